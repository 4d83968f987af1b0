// One generation step's attention over the compressed cache (Sec. 5.1.2: decoding on the
// compressed keys and values).  Per (batch, query head): out = softmax(q . K^T / sqrt(d)) V over
// the `rows` rows of the head's compressed cache.  One query row per head, so this is a
// bandwidth-bound matrix-vector pass: the rows are split over many CTAs (partial maximum, sum and
// unnormalised output each), and a second kernel merges the partials.  Eight lanes share a
// cache row (16-byte vector loads, each lane 1/8 of the head dimension), so a warp works on
// four rows at a time; bf16 products accumulate in fp32, exponentials are exp2 of logits scaled
// by log2(e)/sqrt(d).
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "../../include/snapkv.h"

namespace snapkv {
namespace {

constexpr int DEC_THREADS = 128;
constexpr int DEC_WARPS = DEC_THREADS / 32;
constexpr int DEC_GROUPS = DEC_WARPS * 4;   // row groups (8 lanes each) per CTA
constexpr int DEC_MIN_ROWS = 64;            // a split is not made smaller than this

__device__ __forceinline__ uint4 ld_nc(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}
__device__ __forceinline__ void unpack8(const uint4& x, float* f) {
  const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(w[i] << 16);            // bf16 -> fp32 is a shift
    f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}

// Partial of one split: [0] = running maximum (log2 domain), [1] = sum of exp2, [2 .. 2+D) =
// unnormalised output.
template <int D>
__global__ void __launch_bounds__(DEC_THREADS)
decode_partial_kernel(const uint4* __restrict__ q, const uint4* __restrict__ ck,
                      const uint4* __restrict__ cv, int g, int rows, int rows_per_split, float c2,
                      float* __restrict__ part) {
  constexpr int DPL = D / 8;          // dimensions per lane
  constexpr int VPL = DPL / 8;        // 16-byte vectors per lane and row
  constexpr int VPR = D / 8;          // 16-byte vectors per row
  const int bh = blockIdx.y;
  const int split = blockIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int sub = lane & 7, grp = warp * 4 + (lane >> 3);
  const size_t head = static_cast<size_t>(bh / g) * rows * VPR;
  float qf[DPL];
#pragma unroll
  for (int u = 0; u < VPL; ++u) unpack8(__ldg(q + static_cast<size_t>(bh) * VPR + sub * VPL + u), qf + 8 * u);
  float m = -INFINITY, l = 0.f, acc[DPL];
#pragma unroll
  for (int i = 0; i < DPL; ++i) acc[i] = 0.f;
  const int r0 = split * rows_per_split;
  const int r1 = min(rows, r0 + rows_per_split);
  // The loop is uniform across the warp (its four row groups step together) because the
  // shuffles below are executed by all 32 lanes; a group past the end of the split loads
  // nothing and leaves its state alone.
  for (int rb = r0 + warp * 4; rb < r1; rb += DEC_GROUPS) {
    const int r = rb + (lane >> 3);
    const bool valid = r < r1;
    const size_t off = head + static_cast<size_t>(valid ? r : r0) * VPR + sub * VPL;
    uint4 kx[VPL], vx[VPL];
#pragma unroll
    for (int u = 0; u < VPL; ++u) { kx[u] = ld_nc(ck + off + u); vx[u] = ld_nc(cv + off + u); }
    float s = 0.f;
#pragma unroll
    for (int u = 0; u < VPL; ++u) {
      float kf[8];
      unpack8(kx[u], kf);
#pragma unroll
      for (int i = 0; i < 8; ++i) s = fmaf(qf[8 * u + i], kf[i], s);
    }
    s += __shfl_xor_sync(0xffffffffu, s, 1);
    s += __shfl_xor_sync(0xffffffffu, s, 2);
    s += __shfl_xor_sync(0xffffffffu, s, 4);
    if (valid) {
      s *= c2;
      const float mn = fmaxf(m, s);
      const float corr = exp2f(m - mn);      // 0 on the first row (m = -inf)
      const float p = exp2f(s - mn);
      l = l * corr + p;
#pragma unroll
      for (int u = 0; u < VPL; ++u) {
        float vf[8];
        unpack8(vx[u], vf);
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[8 * u + i] = fmaf(p, vf[i], acc[8 * u + i] * corr);
      }
      m = mn;
    }
  }
  // merge the CTA's row groups in shared memory, in group order
  __shared__ float sm_m[DEC_GROUPS], sm_l[DEC_GROUPS];
  __shared__ float sm_acc[DEC_GROUPS][D];
  if (sub == 0) { sm_m[grp] = m; sm_l[grp] = l; }
#pragma unroll
  for (int i = 0; i < DPL; ++i) sm_acc[grp][sub * DPL + i] = acc[i];
  __syncthreads();
  float M = -INFINITY;
  for (int gi = 0; gi < DEC_GROUPS; ++gi) M = fmaxf(M, sm_m[gi]);
  float* dst = part + (static_cast<size_t>(bh) * gridDim.x + split) * (D + 2);
  for (int t = threadIdx.x; t < D; t += DEC_THREADS) {
    float o = 0.f;
    for (int gi = 0; gi < DEC_GROUPS; ++gi)
      if (sm_m[gi] > -INFINITY) o += sm_acc[gi][t] * exp2f(sm_m[gi] - M);
    dst[2 + t] = o;
  }
  if (threadIdx.x == 0) {
    float L = 0.f;
    for (int gi = 0; gi < DEC_GROUPS; ++gi)
      if (sm_m[gi] > -INFINITY) L += sm_l[gi] * exp2f(sm_m[gi] - M);
    dst[0] = M;
    dst[1] = L;
  }
}

// One CTA of D threads per (batch, query head): folds the splits in split order.
template <int D>
__global__ void __launch_bounds__(D)
decode_merge_kernel(const float* __restrict__ part, int nsplit, float* __restrict__ out,
                    float* __restrict__ out_lse) {
  const int bh = blockIdx.x;
  const float* src = part + static_cast<size_t>(bh) * nsplit * (D + 2);
  float M = -INFINITY;
  for (int s = 0; s < nsplit; ++s) M = fmaxf(M, src[s * (D + 2)]);
  float L = 0.f, o = 0.f;
  for (int s = 0; s < nsplit; ++s) {
    const float ms = src[s * (D + 2)];
    if (ms == -INFINITY) continue;
    const float w = exp2f(ms - M);
    L += src[s * (D + 2) + 1] * w;
    o += src[s * (D + 2) + 2 + threadIdx.x] * w;
  }
  out[static_cast<size_t>(bh) * D + threadIdx.x] = o / L;
  if (out_lse && threadIdx.x == 0) out_lse[bh] = (M + log2f(L)) * 0.6931471805599453f;
}

int decode_nsplit(int heads, int rows) {
  int sms = 148, dev = 0;
  if (cudaGetDevice(&dev) == cudaSuccess) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0) sms = n;
  }
  // about eight CTAs per SM in flight, but no split below DEC_MIN_ROWS rows
  long long want = (8ll * sms + heads - 1) / heads;
  const long long cap = (rows + DEC_MIN_ROWS - 1) / DEC_MIN_ROWS;
  if (want > cap) want = cap;
  if (want < 1) want = 1;
  return static_cast<int>(want);
}

}  // namespace
}  // namespace snapkv

extern "C" size_t snapkv_decode_workspace_size(int B, int Hq, int rows, int d) {
  if (B < 1 || Hq < 1 || rows < 1 || (d != 64 && d != 128)) return 0;
  // the split count depends on the device's SM count; size for the finest split allowed
  const size_t splits = static_cast<size_t>((rows + snapkv::DEC_MIN_ROWS - 1) / snapkv::DEC_MIN_ROWS);
  const size_t heads = static_cast<size_t>(B) * Hq;
  const size_t per_head = (splits < 1184 ? splits : 1184) * (d + 2) * sizeof(float);
  return (heads * per_head + 255) / 256 * 256;
}

extern "C" snapkv_status_t snapkv_decode_attention(const void* q_cur, const void* cache_k,
                                                   const void* cache_v, int B, int Hq, int Hc,
                                                   int rows, int d, float* out, float* out_lse,
                                                   void* workspace, size_t workspace_bytes,
                                                   void* stream) {
  using namespace snapkv;
  if (B < 1 || Hq < 1 || Hc < 1 || rows < 1 || Hq % Hc != 0) return SNAPKV_ERR_INVALID_ARG;
  if (d != 64 && d != 128) return SNAPKV_ERR_UNSUPPORTED;
  if (!q_cur || !cache_k || !cache_v || !out) return SNAPKV_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(q_cur) & 15) || (reinterpret_cast<uintptr_t>(cache_k) & 15) ||
      (reinterpret_cast<uintptr_t>(cache_v) & 15) || (reinterpret_cast<uintptr_t>(out) & 3) ||
      (reinterpret_cast<uintptr_t>(out_lse) & 3))
    return SNAPKV_ERR_INVALID_ARG;
  const long long heads = static_cast<long long>(B) * Hq;
  if (heads > 65535) return SNAPKV_ERR_UNSUPPORTED;
  const int nsplit = decode_nsplit(static_cast<int>(heads), rows);
  const size_t need = static_cast<size_t>(heads) * nsplit * (d + 2) * sizeof(float);
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < need)
    return SNAPKV_ERR_WORKSPACE;
  const int rps = (rows + nsplit - 1) / nsplit;
  const float c2 = static_cast<float>(1.4426950408889634 / sqrt(static_cast<double>(d)));
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  float* part = static_cast<float*>(workspace);
  const dim3 grid(nsplit, static_cast<unsigned>(heads));
  const uint4* q4 = static_cast<const uint4*>(q_cur);
  const uint4* k4 = static_cast<const uint4*>(cache_k);
  const uint4* v4 = static_cast<const uint4*>(cache_v);
  if (d == 128) {
    decode_partial_kernel<128><<<grid, DEC_THREADS, 0, s>>>(q4, k4, v4, Hq / Hc, rows, rps, c2, part);
    decode_merge_kernel<128><<<static_cast<unsigned>(heads), 128, 0, s>>>(part, nsplit, out, out_lse);
  } else {
    decode_partial_kernel<64><<<grid, DEC_THREADS, 0, s>>>(q4, k4, v4, Hq / Hc, rows, rps, c2, part);
    decode_merge_kernel<64><<<static_cast<unsigned>(heads), 64, 0, s>>>(part, nsplit, out, out_lse);
  }
  return cudaGetLastError() == cudaSuccess ? SNAPKV_OK : SNAPKV_ERR_CUDA;
}
