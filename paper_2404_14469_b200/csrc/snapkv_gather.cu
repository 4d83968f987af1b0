// Gather + append (Listing 1's gather and cat): per query head, copy the selected
// prefix rows of K and V in the order of `idx`, then the W window rows, into a dense
// [rows, d] block.  Pure byte movement in 16-byte vectors; a row of d = 128 bf16 is
// 16 vectors, so half a warp reads one source row contiguously and writes one
// destination row contiguously.
#include <cuda_runtime.h>
#include <stdint.h>

#include "snapkv_internal.h"

namespace snapkv {

namespace {

constexpr int GATHER_THREADS = 256;
constexpr int GATHER_UNROLL = 4;

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}
__device__ __forceinline__ void st_stream(uint4* p, const uint4& v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(v.x), "r"(v.y),
               "r"(v.z), "r"(v.w)
               : "memory");
}

// VPR = 16-byte vectors per row.  One thread moves one vector of K and of V for
// GATHER_UNROLL different rows, all loads issued before the first store.
template <int VPR>
__global__ void __launch_bounds__(GATHER_THREADS)
gather_kernel(const uint4* __restrict__ k, const uint4* __restrict__ v,
              const int32_t* __restrict__ idx, int g, int L, int W, int ksel, int out_stride,
              long long total_rows, uint4* __restrict__ out_k, uint4* __restrict__ out_v) {
  const int rows = ksel + W;
  const int n = L - W;
  const long long vec0 = (static_cast<long long>(blockIdx.x) * GATHER_THREADS * GATHER_UNROLL) +
                         threadIdx.x;
  size_t src[GATHER_UNROLL], dst[GATHER_UNROLL];
  bool ok[GATHER_UNROLL];
#pragma unroll
  for (int uu = 0; uu < GATHER_UNROLL; ++uu) {
    const long long gid = vec0 + static_cast<long long>(uu) * GATHER_THREADS;
    const long long grow = gid / VPR;
    const int vec = static_cast<int>(gid - grow * VPR);
    ok[uu] = grow < total_rows;
    src[uu] = dst[uu] = 0;
    if (ok[uu]) {
      const long long bh = grow / rows;
      const int t = static_cast<int>(grow - bh * rows);
      int pos;
      if (t < ksel) pos = idx ? __ldg(idx + bh * ksel + t) : t;
      else pos = n + (t - ksel);
      const long long ukv = bh / g;
      src[uu] = static_cast<size_t>((ukv * L + pos) * VPR + vec);
      dst[uu] = static_cast<size_t>((bh * out_stride + t) * VPR + vec);
    }
  }
  uint4 kk[GATHER_UNROLL], vv[GATHER_UNROLL];
#pragma unroll
  for (int uu = 0; uu < GATHER_UNROLL; ++uu)
    if (ok[uu]) {
      kk[uu] = ld_stream(k + src[uu]);
      vv[uu] = ld_stream(v + src[uu]);
    }
#pragma unroll
  for (int uu = 0; uu < GATHER_UNROLL; ++uu)
    if (ok[uu]) {
      st_stream(out_k + dst[uu], kk[uu]);
      st_stream(out_v + dst[uu], vv[uu]);
    }
}

}  // namespace

cudaError_t launch_gather(const void* k, const void* v, const int32_t* idx, int B, int Hq, int Hkv,
                          int L, int d, int W, int ksel, int out_rows_stride, void* out_k,
                          void* out_v, cudaStream_t stream, int* launches) {
  const int rows = ksel + W;
  const long long total_rows = static_cast<long long>(B) * Hq * rows;
  const int vpr = d * 2 / 16;
  const long long total_vec = total_rows * vpr;
  const long long per_block = static_cast<long long>(GATHER_THREADS) * GATHER_UNROLL;
  const long long blocks = (total_vec + per_block - 1) / per_block;
  if (blocks <= 0) return cudaSuccess;
  if (blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
  const int g = Hq / Hkv;
  const uint4* kp = static_cast<const uint4*>(k);
  const uint4* vp = static_cast<const uint4*>(v);
  uint4* okp = static_cast<uint4*>(out_k);
  uint4* ovp = static_cast<uint4*>(out_v);
  if (vpr == 16)
    gather_kernel<16><<<static_cast<unsigned>(blocks), GATHER_THREADS, 0, stream>>>(
        kp, vp, idx, g, L, W, ksel, out_rows_stride, total_rows, okp, ovp);
  else
    gather_kernel<8><<<static_cast<unsigned>(blocks), GATHER_THREADS, 0, stream>>>(
        kp, vp, idx, g, L, W, ksel, out_rows_stride, total_rows, okp, ovp);
  *launches += 1;
  return cudaGetLastError();
}

}  // namespace snapkv
