// Gather + append (Listing 1's gather and cat): per query head, copy the selected
// prefix rows of K and V in the order of `idx`, then the W window rows, into a dense
// [rows, d] block.  Pure byte movement in 16-byte vectors; a row of d = 128 bf16 is
// 16 vectors, so half a warp reads one source row contiguously and writes one
// destination row contiguously.
#include <cuda_runtime.h>
#include <stdint.h>

#include "launch.cuh"
#include "snapkv_internal.h"

namespace snapkv {

namespace {

constexpr int GATHER_THREADS = 256;
// Two rows in flight per thread and eight blocks per SM (32 registers): the copy is bound by
// memory latency, and 2048 resident threads with four loads each beat 1024 with eight (68 vs
// 85 us for 128 heads x 4096 rows on a cold L2).
constexpr int GATHER_UNROLL = 2;
constexpr int GATHER_MIN_BLOCKS = 8;

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

// Strides of K and of V in 16-byte vectors (batch or page, KV head, position).
struct GatherStrides {
  long long kb, kh, kl, vb, vh, vl;
};

// Block table of a paged cache (table == nullptr: dense addressing).
struct GatherPages {
  const int32_t* table;
  int pages_per_seq, page_size, num_pages;
};

// VPR = 16-byte vectors per row.  blockIdx.y (+ h0) is the (batch, query head) pair, blockIdx.x
// a block of RPB consecutive output rows of that head; one thread moves one vector of K and
// of V for GATHER_UNROLL rows, all loads issued before the first store.
template <int VPR, bool PAGED>
__global__ void __launch_bounds__(GATHER_THREADS, GATHER_MIN_BLOCKS)
gather_kernel(const uint4* __restrict__ k, const uint4* __restrict__ v, const GatherStrides st,
              const GatherPages pg, const int32_t* __restrict__ idx, int h0, int g, int Hkv, int L,
              int W, int ksel, int out_stride, uint4* __restrict__ out_k, uint4* __restrict__ out_v) {
  constexpr int RPT = GATHER_THREADS / VPR;      // rows covered by the block per unrolled step
  constexpr int RPB = RPT * GATHER_UNROLL;       // rows per block
  pdl_wait();  // launched early behind the select kernel: idx is complete only from here on
  const int rows = ksel + W;
  const int n = L - W;
  const int bh = h0 + blockIdx.y;
  const int vec = threadIdx.x % VPR;
  const int t0 = blockIdx.x * RPB + threadIdx.x / VPR;
  const int kvh = bh / g;
  const int b = kvh / Hkv, c = kvh - b * Hkv;
  // dense: the head's first row; paged: the head's first row inside page 0 of the pool
  const uint4* k_head = k + ((PAGED ? 0 : b * st.kb) + c * st.kh + vec);
  const uint4* v_head = v + ((PAGED ? 0 : b * st.vb) + c * st.vh + vec);
  const int32_t* pages = PAGED ? pg.table + static_cast<size_t>(b) * pg.pages_per_seq : nullptr;
  const size_t dst_head = static_cast<size_t>(bh) * out_stride * VPR + vec;
  const int32_t* idx_head = idx ? idx + static_cast<size_t>(bh) * ksel : nullptr;
  int pos[GATHER_UNROLL];
  bool ok[GATHER_UNROLL];
#pragma unroll
  for (int uu = 0; uu < GATHER_UNROLL; ++uu) {
    const int t = t0 + uu * RPT;
    ok[uu] = t < rows;
    pos[uu] = 0;
    if (ok[uu]) pos[uu] = (t < ksel) ? (idx_head ? __ldg(idx_head + t) : t) : n + (t - ksel);
  }
  uint4 kk[GATHER_UNROLL], vv[GATHER_UNROLL];
#pragma unroll
  for (int uu = 0; uu < GATHER_UNROLL; ++uu)
    if (ok[uu]) {
      if (PAGED) {
        const int slot = pos[uu] / pg.page_size;
        const int row = pos[uu] - slot * pg.page_size;
        const int page = __ldg(pages + slot);
        if (static_cast<unsigned>(page) < static_cast<unsigned>(pg.num_pages)) {
          kk[uu] = ld_stream(k_head + page * st.kb + row * st.kl);
          vv[uu] = ld_stream(v_head + page * st.vb + row * st.vl);
        } else {  // an entry that names no page of the pool: zeros, as the scoring pass reads it
          kk[uu] = make_uint4(0u, 0u, 0u, 0u);
          vv[uu] = make_uint4(0u, 0u, 0u, 0u);
        }
      } else {
        kk[uu] = ld_stream(k_head + pos[uu] * st.kl);
        vv[uu] = ld_stream(v_head + pos[uu] * st.vl);
      }
    }
#pragma unroll
  for (int uu = 0; uu < GATHER_UNROLL; ++uu)
    if (ok[uu]) {
      const size_t dst = dst_head + static_cast<size_t>(t0 + uu * RPT) * VPR;
      st_stream(out_k + dst, kk[uu]);
      st_stream(out_v + dst, vv[uu]);
    }
}

// A shard of a longer prompt holds positions [pos0, pos0 + L).  Of a head's ascending list of
// selected positions, the entries inside that range form one contiguous segment.
// seg_kernel finds it, one thread per head (two binary searches): seg[head] = {first entry of
// the segment, entries in it}.  gather_range_kernel then copies those rows and `append`
// trailing rows of the shard (the window rows, on the shard that holds them) into rows
// [0, count + append) of the head's output.
__global__ void seg_kernel(const int32_t* __restrict__ idx, int heads, int ksel, int pos0, int L,
                           int32_t* __restrict__ seg) {
  const int bh = blockIdx.x * blockDim.x + threadIdx.x;
  if (bh >= heads) return;
  const int32_t* idx_head = idx + static_cast<size_t>(bh) * ksel;
  auto lower_bound = [&](int value) {  // first entry >= value
    int lo = 0, hi = ksel;
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (__ldg(idx_head + mid) < value) lo = mid + 1; else hi = mid;
    }
    return lo;
  };
  const int lo = lower_bound(pos0);
  seg[2 * bh] = lo;
  seg[2 * bh + 1] = lower_bound(pos0 + L) - lo;
}

template <int VPR>
__global__ void __launch_bounds__(GATHER_THREADS, GATHER_MIN_BLOCKS)
gather_range_kernel(const uint4* __restrict__ k, const uint4* __restrict__ v, const GatherStrides st,
                    const int32_t* __restrict__ idx, int g, int Hkv, int L, int pos0, int ksel, int append,
                    int out_stride, uint4* __restrict__ out_k, uint4* __restrict__ out_v,
                    const int32_t* __restrict__ seg) {
  constexpr int RPT = GATHER_THREADS / VPR;
  constexpr int RPB = RPT * GATHER_UNROLL;
  __shared__ int s_lo, s_cnt;
  const int bh = blockIdx.y;
  const int32_t* idx_head = idx + static_cast<size_t>(bh) * ksel;
  if (threadIdx.x == 0) {
    s_lo = __ldg(seg + 2 * bh);
    s_cnt = __ldg(seg + 2 * bh + 1);
  }
  __syncthreads();
  const int lo = s_lo, cnt = s_cnt;
  const int rows = cnt + append;
  if (static_cast<int>(blockIdx.x) * RPB >= rows) return;
  const int vec = threadIdx.x % VPR;
  const int t0 = blockIdx.x * RPB + threadIdx.x / VPR;
  const int kvh = bh / g;
  const int b = kvh / Hkv, c = kvh - b * Hkv;
  const uint4* k_head = k + (b * st.kb + c * st.kh + vec);
  const uint4* v_head = v + (b * st.vb + c * st.vh + vec);
  const size_t dst_head = static_cast<size_t>(bh) * out_stride * VPR + vec;
#pragma unroll
  for (int uu = 0; uu < GATHER_UNROLL; ++uu) {
    const int t = t0 + uu * RPT;
    if (t < rows) {
      const int pos = t < cnt ? __ldg(idx_head + lo + t) - pos0 : L - append + (t - cnt);
      const uint4 kk = ld_stream(k_head + pos * st.kl);
      const uint4 vv = ld_stream(v_head + pos * st.vl);
      const size_t dst = dst_head + static_cast<size_t>(t) * VPR;
      st_stream(out_k + dst, kk);
      st_stream(out_v + dst, vv);
    }
  }
}

}  // namespace

cudaError_t launch_gather_range(const void* k, const void* v, const KVStrides& ks, const KVStrides& vs,
                                const int32_t* idx, int B, int Hq, int Hkv, int L, int d, int pos0,
                                int ksel, int append, int out_rows_stride, void* out_k, void* out_v,
                                int32_t* seg, cudaStream_t stream, int* launches) {
  const int vpr = d * 2 / 16;
  const int rpb = GATHER_THREADS / vpr * GATHER_UNROLL;
  const long long heads = static_cast<long long>(B) * Hq;
  if (heads <= 0 || heads > 65535) return cudaErrorInvalidValue;
  const int max_rows = (ksel < L ? ksel : L) + append;
  const GatherStrides st = {ks.b / 8, ks.h / 8, ks.l / 8, vs.b / 8, vs.h / 8, vs.l / 8};
  const dim3 grid(static_cast<unsigned>((max_rows + rpb - 1) / rpb > 0 ? (max_rows + rpb - 1) / rpb : 1),
                  static_cast<unsigned>(heads));
  seg_kernel<<<static_cast<unsigned>((heads + 127) / 128), 128, 0, stream>>>(idx, static_cast<int>(heads), ksel,
                                                                             pos0, L, seg);
  *launches += 1;
  const uint4* kp = static_cast<const uint4*>(k);
  const uint4* vp = static_cast<const uint4*>(v);
  if (vpr == 16)
    gather_range_kernel<16><<<grid, GATHER_THREADS, 0, stream>>>(
        kp, vp, st, idx, Hq / Hkv, Hkv, L, pos0, ksel, append, out_rows_stride,
        static_cast<uint4*>(out_k), static_cast<uint4*>(out_v), seg);
  else
    gather_range_kernel<8><<<grid, GATHER_THREADS, 0, stream>>>(
        kp, vp, st, idx, Hq / Hkv, Hkv, L, pos0, ksel, append, out_rows_stride,
        static_cast<uint4*>(out_k), static_cast<uint4*>(out_v), seg);
  *launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_gather(const void* k, const void* v, const KVStrides& ks, const KVStrides& vs,
                          const int32_t* idx, int B, int Hq, int Hkv, int L, int d, int W, int ksel,
                          int out_rows_stride, void* out_k, void* out_v, cudaStream_t stream,
                          int* launches, const PagedKV* paged) {
  const int rows = ksel + W;
  const int vpr = d * 2 / 16;
  const int rpb = GATHER_THREADS / vpr * GATHER_UNROLL;
  const long long heads = static_cast<long long>(B) * Hq;
  if (rows <= 0 || heads <= 0) return cudaSuccess;
  const int g = Hq / Hkv;
  const uint4* kp = static_cast<const uint4*>(k);
  const uint4* vp = static_cast<const uint4*>(v);
  uint4* okp = static_cast<uint4*>(out_k);
  uint4* ovp = static_cast<uint4*>(out_v);
  // strides are multiples of 8 elements (the callers check): whole 16-byte vectors
  const GatherStrides st = {ks.b / 8, ks.h / 8, ks.l / 8, vs.b / 8, vs.h / 8, vs.l / 8};
  const unsigned gx = static_cast<unsigned>((rows + rpb - 1) / rpb);
  // blockIdx.y is limited to 65535: go through the heads in slabs if there are more
  const long long slab = 65535;
  cudaError_t e = cudaSuccess;
  for (long long h0 = 0; h0 < heads && e == cudaSuccess; h0 += slab) {
    const unsigned gy = static_cast<unsigned>(heads - h0 < slab ? heads - h0 : slab);
    const int h0i = static_cast<int>(h0);
    const dim3 grid(gx, gy);
    if (paged) {
      const GatherPages pg = {paged->table, paged->pages_per_seq, paged->page_size, paged->num_pages};
      if (vpr == 16)
        e = launch_pdl(gather_kernel<16, true>, grid, dim3(GATHER_THREADS), 0, stream, kp, vp, st, pg,
                       idx, h0i, g, Hkv, L, W, ksel, out_rows_stride, okp, ovp);
      else
        e = launch_pdl(gather_kernel<8, true>, grid, dim3(GATHER_THREADS), 0, stream, kp, vp, st, pg,
                       idx, h0i, g, Hkv, L, W, ksel, out_rows_stride, okp, ovp);
    } else {
      const GatherPages pg = {nullptr, 0, 1, 0};
      if (vpr == 16)
        e = launch_pdl(gather_kernel<16, false>, grid, dim3(GATHER_THREADS), 0, stream, kp, vp, st, pg,
                       idx, h0i, g, Hkv, L, W, ksel, out_rows_stride, okp, ovp);
      else
        e = launch_pdl(gather_kernel<8, false>, grid, dim3(GATHER_THREADS), 0, stream, kp, vp, st, pg,
                       idx, h0i, g, Hkv, L, W, ksel, out_rows_stride, okp, ovp);
    }
    *launches += 1;
  }
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace snapkv
