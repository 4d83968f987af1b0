// Pooling and per-head top-k (Listing 1's pool1d and topk; Eq. 2) for rows of a few thousand to
// 131072 positions: one thread-block CLUSTER per row.
//
// A row is cut into C chunks, one CTA of 256 threads each; a thread keeps its EPT consecutive
// pooled keys in registers for the whole kernel.  The CTAs of a row talk through distributed
// shared memory only:
//   1. votes of the chunk (plus the pooling halo) go to shared memory with coalesced loads,
//      each thread pools its own positions and turns them into order-preserving 32-bit keys;
//   2. radix select of the ksel-th largest key, most significant byte first: every CTA
//      histograms its keys that match the prefix found so far (256 bins), the cluster meets at
//      a barrier, every CTA adds up the C histograms (thread t owns bin t, one remote read per
//      peer) and walks the bins from the top - all CTAs get the same digit without a second
//      exchange.  Two histogram buffers alternate, so that a CTA may clear the next one while
//      its peers still read the current one;
//   3. ordered compaction: keys above the threshold, plus the lowest-position keys equal to
//      it until ksel are out; a block scan gives the offset inside the CTA, the CTA totals go
//      round the cluster for the offset of the chunk.
// Ties go to the lower position by construction.  The only waits are cluster barriers (every
// CTA of a cluster is resident by definition and reaches every barrier); a last barrier
// keeps a CTA's shared memory alive until its peers have finished reading it.
//
// Small CTAs with few registers spread a row over up to 16 SMs and fill all of them, where
// one CTA per row leaves SMs idle whenever there are fewer rows than SMs and pays a whole
// row's latency on a single SM.
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "snapkv_internal.h"

namespace snapkv {

namespace {

constexpr int CL_THREADS = 256;
constexpr int CL_WARPS = CL_THREADS / 32;
constexpr int CL_RMAX = 7;          // largest pooling radius this kernel takes
constexpr int CL_MAX_CLUSTER = 16;  // 16 needs the non-portable cluster size
constexpr int CL_BINS = 256;
constexpr int CL_COPIES = 4;        // private histogram copies per CTA (two warps share one)

__device__ __forceinline__ uint32_t float_to_key(float x) {
  const uint32_t b = __float_as_uint(x);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ uint32_t smem_addr(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_size() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
  return r;
}
// All threads of all CTAs of the cluster; orders shared-memory accesses across the cluster.
__device__ __forceinline__ void cluster_barrier() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address of the same shared-memory variable in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t peer_addr(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ int ld_peer(uint32_t addr) {
  int v;
  asm volatile("ld.shared::cluster.s32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ void st_peer(uint32_t addr, int v) {
  asm volatile("st.shared::cluster.s32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}

// slot of position t of the staged chunk: one pad word per 32, so that threads reading
// consecutive runs of EPT positions do not meet in a bank
__device__ __forceinline__ int slot(int t) { return t + (t >> 5); }

// Exclusive prefix sum over the CTA's 256 threads (8 warps); *total_s holds the sum after the
// second barrier inside.
__device__ __forceinline__ uint32_t cta_exclusive_scan(uint32_t x, uint32_t* warp_sums_s, uint32_t* total_s) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t inc = x;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += y;
  }
  if (lane == 31) warp_sums_s[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    const uint32_t w = lane < CL_WARPS ? warp_sums_s[lane] : 0u;
    uint32_t winc = w;
#pragma unroll
    for (int o = 1; o < CL_WARPS; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += y;
    }
    if (lane < CL_WARPS) warp_sums_s[lane] = winc - w;
    if (lane == CL_WARPS - 1) *total_s = winc;
  }
  __syncthreads();
  return warp_sums_s[warp] + inc - x;
}

// R, PT >= 0: the pooling radius is exactly R and the type PT (0 max, 1 avg), no per-tap tests.
// PT = -1: radius r <= R and pool_type are run-time values.
template <int EPT, int R, int PT>
__global__ void __launch_bounds__(CL_THREADS)
pool_topk_cluster_kernel(const float* __restrict__ vote, int n, int gsum, int r, int pool_type,
                         int ksel, int32_t* __restrict__ out_idx) {
  constexpr int CHUNK = CL_THREADS * EPT;
  constexpr int STAGED = CHUNK + 2 * CL_RMAX;
  __shared__ float raw[STAGED + STAGED / 32 + 1];
  __shared__ int hist[2][CL_BINS];        // the CTA's histogram of a round, read by the peers
  __shared__ int hist_w[CL_COPIES][CL_BINS];  // private histograms, one per pair of warps
  __shared__ int totals[CL_MAX_CLUSTER][2];  // per CTA of the cluster: keys above / equal to the threshold
  __shared__ uint32_t warp_sums[CL_WARPS];
  __shared__ uint32_t scan_total;
  __shared__ int sel_bin, sel_above;

  const uint32_t C = cluster_size(), rank = cluster_rank();
  const int row = blockIdx.x / C;
  const int c0 = static_cast<int>(rank) * CHUNK;  // first position of this CTA's chunk
  const float* vrow = vote + static_cast<size_t>(row) * gsum * n;

  // ---- 1. stage the chunk and its halo: position c0 - CL_RMAX + t at slot(t); zero outside the row.
  // All of a thread's loads are issued before the first value is stored: the votes come from
  // L2, and a loop of load-then-store would pay that latency once per element.
  {
    float x[EPT];
#pragma unroll
    for (int i = 0; i < EPT; ++i) {
      const int j = c0 + static_cast<int>(threadIdx.x) + CL_THREADS * i;
      x[i] = (j < n) ? __ldg(vrow + j) : 0.f;
    }
    for (int g = 1; g < gsum; ++g) {  // ascending head order
      const float* src = vrow + static_cast<size_t>(g) * n;
#pragma unroll
      for (int i = 0; i < EPT; ++i) {
        const int j = c0 + static_cast<int>(threadIdx.x) + CL_THREADS * i;
        if (j < n) x[i] += __ldg(src + j);
      }
    }
#pragma unroll
    for (int i = 0; i < EPT; ++i) raw[slot(CL_RMAX + static_cast<int>(threadIdx.x) + CL_THREADS * i)] = x[i];
    if (threadIdx.x < 2 * CL_RMAX) {  // the halo: CL_RMAX positions before the chunk, CL_RMAX after
      const int t = threadIdx.x < CL_RMAX ? static_cast<int>(threadIdx.x)
                                          : CHUNK + static_cast<int>(threadIdx.x);
      const int j = c0 - CL_RMAX + t;
      float h = 0.f;
      if (j >= 0 && j < n) {
        h = __ldg(vrow + j);
        for (int g = 1; g < gsum; ++g) h += __ldg(vrow + static_cast<size_t>(g) * n + j);
      }
      raw[slot(t)] = h;
    }
  }
  __syncthreads();

  // ---- pooling: thread owns positions c0 + base .. c0 + base + EPT - 1
  const int base = threadIdx.x * EPT;
  uint32_t key[EPT];
  {
    float a[EPT + 2 * R];
#pragma unroll
    for (int i = 0; i < EPT + 2 * R; ++i) a[i] = raw[slot(base + (CL_RMAX - R) + i)];
#pragma unroll
    for (int i = 0; i < EPT; ++i) {
      float p = 0.f;  // votes are >= 0: zero is neutral for max and is the avg padding
#pragma unroll
      for (int t = 0; t <= 2 * R; ++t) {
        const int off = t - R;
        if (PT >= 0 || (off >= -r && off <= r))
          p = ((PT >= 0) ? (PT == 0) : (pool_type == 0)) ? fmaxf(p, a[i + t]) : p + a[i + t];
      }
      // average pooling ranks by the window sum: dividing by the kernel size is monotone.
      // Positions past the row's end rank below every real key (votes >= 0 set the top bit).
      key[i] = (c0 + base + i < n) ? float_to_key(p) : 0u;
    }
  }

  // ---- 2. radix select, one byte per round from the top
  // Pairs of warps count into a histogram of their own (pooled neighbours mostly share a bin,
  // and in the first rounds so do most keys of the row: one shared histogram would serialise
  // the whole CTA on a few words); thread t then adds the copies of bin t, publishes the sum
  // in the CTA's histogram of this round and clears the copies for the next round.
  uint32_t prefix = 0u, mask = 0u;
  int krem = ksel;
  const uint32_t hist_base = smem_addr(&hist[0][0]);
  const int warp = threadIdx.x >> 5;
#pragma unroll
  for (int w = 0; w < CL_COPIES; ++w) hist_w[w][threadIdx.x] = 0;  // CL_BINS == CL_THREADS
  __syncthreads();
#pragma unroll 1
  for (int round = 0; round < 4; ++round) {
    const int shift = 24 - 8 * round;
    {
      int* h = hist_w[warp % CL_COPIES];
      int cur = -1, cnt = 0;  // count runs of equal bins
#pragma unroll
      for (int i = 0; i < EPT; ++i) {
        if ((key[i] & mask) == prefix) {
          const int b = static_cast<int>((key[i] >> shift) & 255u);
          if (b != cur) {
            if (cnt) atomicAdd(&h[cur], cnt);
            cur = b;
            cnt = 0;
          }
          ++cnt;
        }
      }
      if (cnt) atomicAdd(&h[cur], cnt);
    }
    __syncthreads();
    {
      int sum = 0;
#pragma unroll
      for (int w = 0; w < CL_COPIES; ++w) {
        sum += hist_w[w][threadIdx.x];
        hist_w[w][threadIdx.x] = 0;
      }
      hist[round & 1][threadIdx.x] = sum;
    }
    cluster_barrier();  // every CTA's histogram of this round is complete
    int cnt_bin = 0;    // thread t owns bin 255 - t: the scan below then runs from the top bin down
    {
      const uint32_t my = hist_base + static_cast<uint32_t>(((round & 1) * CL_BINS + (255 - static_cast<int>(threadIdx.x))) * 4);
      // all remote reads are issued before the first one is used
      int part[CL_MAX_CLUSTER];
#pragma unroll
      for (uint32_t p = 0; p < CL_MAX_CLUSTER; ++p) part[p] = p < C ? ld_peer(peer_addr(my, p)) : 0;
#pragma unroll
      for (uint32_t p = 0; p < CL_MAX_CLUSTER; ++p) cnt_bin += part[p];
    }
    const int above = static_cast<int>(cta_exclusive_scan(static_cast<uint32_t>(cnt_bin), warp_sums, &scan_total));
    if (cnt_bin > 0 && above < krem && krem <= above + cnt_bin) {
      sel_bin = 255 - static_cast<int>(threadIdx.x);
      sel_above = above;
    }
    __syncthreads();
    prefix |= static_cast<uint32_t>(sel_bin) << shift;
    mask |= 255u << shift;
    krem -= sel_above;
    // (sel_bin and the warps' histograms are written again only behind the next barriers; a
    // peer reads hist[round & 1] until it arrives at the next cluster barrier, and this CTA
    // writes that buffer again two rounds on)
  }
  const uint32_t T = prefix;  // key of the ksel-th largest pooled vote of the row
  const int need_eq = krem;   // how many positions equal to it are kept (the lowest ones)

  // ---- 3. ordered compaction
  uint32_t m_gt = 0u, m_eq = 0u;  // EPT <= 32
#pragma unroll
  for (int i = 0; i < EPT; ++i) {
    m_gt |= static_cast<uint32_t>(key[i] > T) << i;
    m_eq |= static_cast<uint32_t>(key[i] == T) << i;
  }
  // two counts of at most CHUNK <= 8192 each in one unsigned word: no carry between the halves
  static_assert(CHUNK < 65536, "two 16-bit counts share one scan word");
  const uint32_t packed = cta_exclusive_scan((static_cast<uint32_t>(__popc(m_gt)) << 16) | __popc(m_eq),
                                             warp_sums, &scan_total);
  if (threadIdx.x == 0) {
    const uint32_t mine = smem_addr(&totals[rank][0]);
    for (uint32_t p = 0; p < C; ++p) {
      st_peer(peer_addr(mine, p), static_cast<int>(scan_total >> 16));
      st_peer(peer_addr(mine + 4, p), static_cast<int>(scan_total & 0xffffu));
    }
  }
  cluster_barrier();  // every CTA has every CTA's totals
  int gt_before = 0, eq_before = 0;
  for (uint32_t p = 0; p < rank; ++p) {
    gt_before += totals[p][0];
    eq_before += totals[p][1];
  }
  int eq_seen = eq_before + static_cast<int>(packed & 0xffffu);
  int out_pos = gt_before + static_cast<int>(packed >> 16) + min(eq_seen, need_eq);
  int32_t* orow = out_idx + static_cast<size_t>(row) * ksel;
  uint32_t rest = m_gt | m_eq;
  while (rest) {
    const int bit = __ffs(rest) - 1;
    rest &= rest - 1;
    const bool is_eq = (m_eq >> bit) & 1u;
    if (!is_eq || eq_seen++ < need_eq) orow[out_pos++] = c0 + base + bit;
  }
  // nobody leaves while a peer may still read its histograms
  cluster_barrier();
}

struct ClusterShape {
  int ept, clusters;  // keys per thread, CTAs per row
};

// How a row of n positions is cut: as many CTAs as the portable cluster size allows, the
// smallest per-thread run that covers the row; rows beyond 8 x 8192 take 16 CTAs.
bool cluster_shape(int n, ClusterShape* s) {
  if (n < 4096 || n > CL_MAX_CLUSTER * CL_THREADS * 32) return false;
  if (n > 8 * CL_THREADS * 32) {
    s->ept = 32;
    s->clusters = 16;
    return true;
  }
  const int per = (n + 7) / 8;
  s->ept = per <= CL_THREADS * 8 ? 8 : (per <= CL_THREADS * 16 ? 16 : 32);
  s->clusters = (n + CL_THREADS * s->ept - 1) / (CL_THREADS * s->ept);
  return true;
}

template <int EPT, int R, int PT>
cudaError_t launch_one(const float* vote, int rows, int n, int gsum, int r, int pool_type, int ksel,
                       int32_t* out_idx, int clusters, cudaStream_t stream) {
  auto kernel = pool_topk_cluster_kernel<EPT, R, PT>;
  if (clusters > 8) {
    static DeviceOnce once;
    if (!once.done()) {
      cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
      if (e != cudaSuccess) return e;
      once.set();
    }
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(rows) * clusters);
  cfg.blockDim = dim3(CL_THREADS);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = clusters;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, vote, n, gsum, r, pool_type, ksel, out_idx);
}

template <int EPT>
cudaError_t launch_ept(const float* vote, int rows, int n, int gsum, int r, int pool_type, int ksel,
                       int32_t* out_idx, int clusters, cudaStream_t stream) {
  const bool mx = pool_type == 0;
#define SNAPKV_CL(RR, PP) launch_one<EPT, RR, PP>(vote, rows, n, gsum, r, pool_type, ksel, out_idx, clusters, stream)
  // the paper's kernel sizes 5, 7 and 13 have instantiations of their own
  if (r == 2) return mx ? SNAPKV_CL(2, 0) : SNAPKV_CL(2, 1);
  if (r == 3) return mx ? SNAPKV_CL(3, 0) : SNAPKV_CL(3, 1);
  if (r == 6) return mx ? SNAPKV_CL(6, 0) : SNAPKV_CL(6, 1);
  return SNAPKV_CL(CL_RMAX, -1);
#undef SNAPKV_CL
}

}  // namespace

// Whether this device can hold a cluster of 16 of these CTAs (asked once per device).
static bool cluster16_ok() {
  constexpr int MAX_DEV = 64;
  static std::atomic<int> state[MAX_DEV] = {};  // 0 unknown, 1 yes, 2 no
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEV) return false;
  int st = state[dev].load(std::memory_order_acquire);
  if (st == 0) {
    auto kernel = pool_topk_cluster_kernel<32, CL_RMAX, -1>;
    int n_clusters = 0;
    bool ok = cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess;
    if (ok) {
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(16);
      cfg.blockDim = dim3(CL_THREADS);
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = 16;
      attr[0].val.clusterDim.y = 1;
      attr[0].val.clusterDim.z = 1;
      cfg.attrs = attr;
      cfg.numAttrs = 1;
      ok = cudaOccupancyMaxActiveClusters(&n_clusters, kernel, &cfg) == cudaSuccess && n_clusters >= 1;
    }
    if (!ok) (void)cudaGetLastError();  // a refusal here is an answer, not an error of the call
    st = ok ? 1 : 2;
    state[dev].store(st, std::memory_order_release);
  }
  return st == 1;
}

bool select_cluster_applies(int rows, int n, int pool_kernel) {
  ClusterShape s;
  if ((pool_kernel >> 1) > CL_RMAX || !cluster_shape(n, &s)) return false;
  if (s.clusters > 8 && !cluster16_ok()) return false;
  // the grid is rows x CTAs per row in one dimension
  return static_cast<long long>(rows) * s.clusters < 2147483647ll;
}

cudaError_t launch_pool_topk_cluster(const float* vote, int rows, int n, int pool_kernel,
                                     int pool_type, int ksel, int32_t* out_idx, cudaStream_t stream,
                                     int* launches, int gsum) {
  ClusterShape s;
  if (!cluster_shape(n, &s)) return cudaErrorInvalidValue;
  const int r = pool_kernel >> 1;
  cudaError_t e;
  if (s.ept == 8) e = launch_ept<8>(vote, rows, n, gsum, r, pool_type, ksel, out_idx, s.clusters, stream);
  else if (s.ept == 16) e = launch_ept<16>(vote, rows, n, gsum, r, pool_type, ksel, out_idx, s.clusters, stream);
  else e = launch_ept<32>(vote, rows, n, gsum, r, pool_type, ksel, out_idx, s.clusters, stream);
  if (e != cudaSuccess) return e;
  *launches += 1;
  return cudaGetLastError();
}

}  // namespace snapkv
