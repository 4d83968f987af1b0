// Pooling and per-head top-k (Listing 1's pool1d and topk; Eq. 2), one CTA per row.
//
// Two kernels: a fast one for rows that fit in shared memory (below) and this generic
// one, which also handles rows of any length through global scratch.
//
//  1. pooled[j] = max or mean of vote[j-r .. j+r] (stride 1, same length; the mean
//     divides by pool_kernel, positions outside the row count as zero), turned into a
//     32-bit key whose unsigned order is the float order.  Keys stay in shared memory
//     when the row fits, otherwise in caller-provided global scratch.
//  2. radix select of the ksel-th largest key: three histogram passes (11 + 11 + 10
//     bits), each followed by a block scan from the top bin down.
//  3. ordered compaction: every key above the threshold, plus the lowest-position keys
//     equal to it until ksel are taken, written in ascending position.
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/snapkv.h"
#include "launch.cuh"
#include "snapkv_internal.h"

namespace snapkv {

namespace {

// Tells L2 that a 128-byte line (global memory, 128-byte aligned) holds nothing worth keeping:
// a dirty line may then be dropped instead of written back.  Its contents are undefined afterwards.
__device__ __forceinline__ void discard_l2_line(const void* p) {
  asm volatile("discard.global.L2 [%0], 128;" ::"l"(__cvta_generic_to_global(p)) : "memory");
}

constexpr int SEL_THREADS = 1024;
constexpr int SEL_WARPS = SEL_THREADS / 32;
constexpr int SEL_SMEM_KEYS = 49152;  // rows up to this length keep their keys on chip
constexpr int NBINS = 2048;

__device__ __forceinline__ uint32_t float_to_key(float x) {
  const uint32_t b = __float_as_uint(x);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// Exclusive prefix sum of one value per thread over the block (SEL_WARPS warps); returns the
// prefix and leaves the block total in *total_s after the second barrier.  T is int, or
// uint32_t when two 16-bit counts travel in one word: unsigned sums wrap, they never overflow.
template <typename T>
__device__ __forceinline__ T block_exclusive_scan(T x, T* warp_sums_s, T* total_s) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  T inc = x;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const T y = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += y;
  }
  if (lane == 31) warp_sums_s[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    T w = warp_sums_s[lane];
    T winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const T y = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += y;
    }
    warp_sums_s[lane] = winc - w;  // exclusive
    if (lane == 31) *total_s = winc;
  }
  __syncthreads();
  return warp_sums_s[warp] + inc - x;
}

// Vote of position j of a selection row.  With shared selection under grouped-query
// attention `gsum` consecutive per-head rows of n votes select together: their sum, taken in
// ascending head order (gsum = 1: the row itself).  `vrow` is the first of those rows.
__device__ __forceinline__ float ld_vote(const float* __restrict__ vrow, int j, int n, int gsum) {
  float x = __ldg(vrow + j);
  for (int t = 1; t < gsum; ++t) x += __ldg(vrow + static_cast<size_t>(t) * n + j);
  return x;
}

__global__ void __launch_bounds__(SEL_THREADS, 1)
pool_topk_kernel(const float* __restrict__ vote, int n, int gsum, int pool_kernel, int pool_type,
                 int ksel, int32_t* __restrict__ out_idx, uint32_t* __restrict__ key_scratch) {
  extern __shared__ uint32_t keys_smem[];
  __shared__ int hist[NBINS];
  __shared__ int warp_sums[SEL_WARPS];
  __shared__ int scan_total;
  __shared__ int sel_bin, sel_above;
  __shared__ int wgt[SEL_WARPS], weq[SEL_WARPS];

  const int row = blockIdx.x;
  const float* vrow = vote + static_cast<size_t>(row) * gsum * n;
  uint32_t* keys = key_scratch ? key_scratch + static_cast<size_t>(row) * n : keys_smem;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int r = pool_kernel >> 1;

  // ---- 1. pooling
  for (int j = threadIdx.x; j < n; j += SEL_THREADS) {
    const int lo = max(0, j - r), hi = min(n - 1, j + r);
    float p;
    if (pool_type == 0) {
      p = ld_vote(vrow, lo, n, gsum);
      for (int t = lo + 1; t <= hi; ++t) p = fmaxf(p, ld_vote(vrow, t, n, gsum));
    } else {
      p = 0.f;
      for (int t = lo; t <= hi; ++t) p += ld_vote(vrow, t, n, gsum);
      p = p / static_cast<float>(pool_kernel);
    }
    keys[j] = float_to_key(p);
  }
  __syncthreads();

  // ---- 2. radix select of the ksel-th largest key
  uint32_t prefix = 0, mask = 0;
  int krem = ksel;
  const int n_round = (n + 31) & ~31;
#pragma unroll 1
  for (int pass = 0; pass < 3; ++pass) {
    const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
    const int nb = pass == 2 ? 1024 : 2048;
    const uint32_t dmask = nb - 1;
    for (int b = threadIdx.x; b < NBINS; b += SEL_THREADS) hist[b] = 0;
    __syncthreads();
    for (int base = warp * 32; base < n_round; base += SEL_THREADS) {
      const int j = base + lane;
      uint32_t key = 0;
      bool live = false;
      if (j < n) {
        key = keys[j];
        live = (key & mask) == prefix;
      }
      // lanes that do not take part get a value no other lane has
      const uint32_t dg = live ? ((key >> shift) & dmask) : (0x80000000u | lane);
      const uint32_t peers = __match_any_sync(0xffffffffu, dg);
      if (live && lane == __ffs(peers) - 1) atomicAdd(&hist[dg], __popc(peers));
    }
    __syncthreads();
    // walk the bins from the top: thread t owns bins nb-1-2t and nb-2-2t
    int c0 = 0, c1 = 0;
    const int b0 = nb - 1 - 2 * static_cast<int>(threadIdx.x);
    if (b0 >= 0) c0 = hist[b0];
    if (b0 - 1 >= 0) c1 = hist[b0 - 1];
    const int before = block_exclusive_scan(c0 + c1, warp_sums, &scan_total);
    if (c0 > 0 && before < krem && krem <= before + c0) {
      sel_bin = b0;
      sel_above = before;
    } else if (c1 > 0 && before + c0 < krem && krem <= before + c0 + c1) {
      sel_bin = b0 - 1;
      sel_above = before + c0;
    }
    __syncthreads();
    prefix |= static_cast<uint32_t>(sel_bin) << shift;
    mask |= dmask << shift;
    krem -= sel_above;
    __syncthreads();
  }
  const uint32_t T = prefix;  // key of the ksel-th largest element
  const int need_eq = krem;   // how many elements equal to T are kept (lowest positions)

  // ---- 3. ordered compaction; warp w owns positions [w*span, (w+1)*span)
  const int span = (((n + SEL_WARPS - 1) / SEL_WARPS) + 31) & ~31;
  const int w_lo = warp * span;
  const int w_hi = min(n, w_lo + span);
  int cg = 0, ce = 0;
  for (int base = w_lo; base < w_hi; base += 32) {
    const int j = base + lane;
    const uint32_t key = (j < w_hi) ? keys[j] : 0u;
    cg += __popc(__ballot_sync(0xffffffffu, j < w_hi && key > T));
    ce += __popc(__ballot_sync(0xffffffffu, j < w_hi && key == T));
  }
  if (lane == 0) {
    wgt[warp] = cg;
    weq[warp] = ce;
  }
  __syncthreads();
  int gt_before = 0, eq_before = 0;
  for (int w = 0; w < warp; ++w) {
    gt_before += wgt[w];
    eq_before += weq[w];
  }
  int out_pos = gt_before + min(eq_before, need_eq);
  int32_t* orow = out_idx + static_cast<size_t>(row) * ksel;
  const uint32_t lt_mask = (1u << lane) - 1u;
  for (int base = w_lo; base < w_hi; base += 32) {
    const int j = base + lane;
    const uint32_t key = (j < w_hi) ? keys[j] : 0u;
    const bool gt = j < w_hi && key > T;
    const bool eq = j < w_hi && key == T;
    const uint32_t be = __ballot_sync(0xffffffffu, eq);
    const bool take = gt || (eq && (eq_before + __popc(be & lt_mask)) < need_eq);
    const uint32_t bt = __ballot_sync(0xffffffffu, take);
    if (take) orow[out_pos + __popc(bt & lt_mask)] = j;
    out_pos += __popc(bt);
    eq_before += __popc(be);
  }
}

// ---------------------------------------------------------------------------------------
// Fast path for rows that fit in shared memory and pooling radii up to RMAX.
// Thread t owns the EPT consecutive positions [t*EPT, (t+1)*EPT): pooling is a sliding
// window over registers, histogram updates are run-length aggregated (pooled neighbours
// fall into the same bin), and the ordered compaction is a single block scan.  Keys sit
// in shared memory at slot j + j/32, which keeps the strided per-thread sweeps free of
// bank conflicts.  The first histogram pass bins (key - min) >> shift with the shift
// chosen from the row's key range, so the bins are spread over the values that occur.
__device__ __forceinline__ int key_slot(int j) { return j + (j >> 5); }
// Layout of the one-CTA-per-row kernel: four pad words after every 32 keys.  A thread's run
// starts at a multiple of 8 keys, so it reads and writes its keys four at a time as aligned
// 16-byte vectors, and the runs of eight neighbouring threads fall into different banks.
__device__ __forceinline__ int key_slot4(int j) { return j + ((j >> 5) << 2); }
__device__ __forceinline__ uint4 ld_keys4(const uint32_t* keys, int j) {
  return *reinterpret_cast<const uint4*>(keys + key_slot4(j));
}
constexpr int FAST_MAX_KEYS = 40960;  // 40 keys per thread: what fits with the padding
constexpr int CAND_CAP = 2048;   // keys of the first-pass bin that are refined from a list
constexpr int MASK_WORDS = 2;    // a thread owns at most 64 positions (SEL_SMEM_KEYS / SEL_THREADS = 48)

// PT = -1: pooling radius r <= RMAX and pool type are run-time values.  PT = 0 (max) or 1
// (avg): the radius is exactly RMAX, so the window loop has no per-element tests.
template <int RMAX, int PT>
__global__ void __launch_bounds__(SEL_THREADS, 1)
pool_topk_fast_kernel(const float* __restrict__ vote, int n, int gsum, int r, int pool_type,
                      int ept, int ksel, int32_t* __restrict__ out_idx, int discard_votes) {
  extern __shared__ __align__(16) uint32_t keys[];
  __shared__ int hist[NBINS];
  __shared__ int warp_sums[SEL_WARPS];
  __shared__ int scan_total;
  __shared__ int sel_bin, sel_above, sel_count, ncand_s;
  __shared__ int above_s, br_lo, br_hi;
  __shared__ uint32_t red_min[SEL_WARPS], red_max[SEL_WARPS];
  __shared__ uint32_t cand[CAND_CAP];
  int ncand = 0;

  const int row = blockIdx.x;
  const float* vrow = vote + static_cast<size_t>(row) * gsum * n;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int base = threadIdx.x * ept;
  // the gather kernel behind this one may become resident now; it waits for this kernel's end
  pdl_launch_dependents();

  // ---- 1. pooling
  // The row is first copied into the key slots with coalesced loads (raw fp32 bits), then
  // every thread pools its own positions in place over a rolling register window.  The
  // values it needs from its neighbours' positions are saved before anybody overwrites.
  uint32_t kmin = 0xffffffffu, kmax = 0u;
  {
    const int total = SEL_THREADS * ept;
    if (gsum == 1) {
      // eight loads in flight per thread before the first store: the votes come from L2, and
      // one load per loop turn would pay that latency once per element (ept is a multiple of 8)
      for (int j0 = threadIdx.x; j0 < total; j0 += 8 * SEL_THREADS) {
        uint32_t x[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int j = j0 + u * SEL_THREADS;
          x[u] = (j < n) ? __float_as_uint(__ldg(vrow + j)) : 0u;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) keys[key_slot4(j0 + u * SEL_THREADS)] = x[u];
      }
    } else {
      // group sum: four positions per thread and step, so that the loads of a step are
      // independent of one another; heads are added in ascending order
      for (int j0 = threadIdx.x; j0 < total; j0 += 4 * SEL_THREADS) {
        float x[4] = {0.f, 0.f, 0.f, 0.f};
        for (int t = 0; t < gsum; ++t) {
          const float* src = vrow + static_cast<size_t>(t) * n;
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int j = j0 + u * SEL_THREADS;
            if (j < n) x[u] += __ldg(src + j);
          }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int j = j0 + u * SEL_THREADS;
          if (j < total) keys[key_slot4(j)] = __float_as_uint(x[u]);
        }
      }
    }
    __syncthreads();
    if (discard_votes && gsum == 1) {
      // The row is in shared memory and its votes are scratch that nobody reads again: drop the
      // whole 128-byte lines inside the row from L2, so that they are not written back to HBM
      // while the gather kernel needs the bandwidth (16.8 MB per layer of the 32K GQA workload).
      // Lines that the row shares with its neighbours stay.
      const uintptr_t b0 = (reinterpret_cast<uintptr_t>(vrow) + 127) & ~static_cast<uintptr_t>(127);
      const uintptr_t b1 = reinterpret_cast<uintptr_t>(vrow + n) & ~static_cast<uintptr_t>(127);
      for (uintptr_t a = b0 + static_cast<uintptr_t>(threadIdx.x) * 128; a < b1;
           a += static_cast<uintptr_t>(SEL_THREADS) * 128)
        discard_l2_line(reinterpret_cast<const void*>(a));
    }
    // a[]: the last RMAX values before the current block of 8, the block, the next block
    float a[RMAX + 16];
    float halo_r[RMAX > 0 ? RMAX : 1];
#pragma unroll
    for (int i = 0; i < RMAX; ++i) {
      const int jl = base - RMAX + i;             // left neighbours
      a[i] = (jl >= 0) ? __uint_as_float(keys[key_slot4(jl)]) : 0.f;
      const int jr = base + ept + i;              // right neighbours
      halo_r[i] = (jr < total) ? __uint_as_float(keys[key_slot4(jr)]) : 0.f;
    }
    auto load8 = [&](int pos, float* dst) {       // own positions pos .. pos + 7
      const uint4 x = ld_keys4(keys, pos), y = ld_keys4(keys, pos + 4);
      dst[0] = __uint_as_float(x.x); dst[1] = __uint_as_float(x.y);
      dst[2] = __uint_as_float(x.z); dst[3] = __uint_as_float(x.w);
      dst[4] = __uint_as_float(y.x); dst[5] = __uint_as_float(y.y);
      dst[6] = __uint_as_float(y.z); dst[7] = __uint_as_float(y.w);
    };
    auto next8 = [&](int sb_next, float* dst) {   // the block after sb_next - 8, or the halo
      if (sb_next < ept) {
        load8(base + sb_next, dst);
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) dst[i] = (i < RMAX) ? halo_r[i < RMAX ? i : 0] : 0.f;
      }
    };
    load8(base, a + RMAX);
    __syncthreads();  // every neighbour value is in registers before anybody overwrites
    next8(8, a + RMAX + 8);
    for (int sb = 0; sb < ept; sb += 8) {
      uint32_t out[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        float p = 0.f;  // votes are >= 0: zero is neutral for max and is the avg padding
#pragma unroll
        for (int t = 0; t <= 2 * RMAX; ++t) {
          const int off = t - RMAX;
          if (PT >= 0 || (off >= -r && off <= r))
            p = ((PT >= 0) ? (PT == 0) : (pool_type == 0)) ? fmaxf(p, a[i + t]) : p + a[i + t];
        }
        const int j = base + sb + i;
        uint32_t key = 0u;  // positions past the row end rank below every real key
        if (j < n) {
          key = float_to_key(p);
          kmin = min(kmin, key);
          kmax = max(kmax, key);
        }
        out[i] = key;
      }
#pragma unroll
      for (int i = 0; i < RMAX + 8; ++i) a[i] = a[i + 8];
      // the block after the next one is still untouched; the current one is done with
      next8(sb + 16, a + RMAX + 8);
      *reinterpret_cast<uint4*>(keys + key_slot4(base + sb)) = make_uint4(out[0], out[1], out[2], out[3]);
      *reinterpret_cast<uint4*>(keys + key_slot4(base + sb + 4)) =
          make_uint4(out[4], out[5], out[6], out[7]);
    }
  }
  kmin = __reduce_min_sync(0xffffffffu, kmin);
  kmax = __reduce_max_sync(0xffffffffu, kmax);
  if (lane == 0) {
    red_min[warp] = kmin;
    red_max[warp] = kmax;
  }
  __syncthreads();
  kmin = red_min[lane];
  kmax = red_max[lane];
  kmin = __reduce_min_sync(0xffffffffu, kmin);
  kmax = __reduce_max_sync(0xffffffffu, kmax);

  // ---- 2. threshold
  // One histogram pass over all keys picks the bin that holds the ksel-th largest key.  A
  // second sweep notes, per thread, which of its keys lie above that bin (kept for sure,
  // one bit each) and which lie inside it, and copies the latter to a small candidate
  // list; the remaining passes refine the threshold on that list alone.
  uint32_t lo = kmin;
  int krem = ksel;
  uint32_t T = kmin;
  uint32_t m_gt[MASK_WORDS], m_in[MASK_WORDS];  // bit i: own key i above / inside the bin
#pragma unroll
  for (int wd = 0; wd < MASK_WORDS; ++wd) { m_gt[wd] = 0u; m_in[wd] = 0u; }
  bool use_list = false;
  if (kmax != kmin) {
    const uint32_t range = kmax - kmin;
    int shift = 32 - __clz(range) - 11;
    if (shift < 0) shift = 0;
    uint32_t width_m1 = range;  // candidates are keys with key - lo <= width_m1
    bool first = true;
    // 2a. A guess from a sample.  Every fourth key goes into the histogram (a quarter of the
    // shared-memory atomics of a full pass, which is what that pass spends its time on); the
    // sample's cumulative counts give a RANGE of bins that should hold the ksel-th key: the
    // bins between the sample ranks 4 standard deviations to either side of ksel/4.  One sweep
    // then counts, exactly, the keys above that range and collects the keys inside it.  If the
    // exact counts confirm that the ksel-th key is inside and the range fits the candidate list,
    // the threshold is refined on the list; otherwise nothing of this is used and the full
    // histogram pass below decides (exactness never rests on the sample).
    {
      for (int b = threadIdx.x; b < NBINS; b += SEL_THREADS) hist[b] = 0;
      if (threadIdx.x == 0) { ncand_s = 0; above_s = 0; br_lo = 0; br_hi = NBINS - 1; }
      __syncthreads();
      for (int i0 = 0; i0 < ept; i0 += 4) {
        const uint32_t key = keys[key_slot4(base + i0)];
        if (key >= kmin) atomicAdd(&hist[(key - kmin) >> shift], 1);  // (padding keys are below kmin)
      }
      __syncthreads();
      int c0 = 0, c1 = 0;
      const int b0 = NBINS - 1 - 2 * static_cast<int>(threadIdx.x);
      if (b0 >= 0) c0 = hist[b0];
      if (b0 - 1 >= 0) c1 = hist[b0 - 1];
      const int before = block_exclusive_scan(c0 + c1, warp_sums, &scan_total);
      const int m_s = scan_total;  // samples in the row
      const float pfrac = static_cast<float>(ksel) / static_cast<float>(n);
      const int delta = static_cast<int>(4.f * sqrtf(static_cast<float>(m_s) * pfrac * (1.f - pfrac))) + 2;
      const int r_mid = static_cast<int>(static_cast<long long>(ksel) * m_s / n);
      const int r_hi = max(1, r_mid - delta);  // sample rank that bounds the range from above
      const int r_lo = r_mid + delta;          // ... from below; beyond the sample: down to the lowest bin
      if (c0 > 0 && before < r_hi && r_hi <= before + c0) br_hi = b0;
      else if (c1 > 0 && before + c0 < r_hi && r_hi <= before + c0 + c1) br_hi = b0 - 1;
      if (c0 > 0 && before < r_lo && r_lo <= before + c0) br_lo = b0;
      else if (c1 > 0 && before + c0 < r_lo && r_lo <= before + c0 + c1) br_lo = b0 - 1;
      __syncthreads();
      const int b_hi = br_hi, b_lo = r_lo > m_s ? 0 : br_lo;
      int cntg = 0, cnti = 0;
      for (int i0 = 0; i0 < ept; i0 += 4) {
        const uint4 kv = ld_keys4(keys, base + i0);
        const uint32_t k4[4] = {kv.x, kv.y, kv.z, kv.w};
        uint32_t bg = 0u, bi = 0u;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const uint32_t key = k4[u];
          const int bin = static_cast<int>((key - kmin) >> shift);
          const bool real = key >= kmin;
          const bool gt = real && bin > b_hi;
          const bool inb = real && bin >= b_lo && bin <= b_hi;
          bg |= static_cast<uint32_t>(gt) << u;
          bi |= static_cast<uint32_t>(inb) << u;
          cntg += gt;
          cnti += inb;
        }
        if (i0 < 32) { m_gt[0] |= bg << i0; m_in[0] |= bi << i0; }
        else { m_gt[1] |= bg << (i0 - 32); m_in[1] |= bi << (i0 - 32); }
      }
      // the keys inside the range go to the candidate list: one atomic per warp reserves the
      // warp's slots (a thousand single appends to one counter would take as long as the pass
      // this replaces), a warp scan places each thread's keys
      {
        int inc = cnti;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int y = __shfl_up_sync(0xffffffffu, inc, o);
          if (lane >= o) inc += y;
        }
        int wbase = 0;
        if (lane == 31 && inc > 0) wbase = atomicAdd(&ncand_s, inc);
        wbase = __shfl_sync(0xffffffffu, wbase, 31);
        int at = wbase + inc - cnti;
#pragma unroll
        for (int wd = 0; wd < MASK_WORDS; ++wd) {
          uint32_t rest = m_in[wd];
          while (rest) {
            const int i = wd * 32 + __ffs(rest) - 1;
            rest &= rest - 1;
            if (at < CAND_CAP) cand[at] = keys[key_slot4(base + i)];
            ++at;
          }
        }
      }
      cntg = __reduce_add_sync(0xffffffffu, cntg);
      if (lane == 0 && cntg) atomicAdd(&above_s, cntg);
      __syncthreads();
      const int above = above_s, inside = ncand_s;
      __syncthreads();  // everybody has read the counts before anybody starts the next pass
      if (above < ksel && ksel <= above + inside && inside <= CAND_CAP) {
        first = false;
        use_list = true;
        ncand = inside;
        krem = ksel - above;
        lo = kmin + (static_cast<uint32_t>(b_lo) << shift);
        const unsigned long long top =
            static_cast<unsigned long long>(kmin) + (static_cast<unsigned long long>(b_hi + 1) << shift) - 1ull;
        const uint32_t hi_key = top > kmax ? kmax : static_cast<uint32_t>(top);
        width_m1 = hi_key - lo;
        shift = 32 - __clz(width_m1 | 1u) - 11;
        if (shift < 0) shift = 0;
      } else {
#pragma unroll
        for (int wd = 0; wd < MASK_WORDS; ++wd) { m_gt[wd] = 0u; m_in[wd] = 0u; }
      }
    }
#pragma unroll 1
    for (;;) {
      for (int b = threadIdx.x; b < NBINS; b += SEL_THREADS) hist[b] = 0;
      __syncthreads();
      if (!use_list) {
        int cur = -1, cnt = 0;
        for (int i0 = 0; i0 < ept; i0 += 4) {
          const uint4 kv = ld_keys4(keys, base + i0);
          const uint32_t k4[4] = {kv.x, kv.y, kv.z, kv.w};
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const uint32_t key = k4[u];
            const uint32_t rel = key - lo;
            if (key >= lo && rel <= width_m1) {
              const int b = static_cast<int>(rel >> shift);
              if (b != cur) {
                if (cnt) atomicAdd(&hist[cur], cnt);
                cur = b;
                cnt = 0;
              }
              ++cnt;
            }
          }
        }
        if (cnt) atomicAdd(&hist[cur], cnt);
      } else {
        for (int c = threadIdx.x; c < ncand; c += SEL_THREADS) {
          const uint32_t rel = cand[c] - lo;  // wraps to a huge value for keys below lo
          if (rel <= width_m1) atomicAdd(&hist[rel >> shift], 1);
        }
      }
      __syncthreads();
      int c0 = 0, c1 = 0;
      const int b0 = NBINS - 1 - 2 * static_cast<int>(threadIdx.x);
      if (b0 >= 0) c0 = hist[b0];
      if (b0 - 1 >= 0) c1 = hist[b0 - 1];
      const int before = block_exclusive_scan(c0 + c1, warp_sums, &scan_total);
      if (c0 > 0 && before < krem && krem <= before + c0) {
        sel_bin = b0;
        sel_above = before;
        sel_count = c0;
      } else if (c1 > 0 && before + c0 < krem && krem <= before + c0 + c1) {
        sel_bin = b0 - 1;
        sel_above = before + c0;
        sel_count = c1;
      }
      if (threadIdx.x == 0) ncand_s = 0;
      __syncthreads();
      krem -= sel_above;
      lo += static_cast<uint32_t>(sel_bin) << shift;
      const int in_bin = sel_count;
      const int done = (shift == 0);
      __syncthreads();
      if (first) {
        // classify own keys against the chosen bin; gather the bin's keys if they fit
        first = false;
        const uint32_t hi_m1 = done ? 0u : ((1u << shift) - 1u);
        use_list = !done && in_bin <= CAND_CAP;
        for (int i0 = 0; i0 < ept; i0 += 4) {
          const uint4 kv = ld_keys4(keys, base + i0);
          const uint32_t k4[4] = {kv.x, kv.y, kv.z, kv.w};
          uint32_t bg = 0u, bi = 0u;  // four bits each
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const uint32_t key = k4[u];
            const bool inb = key >= lo && key - lo <= hi_m1;
            const bool gt = key >= lo && key - lo > hi_m1;
            bg |= static_cast<uint32_t>(gt) << u;
            bi |= static_cast<uint32_t>(inb) << u;
            if (inb && use_list) cand[atomicAdd(&ncand_s, 1)] = key;
          }
          // i0 is a multiple of 4: the four bits never straddle a mask word
          if (i0 < 32) { m_gt[0] |= bg << i0; m_in[0] |= bi << i0; }
          else { m_gt[1] |= bg << (i0 - 32); m_in[1] |= bi << (i0 - 32); }
        }
        __syncthreads();
        ncand = ncand_s;
      }
      if (done) break;
      width_m1 = (1u << shift) - 1u;
      shift = shift > 11 ? shift - 11 : 0;
    }
    T = lo;
  } else {
    // every key equals T
#pragma unroll
    for (int wd = 0; wd < MASK_WORDS; ++wd)
      for (int i = wd * 32; i < min(ept, wd * 32 + 32); ++i)
        if (base + i < n) m_in[wd] |= 1u << (i & 31);
  }
  const int need_eq = krem;

  // ---- 3. ordered compaction
  // Keys inside the first bin are compared with the final threshold (few per thread), the
  // rest is known from the bit masks; one block scan gives every thread its output offset.
  uint32_t m_eq[MASK_WORDS];
  int cg = 0, ce = 0;
#pragma unroll
  for (int wd = 0; wd < MASK_WORDS; ++wd) {
    m_eq[wd] = 0u;
    uint32_t rest = m_in[wd];
    while (rest) {
      const int i = wd * 32 + __ffs(rest) - 1;
      rest &= rest - 1;
      const uint32_t key = keys[key_slot4(base + i)];
      if (key > T) m_gt[wd] |= 1u << (i & 31);
      else if (key == T) m_eq[wd] |= 1u << (i & 31);
    }
    cg += __popc(m_gt[wd]);
    ce += __popc(m_eq[wd]);
  }
  // Two counts in one scan: keys above the threshold in the high half, keys equal to it in
  // the low half.  Either total is at most n <= FAST_MAX_KEYS < 65536, so the low half never
  // carries into the high one, and the word is unsigned so that a high half of 32768 or more
  // (ksel that large is valid) stays a count after the shift.
  static_assert(FAST_MAX_KEYS < 65536, "two 16-bit counts share one scan word");
  uint32_t* scan_u = reinterpret_cast<uint32_t*>(warp_sums);
  const uint32_t packed =
      block_exclusive_scan<uint32_t>((static_cast<uint32_t>(cg) << 16) | static_cast<uint32_t>(ce),
                                     scan_u, reinterpret_cast<uint32_t*>(&scan_total));
  int eq_before = static_cast<int>(packed & 0xffffu);
  int out_pos = static_cast<int>(packed >> 16) + min(eq_before, need_eq);
  int32_t* orow = out_idx + static_cast<size_t>(row) * ksel;
#pragma unroll
  for (int wd = 0; wd < MASK_WORDS; ++wd) {
    uint32_t rest = m_gt[wd] | m_eq[wd];
    while (rest) {
      const int bit = __ffs(rest) - 1;
      rest &= rest - 1;
      const bool is_eq = (m_eq[wd] >> bit) & 1u;
      if (!is_eq || eq_before++ < need_eq) orow[out_pos++] = base + wd * 32 + bit;
    }
  }
}

// ---------------------------------------------------------------------------------------
// Rows too long for one CTA's shared memory: the same radix select spread over many CTAs.
// A row is cut into chunks of WIDE_CHUNK positions, one CTA each; histograms are built per
// CTA in shared memory and added into a per-row histogram in global memory; a one-CTA-per-
// row kernel picks the bin between the passes.  Keys live in global scratch:
//   keys [rows][n] | hist [rows][NBINS] | state [rows][8] | counts [rows][nblk][2]
// state: 0 prefix, 1 mask, 2 remaining rank.  Digits: 11, 11 and 10 bits from the top.
constexpr int WIDE_THREADS = 256;
constexpr int WIDE_EPT = 32;                            // positions per thread, contiguous
constexpr int WIDE_CHUNK = WIDE_THREADS * WIDE_EPT;     // 8192 positions per CTA
constexpr int WIDE_HALO = 31;                           // largest pooling radius

struct WideBufs {
  uint32_t* keys;
  int* hist;
  int* state;
  int* counts;
  int nblk;
};

__device__ __forceinline__ int wide_shift(int pass) { return pass == 0 ? 21 : (pass == 1 ? 10 : 0); }
__device__ __forceinline__ int wide_bins(int pass) { return pass == 2 ? 1024 : 2048; }

// Adds this CTA's keys that match the row's prefix into the row histogram (digit `pass`).
__device__ __forceinline__ void wide_histogram(const uint32_t (&key_of_thread)[32], int valid, int pass,
                                               uint32_t prefix, uint32_t mask, int* hist_s,
                                               int* hist_g) {
  const int shift = wide_shift(pass);
  const uint32_t dmask = wide_bins(pass) - 1;
  for (int b = threadIdx.x; b < NBINS; b += WIDE_THREADS) hist_s[b] = 0;
  __syncthreads();
  int cur = -1, cnt = 0;
#pragma unroll
  for (int i = 0; i < WIDE_EPT; ++i) {
    const uint32_t key = key_of_thread[i];
    if (i < valid && (key & mask) == prefix) {
      const int b = static_cast<int>((key >> shift) & dmask);
      if (b != cur) {
        if (cnt) atomicAdd(&hist_s[cur], cnt);
        cur = b;
        cnt = 0;
      }
      ++cnt;
    }
  }
  if (cnt) atomicAdd(&hist_s[cur], cnt);
  __syncthreads();
  for (int b = threadIdx.x; b < NBINS; b += WIDE_THREADS)
    if (hist_s[b]) atomicAdd(&hist_g[b], hist_s[b]);
}

// Pooling of one chunk (staged through shared memory with its halo), keys to scratch, and
// the first histogram pass.
__global__ void __launch_bounds__(WIDE_THREADS)
wide_pool_kernel(const float* __restrict__ vote, int n, int gsum, int pool_kernel, int pool_type,
                 WideBufs wb) {
  pdl_launch_dependents();  // the kernels behind this one are launched early and wait for its end
  __shared__ float raw[WIDE_CHUNK + 2 * WIDE_HALO + (WIDE_CHUNK + 2 * WIDE_HALO) / 32 + 1];
  __shared__ int hist_s[NBINS];
  const int row = blockIdx.y;
  const int c0 = blockIdx.x * WIDE_CHUNK;
  const int r = pool_kernel >> 1;
  const float* vrow = vote + static_cast<size_t>(row) * gsum * n;
  for (int t = threadIdx.x; t < WIDE_CHUNK + 2 * r; t += WIDE_THREADS) {
    const int j = c0 - r + t;
    raw[key_slot(t)] = (j >= 0 && j < n) ? (gsum == 1 ? __ldg(vrow + j) : ld_vote(vrow, j, n, gsum)) : 0.f;
  }
  __syncthreads();
  uint32_t mine[WIDE_EPT];
  const int base = threadIdx.x * WIDE_EPT;
  int valid = n - (c0 + base);
  valid = valid < 0 ? 0 : (valid > WIDE_EPT ? WIDE_EPT : valid);
#pragma unroll
  for (int i = 0; i < WIDE_EPT; ++i) {
    float p = 0.f;  // votes are >= 0: zero is neutral for max and is the avg padding
    for (int t = 0; t <= 2 * r; ++t) {
      const float x = raw[key_slot(base + i + t)];
      p = (pool_type == 0) ? fmaxf(p, x) : p + x;
    }
    if (pool_type != 0) p = p / static_cast<float>(pool_kernel);
    mine[i] = float_to_key(p);
  }
  // keys go out through shared memory so that the global stores are coalesced
  __syncthreads();  // everybody is done reading the raw votes
  uint32_t* stage = reinterpret_cast<uint32_t*>(raw);
#pragma unroll
  for (int i = 0; i < WIDE_EPT; ++i) stage[key_slot(base + i)] = mine[i];
  __syncthreads();
  uint32_t* krow = wb.keys + static_cast<size_t>(row) * n + c0;
  for (int t = threadIdx.x; t < WIDE_CHUNK && c0 + t < n; t += WIDE_THREADS) krow[t] = stage[key_slot(t)];
  wide_histogram(mine, valid, 0, 0u, 0u, hist_s, wb.hist + static_cast<size_t>(row) * NBINS);
}

// One CTA per row: walk the row histogram from the top, fix the next digit of the
// threshold, clear the histogram for the next pass.
__global__ void __launch_bounds__(SEL_THREADS)
wide_pick_kernel(int pass, int ksel, WideBufs wb) {
  pdl_launch_dependents();
  pdl_wait();  // launched early: the previous kernel's results are complete only from here on
  __shared__ int warp_sums[SEL_WARPS];
  __shared__ int scan_total;
  const int row = blockIdx.x;
  int* hist = wb.hist + static_cast<size_t>(row) * NBINS;
  int* st = wb.state + row * 8;
  const int nb = wide_bins(pass);
  const int krem = pass == 0 ? ksel : st[2];
  const uint32_t prefix = pass == 0 ? 0u : static_cast<uint32_t>(st[0]);
  const uint32_t mask = pass == 0 ? 0u : static_cast<uint32_t>(st[1]);
  int c0 = 0, c1 = 0;
  const int b0 = nb - 1 - 2 * static_cast<int>(threadIdx.x);
  if (b0 >= 0) c0 = hist[b0];
  if (b0 - 1 >= 0) c1 = hist[b0 - 1];
  const int before = block_exclusive_scan(c0 + c1, warp_sums, &scan_total);
  int bin = -1, above = 0;
  if (c0 > 0 && before < krem && krem <= before + c0) { bin = b0; above = before; }
  else if (c1 > 0 && before + c0 < krem && krem <= before + c0 + c1) { bin = b0 - 1; above = before + c0; }
  __syncthreads();  // every thread has read the state and its bins
  if (bin >= 0) {
    const int shift = wide_shift(pass);
    st[0] = static_cast<int>(prefix | (static_cast<uint32_t>(bin) << shift));
    st[1] = static_cast<int>(mask | (static_cast<uint32_t>(nb - 1) << shift));
    st[2] = krem - above;
  }
  for (int b = threadIdx.x; b < NBINS; b += SEL_THREADS) hist[b] = 0;
}

__global__ void __launch_bounds__(WIDE_THREADS)
wide_hist_kernel(int n, int pass, WideBufs wb) {
  pdl_launch_dependents();
  pdl_wait();  // launched early: the previous kernel's results are complete only from here on
  __shared__ int hist_s[NBINS];
  const int row = blockIdx.y;
  // lane-strided reads (coalesced); the order of the keys does not matter here.  Only keys
  // that match the row's prefix count, and those are few after the first pass.
  const int c0 = blockIdx.x * WIDE_CHUNK;
  const uint32_t* krow = wb.keys + static_cast<size_t>(row) * n + c0;
  const int* st = wb.state + row * 8;
  const uint32_t prefix = static_cast<uint32_t>(st[0]), mask = static_cast<uint32_t>(st[1]);
  const int shift = wide_shift(pass);
  const uint32_t dmask = wide_bins(pass) - 1;
  for (int b = threadIdx.x; b < NBINS; b += WIDE_THREADS) hist_s[b] = 0;
  __syncthreads();
#pragma unroll 8
  for (int i = 0; i < WIDE_EPT; ++i) {
    const int t = i * WIDE_THREADS + threadIdx.x;
    if (c0 + t < n) {
      const uint32_t key = krow[t];
      if ((key & mask) == prefix) atomicAdd(&hist_s[(key >> shift) & dmask], 1);
    }
  }
  __syncthreads();
  int* hist_g = wb.hist + static_cast<size_t>(row) * NBINS;
  for (int b = threadIdx.x; b < NBINS; b += WIDE_THREADS)
    if (hist_s[b]) atomicAdd(&hist_g[b], hist_s[b]);
}

// Per chunk: how many keys are above the threshold and how many equal it.
__global__ void __launch_bounds__(WIDE_THREADS)
wide_count_kernel(int n, WideBufs wb) {
  pdl_launch_dependents();
  pdl_wait();  // launched early: the previous kernel's results are complete only from here on
  __shared__ int sg, se;
  const int row = blockIdx.y;
  if (threadIdx.x == 0) { sg = 0; se = 0; }
  __syncthreads();
  const uint32_t T = static_cast<uint32_t>(wb.state[row * 8 + 0]);
  const int c0 = blockIdx.x * WIDE_CHUNK;
  const uint32_t* krow = wb.keys + static_cast<size_t>(row) * n + c0;
  int cg = 0, ce = 0;
#pragma unroll 8
  for (int i = 0; i < WIDE_EPT; ++i) {
    const int t = i * WIDE_THREADS + threadIdx.x;
    if (c0 + t < n) {
      const uint32_t key = krow[t];
      cg += key > T;
      ce += key == T;
    }
  }
  cg = __reduce_add_sync(0xffffffffu, cg);
  ce = __reduce_add_sync(0xffffffffu, ce);
  if ((threadIdx.x & 31) == 0) { atomicAdd(&sg, cg); atomicAdd(&se, ce); }
  __syncthreads();
  if (threadIdx.x == 0) {
    int* c = wb.counts + (static_cast<size_t>(row) * wb.nblk + blockIdx.x) * 2;
    c[0] = sg;
    c[1] = se;
  }
}

// Ordered compaction: every key above the threshold, and the lowest-position keys equal
// to it until ksel positions are out, in ascending position.
__global__ void __launch_bounds__(WIDE_THREADS)
wide_write_kernel(int n, int ksel, int32_t* __restrict__ out_idx, WideBufs wb) {
  pdl_launch_dependents();
  pdl_wait();  // launched early: the previous kernel's results are complete only from here on
  __shared__ int warp_sums[WIDE_THREADS / 32];
  const int row = blockIdx.y;
  const uint32_t T = static_cast<uint32_t>(wb.state[row * 8 + 0]);
  const int need_eq = wb.state[row * 8 + 2];
  // keys selected in the chunks before this one (a short serial sum)
  int gt_before = 0, eq_before = 0;
  const int* c = wb.counts + static_cast<size_t>(row) * wb.nblk * 2;
  for (int b = 0; b < static_cast<int>(blockIdx.x); ++b) {
    gt_before += c[2 * b];
    eq_before += c[2 * b + 1];
  }
  __shared__ uint32_t stage[WIDE_CHUNK + WIDE_CHUNK / 32 + 1];
  const int c0 = blockIdx.x * WIDE_CHUNK;
  {
    const uint32_t* kin = wb.keys + static_cast<size_t>(row) * n + c0;
    for (int t = threadIdx.x; t < WIDE_CHUNK; t += WIDE_THREADS)
      stage[key_slot(t)] = (c0 + t < n) ? kin[t] : 0u;
  }
  __syncthreads();
  const int lbase = threadIdx.x * WIDE_EPT;
  const int base = c0 + lbase;
  uint32_t m_gt = 0u, m_eq = 0u;
#pragma unroll
  for (int i = 0; i < WIDE_EPT; ++i) {
    const uint32_t key = stage[key_slot(lbase + i)];
    const bool in = base + i < n;
    m_gt |= static_cast<uint32_t>(in && key > T) << i;
    m_eq |= static_cast<uint32_t>(in && key == T) << i;
  }
  // Block scan over the 8 warps of this kernel, two counts in one word: keys above the
  // threshold in the high half, keys equal to it in the low half.  A chunk has WIDE_CHUNK =
  // 8192 positions, so either half stays below 2^14 and the packed sums never carry or reach
  // the sign bit; what came before the chunk is added outside the packed word.
  static_assert(WIDE_CHUNK < 32768, "two counts of a chunk share one signed scan word");
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int x = (__popc(m_gt) << 16) | __popc(m_eq);
  int inc = x;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += y;
  }
  if (lane == 31) warp_sums[warp] = inc;
  __syncthreads();
  int wpre = 0;
  for (int w2 = 0; w2 < warp; ++w2) wpre += warp_sums[w2];
  const int packed = wpre + inc - x;
  int eq_seen = eq_before + (packed & 0xffff);
  int out_pos = gt_before + (packed >> 16) + min(eq_seen, need_eq);
  int32_t* orow = out_idx + static_cast<size_t>(row) * ksel;
  uint32_t rest = m_gt | m_eq;
  while (rest) {
    const int bit = __ffs(rest) - 1;
    rest &= rest - 1;
    const bool is_eq = (m_eq >> bit) & 1u;
    if (!is_eq || eq_seen++ < need_eq) orow[out_pos++] = base + bit;
  }
}

__global__ void iota_kernel(int32_t* out, int rows, int n, int row_stride) {
  const long long total = static_cast<long long>(rows) * n;
  for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < total;
       i += static_cast<long long>(gridDim.x) * blockDim.x) {
    const int rw = static_cast<int>(i / n);
    const int j = static_cast<int>(i - static_cast<long long>(rw) * n);
    out[static_cast<size_t>(rw) * row_stride + j] = j;
  }
}

}  // namespace

static DeviceOnce& select_attr_once() {
  static DeviceOnce once;
  return once;
}

static inline int key_slot4_host(int j) { return j + ((j >> 5) << 2); }
constexpr int FAST_SMEM_BYTES = (FAST_MAX_KEYS + FAST_MAX_KEYS / 8 + 64) * 4;

bool select_needs_scratch(int n) { return n > SEL_SMEM_KEYS; }

static inline size_t up256(size_t x) { return (x + 255) / 256 * 256; }
static inline int wide_nblk(int n) { return (n + WIDE_CHUNK - 1) / WIDE_CHUNK; }

// Scratch of the many-CTA path: keys | row histograms | row state | chunk counts.
size_t select_scratch_bytes(int rows, int n) {
  if (!select_needs_scratch(n)) return 0;
  const size_t r = static_cast<size_t>(rows);
  return up256(r * n * 4) + up256(r * NBINS * 4) + up256(r * 8 * 4) + up256(r * wide_nblk(n) * 2 * 4);
}

cudaError_t launch_pool_topk(const float* vote, int rows, int n, int pool_kernel, int pool_type,
                             int ksel, int32_t* out_idx, float* pooled_scratch,
                             cudaStream_t stream, int* launches, int gsum, bool vote_is_scratch) {
  // the opt-in to more than 48 KB of dynamic shared memory is a property of the device's
  // context, so it is made once per device
  DeviceOnce& once = select_attr_once();
  if (!once.done()) {
    cudaError_t e = cudaFuncSetAttribute(pool_topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         SEL_SMEM_KEYS * 4);
    if (e != cudaSuccess) return e;
#define SNAPKV_FAST_ATTR(RM, P)                                                              \
  e = cudaFuncSetAttribute(pool_topk_fast_kernel<RM, P>,                                     \
                           cudaFuncAttributeMaxDynamicSharedMemorySize, FAST_SMEM_BYTES);    \
  if (e != cudaSuccess) return e;
    SNAPKV_FAST_ATTR(3, -1) SNAPKV_FAST_ATTR(7, -1)
    SNAPKV_FAST_ATTR(2, 0) SNAPKV_FAST_ATTR(2, 1) SNAPKV_FAST_ATTR(3, 0) SNAPKV_FAST_ATTR(3, 1)
    SNAPKV_FAST_ATTR(6, 0) SNAPKV_FAST_ATTR(6, 1)
#undef SNAPKV_FAST_ATTR
    once.set();
  }
  const int r = pool_kernel >> 1;
  // One cluster of small CTAs per row: for rows too long for the one-CTA kernel below, and
  // whenever there are too few rows to fill the GPU with one CTA each.  The cluster kernel's
  // chain of cluster barriers takes about 17-21 us whatever the row count (measured: 32 rows
  // of 32736 in 21 us, 64 in 25 us, 128 in 45 us); the one-CTA kernel takes about 26-28 us for
  // any number of rows up to the SM count.
  const bool one_cta_fits = n <= FAST_MAX_KEYS && r <= 7;
  if ((!one_cta_fits || rows <= 48) && select_cluster_applies(rows, n, pool_kernel))
    return launch_pool_topk_cluster(vote, rows, n, pool_kernel, pool_type, ksel, out_idx, stream,
                                    launches, gsum);
  if (one_cta_fits) {
    const int ept = (((n + SEL_THREADS - 1) / SEL_THREADS) + 7) & ~7;
    const int words = key_slot4_host(SEL_THREADS * ept) + 4;
#define SNAPKV_FAST_LAUNCH(RM, P)                                                            \
  pool_topk_fast_kernel<RM, P><<<rows, SEL_THREADS, words * 4, stream>>>(vote, n, gsum, r,    \
                                                                        pool_type, ept, ksel, out_idx, \
                                                                        vote_is_scratch ? 1 : 0)
    // the paper's kernel sizes 5, 7 and 13 have instantiations of their own
    const bool mx = pool_type == 0;
    if (r == 2) { if (mx) SNAPKV_FAST_LAUNCH(2, 0); else SNAPKV_FAST_LAUNCH(2, 1); }
    else if (r == 3) { if (mx) SNAPKV_FAST_LAUNCH(3, 0); else SNAPKV_FAST_LAUNCH(3, 1); }
    else if (r == 6) { if (mx) SNAPKV_FAST_LAUNCH(6, 0); else SNAPKV_FAST_LAUNCH(6, 1); }
    else if (r <= 3) SNAPKV_FAST_LAUNCH(3, -1);
    else SNAPKV_FAST_LAUNCH(7, -1);
#undef SNAPKV_FAST_LAUNCH
    *launches += 1;
    return cudaGetLastError();
  }
  if (!select_needs_scratch(n)) {  // fits one CTA, but the radius is beyond the fast path
    pool_topk_kernel<<<rows, SEL_THREADS, static_cast<size_t>(n) * 4, stream>>>(
        vote, n, gsum, pool_kernel, pool_type, ksel, out_idx, nullptr);
    *launches += 1;
    return cudaGetLastError();
  }
  // long rows: many CTAs per row, state in global scratch
  WideBufs wb;
  uint8_t* p = reinterpret_cast<uint8_t*>(pooled_scratch);
  const size_t nr = static_cast<size_t>(rows);
  wb.nblk = wide_nblk(n);
  wb.keys = reinterpret_cast<uint32_t*>(p);
  p += up256(nr * n * 4);
  wb.hist = reinterpret_cast<int*>(p);
  p += up256(nr * NBINS * 4);
  wb.state = reinterpret_cast<int*>(p);
  p += up256(nr * 8 * 4);
  wb.counts = reinterpret_cast<int*>(p);
  cudaError_t e = cudaMemsetAsync(wb.hist, 0, up256(nr * NBINS * 4), stream);
  if (e != cudaSuccess) return e;
  const dim3 grid(wb.nblk, rows);
  wide_pool_kernel<<<grid, WIDE_THREADS, 0, stream>>>(vote, n, gsum, pool_kernel, pool_type, wb);
  // the seven kernels behind the first are launched with programmatic dependent launch:
  // each becomes resident while its predecessor runs and waits for it before its first read
  const dim3 one(rows), st(SEL_THREADS), wt(WIDE_THREADS);
  e = cudaGetLastError();
  if (e == cudaSuccess) e = launch_pdl(wide_pick_kernel, one, st, 0, stream, 0, ksel, wb);
  if (e == cudaSuccess) e = launch_pdl(wide_hist_kernel, grid, wt, 0, stream, n, 1, wb);
  if (e == cudaSuccess) e = launch_pdl(wide_pick_kernel, one, st, 0, stream, 1, ksel, wb);
  if (e == cudaSuccess) e = launch_pdl(wide_hist_kernel, grid, wt, 0, stream, n, 2, wb);
  if (e == cudaSuccess) e = launch_pdl(wide_pick_kernel, one, st, 0, stream, 2, ksel, wb);
  if (e == cudaSuccess) e = launch_pdl(wide_count_kernel, grid, wt, 0, stream, n, wb);
  if (e == cudaSuccess) e = launch_pdl(wide_write_kernel, grid, wt, 0, stream, n, ksel, out_idx, wb);
  if (e != cudaSuccess) return e;
  *launches += 8;
  return cudaGetLastError();
}

cudaError_t launch_iota_idx(int32_t* out_idx, int rows, int n, int row_stride, cudaStream_t stream,
                            int* launches) {
  if (n <= 0) return cudaSuccess;
  const long long total = static_cast<long long>(rows) * n;
  int blocks = static_cast<int>((total + 255) / 256 < 1184 ? (total + 255) / 256 : 1184);
  iota_kernel<<<blocks, 256, 0, stream>>>(out_idx, rows, n, row_stride);
  *launches += 1;
  return cudaGetLastError();
}

}  // namespace snapkv

// ---------------------------------------------------------------------------------------
// Pool + top-k for callers that cannot hand the library any scratch memory.
//
// The generic kernel above keeps one 32-bit key per vote in global memory.  Here that
// memory is a fixed array inside the library image instead of a caller buffer: 16 MiB that
// every GPU which loads libsnapkv.so holds until the process exits.
static __device__ __align__(256) uint32_t g_static_keys[SNAPKV_STATIC_MAX_KEYS];

namespace snapkv {
namespace {
constexpr int MAX_DEVICES = 64;
uint32_t* g_static_keys_addr[MAX_DEVICES] = {nullptr};

// The array's name is only a handle on the host; the device address has to be asked for,
// once per device, with that device current.
snapkv_status_t static_keys_address(uint32_t** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return SNAPKV_ERR_CUDA;
  if (g_static_keys_addr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_keys) != cudaSuccess || p == nullptr) return SNAPKV_ERR_CUDA;
    g_static_keys_addr[dev] = static_cast<uint32_t*>(p);
  }
  *out = g_static_keys_addr[dev];
  return SNAPKV_OK;
}
}  // namespace
}  // namespace snapkv

extern "C" snapkv_status_t snapkv_pool_topk_static(const float* vote, int rows, int n,
                                                   int pool_kernel, int pool_type, int ksel,
                                                   int32_t* out_idx, void* stream) {
  using namespace snapkv;
  if (rows < 1 || n < 1 || ksel < 1 || ksel > n || !vote || !out_idx) return SNAPKV_ERR_INVALID_ARG;
  if (pool_kernel < 1 || (pool_kernel & 1) == 0) return SNAPKV_ERR_INVALID_ARG;
  if (pool_type != SNAPKV_POOL_MAX && pool_type != SNAPKV_POOL_AVG) return SNAPKV_ERR_INVALID_ARG;
  if (pool_kernel > 63) return SNAPKV_ERR_UNSUPPORTED;
  // more keys than the built-in array holds: refuse before touching the device
  if (static_cast<long long>(rows) * n > static_cast<long long>(SNAPKV_STATIC_MAX_KEYS))
    return SNAPKV_ERR_WORKSPACE;
  uint32_t* keys = nullptr;
  const snapkv_status_t st = static_keys_address(&keys);
  if (st != SNAPKV_OK) return st;
  // Every key the kernel reads was written by the same launch, so nothing has to be
  // cleared between calls; whatever the previous call left behind is overwritten or unused.
  pool_topk_kernel<<<rows, SEL_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(
      vote, n, 1, pool_kernel, pool_type, ksel, out_idx, keys);
  return cudaGetLastError() == cudaSuccess ? SNAPKV_OK : SNAPKV_ERR_CUDA;
}
