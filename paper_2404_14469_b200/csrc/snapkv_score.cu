// Window scoring (Eq. 1; Listing 1's compute_attn and the sum over the window):
//   vote[h, j] = sum_i softmax_i(q_i . k / sqrt(d))[j],  j in [0, n)
// computed in two tensor-core passes over K inside ONE persistent kernel.
//
//  pass S (statistics)  S^T tile = Q_rep[128 x d] . K_tile[128 x d]^T : window rows on
//      TMEM lanes, keys on columns.  Each thread owns one window row and keeps a running
//      (max, sum of exp) over the keys it sees: an online softmax without shuffles.
//      When the unit has fewer than 128 window rows the rows are replicated along M and
//      each replica takes a different slice of the tile's keys, so all four epilogue
//      warps of a warpgroup stay busy.  Each CTA publishes one log2-sum-exp per window row
//      for the keys it saw (its "partial") and bumps the unit's counter.
//  pass V (votes)       S tile = K_tile[128 x d] . Q[ncols x d]^T : keys on TMEM lanes,
//      window rows on columns.  Once the unit's counter shows that every partial has been
//      published, the CTA folds them, in slot order, into one log2-sum-exp per window row;
//      then each thread owns one key and adds exp2(s*c - lse) over the W columns of each
//      head: the sum over the window is a serial add per thread.
//
// Units (batch, KV head, head sub-group) are grouped into waves small enough for L2; the
// kernel walks the phases  S(0), S(1), V(0), S(2), V(1), ...  so that the second sweep
// over a wave's keys is served by L2 and the partials a vote phase needs were published
// a whole phase earlier.  Within a phase the wave's tiles are split evenly over the CTAs.
// One CTA per SM and no more CTAs than SMs, so all of them are resident and waiting on
// another CTA's partials cannot starve it.
//
// Warp roles: warp 0 issues TMA loads (K tiles into a ring of stages, Q per work item
// into two buffers), warp 1 issues tcgen05.mma into four TMEM accumulator buffers, warps
// 2-9 (two warpgroups) read the accumulators back with tcgen05.ld and do the fp32 softmax
// arithmetic; with 64 or more query columns per unit a second set of eight softmax warps
// (12-19) takes every other tile, each warpgroup of a set working on half of the columns:
// the epilogue is bound by instruction latency, and four warps per scheduler hide it where
// two do not.  Warps 10 and 11 are the book-keepers: warp 10 publishes the partial
// statistics the softmax warps leave in shared memory, warp 11 fetches and folds the
// partials of the coming vote items' units while the softmax warps are still busy.  The single-thread roles (TMA and MMA issue) are entered through elect.sync:
// the compiler then keeps descriptors and addresses in uniform registers, which cut the
// time per tcgen05.mma issue by about a third against a lane-index test.
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "launch.cuh"
#include "sm100_ptx.cuh"
#include "snapkv_internal.h"

namespace snapkv {

namespace {

constexpr int STAGES = 4;
constexpr int NBUF = 4;               // TMEM accumulator buffers of 128 columns
constexpr int TMEM_COLS = 512;
constexpr int SUBTILE_BYTES = 128 * 128;  // 128 rows x 64 bf16, 128-byte swizzled
constexpr int EPI_WARPS = 8;           // softmax warps per set (two warpgroups)
// Warps: 0 producer, 1 MMA issuer, 2-9 softmax set 0, 10 publisher, 11 lse fetcher and, in
// split mode, 12-19 softmax set 1.
constexpr int threads_for(bool split) { return split ? 640 : 384; }
#ifndef WAVE_MIB
#define WAVE_MIB 64
#endif
#ifndef WAVE_LAG
#define WAVE_LAG 2
#endif
constexpr long long WAVE_BYTES = static_cast<long long>(WAVE_MIB) << 20;
constexpr int NPB = 2;                // buffers for partial statistics (book-keeper queue)
constexpr int NLB = 8;                // buffers for merged log-sum-exp rows
constexpr int MERGE_SEGS = 40;        // partials staged in shared memory per merge round

struct ScoreArgs {
  int L, n, W, Hkv;
  int hpu, ncols, npad;
  int sub_per_kv, g;
  int units, upw, nwaves;   // units per wave, number of waves
  int T1, T2;               // tiles per unit in the statistics / vote pass
  int maxseg;               // partial slots per unit
  int pipelined;            // how many waves the statistics run ahead of the votes (>= 1)
  int mask_n;               // window row i sees keys j <= mask_n + i (n, or n minus a shard's first position)
  int stats_only;           // 1: statistics pass alone (a shard's partial log-sum-exp), no votes
  int votes_only;           // 1: lse2 and the counters are already set, no statistics pass
  unsigned long long wait_ns;  // time limit of every device-side wait
  const int32_t* page_table;   // paged K: [batch][pages_per_seq] page numbers, else nullptr
  int pages_per_seq, page_size;
  float c2;                 // log2(e) / sqrt(d)
  float* partials;          // [units][maxseg][MAX_COLS] log2-sum-exp of one CTA's share
  float* lse2;              // [units][MAX_COLS] minus the log2-sum-exp per window row, when supplied
  int* counters;            // [units] published partials (a large value when lse2 was supplied)
  int* status;
  float* vote;
};

template <int D>
struct Smem {
  static constexpr int SUBT = D / 64;
  static constexpr int Q_BYTES = SUBT * SUBTILE_BYTES;
  static constexpr int STAGE_BYTES = SUBT * SUBTILE_BYTES;
  static constexpr int OFF_Q = 0;                            // two Q buffers
  static constexpr int OFF_K = 2 * Q_BYTES;
  static constexpr int OFF_BAR = OFF_K + STAGES * STAGE_BYTES;
  // barriers: full[STAGES], empty[STAGES], tf[NBUF], te[NBUF], qfull[2], qempty[2], drain,
  // pfull[NPB], pempty[NPB] (partial statistics), lfull[NLB], lempty[NLB] (log-sum-exp),
  // merge (bulk copy of a unit's partials)
  static constexpr int NBAR = 2 * STAGES + 2 * NBUF + 5 + 2 * NPB + 2 * NLB + 1;
  static constexpr int OFF_MISC = OFF_BAR + ((NBAR * 8 + 15) & ~15);  // tmem ptr, abort flag, wait limit
  static constexpr int OFF_PART = OFF_MISC + 16;              // float2 [NPB][2 sets][8][32]
  static constexpr int OFF_LSE = OFF_PART + NPB * 16 * 32 * 8; // float [NLB][128]
  static constexpr int OFF_MERGE = OFF_LSE + NLB * 128 * 4;   // float [MERGE_SEGS][128]
  static constexpr int TOTAL = OFF_MERGE + MERGE_SEGS * 128 * 4;
  static_assert(OFF_PART % 16 == 0 && OFF_LSE % 16 == 0 && OFF_MERGE % 16 == 0,
                "float4 reads of the lse buffers, bulk copies into the merge buffer");
  static constexpr int DYN_BYTES = TOTAL + 1024;            // slack for 1024-byte alignment
};

// Wait of the abort path (the abort flag is already set, so it is not looked at): for a copy
// or an MMA that is in flight and will complete.
__device__ __forceinline__ bool mbar_wait_drain(uint32_t bar, uint32_t parity,
                                                unsigned long long limit_ns) {
  const unsigned long long t0 = globaltimer_ns();
  for (;;) {
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (globaltimer_ns() - t0 > limit_ns) return false;
  }
}

// Warp-wide wait for a warp that is off the critical path: backs off between polls so
// that it does not take issue slots from the softmax warps of its scheduler.
__device__ __forceinline__ bool mbar_wait_warp_relaxed(uint32_t bar, uint32_t parity,
                                                       volatile int* abort_flag, int code) {
  if (__all_sync(0xffffffffu, mbar_try_wait(bar, parity))) return true;
  const unsigned long long t0 = globaltimer_ns();
  for (;;) {
    __nanosleep(250);
    if (__all_sync(0xffffffffu, mbar_try_wait(bar, parity))) return true;
    int stop = 0;
    if ((threadIdx.x & 31) == 0) {
      if (*abort_flag != 0) stop = 1;
      else if (globaltimer_ns() - t0 > wait_limit_ns(abort_flag)) { *abort_flag = code; stop = 1; }
    }
    if (__shfl_sync(0xffffffffu, stop, 0)) return false;
  }
}

__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// One piece of work: tiles [t0, t1) of one unit in one pass.
struct Item {
  int unit, t0, t1, vote, slot, nseg;
};

// The work items of CTA `cr` in one phase: the phase's TT = nu * T tiles (units u0 .. u0+nu-1,
// T tiles each) are cut into G consecutive shares, CTA c owning tiles [c*TT/G, (c+1)*TT/G); a
// share that crosses a unit boundary is one item per unit.  I is the integer type of the tile
// arithmetic: every warp of a CTA walks the list, at every item, so the divisions are done in
// 32 bits whenever the products fit (64-bit divisions cost about 0.1 us each here).
template <typename I, typename F>
__host__ __device__ __forceinline__ bool phase_items(const ScoreArgs& a, int cr, int G, int u0,
                                                     int nu, int T, int vote, F&& f) {
  const I g = static_cast<I>(G);
  const I TT = static_cast<I>(nu) * static_cast<I>(T);
  const I lo = static_cast<I>(cr) * TT / g, hi = static_cast<I>(cr + 1) * TT / g;
  // where this CTA's partial of a unit goes and how many partials the unit gets follow from
  // the statistics-pass partition of the unit's wave (TT1 tiles)
  const I T1 = static_cast<I>(a.T1);
  const I TT1 = static_cast<I>(nu) * T1;
  // the CTA whose share contains tile x: the largest c with c*TT1/G <= x
  auto cta_of_tile = [&](I x) { return static_cast<int>(((x + 1) * g + TT1 - 1) / TT1) - 1; };
  for (I pos = lo; pos < hi;) {
    const I ul = pos / static_cast<I>(T);
    Item it;
    it.unit = u0 + static_cast<int>(ul);
    it.t0 = static_cast<int>(pos - ul * static_cast<I>(T));
    const I t1 = static_cast<I>(it.t0) + (hi - pos);
    it.t1 = t1 < static_cast<I>(T) ? static_cast<int>(t1) : T;
    it.vote = vote;
    if (TT1 >= g) {  // every CTA has tiles: a unit's owners are consecutive CTAs
      const int cfirst = cta_of_tile(ul * T1);
      const int clast = cta_of_tile((ul + 1) * T1 - 1);
      it.slot = cr - cfirst;
      it.nseg = clast - cfirst + 1;
    } else {         // fewer tiles than CTAs: one tile per owner, one partial per tile
      it.slot = it.t0;
      it.nseg = a.T1;
    }
    pos += static_cast<I>(it.t1 - it.t0);
    if (!f(it)) return false;
  }
  return true;
}

// Calls f(item) for every work item of this CTA in schedule order; stops when f
// returns false.  All warp roles walk the same list.
template <typename F>
__host__ __device__ __forceinline__ void for_each_item(const ScoreArgs& a, int cta, int G, int lag,
                                                       F&& f) {
  // Phase order: statistics run `lag` waves ahead of votes: S(0) .. S(lag-1) V(0) S(lag)
  // V(1) ...; lag = 1 is the plain order S(0) V(0) S(1) V(1) ...
  int s_next = a.votes_only ? a.nwaves : 0, v_next = a.stats_only ? a.nwaves : 0;
  while (v_next < a.nwaves || s_next < a.nwaves) {
    int w, vote;
    if (s_next < a.nwaves && (v_next >= a.nwaves || s_next - v_next < lag)) { w = s_next++; vote = 0; }
    else { w = v_next++; vote = 1; }
    const int u0 = w * a.upw;
    const int nu = a.upw < a.units - u0 ? a.upw : a.units - u0;
    const int T = vote ? a.T2 : a.T1;
    // TT is seldom a multiple of G, so some CTAs get one tile less than the others; which
    // ones moves on by one CTA from phase to phase, so that over the phases of a launch no
    // CTA carries the longer share every time
    const int cr = (cta + 2 * w + vote) % G;
    const long long tmax = static_cast<long long>(nu) * (a.T1 > T ? a.T1 : T);
    const bool fits32 = (tmax + 1) * (G + 1) < (1ll << 32);
    const bool go_on = fits32 ? phase_items<uint32_t>(a, cr, G, u0, nu, T, vote, f)
                              : phase_items<unsigned long long>(a, cr, G, u0, nu, T, vote, f);
    if (!go_on) return;
  }
}

// NCH = npad / 32: how many 32-column chunks of the accumulator a thread reads per tile.
template <int D, int NCH, bool SPLIT>
__global__ void __launch_bounds__(threads_for(SPLIT), 1)
score_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmQ,
             const ScoreArgs a) {
  pdl_launch_dependents();
  using SM = Smem<D>;
  constexpr int SUBT = SM::SUBT;
  constexpr int NPAD = NCH * 32;
  constexpr int REPS = 128 / NPAD;
  constexpr int NSET = SPLIT ? 2 : 1;  // sets of softmax warps
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  const uint32_t sbase = smem_u32(smem);
  const uint32_t k_s = sbase + SM::OFF_K;
  const uint32_t bar0 = sbase + SM::OFF_BAR;
  auto q_s = [&](int b) { return sbase + SM::OFF_Q + b * SM::Q_BYTES; };
  // Stages 2p and 2p+1 interleave so that each 64-element half of the head dimension is one
  // 256-row tile across the pair: [half 0: stage 2p rows, stage 2p+1 rows][half 1: ...].
  auto stage_addr = [&](int s, int sb) {
    return k_s + (s >> 1) * (2 * SM::STAGE_BYTES) + sb * (2 * SUBTILE_BYTES) + (s & 1) * SUBTILE_BYTES;
  };
  auto bar_full = [&](int s) { return bar0 + 8u * s; };
  auto bar_empty = [&](int s) { return bar0 + 8u * (STAGES + s); };
  auto bar_tf = [&](int b) { return bar0 + 8u * (2 * STAGES + b); };
  auto bar_te = [&](int b) { return bar0 + 8u * (2 * STAGES + NBUF + b); };
  auto bar_qf = [&](int b) { return bar0 + 8u * (2 * STAGES + 2 * NBUF + b); };
  auto bar_qe = [&](int b) { return bar0 + 8u * (2 * STAGES + 2 * NBUF + 2 + b); };
  const uint32_t bar_drain = bar0 + 8u * (2 * STAGES + 2 * NBUF + 4);
  constexpr int BAR_P = 2 * STAGES + 2 * NBUF + 5;
  auto bar_pf = [&](int b) { return bar0 + 8u * (BAR_P + b); };
  auto bar_pe = [&](int b) { return bar0 + 8u * (BAR_P + NPB + b); };
  auto bar_lf = [&](int b) { return bar0 + 8u * (BAR_P + 2 * NPB + b); };
  auto bar_le = [&](int b) { return bar0 + 8u * (BAR_P + 2 * NPB + NLB + b); };
  const uint32_t bar_merge = bar0 + 8u * (BAR_P + 2 * NPB + 2 * NLB);
  volatile uint32_t* tmem_ptr_s = reinterpret_cast<volatile uint32_t*>(smem + SM::OFF_MISC);
  volatile int* abort_s = reinterpret_cast<volatile int*>(smem + SM::OFF_MISC + 4);
  float2* part_s = reinterpret_cast<float2*>(smem + SM::OFF_PART);
  float* lse_s = reinterpret_cast<float*>(smem + SM::OFF_LSE);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int cta = blockIdx.x;
  const int G = gridDim.x;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(bar_full(s), 1);
      mbar_init(bar_empty(s), 1);
    }
    for (int b = 0; b < NBUF; ++b) {
      mbar_init(bar_tf(b), 1);
      mbar_init(bar_te(b), EPI_WARPS);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_qf(b), 1);
      mbar_init(bar_qe(b), 1);
    }
    for (int b = 0; b < NPB; ++b) {
      mbar_init(bar_pf(b), EPI_WARPS * NSET);
      mbar_init(bar_pe(b), 1);
    }
    for (int b = 0; b < NLB; ++b) {
      mbar_init(bar_lf(b), 1);
      mbar_init(bar_le(b), EPI_WARPS * NSET);
    }
    mbar_init(bar_drain, 1);
    mbar_init(bar_merge, 1);
    *abort_s = 0;
    *reinterpret_cast<volatile unsigned long long*>(abort_s + 1) = a.wait_ns;
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_ptr_s)), TMEM_COLS);
    tmem_relinquish();
  }
  // everything above touched only this CTA's shared memory and TMEM; from here on the
  // kernel reads and writes global memory, so the previous kernel must be complete
  pdl_wait();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_ptr_s;

  // tile visited at step k of an item: ascending, except that the sequential schedule
  // sweeps the vote pass backwards (the keys read last are the likeliest to be in L2)
  auto tile_of = [&](const Item& it, int k) {
    return (it.vote && a.pipelined == 1) ? (it.t1 - 1 - k) : (it.t0 + k);
  };
  auto first_head = [&](int unit, int* ukv) {
    *ukv = unit / a.sub_per_kv;
    return *ukv * a.g + (unit - *ukv * a.sub_per_kv) * a.hpu;  // flat over the batch
  };

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (elect_one()) {
      tma_prefetch_desc(&tmK);
      tma_prefetch_desc(&tmQ);
      const uint64_t pol_first = l2_policy_evict_first();
      int git = 0;      // tiles issued so far (ring position)
      int nitem = 0;    // items started so far (Q buffer position)
      for_each_item(a, cta, G, a.pipelined, [&](const Item& it) {
        int ukv;
        const int qrow0 = first_head(it.unit, &ukv) * a.W;
        const int qb = nitem & 1;
        if (!mbar_wait_thread(bar_qe(qb), ((nitem >> 1) & 1) ^ 1, abort_s, WAIT_Q_FULL)) return false;
        if (it.vote) {
          mbar_expect_tx(bar_qf(qb), SUBT * NPAD * 128);
          for (int sb = 0; sb < SUBT; ++sb)
            tma_load_2d(q_s(qb) + sb * SUBTILE_BYTES, &tmQ, bar_qf(qb), sb * 64, qrow0);
        } else {
          mbar_expect_tx(bar_qf(qb), SUBT * 128 * 128);
          for (int rep = 0; rep < REPS; ++rep)
            for (int sb = 0; sb < SUBT; ++sb)
              tma_load_2d(q_s(qb) + sb * SUBTILE_BYTES + rep * NPAD * 128, &tmQ, bar_qf(qb),
                          sb * 64, qrow0);
        }
        ++nitem;
        const int kb = ukv / a.Hkv, kh = ukv - kb * a.Hkv;  // the K map is (d, L, Hkv, B)
        const int nt = it.t1 - it.t0;
        for (int k = 0; k < nt; ++k, ++git) {
          const int s = git % STAGES;
          const uint32_t ph = (git / STAGES) & 1;
          if (!mbar_wait_thread(bar_empty(s), ph ^ 1, abort_s, WAIT_PRODUCER_EMPTY)) return false;
          mbar_expect_tx(bar_full(s), SM::STAGE_BYTES);
          int key0 = tile_of(it, k) * TILE_KEYS;
          int kslab = kb;  // outermost coordinate of the K map: the batch, or the page of the pool
          if (a.page_table) {
            // a page holds a whole number of tiles: the tile's 128 keys sit in one page
            const int pg = key0 / a.page_size;
            kslab = __ldg(a.page_table + static_cast<size_t>(kb) * a.pages_per_seq + pg);
            key0 -= pg * a.page_size;
          }
          // the vote pass is the last reader of a key tile: its lines may leave L2 first,
          // which keeps the next wave's statistics-pass lines resident instead
          for (int sb = 0; sb < SUBT; ++sb) {
            if (it.vote)
              tma_load_4d_hint(stage_addr(s, sb), &tmK, bar_full(s), sb * 64, key0, kh, kslab, pol_first);
            else
              tma_load_4d(stage_addr(s, sb), &tmK, bar_full(s), sb * 64, key0, kh, kslab);
          }
        }
        return true;
      });
      if (*abort_s != 0) {
        // let every copy in flight land before the CTA's shared memory goes away
        for (int b = 0; b < 2; ++b) {
          int last = -1;
          for (int i = b; i < nitem; i += 2) last = i;
          if (last >= 0) mbar_wait_drain(bar_qf(b), (last >> 1) & 1, a.wait_ns);
        }
        for (int s = 0; s < STAGES; ++s) {
          int last = -1;
          for (int i = s; i < git; i += STAGES) last = i;
          if (last >= 0) mbar_wait_drain(bar_full(s), (last / STAGES) & 1, a.wait_ns);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    // The tensor pipe takes about as long for a 128 x N x 16 instruction with N <= 128 as
    // for N = 256, so the statistics pass (keys on N) covers two key tiles per instruction
    // whenever two tiles of an item sit in an aligned pair of stages: their accumulators
    // are adjacent 128-column TMEM buffers, so the softmax warps see two ordinary tiles.
    if (elect_one()) {
      const uint32_t idesc_s = umma_idesc_bf16(128, 128);
      const uint32_t idesc_s2 = umma_idesc_bf16(128, 256);
      const uint32_t idesc_v = umma_idesc_bf16(128, NPAD);
      int git = 0, nitem = 0;
      for_each_item(a, cta, G, a.pipelined, [&](const Item& it) {
        const int qb = nitem & 1;
        if (!mbar_wait_thread(bar_qf(qb), (nitem >> 1) & 1, abort_s, WAIT_Q_FULL)) return false;
        ++nitem;
        const uint64_t qd0 = umma_desc_k128(q_s(qb));
        const int nt = it.t1 - it.t0;
        for (int k = 0; k < nt;) {
          const int s = git % STAGES;
          const uint32_t ph = (git / STAGES) & 1;
          const int buf = git & (NBUF - 1);
          const uint32_t ub = (git / NBUF) & 1;
          const bool pair = !it.vote && (git & 1) == 0 && k + 1 < nt;
          if (!mbar_wait_thread(bar_full(s), ph, abort_s, WAIT_MMA_FULL)) return false;
          if (!mbar_wait_thread(bar_te(buf), ub ^ 1, abort_s, WAIT_MMA_TMEM_EMPTY)) return false;
          if (pair) {  // stage s + 1 and buffer buf + 1 are in the same round of their rings
            if (!mbar_wait_thread(bar_full(s + 1), ph, abort_s, WAIT_MMA_FULL)) return false;
            if (!mbar_wait_thread(bar_te(buf + 1), ub ^ 1, abort_s, WAIT_MMA_TMEM_EMPTY)) return false;
          }
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + buf * 128;
          // One descriptor per operand and tile; the eight K-slices of the tile differ from it
          // by constants (the start-address field counts 16-byte units and the operands sit
          // below 256 KB, so adding to the low word never carries into another field).  The
          // issuing thread is a single in-order instruction stream: every instruction saved
          // per tcgen05.mma shortens the time between two of them.
          const uint64_t kd0 = umma_desc_k128(stage_addr(s, 0));
          constexpr uint64_t K_SB = (2 * SUBTILE_BYTES) >> 4;  // next 64 elements of d (stage pairs interleave)
          constexpr uint64_t Q_SB = SUBTILE_BYTES >> 4;
          if (it.vote) {
#pragma unroll
            for (int sb = 0; sb < SUBT; ++sb)
#pragma unroll
              for (int kk = 0; kk < 4; ++kk)
                tc_mma_bf16(d_tmem, kd0 + (sb * K_SB + kk * 2), qd0 + (sb * Q_SB + kk * 2), idesc_v,
                            (sb | kk) != 0);
          } else {
            const uint32_t idesc = pair ? idesc_s2 : idesc_s;
#pragma unroll
            for (int sb = 0; sb < SUBT; ++sb)
#pragma unroll
              for (int kk = 0; kk < 4; ++kk)
                tc_mma_bf16(d_tmem, qd0 + (sb * Q_SB + kk * 2), kd0 + (sb * K_SB + kk * 2), idesc,
                            (sb | kk) != 0);
          }
          tc_commit(bar_empty(s));
          if (pair) tc_commit(bar_empty(s + 1));
          tc_commit(bar_tf(buf));
          if (pair) tc_commit(bar_tf(buf + 1));
          const int step = pair ? 2 : 1;
          k += step;
          git += step;
        }
        tc_commit(bar_qe(qb));  // the item's MMAs are the last readers of its Q buffer
        return true;
      });
      if (*abort_s != 0) {
        tc_commit(bar_drain);
        mbar_wait_drain(bar_drain, 0, a.wait_ns);
      }
    }
  } else if (warp < 2 + EPI_WARPS || warp >= 4 + EPI_WARPS) {
    // ------------------------------------------------------------ softmax warps
    // SPLIT: both warpgroups work on every tile, each on half of the accumulator columns
    // (CPT columns per thread); the -lse values of a vote item then fit in registers.
    // Otherwise the warpgroups alternate tiles and take all NPAD columns.
    constexpr int CPT = SPLIT ? NPAD / 2 : NPAD;
    constexpr int VCH = CPT / 32;
    // SPLIT also has two sets of softmax warps: set 0 takes the even tiles (by ring position)
    // and set 1 the odd ones, so four warps per scheduler hide each other's latencies.
    const int set = warp >= 4 + EPI_WARPS ? 1 : 0;
    const int wg = ((set ? warp - (4 + EPI_WARPS) : warp - 2) >> 2);
    const int q = warp & 3;  // TMEM lane quarter this warp may read
    const uint32_t lane_sel = static_cast<uint32_t>(32 * q) << 16;
    const int rrow = 32 * q + lane;  // TMEM lane
    const int rep = rrow / NPAD;
    const int qcol = rrow - rep * NPAD;
    const int jmax = min(a.L - 1, a.mask_n + (qcol % a.W));  // last key window row qcol % W sees
    const int jfree = min(a.L - 1, a.mask_n);  // keys up to here are seen by every row
    const int coff = SPLIT ? wg * CPT : 0;               // first accumulator column of this thread
    const bool w16 = (a.W & 15) == 0;
    const int gpw = a.W >> 4;  // 16-column groups per head (when W is a multiple of 16)
    const uint32_t te_arrivals = SPLIT ? 1 : 2;          // the barrier expects 8 per tile
    int git = 0, nstat = 0, nvote = 0;
    for_each_item(a, cta, G, a.pipelined, [&](const Item& it) {
      const int nt = it.t1 - it.t0;
      int ukv;
      const int hq0 = first_head(it.unit, &ukv);
      if (!it.vote) {
        // ---------------------------------------------------------- statistics
        float m2 = -INFINITY;  // running max, log2 domain
        float l = 0.f;         // running sum of exp2(x - m2)
        for (int k = 0; k < nt; ++k, ++git) {
          if ((git & 1) != (SPLIT ? set : wg)) continue;
          const int buf = git & (NBUF - 1);
          const uint32_t ub = (git / NBUF) & 1;
          if (!mbar_wait_warp(bar_tf(buf), ub, abort_s, WAIT_EPI_TMEM_FULL)) return false;
          tc_fence_after();
          const int key0 = tile_of(it, k) * TILE_KEYS;
          // this thread's slice of its window row: CPT key columns
          float v[VCH][32];
          const uint32_t taddr = tmem_base + lane_sel + buf * 128 + rep * NPAD + coff;
#pragma unroll
          for (int ch = 0; ch < VCH; ++ch) tmem_ld32(taddr + ch * 32, v[ch]);
          tmem_wait_ld();
          // the accumulator is in registers now: hand the buffer back to the MMA warp
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_n(bar_te(buf), te_arrivals);
          if (key0 + TILE_KEYS - 1 > jfree) {  // tile touches the window or the end of the keys
            const int kb = key0 + rep * NPAD + coff;
#pragma unroll
            for (int ch = 0; ch < VCH; ++ch)
#pragma unroll
              for (int c = 0; c < 32; ++c)
                v[ch][c] = (kb + ch * 32 + c <= jmax) ? v[ch][c] : -INFINITY;
          }
          float c0 = v[0][0], c1 = v[0][1], c2m = v[0][2], c3 = v[0][3];
#pragma unroll
          for (int ch = 0; ch < VCH; ++ch)
#pragma unroll
            for (int c = (ch == 0 ? 4 : 0); c < 32; c += 4) {
              c0 = fmaxf(c0, v[ch][c + 0]);
              c1 = fmaxf(c1, v[ch][c + 1]);
              c2m = fmaxf(c2m, v[ch][c + 2]);
              c3 = fmaxf(c3, v[ch][c + 3]);
            }
          const float cmax = fmaxf(fmaxf(c0, c1), fmaxf(c2m, c3));
          const float mnew = fmaxf(fmaxf(cmax * a.c2, m2), -1e30f);
          l *= ex2_approx(m2 - mnew);
          float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
          for (int ch = 0; ch < VCH; ++ch)
#pragma unroll
            for (int c = 0; c < 32; c += 4) {
              s0 += ex2_approx(fmaf(v[ch][c + 0], a.c2, -mnew));
              s1 += ex2_approx(fmaf(v[ch][c + 1], a.c2, -mnew));
              s2 += ex2_approx(fmaf(v[ch][c + 2], a.c2, -mnew));
              s3 += ex2_approx(fmaf(v[ch][c + 3], a.c2, -mnew));
            }
          l += (s0 + s1) + (s2 + s3);
          m2 = mnew;
        }
        // leave this warp's (max, sum) per TMEM lane for the book-keeper
        const int pb = nstat % NPB;
        if (!mbar_wait_warp(bar_pe(pb), ((nstat / NPB) & 1) ^ 1, abort_s, WAIT_PART_EMPTY))
          return false;
        part_s[((pb * 2 + set) * 8 + wg * 4 + q) * 32 + lane] = make_float2(m2, l);
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_pf(pb));
        ++nstat;
        return true;
      }
      // ------------------------------------------------------------ votes
      const int lb = nvote % NLB;
      if (!mbar_wait_warp(bar_lf(lb), (nvote / NLB) & 1, abort_s, WAIT_LSE_FULL)) return false;
      const float* lse_b = lse_s + lb * MAX_COLS;
      for (int k = 0; k < nt; ++k, ++git) {
        if ((git & 1) != (SPLIT ? set : wg)) continue;
        const int buf = git & (NBUF - 1);
        const uint32_t ub = (git / NBUF) & 1;
        if (!mbar_wait_warp(bar_tf(buf), ub, abort_s, WAIT_EPI_TMEM_FULL)) return false;
        tc_fence_after();
        const int j = tile_of(it, k) * TILE_KEYS + 32 * q + lane;
        const uint32_t taddr = tmem_base + lane_sel + buf * 128 + coff;
        float g16[VCH * 2];
        float v[SPLIT ? 1 : VCH][32];
        if (!SPLIT) {
#pragma unroll
          for (int ch = 0; ch < VCH; ++ch) tmem_ld32(taddr + ch * 32, v[ch]);
          tmem_wait_ld();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_n(bar_te(buf), te_arrivals);
        }
        if (SPLIT || w16) {
#pragma unroll
          for (int ch = 0; ch < VCH; ++ch) {
            if (SPLIT) {
              tmem_ld32(taddr + ch * 32, v[0]);
              tmem_wait_ld();
              if (ch == VCH - 1) {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_n(bar_te(buf), te_arrivals);
              }
            }
            const float(&vc)[32] = v[SPLIT ? 0 : ch];
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
              float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
              for (int t4 = 0; t4 < 4; ++t4) {
                // -lse of four adjacent columns: one broadcast read for the whole warp
                const float4 z =
                    *reinterpret_cast<const float4*>(lse_b + coff + ch * 32 + hf * 16 + 4 * t4);
                a0 += ex2_approx(fmaf(vc[hf * 16 + 4 * t4 + 0], a.c2, z.x));
                a1 += ex2_approx(fmaf(vc[hf * 16 + 4 * t4 + 1], a.c2, z.y));
                a2 += ex2_approx(fmaf(vc[hf * 16 + 4 * t4 + 2], a.c2, z.z));
                a3 += ex2_approx(fmaf(vc[hf * 16 + 4 * t4 + 3], a.c2, z.w));
              }
              g16[ch * 2 + hf] = (a0 + a1) + (a2 + a3);
            }
          }
          int hl = coff / a.W, left = gpw;  // SPLIT: coff is a multiple of W
          float acc = 0.f;
#pragma unroll
          for (int gi = 0; gi < VCH * 2; ++gi) {
            acc += g16[gi];
            if (--left == 0) {
              if (hl < a.hpu && j < a.n) a.vote[static_cast<size_t>(hq0 + hl) * a.n + j] = acc;
              acc = 0.f;
              left = gpw;
              ++hl;
            }
          }
        } else {
          int hl = 0, left = a.W;
          float acc = 0.f;
#pragma unroll
          for (int ch = 0; ch < VCH; ++ch)
#pragma unroll
            for (int c = 0; c < 32; ++c) {
              const int col = ch * 32 + c;
              if (col < a.ncols) {
                acc += ex2_approx(fmaf(v[ch][c], a.c2, lse_b[col]));
                if (--left == 0) {
                  if (j < a.n) a.vote[static_cast<size_t>(hq0 + hl) * a.n + j] = acc;
                  acc = 0.f;
                  left = a.W;
                  ++hl;
                }
              }
            }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_le(lb));  // this warp is done reading lse_s[lb]
      ++nvote;
      return true;
    });
  } else {
    // ------------------------------------------------------------ book-keeper warps
    // Warp 10 publishes this CTA's statistics partials; warp 11 fetches the unit's partials
    // for every vote item and folds them into the log-sum-exp row the item needs.  Each
    // walks its own kind of item in schedule order, so publishing never waits for another
    // CTA and the fetcher runs as far ahead as its shared-memory buffers allow.
    const bool publisher = warp == 2 + EPI_WARPS;  // warp 10; warp 11 is the fetcher
    int nstat = 0, nvote = 0, nmerge = 0;
    const float* merge_s = reinterpret_cast<const float*>(smem + SM::OFF_MERGE);
    for_each_item(a, cta, G, /*lag=*/1, [&](const Item& it) {
      if ((it.vote != 0) == publisher) return true;  // the other warp's kind of item
      if (!it.vote) {
        // merge the replicas and the two warpgroups (fixed order), publish, count
        const int pb = nstat % NPB;
        if (!mbar_wait_warp_relaxed(bar_pf(pb), (nstat / NPB) & 1, abort_s, WAIT_PART_FULL))
          return false;
        const float2* ps = part_s + pb * 16 * 32;
        for (int c = lane; c < a.ncols; c += 32) {
          float M = -INFINITY;
          for (int w2 = 0; w2 < 2 * NSET; ++w2)
            for (int r = 0; r < REPS; ++r) {
              const int row = r * NPAD + c;
              M = fmaxf(M, ps[(w2 * 4 + (row >> 5)) * 32 + (row & 31)].x);
            }
          M = fmaxf(M, -1e30f);
          float S = 0.f;
          for (int w2 = 0; w2 < 2 * NSET; ++w2)
            for (int r = 0; r < REPS; ++r) {
              const int row = r * NPAD + c;
              const float2 p = ps[(w2 * 4 + (row >> 5)) * 32 + (row & 31)];
              S += p.y * ex2_approx(p.x - M);
            }
          // log2 of this CTA's share of the row's softmax normaliser (-inf if it saw no key)
          a.partials[(static_cast<size_t>(it.unit) * a.maxseg + it.slot) * MAX_COLS + c] =
              M + log2f(S);
        }
        // release: the partial is visible to whoever sees the count
        __threadfence();
        __syncwarp();
        if (lane == 0) {
          atomicAdd(a.counters + it.unit, 1);
          mbar_arrive(bar_pe(pb));
        }
        ++nstat;
        return true;
      }
      // Fetcher.  A vote item needs minus the log2-sum-exp of every window row of its unit.
      // With a supplied normaliser that row is in global memory already.  Otherwise it is
      // the fold of the unit's partials: as soon as the unit's count says that all of them
      // are published (bounded wait), this warp pulls them into shared memory with bulk
      // copies (they are contiguous, 512 bytes each) and folds them in slot order, the same
      // order in every CTA and every run, so all CTAs get bit-identical rows without a
      // second hand-over through global memory.
      const int lb = nvote % NLB;
      const int ready = a.votes_only ? 0 : it.nseg - 1;  // count must exceed this
      int stop = 0;
      if (lane == 0 && ld_acquire(a.counters + it.unit) <= ready) {
        const unsigned long long t0 = globaltimer_ns();
        for (;;) {
          if (ld_acquire(a.counters + it.unit) > ready) break;
          if (*abort_s != 0) { stop = 1; break; }
          // half the limit: the roles of this CTA that wait for this row then still see the
          // abort flag, not their own time-out, and the status names the wait that failed
          if (globaltimer_ns() - t0 > a.wait_ns / 2) { *abort_s = WAIT_UNIT_STATS; stop = 1; break; }
          __nanosleep(100);
        }
      }
      if (__shfl_sync(0xffffffffu, stop, 0)) return false;
      (void)ld_acquire(a.counters + it.unit);  // every lane orders its reads after the count
      const int c4 = lane * 4;
      float4 val = make_float4(0.f, 0.f, 0.f, 0.f);
      if (a.votes_only) {
        if (c4 < a.ncols)
          val = __ldcg(reinterpret_cast<const float4*>(a.lse2 + static_cast<size_t>(it.unit) * MAX_COLS + c4));
      } else {
        fence_proxy_async();
        const float* pp = a.partials + static_cast<size_t>(it.unit) * a.maxseg * MAX_COLS;
        float M[4], S[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) { M[t] = -INFINITY; S[t] = 0.f; }
        for (int s0 = 0; s0 < it.nseg; s0 += MERGE_SEGS, ++nmerge) {
          const int ns = min(MERGE_SEGS, it.nseg - s0);
          if (lane == 0) {
            mbar_expect_tx(bar_merge, ns * MAX_COLS * 4);
            bulk_load(sbase + SM::OFF_MERGE, pp + static_cast<size_t>(s0) * MAX_COLS,
                      ns * MAX_COLS * 4, bar_merge);
          }
          if (!mbar_wait_warp_relaxed(bar_merge, nmerge & 1, abort_s, WAIT_MERGE_COPY)) {
            mbar_wait_drain(bar_merge, nmerge & 1, a.wait_ns);  // never leave with the copy in flight
            return false;
          }
          if (c4 < a.ncols) {
            for (int sg = 0; sg < ns; ++sg) {
              const float4 x = *reinterpret_cast<const float4*>(merge_s + sg * MAX_COLS + c4);
              const float pv[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
              for (int t = 0; t < 4; ++t) {
                const float Mn = fmaxf(fmaxf(M[t], pv[t]), -1e30f);
                S[t] = S[t] * ex2_approx(M[t] - Mn) + ex2_approx(pv[t] - Mn);
                M[t] = Mn;
              }
            }
          }
          __syncwarp();  // all lanes are done with the buffer before the next copy lands
        }
        if (c4 < a.ncols) {
          val.x = -(M[0] + log2f(S[0]));
          val.y = -(M[1] + log2f(S[1]));
          val.z = -(M[2] + log2f(S[2]));
          val.w = -(M[3] + log2f(S[3]));
        }
      }
      // the softmax warps must be done with this buffer's previous row
      if (!mbar_wait_warp_relaxed(bar_le(lb), ((nvote / NLB) & 1) ^ 1, abort_s, WAIT_LSE_EMPTY))
        return false;
      *reinterpret_cast<float4*>(lse_s + lb * MAX_COLS + c4) = val;
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_lf(lb));
      ++nvote;
      return true;
    });
  }

  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_s != 0) {
    if (atomicCAS(a.status, 0, 5 /* SNAPKV_ERR_TIMEOUT */) == 0) a.status[1] = *abort_s;
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) ==
            cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

bool encode_map(CUtensorMap* m, const void* base, int rank, const cuuint64_t* dims,
                const cuuint64_t* strides_bytes, const cuuint32_t* box) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank, const_cast<void*>(base), dims,
            strides_bytes, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int sm_count() {
  static int cached[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SM_COUNT_HINT;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1)
      n = SM_COUNT_HINT;
    cached[dev] = n;
  }
  return cached[dev];
}

// Supplied-normaliser variant: the caller hands in each window row's natural-log sum-exp
// (what a prefill attention kernel keeps per query row).  This kernel puts it where the vote
// pass expects the merged statistics - minus the log2-sum-exp, one row of MAX_COLS per unit -
// and marks every unit as merged, so the scoring kernel runs its vote phases only.
constexpr int COUNTER_READY = 1 << 30;
__global__ void lse_prep_kernel(const float* __restrict__ lse_obs, float* __restrict__ lse2,
                                int* __restrict__ counters, int* __restrict__ status,
                                int keep_status, int units, int sub_per_kv, int g, int hpu, int W,
                                int ncols) {
  pdl_launch_dependents();
  pdl_wait();
  const int u = blockIdx.x, c = threadIdx.x;  // one block per unit, one thread per column
  // this kernel stands in for the clear kernel of the two-sweep path: the status block too,
  // unless an earlier part of the same logical call may have left an error there
  if (u == 0 && c < STATUS_BYTES / 4 && !keep_status) status[c] = 0;
  if (u >= units || c >= MAX_COLS) return;
  const int ukv = u / sub_per_kv;
  const int hq0 = ukv * g + (u - ukv * sub_per_kv) * hpu;  // flat over the batch
  float out = 0.f;
  if (c < ncols) {
    const int hl = c / W, i = c - hl * W;
    out = -lse_obs[static_cast<size_t>(hq0 + hl) * W + i] * 1.4426950408889634f;
  }
  lse2[static_cast<size_t>(u) * MAX_COLS + c] = out;
  if (c == 0) counters[u] = COUNTER_READY;
}

// After a statistics-only launch: folds every unit's partials, in slot order as the vote sweep
// would, into one natural-log sum-exp per window row (counters[u] is the number of partials the
// unit got).  One block per unit, one thread per window column.
__global__ void lse_finish_kernel(const float* __restrict__ partials, const int* __restrict__ counters,
                                  float* __restrict__ lse_out, int units, int maxseg, int sub_per_kv,
                                  int g, int hpu, int W, int ncols) {
  const int u = blockIdx.x, c = threadIdx.x;
  if (u >= units || c >= ncols) return;
  const int nseg = counters[u];
  const float* pp = partials + static_cast<size_t>(u) * maxseg * MAX_COLS + c;
  float M = -INFINITY, S = 0.f;
  for (int sg = 0; sg < nseg; ++sg) {
    const float pv = pp[static_cast<size_t>(sg) * MAX_COLS];
    const float Mn = fmaxf(fmaxf(M, pv), -1e30f);
    S = S * ex2_approx(M - Mn) + ex2_approx(pv - Mn);
    M = Mn;
  }
  const int ukv = u / sub_per_kv;
  const int hq0 = ukv * g + (u - ukv * sub_per_kv) * hpu;
  const int hl = c / W, i = c - hl * W;
  // log2 -> natural log; a row that saw no key of this shard has S = 0: log gives -inf
  lse_out[static_cast<size_t>(hq0 + hl) * W + i] = (M + log2f(S)) * 0.6931471805599453f;
}

template <int D, int NCH, bool SPLIT>
cudaError_t run_scores(const CUtensorMap& tmK, const CUtensorMap& tmQ, const ScoreArgs& a,
                       int grid, cudaStream_t stream, int* launches) {
  static DeviceOnce once;  // one flag set per instantiation: the attribute is per function and device
  if (!once.done()) {
    cudaError_t e = cudaFuncSetAttribute(score_kernel<D, NCH, SPLIT>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         Smem<D>::DYN_BYTES);
    if (e != cudaSuccess) return e;
    once.set();
  }
  // One CTA per SM (the shared-memory footprint allows no second one), grid no larger
  // than the SM count: every CTA becomes resident as soon as the stream's earlier work
  // has drained, so a CTA that waits for another CTA's partial statistics is waiting for
  // a CTA that runs.  The waits are bounded in any case.
  cudaError_t e = launch_pdl(score_kernel<D, NCH, SPLIT>, dim3(grid), dim3(threads_for(SPLIT)),
                             Smem<D>::DYN_BYTES, stream, tmK, tmQ, a);
  if (e != cudaSuccess) return e;
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  *launches += 1;
  return cudaSuccess;
}

}  // namespace

// The part of the kernel's arguments that fixes the schedule (what for_each_item reads).
static ScoreArgs schedule_args(const ScorePlan& plan, int L, int W, int Hkv, int votes_only) {
  ScoreArgs a = {};
  a.L = L;
  a.n = plan.n_vote;
  a.mask_n = L - W;
  a.stats_only = 0;
  a.W = W;
  a.Hkv = Hkv;
  a.hpu = plan.hpu;
  a.ncols = plan.ncols;
  a.npad = plan.npad;
  a.sub_per_kv = plan.sub_per_kv;
  a.g = plan.g;
  a.units = plan.units;
  a.upw = plan.units_per_wave;
  a.nwaves = plan.nwaves;
  a.T1 = plan.tiles_stats;
  a.T2 = plan.tiles_vote;
  a.maxseg = plan.maxseg;
  a.pipelined = plan.pipelined;
  a.votes_only = votes_only;
  if (votes_only) {  // nothing couples the units any more: one phase over all of them
    a.upw = plan.units;
    a.nwaves = 1;
  }
  return a;
}

int list_schedule_items(const ScorePlan& plan, int L, int W, int Hkv, int votes_only, int grid,
                        int cta, int32_t* out, int max_items) {
  const ScoreArgs a = schedule_args(plan, L, W, Hkv, votes_only);
  int count = 0;
  for_each_item(a, cta, grid, a.pipelined, [&](const Item& it) {
    if (count < max_items) {
      int32_t* o = out + static_cast<size_t>(count) * 6;
      o[0] = it.unit; o[1] = it.t0; o[2] = it.t1; o[3] = it.vote; o[4] = it.slot; o[5] = it.nseg;
    }
    ++count;
    return true;
  });
  return count;
}

bool make_score_plan(int B, int Hq, int Hkv, int L, int d, int W, ScorePlan* plan, int n_vote) {
  if (B < 1 || Hq < 1 || Hkv < 1 || L < 1 || W < 1 || W > L || Hq % Hkv != 0) return false;
  if (n_vote > L) return false;
  if (W > MAX_COLS || (d != 64 && d != 128)) return false;
  ScorePlan p;
  p.g = Hq / Hkv;
  p.hpu = 1;
  for (int h = 1; h <= p.g; ++h)
    if (p.g % h == 0 && h * W <= MAX_COLS) p.hpu = h;
  p.sub_per_kv = p.g / p.hpu;
  const long long units = static_cast<long long>(B) * Hkv * p.sub_per_kv;
  if (units > (1 << 24)) return false;
  p.units = static_cast<int>(units);
  p.ncols = p.hpu * W;
  p.npad = p.ncols <= 32 ? 32 : (p.ncols <= 64 ? 64 : 128);
  const int n = n_vote >= 0 ? n_vote : L - W;
  p.n_vote = n;
  p.tiles_stats = (L + TILE_KEYS - 1) / TILE_KEYS;
  p.tiles_vote = (n + TILE_KEYS - 1) / TILE_KEYS;
  // A wave is a set of units whose keys are swept twice, WAVE_BYTES of keys; the statistics
  // run WAVE_LAG waves ahead of the votes.  Units too big for a wave take one wave each.
  const long long kbytes = static_cast<long long>(L) * d * 2;
  // With 128 window columns on one unit per KV head a vote tile costs the same from L2 as from
  // HBM (the softmax warps are its bound), so nothing is lost by waves too big for L2, and fewer,
  // longer phases split more evenly over the CTAs: such shapes take waves of twice the size
  // (191.6 vs 193.6 us per layer on the 32K GQA workload; narrower units and KV heads with
  // two sub-groups, whose vote tiles do gain from L2, are 3-5 % slower that way).
  const long long wave_bytes = (p.ncols == 128 && p.sub_per_kv == 1) ? 2 * WAVE_BYTES : WAVE_BYTES;
  long long kv_per_wave = wave_bytes / kbytes;
  // units bigger than a wave run one per wave: their second sweep comes from HBM, but the
  // statistics of the next unit still hide the hand-over between the two passes
  p.pipelined = WAVE_LAG;
  if (kv_per_wave < 1) kv_per_wave = 1;
  long long upw = kv_per_wave * p.sub_per_kv;
  // at most 128 units per wave: a CTA's share of a phase then spans few units, which
  // bounds the work items per phase (the book-keeper's buffers are sized for that)
  if (upw > 128) upw = 128 / p.sub_per_kv * p.sub_per_kv;
  if (upw < p.sub_per_kv) upw = p.sub_per_kv;
  if (upw > units) upw = units;
  // the bigger waves must not leave a single wave where two of the plain size were possible:
  // with one wave the votes start right behind the statistics and wait for the hand-over
  // (60.2 -> 57.2 us for 2 x 8 KV heads of 32K keys)
  if (wave_bytes != WAVE_BYTES && upw >= units && units >= 2 * p.sub_per_kv)
    upw = ((units / p.sub_per_kv + 1) / 2) * p.sub_per_kv;
  p.units_per_wave = static_cast<int>(upw);
  p.nwaves = (p.units + p.units_per_wave - 1) / p.units_per_wave;
  // partial slots per unit: a unit of T1 tiles is shared by at most ceil(T1 / q) + 1 CTAs
  // when every CTA gets at least q = floor(TT / G) tiles of the wave (G up to MAX_GRID)
  auto segs = [&](int nu) {
    const long long TT = static_cast<long long>(nu) * p.tiles_stats;
    const long long q = TT / MAX_GRID;
    long long s = q >= 1 ? (p.tiles_stats + q - 1) / q + 1 : p.tiles_stats;
    if (s > MAX_GRID) s = MAX_GRID;
    return static_cast<int>(s);
  };
  const int last_nu = p.units - (p.nwaves - 1) * p.units_per_wave;
  p.maxseg = segs(p.units_per_wave);
  if (segs(last_nu) > p.maxseg) p.maxseg = segs(last_nu);
  *plan = p;
  return true;
}

cudaError_t launch_window_scores(const void* q_obs, const void* k, const KVStrides& ks, int B,
                                 int Hq, int Hkv, int L, int d, int W, const ScorePlan& plan,
                                 float* vote, int* status,
                                 int* counters, float* partials, float* lse2, cudaStream_t stream,
                                 int* launches, const float* lse_obs, bool keep_status,
                                 bool never_ready, const PagedKV* paged, const ShardMode* shard) {
  CUtensorMap tmK, tmQ;
  {
    // (d, position, KV head, batch) with the caller's strides: any layout whose rows of d
    // elements are contiguous is one tensor map, e.g. [B, L, Hkv, d] as well as [B, Hkv, L, d].
    // A paged cache is the same map over the pool: (d, position in page, KV head, page); rows
    // past a page's end or pages outside the pool read as zeros.
    cuuint64_t dims[4] = {static_cast<cuuint64_t>(d),
                          static_cast<cuuint64_t>(paged ? paged->page_size : L),
                          static_cast<cuuint64_t>(Hkv),
                          static_cast<cuuint64_t>(paged ? paged->num_pages : B)};
    cuuint64_t strides[3] = {static_cast<cuuint64_t>(ks.l) * 2, static_cast<cuuint64_t>(ks.h) * 2,
                             static_cast<cuuint64_t>(ks.b) * 2};
    cuuint32_t box[4] = {64, TILE_KEYS, 1, 1};
    if (!encode_map(&tmK, k, 4, dims, strides, box)) return cudaErrorInvalidValue;
  }
  {
    cuuint64_t dims[2] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(B) * Hq * W};
    cuuint64_t strides[1] = {static_cast<cuuint64_t>(d) * 2};
    cuuint32_t box[2] = {64, static_cast<cuuint32_t>(plan.npad)};
    if (!encode_map(&tmQ, q_obs, 2, dims, strides, box)) return cudaErrorInvalidValue;
  }
  ScoreArgs a = schedule_args(plan, L, W, Hkv, (lse_obs || never_ready) ? 1 : 0);
  a.wait_ns = wait_limit_setting();
  if (shard) {
    a.mask_n = shard->mask_n;
    a.stats_only = shard->lse_out ? 1 : 0;
  }
  a.page_table = paged ? paged->table : nullptr;
  a.pages_per_seq = paged ? paged->pages_per_seq : 0;
  a.page_size = paged ? paged->page_size : 1;
  a.c2 = static_cast<float>(1.4426950408889634 / sqrt(static_cast<double>(d)));
  a.partials = partials;
  a.lse2 = lse2;
  a.counters = counters;
  a.status = status;
  a.vote = vote;
  if (lse_obs) {
    const cudaError_t e =
        launch_pdl(lse_prep_kernel, dim3(plan.units), dim3(MAX_COLS), 0, stream, lse_obs, lse2,
                   counters, status, keep_status ? 1 : 0, plan.units, plan.sub_per_kv, plan.g,
                   plan.hpu, W, plan.ncols);
    if (e != cudaSuccess) return e;
    *launches += 1;
  }
  int grid = sm_count();
  if (grid > MAX_GRID) grid = MAX_GRID;
  const int nch = plan.npad >> 5;
  // column-split epilogue when each warpgroup's half of the columns is whole heads
  const bool split = nch >= 2 && (W % 16) == 0 && ((plan.npad / 2) % W) == 0;
  cudaError_t e;
  if (d == 64) {
    if (nch == 1) e = run_scores<64, 1, false>(tmK, tmQ, a, grid, stream, launches);
    else if (nch == 2)
      e = split ? run_scores<64, 2, true>(tmK, tmQ, a, grid, stream, launches)
                : run_scores<64, 2, false>(tmK, tmQ, a, grid, stream, launches);
    else
      e = split ? run_scores<64, 4, true>(tmK, tmQ, a, grid, stream, launches)
                : run_scores<64, 4, false>(tmK, tmQ, a, grid, stream, launches);
  } else {
    if (nch == 1) e = run_scores<128, 1, false>(tmK, tmQ, a, grid, stream, launches);
    else if (nch == 2)
      e = split ? run_scores<128, 2, true>(tmK, tmQ, a, grid, stream, launches)
                : run_scores<128, 2, false>(tmK, tmQ, a, grid, stream, launches);
    else
      e = split ? run_scores<128, 4, true>(tmK, tmQ, a, grid, stream, launches)
                : run_scores<128, 4, false>(tmK, tmQ, a, grid, stream, launches);
  }
  if (e != cudaSuccess || !a.stats_only) return e;
  lse_finish_kernel<<<plan.units, MAX_COLS, 0, stream>>>(partials, counters, shard->lse_out, plan.units,
                                                        plan.maxseg, plan.sub_per_kv, plan.g, plan.hpu,
                                                        W, plan.ncols);
  *launches += 1;
  return cudaGetLastError();
}

}  // namespace snapkv
