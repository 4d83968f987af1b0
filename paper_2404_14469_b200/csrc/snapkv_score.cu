// Window scoring (Eq. 1; Listing 1's compute_attn and the sum over the window):
//   vote[h, j] = sum_i softmax_i(q_i . k / sqrt(d))[j],  j in [0, n)
// computed in two tensor-core passes over K.
//
//  pass 1 (statistics)  S^T tile = Q_rep[128 x d] . K_tile[128 x d]^T : window rows on
//      TMEM lanes, keys on columns.  Each thread owns one window row and keeps a running
//      (max, sum of exp) over the keys it sees: an online softmax without shuffles.
//      When the unit has fewer than 128 window rows the rows are replicated along M and
//      each replica takes a different slice of the tile's keys, so all four epilogue
//      warps of a warpgroup stay busy.  The last CTA of a unit to finish merges the
//      partial (max, sum) pairs into one log2-sum-exp per window row.
//  pass 2 (votes)       S tile = K_tile[128 x d] . Q[ncols x d]^T : keys on TMEM lanes,
//      window rows on columns.  Each thread owns one key and adds exp2(s*c - lse) over
//      the W columns of each head: the sum over the window is a serial add per thread.
//
// Both passes share one warp-specialised skeleton: warp 0 issues TMA loads of K tiles
// into a ring of shared-memory stages, warp 1 issues tcgen05.mma into four TMEM
// accumulator buffers, warps 2-9 (two warpgroups, alternating tiles) read the
// accumulators back with tcgen05.ld and do the fp32 softmax arithmetic.
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "sm100_ptx.cuh"
#include "snapkv_internal.h"

namespace snapkv {

namespace {

constexpr int STAGES = 4;
constexpr int NBUF = 4;               // TMEM accumulator buffers of 128 columns
constexpr int TMEM_COLS = 512;
constexpr int SUBTILE_BYTES = 128 * 128;  // 128 rows x 64 bf16, 128-byte swizzled
constexpr int THREADS = 320;          // producer warp, MMA warp, 8 epilogue warps
constexpr int EPI_THREADS = 256;

struct ScoreArgs {
  int L, n, W;
  int hpu, ncols, npad;
  int sub_per_kv, g;
  int tiles, chunks, unit0;
  float c2;  // log2(e) / sqrt(d)
  float2* partials;
  float* lse2;
  int* counters;
  int* status;
  float* vote;
};

template <int D>
struct Smem {
  static constexpr int SUBT = D / 64;
  static constexpr int Q_BYTES = SUBT * SUBTILE_BYTES;
  static constexpr int STAGE_BYTES = SUBT * SUBTILE_BYTES;
  static constexpr int OFF_Q = 0;
  static constexpr int OFF_K = Q_BYTES;
  static constexpr int OFF_BAR = OFF_K + STAGES * STAGE_BYTES;
  // barriers: full[STAGES], empty[STAGES], tf[NBUF], te[NBUF], qfull, drain
  static constexpr int NBAR = 2 * STAGES + 2 * NBUF + 2;
  static constexpr int OFF_MISC = OFF_BAR + NBAR * 8;       // tmem ptr, abort, last flag
  static constexpr int OFF_PART = OFF_MISC + 16;            // float2 [8][32]
  static constexpr int OFF_LSE = OFF_PART + 8 * 32 * 8;     // float [128]
  static constexpr int TOTAL = OFF_LSE + 128 * 4;
  static constexpr int DYN_BYTES = TOTAL + 1024;            // slack for 1024-byte alignment
};

__device__ __forceinline__ bool mbar_wait_drain(uint32_t bar, uint32_t parity) {
  const unsigned long long t0 = globaltimer_ns();
  for (;;) {
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (globaltimer_ns() - t0 > WAIT_LIMIT_NS) return false;
  }
}

// NCH = npad / 32: how many 32-column chunks of the accumulator a thread reads per tile.
template <int D, bool VOTE, int NCH>
__global__ void __launch_bounds__(THREADS, 1)
score_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmQ,
             const ScoreArgs a) {
  using SM = Smem<D>;
  constexpr int SUBT = SM::SUBT;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  const uint32_t sbase = smem_u32(smem);
  const uint32_t q_s = sbase + SM::OFF_Q;
  const uint32_t k_s = sbase + SM::OFF_K;
  const uint32_t bar0 = sbase + SM::OFF_BAR;
  auto bar_full = [&](int s) { return bar0 + 8u * s; };
  auto bar_empty = [&](int s) { return bar0 + 8u * (STAGES + s); };
  auto bar_tf = [&](int b) { return bar0 + 8u * (2 * STAGES + b); };
  auto bar_te = [&](int b) { return bar0 + 8u * (2 * STAGES + NBUF + b); };
  const uint32_t bar_q = bar0 + 8u * (2 * STAGES + 2 * NBUF);
  const uint32_t bar_drain = bar_q + 8u;
  volatile uint32_t* tmem_ptr_s = reinterpret_cast<volatile uint32_t*>(smem + SM::OFF_MISC);
  volatile int* abort_s = reinterpret_cast<volatile int*>(smem + SM::OFF_MISC + 4);
  volatile int* last_s = reinterpret_cast<volatile int*>(smem + SM::OFF_MISC + 8);
  float2* part_s = reinterpret_cast<float2*>(smem + SM::OFF_PART);
  float* lse_s = reinterpret_cast<float*>(smem + SM::OFF_LSE);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int chunk = blockIdx.x;
  const int u = a.unit0 + blockIdx.y;          // unit
  const int ukv = u / a.sub_per_kv;            // flat (batch, KV head)
  const int sub = u - ukv * a.sub_per_kv;
  const int hq0 = ukv * a.g + sub * a.hpu;     // first query head of the unit, flat over batch
  const int t_begin = static_cast<int>((static_cast<long long>(chunk) * a.tiles) / a.chunks);
  const int t_end = static_cast<int>((static_cast<long long>(chunk + 1) * a.tiles) / a.chunks);
  const int nt = t_end - t_begin;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(bar_full(s), 1);
      mbar_init(bar_empty(s), 1);
    }
    for (int b = 0; b < NBUF; ++b) {
      mbar_init(bar_tf(b), 1);
      mbar_init(bar_te(b), 4);
    }
    mbar_init(bar_q, 1);
    mbar_init(bar_drain, 1);
    *abort_s = 0;
    *last_s = 0;
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_ptr_s)), TMEM_COLS);
    tmem_relinquish();
  }
  if (VOTE) {
    // -lse2 of this unit's window rows, written by the statistics pass
    if (threadIdx.x >= 64 && threadIdx.x < 64 + 128) {
      const int c = threadIdx.x - 64;
      lse_s[c] = (c < a.ncols) ? -__ldcg(a.lse2 + static_cast<size_t>(u) * MAX_COLS + c) : 0.f;
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_ptr_s;

  // tile visited at iteration `it`: ascending in the statistics pass, descending in the
  // vote pass (the tiles read last by pass 1 are the most likely to still be in L2)
  auto tile_of = [&](int it) { return VOTE ? (t_end - 1 - it) : (t_begin + it); };

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&tmK);
      tma_prefetch_desc(&tmQ);
      const int qrow0 = hq0 * a.W;
      if (VOTE) {
        mbar_expect_tx(bar_q, SUBT * a.npad * 128);
        for (int sb = 0; sb < SUBT; ++sb)
          tma_load_2d(q_s + sb * SUBTILE_BYTES, &tmQ, bar_q, sb * 64, qrow0);
      } else {
        mbar_expect_tx(bar_q, SUBT * 128 * 128);
        const int reps = 128 / a.npad;
        for (int rep = 0; rep < reps; ++rep)
          for (int sb = 0; sb < SUBT; ++sb)
            tma_load_2d(q_s + sb * SUBTILE_BYTES + rep * a.npad * 128, &tmQ, bar_q, sb * 64, qrow0);
      }
      int issued = 0;
      for (int it = 0; it < nt; ++it) {
        const int s = it % STAGES;
        const uint32_t ph = (it / STAGES) & 1;
        if (!mbar_wait_thread(bar_empty(s), ph ^ 1, abort_s, WAIT_PRODUCER_EMPTY)) break;
        mbar_expect_tx(bar_full(s), SM::STAGE_BYTES);
        const int key0 = tile_of(it) * TILE_KEYS;
        for (int sb = 0; sb < SUBT; ++sb)
          tma_load_3d(k_s + s * SM::STAGE_BYTES + sb * SUBTILE_BYTES, &tmK, bar_full(s), sb * 64,
                      key0, ukv);
        issued = it + 1;
      }
      if (*abort_s != 0) {
        // let every copy in flight land before the CTA's shared memory goes away
        mbar_wait_drain(bar_q, 0);
        for (int s = 0; s < STAGES; ++s) {
          int last = -1;
          for (int it = s; it < issued; it += STAGES) last = it;
          if (last >= 0) mbar_wait_drain(bar_full(s), (last / STAGES) & 1);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = VOTE ? umma_idesc_bf16(128, a.npad) : umma_idesc_bf16(128, 128);
      bool ok = mbar_wait_thread(bar_q, 0, abort_s, WAIT_Q_FULL);
      for (int it = 0; ok && it < nt; ++it) {
        const int s = it % STAGES;
        const uint32_t ph = (it / STAGES) & 1;
        const int buf = it & (NBUF - 1);
        const uint32_t ub = (it / NBUF) & 1;
        if (!mbar_wait_thread(bar_full(s), ph, abort_s, WAIT_MMA_FULL)) break;
        if (!mbar_wait_thread(bar_te(buf), ub ^ 1, abort_s, WAIT_MMA_TMEM_EMPTY)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * 128;
#pragma unroll
        for (int sb = 0; sb < SUBT; ++sb) {
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            const uint64_t kd =
                umma_desc_k128(k_s + s * SM::STAGE_BYTES + sb * SUBTILE_BYTES + kk * 32);
            const uint64_t qd = umma_desc_k128(q_s + sb * SUBTILE_BYTES + kk * 32);
            if (VOTE) tc_mma_bf16(d_tmem, kd, qd, idesc, (sb | kk) != 0);
            else tc_mma_bf16(d_tmem, qd, kd, idesc, (sb | kk) != 0);
          }
        }
        tc_commit(bar_empty(s));
        tc_commit(bar_tf(buf));
      }
      if (*abort_s != 0) {
        tc_commit(bar_drain);
        mbar_wait_drain(bar_drain, 0);
      }
    }
  } else {
    // ------------------------------------------------------------ softmax warps
    const int e = warp - 2;
    const int wg = e >> 2;
    const int q = warp & 3;  // TMEM lane quarter this warp may read
    const uint32_t lane_sel = static_cast<uint32_t>(32 * q) << 16;
    if (!VOTE) {
      const int rrow = 32 * q + lane;
      const int rep = rrow / a.npad;
      const int qcol = rrow - rep * a.npad;
      const int i = qcol % a.W;
      const int jmax = min(a.L - 1, a.n + i);
      float m2 = -INFINITY;  // running max, log2 domain
      float l = 0.f;         // running sum of exp2(x - m2)
      for (int it = wg; it < nt; it += 2) {
        const int buf = it & (NBUF - 1);
        const uint32_t ub = (it / NBUF) & 1;
        if (!mbar_wait_warp(bar_tf(buf), ub, abort_s, WAIT_EPI_TMEM_FULL)) break;
        tc_fence_after();
        const int key0 = tile_of(it) * TILE_KEYS;
        // the whole slice of this thread's row: NCH * 32 key columns
        float v[NCH][32];
        const uint32_t taddr = tmem_base + lane_sel + buf * 128 + rep * (NCH * 32);
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch) tmem_ld32(taddr + ch * 32, v[ch]);
        tmem_wait_ld();
        // the accumulator is in registers now: hand the buffer back to the MMA warp
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_te(buf));
        if (key0 + TILE_KEYS - 1 > a.n) {  // tile touches the window or the end of the prompt
          const int kb = key0 + rep * (NCH * 32);
#pragma unroll
          for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
            for (int c = 0; c < 32; ++c)
              v[ch][c] = (kb + ch * 32 + c <= jmax) ? v[ch][c] : -INFINITY;
        }
        float c0 = v[0][0], c1 = v[0][1], c2m = v[0][2], c3 = v[0][3];
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch)
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
        for (int ch = 0; ch < NCH; ++ch)
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
      part_s[(wg * 4 + q) * 32 + lane] = make_float2(m2, l);
      named_bar_sync(1, EPI_THREADS);
      const int tid = threadIdx.x - 64;
      const bool aborted = (*abort_s != 0);
      if (!aborted && tid < a.ncols) {
        // merge the replicas and the two warpgroups of this CTA, fixed order
        const int reps = 128 / a.npad;
        float M = -INFINITY;
        for (int w2 = 0; w2 < 2; ++w2)
          for (int r = 0; r < reps; ++r) {
            const int row = r * a.npad + tid;
            M = fmaxf(M, part_s[(w2 * 4 + (row >> 5)) * 32 + (row & 31)].x);
          }
        float S = 0.f;
        for (int w2 = 0; w2 < 2; ++w2)
          for (int r = 0; r < reps; ++r) {
            const int row = r * a.npad + tid;
            const float2 p = part_s[(w2 * 4 + (row >> 5)) * 32 + (row & 31)];
            S += p.y * exp2f(p.x - M);
          }
        a.partials[(static_cast<size_t>(u) * a.chunks + chunk) * MAX_COLS + tid] = make_float2(M, S);
      }
      __threadfence();
      named_bar_sync(1, EPI_THREADS);
      if (tid == 0 && !aborted) {
        const int old = atomicAdd(a.counters + u, 1);
        *last_s = (old == a.chunks - 1) ? 1 : 0;
      }
      named_bar_sync(1, EPI_THREADS);
      if (*last_s != 0 && tid < a.ncols) {
        // this CTA finished last for the unit: every partial is visible now
        __threadfence();
        const float2* pp = a.partials + static_cast<size_t>(u) * a.chunks * MAX_COLS + tid;
        float M = -INFINITY;
        for (int c = 0; c < a.chunks; ++c) M = fmaxf(M, __ldcg(pp + c * MAX_COLS).x);
        float S = 0.f;
        for (int c = 0; c < a.chunks; ++c) {
          const float2 p = __ldcg(pp + c * MAX_COLS);
          S += p.y * exp2f(p.x - M);
        }
        a.lse2[static_cast<size_t>(u) * MAX_COLS + tid] = M + log2f(S);
      }
    } else {
      // ---------------------------------------------------------- votes
      const bool w16 = (a.W & 15) == 0;
      const int gpw = a.W >> 4;  // 16-column groups per head (when W is a multiple of 16)
      for (int it = wg; it < nt; it += 2) {
        const int buf = it & (NBUF - 1);
        const uint32_t ub = (it / NBUF) & 1;
        if (!mbar_wait_warp(bar_tf(buf), ub, abort_s, WAIT_EPI_TMEM_FULL)) break;
        tc_fence_after();
        const int j = tile_of(it) * TILE_KEYS + 32 * q + lane;
        const uint32_t taddr = tmem_base + lane_sel + buf * 128;
        // this key's logits against every window row of the unit
        float v[NCH][32];
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch) tmem_ld32(taddr + ch * 32, v[ch]);
        tmem_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_te(buf));
        if (w16) {
          // exp2(s * c2 - lse2) summed over each group of 16 columns, then groups -> heads
          float g16[NCH * 2];
#pragma unroll
          for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
              const float4* nl = reinterpret_cast<const float4*>(lse_s + ch * 32 + hf * 16);
              float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
              for (int t4 = 0; t4 < 4; ++t4) {
                const float4 z = nl[t4];
                a0 += ex2_approx(fmaf(v[ch][hf * 16 + 4 * t4 + 0], a.c2, z.x));
                a1 += ex2_approx(fmaf(v[ch][hf * 16 + 4 * t4 + 1], a.c2, z.y));
                a2 += ex2_approx(fmaf(v[ch][hf * 16 + 4 * t4 + 2], a.c2, z.z));
                a3 += ex2_approx(fmaf(v[ch][hf * 16 + 4 * t4 + 3], a.c2, z.w));
              }
              g16[ch * 2 + hf] = (a0 + a1) + (a2 + a3);
            }
          int hl = 0, left = gpw;
          float acc = 0.f;
#pragma unroll
          for (int gi = 0; gi < NCH * 2; ++gi) {
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
          for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
            for (int c = 0; c < 32; ++c) {
              const int col = ch * 32 + c;
              if (col < a.ncols) {
                acc += ex2_approx(fmaf(v[ch][c], a.c2, lse_s[col]));
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
    }
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
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank, const_cast<void*>(base), dims,
            strides_bytes, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D, int NCH>
cudaError_t run_passes(const CUtensorMap& tmK, const CUtensorMap& tmQ, ScoreArgs a,
                       const ScorePlan& p, cudaStream_t stream, int* launches) {
  static bool attr_done = false;
  if (!attr_done) {
    cudaError_t e = cudaFuncSetAttribute(score_kernel<D, false, NCH>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         Smem<D>::DYN_BYTES);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(score_kernel<D, true, NCH>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<D>::DYN_BYTES);
    if (e != cudaSuccess) return e;
    attr_done = true;
  }
  for (int u0 = 0; u0 < p.units; u0 += p.units_per_wave) {
    const int nu = (p.units - u0 < p.units_per_wave) ? (p.units - u0) : p.units_per_wave;
    a.unit0 = u0;
    a.tiles = p.tiles_stats;
    a.chunks = p.chunks_stats;
    score_kernel<D, false, NCH><<<dim3(p.chunks_stats, nu), THREADS, Smem<D>::DYN_BYTES, stream>>>(
        tmK, tmQ, a);
    a.tiles = p.tiles_vote;
    a.chunks = p.chunks_vote;
    score_kernel<D, true, NCH><<<dim3(p.chunks_vote, nu), THREADS, Smem<D>::DYN_BYTES, stream>>>(
        tmK, tmQ, a);
    *launches += 2;
  }
  return cudaGetLastError();
}

}  // namespace

bool make_score_plan(int B, int Hq, int Hkv, int L, int d, int W, ScorePlan* plan) {
  if (B < 1 || Hq < 1 || Hkv < 1 || L < 1 || W < 1 || W > L || Hq % Hkv != 0) return false;
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
  const int n = L - W;
  p.tiles_stats = (L + TILE_KEYS - 1) / TILE_KEYS;
  p.tiles_vote = (n + TILE_KEYS - 1) / TILE_KEYS;
  // A wave is the set of units whose keys are swept twice back to back; it is sized so
  // that the second sweep finds the keys in L2 (64 MiB of K per wave).
  const long long kbytes = static_cast<long long>(L) * d * 2;
  long long kv_per_wave = (64ll << 20) / kbytes;
  if (kv_per_wave < 1) kv_per_wave = 1;
  if (kv_per_wave > 4096) kv_per_wave = 4096;
  long long upw = kv_per_wave * p.sub_per_kv;
  if (upw > units) upw = units;
  p.units_per_wave = static_cast<int>(upw);
  auto chunks_for = [&](int tiles) {
    int c = SM_COUNT_HINT / p.units_per_wave;
    if (c < 1) c = 1;
    if (c > tiles) c = tiles;
    if (c < 1) c = 1;
    return c;
  };
  p.chunks_stats = chunks_for(p.tiles_stats);
  p.chunks_vote = chunks_for(p.tiles_vote);
  *plan = p;
  return true;
}

cudaError_t launch_window_scores(const void* q_obs, const void* k, int B, int Hq, int Hkv, int L,
                                 int d, int W, const ScorePlan& plan, float* vote, int* status,
                                 int* counters, float2* partials, float* lse2, cudaStream_t stream,
                                 int* launches) {
  CUtensorMap tmK, tmQ;
  {
    cuuint64_t dims[3] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(L),
                          static_cast<cuuint64_t>(B) * Hkv};
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(d) * 2, static_cast<cuuint64_t>(L) * d * 2};
    cuuint32_t box[3] = {64, TILE_KEYS, 1};
    if (!encode_map(&tmK, k, 3, dims, strides, box)) return cudaErrorInvalidValue;
  }
  {
    cuuint64_t dims[2] = {static_cast<cuuint64_t>(d), static_cast<cuuint64_t>(B) * Hq * W};
    cuuint64_t strides[1] = {static_cast<cuuint64_t>(d) * 2};
    cuuint32_t box[2] = {64, static_cast<cuuint32_t>(plan.npad)};
    if (!encode_map(&tmQ, q_obs, 2, dims, strides, box)) return cudaErrorInvalidValue;
  }
  cudaError_t e = cudaMemsetAsync(counters, 0, sizeof(int) * plan.units, stream);
  if (e != cudaSuccess) return e;
  ScoreArgs a;
  a.L = L;
  a.n = L - W;
  a.W = W;
  a.hpu = plan.hpu;
  a.ncols = plan.ncols;
  a.npad = plan.npad;
  a.sub_per_kv = plan.sub_per_kv;
  a.g = plan.g;
  a.tiles = 0;
  a.chunks = 0;
  a.unit0 = 0;
  a.c2 = static_cast<float>(1.4426950408889634 / sqrt(static_cast<double>(d)));
  a.partials = partials;
  a.lse2 = lse2;
  a.counters = counters;
  a.status = status;
  a.vote = vote;
  const int nch = plan.npad >> 5;
  if (d == 64) {
    if (nch == 1) return run_passes<64, 1>(tmK, tmQ, a, plan, stream, launches);
    if (nch == 2) return run_passes<64, 2>(tmK, tmQ, a, plan, stream, launches);
    return run_passes<64, 4>(tmK, tmQ, a, plan, stream, launches);
  }
  if (nch == 1) return run_passes<128, 1>(tmK, tmQ, a, plan, stream, launches);
  if (nch == 2) return run_passes<128, 2>(tmK, tmQ, a, plan, stream, launches);
  return run_passes<128, 4>(tmK, tmQ, a, plan, stream, launches);
}

}  // namespace snapkv
