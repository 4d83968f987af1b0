// C ABI of libsnapkv: argument validation, workspace layout, and the sequence of
// launches that makes up the compression step (Listing 1).
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <mutex>

#include "../../include/snapkv.h"
#include "launch.cuh"
#include "snapkv_internal.h"

namespace snapkv {

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Clears the status block and the unit counters behind it (a multiple of 256 bytes).  A
// kernel rather than a memset so that the scoring kernel behind it can be made resident early.
__global__ void clear_kernel(uint4* p, int n16) {
  pdl_launch_dependents();
  pdl_wait();
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += gridDim.x * blockDim.x)
    p[i] = make_uint4(0u, 0u, 0u, 0u);
}

// `keep_status`: leave the status block alone (a later part of one logical call must not wipe
// an error an earlier part recorded) and clear the counters only.
static cudaError_t launch_clear(uint8_t* ws, const WorkspaceLayout& w, cudaStream_t s,
                                bool keep_status = false) {
  const size_t from = keep_status ? w.off_counters : w.off_status;
  const int n16 = static_cast<int>((w.off_partials - from) / 16);
  const int blocks = n16 > 256 * 64 ? 64 : (n16 + 255) / 256;
  return launch_pdl(clear_kernel, dim3(blocks), dim3(256), 0, s,
                    reinterpret_cast<uint4*>(ws + from), n16);
}

// Zeroes the status block alone.  Entry points that run several single-sequence steps on one
// workspace do this once, up front, and then run every step with keep_status set, so that the
// block ends up holding the first error of any step.
static cudaError_t clear_status(void* ws, cudaStream_t s) {
  return cudaMemsetAsync(ws, 0, STATUS_BYTES, s);
}

static bool workspace_ok(const void* ws, size_t bytes, size_t need) {
  return ws && (reinterpret_cast<uintptr_t>(ws) & 255) == 0 && bytes >= need;
}

WorkspaceLayout make_layout(const ScorePlan& p, int B, int Hq, int n, bool need_vote,
                            bool need_pooled) {
  WorkspaceLayout w;
  size_t off = 0;
  w.off_status = off;
  off += STATUS_BYTES;
  w.off_counters = off;
  off = align_up(off + sizeof(int) * static_cast<size_t>(p.units), 256);
  w.off_partials = off;
  off = align_up(off + sizeof(float) * static_cast<size_t>(p.units) * p.maxseg * MAX_COLS, 256);
  w.off_lse = off;
  off = align_up(off + sizeof(float) * static_cast<size_t>(p.units) * MAX_COLS, 256);
  w.off_vote = off;
  const size_t row_bytes = sizeof(float) * static_cast<size_t>(B) * Hq * (n > 0 ? n : 0);
  if (need_vote) off = align_up(off + row_bytes, 256);
  w.off_pooled = off;
  if (need_pooled) off = align_up(off + select_scratch_bytes(B * Hq, n), 256);
  w.total = off;
  return w;
}

static thread_local int g_last_launches = 0;

static std::atomic<unsigned long long> g_wait_limit_ns{1000ull * 1000ull * 1000ull};
unsigned long long wait_limit_setting() { return g_wait_limit_ns.load(std::memory_order_relaxed); }

// Side stream and events of snapkv_compress_host, one set per device, created on first use
// and kept for the life of the process (nullptr if they cannot be created: the entry point
// then copies back on the caller's stream).
constexpr int HOST_PARTS = 8;
struct HostSide {
  cudaStream_t stream;
  cudaEvent_t computed[HOST_PARTS];
  cudaEvent_t done;
};
static HostSide* host_side() {
  constexpr int MAX_DEV = 64;
  static std::mutex mu;
  static HostSide* table[MAX_DEV] = {};
  static bool failed[MAX_DEV] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEV) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  if (table[dev] || failed[dev]) return table[dev];
  HostSide* h = new HostSide();
  bool ok = cudaStreamCreateWithFlags(&h->stream, cudaStreamNonBlocking) == cudaSuccess;
  for (int i = 0; ok && i < HOST_PARTS; ++i)
    ok = cudaEventCreateWithFlags(&h->computed[i], cudaEventDisableTiming) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&h->done, cudaEventDisableTiming) == cudaSuccess;
  if (!ok) {
    failed[dev] = true;
    delete h;
    return nullptr;
  }
  table[dev] = h;
  return h;
}

static snapkv_status_t check_common(int B, int Hq, int Hkv, int L, int d, int W) {
  if (B < 1 || Hq < 1 || Hkv < 1 || L < 1 || d < 1 || W < 1) return SNAPKV_ERR_INVALID_ARG;
  if (Hq % Hkv != 0 || W > L) return SNAPKV_ERR_INVALID_ARG;
  if (d != 64 && d != 128) return SNAPKV_ERR_UNSUPPORTED;
  if (W > MAX_COLS) return SNAPKV_ERR_UNSUPPORTED;
  if (static_cast<double>(B) * Hkv * L * d >= 1099511627776.0) return SNAPKV_ERR_UNSUPPORTED;
  if (static_cast<double>(B) * Hq * L >= 2147483647.0 * 16) return SNAPKV_ERR_UNSUPPORTED;
  return SNAPKV_OK;
}

static snapkv_status_t check_pool(int pool_kernel, int pool_type) {
  if (pool_kernel < 1 || (pool_kernel & 1) == 0) return SNAPKV_ERR_INVALID_ARG;
  if (pool_type != SNAPKV_POOL_MAX && pool_type != SNAPKV_POOL_AVG) return SNAPKV_ERR_INVALID_ARG;
  if (pool_kernel > 63) return SNAPKV_ERR_UNSUPPORTED;
  return SNAPKV_OK;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// out[i] = log sum_r exp(parts[r][i]), folded in the order of r (the same on every rank).
__global__ void lse_merge_kernel(const float* __restrict__ parts, int R, int count, float* __restrict__ out) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= count) return;
  float M = -INFINITY, S = 0.f;
  for (int r = 0; r < R; ++r) {
    const float p = parts[static_cast<size_t>(r) * count + i];
    const float Mn = fmaxf(fmaxf(M, p), -1e30f);
    S = S * expf(M - Mn) + expf(p - Mn);
    M = Mn;
  }
  out[i] = M + logf(S);
}

}  // namespace snapkv

using namespace snapkv;

extern "C" {

const char* snapkv_status_string(int status) {
  switch (status) {
    case SNAPKV_OK: return "SNAPKV_OK";
    case SNAPKV_ERR_INVALID_ARG: return "SNAPKV_ERR_INVALID_ARG";
    case SNAPKV_ERR_UNSUPPORTED: return "SNAPKV_ERR_UNSUPPORTED";
    case SNAPKV_ERR_WORKSPACE: return "SNAPKV_ERR_WORKSPACE";
    case SNAPKV_ERR_CUDA: return "SNAPKV_ERR_CUDA";
    case SNAPKV_ERR_TIMEOUT: return "SNAPKV_ERR_TIMEOUT";
    default: return "SNAPKV_UNKNOWN_STATUS";
  }
}

int snapkv_out_rows(int L, int budget) { return budget < L ? budget : L; }

int snapkv_last_launch_count(void) { return g_last_launches; }

size_t snapkv_workspace_size(int B, int Hq, int Hkv, int L, int d, int W, int pool_kernel,
                             int pool_type, int budget) {
  if (check_common(B, Hq, Hkv, L, d, W) != SNAPKV_OK) return 0;
  if (check_pool(pool_kernel, pool_type) != SNAPKV_OK) return 0;
  if (budget <= W) return 0;
  ScorePlan p;
  if (!make_score_plan(B, Hq, Hkv, L, d, W, &p)) return 0;
  const int n = L - W;
  return make_layout(p, B, Hq, n, true, select_needs_scratch(n)).total;
}

size_t snapkv_pool_topk_workspace_size(int rows, int n) {
  if (rows < 1 || n < 1) return 0;
  return select_scratch_bytes(rows, n);
}

static snapkv_status_t window_scores_impl(const void* q_obs, const void* k, const float* lse_obs,
                                          int B, int Hq, int Hkv, int L, int d, int W,
                                          float* out_vote, void* workspace,
                                          size_t workspace_bytes, void* stream) {
  snapkv_status_t st = check_common(B, Hq, Hkv, L, d, W);
  if (st != SNAPKV_OK) return st;
  if (W >= L) return SNAPKV_ERR_INVALID_ARG;
  if (!q_obs || !k || !out_vote) return SNAPKV_ERR_INVALID_ARG;
  if (!aligned16(q_obs) || !aligned16(k) || (reinterpret_cast<uintptr_t>(out_vote) & 3))
    return SNAPKV_ERR_INVALID_ARG;
  ScorePlan p;
  if (!make_score_plan(B, Hq, Hkv, L, d, W, &p)) return SNAPKV_ERR_UNSUPPORTED;
  const WorkspaceLayout w = make_layout(p, B, Hq, L - W, false, false);
  if (!workspace_ok(workspace, workspace_bytes, w.total)) return SNAPKV_ERR_WORKSPACE;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // with a supplied normaliser the conversion kernel clears what the clear kernel would
  int launches = 0;
  if (!lse_obs) {
    if (launch_clear(ws, w, s) != cudaSuccess) return SNAPKV_ERR_CUDA;
    launches = 1;
  }
  cudaError_t e = launch_window_scores(
      q_obs, k, dense_strides(Hkv, L, d), B, Hq, Hkv, L, d, W, p, out_vote, reinterpret_cast<int*>(ws + w.off_status),
      reinterpret_cast<int*>(ws + w.off_counters), reinterpret_cast<float*>(ws + w.off_partials),
      reinterpret_cast<float*>(ws + w.off_lse), s, &launches, lse_obs);
  if (e != cudaSuccess) return SNAPKV_ERR_CUDA;
  g_last_launches = launches;
  return SNAPKV_OK;
}

snapkv_status_t snapkv_window_scores(const void* q_obs, const void* k, int B, int Hq, int Hkv,
                                     int L, int d, int W, float* out_vote, void* workspace,
                                     size_t workspace_bytes, void* stream) {
  return window_scores_impl(q_obs, k, nullptr, B, Hq, Hkv, L, d, W, out_vote, workspace,
                            workspace_bytes, stream);
}

snapkv_status_t snapkv_window_scores_lse(const void* q_obs, const void* k, const float* lse_obs,
                                         int B, int Hq, int Hkv, int L, int d, int W,
                                         float* out_vote, void* workspace, size_t workspace_bytes,
                                         void* stream) {
  if (!lse_obs || (reinterpret_cast<uintptr_t>(lse_obs) & 3)) return SNAPKV_ERR_INVALID_ARG;
  return window_scores_impl(q_obs, k, lse_obs, B, Hq, Hkv, L, d, W, out_vote, workspace,
                            workspace_bytes, stream);
}

snapkv_status_t snapkv_pool_topk(const float* vote, int rows, int n, int pool_kernel, int pool_type,
                                 int ksel, int32_t* out_idx, void* workspace,
                                 size_t workspace_bytes, void* stream) {
  if (rows < 1 || n < 1 || ksel < 1 || ksel > n || !vote || !out_idx) return SNAPKV_ERR_INVALID_ARG;
  snapkv_status_t st = check_pool(pool_kernel, pool_type);
  if (st != SNAPKV_OK) return st;
  const size_t need = snapkv_pool_topk_workspace_size(rows, n);
  if (need > 0 &&
      (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < need))
    return SNAPKV_ERR_WORKSPACE;
  int launches = 0;
  cudaError_t e = launch_pool_topk(vote, rows, n, pool_kernel, pool_type, ksel, out_idx,
                                   static_cast<float*>(workspace),
                                   static_cast<cudaStream_t>(stream), &launches);
  return e == cudaSuccess ? SNAPKV_OK : SNAPKV_ERR_CUDA;
}

snapkv_status_t snapkv_gather(const void* k, const void* v, const int32_t* idx, int B, int Hq,
                              int Hkv, int L, int d, int W, int ksel, void* out_k, void* out_v,
                              void* stream) {
  snapkv_status_t st = check_common(B, Hq, Hkv, L, d, W);
  if (st != SNAPKV_OK) return st;
  if (ksel < 0 || ksel > L - W || !k || !v || !out_k || !out_v || (ksel > 0 && !idx))
    return SNAPKV_ERR_INVALID_ARG;
  if (!aligned16(k) || !aligned16(v) || !aligned16(out_k) || !aligned16(out_v))
    return SNAPKV_ERR_INVALID_ARG;
  int launches = 0;
  const KVStrides ds = dense_strides(Hkv, L, d);
  cudaError_t e = launch_gather(k, v, ds, ds, idx, B, Hq, Hkv, L, d, W, ksel, ksel + W, out_k,
                                out_v, static_cast<cudaStream_t>(stream), &launches);
  return e == cudaSuccess ? SNAPKV_OK : SNAPKV_ERR_CUDA;
}

static snapkv_status_t compress_impl(const void* q_obs, const void* k, const void* v, int B, int Hq,
                                     int Hkv, int L, int d, int W, int pool_kernel, int pool_type,
                                     int budget, void* out_k, void* out_v, int32_t* out_idx,
                                     void* workspace, size_t workspace_bytes, void* stream,
                                     bool keep_status, const float* lse_obs = nullptr,
                                     const KVStrides* k_str = nullptr,
                                     const KVStrides* v_str = nullptr, bool grouped = false,
                                     const PagedKV* paged = nullptr) {
  snapkv_status_t st = check_common(B, Hq, Hkv, L, d, W);
  if (st != SNAPKV_OK) return st;
  st = check_pool(pool_kernel, pool_type);
  if (st != SNAPKV_OK) return st;
  if (budget <= W) return SNAPKV_ERR_INVALID_ARG;
  if (!q_obs || !k || !v || !out_k || !out_v) return SNAPKV_ERR_INVALID_ARG;
  if (!aligned16(q_obs) || !aligned16(k) || !aligned16(v) || !aligned16(out_k) || !aligned16(out_v))
    return SNAPKV_ERR_INVALID_ARG;
  const int n = L - W;
  if (!out_idx && n > 0) return SNAPKV_ERR_INVALID_ARG;
  const KVStrides ks = k_str ? *k_str : dense_strides(Hkv, L, d);
  const KVStrides vs = v_str ? *v_str : dense_strides(Hkv, L, d);
  // shared selection: the votes of a group's query heads are summed when the select kernel
  // loads them, and the cache keeps Hkv heads
  const int Ho = grouped ? Hkv : Hq;
  const int gsum = grouped ? Hq / Hkv : 1;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int launches = 0;
  if (budget >= L) {
    // Listing 1's early return: nothing is dropped, the cache is expanded to Hq heads.
    if (launch_iota_idx(out_idx, B * Ho, n, budget - W, s, &launches) != cudaSuccess)
      return SNAPKV_ERR_CUDA;
    if (launch_gather(k, v, ks, vs, nullptr, B, Ho, Hkv, L, d, W, n, budget, out_k, out_v, s,
                      &launches, paged) != cudaSuccess)
      return SNAPKV_ERR_CUDA;
    // no kernel of this path can time out, but a caller that passes a workspace may read its
    // status afterwards: it must not find what an earlier use of the memory left there
    if (!keep_status && workspace_ok(workspace, workspace_bytes, STATUS_BYTES) &&
        clear_status(workspace, s) != cudaSuccess)
      return SNAPKV_ERR_CUDA;
    g_last_launches = launches;
    return SNAPKV_OK;
  }
  ScorePlan p;
  if (!make_score_plan(B, Hq, Hkv, L, d, W, &p)) return SNAPKV_ERR_UNSUPPORTED;
  const bool scratch = select_needs_scratch(n);
  const WorkspaceLayout w = make_layout(p, B, Hq, n, true, scratch);
  if (!workspace_ok(workspace, workspace_bytes, w.total)) return SNAPKV_ERR_WORKSPACE;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  if (!lse_obs) {
    if (launch_clear(ws, w, s, keep_status) != cudaSuccess) return SNAPKV_ERR_CUDA;
    launches += 1;
  }
  float* vote = reinterpret_cast<float*>(ws + w.off_vote);
  const int ksel = budget - W;
  if (launch_window_scores(q_obs, k, ks, B, Hq, Hkv, L, d, W, p, vote,
                           reinterpret_cast<int*>(ws + w.off_status),
                           reinterpret_cast<int*>(ws + w.off_counters),
                           reinterpret_cast<float*>(ws + w.off_partials),
                           reinterpret_cast<float*>(ws + w.off_lse), s, &launches, lse_obs,
                           keep_status, false, paged) != cudaSuccess)
    return SNAPKV_ERR_CUDA;
  if (launch_pool_topk(vote, B * Ho, n, pool_kernel, pool_type, ksel, out_idx,
                       scratch ? reinterpret_cast<float*>(ws + w.off_pooled) : nullptr, s,
                       &launches, gsum, /*vote_is_scratch=*/true) != cudaSuccess)
    return SNAPKV_ERR_CUDA;
  if (launch_gather(k, v, ks, vs, out_idx, B, Ho, Hkv, L, d, W, ksel, budget, out_k, out_v, s,
                    &launches, paged) != cudaSuccess)
    return SNAPKV_ERR_CUDA;
  g_last_launches = launches;
  return SNAPKV_OK;
}

snapkv_status_t snapkv_compress(const void* q_obs, const void* k, const void* v, int B, int Hq,
                                int Hkv, int L, int d, int W, int pool_kernel, int pool_type,
                                int budget, void* out_k, void* out_v, int32_t* out_idx,
                                void* workspace, size_t workspace_bytes, void* stream) {
  return compress_impl(q_obs, k, v, B, Hq, Hkv, L, d, W, pool_kernel, pool_type, budget, out_k,
                       out_v, out_idx, workspace, workspace_bytes, stream, false);
}

snapkv_status_t snapkv_compress_lse(const void* q_obs, const void* k, const void* v,
                                    const float* lse_obs, int B, int Hq, int Hkv, int L, int d,
                                    int W, int pool_kernel, int pool_type, int budget, void* out_k,
                                    void* out_v, int32_t* out_idx, void* workspace,
                                    size_t workspace_bytes, void* stream) {
  if (!lse_obs || (reinterpret_cast<uintptr_t>(lse_obs) & 3)) return SNAPKV_ERR_INVALID_ARG;
  return compress_impl(q_obs, k, v, B, Hq, Hkv, L, d, W, pool_kernel, pool_type, budget, out_k,
                       out_v, out_idx, workspace, workspace_bytes, stream, false, lse_obs);
}

// One stride triple of snapkv_compress_strided: positive, whole 16-byte vectors, rows of d
// elements do not overlap, and within what a tensor map can address (byte stride < 2^40).
static bool strides_ok(const int64_t* st, int d, KVStrides* out) {
  if (!st) return false;
  for (int i = 0; i < 3; ++i)
    if (st[i] <= 0 || (st[i] & 7) != 0 || st[i] >= (1ll << 39)) return false;
  if (st[2] < d) return false;
  out->b = st[0];
  out->h = st[1];
  out->l = st[2];
  return true;
}

snapkv_status_t snapkv_compress_strided(const void* q_obs, const void* k, const void* v,
                                        const int64_t* k_strides, const int64_t* v_strides,
                                        const float* lse_obs, int B, int Hq, int Hkv, int L,
                                        int d, int W, int pool_kernel, int pool_type, int budget,
                                        void* out_k, void* out_v, int32_t* out_idx,
                                        void* workspace, size_t workspace_bytes, void* stream) {
  KVStrides ks, vs;
  if (!strides_ok(k_strides, d, &ks) || !strides_ok(v_strides, d, &vs))
    return SNAPKV_ERR_INVALID_ARG;
  if (lse_obs && (reinterpret_cast<uintptr_t>(lse_obs) & 3)) return SNAPKV_ERR_INVALID_ARG;
  return compress_impl(q_obs, k, v, B, Hq, Hkv, L, d, W, pool_kernel, pool_type, budget, out_k,
                       out_v, out_idx, workspace, workspace_bytes, stream, false, lse_obs, &ks,
                       &vs);
}

snapkv_status_t snapkv_compress_grouped(const void* q_obs, const void* k, const void* v,
                                        const int64_t* k_strides, const int64_t* v_strides,
                                        const float* lse_obs, int B, int Hq, int Hkv, int L,
                                        int d, int W, int pool_kernel, int pool_type, int budget,
                                        void* out_k, void* out_v, int32_t* out_idx,
                                        void* workspace, size_t workspace_bytes, void* stream) {
  KVStrides ks, vs;
  if ((k_strides && !strides_ok(k_strides, d, &ks)) || (v_strides && !strides_ok(v_strides, d, &vs)))
    return SNAPKV_ERR_INVALID_ARG;
  if (lse_obs && (reinterpret_cast<uintptr_t>(lse_obs) & 3)) return SNAPKV_ERR_INVALID_ARG;
  return compress_impl(q_obs, k, v, B, Hq, Hkv, L, d, W, pool_kernel, pool_type, budget, out_k,
                       out_v, out_idx, workspace, workspace_bytes, stream, false, lse_obs,
                       k_strides ? &ks : nullptr, v_strides ? &vs : nullptr, true);
}

snapkv_status_t snapkv_compress_varlen(const void* q_obs, const void* k, const void* v,
                                       const int64_t* k_strides, const int64_t* v_strides,
                                       const int64_t* k_seq_offsets, const int64_t* v_seq_offsets,
                                       const int32_t* seq_lens, const float* lse_obs, int B,
                                       int Hq, int Hkv, int Lmax, int d, int W, int pool_kernel,
                                       int pool_type, int budget, void* out_k, void* out_v,
                                       int32_t* out_idx, void* workspace, size_t workspace_bytes,
                                       void* stream) {
  snapkv_status_t st = check_common(B, Hq, Hkv, Lmax, d, W);
  if (st != SNAPKV_OK) return st;
  if (!seq_lens || budget <= W || !q_obs || !k || !v || !out_k || !out_v)
    return SNAPKV_ERR_INVALID_ARG;
  KVStrides ks = dense_strides(Hkv, Lmax, d), vs = ks;
  if ((k_strides && !strides_ok(k_strides, d, &ks)) || (v_strides && !strides_ok(v_strides, d, &vs)))
    return SNAPKV_ERR_INVALID_ARG;
  if (lse_obs && (reinterpret_cast<uintptr_t>(lse_obs) & 3)) return SNAPKV_ERR_INVALID_ARG;
  // every sequence, every pointer and the workspace are checked before the first launch
  st = check_pool(pool_kernel, pool_type);
  if (st != SNAPKV_OK) return st;
  if (!aligned16(q_obs) || !aligned16(k) || !aligned16(v) || !aligned16(out_k) || !aligned16(out_v))
    return SNAPKV_ERR_INVALID_ARG;
  for (int b = 0; b < B; ++b) {
    if (seq_lens[b] < W || seq_lens[b] > Lmax) return SNAPKV_ERR_INVALID_ARG;
    if (k_seq_offsets && (k_seq_offsets[b] < 0 || (k_seq_offsets[b] & 7))) return SNAPKV_ERR_INVALID_ARG;
    if (v_seq_offsets && (v_seq_offsets[b] < 0 || (v_seq_offsets[b] & 7))) return SNAPKV_ERR_INVALID_ARG;
    if (!out_idx && seq_lens[b] > W) return SNAPKV_ERR_INVALID_ARG;
  }
  for (int b = 0; b < B; ++b) {
    if (budget >= seq_lens[b]) continue;  // copied through: no scratch
    const size_t need =
        snapkv_workspace_size(1, Hq, Hkv, seq_lens[b], d, W, pool_kernel, pool_type, budget);
    if (need == 0) return SNAPKV_ERR_INVALID_ARG;
    if (!workspace_ok(workspace, workspace_bytes, need)) return SNAPKV_ERR_WORKSPACE;
  }
  // one clear of the status block for the whole call, whichever path the first sequence takes
  const bool have_ws = workspace_ok(workspace, workspace_bytes, STATUS_BYTES);
  if (have_ws && clear_status(workspace, static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return SNAPKV_ERR_CUDA;
  const size_t head_rows = static_cast<size_t>(Hq) * budget * d * 2;  // bytes of one sequence's out_k
  int launches = 0;
  for (int b = 0; b < B; ++b) {
    const long long ko = k_seq_offsets ? k_seq_offsets[b] : b * ks.b;
    const long long vo = v_seq_offsets ? v_seq_offsets[b] : b * vs.b;
    // the sequences are independent (Sec. 4.1): one single-sequence step each, on the same
    // stream and workspace; the status block keeps the first error of any of them
    st = compress_impl(static_cast<const uint8_t*>(q_obs) + static_cast<size_t>(b) * Hq * W * d * 2,
                       static_cast<const uint8_t*>(k) + ko * 2,
                       static_cast<const uint8_t*>(v) + vo * 2, 1, Hq, Hkv, seq_lens[b], d, W,
                       pool_kernel, pool_type, budget,
                       static_cast<uint8_t*>(out_k) + b * head_rows,
                       static_cast<uint8_t*>(out_v) + b * head_rows,
                       out_idx ? out_idx + static_cast<size_t>(b) * Hq * (budget - W) : nullptr,
                       workspace, workspace_bytes, stream, /*keep_status=*/true,
                       lse_obs ? lse_obs + static_cast<size_t>(b) * Hq * W : nullptr, &ks, &vs);
    if (st != SNAPKV_OK) return st;
    launches += g_last_launches;
  }
  g_last_launches = launches;
  return SNAPKV_OK;
}

snapkv_status_t snapkv_compress_paged(const void* q_obs, const void* k_pool, const void* v_pool,
                                      const int64_t* k_strides, const int64_t* v_strides,
                                      const int32_t* page_table, int pages_per_seq, int page_size,
                                      int num_pages, const int32_t* seq_lens, const float* lse_obs,
                                      int B, int Hq, int Hkv, int L, int d, int W, int pool_kernel,
                                      int pool_type, int budget, void* out_k, void* out_v,
                                      int32_t* out_idx, void* workspace, size_t workspace_bytes,
                                      void* stream) {
  snapkv_status_t st = check_common(B, Hq, Hkv, L, d, W);
  if (st != SNAPKV_OK) return st;
  st = check_pool(pool_kernel, pool_type);
  if (st != SNAPKV_OK) return st;
  if (budget <= W || !q_obs || !k_pool || !v_pool || !out_k || !out_v || !page_table)
    return SNAPKV_ERR_INVALID_ARG;
  if (!aligned16(q_obs) || !aligned16(k_pool) || !aligned16(v_pool) || !aligned16(out_k) ||
      !aligned16(out_v) || (reinterpret_cast<uintptr_t>(page_table) & 3))
    return SNAPKV_ERR_INVALID_ARG;
  if (lse_obs && (reinterpret_cast<uintptr_t>(lse_obs) & 3)) return SNAPKV_ERR_INVALID_ARG;
  // a tile of TILE_KEYS keys must lie inside one page
  if (page_size < TILE_KEYS || page_size % TILE_KEYS != 0 || num_pages < 1 || pages_per_seq < 1)
    return SNAPKV_ERR_INVALID_ARG;
  if (static_cast<long long>(pages_per_seq) * page_size < L) return SNAPKV_ERR_INVALID_ARG;
  KVStrides ks, vs;
  if (!strides_ok(k_strides, d, &ks) || !strides_ok(v_strides, d, &vs)) return SNAPKV_ERR_INVALID_ARG;
  const PagedKV paged_all = {page_table, pages_per_seq, page_size, num_pages};
  if (!seq_lens)
    return compress_impl(q_obs, k_pool, v_pool, B, Hq, Hkv, L, d, W, pool_kernel, pool_type, budget,
                         out_k, out_v, out_idx, workspace, workspace_bytes, stream, false, lse_obs,
                         &ks, &vs, false, &paged_all);
  // per-sequence lengths: one single-sequence step each, as in snapkv_compress_varlen; every
  // sequence and the workspace are checked before the first launch
  for (int b = 0; b < B; ++b) {
    if (seq_lens[b] < W || seq_lens[b] > L) return SNAPKV_ERR_INVALID_ARG;
    if (!out_idx && seq_lens[b] > W) return SNAPKV_ERR_INVALID_ARG;
  }
  for (int b = 0; b < B; ++b) {
    if (budget >= seq_lens[b]) continue;
    const size_t need =
        snapkv_workspace_size(1, Hq, Hkv, seq_lens[b], d, W, pool_kernel, pool_type, budget);
    if (need == 0) return SNAPKV_ERR_INVALID_ARG;
    if (!workspace_ok(workspace, workspace_bytes, need)) return SNAPKV_ERR_WORKSPACE;
  }
  if (workspace_ok(workspace, workspace_bytes, STATUS_BYTES) &&
      clear_status(workspace, static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return SNAPKV_ERR_CUDA;
  const size_t head_rows = static_cast<size_t>(Hq) * budget * d * 2;
  int launches = 0;
  for (int b = 0; b < B; ++b) {
    const PagedKV one = {page_table + static_cast<size_t>(b) * pages_per_seq, pages_per_seq,
                         page_size, num_pages};
    st = compress_impl(static_cast<const uint8_t*>(q_obs) + static_cast<size_t>(b) * Hq * W * d * 2,
                       k_pool, v_pool, 1, Hq, Hkv, seq_lens[b], d, W, pool_kernel, pool_type, budget,
                       static_cast<uint8_t*>(out_k) + b * head_rows,
                       static_cast<uint8_t*>(out_v) + b * head_rows,
                       out_idx ? out_idx + static_cast<size_t>(b) * Hq * (budget - W) : nullptr,
                       workspace, workspace_bytes, stream, /*keep_status=*/true,
                       lse_obs ? lse_obs + static_cast<size_t>(b) * Hq * W : nullptr, &ks, &vs, false,
                       &one);
    if (st != SNAPKV_OK) return st;
    launches += g_last_launches;
  }
  g_last_launches = launches;
  return SNAPKV_OK;
}

// ---- a prompt sharded along its length over several GPUs: the per-shard steps
static snapkv_status_t shard_common(const void* q_obs, const void* k_shard, int B, int Hq, int Hkv,
                                    int Ls, int d, int W) {
  snapkv_status_t st = check_common(B, Hq, Hkv, Ls, d, W);
  if (st != SNAPKV_OK) return st;
  if (!q_obs || !k_shard || !aligned16(q_obs) || !aligned16(k_shard)) return SNAPKV_ERR_INVALID_ARG;
  return SNAPKV_OK;
}

snapkv_status_t snapkv_shard_lse(const void* q_obs, const void* k_shard, int B, int Hq, int Hkv,
                                 int Ls, int d, int W, int mask_n, float* out_lse, void* workspace,
                                 size_t workspace_bytes, void* stream) {
  snapkv_status_t st = shard_common(q_obs, k_shard, B, Hq, Hkv, Ls, d, W);
  if (st != SNAPKV_OK) return st;
  if (!out_lse || (reinterpret_cast<uintptr_t>(out_lse) & 3)) return SNAPKV_ERR_INVALID_ARG;
  ScorePlan p;
  if (!make_score_plan(B, Hq, Hkv, Ls, d, W, &p)) return SNAPKV_ERR_UNSUPPORTED;
  const WorkspaceLayout w = make_layout(p, B, Hq, 0, false, false);
  if (!workspace_ok(workspace, workspace_bytes, w.total)) return SNAPKV_ERR_WORKSPACE;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (launch_clear(ws, w, s) != cudaSuccess) return SNAPKV_ERR_CUDA;
  int launches = 1;
  const ShardMode shard = {mask_n, out_lse};
  if (launch_window_scores(q_obs, k_shard, dense_strides(Hkv, Ls, d), B, Hq, Hkv, Ls, d, W, p, nullptr,
                           reinterpret_cast<int*>(ws + w.off_status),
                           reinterpret_cast<int*>(ws + w.off_counters),
                           reinterpret_cast<float*>(ws + w.off_partials),
                           reinterpret_cast<float*>(ws + w.off_lse), s, &launches, nullptr, false,
                           false, nullptr, &shard) != cudaSuccess)
    return SNAPKV_ERR_CUDA;
  g_last_launches = launches;
  return SNAPKV_OK;
}

snapkv_status_t snapkv_lse_merge(const float* parts, int R, int count, float* out, void* stream) {
  if (!parts || !out || R < 1 || count < 1) return SNAPKV_ERR_INVALID_ARG;
  lse_merge_kernel<<<(count + 255) / 256, 256, 0, static_cast<cudaStream_t>(stream)>>>(parts, R, count, out);
  g_last_launches = 1;
  return cudaGetLastError() == cudaSuccess ? SNAPKV_OK : SNAPKV_ERR_CUDA;
}

snapkv_status_t snapkv_shard_votes(const void* q_obs, const void* k_shard, const float* lse_obs,
                                   int B, int Hq, int Hkv, int Ls, int d, int W, int n_vote,
                                   float* out_vote, void* workspace, size_t workspace_bytes,
                                   void* stream) {
  snapkv_status_t st = shard_common(q_obs, k_shard, B, Hq, Hkv, Ls, d, W);
  if (st != SNAPKV_OK) return st;
  if (!lse_obs || !out_vote || n_vote < 1 || n_vote > Ls) return SNAPKV_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(lse_obs) & 3) || (reinterpret_cast<uintptr_t>(out_vote) & 3))
    return SNAPKV_ERR_INVALID_ARG;
  ScorePlan p;
  if (!make_score_plan(B, Hq, Hkv, Ls, d, W, &p, n_vote)) return SNAPKV_ERR_UNSUPPORTED;
  const WorkspaceLayout w = make_layout(p, B, Hq, 0, false, false);
  if (!workspace_ok(workspace, workspace_bytes, w.total)) return SNAPKV_ERR_WORKSPACE;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  int launches = 0;
  if (launch_window_scores(q_obs, k_shard, dense_strides(Hkv, Ls, d), B, Hq, Hkv, Ls, d, W, p, out_vote,
                           reinterpret_cast<int*>(ws + w.off_status),
                           reinterpret_cast<int*>(ws + w.off_counters),
                           reinterpret_cast<float*>(ws + w.off_partials),
                           reinterpret_cast<float*>(ws + w.off_lse), static_cast<cudaStream_t>(stream),
                           &launches, lse_obs) != cudaSuccess)
    return SNAPKV_ERR_CUDA;
  g_last_launches = launches;
  return SNAPKV_OK;
}

snapkv_status_t snapkv_gather_range(const void* k_shard, const void* v_shard, const int32_t* idx,
                                    int B, int Hq, int Hkv, int Ls, int d, int pos0, int ksel,
                                    int append, void* out_k, void* out_v, int out_rows,
                                    int32_t* seg, void* stream) {
  if (B < 1 || Hq < 1 || Hkv < 1 || Hq % Hkv != 0 || Ls < 1 || (d != 64 && d != 128))
    return SNAPKV_ERR_INVALID_ARG;
  if (pos0 < 0 || ksel < 0 || append < 0 || append > Ls || !k_shard || !v_shard || !out_k || !out_v || !seg ||
      (ksel > 0 && !idx))
    return SNAPKV_ERR_INVALID_ARG;
  if (!aligned16(k_shard) || !aligned16(v_shard) || !aligned16(out_k) || !aligned16(out_v))
    return SNAPKV_ERR_INVALID_ARG;
  if (static_cast<long long>(B) * Hq > 65535) return SNAPKV_ERR_UNSUPPORTED;
  const int most = (ksel < Ls ? ksel : Ls) + append;  // rows a head can get from this shard
  if (out_rows < most) return SNAPKV_ERR_INVALID_ARG;
  int launches = 0;
  const KVStrides ds = dense_strides(Hkv, Ls, d);
  const cudaError_t e = launch_gather_range(k_shard, v_shard, ds, ds, idx, B, Hq, Hkv, Ls, d, pos0, ksel,
                                            append, out_rows, out_k, out_v, seg,
                                            static_cast<cudaStream_t>(stream), &launches);
  g_last_launches = launches;
  return e == cudaSuccess ? SNAPKV_OK : SNAPKV_ERR_CUDA;
}

size_t snapkv_host_staging_size(int B, int Hq, int Hkv, int L, int d, int W, int pool_kernel,
                                int pool_type, int budget) {
  if (check_common(B, Hq, Hkv, L, d, W) != SNAPKV_OK) return 0;
  if (check_pool(pool_kernel, pool_type) != SNAPKV_OK || budget <= W) return 0;
  const size_t qb = align_up(static_cast<size_t>(B) * Hq * W * d * 2, 256);
  const size_t kb = align_up(static_cast<size_t>(B) * Hkv * L * d * 2, 256);
  const size_t ob = align_up(static_cast<size_t>(B) * Hq * budget * d * 2, 256);
  const size_t ib = align_up(static_cast<size_t>(B) * Hq * (budget - W) * 4, 256);
  size_t ws = 0;
  if (budget < L) {
    // the entry point works through the (batch, KV head) pairs in parts, each a problem of
    // its own; the workspace must hold the largest of them (and the whole, if it runs as one)
    ws = snapkv_workspace_size(B, Hq, Hkv, L, d, W, pool_kernel, pool_type, budget);
    const int pairs = B * Hkv, g = Hq / Hkv;
    const int parts = pairs < HOST_PARTS ? pairs : HOST_PARTS;
    const int per = (pairs + parts - 1) / parts;
    const int sizes[2] = {per, pairs % per};
    for (int np : sizes)
      if (np > 0) {
        const size_t w1 = snapkv_workspace_size(1, np * g, np, L, d, W, pool_kernel, pool_type, budget);
        if (w1 > ws) ws = w1;
      }
  }
  return qb + 2 * kb + 2 * ob + ib + align_up(ws, 256);
}

snapkv_status_t snapkv_compress_host(const void* q_obs, const void* k, const void* v, int B, int Hq,
                                     int Hkv, int L, int d, int W, int pool_kernel, int pool_type,
                                     int budget, void* out_k, void* out_v, int32_t* out_idx,
                                     void* staging, size_t staging_bytes, void* stream) {
  const size_t need =
      snapkv_host_staging_size(B, Hq, Hkv, L, d, W, pool_kernel, pool_type, budget);
  if (need == 0) {
    snapkv_status_t st = check_common(B, Hq, Hkv, L, d, W);
    if (st != SNAPKV_OK) return st;
    st = check_pool(pool_kernel, pool_type);
    return st != SNAPKV_OK ? st : SNAPKV_ERR_INVALID_ARG;
  }
  if (!q_obs || !k || !v || !out_k || !out_v || !out_idx) return SNAPKV_ERR_INVALID_ARG;
  if (!staging || (reinterpret_cast<uintptr_t>(staging) & 255) || staging_bytes < need)
    return SNAPKV_ERR_WORKSPACE;
  const size_t q_raw = static_cast<size_t>(B) * Hq * W * d * 2;
  const size_t k_raw = static_cast<size_t>(B) * Hkv * L * d * 2;
  const size_t o_raw = static_cast<size_t>(B) * Hq * budget * d * 2;
  const size_t i_raw = static_cast<size_t>(B) * Hq * (budget - W) * 4;
  uint8_t* p = static_cast<uint8_t*>(staging);
  uint8_t* dq = p; p += align_up(q_raw, 256);
  uint8_t* dk = p; p += align_up(k_raw, 256);
  uint8_t* dv = p; p += align_up(k_raw, 256);
  uint8_t* dok = p; p += align_up(o_raw, 256);
  uint8_t* dov = p; p += align_up(o_raw, 256);
  uint8_t* di = p; p += align_up(i_raw, 256);
  uint8_t* dws = p;
  const size_t ws_bytes = staging_bytes - static_cast<size_t>(dws - static_cast<uint8_t*>(staging));
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // The (batch, KV head) pairs are independent: they go through in up to HOST_PARTS parts so
  // that the copy back of one part (on a side stream) runs while the next part's inputs are
  // still coming in; PCIe carries both directions at once.
  const int pairs = B * Hkv, g = Hq / Hkv;
  HostSide* side = host_side();
  int parts = side ? (pairs < HOST_PARTS ? pairs : HOST_PARTS) : 1;
  const int per = (pairs + parts - 1) / parts;
  parts = (pairs + per - 1) / per;
  const size_t q_pair = static_cast<size_t>(g) * W * d * 2, k_pair = static_cast<size_t>(L) * d * 2;
  const size_t o_pair = static_cast<size_t>(g) * budget * d * 2;
  const size_t i_pair = static_cast<size_t>(g) * (budget - W) * 4;
  int launches = 0;
  // (no workspace part in the staging buffer when the cache is copied through, budget >= L)
  if (workspace_ok(dws, ws_bytes, STATUS_BYTES) && clear_status(dws, s) != cudaSuccess)
    return SNAPKV_ERR_CUDA;
  for (int c = 0; c < parts; ++c) {
    const int p0 = c * per, np = (pairs - p0 < per) ? pairs - p0 : per;
    const size_t qo = p0 * q_pair, ko = p0 * k_pair, oo = p0 * o_pair, io = p0 * i_pair;
    if (cudaMemcpyAsync(dq + qo, static_cast<const uint8_t*>(q_obs) + qo, np * q_pair,
                        cudaMemcpyHostToDevice, s) != cudaSuccess ||
        cudaMemcpyAsync(dk + ko, static_cast<const uint8_t*>(k) + ko, np * k_pair,
                        cudaMemcpyHostToDevice, s) != cudaSuccess ||
        cudaMemcpyAsync(dv + ko, static_cast<const uint8_t*>(v) + ko, np * k_pair,
                        cudaMemcpyHostToDevice, s) != cudaSuccess)
      return SNAPKV_ERR_CUDA;
    // one part is a problem of its own with batch 1 and np KV heads (the layouts are flat
    // over batch and KV head); the parts share the workspace, which the stream serialises
    const snapkv_status_t st = compress_impl(
        dq + qo, dk + ko, dv + ko, 1, np * g, np, L, d, W, pool_kernel, pool_type, budget,
        dok + oo, dov + oo, reinterpret_cast<int32_t*>(di + io), dws, ws_bytes, stream,
        /*keep_status=*/true);
    if (st != SNAPKV_OK) return st;
    launches += g_last_launches;
    cudaStream_t back = s;
    if (side) {
      if (cudaEventRecord(side->computed[c], s) != cudaSuccess ||
          cudaStreamWaitEvent(side->stream, side->computed[c], 0) != cudaSuccess)
        return SNAPKV_ERR_CUDA;
      back = side->stream;
    }
    if (cudaMemcpyAsync(static_cast<uint8_t*>(out_k) + oo, dok + oo, np * o_pair,
                        cudaMemcpyDeviceToHost, back) != cudaSuccess ||
        cudaMemcpyAsync(static_cast<uint8_t*>(out_v) + oo, dov + oo, np * o_pair,
                        cudaMemcpyDeviceToHost, back) != cudaSuccess ||
        cudaMemcpyAsync(reinterpret_cast<uint8_t*>(out_idx) + io, di + io, np * i_pair,
                        cudaMemcpyDeviceToHost, back) != cudaSuccess)
      return SNAPKV_ERR_CUDA;
  }
  if (side) {  // the caller's stream is complete only when the last copy back is
    if (cudaEventRecord(side->done, side->stream) != cudaSuccess ||
        cudaStreamWaitEvent(s, side->done, 0) != cudaSuccess)
      return SNAPKV_ERR_CUDA;
  }
  g_last_launches = launches;
  return SNAPKV_OK;
}

int snapkv_schedule_items(int B, int Hq, int Hkv, int L, int d, int W, int votes_only, int grid,
                          int cta, int32_t* out_items, int max_items, int32_t* out_plan) {
  if (check_common(B, Hq, Hkv, L, d, W) != SNAPKV_OK || W >= L) return -1;
  if (grid < 1 || grid > MAX_GRID || cta < 0 || cta >= grid || max_items < 0) return -1;
  if (max_items > 0 && !out_items) return -1;
  ScorePlan p;
  if (!make_score_plan(B, Hq, Hkv, L, d, W, &p)) return -1;
  if (out_plan) {
    out_plan[0] = p.units;
    out_plan[1] = votes_only ? p.units : p.units_per_wave;
    out_plan[2] = votes_only ? 1 : p.nwaves;
    out_plan[3] = p.tiles_stats;
    out_plan[4] = p.tiles_vote;
    out_plan[5] = p.maxseg;
    out_plan[6] = p.pipelined;
    out_plan[7] = p.ncols;
  }
  return list_schedule_items(p, L, W, Hkv, votes_only ? 1 : 0, grid, cta, out_items, max_items);
}

unsigned long long snapkv_set_wait_limit_ns(unsigned long long limit_ns) {
  // at least a millisecond: a limit near the length of an ordinary wait would turn a busy
  // memory system into an error
  if (limit_ns < 1000000ull) limit_ns = 1000000ull;
  return g_wait_limit_ns.exchange(limit_ns, std::memory_order_relaxed);
}

snapkv_status_t snapkv_selftest_stalled_scores(const void* q_obs, const void* k, int B, int Hq,
                                               int Hkv, int L, int d, int W, float* out_vote,
                                               void* workspace, size_t workspace_bytes,
                                               void* stream) {
  snapkv_status_t st = check_common(B, Hq, Hkv, L, d, W);
  if (st != SNAPKV_OK) return st;
  if (W >= L || !q_obs || !k || !out_vote) return SNAPKV_ERR_INVALID_ARG;
  if (!aligned16(q_obs) || !aligned16(k) || (reinterpret_cast<uintptr_t>(out_vote) & 3))
    return SNAPKV_ERR_INVALID_ARG;
  ScorePlan p;
  if (!make_score_plan(B, Hq, Hkv, L, d, W, &p)) return SNAPKV_ERR_UNSUPPORTED;
  const WorkspaceLayout w = make_layout(p, B, Hq, L - W, false, false);
  if (!workspace_ok(workspace, workspace_bytes, w.total)) return SNAPKV_ERR_WORKSPACE;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int launches = 1;
  // counters cleared and never raised: every unit looks as if its statistics were still
  // on their way, for ever
  if (launch_clear(ws, w, s) != cudaSuccess) return SNAPKV_ERR_CUDA;
  cudaError_t e = launch_window_scores(
      q_obs, k, dense_strides(Hkv, L, d), B, Hq, Hkv, L, d, W, p, out_vote,
      reinterpret_cast<int*>(ws + w.off_status), reinterpret_cast<int*>(ws + w.off_counters),
      reinterpret_cast<float*>(ws + w.off_partials), reinterpret_cast<float*>(ws + w.off_lse), s,
      &launches, nullptr, false, /*never_ready=*/true);
  if (e != cudaSuccess) return SNAPKV_ERR_CUDA;
  g_last_launches = launches;
  return SNAPKV_OK;
}

snapkv_status_t snapkv_device_status(const void* workspace, void* stream, int* detail) {
  if (!workspace) return SNAPKV_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int host[2] = {0, 0};
  if (cudaMemcpyAsync(host, workspace, sizeof(host), cudaMemcpyDeviceToHost, s) != cudaSuccess)
    return SNAPKV_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return SNAPKV_ERR_CUDA;
  if (detail) *detail = host[1];
  return host[0] == 0 ? SNAPKV_OK : static_cast<snapkv_status_t>(host[0]);
}

}  // extern "C"
