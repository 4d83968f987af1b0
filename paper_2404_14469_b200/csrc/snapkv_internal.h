// Internal interfaces between the translation units of libsnapkv (not part of the ABI).
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <atomic>

namespace snapkv {

constexpr int TILE_KEYS = 128;      // keys per MMA tile
constexpr int MAX_COLS = 128;       // window-query columns handled by one unit
constexpr int STATUS_BYTES = 256;   // status block at the start of every workspace
constexpr int SM_COUNT_HINT = 148;  // B200
constexpr int MAX_GRID = 192;       // the scoring kernel runs one CTA per SM, at most this many

// Codes stored in the workspace status block's second word when a wait gives up.
enum WaitCode {
  WAIT_NONE = 0,
  WAIT_PRODUCER_EMPTY = 1,
  WAIT_MMA_FULL = 2,
  WAIT_MMA_TMEM_EMPTY = 3,
  WAIT_EPI_TMEM_FULL = 4,
  WAIT_Q_FULL = 5,
  /* 6 is not used */
  WAIT_UNIT_STATS = 7,
  WAIT_PART_EMPTY = 8,
  WAIT_PART_FULL = 9,
  WAIT_LSE_FULL = 10,
  WAIT_LSE_EMPTY = 11,
  WAIT_MERGE_COPY = 12,
};

// How the scoring passes split the work.  A "unit" is one (batch, KV head, head
// sub-group): `hpu` query heads that share the KV head, hpu * W <= MAX_COLS columns.
struct ScorePlan {
  int g;            // Hq / Hkv
  int hpu;          // query heads per unit
  int sub_per_kv;   // g / hpu
  int units;        // B * Hkv * sub_per_kv
  int ncols;        // hpu * W
  int npad;         // ncols rounded up to 32, 64 or 128
  int tiles_stats;  // ceil(L / TILE_KEYS): the normaliser covers every key
  int n_vote;       // keys that get a vote: L - W, or what a shard of a longer prompt asks for
  int tiles_vote;   // ceil(n_vote / TILE_KEYS): votes exist for prefix keys only
  int units_per_wave;
  int nwaves;
  int maxseg;       // partial-statistics slots per unit
  int pipelined;    // how many waves the statistics pass runs ahead of the vote pass (>= 1)
};

// Where a K or V tensor's rows are: element strides between consecutive batches, KV heads and
// positions of a tensor addressed as [batch][KV head][position][d] with d contiguous.  The
// dense [B, Hkv, L, d] cache of Listing 1 is {Hkv*L*d, L*d, d}.
struct KVStrides {
  long long b, h, l;
};
inline KVStrides dense_strides(int Hkv, int L, int d) {
  return KVStrides{static_cast<long long>(Hkv) * L * d, static_cast<long long>(L) * d, d};
}

// "Done once on this device" flag for set-up that belongs to a device's context (function
// attributes).  done() and set() refer to the calling thread's current device; devices beyond
// the table are never marked, so their set-up is simply repeated on every call.
class DeviceOnce {
 public:
  bool done() const {
    const int dev = current();
    return dev >= 0 && flags_[dev].load(std::memory_order_acquire);
  }
  void set() {
    const int dev = current();
    if (dev >= 0) flags_[dev].store(true, std::memory_order_release);
  }

 private:
  static constexpr int MAX_DEV = 64;
  static int current() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEV) return -1;
    return dev;
  }
  std::atomic<bool> flags_[MAX_DEV] = {};
};

// Block-table addressing of K and V (a serving stack's paged cache): position p of sequence b
// is row p % page_size of page table[b * pages_per_seq + p / page_size] of a pool of pages.
// With a table, a KVStrides' `b` is the element stride between consecutive PAGES of the pool,
// `h` between KV heads inside a page and `l` between positions inside a page.
struct PagedKV {
  const int32_t* table;  // device memory; nullptr = not paged
  int pages_per_seq;     // entries per sequence (row stride of the table)
  int page_size;         // positions per page, a multiple of TILE_KEYS
  int num_pages;         // pages in the pool; an entry outside [0, num_pages) reads as zeros
};

// A shard of a longer prompt (the positions [pos0, pos0 + L) of it).  `mask_n`: window row i
// sees the shard's keys j <= mask_n + i (the whole prompt's prefix length minus pos0; may be
// negative or beyond L).  With `lse_out` the statistics sweep alone runs and the shard's partial
// natural-log sum-exp of every window row goes to lse_out [B*Hq, W] (-inf where a row sees
// none of the shard's keys); `vote` is then not touched.
struct ShardMode {
  int mask_n;
  float* lse_out;
};

struct WorkspaceLayout {
  size_t off_status, off_counters, off_partials, off_lse, off_vote, off_pooled, total;
};

// The work items of block `cta` of a grid of `grid` blocks, in the order the scoring kernel
// walks them (the very routine the kernel runs, on the host).  Writes up to `max_items`
// records {unit, first tile, end tile, 1 for the vote sweep, partial slot, partials of the unit}
// and returns how many items there are.
int list_schedule_items(const ScorePlan& plan, int L, int W, int Hkv, int votes_only, int grid,
                        int cta, int32_t* out, int max_items);

// Time limit, in nanoseconds, that kernels launched from now on give each of their device-side
// waits (process-wide; one second unless snapkv_set_wait_limit_ns changed it).
unsigned long long wait_limit_setting();

// `n_vote` < 0: the keys that get a vote are the L - W prefix keys (the whole prompt is here).
bool make_score_plan(int B, int Hq, int Hkv, int L, int d, int W, ScorePlan* plan, int n_vote = -1);
WorkspaceLayout make_layout(const ScorePlan& p, int B, int Hq, int n, bool need_vote,
                            bool need_pooled);
bool select_needs_scratch(int n);
size_t select_scratch_bytes(int rows, int n);  // 0 when the rows fit one CTA

// Enqueue both scoring passes.  `vote` is fp32 [B*Hq, n].  `counters` must be zero when the
// kernel starts (the callers clear it together with the status block).  With `lse_obs`
// (device fp32 [B*Hq, W], natural-log sum-exp of every window row) the statistics pass is
// skipped: a small kernel converts the rows first, then only the vote pass runs; that kernel
// also zeroes the status block unless `keep_status` is set.  `never_ready` (self-test of the
// time-out path): the vote pass alone is launched and nothing marks the units' statistics as
// present, so its wait for them must run out.
cudaError_t launch_window_scores(const void* q_obs, const void* k, const KVStrides& ks, int B,
                                 int Hq, int Hkv, int L, int d, int W, const ScorePlan& plan,
                                 float* vote, int* status,
                                 int* counters, float* partials, float* lse2, cudaStream_t stream,
                                 int* launches, const float* lse_obs = nullptr,
                                 bool keep_status = false, bool never_ready = false,
                                 const PagedKV* paged = nullptr, const ShardMode* shard = nullptr);

// Pool + top-k over `rows` rows of fp32 votes.  `pooled_scratch` (select_scratch_bytes bytes)
// is only touched when select_needs_scratch(n).  With gsum > 1 a selection row is the sum of
// gsum consecutive rows of `vote` (which then holds rows * gsum rows): the query heads of a
// group selecting together.  vote_is_scratch: nobody reads `vote` after this call, so a
// kernel may leave its contents undefined (dirty L2 lines dropped instead of written back).
cudaError_t launch_pool_topk(const float* vote, int rows, int n, int pool_kernel, int pool_type,
                             int ksel, int32_t* out_idx, float* pooled_scratch,
                             cudaStream_t stream, int* launches, int gsum = 1,
                             bool vote_is_scratch = false);

// The one-cluster-per-row select kernel: whether it takes rows of this length and pooling
// kernel on the current device, and its launch (same contract as launch_pool_topk, no scratch).
bool select_cluster_applies(int rows, int n, int pool_kernel);
cudaError_t launch_pool_topk_cluster(const float* vote, int rows, int n, int pool_kernel,
                                     int pool_type, int ksel, int32_t* out_idx, cudaStream_t stream,
                                     int* launches, int gsum);

// Gather + append.  idx == nullptr copies rows 0..ksel-1 (identity path).
cudaError_t launch_gather(const void* k, const void* v, const KVStrides& ks, const KVStrides& vs,
                          const int32_t* idx, int B, int Hq, int Hkv, int L, int d, int W, int ksel,
                          int out_rows_stride, void* out_k, void* out_v, cudaStream_t stream,
                          int* launches, const PagedKV* paged = nullptr);

// A shard's part of the gather: rows of `idx` (global positions) that lie in [pos0, pos0 + L),
// then `append` trailing rows of the shard; seg [B*Hq][2] = {first entry, entries} per head.
cudaError_t launch_gather_range(const void* k, const void* v, const KVStrides& ks, const KVStrides& vs,
                                const int32_t* idx, int B, int Hq, int Hkv, int L, int d, int pos0,
                                int ksel, int append, int out_rows_stride, void* out_k, void* out_v,
                                int32_t* seg, cudaStream_t stream, int* launches);

cudaError_t launch_iota_idx(int32_t* out_idx, int rows, int n, int row_stride, cudaStream_t stream,
                            int* launches);

}  // namespace snapkv
