/*
 * snapkv.h - C ABI of the SnapKV prompt KV-cache compression step for NVIDIA B200.
 *
 * The step follows arXiv 2404.14469, Sec. 4 (Eq. 1-2) and Listing 1: the last W
 * prompt queries (the observation window) score every prompt key, the softmax
 * probabilities are summed over the window, pooled along the sequence, the
 * top-(budget - W) prefix positions are chosen per head, and those K/V rows plus
 * the window's own rows form the compressed cache.
 *
 * Notation: L prompt length, W window, n = L - W prefix length, d head dimension,
 * ksel = budget - W selected rows per head, g = Hq / Hkv (query head h reads KV
 * head h / g; each query head selects its own positions).
 *
 * Conventions for every entry point
 *   - All tensors are dense, row-major, in the stated shape; "bf16" is the 16-bit
 *     brain-float bit pattern.  Device pointers must be 16-byte aligned and must
 *     not alias one another.
 *   - The caller owns every buffer the entry points read or write.  The library itself
 *     holds, for the life of the process: one fixed 16 MiB device array on every GPU
 *     that loads it (the scratch of snapkv_pool_topk_static), and, per device and
 *     created on the first snapkv_compress_host call there, one side stream and a
 *     handful of events.  It caches driver entry points, the SM count and "attribute
 *     set" flags per device.  Nothing else is allocated and no per-call state is kept.
 *   - One call at a time per device.  The scoring kernel behind snapkv_compress*,
 *     snapkv_window_scores* is a persistent grid of one block per SM whose blocks wait
 *     for one another's partial results; that is safe because all of them are resident
 *     at once, which needs the whole GPU.  If another kernel holds SMs (a second
 *     library call on another stream, other work of the caller, another tenant of the
 *     GPU), blocks of the grid may not get an SM while the resident ones wait for them:
 *     the waits then run into their one-second limit, the call's outputs are left
 *     unwritten and SNAPKV_ERR_TIMEOUT is recorded in the status block.  So do not let
 *     two scoring/compress calls, or such a call and other large kernels, overlap on one
 *     GPU; calls on one stream never do.  snapkv_compress_host in addition shares its
 *     side stream and events among all calls on a device: one caller per device at a
 *     time.
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL is the
 *     default stream).  Calls return without synchronising unless stated.  Several of
 *     the kernels are launched with programmatic dependent launch: their blocks may
 *     become resident while the stream's previous kernel - the caller's included - is
 *     still running, but they read and write nothing before that kernel has completed
 *     and its writes are visible, so stream order holds for every buffer.
 *   - Errors come back as a snapkv_status_t; nothing aborts or throws.  Argument
 *     errors are found on the host before anything is launched.
 *   - A device-side wait that exceeds its time limit stops the kernel early and
 *     records SNAPKV_ERR_TIMEOUT in the first word of the workspace; read it with
 *     snapkv_device_status after the stream has drained.
 */
#ifndef SNAPKV_H_
#define SNAPKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SNAPKV_OK = 0,
  SNAPKV_ERR_INVALID_ARG = 1, /* a size, enum or pointer is not acceptable            */
  SNAPKV_ERR_UNSUPPORTED = 2, /* valid for the method, not implemented by the kernels  */
  SNAPKV_ERR_WORKSPACE = 3,   /* workspace missing, misaligned or too small            */
  SNAPKV_ERR_CUDA = 4,        /* a CUDA runtime/driver call or a launch failed         */
  SNAPKV_ERR_TIMEOUT = 5      /* a bounded device-side wait gave up                    */
} snapkv_status_t;

enum { SNAPKV_POOL_MAX = 0, SNAPKV_POOL_AVG = 1 };

/* Supported range: d in {64, 128}; 1 <= W <= 128 and W <= L; pool_kernel odd in
 * [1, 63]; W < budget; Hq % Hkv == 0; B*Hkv*L*d < 2^40.  Anything else that is
 * meaningful for the method returns SNAPKV_ERR_UNSUPPORTED, anything meaningless
 * SNAPKV_ERR_INVALID_ARG. */

/* Human-readable name of a status code (static storage). */
const char* snapkv_status_string(int status);

/* Rows written per head by snapkv_compress: min(budget, L).  Listing 1 returns the
 * cache unchanged when the prompt is not longer than the budget.  Host only. */
int snapkv_out_rows(int L, int budget);

/* Bytes of device scratch snapkv_compress / snapkv_window_scores / snapkv_pool_topk
 * need for these sizes (the maximum over the three); 0 if the arguments are not
 * acceptable.  Host only, no CUDA calls.  The workspace must be 256-byte aligned. */
size_t snapkv_workspace_size(int B, int Hq, int Hkv, int L, int d, int W,
                             int pool_kernel, int pool_type, int budget);

/*
 * The whole step (Listing 1; Sec. 4.1 "vote" then "update and store").
 *   q_obs   bf16 [B, Hq, W, d]   device  the last W prompt queries (post-RoPE)
 *   k, v    bf16 [B, Hkv, L, d]  device  prompt keys / values as cached
 *   out_k/v bf16 [B, Hq, budget, d] device.  Per head: rows [0, ksel) are the selected
 *           prefix rows in ascending position, rows [ksel, budget) the window rows.
 *   out_idx int32 [B, Hq, budget - W] device: the selected prefix positions,
 *           strictly ascending, each in [0, n).
 * Logits are q.k/sqrt(d) with a causal mask inside the window; the softmax
 * normaliser covers every visible key; average pooling divides by pool_kernel;
 * ties go to the lower position.
 * If budget >= L the cache is copied through (expanded to Hq heads): per head rows
 * [0, L) of out_k/out_v are written with row stride unchanged (budget rows per
 * head), out_idx[..., 0:n] = 0..n-1 (row stride budget - W), everything else is
 * left untouched.
 */
snapkv_status_t snapkv_compress(const void* q_obs, const void* k, const void* v,
                                int B, int Hq, int Hkv, int L, int d, int W,
                                int pool_kernel, int pool_type, int budget,
                                void* out_k, void* out_v, int32_t* out_idx,
                                void* workspace, size_t workspace_bytes, void* stream);

/*
 * Steps "score" and "vote" alone (Eq. 1; Listing 1's compute_attn and .sum):
 *   out_vote fp32 [B, Hq, n] device, vote[j] = sum over window rows i of
 *   softmax_i(q_i.k/sqrt(d))[j], j in [0, n).  fp32 accumulation of bf16 products.
 * Requires W < L.
 */
snapkv_status_t snapkv_window_scores(const void* q_obs, const void* k,
                                     int B, int Hq, int Hkv, int L, int d, int W,
                                     float* out_vote,
                                     void* workspace, size_t workspace_bytes, void* stream);

/*
 * Steps "pool" and "top-k" alone (Listing 1's pool1d and topk; Eq. 2) on `rows`
 * independent rows:
 *   vote    fp32 [rows, n] device, finite and >= 0
 *   out_idx int32 [rows, ksel] device, ascending positions of the ksel largest pooled
 *           votes; among equal pooled votes the lower positions win.
 * Requires 1 <= ksel <= n.  `workspace` must hold snapkv_pool_topk_workspace_size
 * bytes (may be NULL when that is 0).
 */
size_t snapkv_pool_topk_workspace_size(int rows, int n);
snapkv_status_t snapkv_pool_topk(const float* vote, int rows, int n,
                                 int pool_kernel, int pool_type, int ksel,
                                 int32_t* out_idx,
                                 void* workspace, size_t workspace_bytes, void* stream);

/*
 * Pool + top-k without any caller-provided scratch.  The paper has no counterpart to this
 * entry point: it exists for hosts that may not allocate device memory at the time of the
 * call - an inference server whose memory pool was sized and frozen at start-up, code
 * running between the launches of a latency-critical decode loop where a cudaMalloc would
 * synchronise the device, or a plug-in that is handed tensors but no allocator.  Same
 * inputs, outputs and result as snapkv_pool_topk; the per-vote keys go into a 16 MiB array
 * that is part of the library image (every GPU that loads the library holds it until the
 * process ends), so rows * n may not exceed SNAPKV_STATIC_MAX_KEYS: larger requests return
 * SNAPKV_ERR_WORKSPACE and launch nothing.  The call allocates and frees nothing.
 * The first call on each device looks up the array's device address (the device must be
 * current); make that first call outside any stream capture.
 * All calls share the one array and it keeps what the last call wrote.  Nothing in it has
 * to start at zero - each launch writes every key before reading it - but two calls whose
 * kernels overlap on the GPU (different streams, no dependency between them) race on it:
 * order them.
 */
#define SNAPKV_STATIC_MAX_KEYS (4 * 1024 * 1024)
snapkv_status_t snapkv_pool_topk_static(const float* vote, int rows, int n,
                                        int pool_kernel, int pool_type, int ksel,
                                        int32_t* out_idx, void* stream);

/*
 * Step "gather + append" alone (Listing 1's gather and cat): with idx int32
 * [B, Hq, ksel] device (positions in [0, L - W)), writes per head the rows k[idx],
 * then the last W rows of k, to out_k [B, Hq, ksel + W, d]; same for v.
 * Byte copies: bit-exact.
 */
snapkv_status_t snapkv_gather(const void* k, const void* v, const int32_t* idx,
                              int B, int Hq, int Hkv, int L, int d, int W, int ksel,
                              void* out_k, void* out_v, void* stream);

/*
 * Supplied-normaliser variant of snapkv_window_scores and snapkv_compress.  The paper's
 * listing recomputes the window rows' softmax after the prompt phase (Listing 1,
 * compute_attn), although the attention kernel of the prompt phase already held each
 * row's normaliser.  Here the caller passes it in: lse_obs, DEVICE fp32 [B, Hq, W],
 * lse_obs[b,h,i] = natural log of the sum over the keys j <= L - W + i of
 * exp(q_obs[b,h,i] . k[b,kv(h),j] / sqrt(d)) (the log-sum-exp flash-attention style
 * kernels return).  Votes are then vote[j] = sum_i exp(logit[i,j] - lse_obs[i]) (Eq. 1
 * with the softmax written out), computed in ONE sweep over K: no statistics pass, half
 * of the exponentials and of the K traffic.  Everything after the vote (pooling, top-k,
 * gather) is the same as in snapkv_compress; with the rows' true log-sum-exp the results
 * agree with it to rounding.  Same arguments, workspace size, errors and ownership as the
 * functions they mirror; lse_obs is read only, must be 4-byte aligned and is consumed by
 * the time the stream's work completes.  A wrong lse_obs scales that row's contribution;
 * nothing checks it.
 */
snapkv_status_t snapkv_window_scores_lse(const void* q_obs, const void* k, const float* lse_obs,
                                         int B, int Hq, int Hkv, int L, int d, int W,
                                         float* out_vote, void* workspace,
                                         size_t workspace_bytes, void* stream);
snapkv_status_t snapkv_compress_lse(const void* q_obs, const void* k, const void* v,
                                    const float* lse_obs,
                                    int B, int Hq, int Hkv, int L, int d, int W,
                                    int pool_kernel, int pool_type, int budget,
                                    void* out_k, void* out_v, int32_t* out_idx,
                                    void* workspace, size_t workspace_bytes, void* stream);

/*
 * The whole step (Listing 1) on caches that are not stored as dense [B, Hkv, L, d].
 * Listing 1 takes key_states / value_states in the framework's [batch, heads, length, d]
 * order; serving stacks often keep the prompt cache as [B, L, Hkv, d], as one fused K/V
 * buffer, or as a slice of a larger allocation.  Here k and v are addressed as
 *   element(b, c, j, t) = base + b * strides[0] + c * strides[1] + j * strides[2] + t
 * with k_strides / v_strides HOST arrays of three element strides (batch, KV head,
 * position), read during the call.  Rows of d elements are contiguous.  Every stride must
 * be positive, a multiple of 8 elements (16 bytes), below 2^39 elements, and the position
 * stride at least d; otherwise SNAPKV_ERR_INVALID_ARG.  k and v need 16-byte aligned bases
 * and may have different strides.  lse_obs may be NULL (the normalisers are recomputed,
 * as in snapkv_compress) or DEVICE fp32 [B, Hq, W] as in snapkv_compress_lse.  q_obs, the
 * outputs (dense, as in snapkv_compress), the workspace size, errors, ownership and the
 * results are those of snapkv_compress: the same tiles reach the same arithmetic in the
 * same order, so the outputs are bit-identical to a call on a dense copy of the cache.
 */
snapkv_status_t snapkv_compress_strided(const void* q_obs, const void* k, const void* v,
                                        const int64_t* k_strides, const int64_t* v_strides,
                                        const float* lse_obs,
                                        int B, int Hq, int Hkv, int L, int d, int W,
                                        int pool_kernel, int pool_type, int budget,
                                        void* out_k, void* out_v, int32_t* out_idx,
                                        void* workspace, size_t workspace_bytes, void* stream);

/*
 * The step with ONE selection per KV head under grouped-query attention, so that the
 * compressed cache keeps Hkv heads instead of being expanded to Hq.  Listing 1 has a single
 * num_heads; here Eq. 1's sum over the window queries runs over the window rows of ALL the
 * query heads of a group: vote_group[b, c, j] = sum over h with kv(h) = c and over window rows
 * i of softmax_i(q[b,h,i] . k[b,c] / sqrt(d))[j], added in ascending head order in fp32.
 * Pooling, top-k (Eq. 2) and the gather then run once per KV head:
 *   out_k/v bf16 [B, Hkv, budget, d], out_idx int32 [B, Hkv, budget - W]  (device)
 * with the row order, ties and identity rule (budget >= L: rows [0, L) copied per KV head)
 * of snapkv_compress.  With Hq == Hkv the results are those of snapkv_compress.
 * k_strides / v_strides: NULL for dense [B, Hkv, L, d], else as in snapkv_compress_strided;
 * lse_obs: NULL, or DEVICE fp32 [B, Hq, W] as in snapkv_compress_lse.  Workspace size,
 * errors and ownership as in snapkv_compress (snapkv_workspace_size with the same
 * arguments: the per-head votes still go through the workspace).
 */
snapkv_status_t snapkv_compress_grouped(const void* q_obs, const void* k, const void* v,
                                        const int64_t* k_strides, const int64_t* v_strides,
                                        const float* lse_obs,
                                        int B, int Hq, int Hkv, int L, int d, int W,
                                        int pool_kernel, int pool_type, int budget,
                                        void* out_k, void* out_v, int32_t* out_idx,
                                        void* workspace, size_t workspace_bytes, void* stream);

/*
 * The whole step (Listing 1) on a batch whose prompts differ in length.  Listing 1 has one
 * q_len for the batch; the sequences are independent of one another (Sec. 4.1), so each is
 * compressed as a single-sequence step of its own length, one after the other on `stream`.
 *   seq_lens       HOST int32 [B]: L_b, W <= L_b <= Lmax.  Sequence b's window is its last W
 *                  positions, its prefix the L_b - W before them.
 *   k, v           as in snapkv_compress_strided (k_strides / v_strides NULL: dense
 *                  [B, Hkv, Lmax, d], each sequence's rows at positions [0, L_b)).
 *   k_seq_offsets / v_seq_offsets  HOST int64 [B] or NULL: element offset of sequence b's
 *                  position 0 of KV head 0 from the base pointer (multiples of 8, >= 0); NULL
 *                  means b * strides[0].  With offsets = Hkv * d * (tokens before b) and
 *                  strides {any, d, Hkv * d} this reads a packed [total_tokens, Hkv, d] cache.
 *   q_obs          bf16 [B, Hq, W, d]: each sequence's own last W queries.
 *   lse_obs        NULL or DEVICE fp32 [B, Hq, W] (as in snapkv_compress_lse, per sequence).
 *   out_k/v        bf16 [B, Hq, budget, d], out_idx int32 [B, Hq, budget - W] (device).
 *                  A sequence with budget >= L_b is copied through as in snapkv_compress: rows
 *                  [0, L_b) written, out_idx[b, :, 0:L_b - W] = 0.., the rest left untouched.
 * The host arrays are read during the call.  All sequences are validated before anything is
 * launched (SNAPKV_ERR_INVALID_ARG; SNAPKV_ERR_WORKSPACE if the workspace is smaller than the
 * largest snapkv_workspace_size(1, Hq, Hkv, L_b, ...) over the sequences with L_b > budget);
 * the status block keeps the first error of any sequence.  Each sequence's result is that of snapkv_compress on that sequence alone.
 */
snapkv_status_t snapkv_compress_varlen(const void* q_obs, const void* k, const void* v,
                                       const int64_t* k_strides, const int64_t* v_strides,
                                       const int64_t* k_seq_offsets, const int64_t* v_seq_offsets,
                                       const int32_t* seq_lens, const float* lse_obs,
                                       int B, int Hq, int Hkv, int Lmax, int d, int W,
                                       int pool_kernel, int pool_type, int budget,
                                       void* out_k, void* out_v, int32_t* out_idx,
                                       void* workspace, size_t workspace_bytes, void* stream);

/*
 * snapkv_compress for callers whose tensors live in host memory (pinned memory
 * gives asynchronous copies).  q_obs, k, v, out_k, out_v, out_idx are HOST pointers
 * with the shapes above (out_k/out_v [B,Hq,budget,d], out_idx [B,Hq,budget-W]).
 * `staging` is DEVICE scratch of at least snapkv_host_staging_size(...) bytes,
 * 256-byte aligned, holding the device copies and the workspace.  Copies in,
 * compresses, copies out; returns after enqueueing (synchronise `stream` before
 * reading the outputs).  The (batch, KV head) pairs are independent (Sec. 4.1: every
 * head selects on its own), so they go through in up to eight parts: a part's
 * results are copied back on a side stream of the library while the next part's
 * inputs are still arriving on `stream`, and `stream` waits for the last copy back
 * before the call's work counts as complete.  The side stream and its events are
 * created on the first call on a device and kept for the life of the process (make
 * that first call outside any stream capture); if they cannot be created everything
 * runs on `stream`.  The status block (snapkv_device_status on the workspace part of
 * `staging`) keeps the first error of any part.
 */
size_t snapkv_host_staging_size(int B, int Hq, int Hkv, int L, int d, int W,
                                int pool_kernel, int pool_type, int budget);
snapkv_status_t snapkv_compress_host(const void* q_obs, const void* k, const void* v,
                                     int B, int Hq, int Hkv, int L, int d, int W,
                                     int pool_kernel, int pool_type, int budget,
                                     void* out_k, void* out_v, int32_t* out_idx,
                                     void* staging, size_t staging_bytes, void* stream);

/*
 * Hit rate of a selection (Sec. 3, Eq. 3-7).  a_cur fp32 [rows, n] device: the attention
 * features of one generated query over the n prefix keys, one row per head; idx int32
 * [rows, k] device: the positions the vote selected (distinct within a row; entries outside
 * [0, n) are ignored); theta: the importance threshold, compared in fp32 with a strict >
 * (Eq. 5).  Writes out_counts int32 [rows, 2] device: per head {sum of O (Eq. 6: selected
 * positions whose feature exceeds theta), sum of M_threshold_cur (features exceeding theta)}.
 * H of Eq. 7 is the ratio of the column sums; the per-row ratios are the per-head rates.
 * Integer counting: exact, independent of scheduling.  Enqueued on `stream` (a clear of
 * out_counts, then one kernel); no workspace.  rows <= 65535.
 */
snapkv_status_t snapkv_hit_counts(const float* a_cur, const int32_t* idx, int rows, int n, int k,
                                  float theta, int32_t* out_counts, void* stream);

/*
 * One generation step's attention over the compressed cache (Sec. 5.1.2: decoding on the
 * compressed keys and values; Sec. 4.1: later steps attend to what the step kept).
 *   q_cur     bf16 [B, Hq, d]        device  the generated token's queries (post-RoPE)
 *   cache_k/v bf16 [B, Hc, rows, d]  device  the compressed cache, every row visible; Hc
 *             divides Hq and query head h reads cache head h / (Hq / Hc): Hc = Hq for the
 *             output of snapkv_compress, Hc = Hkv for that of snapkv_compress_grouped
 *   out       fp32 [B, Hq, d]        device  softmax_j(q . k_j / sqrt(d)) applied to the values
 *   out_lse   fp32 [B, Hq] device or NULL: natural-log sum-exp of the logits (lets the
 *             caller merge with attention over rows kept elsewhere, e.g. newly generated ones)
 * bf16 products accumulated in fp32; the rows are split over many blocks and merged in a
 * fixed order, so results are reproducible run to run.  `workspace`: device scratch of
 * snapkv_decode_workspace_size(B, Hq, rows, d) bytes, 256-byte aligned (0 from the size
 * query means unacceptable arguments).  Enqueued on `stream`: two kernels, no allocation.
 * d must be 64 or 128 (SNAPKV_ERR_UNSUPPORTED otherwise), B * Hq <= 65535.
 */
size_t snapkv_decode_workspace_size(int B, int Hq, int rows, int d);
snapkv_status_t snapkv_decode_attention(const void* q_cur, const void* cache_k, const void* cache_v,
                                        int B, int Hq, int Hc, int rows, int d,
                                        float* out, float* out_lse,
                                        void* workspace, size_t workspace_bytes, void* stream);

/*
 * Synchronises `stream`, reads the status word the kernels keep at the start of
 * `workspace` and returns it (SNAPKV_OK or SNAPKV_ERR_TIMEOUT), or SNAPKV_ERR_CUDA
 * if the stream reports an error.  `detail`, if not NULL, receives a code telling
 * which wait gave up (0 if none).
 */
snapkv_status_t snapkv_device_status(const void* workspace, void* stream, int* detail);

/*
 * The step on a PAGED cache (Listing 1 takes dense key_states / value_states; serving
 * stacks keep the prompt's K and V in fixed-size pages of a shared pool and a per-sequence
 * block table).  Position p of sequence b is row p % page_size of page
 * page_table[b * pages_per_seq + p / page_size].
 *   k_pool, v_pool  bf16, device: the pools.  Addressed as [page][KV head][row][d] with
 *                   element strides k_strides[3] = {page, KV head, row} (v_strides likewise);
 *                   rows of d elements contiguous, strides positive multiples of 8 elements,
 *                   e.g. {Hkv*page_size*d, page_size*d, d} or {page_size*Hkv*d, d, Hkv*d}.
 *   page_table      int32, device, [B][pages_per_seq].  Entries of pages a sequence does
 *                   not reach are never read; an entry outside [0, num_pages) reads as
 *                   zeros.  Pages may be shared between sequences (common prefixes).
 *   page_size       positions per page: a multiple of 128, so that a tile of 128 keys lies in
 *                   one page (SNAPKV_ERR_INVALID_ARG otherwise); pages_per_seq * page_size >= L.
 *   seq_lens        host int32[B] or NULL.  NULL: every sequence has L positions.  Otherwise
 *                   sequence b has seq_lens[b] in [W, L] positions and the call runs one
 *                   single-sequence step per prompt (as snapkv_compress_varlen does), a
 *                   sequence with budget >= its length being copied through.
 *   lse_obs         optional, as in snapkv_compress_lse.
 * What lies in a page behind a sequence's last position is never used (it may be anything).
 * Outputs and workspace as for snapkv_compress (with seq_lens: as for
 * snapkv_compress_varlen; the workspace must hold snapkv_workspace_size(1, Hq, Hkv, L_b, ...)
 * of the longest sequence).  Results are bit-identical to snapkv_compress on a dense copy.
 */
snapkv_status_t snapkv_compress_paged(const void* q_obs, const void* k_pool, const void* v_pool,
                                      const int64_t* k_strides, const int64_t* v_strides,
                                      const int32_t* page_table, int pages_per_seq, int page_size,
                                      int num_pages, const int32_t* seq_lens, const float* lse_obs,
                                      int B, int Hq, int Hkv, int L, int d, int W,
                                      int pool_kernel, int pool_type, int budget,
                                      void* out_k, void* out_v, int32_t* out_idx,
                                      void* workspace, size_t workspace_bytes, void* stream);

/*
 * A prompt sharded along its length (context parallelism).  The paper stops at what one GPU
 * holds (Sec. 5.1.1: 380K tokens; Sec. 6 leaves prompt processing aside); Eq. 1-2 decompose
 * over ranges of keys, which is what these four per-shard steps implement.  A shard holds
 * the keys and values of positions [pos0, pos0 + Ls) of every sequence, dense
 * [B, Hkv, Ls, d], and all shards know q_obs (the last W queries of the whole prompt).  With
 * n = L_total - W the whole prompt's prefix length:
 *
 * 1. snapkv_shard_lse: the shard's share of each window row's softmax normaliser.
 *    out_lse fp32 [B, Hq, W] = log sum over the shard's keys j visible to window row i
 *    (global position pos0 + j <= n + i, i.e. local j <= mask_n + i with mask_n = n - pos0,
 *    which may be negative or exceed Ls) of exp(q_i.k_j / sqrt(d)); -inf where a row sees no
 *    key of the shard.  Requires W <= Ls.
 * 2. snapkv_lse_merge: out[i] = log sum_r exp(parts[r][i]) over R shards' results laid out
 *    [R][count] (count = B*Hq*W), folded in the order of r, so every rank that merges the same
 *    gathered buffer gets the same bits.  This is lse_obs of snapkv_window_scores_lse.
 * 3. snapkv_shard_votes: Eq. 1 for the shard's first n_vote keys (those of its keys that are
 *    prefix keys: min(Ls, n - pos0)) given the merged lse_obs:
 *    out_vote fp32 [B, Hq, n_vote].  Concatenated over the shards these are the votes of the
 *    whole prompt; pooling and top-k then run on the whole rows (snapkv_pool_topk).
 * 4. snapkv_gather_range: the shard's part of the gather.  idx int32 [B, Hq, ksel] holds a
 *    head's selected GLOBAL positions, ascending; the entries inside [pos0, pos0 + Ls) form
 *    one segment.  Their K/V rows are copied to rows [0, count) of out_k/out_v
 *    [B, Hq, out_rows, d], followed by the shard's last `append` rows (the window rows, on
 *    the shard that holds them; 0 elsewhere); seg int32 [B, Hq, 2] = {first entry of the
 *    segment, count}.  out_rows >= min(ksel, Ls) + append.  The whole compressed cache of a
 *    head is the shards' segments in shard order, then the window rows.
 * Workspaces: snapkv_workspace_size(B, Hq, Hkv, Ls, d, W, 1, 0, W + 1) bytes suffice for
 * steps 1 and 3.  Everything else as for the single-GPU entry points.
 */
snapkv_status_t snapkv_shard_lse(const void* q_obs, const void* k_shard,
                                 int B, int Hq, int Hkv, int Ls, int d, int W, int mask_n,
                                 float* out_lse,
                                 void* workspace, size_t workspace_bytes, void* stream);
snapkv_status_t snapkv_lse_merge(const float* parts, int R, int count, float* out, void* stream);
snapkv_status_t snapkv_shard_votes(const void* q_obs, const void* k_shard, const float* lse_obs,
                                   int B, int Hq, int Hkv, int Ls, int d, int W, int n_vote,
                                   float* out_vote,
                                   void* workspace, size_t workspace_bytes, void* stream);
snapkv_status_t snapkv_gather_range(const void* k_shard, const void* v_shard, const int32_t* idx,
                                    int B, int Hq, int Hkv, int Ls, int d, int pos0, int ksel,
                                    int append, void* out_k, void* out_v, int out_rows,
                                    int32_t* seg, void* stream);

/*
 * The scoring kernel's schedule, for inspection (no counterpart in the paper).  The kernel
 * is a persistent grid; every block walks a fixed list of work items - tiles [t0, t1) of 128
 * keys of one unit (a batch, a KV head and up to 128 window columns of its query heads), in
 * the statistics sweep or in the vote sweep of Eq. 1 - and the blocks that share a unit's
 * statistics sweep each publish one partial (slot s of nseg).  This routine runs the
 * kernel's own item walk on the host for block `cta` of `grid`: it writes up to max_items
 * records of six int32 {unit, t0, t1, vote (0/1), slot, nseg} to out_items (host memory)
 * and returns the number of items, or -1 if the arguments are not acceptable.  out_plan,
 * if not NULL, receives eight int32: units, units per wave, waves, tiles per unit in the
 * statistics sweep, tiles per unit in the vote sweep, partial slots per unit, waves the
 * statistics run ahead of the votes, window columns per unit.  Host only, no CUDA calls.
 */
int snapkv_schedule_items(int B, int Hq, int Hkv, int L, int d, int W, int votes_only,
                          int grid, int cta, int32_t* out_items, int max_items,
                          int32_t* out_plan);

/*
 * Time limit of the device-side waits (no counterpart in the paper; the scoring kernel's
 * blocks wait for one another's partial softmax statistics of Eq. 1's normaliser, and for
 * their own copies and tensor-core operations).  Every such wait gives up after `limit_ns`
 * nanoseconds (one second unless changed; values below one millisecond are raised to
 * that); a wait on another block gives up after half of it, so that the detail word
 * names the wait that failed and not one downstream of it.  Process-wide, applies to
 * kernels launched afterwards, returns the previous limit.  Host only.
 */
unsigned long long snapkv_set_wait_limit_ns(unsigned long long limit_ns);

/*
 * Self-test of the time-out path (no counterpart in the paper).  Same arguments as
 * snapkv_window_scores, but only the vote sweep is launched and nothing ever supplies the
 * softmax statistics it waits for: every block's wait runs into the limit, the blocks drain
 * their copies, release tensor memory and return; out_vote is left unwritten.  Afterwards
 * snapkv_device_status(workspace) reports SNAPKV_ERR_TIMEOUT with detail 7 (the wait for a
 * unit's statistics) and the context is usable as before.  The call occupies the GPU for
 * about half the wait limit: lower the limit first (snapkv_set_wait_limit_ns) and restore
 * it afterwards.
 */
snapkv_status_t snapkv_selftest_stalled_scores(const void* q_obs, const void* k,
                                               int B, int Hq, int Hkv, int L, int d, int W,
                                               float* out_vote,
                                               void* workspace, size_t workspace_bytes,
                                               void* stream);

/* Number of kernel launches the last successful snapkv_compress /
 * snapkv_window_scores call of this thread enqueued (for accounting in benchmarks).
 * Host only. */
int snapkv_last_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SNAPKV_H_ */
