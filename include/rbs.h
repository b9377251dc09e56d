/*
 * rbs.h -- C ABI of the RBS-Attention prefill hot path for NVIDIA B200 (sm_100a).
 *
 * Three calls per layer follow Algorithm 1 of the paper:
 *   rbs_block_stats     key-block centroids and radii                    (Sec. 3.1)
 *   rbs_select          rescue coefficients, dual-branch block selection (Sec. 3.1-3.2)
 *   rbs_sparse_prefill  causal block-sparse attention over the mask      (Sec. 3.3, Eq. 1 when dense)
 *
 * Conventions for every entry point
 *   - All data pointers are DEVICE pointers unless a parameter says "host".  The caller owns every
 *     buffer; the library allocates nothing on these paths and keeps no state between calls.
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = the legacy default
 *     stream) and the call returns without waiting for it.
 *   - Argument errors are detected on the host before anything is launched and reported through
 *     the return value; nothing is written in that case.  There is no CPU fallback.
 *   - Q/K/V/O are bf16 tensors with the head dimension contiguous, addressed as
 *       element(l, t, h, j) = ptr[l*stride_batch + t*stride_token + h*stride_head + j]
 *     (strides in elements, multiples of 8; ptr 16-byte aligned).  The natural layout is
 *     [batch][token][head][head_dim].  `batch` is prompts x layers: every (batch, KV head) is an
 *     independent problem.
 *   - Notation: N = seqlen, B = block, M = ceil(N / B) blocks (a short last block is allowed), Hq / Hkv query / KV heads,
 *     G = Hq / Hkv, query head h reads KV head h / G, d = head_dim, W = ceil(M / 32).
 *   - Supported: head_dim == 128, block in {64, 128, 256}, seqlen positive,
 *     Hq a multiple of Hkv, M <= 8192.  Anything else returns RBS_ERR_UNSUPPORTED.
 */
#ifndef RBS_H_
#define RBS_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define RBS_API __attribute__((visibility("default")))
#else
#define RBS_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  RBS_OK = 0,
  RBS_ERR_INVALID_ARG = 1, /* null pointer, misaligned pointer or stride, alpha <= 0, negative count */
  RBS_ERR_UNSUPPORTED = 2, /* shape outside the supported set listed above */
  RBS_ERR_WORKSPACE = 3,   /* workspace missing or smaller than rbs_workspace_bytes() */
  RBS_ERR_CUDA = 4,        /* a CUDA runtime / driver call failed (launch, tensor-map encode, ...) */
  RBS_ERR_TIMEOUT = 5,     /* a bounded device-side wait gave up  */
  RBS_ERR_DEBUG_CHECK = 6  /* debug build only: a device-side index check failed (rbs_device_status) */
} rbs_status;

typedef struct {
  int batch;      /* L: prompts x layers */
  int seqlen;     /* N */
  int n_q_heads;  /* Hq */
  int n_kv_heads; /* Hkv */
  int head_dim;   /* d */
  int block;      /* B: block size of queries and of keys (Sec. 4.4: 128 by default) */
} rbs_shape;

typedef struct {
  void* ptr;            /* device, bf16 */
  int64_t stride_batch; /* elements */
  int64_t stride_token;
  int64_t stride_head;
} rbs_tensor;

/* Per-block key statistics (Sec. 3.1), all device fp32, dense row-major in the index order shown. */
typedef struct {
  float* centroid; /* [L][Hkv][M][d]  c_b = mean of the block's keys */
  float* radius;   /* [L][Hkv][M]     r_b = max_k ||k - c_b||_2 */
  float* beta;     /* [L][Hkv][M]     rescue coefficient, Eq. (beta) */
  float* rq;       /* [L][Hkv][2]     (r_low, r_high) = radius quantiles 0.5 and 0.9 */
} rbs_stats;

/* Per-block coordinate-wise key minima and maxima (App. D.2: a_b, u_b), device fp32, the statistics of the Quest-style
 * comparison selector. */
typedef struct {
  float* lo; /* [L][Hkv][M][d]  a_bj = min over the block's keys of k_j */
  float* hi; /* [L][Hkv][M][d]  u_bj = max over the block's keys of k_j */
} rbs_box;

enum { RBS_OP_BLOCK_STATS = 0, RBS_OP_SELECT = 1, RBS_OP_SPARSE_PREFILL = 2, RBS_OP_SELECT_BOX = 3 };

/* Bytes of device workspace the given call needs for this shape (0 if none).  Workspace must be
 * 256-byte aligned; its contents need not be initialised and are undefined afterwards. */
RBS_API size_t rbs_workspace_bytes(int op, const rbs_shape* shape);

/*
 * Sec. 3.1 / Algorithm 1, first loop.  Reads K once and writes, for every (l, KV head, block b),
 *   stats.centroid = (1/B) sum of the block's keys                  (fp32 accumulation of bf16 keys)
 *   stats.radius   = max over the block's keys of ||k - c_b||_2     (difference form, fp32)
 * stats.beta and stats.rq are not touched.  Needs no workspace.
 */
RBS_API rbs_status rbs_block_stats(const rbs_shape* shape, rbs_tensor K, rbs_stats stats, void* stream);

/*
 * Sec. 3.1-3.2 / Algorithm 1, second and third loops.
 *   1. per (l, KV head): r_low = quantile(r, 0.5), r_high = quantile(r, 0.9) (linear interpolation
 *      between order statistics at p*(M-1)); beta_b = clamp((r_b - r_low)/(r_high - r_low), 0, 1),
 *      beta = 0 when r_high <= r_low.  Written to stats.rq and stats.beta.
 *   2. per (l, query head h, query block i), for every causal key block b <= i:
 *        S_base[i,b]   = sum_{t in Q_i} exp( q_t.c_b / sqrt(d) - m )
 *        S_rescue[i,b] = sum_{t in Q_i} exp((q_t.c_b + ||q_t|| r_b beta_b) / sqrt(d) - m')
 *      (Eq. base_score, rescue_score, block_aggregation; evaluated as per-block log-sum-exp), then
 *        keep b  iff  S_base >= alpha_base * max_b' S_base   or   S_rescue >= alpha_rescue * max_b' S_rescue
 *        or b is forced: b < n_sink, or i - n_local < b <= i, or i >= M - n_recent
 *      (Eq. branch_thresholds and the mask union).
 *   3. density[l][h] = kept causal pairs / (M (M+1) / 2)              (Eq. actual_density).
 * stats.centroid and stats.radius are inputs (from rbs_block_stats).
 * mask: uint32 [L][Hq][M][W]; key block b of query block i is bit (b % 32) of word b / 32; bits
 *   with b > i are written as 0.  dbg_base_mask / dbg_rescue_mask (same layout) receive the two
 *   branch masks before the union when non-NULL.
 * alpha > 1 disables that branch (empty set).  alpha must be > 0.
 * Workspace: rbs_workspace_bytes(RBS_OP_SELECT, shape).
 */
RBS_API rbs_status rbs_select(const rbs_shape* shape, rbs_tensor Q, rbs_stats stats, float alpha_base,
                      float alpha_rescue, int n_sink, int n_local, int n_recent, uint32_t* mask,
                      float* density, uint32_t* dbg_base_mask, uint32_t* dbg_rescue_mask,
                      void* workspace, size_t workspace_bytes, void* stream);

/*
 * Sec. 3.3 / Algorithm 1, last step; Eq. (1) when mask == NULL.
 * For token t of query block i and query head h:
 *   O_t = sum_j softmax_j(q_t.k_j * scale) v_j  over keys j <= t whose block is set in mask row (l,h,i),
 * the softmax normalised over those retained keys only.  bf16 inputs, fp32 accumulation and
 * softmax, bf16 output.  mask == NULL selects every causal block (the dense baseline, density 1).
 * Mask bits with b > i are ignored.  A row with no retained key outputs zeros and lse = -inf.
 * lse (nullable): fp32 [L][Hq][N], natural-log-sum-exp of the scaled retained logits.
 * softmax_scale == 0 means 1/sqrt(d).
 * Workspace: optional (NULL / 0: none).  With mask != NULL, block >= 128 and a workspace of at least
 * rbs_workspace_bytes(RBS_OP_SPARSE_PREFILL, shape) bytes (256-byte aligned; RBS_ERR_WORKSPACE if too small or
 * misaligned) the call derives a schedule from the mask first -- per-row counts of selected blocks, rows of more than
 * 256 key tiles of 128 cut into up to 4 parts of equal length (the index compaction of Sec. 3.3's cost paragraph,
 * O(M K_avg) entries, reduced to what the kernel needs) -- runs the parts as separate thread blocks and merges their
 * partial results in a fixed order (bitwise repeatable; the cut depends only on the row, so a row gives the same
 * bits in a whole-sequence call and in any chunked call that is also given a workspace; against a call without
 * workspace a cut row agrees to rounding only).  This pays when a call is short next to its longest rows, as chunked
 * calls are (the last 64 query blocks of a 128K layer: 1.4 against 2.3 ms); on a whole 128K layer it costs about 2 %.
 * The size depends on the shape only: one buffer serves the whole-sequence call and every chunked call.
 */
RBS_API rbs_status rbs_sparse_prefill(const rbs_shape* shape, rbs_tensor Q, rbs_tensor K, rbs_tensor V,
                              const uint32_t* mask, rbs_tensor O, float* lse, float softmax_scale,
                              void* workspace, size_t workspace_bytes, void* stream);

/*
 * The same two steps for a range of query blocks only (chunked prefill; prefill against a key/value prefix).
 * Algorithm 1 treats every query block independently (its third loop and the sparse attention), so a caller may
 * process the queries of tokens [q_start_block * B, q_start_block * B + n_q_tokens) in one call and the rest in
 * others, against the keys / values / statistics of the whole sequence (`shape->seqlen` tokens; keys after a query
 * are hidden by causality, so they need not be final yet).  In these calls
 *   - Q, O hold only the chunk's tokens (token 0 of the tensor = first token of the chunk), lse is [L][Hq][n_q_tokens];
 *   - mask / debug masks are [L][Hq][Mq][W] with Mq = ceil(n_q_tokens / B) rows (row 0 = query block q_start_block)
 *     and W = ceil(M / 32) words per row as usual;
 *   - density[l][h] = kept pairs of the chunk / causal pairs of the chunk (sum over its query blocks i of i + 1);
 *   - the "recent" rule still refers to the last n_recent query blocks of the whole sequence.
 * The chunk must start on a block boundary, lie inside the sequence, and may end inside a block only at the end of
 * the sequence (RBS_ERR_INVALID_ARG otherwise).  rbs_select_chunk recomputes stats.beta / stats.rq from all M radii on
 * every call.  With q_start_block = 0 and n_q_tokens = seqlen they are rbs_select / rbs_sparse_prefill.
 */
RBS_API rbs_status rbs_select_chunk(const rbs_shape* shape, int q_start_block, int n_q_tokens, rbs_tensor Q,
                                    rbs_stats stats, float alpha_base, float alpha_rescue, int n_sink, int n_local,
                                    int n_recent, uint32_t* mask, float* density, uint32_t* dbg_base_mask,
                                    uint32_t* dbg_rescue_mask, void* workspace, size_t workspace_bytes, void* stream);
RBS_API rbs_status rbs_sparse_prefill_chunk(const rbs_shape* shape, int q_start_block, int n_q_tokens, rbs_tensor Q,
                                            rbs_tensor K, rbs_tensor V, const uint32_t* mask, rbs_tensor O, float* lse,
                                            float softmax_scale, void* workspace, size_t workspace_bytes, void* stream);

/*
 * The selector variants the paper compares with in a shared backend (Sec. 4.2, the selector ablation), through
 * the same kernels:
 *   RBS_SELECTOR_RBS            the method itself; identical to rbs_select.
 *   RBS_SELECTOR_CENTROID_ONLY  mean-only scoring: beta = 0 everywhere, one relative threshold alpha_base on the
 *                               centroid score (alpha_rescue is ignored), union with the forced blocks.
 *   RBS_SELECTOR_FULL_L2        the unattenuated bound of Eq. (full_l2_bound) as a single ranking score: beta = 1
 *                               everywhere, one relative threshold alpha_rescue (alpha_base is ignored), union with
 *                               the forced blocks.
 * stats.beta receives the beta actually used; stats.rq the quantiles (computed in every variant).
 * Everything else is as for rbs_select.
 */
typedef enum { RBS_SELECTOR_RBS = 0, RBS_SELECTOR_CENTROID_ONLY = 1, RBS_SELECTOR_FULL_L2 = 2 } rbs_selector;
RBS_API rbs_status rbs_select_variant(const rbs_shape* shape, rbs_tensor Q, rbs_stats stats, rbs_selector which,
                                      float alpha_base, float alpha_rescue, int n_sink, int n_local, int n_recent,
                                      uint32_t* mask, float* density, uint32_t* dbg_base_mask,
                                      uint32_t* dbg_rescue_mask, void* workspace, size_t workspace_bytes,
                                      void* stream);

/*
 * The Quest-style comparison selector of the paper's ablation (Sec. 4.2; App. D.2, Eq. quest_box), in the same backend.
 *   rbs_block_stats_box  as rbs_block_stats, and from the same single read of K also box.lo / box.hi: the
 *                        per-coordinate minimum and maximum of each block's keys.
 *   rbs_select_box       block logit = the box upper bound  U_b(q) = sum_j max(q_j a_bj, q_j u_bj) = q.v_b + |q|.h_b
 *                        (v_b, h_b the box centre and half-width), aggregated over the query block's tokens exactly as the
 *                        other selectors' logits are (Eq. block_aggregation); query block i then keeps its
 *                        ceil(density_param * (i + 1)) best causal key blocks -- blocks whose score equals the last kept
 *                        one included -- united with the forced blocks of rbs_select.
 * The paper states the policy only as "per-dimension key minima/maxima and query-dependent block selection" with a
 * "density parameter" (0.0405 in its comparison); aggregation and the meaning of the parameter are this library's
 * reading.  mask, density: as rbs_select.  dbg_chosen_mask (nullable): the choice before the union with the forced
 * blocks.  Blocks of 64 and 128 only (RBS_ERR_UNSUPPORTED for 256).  density_param in (0, 1].
 * Workspace: rbs_workspace_bytes(RBS_OP_SELECT_BOX, shape).
 */
RBS_API rbs_status rbs_block_stats_box(const rbs_shape* shape, rbs_tensor K, rbs_stats stats, rbs_box box, void* stream);
RBS_API rbs_status rbs_select_box(const rbs_shape* shape, rbs_tensor Q, rbs_box box, double density_param, int n_sink,
                                  int n_local, int n_recent, uint32_t* mask, float* density, uint32_t* dbg_chosen_mask,
                                  void* workspace, size_t workspace_bytes, void* stream);

/*
 * rbs_select for callers that have no device memory to hand over and must not allocate any.
 * (The paper has no counterpart: this is a packaging variant of rbs_select, same arithmetic, same outputs.)
 *
 * Who needs it: code that runs after the application has claimed the whole GPU for its own pools (a
 * serving engine that sized its KV cache to the last free byte, so a cudaMalloc would fail or evict),
 * code on a latency-critical path where the implicit device-wide synchronisation of cudaMalloc/cudaFree
 * is not acceptable, and plug-ins that are called from inside someone else's memory-managed region and
 * are simply not given an allocator.  Such callers still pass Q, the statistics and the output buffers;
 * only the scratch space differs.
 *
 * The scratch lives in a fixed array of RBS_SELECT_STATIC_SCRATCH_BYTES inside the library's device
 * image: every GPU on which the library is loaded holds that much memory until the process exits.
 * Shapes whose rbs_workspace_bytes(RBS_OP_SELECT) exceed it are rejected with RBS_ERR_WORKSPACE and
 * nothing is launched (the limit covers about 8,100 centroid rows = batch * n_kv_heads * M rounded up to 128,
 * e.g. one 128K-token layer with 4 KV heads at block 128 needs about half of it).
 * The call itself performs no cudaMalloc / cudaFree and calls no allocating library routine.
 * The first call on each device looks up the array's device address (and, like any first use of a CUDA
 * module, lets the driver load the kernels, which is also when the driver places the array in device memory);
 * make that first call outside stream capture and before the application claims the rest of the device's memory --
 * a caller that has already taken every free byte gets RBS_ERR_CUDA from it.
 * All calls on one device share the one array: it keeps whatever the previous call left there, the
 * parts that must start at zero are cleared by every call, and two calls whose kernels may overlap on
 * the GPU (different streams without an ordering between them) race on it -- order them.
 * Calls to rbs_select with a caller-owned workspace are unaffected.
 * Arguments, outputs and error codes are those of rbs_select.
 */
#define RBS_SELECT_STATIC_SCRATCH_BYTES (4u << 20)
RBS_API rbs_status rbs_select_static(const rbs_shape* shape, rbs_tensor Q, rbs_stats stats, float alpha_base,
                                     float alpha_rescue, int n_sink, int n_local, int n_recent, uint32_t* mask,
                                     float* density, uint32_t* dbg_base_mask, uint32_t* dbg_rescue_mask,
                                     void* stream);

/*
 * Group-shared masks under grouped-query attention: replaces, in place, the mask rows of the G query heads that
 * share a KV head by their union, and recomputes density.  The paper's selector is applied per query head
 * (Sec. 3.2: the scores S are taken over one head's query block); sharing the union inside a KV group is a
 * variant with no counterpart in the paper: every head of the group then attends the same key blocks, so a
 * kernel can fetch each selected K/V block once per group, at the price of a higher density.
 *   mask    device, [batch][n_q_heads][Mq][W] as written by rbs_select / rbs_select_chunk; updated in place
 *   density device, [batch][n_q_heads] fp32, overwritten: kept pairs / causal pairs of the call's query blocks
 *           (the same value for the G heads of a group)
 *   q_start_block, n_q_tokens: the query range the mask covers, as in rbs_select_chunk (n_q_tokens < 0: the whole
 *           sequence).
 * Errors as rbs_select_chunk.  Asynchronous on `stream`; no workspace.
 */
RBS_API rbs_status rbs_mask_group_union(const rbs_shape* shape, int q_start_block, int n_q_tokens, uint32_t* mask,
                                        float* density, void* stream);

/*
 * rbs_sparse_prefill for group-shared masks: the caller states that the G query heads of every KV group have identical
 * mask rows (as rbs_mask_group_union leaves them).  Two heads of a group are then served by one thread block that brings
 * every selected K/V tile into shared memory once for both (head-packed query tiles), instead of once per head.  The
 * paper's selector is per query head (Sec. 3.2), so this execution variant has no counterpart there; the attention it
 * computes is Sec. 3.3's.  Arguments and outputs as rbs_sparse_prefill (whole sequence only, no workspace); the mask is
 * read from the first head of each pair.  Needs block >= 128 and an even group size (RBS_ERR_UNSUPPORTED otherwise)
 * and a mask (RBS_ERR_INVALID_ARG for NULL).
 */
RBS_API rbs_status rbs_sparse_prefill_grouped(const rbs_shape* shape, rbs_tensor Q, rbs_tensor K, rbs_tensor V,
                                              const uint32_t* mask, rbs_tensor O, float* lse, float softmax_scale,
                                              void* stream);

/*
 * A batch of prompts of different lengths packed back to back along the token axis (no padding).  Every prompt is
 * selected and attended on its own, exactly as by rbs_block_stats + rbs_select + rbs_sparse_prefill on its rows
 * (Sec. 4.1: requests are not concatenated into one causal sequence); results are bit-identical to those calls.
 *   cu_seqlens   HOST array of n_prompts + 1 ints: cu_seqlens[0] = 0, prompt k holds tokens [cu_seqlens[k], cu_seqlens[k+1])
 *   Q, O         packed [T][Hq][d]; K, V packed [T][Hkv][d] (stride_token, stride_head in elements; stride_batch ignored)
 *   density      device, [n_prompts][Hq] fp32
 *   workspace    device, rbs_varlen_workspace_bytes(...) bytes, 256-byte aligned: statistics, mask and selector scratch
 *                of the longest prompt, reused from prompt to prompt in stream order (nothing is allocated, no tensor
 *                outlives the call; the per-prompt masks and statistics are not returned).
 * Errors: RBS_ERR_INVALID_ARG for a malformed cu_seqlens (not starting at 0, not strictly increasing), otherwise as the
 * three calls.  All prompts are enqueued on `stream` one after the other.
 */
RBS_API size_t rbs_varlen_workspace_bytes(int n_prompts, const int* cu_seqlens, int n_q_heads, int n_kv_heads,
                                          int head_dim, int block);
RBS_API rbs_status rbs_prefill_varlen(int n_prompts, const int* cu_seqlens, int n_q_heads, int n_kv_heads, int head_dim,
                                      int block, rbs_tensor Q, rbs_tensor K, rbs_tensor V, rbs_tensor O, float alpha_base,
                                      float alpha_rescue, int n_sink, int n_local, int n_recent, float* density,
                                      void* workspace, size_t workspace_bytes, void* stream);

/*
 * Kernels that wait on hardware barriers (TMA arrival, tensor-core completion) give every wait an
 * iteration limit.  A wait that runs out records a non-zero code in a device-side status word, lets the
 * kernel drain and return, and leaves the CUDA context usable; outputs of that launch are then
 * undefined.  This call synchronises `stream`, reads the word into *code_out (nullable) and, if
 * `clear` is non-zero, resets it.  Returns RBS_OK when the word is 0, RBS_ERR_TIMEOUT for a wait that ran out
 * (codes 1 .. 7: which kind of wait) and RBS_ERR_DEBUG_CHECK for a failed index check of the debug build
 * (code 0x100 + site; the library built with -DRBS_DEBUG checks the indices of its writes and of its
 * tile walks and skips an access that fails; the release build has no such checks).
 * (No counterpart in the paper: an operational check.)
 */
RBS_API rbs_status rbs_device_status(void* stream, unsigned int* code_out, int clear);

/* Human-readable name of a status code (static storage, never NULL). */
RBS_API const char* rbs_status_string(rbs_status status);

/* Library version string (static storage), e.g. for logging next to measurements. */
RBS_API const char* rbs_version(void);

#ifdef __cplusplus
}
#endif
#endif /* RBS_H_ */
