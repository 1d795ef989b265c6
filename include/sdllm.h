/*
 * libsdllm — cache refresh and sparse block attention for diffusion LLMs (Sparse-dLLM), C ABI.
 *
 * One layer, one decoding block. At the refresh step of a block (cache_state 1 of the paper's
 * Algorithm 2) the block's b query rows attend over the whole bidirectional K/V, a saliency score
 * per key is reduced over the block queries and pooled along the key axis, a per-KV-head top-k at
 * the retention ratio r picks the prefix/suffix entries to keep, and the kept K/V rows are gathered
 * into a compacted cache (Algorithm 1). Every later step of the block (cache_state 2, Algorithm 3)
 * attends over Concat(K_c, K_n): the compacted cache followed by the block's fresh K/V.
 *
 * Conventions for every call
 *   - All data pointers are DEVICE pointers unless a parameter says "host". The library never
 *     allocates, frees or keeps a pointer; buffers and workspace belong to the caller.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL = default stream).
 *     No call synchronises with the host.
 *   - Layout: the last axis (head_dim, D) is contiguous. The other axes (batch, head, position) are
 *     addressed through the *_stride arrays of sdllm_desc, given in ELEMENTS. Every base pointer and
 *     every stride*element_size must be a multiple of 16 bytes.
 *   - Query head h reads KV head h / G, G = n_q_heads / n_kv_heads.
 *   - Arguments are validated on the host before anything is launched: a bad argument returns a
 *     status and launches nothing. Kernels never trap or assert.
 *   - Positions >= seq_len[i] of sequence i are padding and are ignored.
 */
#ifndef SDLLM_H_
#define SDLLM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SDLLM_VERSION 100

typedef enum {
  SDLLM_OK = 0,
  SDLLM_ERR_INVALID_ARG = 1, /* null/misaligned pointer, inconsistent shape, even pool window, r outside [0,1] ... */
  SDLLM_ERR_UNSUPPORTED = 2, /* shape or mode outside what the kernels cover, or not an sm_100 device */
  SDLLM_ERR_WORKSPACE = 3,   /* workspace NULL or smaller than sdllm_workspace_bytes() */
  SDLLM_ERR_CUDA = 4,        /* a CUDA runtime call or launch failed */
  SDLLM_ERR_TIMEOUT = 5      /* a bounded device-side wait gave up (sdllm_read_status) */
} sdllm_status;

typedef enum { SDLLM_F32 = 0, SDLLM_BF16 = 1 } sdllm_dtype;

/* Saliency of a candidate key (Algorithm 1, "Calculate attention scores").
 * LOGIT_MEAN: a_c = scale * <Mean(Q_b), k_c>, the pre-softmax score of the paper's equation and pseudocode.
 * PROB_MEAN : a_c = mean over the block queries of softmax(scale * Q_b K^T)[., c], normalised over all keys. It costs a
 *             second pass over K, needs `out` (the attention output) to be requested with the scores, and is available
 *             for bf16 with block lengths that are multiples of 16 (other shapes: SDLLM_ERR_UNSUPPORTED). */
typedef enum { SDLLM_SCORE_LOGIT_MEAN = 0, SDLLM_SCORE_PROB_MEAN = 1 } sdllm_score_kind;

/* Key-axis pooling (Algorithm 1, MaxPool1D with kernel_size = s, padding = s/2, stride 1). AVG is the
 * paper's AvgPool ablation: padding counts as zero and the divisor is always s. */
typedef enum { SDLLM_POOL_MAX = 0, SDLLM_POOL_AVG = 1 } sdllm_pool_kind;

/* How many entries are kept and from where.
 * JOINT_FLOOR     : Algorithm 1 as printed. One top-n over Concat(prefix, suffix), n = floor((L-b)*r);
 *                   the pooling window runs across the prefix/suffix seam.
 * PER_REGION_CEIL : ceil(r*o) from the prefix and ceil(r*(L-o-b)) from the suffix, pooled per region.
 * PREFIX_ONLY     : Algorithm 5 (prefix-sparse). floor(o*r) from the prefix, the whole suffix is kept. */
typedef enum { SDLLM_SELECT_JOINT_FLOOR = 0, SDLLM_SELECT_PER_REGION_CEIL = 1, SDLLM_SELECT_PREFIX_ONLY = 2 } sdllm_select_mode;

typedef enum {
  SDLLM_OP_REFRESH_SCORES = 0,
  SDLLM_OP_SELECT_TOPK = 1,
  SDLLM_OP_COMPACT_KV = 2,
  SDLLM_OP_SPARSE_BLOCK_ATTN = 3,
  SDLLM_OP_DENSE_ATTN = 4,
  SDLLM_OP_SELECT_COMPACT = 5
} sdllm_op;

/* Problem description, filled by the caller. Plain data; set struct_size = sizeof(sdllm_desc). */
typedef struct sdllm_desc {
  uint32_t struct_size;
  int32_t batch;        /* B: independent sequences */
  int32_t n_q_heads;    /* Hq */
  int32_t n_kv_heads;   /* Hkv, divides Hq */
  int32_t head_dim;     /* D: 64 or 128 */
  int32_t seq_len_max;  /* padded length of the position axis of k, v and pooled_scores (>= every seq_len[i]) */
  int32_t block_len;    /* b: rows of the current decoding block; b * G <= 256 */
  int32_t dtype;        /* sdllm_dtype of q, k, v, out, k_c, v_c */
  float softmax_scale;  /* 0 selects 1/sqrt(D) */
  int32_t pool_window;  /* s: odd, >= 1 */
  int32_t pool;         /* sdllm_pool_kind */
  int32_t score;        /* sdllm_score_kind */
  int32_t select;       /* sdllm_select_mode */
  int32_t n_keep_max;   /* rows per (sequence, KV head) of kept_idx, k_c and v_c; kept counts are clamped to it */
  double retention;     /* r in [0, 1] */
  /* strides in elements for the (batch, head, position) axes */
  int64_t q_stride[3];   /* q_blk  [B, Hq,  b,          D] */
  int64_t kv_stride[3];  /* k, v   [B, Hkv, seq_len_max, D] */
  int64_t o_stride[3];   /* out    [B, Hq,  b,          D] */
  int64_t c_stride[3];   /* k_c,v_c[B, Hkv, n_keep_max, D] */
  int64_t blk_stride[3]; /* k_blk,v_blk [B, Hkv, b,     D] */
} sdllm_desc;

/* Library version (SDLLM_VERSION of the build). */
int sdllm_version(void);

/* Static, human-readable name of a status code. */
const char* sdllm_status_string(sdllm_status status);

/* Bytes of device workspace a call of `op` needs for this description (host-only, no GPU needed).
 * Returns 0 for an invalid description or when the op needs none. The workspace needs 256-byte alignment and the
 * caller zeroes ALL of it once after allocating it: its first 4 bytes are a status word (see sdllm_read_status) and
 * it holds completion counters that every call leaves at zero again; the rest is unspecified after a call. One
 * workspace may serve any number of calls that run one after another on the GPU, never two that overlap.
 * After a call whose status word reads non-zero (SDLLM_ERR_TIMEOUT) zero the whole workspace again before reusing it:
 * the status word is sticky, and the call that gave up may have left its counters anywhere. */
size_t sdllm_workspace_bytes(const sdllm_desc* desc, int op);

/* Host-only. Number of cache entries kept for a sequence of length seq_len whose block starts at block_off:
 * n = floor(|I| * r) of Algorithm 1 (or the other policies of sdllm_select_mode), products taken in double.
 * n_total is always written; n_prefix / n_suffix receive the per-region quotas, or -1 when the split is data
 * dependent (JOINT_FLOOR). Not clamped to n_keep_max. Any output pointer may be NULL. */
sdllm_status sdllm_keep_count(const sdllm_desc* desc, int32_t seq_len, int32_t block_off, int32_t* n_total,
                              int32_t* n_prefix, int32_t* n_suffix);

/* Host-only. Cache state of step i within a block for delay step x (Algorithm 2 is x = 1; Algorithm 4 general):
 * 0 = dense step (cache unused), 1 = refresh (run Algorithm 1), 2 = reuse the compacted cache. */
int32_t sdllm_cache_state(int32_t step_in_block, int32_t delay);

/* Host-only. Number of kernels one call of `op` launches for this description (refresh with all outputs requested);
 * -1 for an invalid description or op. Lets a caller account for its launches without tracing them. */
int32_t sdllm_launch_count(const sdllm_desc* desc, int op);

/* Host-only; the paper has no counterpart. Writes a short NUL-terminated description of the launch plan of an attention
 * call (`op` = SDLLM_OP_REFRESH_SCORES or SDLLM_OP_SPARSE_BLOCK_ATTN) into buf[0..buf_bytes): the kernel's name first,
 * then its grid in words, e.g. "attn_kt_kernel splits=6 cluster=6 stages=1 threads=192". For logs and for naming the
 * kernel a measurement belongs to; the text is not a stable format. The plan depends on the current device's SM
 * count and on sdllm_tuning_set. Returns SDLLM_ERR_INVALID_ARG for a bad description, op, or a NULL / empty buffer. */
sdllm_status sdllm_plan_describe(const sdllm_desc* desc, int op, char* buf, size_t buf_bytes);

/* Reads the device status word kept in the first 4 bytes of an attention workspace. The kernels bound every wait
 * on a shared-memory barrier; if one ever expires they record a non-zero code there and run to the end instead of
 * hanging (the outputs of that call are then invalid). The caller zeroes those 4 bytes once after allocating the
 * workspace. This call copies the word to the host and SYNCHRONISES the stream (the only call that does).
 * Returns SDLLM_OK when the word is zero, SDLLM_ERR_TIMEOUT otherwise; *device_status receives the raw code. */
sdllm_status sdllm_read_status(const void* workspace, void* cuda_stream, int32_t* device_status);

/* Refresh step, part 1 (cache_state 1; Algorithm 1 up to the importance scores).
 *   out[i, h, :, :]  = softmax(scale * Q_b K^T) V for the block rows over ALL seq_len[i] keys (prefix+block+suffix)
 *   lse[i, h, :]     = log-sum-exp of the scaled logits per row            [B, Hq, b] fp32, nullable
 *   pooled_scores    = importance I after saliency + key-axis pooling      [B, Hkv, seq_len_max] fp32, nullable;
 *                      indexed by ABSOLUTE position; block positions and padding hold -inf.
 * `out` may be NULL (scores only). seq_len NULL means every sequence has seq_len_max keys. block_off[i] = o.
 * The probability matrix is never written to memory. */
sdllm_status sdllm_refresh_scores(const sdllm_desc* desc, const void* q_blk, const void* k, const void* v,
                                  const int32_t* seq_len, const int32_t* block_off, void* out, float* lse,
                                  float* pooled_scores, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Refresh step, part 2 (Algorithm 1, "n <- floor(|I| r)", "TopKIndices"). Per (sequence, KV head): the n
 * candidates with the largest pooled score; equal scores go to the lower position; written as ascending
 * absolute positions into kept_idx [B, Hkv, n_keep_max] int32, entries past the count are -1.
 * kept_cnt [B] int32 receives min(n, n_keep_max) (the same for every head of a sequence). */
sdllm_status sdllm_select_topk(const sdllm_desc* desc, const float* pooled_scores, const int32_t* seq_len,
                               const int32_t* block_off, int32_t* kept_idx, int32_t* kept_cnt, void* workspace,
                               size_t workspace_bytes, void* cuda_stream);

/* Refresh step, part 3 (Algorithm 1, "Select" and the cache store): k_c[i, g, j, :] = k[i, g, kept_idx[i, g, j], :],
 * same for v, bit-exact. Rows j >= kept_cnt[i] are zero-filled. */
sdllm_status sdllm_compact_kv(const sdllm_desc* desc, const void* k, const void* v, const int32_t* kept_idx,
                              const int32_t* kept_cnt, void* k_c, void* v_c, void* cuda_stream);

/* Refresh step, parts 2 and 3 in one call (Algorithm 1 from "n <- floor(|I| r)" to the cache store): exactly the results of
 * sdllm_select_topk followed by sdllm_compact_kv - the same kept_idx, kept_cnt, k_c and v_c, bit for bit - but, while the
 * candidates of a head fit the shared memory of a CTA (seq_len_max - block_len <= 8192), in ONE launch: the CTAs that
 * select a head's entries copy its rows themselves, so the index list makes no round trip through memory. Longer
 * sequences run the two kernels one after the other inside this call (sdllm_launch_count tells which). The launch may
 * start while the kernel in front of it in the stream is finishing and reads pooled_scores only once that kernel has
 * completed; it holds its own dependents back until it has completed, so the reuse step that follows may read the
 * compacted cache early (see sdllm_sparse_block_attn). seq_len and block_off are older than the scores (the refresh
 * attention in front has read them too) and are read early, under the rule stated at sdllm_sparse_block_attn: only a
 * caller's own kernel that releases its dependents early must not be the one that writes them directly in front. */
sdllm_status sdllm_select_compact(const sdllm_desc* desc, const float* pooled_scores, const int32_t* seq_len,
                                  const int32_t* block_off, const void* k, const void* v, int32_t* kept_idx,
                                  int32_t* kept_cnt, void* k_c, void* v_c, void* cuda_stream);

/* Reuse step (cache_state 2, Algorithm 3): out = softmax(scale * Q_b' [K_c ; K_n]^T) [V_c ; V_n] over the first
 * kept_cnt[i] rows of the compacted cache followed by the block's b fresh rows k_blk, v_blk.
 * The compacted cache is older than the step that reuses it, and the call takes advantage of that: it starts streaming
 * k_c, v_c (and reads kept_cnt) while the kernel in front of it in the stream may still be finishing. This is safe
 * after every call of this library and after any kernel that holds its dependents back until it has completed (the
 * default). Only a caller's own kernel that releases its dependents early (programmatic dependent launch) must not be
 * the one that writes k_c, v_c or kept_cnt directly in front of this call. q_blk, k_blk and v_blk are read only
 * after the preceding kernel has completed. */
sdllm_status sdllm_sparse_block_attn(const sdllm_desc* desc, const void* q_blk, const void* k_c, const void* v_c,
                                     const int32_t* kept_cnt, const void* k_blk, const void* v_blk, void* out,
                                     void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Dense step (cache_state 0, and the full-sequence part of cache_state 1; Algorithm 3, "all L rows"): bidirectional
 * attention of every row of a sequence over all of its keys,
 *   out[i, h, t, :] = softmax_u(scale * q[i, h, t, :] . k[i, h / G, u, :]) v[i, h / G, u, :],   t, u < seq_len[i].
 *   q   [B, Hq, seq_len_max, D], strides q_stride[3] = (batch, head, row) in ELEMENTS, rows of D contiguous elements
 *   k,v [B, Hkv, seq_len_max, D] with desc->kv_stride
 *   out [B, Hq, seq_len_max, D] with o_stride[3]; rows t >= seq_len[i] are not written
 *   lse [B, Hq, seq_len_max] fp32, nullable: log-sum-exp of the scaled logits per written row
 * seq_len NULL means every sequence has seq_len_max rows. desc->block_len, retention and the selection fields are
 * not used. bf16 only, D in {64, 128}, at most 65535 query heads; anything else returns
 * SDLLM_ERR_UNSUPPORTED. The probability matrix is never written to memory. Workspace:
 * sdllm_workspace_bytes(desc, SDLLM_OP_DENSE_ATTN) bytes (the status word), zeroed once by the caller; a workspace of
 * the other attention calls serves as well. */
sdllm_status sdllm_dense_attn(const sdllm_desc* desc, const void* q, const int64_t* q_stride, const void* k, const void* v,
                              const int32_t* seq_len, void* out, const int64_t* o_stride, float* lse, void* workspace,
                              size_t workspace_bytes, void* cuda_stream);

/* The reuse step for callers that cannot allocate device memory. The paper has no counterpart for this call: it
 * computes exactly what sdllm_sparse_block_attn computes, but takes no workspace. Some hosts of this library run under
 * a fixed memory plan - an inference server that sized every buffer at start-up, a plug-in whose host owns the
 * allocator - and must not call cudaMalloc (or any allocating library routine) once they are running; they have
 * nowhere to get the workspace from. For them the scratch (status word, completion counters, key-split partials) is a
 * 8 MiB array built into the library image; every GPU that loads the library holds one copy until the process exits.
 *   - Shapes whose workspace (sdllm_workspace_bytes(desc, SDLLM_OP_SPARSE_BLOCK_ATTN)) exceeds 8 MiB are refused with
 *     SDLLM_ERR_WORKSPACE; use sdllm_sparse_block_attn with a caller-owned workspace for those.
 *   - The call allocates and frees nothing. The first call on each device looks the array's device address up
 *     (cudaGetSymbolAddress, with that device current); make that first call before any stream capture.
 *   - All calls on a device share the one array and it keeps what the last call left; each call clears the part that
 *     has to start at zero on its stream. Two calls that overlap on the GPU (different streams) race on it: keep the
 *     calls of one device in one stream order.
 *   - There is no workspace pointer to hand to sdllm_read_status; a bounded wait that expired shows as wrong output.
 * Inputs, outputs, layouts and errors are otherwise those of sdllm_sparse_block_attn. */
sdllm_status sdllm_sparse_block_attn_static(const sdllm_desc* desc, const void* q_blk, const void* k_c, const void* v_c,
                                            const int32_t* kept_cnt, const void* k_blk, const void* v_blk, void* out,
                                            void* cuda_stream);

/* Tuning and test aid; the paper has no counterpart. Overrides one decision of the launch planner, process-wide, until
 * sdllm_tuning_reset(). The library never reads the environment: these overrides are the only hidden input of the
 * planner, so sdllm_workspace_bytes, sdllm_launch_count and the launches agree as long as no override changes between
 * them. Host-only, thread-safe; takes effect for calls made afterwards. `name` is a NUL-terminated host string:
 *   "splits"      > 0: key splits per (sequence, KV head) of the attention calls
 *   "kernel"      attention kernel family: 0 automatic, 1 cp.async, 2 tcgen05 with the queries on the accumulator rows,
 *                 3 tcgen05 with the keys on the accumulator rows (only where that kernel covers the shape)
 *   "pdl"         0: no programmatic dependent launch     "early_loads" 0: no loads ahead of the grid dependency
 *   "cluster", "fused_tail", "dual", "key_tile", "lpt", "stages", "trigger", "persist"   plan details of the tcgen05 kernels
 *   "select"      top-k kernel: 1 one CTA per head, 2 one cluster per head
 *   "wait_cycles" limit, in SM clock cycles, of every abortable device-side wait (default 400 000 000, ~0.2 s). A limit
 *                 of a few cycles makes the first wait that is not already satisfied give up: the call still returns,
 *                 its outputs are invalid and sdllm_read_status reports SDLLM_ERR_TIMEOUT (how the tests exercise
 *                 that path without hanging anything).
 *   "debug"       1: print the CUDA error behind an SDLLM_ERR_CUDA to stderr
 * Returns SDLLM_ERR_INVALID_ARG for an unknown name. */
sdllm_status sdllm_tuning_set(const char* name, int64_t value);
void sdllm_tuning_reset(void);

#ifdef __cplusplus
}
#endif
#endif /* SDLLM_H_ */
