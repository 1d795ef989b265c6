// C ABI of libsdllm: argument validation, workspace layout and kernel dispatch. Host code only.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>

#include <mutex>

#include "common.cuh"
#include "tuning.cuh"

using namespace sdllm;

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline int elem_size(int dtype) { return dtype == SDLLM_BF16 ? 2 : 4; }

bool strides_ok(const int64_t* s, int es) {
  for (int i = 0; i < 3; ++i)
    if (s[i] < 0 || (s[i] * es) % 16 != 0) return false;
  return true;
}

// Shape and policy checks shared by every entry point.
sdllm_status check_desc(const sdllm_desc* d) {
  if (d == nullptr || d->struct_size != sizeof(sdllm_desc)) return SDLLM_ERR_INVALID_ARG;
  if (d->batch < 1 || d->n_q_heads < 1 || d->n_kv_heads < 1 || d->block_len < 1 || d->seq_len_max < 1) return SDLLM_ERR_INVALID_ARG;
  if (d->n_q_heads % d->n_kv_heads != 0) return SDLLM_ERR_INVALID_ARG;
  if (d->dtype != SDLLM_F32 && d->dtype != SDLLM_BF16) return SDLLM_ERR_INVALID_ARG;
  if (d->pool_window < 1 || d->pool_window % 2 == 0) return SDLLM_ERR_INVALID_ARG;
  if (d->pool != SDLLM_POOL_MAX && d->pool != SDLLM_POOL_AVG) return SDLLM_ERR_INVALID_ARG;
  if (d->score != SDLLM_SCORE_LOGIT_MEAN && d->score != SDLLM_SCORE_PROB_MEAN) return SDLLM_ERR_INVALID_ARG;
  if (d->select < SDLLM_SELECT_JOINT_FLOOR || d->select > SDLLM_SELECT_PREFIX_ONLY) return SDLLM_ERR_INVALID_ARG;
  if (!(d->retention >= 0.0 && d->retention <= 1.0)) return SDLLM_ERR_INVALID_ARG;
  if (!(d->softmax_scale >= 0.f) || isinf(d->softmax_scale)) return SDLLM_ERR_INVALID_ARG;
  if (d->n_keep_max < 0 || d->block_len > d->seq_len_max) return SDLLM_ERR_INVALID_ARG;
  const int es = elem_size(d->dtype);
  if (!strides_ok(d->q_stride, es) || !strides_ok(d->kv_stride, es) || !strides_ok(d->o_stride, es) ||
      !strides_ok(d->c_stride, es) || !strides_ok(d->blk_stride, es))
    return SDLLM_ERR_INVALID_ARG;
  if (d->head_dim != 64 && d->head_dim != 128) return SDLLM_ERR_UNSUPPORTED;
  if ((int64_t)d->block_len * (d->n_q_heads / d->n_kv_heads) > kMaxRows) return SDLLM_ERR_UNSUPPORTED;
  if (d->batch > 65535 || d->n_kv_heads > 65535) return SDLLM_ERR_UNSUPPORTED;
  // the softmax-probability saliency exists in the tcgen05 kernel only
  if (d->score == SDLLM_SCORE_PROB_MEAN &&
      !umma_supported(d->dtype, d->head_dim, d->n_q_heads / d->n_kv_heads * d->block_len, d->block_len))
    return SDLLM_ERR_UNSUPPORTED;
  return SDLLM_OK;
}

// Pointer checks of the reuse step (both entry points).
sdllm_status check_sparse_args(const sdllm_desc* d, const void* q_blk, const void* k_c, const void* v_c, const int32_t* kept_cnt,
                               const void* k_blk, const void* v_blk, const void* out) {
  if (!q_blk || !k_blk || !v_blk || !out || !kept_cnt) return SDLLM_ERR_INVALID_ARG;
  if (d->n_keep_max > 0 && (!k_c || !v_c)) return SDLLM_ERR_INVALID_ARG;
  if (!aligned16(q_blk) || !aligned16(k_c) || !aligned16(v_c) || !aligned16(k_blk) || !aligned16(v_blk) || !aligned16(out))
    return SDLLM_ERR_INVALID_ARG;
  return SDLLM_OK;
}

// The kernels are built for sm_100a only.
sdllm_status check_device() {
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SDLLM_ERR_CUDA;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return SDLLM_ERR_CUDA;
  return major == 10 ? SDLLM_OK : SDLLM_ERR_UNSUPPORTED;
}

// With the tuning field "debug" set, the CUDA error behind an SDLLM_ERR_CUDA is printed to stderr.
bool cuda_failed(cudaError_t e, const char* what) {
  if (e == cudaSuccess) return false;
  if (tuning().debug != 0) fprintf(stderr, "libsdllm: %s: %s\n", what, cudaGetErrorString(e));
  (void)cudaGetLastError();
  return true;
}

float scale_of(const sdllm_desc* d) { return d->softmax_scale > 0.f ? d->softmax_scale : 1.0f / sqrtf((float)d->head_dim); }

struct WsLayout {
  size_t status, counters, part_o, part_ml, raw, lse, total;
};

WsLayout attn_ws(const sdllm_desc* d, const AttnPlan& pl, bool scores) {
  WsLayout w{};
  const int G = d->n_q_heads / d->n_kv_heads, M = G * d->block_len;
  size_t off = 0;
  w.status = off;
  (void)M;
  off += 256;                          // device status word (sdllm_read_status)
  w.counters = off;                    // completion counters: zero between calls
  off += align_up(pl.n_counters * 4, 256);
  w.part_o = off;
  off += align_up((size_t)d->batch * d->n_kv_heads * pl.part_rows * d->head_dim * 4, 256);
  w.part_ml = off;
  off += align_up((size_t)d->batch * d->n_kv_heads * pl.part_rows * 2 * 4, 256);
  w.raw = off;
  const bool prob = d->score == SDLLM_SCORE_PROB_MEAN;
  if (scores) off += align_up((size_t)d->batch * d->n_kv_heads * d->seq_len_max * 4 * (prob ? pl.row_tiles : 1), 256);
  w.lse = off;                         // probability saliency: the rows' log-sum-exp between its two passes
  if (scores && prob) off += align_up((size_t)d->batch * d->n_q_heads * d->block_len * 4, 256);
  w.total = off;
  return w;
}

AttnPlan plan_for(const sdllm_desc* d, int op) {
  const int G = d->n_q_heads / d->n_kv_heads;
  const bool refresh = op == SDLLM_OP_REFRESH_SCORES;
  return plan_attention(d->dtype, d->head_dim, G * d->block_len, d->block_len, d->batch, d->n_kv_heads,
                        refresh ? d->seq_len_max : d->n_keep_max, refresh ? 0 : d->block_len,
                        refresh && d->score == SDLLM_SCORE_PROB_MEAN);
}

void fill_common(AttnParams& p, const sdllm_desc* d, const AttnPlan& pl) {
  p.B = d->batch; p.Hq = d->n_q_heads; p.Hkv = d->n_kv_heads; p.G = p.Hq / p.Hkv; p.b = d->block_len; p.M = p.G * p.b;
  p.splits = pl.splits;
  p.splits_total = pl.splits * pl.cluster;
  p.scale = scale_of(d);
  p.scale_log2 = p.scale * kLog2e;
  p.wait_cycles = tuning().wait_cycles;
  for (int i = 0; i < 3; ++i) { p.q_stride[i] = d->q_stride[i]; p.o_stride[i] = d->o_stride[i]; }
}

// Full-sequence attention runs on its own tcgen05 kernel: bf16, D in {64, 128}, one grid row per query head.
// Its workspace is the status word alone.
constexpr size_t kDenseWorkspaceBytes = 256;
bool dense_supported(const sdllm_desc* d) {
  return umma_supported(d->dtype, d->head_dim, 128, 128) && d->n_q_heads <= 65535;
}

// Built-in scratch of sdllm_sparse_block_attn_static: lives in the library image, one copy per GPU that loads it.
constexpr size_t kStaticScratchBytes = (size_t)8 << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
std::mutex g_static_mutex;
void* g_static_scratch_ptr[kMaxDevices] = {};      // device address of g_static_scratch on each device, once looked up

// The array's name is only a handle on the host; the address a kernel can use comes from the runtime, per device.
sdllm_status static_scratch_address(void** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SDLLM_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return SDLLM_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (g_static_scratch_ptr[dev] == nullptr) {
    void* ptr = nullptr;
    if (cuda_failed(cudaGetSymbolAddress(&ptr, g_static_scratch), "cudaGetSymbolAddress") || ptr == nullptr) return SDLLM_ERR_CUDA;
    g_static_scratch_ptr[dev] = ptr;
  }
  *out = g_static_scratch_ptr[dev];
  return SDLLM_OK;
}

}  // namespace

extern "C" {

int sdllm_version(void) { return SDLLM_VERSION; }

sdllm_status sdllm_tuning_set(const char* name, int64_t value) {
  return tuning_set(name, (long long)value) ? SDLLM_OK : SDLLM_ERR_INVALID_ARG;
}

void sdllm_tuning_reset(void) { tuning_reset(); }

const char* sdllm_status_string(sdllm_status s) {
  switch (s) {
    case SDLLM_OK: return "ok";
    case SDLLM_ERR_INVALID_ARG: return "invalid argument";
    case SDLLM_ERR_UNSUPPORTED: return "unsupported shape, mode or device";
    case SDLLM_ERR_WORKSPACE: return "workspace missing or too small";
    case SDLLM_ERR_CUDA: return "CUDA error";
    case SDLLM_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

size_t sdllm_workspace_bytes(const sdllm_desc* d, int op) {
  if (check_desc(d) != SDLLM_OK) return 0;
  if (op == SDLLM_OP_REFRESH_SCORES) return attn_ws(d, plan_for(d, op), true).total;
  if (op == SDLLM_OP_SPARSE_BLOCK_ATTN) return attn_ws(d, plan_for(d, op), false).total;
  if (op == SDLLM_OP_DENSE_ATTN && dense_supported(d)) return kDenseWorkspaceBytes;
  return 0;
}

sdllm_status sdllm_keep_count(const sdllm_desc* d, int32_t seq_len, int32_t block_off, int32_t* n_total, int32_t* n_prefix,
                              int32_t* n_suffix) {
  const sdllm_status st = check_desc(d);
  if (st != SDLLM_OK) return st;
  if (seq_len < d->block_len || block_off < 0 || block_off + d->block_len > seq_len) return SDLLM_ERR_INVALID_ARG;
  int np, ns;
  const int nt = keep_count_total(block_off, seq_len - block_off - d->block_len, d->retention, d->select, &np, &ns);
  if (n_total) *n_total = nt;
  if (n_prefix) *n_prefix = np;
  if (n_suffix) *n_suffix = ns;
  return SDLLM_OK;
}

sdllm_status sdllm_plan_describe(const sdllm_desc* d, int op, char* buf, size_t buf_bytes) {
  if (buf == nullptr || buf_bytes == 0) return SDLLM_ERR_INVALID_ARG;
  buf[0] = 0;
  if (check_desc(d) != SDLLM_OK || (op != SDLLM_OP_REFRESH_SCORES && op != SDLLM_OP_SPARSE_BLOCK_ATTN)) return SDLLM_ERR_INVALID_ARG;
  const AttnPlan pl = plan_for(d, op);
  const char* name = pl.kind == 3 ? (pl.persistent ? "attn_kt_stream_kernel" : "attn_kt_kernel")
                                  : (pl.kind == 2 ? "attn_umma_bf16_kernel" : (d->dtype == SDLLM_BF16 ? "attn_bf16_kernel" : "attn_f32_kernel"));
  if (pl.kind == 3)
    snprintf(buf, buf_bytes, "%s splits=%d cluster=%d stages=%d softmax_warpgroups=%d threads=%d smem=%zu", name, pl.cluster, pl.cluster,
             pl.stages, pl.c_warps * pl.warp_keys, pl.threads, pl.smem_bytes);
  else
    snprintf(buf, buf_bytes, "%s splits=%d cluster=%d stages=%d key_tile=%d threads=%d smem=%zu", name, pl.splits, pl.cluster, pl.stages,
             pl.key_tile, pl.threads, pl.smem_bytes);
  return SDLLM_OK;
}

int32_t sdllm_launch_count(const sdllm_desc* d, int op) {
  if (check_desc(d) != SDLLM_OK) return -1;
  if (op == SDLLM_OP_SELECT_TOPK) return 1;
  if (op == SDLLM_OP_COMPACT_KV) return d->n_keep_max > 0 ? 1 : 0;
  if (op == SDLLM_OP_SELECT_COMPACT)
    return select_compact_is_fused(d->seq_len_max, d->block_len, d->n_keep_max) ? 1 : 1 + (d->n_keep_max > 0 ? 1 : 0);
  if (op == SDLLM_OP_DENSE_ATTN) return dense_supported(d) ? 1 : -1;
  if (op != SDLLM_OP_REFRESH_SCORES && op != SDLLM_OP_SPARSE_BLOCK_ATTN) return -1;
  const bool refresh = op == SDLLM_OP_REFRESH_SCORES;
  const AttnPlan pl = plan_for(d, op);
  const int M = d->n_q_heads / d->n_kv_heads * d->block_len;
  if (pl.kind == 3) return 1;       // the key splits merge, and the scores are pooled, inside the one launch
  if (pl.kind == 2) {
    const int n1 = refresh ? d->seq_len_max : d->n_keep_max;
    if (refresh && d->score == SDLLM_SCORE_PROB_MEAN)     // attention pass (+ its merge) and saliency pass (+ its pooling)
      return 1 + ((pl.splits > 1 && !umma_tail_is_fused(pl, d->head_dim, M, n1, false, true)) ? 1 : 0) + 1 +
             (umma_tail_is_fused(pl, d->head_dim, M, n1, true, false) ? 0 : 1);
    const bool tail_work = pl.splits > 1 || refresh;
    return 1 + ((tail_work && !umma_tail_is_fused(pl, d->head_dim, M, n1, refresh, true)) ? 1 : 0);
  }
  return 1 + ((refresh || pl.splits > 1) ? 1 : 0);
}

int32_t sdllm_cache_state(int32_t i, int32_t delay) { return i > delay ? 2 : (i == delay ? 1 : 0); }

sdllm_status sdllm_read_status(const void* workspace, void* cuda_stream, int32_t* device_status) {
  if (!workspace || !device_status) return SDLLM_ERR_INVALID_ARG;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  int32_t v = 0;
  if (cudaMemcpyAsync(&v, workspace, sizeof(v), cudaMemcpyDeviceToHost, stream) != cudaSuccess) return SDLLM_ERR_CUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return SDLLM_ERR_CUDA;
  *device_status = v;
  return v == 0 ? SDLLM_OK : SDLLM_ERR_TIMEOUT;
}

sdllm_status sdllm_refresh_scores(const sdllm_desc* d, const void* q_blk, const void* k, const void* v, const int32_t* seq_len,
                                  const int32_t* block_off, void* out, float* lse, float* pooled_scores, void* ws, size_t ws_bytes,
                                  void* cuda_stream) {
  sdllm_status st = check_desc(d);
  if (st != SDLLM_OK) return st;
  if (!q_blk || !k || !v || !block_off || (!out && !pooled_scores)) return SDLLM_ERR_INVALID_ARG;
  if (!aligned16(q_blk) || !aligned16(k) || !aligned16(v) || !aligned16(out) || !aligned16(pooled_scores) || !aligned16(lse))
    return SDLLM_ERR_INVALID_ARG;
  if (lse && !out) return SDLLM_ERR_INVALID_ARG;
  const AttnPlan pl = plan_for(d, SDLLM_OP_REFRESH_SCORES);
  const WsLayout w = attn_ws(d, pl, true);
  if (w.total > 0 && (ws == nullptr || ws_bytes < w.total || (reinterpret_cast<uintptr_t>(ws) & 255u))) return SDLLM_ERR_WORKSPACE;
  if ((st = check_device()) != SDLLM_OK) return st;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  char* wsb = reinterpret_cast<char*>(ws);

  AttnParams p{};
  fill_common(p, d, pl);
  p.q = q_blk; p.k1 = k; p.v1 = v; p.k2 = nullptr; p.v2 = nullptr;
  p.n1_per_seq = seq_len; p.block_off = block_off;
  p.out = out; p.lse = lse;
  p.status = reinterpret_cast<int32_t*>(wsb + w.status);
  p.part_o = reinterpret_cast<float*>(wsb + w.part_o);
  p.part_ml = reinterpret_cast<float*>(wsb + w.part_ml);
  p.raw_scores = pooled_scores ? reinterpret_cast<float*>(wsb + w.raw) : nullptr;
  p.n1_max = d->seq_len_max; p.n2 = 0;
  p.want_scores = pooled_scores != nullptr;
  p.counters = reinterpret_cast<int32_t*>(wsb + w.counters);
  p.pooled = pooled_scores; p.window = d->pool_window; p.pool_kind = d->pool;
  p.per_region = d->select != SDLLM_SELECT_JOINT_FLOOR;
  for (int i = 0; i < 3; ++i) { p.k1_stride[i] = d->kv_stride[i]; p.k2_stride[i] = 0; }
  if (d->score == SDLLM_SCORE_PROB_MEAN && pooled_scores != nullptr) {
    // Softmax-probability saliency: the probabilities need each row's final normaliser, so the scores come from a
    // second pass over K once the attention pass has left the rows' log-sum-exp.
    if (!out) return SDLLM_ERR_INVALID_ARG;
    AttnParams a = p;
    a.want_scores = 0; a.pooled = nullptr; a.raw_scores = nullptr;
    if (!a.lse) a.lse = reinterpret_cast<float*>(wsb + w.lse);
    if (cuda_failed(launch_attn_partial(a, pl, d->dtype, d->head_dim, stream), "attention launch")) return SDLLM_ERR_CUDA;
    AttnParams s2 = p;
    s2.out = nullptr; s2.lse = nullptr; s2.lse_in = a.lse; s2.prob_pass = 1; s2.want_scores = 0;
    if (cuda_failed(launch_attn_partial(s2, pl, d->dtype, d->head_dim, stream), "saliency launch")) return SDLLM_ERR_CUDA;
    return SDLLM_OK;
  }
  if (cuda_failed(launch_attn_partial(p, pl, d->dtype, d->head_dim, stream), "attention launch")) return SDLLM_ERR_CUDA;
  if (pl.fused_tail) return SDLLM_OK;

  MergeParams m{};
  m.part_o = (out && pl.splits > 1) ? p.part_o : nullptr;
  m.part_ml = p.part_ml; m.out = out; m.lse = lse;
  m.B = p.B; m.Hq = p.Hq; m.Hkv = p.Hkv; m.G = p.G; m.b = p.b; m.M = p.M; m.D = d->head_dim; m.splits = pl.splits; m.dtype = d->dtype;
  for (int i = 0; i < 3; ++i) m.o_stride[i] = d->o_stride[i];
  m.raw_scores = p.raw_scores; m.pooled = pooled_scores; m.seq_len = seq_len; m.block_off = block_off;
  m.Lmax = d->seq_len_max; m.window = d->pool_window; m.pool_kind = d->pool;
  m.per_region = d->select != SDLLM_SELECT_JOINT_FLOOR;
  if (cuda_failed(launch_merge_pool(m, stream), "merge/pool launch")) return SDLLM_ERR_CUDA;
  return SDLLM_OK;
}

sdllm_status sdllm_select_topk(const sdllm_desc* d, const float* pooled_scores, const int32_t* seq_len, const int32_t* block_off,
                               int32_t* kept_idx, int32_t* kept_cnt, void* ws, size_t ws_bytes, void* cuda_stream) {
  (void)ws; (void)ws_bytes;
  sdllm_status st = check_desc(d);
  if (st != SDLLM_OK) return st;
  if (!pooled_scores || !block_off || !kept_idx || !kept_cnt) return SDLLM_ERR_INVALID_ARG;
  if (!aligned16(pooled_scores) || !aligned16(kept_idx)) return SDLLM_ERR_INVALID_ARG;
  if ((st = check_device()) != SDLLM_OK) return st;
  SelectParams p{};
  p.pooled = pooled_scores; p.seq_len = seq_len; p.block_off = block_off; p.kept_idx = kept_idx; p.kept_cnt = kept_cnt;
  p.B = d->batch; p.Hkv = d->n_kv_heads; p.Lmax = d->seq_len_max; p.b = d->block_len; p.n_keep_max = d->n_keep_max;
  p.mode = d->select; p.retention = d->retention;
  const int cand = d->seq_len_max - d->block_len;
  p.smem_keys = cand <= 45056 ? cand : 0;
  if (cuda_failed(launch_select_topk(p, reinterpret_cast<cudaStream_t>(cuda_stream)), "select launch")) return SDLLM_ERR_CUDA;
  return SDLLM_OK;
}

sdllm_status sdllm_compact_kv(const sdllm_desc* d, const void* k, const void* v, const int32_t* kept_idx, const int32_t* kept_cnt,
                              void* k_c, void* v_c, void* cuda_stream) {
  sdllm_status st = check_desc(d);
  if (st != SDLLM_OK) return st;
  if (!k || !v || !kept_idx || !kept_cnt || !k_c || !v_c) return SDLLM_ERR_INVALID_ARG;
  if (!aligned16(k) || !aligned16(v) || !aligned16(k_c) || !aligned16(v_c)) return SDLLM_ERR_INVALID_ARG;
  if ((st = check_device()) != SDLLM_OK) return st;
  const int es = elem_size(d->dtype);
  CompactParams p{};
  p.k = k; p.v = v; p.kept_idx = kept_idx; p.kept_cnt = kept_cnt; p.k_c = k_c; p.v_c = v_c;
  p.B = d->batch; p.Hkv = d->n_kv_heads; p.n_keep_max = d->n_keep_max; p.row_bytes = d->head_dim * es; p.Lmax = d->seq_len_max;
  for (int i = 0; i < 3; ++i) { p.kv_stride_bytes[i] = d->kv_stride[i] * es; p.c_stride_bytes[i] = d->c_stride[i] * es; }
  if (cuda_failed(launch_compact(p, reinterpret_cast<cudaStream_t>(cuda_stream)), "compact launch")) return SDLLM_ERR_CUDA;
  return SDLLM_OK;
}

sdllm_status sdllm_select_compact(const sdllm_desc* d, const float* pooled_scores, const int32_t* seq_len, const int32_t* block_off,
                                  const void* k, const void* v, int32_t* kept_idx, int32_t* kept_cnt, void* k_c, void* v_c,
                                  void* cuda_stream) {
  sdllm_status st = check_desc(d);
  if (st != SDLLM_OK) return st;
  if (!pooled_scores || !block_off || !kept_idx || !kept_cnt) return SDLLM_ERR_INVALID_ARG;
  if (d->n_keep_max > 0 && (!k || !v || !k_c || !v_c)) return SDLLM_ERR_INVALID_ARG;
  if (!aligned16(pooled_scores) || !aligned16(kept_idx) || !aligned16(k) || !aligned16(v) || !aligned16(k_c) || !aligned16(v_c))
    return SDLLM_ERR_INVALID_ARG;
  if ((st = check_device()) != SDLLM_OK) return st;
  const int es = elem_size(d->dtype);
  SelectParams p{};
  p.pooled = pooled_scores; p.seq_len = seq_len; p.block_off = block_off; p.kept_idx = kept_idx; p.kept_cnt = kept_cnt;
  p.B = d->batch; p.Hkv = d->n_kv_heads; p.Lmax = d->seq_len_max; p.b = d->block_len; p.n_keep_max = d->n_keep_max;
  p.mode = d->select; p.retention = d->retention;
  const int cand = d->seq_len_max - d->block_len;
  p.smem_keys = cand <= 45056 ? cand : 0;
  p.early_inputs = (tuning().pdl != 0 && tuning().early_loads != 0) ? 1 : 0;
  CompactParams c{};
  c.k = k; c.v = v; c.kept_idx = kept_idx; c.kept_cnt = kept_cnt; c.k_c = k_c; c.v_c = v_c;
  c.B = d->batch; c.Hkv = d->n_kv_heads; c.n_keep_max = d->n_keep_max; c.row_bytes = d->head_dim * es; c.Lmax = d->seq_len_max;
  for (int i = 0; i < 3; ++i) { c.kv_stride_bytes[i] = d->kv_stride[i] * es; c.c_stride_bytes[i] = d->c_stride[i] * es; }
  if (cuda_failed(launch_select_compact(p, c, reinterpret_cast<cudaStream_t>(cuda_stream)), "select + compact launch")) return SDLLM_ERR_CUDA;
  return SDLLM_OK;
}

sdllm_status sdllm_sparse_block_attn(const sdllm_desc* d, const void* q_blk, const void* k_c, const void* v_c, const int32_t* kept_cnt,
                                     const void* k_blk, const void* v_blk, void* out, void* ws, size_t ws_bytes, void* cuda_stream) {
  sdllm_status st = check_desc(d);
  if (st != SDLLM_OK) return st;
  if ((st = check_sparse_args(d, q_blk, k_c, v_c, kept_cnt, k_blk, v_blk, out)) != SDLLM_OK) return st;
  const AttnPlan pl = plan_for(d, SDLLM_OP_SPARSE_BLOCK_ATTN);
  const WsLayout w = attn_ws(d, pl, false);
  if (w.total > 0 && (ws == nullptr || ws_bytes < w.total || (reinterpret_cast<uintptr_t>(ws) & 255u))) return SDLLM_ERR_WORKSPACE;
  if ((st = check_device()) != SDLLM_OK) return st;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  char* wsb = reinterpret_cast<char*>(ws);

  AttnParams p{};
  fill_common(p, d, pl);
  p.q = q_blk; p.k1 = k_c ? k_c : k_blk; p.v1 = v_c ? v_c : v_blk; p.k2 = k_blk; p.v2 = v_blk;
  p.n1_per_seq = kept_cnt; p.block_off = nullptr;
  p.out = out; p.lse = nullptr;
  p.status = reinterpret_cast<int32_t*>(wsb + w.status);
  p.part_o = reinterpret_cast<float*>(wsb + w.part_o);
  p.part_ml = reinterpret_cast<float*>(wsb + w.part_ml);
  p.raw_scores = nullptr;
  p.n1_max = d->n_keep_max; p.n2 = d->block_len;
  p.want_scores = 0;
  p.counters = reinterpret_cast<int32_t*>(wsb + w.counters);
  p.pooled = nullptr;
  for (int i = 0; i < 3; ++i) { p.k1_stride[i] = d->c_stride[i]; p.k2_stride[i] = d->blk_stride[i]; }
  if (cuda_failed(launch_attn_partial(p, pl, d->dtype, d->head_dim, stream), "attention launch")) return SDLLM_ERR_CUDA;
  if (pl.splits > 1 && !pl.fused_tail) {
    MergeParams m{};
    m.part_o = p.part_o; m.part_ml = p.part_ml; m.out = out; m.lse = nullptr;
    m.B = p.B; m.Hq = p.Hq; m.Hkv = p.Hkv; m.G = p.G; m.b = p.b; m.M = p.M; m.D = d->head_dim; m.splits = pl.splits; m.dtype = d->dtype;
    for (int i = 0; i < 3; ++i) m.o_stride[i] = d->o_stride[i];
    if (cuda_failed(launch_merge_pool(m, stream), "merge/pool launch")) return SDLLM_ERR_CUDA;
  }
  return SDLLM_OK;
}

sdllm_status sdllm_dense_attn(const sdllm_desc* d, const void* q, const int64_t* q_stride, const void* k, const void* v,
                              const int32_t* seq_len, void* out, const int64_t* o_stride, float* lse, void* ws, size_t ws_bytes,
                              void* cuda_stream) {
  sdllm_status st = check_desc(d);
  if (st != SDLLM_OK) return st;
  if (!q || !k || !v || !out || !q_stride || !o_stride) return SDLLM_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || !aligned16(lse)) return SDLLM_ERR_INVALID_ARG;
  if (!strides_ok(q_stride, elem_size(d->dtype)) || !strides_ok(o_stride, elem_size(d->dtype))) return SDLLM_ERR_INVALID_ARG;
  if (!dense_supported(d)) return SDLLM_ERR_UNSUPPORTED;
  if (ws == nullptr || ws_bytes < kDenseWorkspaceBytes || (reinterpret_cast<uintptr_t>(ws) & 255u)) return SDLLM_ERR_WORKSPACE;
  if ((st = check_device()) != SDLLM_OK) return st;
  if (cuda_failed(launch_dense_pair(q, q_stride, k, v, d->kv_stride, seq_len, out, o_stride, lse, reinterpret_cast<int32_t*>(ws),
                                    d->batch, d->n_q_heads, d->n_kv_heads, d->seq_len_max, d->head_dim, scale_of(d),
                                    reinterpret_cast<cudaStream_t>(cuda_stream)), "dense attention launch"))
    return SDLLM_ERR_CUDA;
  return SDLLM_OK;
}

sdllm_status sdllm_sparse_block_attn_static(const sdllm_desc* d, const void* q_blk, const void* k_c, const void* v_c,
                                            const int32_t* kept_cnt, const void* k_blk, const void* v_blk, void* out, void* cuda_stream) {
  sdllm_status st = check_desc(d);
  if (st != SDLLM_OK) return st;
  if ((st = check_sparse_args(d, q_blk, k_c, v_c, kept_cnt, k_blk, v_blk, out)) != SDLLM_OK) return st;
  const WsLayout w = attn_ws(d, plan_for(d, SDLLM_OP_SPARSE_BLOCK_ATTN), false);
  if (w.total > kStaticScratchBytes) return SDLLM_ERR_WORKSPACE;       // this shape needs more than the built-in scratch
  if ((st = check_device()) != SDLLM_OK) return st;
  void* scratch = nullptr;
  if ((st = static_scratch_address(&scratch)) != SDLLM_OK) return st;
  // the status word and the completion counters must start at zero whatever the last call left behind
  if (cuda_failed(cudaMemsetAsync(scratch, 0, w.part_o, reinterpret_cast<cudaStream_t>(cuda_stream)), "scratch clear")) return SDLLM_ERR_CUDA;
  return sdllm_sparse_block_attn(d, q_blk, k_c, v_c, kept_cnt, k_blk, v_blk, out, scratch, kStaticScratchBytes, cuda_stream);
}

}  // extern "C"
