// Shared declarations of the libsdllm CUDA sources (sm_100a only).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sdllm.h"

namespace sdllm {

constexpr int kMaxRows = 256;         // b * G rows of one KV head handled by one CTA
constexpr int kMaxSplits = 64;        // key-axis splits per (sequence, KV head)
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// How one attention launch is cut into CTAs; a pure function of the description so that the workspace
// query and the launch always agree.
struct AttnPlan {
  int key_tile;     // keys per pipeline stage
  int m_warps;      // warps along the query rows (16 rows each, bf16) / row chunks (32 rows each, fp32)
  int c_warps;      // warps along the keys of a tile (bf16 only)
  int warp_keys;    // keys per warp per tile (cp.async bf16 kernel)
  int stages;       // shared-memory pipeline depth
  int cluster;      // > 1: the key splits of a unit form a thread-block cluster and merge through distributed shared memory
  int splits;       // partials per (sequence, KV head) left in the workspace (1 = final output written directly)
  int threads;
  bool tma;         // the kernel is fed by TMA (tcgen05 kernel), else by cp.async
  size_t smem_bytes;
  int kind;         // 0: cp.async kernels (fp32 FMA / bf16 mma.sync), 2: tcgen05 kernel, queries on the accumulator rows,
                    // 3: tcgen05 kernel, keys on the accumulator rows (its key splits merge inside their cluster)
  int key_tile2;    // tcgen05 kernel: keys per tile of source 2
  int rep;          // tcgen05 kernel: replicas of the query rows along the 128 accumulator rows
  int row_tiles;    // tcgen05 kernel: 128-row tiles of the b*G rows
  int parts;        // partials per (sequence, KV head, row tile) = splits * rep
  int rows_rep;     // rows of one partial
  bool fused_tail;  // the attention kernel merges the partials and pools the scores itself
  bool dual;        // tcgen05 kernel, small-footprint variant: two CTAs per SM
  bool persistent;  // key-row kernel, streaming variant: one resident CTA per SM walks the units
  size_t part_rows; // partial rows per (sequence, KV head) in the workspace (0: none)
  size_t n_counters;// completion counters in the workspace
};

// Key sources of one attention launch. The virtual key axis is [src1 rows 0..n1) ++ [src2 rows 0..n2).
// refresh: src1 = full K/V with n1 = seq_len[i], n2 = 0.  reuse: src1 = compacted cache with n1 = kept_cnt[i],
// src2 = the block's fresh rows with n2 = b.
struct AttnParams {
  const void* q;
  const void* k1; const void* v1;
  const void* k2; const void* v2;
  const int32_t* n1_per_seq;   // nullable -> n1_max
  const int32_t* block_off;    // refresh only
  void* out;                   // nullable
  float* lse;                  // nullable
  float* part_o;               // [B][Hkv][splits][M][D]
  float* part_ml;              // [B][Hkv][splits][M][2]  (running max in log2 units, running sum)
  float* raw_scores;           // [B][Hkv][n1_max] or null
  int B, Hq, Hkv, G, b, M;     // M = G * b rows per KV head
  int n1_max, n2;
  int splits;                  // partials per (sequence, KV head) in the workspace
  int splits_total;            // CTAs along the key axis per (sequence, KV head) = splits * cluster size
  int32_t* status;             // device status word: set non-zero when a bounded wait gave up
  long long wait_cycles;       // limit of an abortable device-side wait, in clock cycles
  int32_t* counters;           // completion counters (tcgen05 kernel), zero between calls
  float* pooled;               // refresh with a fused tail: pooled scores [B][Hkv][n1_max], else null
  int window, pool_kind, per_region;
  const float* lse_in;         // probability saliency, second pass: log-sum-exp of every block row [B][Hq][b]
  int prob_pass;               // 1: this launch is that second pass (tcgen05 kernel only)
  int want_scores;             // compute mean-query logit scores for src1 keys
  float scale;                 // softmax scale
  float scale_log2;            // scale * log2(e)
  int64_t q_stride[3], k1_stride[3], k2_stride[3], o_stride[3];
};

struct MergeParams {
  const float* part_o; const float* part_ml;
  void* out; float* lse;
  int B, Hq, Hkv, G, b, M, D, splits, dtype;
  int64_t o_stride[3];
  int merge_blocks;            // blocks [0, merge_blocks) merge; the rest pool
  // pooling of raw scores -> pooled scores
  const float* raw_scores; float* pooled;
  const int32_t* seq_len; const int32_t* block_off;
  int Lmax, window, pool_kind, per_region;
};

struct SelectParams {
  const float* pooled; const int32_t* seq_len; const int32_t* block_off;
  int32_t* kept_idx; int32_t* kept_cnt;
  int B, Hkv, Lmax, b, n_keep_max, mode;
  double retention;
  int smem_keys;               // candidates cached in shared memory (0 = read global every pass)
  int early_inputs;            // fused kernel: seq_len and block_off are read ahead of the grid dependency
};

struct CompactParams {
  const void* k; const void* v; const int32_t* kept_idx; const int32_t* kept_cnt;
  void* k_c; void* v_c;
  int B, Hkv, n_keep_max, row_bytes, Lmax;
  int64_t kv_stride_bytes[3], c_stride_bytes[3];
};

AttnPlan plan_attention(int dtype, int D, int M, int b, int B, int Hkv, int n1_max, int n2, bool prob_scores);

bool umma_tail_is_fused(const AttnPlan& pl, int D, int M, int n1_max, bool pool, bool merge);
bool umma_supported(int dtype, int D, int M, int b);
// Full-sequence attention, two query tiles per CTA (attn_dense.cu).
cudaError_t launch_dense_pair(const void* q, const int64_t* q_stride, const void* k, const void* v, const int64_t* kv_stride,
                              const int32_t* seq_len, void* out, const int64_t* o_stride, float* lse, int32_t* status, int B, int Hq,
                              int Hkv, int L, int D, float scale, cudaStream_t st);
cudaError_t launch_attn_partial(const AttnParams& p, const AttnPlan& plan, int dtype, int D, cudaStream_t st);
cudaError_t launch_merge_pool(const MergeParams& p, cudaStream_t st);
cudaError_t launch_select_topk(const SelectParams& p, cudaStream_t st);
cudaError_t launch_compact(const CompactParams& p, cudaStream_t st);
cudaError_t launch_select_compact(const SelectParams& p, const CompactParams& cp, cudaStream_t st);
bool select_compact_is_fused(int Lmax, int b, int n_keep_max);

__host__ __device__ inline int keep_count_total(int pre, int suf, double r, int mode, int* n_pre, int* n_suf) {
  // Algorithm 1: n = floor(|I| * r) in double; the other policies are described in sdllm.h.
  auto clampll = [](long long x, int hi) { return (int)(x < 0 ? 0 : (x > hi ? hi : x)); };
  if (mode == SDLLM_SELECT_JOINT_FLOOR) {
    *n_pre = -1; *n_suf = -1;
    return clampll((long long)floor((double)(pre + suf) * r), pre + suf);
  }
  if (mode == SDLLM_SELECT_PER_REGION_CEIL) {
    *n_pre = clampll((long long)ceil((double)pre * r), pre);
    *n_suf = clampll((long long)ceil((double)suf * r), suf);
    return *n_pre + *n_suf;
  }
  *n_pre = clampll((long long)floor((double)pre * r), pre);
  *n_suf = suf;
  return *n_pre + *n_suf;
}

}  // namespace sdllm
