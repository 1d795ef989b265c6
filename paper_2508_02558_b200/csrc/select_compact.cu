// Top-k selection over the pooled importance scores and the K/V gather-compaction
// (Algorithm 1: "n <- floor(|I| r)", "TopKIndices(I, n)", "Select(K_f, I)", "Select(V_f, I)").
#include "common.cuh"

namespace sdllm {
namespace {

// Order-preserving map fp32 -> u32 (larger float <=> larger key). -0 is folded onto +0 and NaN sorts lowest so the
// order agrees with a numeric comparison of the values.
__device__ __forceinline__ uint32_t score_key(float x) {
  if (x != x) return 0u;
  if (x == 0.f) x = 0.f;
  const uint32_t u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

constexpr int SEL_THREADS = 1024;
constexpr int SEL_WARPS = SEL_THREADS / 32;

struct Segment { int c_lo, c_hi, n; };   // candidate range and how many to keep

// One CTA per (sequence, KV head). Radix select (4 passes of 8 bits, most significant first) finds the key of the
// n-th largest candidate and how many candidates are strictly greater; a final ordered pass writes, in ascending
// position order, every candidate above the threshold plus the lowest-index candidates equal to it. No step depends
// on the order in which threads run, so the result is deterministic.
__global__ void __launch_bounds__(SEL_THREADS) select_topk_kernel(const SelectParams p) {
  extern __shared__ uint32_t keys_s[];                 // optional cache of the candidate keys
  __shared__ uint32_t hist[SEL_WARPS][256];
  __shared__ uint32_t warp_cnt[2][SEL_WARPS];
  __shared__ uint32_t sh_prefix, sh_remaining, sh_run_eq, sh_run_out;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = blockIdx.x, bi = blockIdx.y;
  int L = p.seq_len ? p.seq_len[bi] : p.Lmax;
  L = min(max(L, 0), p.Lmax);
  const int b = p.b;
  int o = p.block_off[bi];
  o = min(max(o, 0), max(L - b, 0));
  const int C = max(L - b, 0);
  const float* sc = p.pooled + (int64_t)(bi * p.Hkv + g) * p.Lmax;
  int32_t* out = p.kept_idx + (int64_t)(bi * p.Hkv + g) * p.n_keep_max;
  const bool cached = C <= p.smem_keys;

  auto cand_pos = [&](int c) { return c < o ? c : c + b; };
  auto key_at = [&](int c) -> uint32_t { return cached ? keys_s[c] : score_key(sc[cand_pos(c)]); };

  if (cached)
    for (int c = tid; c < C; c += SEL_THREADS) keys_s[c] = score_key(sc[cand_pos(c)]);

  int n_pre, n_suf;
  const int n_total = keep_count_total(o, C - o, p.retention, p.mode, &n_pre, &n_suf);
  Segment seg[2];
  int n_seg;
  if (p.mode == SDLLM_SELECT_JOINT_FLOOR) {
    seg[0] = {0, C, min(n_total, p.n_keep_max)};
    n_seg = 1;
  } else {
    const int np = min(n_pre, p.n_keep_max);
    seg[0] = {0, o, np};
    seg[1] = {o, C, min(n_suf, p.n_keep_max - np)};
    n_seg = 2;
  }
  if (tid == 0) { sh_run_out = 0; }
  __syncthreads();

  for (int si = 0; si < n_seg; ++si) {
    const int c_lo = seg[si].c_lo, c_hi = seg[si].c_hi, n = seg[si].n;
    const int len = c_hi - c_lo;
    if (n <= 0 || len <= 0) continue;
    uint32_t thr = 0u, need_eq = 0u;
    const bool take_all = n >= len;
    if (!take_all) {
      // ---- radix select of the n-th largest key ----
      if (tid == 0) { sh_prefix = 0u; sh_remaining = (uint32_t)n; }
      for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        for (int i = tid; i < SEL_WARPS * 256; i += SEL_THREADS) (&hist[0][0])[i] = 0u;
        __syncthreads();
        const uint32_t prefix = sh_prefix;
        const uint32_t remaining = sh_remaining;
        const uint32_t himask = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + 8));
        for (int c0 = c_lo; c0 < c_hi; c0 += SEL_THREADS) {
          const int c = c0 + tid;
          const bool in = c < c_hi;
          const uint32_t k = in ? key_at(c) : 0u;
          const bool match = in && ((k & himask) == prefix);
          const uint32_t digit = (k >> shift) & 0xFFu;
          // aggregate equal digits inside the warp, one shared-memory add per distinct digit
          const uint32_t active = __ballot_sync(0xffffffffu, match);
          if (match) {
            const uint32_t peers = __match_any_sync(active, digit);
            if ((int)(__ffs(peers) - 1) == lane) hist[warp][digit] += __popc(peers);
          }
        }
        __syncthreads();
        // column sums of the per-warp histograms, then a scan from the top bin by warp 0
        if (tid < 256) {
          uint32_t s = 0;
          for (int w = 0; w < SEL_WARPS; ++w) s += hist[w][tid];
          hist[0][tid] = s;
        }
        __syncthreads();
        if (warp == 0) {
          // lane handles bins [255 - 8*lane - 7, 255 - 8*lane], scanning downward
          uint32_t local[8], sum = 0;
#pragma unroll
          for (int i = 0; i < 8; ++i) { local[i] = hist[0][255 - (8 * lane + i)]; sum += local[i]; }
          uint32_t incl = sum;
#pragma unroll
          for (int d = 1; d < 32; d <<= 1) {
            const uint32_t y = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += y;
          }
          uint32_t above = incl - sum;            // candidates in bins above this lane's range
          if (above < remaining && incl >= remaining) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              if (above + local[i] >= remaining) {
                sh_prefix = prefix | ((uint32_t)(255 - (8 * lane + i)) << shift);
                sh_remaining = remaining - above;
                break;
              }
              above += local[i];
            }
          }
        }
        __syncthreads();
      }
      thr = sh_prefix;
      need_eq = sh_remaining;                     // how many candidates equal to thr are still to be kept (>= 1)
    }
    // ---- ordered emission ----
    if (tid == 0) sh_run_eq = 0u;
    __syncthreads();
    for (int c0 = c_lo; c0 < c_hi; c0 += SEL_THREADS) {
      const int c = c0 + tid;
      const bool in = c < c_hi;
      const uint32_t k = in ? key_at(c) : 0u;
      const bool gt = in && (take_all || k > thr);
      const bool eq = in && !take_all && k == thr;
      const uint32_t beq = __ballot_sync(0xffffffffu, eq);
      if (lane == 0) warp_cnt[0][warp] = __popc(beq);
      __syncthreads();
      uint32_t eq_before = sh_run_eq;
      for (int w = 0; w < warp; ++w) eq_before += warp_cnt[0][w];
      eq_before += __popc(beq & ((1u << lane) - 1u));
      const bool keep = gt || (eq && eq_before < need_eq);
      const uint32_t bk = __ballot_sync(0xffffffffu, keep);
      if (lane == 0) warp_cnt[1][warp] = __popc(bk);
      __syncthreads();
      uint32_t out_before = sh_run_out;
      for (int w = 0; w < warp; ++w) out_before += warp_cnt[1][w];
      out_before += __popc(bk & ((1u << lane) - 1u));
      if (keep && out_before < (uint32_t)p.n_keep_max) out[out_before] = cand_pos(c);
      __syncthreads();
      if (tid == 0) {
        uint32_t te = 0, tk = 0;
        for (int w = 0; w < SEL_WARPS; ++w) { te += warp_cnt[0][w]; tk += warp_cnt[1][w]; }
        sh_run_eq += te; sh_run_out += tk;
      }
      __syncthreads();
    }
  }
  __syncthreads();
  const int kept = min((int)sh_run_out, p.n_keep_max);
  for (int i = kept + tid; i < p.n_keep_max; i += SEL_THREADS) out[i] = -1;
  if (g == 0 && tid == 0) p.kept_cnt[bi] = kept;
}

// Gather of the kept rows: 16 bytes per thread, four rows of K and of V in flight per thread.
constexpr int CP_ROWS_PER_THREAD = 4;

__global__ void __launch_bounds__(256) compact_kv_kernel(const CompactParams p) {
  const int chunks = p.row_bytes / 16;                 // threads per row
  const int rows_per_pass = 256 / chunks;
  const int tid = threadIdx.x;
  const int c = tid % chunks, rl = tid / chunks;
  const int g = blockIdx.y, bi = blockIdx.z;
  const int cnt = min(max(p.kept_cnt[bi], 0), p.n_keep_max);
  const int32_t* idx = p.kept_idx + (int64_t)(bi * p.Hkv + g) * p.n_keep_max;
  const char* kb = reinterpret_cast<const char*>(p.k) + bi * p.kv_stride_bytes[0] + g * p.kv_stride_bytes[1];
  const char* vb = reinterpret_cast<const char*>(p.v) + bi * p.kv_stride_bytes[0] + g * p.kv_stride_bytes[1];
  char* kc = reinterpret_cast<char*>(p.k_c) + bi * p.c_stride_bytes[0] + g * p.c_stride_bytes[1];
  char* vc = reinterpret_cast<char*>(p.v_c) + bi * p.c_stride_bytes[0] + g * p.c_stride_bytes[1];
  const int row0 = blockIdx.x * rows_per_pass * CP_ROWS_PER_THREAD + rl;

  uint4 kv[CP_ROWS_PER_THREAD], vv[CP_ROWS_PER_THREAD];
#pragma unroll
  for (int u = 0; u < CP_ROWS_PER_THREAD; ++u) {
    const int i = row0 + u * rows_per_pass;
    kv[u] = make_uint4(0u, 0u, 0u, 0u);
    vv[u] = make_uint4(0u, 0u, 0u, 0u);
    if (i < cnt) {
      const int src = idx[i];
      if (src >= 0 && src < p.Lmax) {
        kv[u] = __ldg(reinterpret_cast<const uint4*>(kb + (int64_t)src * p.kv_stride_bytes[2]) + c);
        vv[u] = __ldg(reinterpret_cast<const uint4*>(vb + (int64_t)src * p.kv_stride_bytes[2]) + c);
      }
    }
  }
#pragma unroll
  for (int u = 0; u < CP_ROWS_PER_THREAD; ++u) {
    const int i = row0 + u * rows_per_pass;
    if (i < p.n_keep_max) {
      reinterpret_cast<uint4*>(kc + (int64_t)i * p.c_stride_bytes[2])[c] = kv[u];
      reinterpret_cast<uint4*>(vc + (int64_t)i * p.c_stride_bytes[2])[c] = vv[u];
    }
  }
}

}  // namespace

cudaError_t launch_select_topk(const SelectParams& p, cudaStream_t st) {
  static size_t configured = 0;
  const size_t smem = (size_t)p.smem_keys * 4;
  if (smem > configured) {
    const cudaError_t e = cudaFuncSetAttribute(select_topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    configured = smem;
  }
  select_topk_kernel<<<dim3(p.Hkv, p.B), SEL_THREADS, smem, st>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_compact(const CompactParams& p, cudaStream_t st) {
  if (p.n_keep_max <= 0) return cudaSuccess;
  const int rows_per_block = (256 / (p.row_bytes / 16)) * CP_ROWS_PER_THREAD;
  const dim3 grid((p.n_keep_max + rows_per_block - 1) / rows_per_block, p.Hkv, p.B);
  compact_kv_kernel<<<grid, 256, 0, st>>>(p);
  return cudaGetLastError();
}

}  // namespace sdllm
