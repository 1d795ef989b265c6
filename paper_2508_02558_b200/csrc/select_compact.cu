// Top-k selection over the pooled importance scores and the K/V gather-compaction
// (Algorithm 1: "n <- floor(|I| r)", "TopKIndices(I, n)", "Select(K_f, I)", "Select(V_f, I)").
#include "common.cuh"
#include "tuning.cuh"

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
constexpr int SEL_HIST = 8;               // histogram copies, one per group of warps, to spread shared-memory atomics

struct Segment { int c_lo, c_hi, n; };   // candidate range and how many to keep
constexpr int CP_ROWS_PER_THREAD = 4;    // gather: rows of K and of V in flight per thread

// Exclusive prefix sum of one value per thread over the whole CTA (thread order); `total` receives the sum.
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t* warp_tot, uint32_t* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t incl = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t y = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += y;
  }
  __syncthreads();                        // warp_tot may still be read from a previous scan
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const uint32_t t = warp_tot[lane];
    uint32_t ti = t;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const uint32_t y = __shfl_up_sync(0xffffffffu, ti, d);
      if (lane >= d) ti += y;
    }
    warp_tot[lane] = ti - t;              // exclusive offset of each warp
    if (lane == 31) warp_tot[32] = ti;    // grand total
  }
  __syncthreads();
  *total = warp_tot[32];
  return warp_tot[warp] + incl - v;
}

// One CTA per (sequence, KV head). The candidate keys are staged once in shared memory (coalesced loads, one padding
// word per 32 so that a thread can walk its own contiguous run of candidates without bank conflicts). A radix select
// (4 passes of 8 bits, most significant first, histograms by shared-memory atomics) finds the key of the n-th largest
// candidate and how many candidates equal to it are still to be kept; then every thread counts the survivors of its run,
// two CTA-wide prefix sums turn the counts into output offsets, and the kept positions are written in ascending
// order, ties going to the lowest positions. Counts are integers, so nothing depends on the order in which threads or
// atomics run: the result is deterministic.
__global__ void __launch_bounds__(SEL_THREADS) select_topk_kernel(const SelectParams p) {
  extern __shared__ uint32_t keys_s[];                 // optional cache of the candidate keys, index c + c / 32
  __shared__ uint32_t hist[SEL_HIST][256];
  __shared__ uint32_t warp_tot[SEL_WARPS + 1];
  __shared__ uint32_t sh_prefix, sh_remaining;

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
  auto key_at = [&](int c) -> uint32_t { return cached ? keys_s[c + (c >> 5)] : score_key(sc[cand_pos(c)]); };

  if (cached)
    for (int c = tid; c < C; c += SEL_THREADS) keys_s[c + (c >> 5)] = score_key(sc[cand_pos(c)]);

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
  uint32_t run_out = 0;                                // entries written so far (same value in every thread)
  __syncthreads();

  for (int si = 0; si < n_seg; ++si) {
    const int c_lo = seg[si].c_lo, c_hi = seg[si].c_hi, n = seg[si].n;
    const int len = c_hi - c_lo;
    if (n <= 0 || len <= 0) continue;
    const int kpt = (len + SEL_THREADS - 1) / SEL_THREADS;   // candidates per thread, a contiguous run
    const int my_lo = min(c_lo + tid * kpt, c_hi), my_hi = min(my_lo + kpt, c_hi);
    uint32_t thr = 0u, need_eq = 0u;
    const bool take_all = n >= len;
    if (!take_all) {
      // ---- radix select of the n-th largest key ----
      if (tid == 0) { sh_prefix = 0u; sh_remaining = (uint32_t)n; }
      for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        for (int i = tid; i < SEL_HIST * 256; i += SEL_THREADS) (&hist[0][0])[i] = 0u;
        __syncthreads();
        const uint32_t prefix = sh_prefix;
        const uint32_t remaining = sh_remaining;
        const uint32_t himask = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + 8));
        uint32_t* my_hist = hist[warp & (SEL_HIST - 1)];
        for (int c = my_lo; c < my_hi; ++c) {
          const uint32_t k = key_at(c);
          if ((k & himask) == prefix) atomicAdd(&my_hist[(k >> shift) & 0xFFu], 1u);
        }
        __syncthreads();
        if (tid < 256) {
          uint32_t s = 0;
#pragma unroll
          for (int w = 0; w < SEL_HIST; ++w) s += hist[w][tid];
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
    // ---- ordered emission: a thread's run is contiguous, so thread order is position order ----
    uint32_t my_eq = 0, my_gt = 0;
    for (int c = my_lo; c < my_hi; ++c) {
      const uint32_t k = key_at(c);
      my_gt += (take_all || k > thr) ? 1u : 0u;
      my_eq += (!take_all && k == thr) ? 1u : 0u;
    }
    uint32_t total_eq, total_keep;
    const uint32_t eq_before = block_exclusive_scan(my_eq, warp_tot, &total_eq);
    const uint32_t eq_quota = need_eq > eq_before ? min(need_eq - eq_before, my_eq) : 0u;   // ties kept from this run: its first ones
    const uint32_t out_before = block_exclusive_scan(my_gt + eq_quota, warp_tot, &total_keep);
    uint32_t w = run_out + out_before, eq_seen = 0;
    for (int c = my_lo; c < my_hi; ++c) {
      const uint32_t k = key_at(c);
      bool keep = take_all || k > thr;
      if (!take_all && k == thr) { keep = eq_seen < eq_quota; ++eq_seen; }
      if (keep) {
        if (w < (uint32_t)p.n_keep_max) out[w] = cand_pos(c);
        ++w;
      }
    }
    run_out += total_keep;
  }
  __syncthreads();
  const int kept = min((int)run_out, p.n_keep_max);
  for (int i = kept + tid; i < p.n_keep_max; i += SEL_THREADS) out[i] = -1;
  if (g == 0 && tid == 0) p.kept_cnt[bi] = kept;
}

// ---------------------------------------------------------------------------------------------------------
// Long sequences: the same selection by a thread-block cluster. One CTA per (sequence, KV head) leaves the GPU to a
// handful of SMs when there are few heads and tens of thousands of candidates, so here SELC_CTAS CTAs share a head:
// each stages a contiguous slice of the candidates, the radix passes add the slices' histograms up through
// distributed shared memory (every CTA ends up with the same global histogram and takes the same decision), and the
// ordered emission gets its offsets from the counts of the CTAs before it in position order. All counts are
// integers: the result is the single-CTA kernel's, bit for bit.
constexpr int SELC_CTAS = 8;
constexpr int SELC_SLICE = 8192;          // candidates one CTA can stage

__device__ __forceinline__ void cluster_barrier() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;\n" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;\n" : "=r"(r));
  return r;
}
// Reads the word that lives at `local` in the shared memory of CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t peer_ld_u32(const uint32_t* local, uint32_t rank) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(local);
  uint32_t ra, v;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(ra) : "r"(a), "r"(rank));
  asm volatile("ld.shared::cluster.u32 %0, [%1];\n" : "=r"(v) : "r"(ra) : "memory");
  return v;
}

__global__ void __launch_bounds__(SEL_THREADS) select_topk_cluster_kernel(const SelectParams p) {
  __shared__ uint32_t keys_s[SELC_SLICE + SELC_SLICE / 32 + 1];   // this CTA's slice, index i + i / 32
  __shared__ uint32_t hist[SEL_HIST][256];
  __shared__ uint32_t fold[2][256];       // this CTA's histogram of a pass (two in turn), read by the peers
  __shared__ uint32_t ghist[256];         // the cluster's histogram
  __shared__ uint32_t warp_tot[SEL_WARPS + 1];
  __shared__ uint32_t sh_prefix, sh_remaining;
  __shared__ uint32_t pub_eq[2], pub_keep[2];   // per segment: this CTA's tie and keep counts, read by the peers

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int rank = (int)cluster_rank();
  const int g = blockIdx.y, bi = blockIdx.z;
  int L = p.seq_len ? p.seq_len[bi] : p.Lmax;
  L = min(max(L, 0), p.Lmax);
  const int b = p.b;
  int o = p.block_off[bi];
  o = min(max(o, 0), max(L - b, 0));
  const int C = max(L - b, 0);
  const float* sc = p.pooled + (int64_t)(bi * p.Hkv + g) * p.Lmax;
  int32_t* out = p.kept_idx + (int64_t)(bi * p.Hkv + g) * p.n_keep_max;
  auto cand_pos = [&](int c) { return c < o ? c : c + b; };

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
  uint32_t run_out = 0;                                // entries written so far (same value in every thread of every CTA)
  int pass_id = 0;                                     // radix passes done so far (the same in every CTA)

  for (int si = 0; si < n_seg; ++si) {
    const int c_lo = seg[si].c_lo, c_hi = seg[si].c_hi, n = seg[si].n;
    const int len = c_hi - c_lo;
    if (n <= 0 || len <= 0) continue;                  // the same decision in every CTA of the cluster
    // this CTA's slice of the segment (slices in rank order are in position order), staged in shared memory
    const int chunk = (len + SELC_CTAS - 1) / SELC_CTAS;
    const int s_lo = min(c_lo + rank * chunk, c_hi), s_hi = min(s_lo + chunk, c_hi);
    const int slen = s_hi - s_lo;
    __syncthreads();                                   // the previous segment's keys are no longer read
    for (int i = tid; i < slen; i += SEL_THREADS) keys_s[i + (i >> 5)] = score_key(sc[cand_pos(s_lo + i)]);
    const int kpt = (slen + SEL_THREADS - 1) / SEL_THREADS;   // candidates per thread, a contiguous run of the slice
    const int my_lo = min(tid * kpt, slen), my_hi = min(my_lo + kpt, slen);
    __syncthreads();
    uint32_t thr = 0u, need_eq = 0u;
    const bool take_all = n >= len;
    if (!take_all) {
      // ---- radix select of the n-th largest key of the whole segment ----
      uint32_t prefix = 0u, remaining = (uint32_t)n;
      for (int pass = 0; pass < 4; ++pass, ++pass_id) {
        const int shift = 24 - 8 * pass;
        for (int i = tid; i < SEL_HIST * 256; i += SEL_THREADS) (&hist[0][0])[i] = 0u;
        __syncthreads();
        const uint32_t himask = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + 8));
        uint32_t* my_hist = hist[warp & (SEL_HIST - 1)];
        for (int i = my_lo; i < my_hi; ++i) {
          const uint32_t k = keys_s[i + (i >> 5)];
          if ((k & himask) == prefix) atomicAdd(&my_hist[(k >> shift) & 0xFFu], 1u);
        }
        __syncthreads();
        if (tid < 256) {
          uint32_t s2 = 0;
#pragma unroll
          for (int w = 0; w < SEL_HIST; ++w) s2 += hist[w][tid];
          fold[pass_id & 1][tid] = s2;
        }
        // every CTA's histogram of this pass is complete (and everybody is done with the one of two passes ago)
        cluster_barrier();
        if (tid < 256) {
          uint32_t s2 = 0;
#pragma unroll
          for (int q = 0; q < SELC_CTAS; ++q) s2 += peer_ld_u32(&fold[pass_id & 1][tid], (uint32_t)q);
          ghist[tid] = s2;
        }
        __syncthreads();
        if (warp == 0) {
          // lane handles bins [255 - 8*lane - 7, 255 - 8*lane], scanning downward
          uint32_t local[8], sum = 0;
#pragma unroll
          for (int i = 0; i < 8; ++i) { local[i] = ghist[255 - (8 * lane + i)]; sum += local[i]; }
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
        prefix = sh_prefix;
        remaining = sh_remaining;
      }
      thr = prefix;
      need_eq = remaining;                        // how many candidates equal to thr are still to be kept (>= 1)
    }
    // ---- ordered emission: runs in thread order and slices in rank order are in position order ----
    uint32_t my_eq = 0, my_gt = 0;
    for (int i = my_lo; i < my_hi; ++i) {
      const uint32_t k = keys_s[i + (i >> 5)];
      my_gt += (take_all || k > thr) ? 1u : 0u;
      my_eq += (!take_all && k == thr) ? 1u : 0u;
    }
    uint32_t total_eq, total_keep;
    uint32_t eq_before = block_exclusive_scan(my_eq, warp_tot, &total_eq);
    if (tid == 0) pub_eq[si] = total_eq;
    cluster_barrier();
    for (int q = 0; q < rank; ++q) eq_before += peer_ld_u32(&pub_eq[si], (uint32_t)q);
    const uint32_t eq_quota = need_eq > eq_before ? min(need_eq - eq_before, my_eq) : 0u;   // ties kept from this run: its first ones
    const uint32_t out_before = block_exclusive_scan(my_gt + eq_quota, warp_tot, &total_keep);
    if (tid == 0) pub_keep[si] = total_keep;
    cluster_barrier();
    uint32_t keep_before = 0, keep_all = 0;
#pragma unroll
    for (int q = 0; q < SELC_CTAS; ++q) {
      const uint32_t v = peer_ld_u32(&pub_keep[si], (uint32_t)q);
      keep_all += v;
      if (q < rank) keep_before += v;
    }
    uint32_t w = run_out + keep_before + out_before, eq_seen = 0;
    for (int i = my_lo; i < my_hi; ++i) {
      const uint32_t k = keys_s[i + (i >> 5)];
      bool keep = take_all || k > thr;
      if (!take_all && k == thr) { keep = eq_seen < eq_quota; ++eq_seen; }
      if (keep) {
        if (w < (uint32_t)p.n_keep_max) out[w] = cand_pos(s_lo + i);
        ++w;
      }
    }
    run_out += keep_all;
  }
  cluster_barrier();                                   // nobody leaves while a peer may still read its shared memory
  if (rank == 0) {
    const int kept = min((int)run_out, p.n_keep_max);
    for (int i = kept + tid; i < p.n_keep_max; i += SEL_THREADS) out[i] = -1;
    if (g == 0 && tid == 0) p.kept_cnt[bi] = kept;
  }
}

// Gather of the kept rows: 16 bytes per thread, four rows of K and of V in flight per thread.

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

// ---------------------------------------------------------------------------------------------------------
// Selection and gather in one launch (Algorithm 1 from "n <- floor(|I| r)" to the cache store). R CTAs share a
// (sequence, KV head): every one of them runs the whole selection of the head on its own - the candidates of a head
// are a few kilobytes, so repeating the radix select costs no time and needs no exchange - and leaves the ascending
// list of kept positions in its shared memory. Then CTA r writes the r-th share of kept_idx and copies the K and V rows
// of that share into the compacted cache, 16 bytes per thread with several rows in flight (zero rows and -1 past the
// count). The index list never makes a round trip through global memory and one launch is gone.
// Same integer arithmetic as select_topk_kernel: the result is that kernel's, bit for bit.
template <int NT>
__device__ __forceinline__ uint32_t block_exclusive_scan_t(uint32_t v, uint32_t* warp_tot, uint32_t* total) {
  constexpr int NW = NT / 32;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t incl = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t y = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += y;
  }
  __syncthreads();                        // warp_tot may still be read from a previous scan
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const uint32_t t = lane < NW ? warp_tot[lane] : 0u;
    uint32_t ti = t;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const uint32_t y = __shfl_up_sync(0xffffffffu, ti, d);
      if (lane >= d) ti += y;
    }
    if (lane < NW) warp_tot[lane] = ti - t;   // exclusive offset of each warp
    if (lane == 31) warp_tot[NW] = ti;        // grand total
  }
  __syncthreads();
  *total = warp_tot[NW];
  return warp_tot[warp] + incl - v;
}

template <int NT>
__global__ void __launch_bounds__(NT) select_gather_kernel(const SelectParams p, const CompactParams cp) {
  constexpr int NW = NT / 32;
  constexpr int HC = NW < SEL_HIST ? NW : SEL_HIST;    // histogram copies
  extern __shared__ uint32_t dyn_s[];                  // candidate keys (index c + c / 32), then the kept positions
  __shared__ uint32_t hist[4][HC][256];                // one set per radix pass, cleared once per segment
  __shared__ uint32_t warp_tot[NW + 1];
  __shared__ uint32_t sh_prefix, sh_remaining;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int r = blockIdx.x, R = gridDim.x, g = blockIdx.y, bi = blockIdx.z;
  // Ahead of the grid dependency: what does not depend on the kernel in front - the first segment's histograms and (the
  // caller's lengths and block offsets are older than the scores) the two words that place the block.
  int L = p.Lmax, o = 0;
  if (p.early_inputs) {
    if (p.seq_len) L = __ldcg(p.seq_len + bi);
    o = __ldcg(p.block_off + bi);
  }
  for (int i = tid; i < 4 * HC * 256; i += NT) (&hist[0][0][0])[i] = 0u;
  asm volatile("griddepcontrol.wait;\n" ::: "memory");  // the pooled scores come from the kernel in front
  if (!p.early_inputs) {
    if (p.seq_len) L = p.seq_len[bi];
    o = p.block_off[bi];
  }
  L = min(max(L, 0), p.Lmax);
  const int b = p.b;
  o = min(max(o, 0), max(L - b, 0));
  const int C = max(L - b, 0);
  const float* sc = p.pooled + (int64_t)(bi * p.Hkv + g) * p.Lmax;
  uint32_t* keys_s = dyn_s;
  int32_t* kept_s = reinterpret_cast<int32_t*>(dyn_s + (p.Lmax - b) + (p.Lmax - b) / 32 + 1);
  auto cand_pos = [&](int c) { return c < o ? c : c + b; };
  for (int c = tid; c < C; c += NT) keys_s[c + (c >> 5)] = score_key(sc[cand_pos(c)]);

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
  uint32_t run_out = 0;                                // entries written so far (same value in every thread)
  bool hist_used = false;
  __syncthreads();

  for (int si = 0; si < n_seg; ++si) {
    const int c_lo = seg[si].c_lo, c_hi = seg[si].c_hi, n = seg[si].n;
    const int len = c_hi - c_lo;
    if (n <= 0 || len <= 0) continue;
    const int kpt = (len + NT - 1) / NT;               // candidates per thread, a contiguous run
    const int my_lo = min(c_lo + tid * kpt, c_hi), my_hi = min(my_lo + kpt, c_hi);
    uint32_t thr = 0u, need_eq = 0u;
    const bool take_all = n >= len;
    if (!take_all) {
      // ---- radix select of the n-th largest key: four passes of 8 bits, most significant first ----
      if (tid == 0) { sh_prefix = 0u; sh_remaining = (uint32_t)n; }
      if (hist_used)                               // (the first select finds the histograms cleared at the kernel's start)
        for (int i = tid; i < 4 * HC * 256; i += NT) (&hist[0][0][0])[i] = 0u;
      hist_used = true;
      __syncthreads();
      for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        const uint32_t prefix = sh_prefix;
        const uint32_t remaining = sh_remaining;
        const uint32_t himask = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + 8));
        uint32_t* my_hist = hist[pass][warp % HC];
        // Pooled scores of one head share their leading bits, so most keys of a warp fall into one bin: the lanes of a
        // warp that hit the same bin are counted by one of them (one shared-memory atomic per distinct bin and warp).
        for (int j = 0; j < kpt; ++j) {
          const int c = my_lo + j;
          uint32_t k = 0u;
          bool act = c < my_hi;
          if (act) { k = keys_s[c + (c >> 5)]; act = (k & himask) == prefix; }
          const uint32_t bin = (k >> shift) & 0xFFu;
          const uint32_t same = __match_any_sync(0xffffffffu, act ? bin : 0x100u);
          if (act && (uint32_t)lane == (uint32_t)(__ffs(same) - 1)) atomicAdd(&my_hist[bin], (uint32_t)__popc(same));
        }
        __syncthreads();
        if (tid < 256) {
          uint32_t h = 0;
#pragma unroll
          for (int w = 0; w < HC; ++w) h += hist[pass][w][tid];
          hist[pass][0][tid] = h;
        }
        __syncthreads();
        if (warp == 0) {
          // lane handles bins [255 - 8*lane - 7, 255 - 8*lane], scanning downward
          uint32_t local[8], sum = 0;
#pragma unroll
          for (int i = 0; i < 8; ++i) { local[i] = hist[pass][0][255 - (8 * lane + i)]; sum += local[i]; }
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
    // ---- ordered emission into shared memory: a thread's run is contiguous, so thread order is position order ----
    uint32_t my_eq = 0, my_gt = 0;
    for (int c = my_lo; c < my_hi; ++c) {
      const uint32_t k = keys_s[c + (c >> 5)];
      my_gt += (take_all || k > thr) ? 1u : 0u;
      my_eq += (!take_all && k == thr) ? 1u : 0u;
    }
    uint32_t total_eq, total_keep;
    const uint32_t eq_before = block_exclusive_scan_t<NT>(my_eq, warp_tot, &total_eq);
    const uint32_t eq_quota = need_eq > eq_before ? min(need_eq - eq_before, my_eq) : 0u;   // ties kept from this run: its first ones
    const uint32_t out_before = block_exclusive_scan_t<NT>(my_gt + eq_quota, warp_tot, &total_keep);
    uint32_t w = run_out + out_before, eq_seen = 0;
    for (int c = my_lo; c < my_hi; ++c) {
      const uint32_t k = keys_s[c + (c >> 5)];
      bool keep = take_all || k > thr;
      if (!take_all && k == thr) { keep = eq_seen < eq_quota; ++eq_seen; }
      if (keep) {
        if (w < (uint32_t)p.n_keep_max) kept_s[w] = cand_pos(c);
        ++w;
      }
    }
    run_out += total_keep;
  }
  __syncthreads();
  const int kept = min((int)run_out, p.n_keep_max);
  if (g == 0 && r == 0 && tid == 0) p.kept_cnt[bi] = kept;

  // ---- this CTA's share of the (padded) list: indices out, rows gathered ----
  const int i_lo = (int)(((long long)r * p.n_keep_max) / R), i_hi = (int)(((long long)(r + 1) * p.n_keep_max) / R);
  int32_t* out = p.kept_idx + (int64_t)(bi * p.Hkv + g) * p.n_keep_max;
  for (int i = i_lo + tid; i < i_hi; i += NT) out[i] = i < kept ? kept_s[i] : -1;
  const int chunks = cp.row_bytes / 16;                // threads per row
  const int rows_per_pass = NT / chunks;
  const int c16 = tid % chunks, rl = tid / chunks;
  const char* kb = reinterpret_cast<const char*>(cp.k) + bi * cp.kv_stride_bytes[0] + g * cp.kv_stride_bytes[1];
  const char* vb = reinterpret_cast<const char*>(cp.v) + bi * cp.kv_stride_bytes[0] + g * cp.kv_stride_bytes[1];
  char* kc = reinterpret_cast<char*>(cp.k_c) + bi * cp.c_stride_bytes[0] + g * cp.c_stride_bytes[1];
  char* vc = reinterpret_cast<char*>(cp.v_c) + bi * cp.c_stride_bytes[0] + g * cp.c_stride_bytes[1];
  if (rl < rows_per_pass)
    for (int i0 = i_lo + rl; i0 < i_hi; i0 += CP_ROWS_PER_THREAD * rows_per_pass) {
      uint4 kv[CP_ROWS_PER_THREAD], vv[CP_ROWS_PER_THREAD];
#pragma unroll
      for (int u = 0; u < CP_ROWS_PER_THREAD; ++u) {
        const int i = i0 + u * rows_per_pass;
        kv[u] = make_uint4(0u, 0u, 0u, 0u);
        vv[u] = make_uint4(0u, 0u, 0u, 0u);
        if (i < i_hi && i < kept) {
          const int src = kept_s[i];
          kv[u] = __ldg(reinterpret_cast<const uint4*>(kb + (int64_t)src * cp.kv_stride_bytes[2]) + c16);
          vv[u] = __ldg(reinterpret_cast<const uint4*>(vb + (int64_t)src * cp.kv_stride_bytes[2]) + c16);
        }
      }
#pragma unroll
      for (int u = 0; u < CP_ROWS_PER_THREAD; ++u) {
        const int i = i0 + u * rows_per_pass;
        if (i < i_hi) {
          reinterpret_cast<uint4*>(kc + (int64_t)i * cp.c_stride_bytes[2])[c16] = kv[u];
          reinterpret_cast<uint4*>(vc + (int64_t)i * cp.c_stride_bytes[2])[c16] = vv[u];
        }
      }
    }
}

}  // namespace

cudaError_t launch_select_topk(const SelectParams& p, cudaStream_t st) {
  // Tens of thousands of candidates per head and few heads (all clusters resident at once): a cluster of CTAs per head;
  // with many heads one CTA per head already fills the GPU and measured several times faster than clusters.
  // Tuning::select forces either wherever the cluster kernel applies.
  const int cand = p.Lmax - p.b;
  bool clustered = cand > 8192 && (long long)p.B * p.Hkv * SELC_CTAS <= sm_count();
  const int forced = tuning().select;
  if (forced != 0) clustered = forced == 2;
  if (clustered && cand >= 1 && cand <= SELC_CTAS * SELC_SLICE) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(SELC_CTAS, p.Hkv, p.B);
    cfg.blockDim = dim3(SEL_THREADS);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = SELC_CTAS; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, select_topk_cluster_kernel, p);
  }
  static SmemConfig configured;
  const size_t smem = ((size_t)p.smem_keys + p.smem_keys / 32 + 1) * 4;
  const cudaError_t e = configure_smem(reinterpret_cast<const void*>(select_topk_kernel), smem, configured, false);
  if (e != cudaSuccess) return e;
  select_topk_kernel<<<dim3(p.Hkv, p.B), SEL_THREADS, smem, st>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_compact(const CompactParams& p, cudaStream_t st);

// Whether selection and gather run as one launch: the candidates and the kept list of a head must fit the shared memory
// of a CTA; longer sequences take the two kernels above one after the other.
bool select_compact_is_fused(int Lmax, int b, int n_keep_max) {
  const int cand = Lmax - b;
  return cand >= 1 && cand <= 8192 && n_keep_max >= 1 && tuning().select == 0;
}

cudaError_t launch_select_compact(const SelectParams& p, const CompactParams& cp, cudaStream_t st) {
  if (!select_compact_is_fused(p.Lmax, p.b, p.n_keep_max)) {
    const cudaError_t e = launch_select_topk(p, st);
    return e != cudaSuccess ? e : launch_compact(cp, st);
  }
  const int cand = p.Lmax - p.b;
  const size_t smem = ((size_t)cand + cand / 32 + 1 + p.n_keep_max) * 4;
  // CTAs per head: fill the SMs, but leave every CTA at least 64 rows to copy
  long long R = sm_count() / ((long long)p.B * p.Hkv);
  if (R > p.n_keep_max / 64) R = p.n_keep_max / 64;
  if (tuning().splits > 0) R = tuning().splits;
  if (R > 16) R = 16;
  if (R < 1) R = 1;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)R, p.Hkv, p.B);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  int na = 0;
  if (tuning().pdl != 0) {      // starts while the kernel in front finishes; never releases its own dependents early
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  cfg.attrs = attr; cfg.numAttrs = na;
  static SmemConfig configured;
  const cudaError_t e = configure_smem(reinterpret_cast<const void*>(select_gather_kernel<SEL_THREADS>), smem, configured, false);
  if (e != cudaSuccess) return e;
  cfg.blockDim = dim3(SEL_THREADS);
  return cudaLaunchKernelEx(&cfg, select_gather_kernel<SEL_THREADS>, p, cp);
}

cudaError_t launch_compact(const CompactParams& p, cudaStream_t st) {
  if (p.n_keep_max <= 0) return cudaSuccess;
  const int rows_per_block = (256 / (p.row_bytes / 16)) * CP_ROWS_PER_THREAD;
  const dim3 grid((p.n_keep_max + rows_per_block - 1) / rows_per_block, p.Hkv, p.B);
  compact_kv_kernel<<<grid, 256, 0, st>>>(p);
  return cudaGetLastError();
}

}  // namespace sdllm
