// bf16 block-query attention on the fifth-generation tensor cores (tcgen05) of sm_100a.
//
// One CTA owns (sequence, KV head, 128-row tile of the head's b*G query rows, key split) and streams its share of
// the key axis  [source 1 rows 0..n1) ++ [source 2 rows 0..n2)  exactly once:
//   refresh step : source 1 = the full K/V of the sequence, no source 2;
//   reuse step   : source 1 = the compacted cache, source 2 = the block's fresh rows (Algorithm 3, Concat(K_c, K_n)).
// Warp roles (256 threads):
//   warp 0      TMA producer: K and V tiles (128-byte swizzle) into a shared-memory ring, one mbarrier pair per slot
//   warp 1      one thread issues tcgen05.mma: S = Q K^T (A, B from shared memory) into TMEM, then
//               O_tile = P V with P read from TMEM (A) and V from shared memory (B, MN-major)
//   warps 2-5   softmax: each thread owns one of the 128 accumulator rows (TMEM lane), reads its S row with
//               tcgen05.ld, keeps the running max / sum and writes P (bf16) over S in TMEM; O accumulates in TMEM
//               across the tiles and is rescaled in place only when a row's maximum grows by more than 2^8
//   warps 6-7   refresh only: mean-query saliency of every streamed key (Algorithm 1, "qbar <- Mean(Q_b)",
//               "A <- MatMul(qbar, K_f^T)") from the K tile in shared memory, fp32
// When b*G <= 64 the query rows are replicated R = 2 or 4 times along the 128 accumulator rows and every replica
// takes its own slice of each key tile, so all four softmax warps work; the replicas are merged like key splits.
// The replicas are merged inside the CTA through shared memory. Key splits leave (max, sum, O) partials in the
// workspace. While the tail is small, the last CTA of a (sequence, KV head, row tile) to finish - found with one
// atomic counter, nobody waits - merges them, writes the output and, at the refresh step, pools the head's saliency
// along the key axis (Algorithm 1, MaxPool1D); for large partial volumes or long sequences a second small launch
// does the same work spread over the whole GPU.
//
// Every wait on an mbarrier is bounded. On expiry the thread sets an abort flag that all other waits poll, records a
// code in the status word and the CTA runs to its end (freeing its TMEM); the outputs of that call are then invalid.
#include <cuda.h>
#include <string.h>

#include "attn_device.cuh"
#include "tuning.cuh"
#include "umma_host.cuh"

namespace sdllm {
using namespace dev;
namespace {

constexpr int UM_THREADS = 256;
constexpr int UM_STAGES = 3;

struct UmmaMaps {
  CUtensorMap q, k1, v1, k2, v2;
};

struct UmmaParams {
  AttnParams a;
  int KT;            // rows of a source-1 tile (64 or 128)
  int KT2;           // rows of a source-2 tile (<= KT, multiple of 16)
  int R;             // replicas of the query rows along the 128 accumulator rows (1, 2, 4)
  int row_tiles;     // 128-row tiles of the b*G rows
  int heads_rt;      // query heads per row tile
  int fused_tail;    // 1: the last CTA of a unit merges and pools; 0: umma_tail_kernel does
  int early_src1;    // 1: source 1 and its count are older than the previous kernel in the stream (reuse step)
  int prob_pass;     // 1: second pass of the probability saliency: S and the rows' log-sum-exp give column means of P
  int cluster;       // > 1: the key splits of a unit form a thread-block cluster and merge through distributed shared memory
  int lpt;           // 1: grid z counts the sequences from the longest to the shortest (several waves of ragged work)
};

#include "umma_ptx.cuh"

// Importance of one absolute position: Algorithm 1, MaxPool1D(A, kernel_size = s, padding = s/2) over the candidate
// axis Concat(prefix, suffix) (AvgPool for the ablation); block positions and padding get -inf. `a` holds the raw
// saliency by absolute position.
__device__ __forceinline__ float pool_at(const AttnParams& p, const float* a, int L, int o_in, int pos, int n_arr = 1,
                                         int64_t arr_stride = 0) {
  const int b = p.b;
  const int o = min(max(o_in, 0), max(L - b, 0));
  if (pos >= L || (pos >= o && pos < o + b)) return -INFINITY;
  const int C = max(L - b, 0), w = (p.window - 1) / 2;
  const int c = pos < o ? pos : pos - b;
  int lo = 0, hi = C;
  if (p.per_region) { if (c < o) hi = o; else lo = o; }
  float mx = -INFINITY, sum = 0.f;
  for (int t = c - w; t <= c + w; ++t) {
    if (t < lo || t >= hi) continue;
    float x = a[t < o ? t : t + b];
    for (int r2 = 1; r2 < n_arr; ++r2) x += a[r2 * arr_stride + (t < o ? t : t + b)];   // one array per row tile
    mx = fmaxf(mx, x);
    sum += x;
  }
  return p.pool_kind == SDLLM_POOL_MAX ? mx : sum / (float)p.window;
}

// The same, reading the raw saliency from global memory through L2 (other CTAs wrote it during this launch).
__device__ __forceinline__ float pool_at_ldcg(const AttnParams& p, const float* a, int L, int o_in, int pos) {
  const int b = p.b;
  const int o = min(max(o_in, 0), max(L - b, 0));
  if (pos >= L || (pos >= o && pos < o + b)) return -INFINITY;
  const int C = max(L - b, 0), w = (p.window - 1) / 2;
  const int c = pos < o ? pos : pos - b;
  int lo = 0, hi = C;
  if (p.per_region) { if (c < o) hi = o; else lo = o; }
  float mx = -INFINITY, sum = 0.f;
  for (int t = c - w; t <= c + w; ++t) {
    if (t < lo || t >= hi) continue;
    const float x = __ldcg(a + (t < o ? t : t + b));
    mx = fmaxf(mx, x);
    sum += x;
  }
  return p.pool_kind == SDLLM_POOL_MAX ? mx : sum / (float)p.window;
}

// Merge of the key-split partials of S (row, float4 column) slots of a unit and the final stores. slot[s] < 0 marks
// an unused entry. The partials are read in batches of MB per slot with the loads of all slots and of the whole batch
// in flight together (one L2 latency per batch) and folded with a running maximum, so that four splits cost a single
// round trip for everything a thread merges.
template <int D, int MB, int S>
__device__ __forceinline__ void merge_slots(const AttnParams& p, int64_t unit, int bi, int g, int rt, const int (&slot)[S]) {
  constexpr int D4 = D / 4;
  const int P = p.splits;
  const int prt = min(p.M, 128);                      // rows of one partial
  const float2* ml_base = reinterpret_cast<const float2*>(p.part_ml) + unit * P * prt;
  const float4* po_base = reinterpret_cast<const float4*>(p.part_o + unit * P * prt * D);
  float4 acc[S];
  float l[S], m_run[S];
  int m_local[S], d4[S];
#pragma unroll
  for (int s = 0; s < S; ++s) {
    acc[s] = make_float4(0.f, 0.f, 0.f, 0.f); l[s] = 0.f; m_run[s] = -INFINITY;
    const int sl = max(slot[s], 0);
    m_local[s] = sl / D4; d4[s] = sl - m_local[s] * D4;
  }
  for (int p0 = 0; p0 < P; p0 += MB) {
    float2 x[S][MB];
    float4 o[S][MB];
#pragma unroll
    for (int s = 0; s < S; ++s)
#pragma unroll
      for (int u = 0; u < MB; ++u) {
        const int pi = min(p0 + u, P - 1);
        x[s][u] = __ldcg(ml_base + (int64_t)pi * prt + m_local[s]);
        o[s][u] = __ldcg(po_base + ((int64_t)pi * prt + m_local[s]) * D4 + d4[s]);
      }
#pragma unroll
    for (int s = 0; s < S; ++s) {
      float bm = m_run[s];
#pragma unroll
      for (int u = 0; u < MB; ++u)
        if (p0 + u < P && x[s][u].y > 0.f) bm = fmaxf(bm, x[s][u].x);
      const float a = (bm == -INFINITY) ? 1.f : fast_exp2(m_run[s] - bm);    // 0 on the first batch with data
      acc[s].x *= a; acc[s].y *= a; acc[s].z *= a; acc[s].w *= a; l[s] *= a;
      m_run[s] = bm;
#pragma unroll
      for (int u = 0; u < MB; ++u) {
        if (p0 + u >= P || !(x[s][u].y > 0.f)) continue;
        const float w = fast_exp2(x[s][u].x - bm);
        l[s] = fmaf(x[s][u].y, w, l[s]);
        acc[s].x = fmaf(o[s][u].x, w, acc[s].x); acc[s].y = fmaf(o[s][u].y, w, acc[s].y);
        acc[s].z = fmaf(o[s][u].z, w, acc[s].z); acc[s].w = fmaf(o[s][u].w, w, acc[s].w);
      }
    }
  }
#pragma unroll
  for (int s = 0; s < S; ++s) {
    if (slot[s] < 0) continue;
    const float inv = l[s] > 0.f ? 1.f / l[s] : 0.f;
    const int m = rt * 128 + m_local[s];
    const int hg = m / p.b, i = m - hg * p.b;
    __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(p.out) + (int64_t)bi * p.o_stride[0] +
                         (int64_t)(g * p.G + hg) * p.o_stride[1] + (int64_t)i * p.o_stride[2] + d4[s] * 4;
    uint2 w2;
    w2.x = pack_bf16(acc[s].x * inv, acc[s].y * inv);
    w2.y = pack_bf16(acc[s].z * inv, acc[s].w * inv);
    *reinterpret_cast<uint2*>(out) = w2;
    if (d4[s] == 0 && p.lse) p.lse[((int64_t)bi * p.Hq + g * p.G + hg) * p.b + i] = (m_run[s] + log2f(l[s])) * kLn2;
  }
}

// Deferred tail (large partial volumes or long sequences): one launch that merges the key splits, one thread per
// (row, float4 column), and pools the saliency, one thread per position.
template <int D>
__global__ void __launch_bounds__(256) umma_tail_kernel(const UmmaParams up, const int merge_blocks) {
  const AttnParams& p = up.a;
  grid_dependency_wait();
  grid_launch_dependents();
  if ((int)blockIdx.x < merge_blocks) {
    constexpr int D4 = D / 4;
    const int64_t slot = (int64_t)blockIdx.x * 256 + threadIdx.x;
    const int d4 = (int)(slot % D4);
    const int64_t r = slot / D4;
    const int m_local = (int)(r % 128);
    const int64_t unit = r / 128;
    if (unit >= (int64_t)p.B * p.Hkv * up.row_tiles) return;
    const int rt = (int)(unit % up.row_tiles);
    const int64_t bg = unit / up.row_tiles;
    const int g = (int)(bg % p.Hkv), bi = (int)(bg / p.Hkv);
    if (m_local >= min(p.M - rt * 128, 128)) return;
    const int one[1] = {m_local * D4 + d4};
    merge_slots<D, 8, 1>(p, unit, bi, g, rt, one);
    return;
  }
  const int64_t idx = (int64_t)(blockIdx.x - merge_blocks) * 256 + threadIdx.x;
  if (idx >= (int64_t)p.B * p.Hkv * p.n1_max) return;
  const int pos = (int)(idx % p.n1_max);
  const int64_t bh = idx / p.n1_max;
  const int bi = (int)(bh / p.Hkv);
  int L = p.n1_per_seq ? p.n1_per_seq[bi] : p.n1_max;
  L = min(max(L, 0), p.n1_max);
  p.pooled[idx] = pool_at(p, p.raw_scores + bh * p.n1_max, L, p.block_off[bi], pos, up.prob_pass ? up.row_tiles : 1,
                          (int64_t)p.B * p.Hkv * p.n1_max);
}

// PROB selects the second pass of the probability saliency; it is a template parameter so that the attention kernel proper
// does not carry that pass's code.
// DUAL is the small-footprint variant for grids of several waves: 64-key tiles, a two-slot ring, 256 TMEM columns and at
// most 128 registers per thread, so that two CTAs share an SM and one's set-up and way out overlap the other's streaming.
template <int D, bool PROB, bool DUAL>
__global__ void __launch_bounds__(UM_THREADS, DUAL ? 2 : 1) attn_umma_bf16_kernel(const __grid_constant__ UmmaMaps tm, const UmmaParams up) {
  constexpr int H = D / 64;            // 128-byte column halves of a row
  constexpr int NS = DUAL ? 2 : UM_STAGES;
  constexpr int NCH = DUAL ? 2 : 4;    // 32-column chunks of a key tile
  constexpr uint32_t S_STRIDE = DUAL ? 64 : 128;   // TMEM columns: the two S/P buffers, then the O accumulator
  constexpr uint32_t O_COL = 2 * S_STRIDE;
  constexpr uint32_t TMEM_COLS = DUAL ? 256 : 512;
  constexpr int CTRL = DUAL ? 4096 : 1024;         // control block: barriers, flags, qbar (and the merge scratch if DUAL)
  const AttnParams& p = up.a;
  extern __shared__ unsigned char smem_raw[];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int KT = up.KT, KT2 = up.KT2, R = up.R;
  const int rows_rep = 128 / R;
  // Which sequence: grid z itself, or, for ragged batches that take several waves, the sequence of that rank when the
  // batch is ordered from the longest to the shortest - CTAs are handed out in grid order, so the long ones start first
  // and the short ones fill the tail. Every warp ranks the (at most 64) lengths on its own: no shared memory, no barrier.
  int bi = blockIdx.z;
  if (up.lpt) {
    if (!up.early_src1) grid_dependency_wait();        // the lengths may come from the kernel in front
    const int lane_ = threadIdx.x & 31;
    const int l0 = lane_ < p.B ? p.n1_per_seq[lane_] : -1, l1 = lane_ + 32 < p.B ? p.n1_per_seq[lane_ + 32] : -1;
    int r0 = 0, r1 = 0;                                // how many sequences come before mine (longer, or equal and earlier)
    for (int i = 0; i < p.B; ++i) {
      const int li = __shfl_sync(0xffffffffu, i < 32 ? l0 : l1, i & 31);
      r0 += (li > l0 || (li == l0 && i < lane_)) ? 1 : 0;
      r1 += (li > l1 || (li == l1 && i < lane_ + 32)) ? 1 : 0;
    }
    const unsigned hit0 = __ballot_sync(0xffffffffu, lane_ < p.B && r0 == (int)blockIdx.z);
    const unsigned hit1 = __ballot_sync(0xffffffffu, lane_ + 32 < p.B && r1 == (int)blockIdx.z);
    bi = hit0 ? __ffs(hit0) - 1 : (hit1 ? __ffs(hit1) + 31 : (int)blockIdx.z);
  }
  const int g = blockIdx.y / up.row_tiles, rt = blockIdx.y - g * up.row_tiles;
  const int split = blockIdx.x;
  const int tiles1 = (p.n1_max + KT - 1) / KT;
  const int tiles2 = (p.n2 + KT2 - 1) / KT2;
  const int tiles_all = tiles1 + tiles2;
  const int t_begin = (int)(((long long)split * tiles_all) / p.splits);
  const int t_end = (int)(((long long)(split + 1) * tiles_all) / p.splits);
  const int M_rt = min(p.M - rt * 128, 128);          // valid query rows of this row tile (<= rows_rep when R > 1)
  constexpr bool prob_pass = PROB;                      // no V, no PV: S tiles only, reduced over the query rows
  const bool do_attn = p.out != nullptr && !prob_pass;
  const bool do_s = do_attn || prob_pass;              // Q and the S = Q K^T tiles are needed
  const bool do_scores = p.want_scores && rt == 0 && !prob_pass;   // mean-query logit saliency (saliency warps)
  const int n2 = p.n2;

  // ---- shared memory carve-up (1024-byte aligned for the 128-byte swizzle) ----
  const uint32_t raw_addr = smem_u32(smem_raw);
  unsigned char* smem = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
  const uint32_t bars = smem_u32(smem);
  auto BAR = [&](int i) { return bars + 8u * (uint32_t)i; };
  const int Q_FULL = 0, FULL_K = 1, FULL_V = 1 + NS, EMPTY_K = 1 + 2 * NS, EMPTY_V = 1 + 3 * NS;
  const int S_FULL = 1 + 4 * NS, P_FULL = S_FULL + 2, PV_DONE = S_FULL + 4, DRAIN = S_FULL + 6;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + 256);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + 260);
  int* last_flag = reinterpret_cast<int*>(smem + 264);
  float* qbar_s = reinterpret_cast<float*>(smem + 512);
  unsigned char* q_s = smem + CTRL;
  unsigned char* stage0 = q_s + H * 128 * 128;
  const int half_bytes = KT * 128;                     // one 64-column half of a K or V tile
  const int kv_bytes = H * half_bytes;                 // a whole K (or V) tile
  const int stage_bytes = 2 * kv_bytes;
  // The Q box (b rows x the row tile's heads) is loaded as many times as it fits into the 128 accumulator rows: every
  // replica starts on a copy, and rows past the valid ones hold real data whose results are simply not used. Only a box
  // that does not divide 128 leaves rows uncovered; those must not hold non-finite garbage and are cleared first.
  const int q_rows = p.b * up.heads_rt;
  const int q_copies = (128 % q_rows == 0) ? 128 / q_rows : R;
  const int q_step = (128 % q_rows == 0) ? q_rows : rows_rep;
  const bool zero_q = do_s && 128 % q_rows != 0 && q_rows < rows_rep;
  if (tid == 0) {                        // the descriptors live in the kernel parameters: fetch them while the CTA sets up
    prefetch_tmap(&tm.k1); prefetch_tmap(&tm.v1);
    if (n2 > 0) { prefetch_tmap(&tm.k2); prefetch_tmap(&tm.v2); }
    if (do_s) prefetch_tmap(&tm.q);
  }

  // The producer lane sets the barriers up and, unless the Q tile has to be cleared first, starts the first loads
  // before the rest of the CTA is ready: the loads need nothing but the barriers.
  int prod_it = 0, prod_t = t_begin, prod_n1 = 0;
  bool prod_ok = true;
  bool q_issued = false;
  auto issue_q = [&]() {              // the Q tile (replicated R times along the accumulator rows)
    q_issued = true;
    if (!do_s) return;
    mbar_expect_tx(BAR(Q_FULL), (uint32_t)(q_copies * H * q_rows * 128));
    for (int c = 0; c < q_copies; ++c)
      for (int h = 0; h < H; ++h)
        tma_load_4d(smem_u32(q_s + h * 128 * 128 + c * q_step * 128), &tm.q, BAR(Q_FULL), h * 64, 0,
                    g * p.G + rt * up.heads_rt, bi);
  };
  // issue loads for up to `limit` further tiles (producer lane only); with src1_only, stop in front of source 2
  auto produce = [&](int limit, bool src1_only) {
    while (prod_t < t_end && limit > 0 && prod_ok) {
      const Tile x = tile_of(prod_t, tiles1, KT, KT2, prod_n1, n2);
      if (src1_only && !x.src1) break;
      ++prod_t;
      if (x.nv == 0) continue;
      const int it = prod_it, s = it % NS;
      const uint32_t ph = ((it / NS) - 1) & 1;
      const uint32_t kdst = smem_u32(stage0 + (size_t)s * stage_bytes), vdst = kdst + kv_bytes;
      const CUtensorMap* mk = x.src1 ? &tm.k1 : &tm.k2;
      const CUtensorMap* mv = x.src1 ? &tm.v1 : &tm.v2;
      const uint32_t tile_tx = (uint32_t)(H * (x.src1 ? KT : KT2) * 128);
      if (it >= NS && !wait_bar(BAR(EMPTY_K + s), ph, abort_flag, p.status, 1, p.wait_cycles)) { prod_ok = false; break; }
      mbar_expect_tx(BAR(FULL_K + s), tile_tx);
      for (int h = 0; h < H; ++h) tma_load_4d(kdst + h * half_bytes, mk, BAR(FULL_K + s), h * 64, x.row0, g, bi);
      if (do_attn) {
        if (it >= NS && !wait_bar(BAR(EMPTY_V + s), ph, abort_flag, p.status, 2, p.wait_cycles)) { prod_ok = false; break; }
        mbar_expect_tx(BAR(FULL_V + s), tile_tx);
        for (int h = 0; h < H; ++h) tma_load_4d(vdst + h * half_bytes, mv, BAR(FULL_V + s), h * 64, x.row0, g, bi);
      }
      ++prod_it;
      --limit;
    }
  };

  if (tid == 0) {
    mbar_init(BAR(Q_FULL), 1);
    for (int s = 0; s < NS; ++s) {
      mbar_init(BAR(FULL_K + s), 1);
      mbar_init(BAR(FULL_V + s), 1);
      mbar_init(BAR(EMPTY_K + s), max((do_s ? 1 : 0) + (do_scores ? 2 : 0), 1));
      mbar_init(BAR(EMPTY_V + s), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(BAR(S_FULL + i), 1);
      mbar_init(BAR(P_FULL + i), 4);
      mbar_init(BAR(PV_DONE + i), 1);
    }
    mbar_init(BAR(DRAIN), 1);
    *abort_flag = 0;
    *last_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    if (!zero_q && (do_s || do_scores)) {
      if (up.early_src1) {
        // Reuse step: the compacted cache and its count were written before the previous kernel in the stream even
        // started, so their tiles may stream in while that kernel is still finishing.
        prod_n1 = p.n1_per_seq ? p.n1_per_seq[bi] : p.n1_max;
        prod_n1 = min(max(prod_n1, 0), p.n1_max);
        produce(NS, true);             // the first NS slots are free: no waiting here
      }
      grid_dependency_wait();          // the loads below read what earlier kernels in the stream wrote
      if (!up.early_src1) {
        prod_n1 = p.n1_per_seq ? p.n1_per_seq[bi] : p.n1_max;
        prod_n1 = min(max(prod_n1, 0), p.n1_max);
      }
      issue_q();
      produce(NS - prod_it, false);
    }
  }
  if (zero_q)
    for (int i = tid; i < H * 128 * 128 / 16; i += UM_THREADS) reinterpret_cast<uint4*>(q_s)[i] = make_uint4(0u, 0u, 0u, 0u);
  if (warp == 1) {                     // the MMA warp owns the tensor memory
    tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
    tmem_relinquish();
  }
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  grid_dependency_wait();              // everything below may read what earlier kernels in the stream wrote
  grid_launch_dependents();

  int n1 = p.n1_per_seq ? p.n1_per_seq[bi] : p.n1_max;
  n1 = min(max(n1, 0), p.n1_max);

  // softmax state of this thread's accumulator row (softmax warps only)
  float m_run = -INFINITY, l_run = 0.f;
  bool sm_ok = true;
  int sm_tiles = 0;

  if (warp == 0) {
    // ======================================= TMA producer =======================================
    if (lane == 0 && (do_s || do_scores)) {
      prod_n1 = n1;
      if (!q_issued) issue_q();
      produce(1 << 30, false);
      if (*abort_flag) {
        // let the copies that were issued land before the CTA retires
        for (int j = max(prod_it - NS, 0); j < prod_it; ++j) {
          drain_bar(BAR(FULL_K + j % NS), (j / NS) & 1);
          if (do_attn) drain_bar(BAR(FULL_V + j % NS), (j / NS) & 1);
        }
        if (do_s && q_issued) drain_bar(BAR(Q_FULL), 0);
      }
    }
  } else if (warp == 1) {
    // ======================================= MMA issuer =======================================
    if (lane == 0 && do_s) {
      const uint32_t idesc_pv = instr_desc(D, true);
      bool ok = true, have_q = false;
      int it = 0;
      Tile prev{}; int prev_it = -1;
      auto issue_pv = [&](const Tile& x, int j) -> bool {
        const int s = j % NS, pb = j & 1;
        if (!wait_bar(BAR(P_FULL + pb), (j >> 1) & 1, abort_flag, p.status, 4, p.wait_cycles)) return false;
        if (!wait_bar(BAR(FULL_V + s), (j / NS) & 1, abort_flag, p.status, 5, p.wait_cycles)) return false;
        tc_fence_after();
        const uint32_t vsm = smem_u32(stage0 + (size_t)s * stage_bytes) + kv_bytes;
        const uint32_t a_t = tmem_base + (uint32_t)pb * S_STRIDE;
        for (int ks = 0; ks < x.n_mma / 16; ++ks)
          mma_ts(tmem_base + O_COL, a_t + ks * 8, smem_desc(vsm + ks * 2048, (uint32_t)half_bytes, 1024u), idesc_pv,
                 (j > 0 || ks > 0) ? 1u : 0u);
        tc_commit(BAR(PV_DONE + pb));  // two alternating barriers: a waiter is never a whole phase ahead of either
        tc_commit(BAR(EMPTY_V + s));
        return true;
      };
      for (int t = t_begin; t < t_end && ok; ++t) {
        const Tile x = tile_of(t, tiles1, KT, KT2, n1, n2);
        if (x.nv == 0) continue;
        const int s = it % NS, sb = it & 1;
        if (!wait_bar(BAR(FULL_K + s), (it / NS) & 1, abort_flag, p.status, 7, p.wait_cycles)) { ok = false; break; }
        if (!have_q) {
          if (!wait_bar(BAR(Q_FULL), 0, abort_flag, p.status, 3, p.wait_cycles)) { ok = false; break; }
          have_q = true;
        }
        // without PV nothing else orders the reuse of an S buffer: wait until the softmax warps have read tile it - 2
        if (prob_pass && it >= 2 && !wait_bar(BAR(P_FULL + sb), ((it >> 1) - 1) & 1, abort_flag, p.status, 12, p.wait_cycles)) { ok = false; break; }
        tc_fence_after();
        const uint32_t ksm = smem_u32(stage0 + (size_t)s * stage_bytes);
        const uint32_t qsm = smem_u32(q_s);
        const uint32_t idesc_s = instr_desc(x.n_mma, false);
        const uint32_t d_t = tmem_base + (uint32_t)sb * S_STRIDE;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint32_t hq = (ks >> 2) * (128 * 128) + (ks & 3) * 32;
          const uint32_t hk = (ks >> 2) * half_bytes + (ks & 3) * 32;
          mma_ss(d_t, smem_desc(qsm + hq, 16u, 1024u), smem_desc(ksm + hk, 16u, 1024u), idesc_s, ks > 0 ? 1u : 0u);
        }
        tc_commit(BAR(S_FULL + sb));
        tc_commit(BAR(EMPTY_K + s));
        if (do_attn && prev_it >= 0 && !issue_pv(prev, prev_it)) { ok = false; break; }
        prev = x; prev_it = it;
        ++it;
      }
      if (do_attn && ok && prev_it >= 0) ok = issue_pv(prev, prev_it);
      // a CTA whose slice holds no valid key never used Q: its load must still have landed before the CTA retires
      if (ok && !have_q) ok = wait_bar(BAR(Q_FULL), 0, abort_flag, p.status, 3, p.wait_cycles);
      if (*abort_flag) {               // wait for the tensor pipe to finish what was issued before TMEM is freed
        tc_commit(BAR(DRAIN));
        drain_bar(BAR(DRAIN), 0);
      }
    }
  } else if (warp < 6) {
    // ======================================= softmax warps =======================================
    if constexpr (PROB) {
      // Probability saliency, second pass: with the rows' log-sum-exp known, P_ij = exp(S_ij - lse_i) is final, and
      // the saliency of key j is the mean of column j over the b*G query rows. Each warp sums its 32 rows of a
      // 32-column chunk with a shuffle transpose (lane i ends up with column i); the four warps' sums meet in shared
      // memory (the V half of ring slot 0, never loaded in this pass), double-buffered by tile parity.
      const int q4 = warp & 3;
      const int row = q4 * 32 + lane;
      const int rep = row / rows_rep, m_local = row - rep * rows_rep;
      const uint32_t lane_addr = tmem_base + ((uint32_t)(q4 * 32) << 16);
      const int chunk_keys = KT / R;
      float* colsum = reinterpret_cast<float*>(stage0 + kv_bytes);          // [2][4][KT]
      float lse2 = INFINITY;                           // rows outside the tile contribute exp2(-inf) = 0
      if (m_local < M_rt) {
        const int m = rt * 128 + m_local;
        const int hg = m / p.b, i = m - hg * p.b;
        lse2 = p.lse_in[((int64_t)bi * p.Hq + g * p.G + hg) * p.b + i] * kLog2e;
      }
      const float inv_rows = 1.f / (float)p.M;
      float* raw = p.raw_scores + ((int64_t)rt * p.B * p.Hkv + (int64_t)(bi * p.Hkv + g)) * p.n1_max;
      const int st = (warp - 2) * 32 + lane;
      int it = 0;
      bool dead = false;
      for (int t = t_begin; t < t_end; ++t) {
        const Tile x = tile_of(t, tiles1, KT, KT2, n1, n2);
        if (x.nv == 0) continue;
        const int sb = it & 1;
        const int c_lo = min(rep * chunk_keys, x.nv), c_hi = min((rep + 1) * chunk_keys, x.nv);
        // a warp that gave up keeps walking the tiles so that the four warps meet at every barrier below
        if (!dead && !wait_bar_warp(BAR(S_FULL + sb), (it >> 1) & 1, abort_flag, p.status, 9, p.wait_cycles)) dead = true;
        tc_fence_after();
        float* cs = colsum + (size_t)sb * 4 * KT + (size_t)(warp - 2) * KT;
#pragma unroll 1
        for (int c = 0; c * 32 < KT && !dead; ++c) {
          float v[32];
          if (c * 32 < c_hi && c * 32 + 32 > c_lo) {
            uint32_t sv[32];
            tmem_ld32(lane_addr + (uint32_t)sb * S_STRIDE + c * 32, sv);
            tc_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const bool in = c * 32 + i >= c_lo && c * 32 + i < c_hi;
              v[i] = in ? fast_exp2(fmaf(__uint_as_float(sv[i]), p.scale_log2, -lse2)) : 0.f;
            }
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) {
              const bool up_half = (lane & off) != 0;
#pragma unroll
              for (int k = 0; k < off; ++k) {
                const float send = up_half ? v[k] : v[k + off];
                const float keep = up_half ? v[k + off] : v[k];
                v[k] = keep + __shfl_xor_sync(0xffffffffu, send, off);
              }
            }
          } else {
            v[0] = 0.f;
          }
          cs[c * 32 + lane] = v[0];
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(BAR(P_FULL + sb));        // the S buffer may be overwritten
        asm volatile("bar.sync 2, 128;\n" ::: "memory");
        if (st < x.nv && x.src1 && !dead) {
          const float* c4 = colsum + (size_t)sb * 4 * KT + st;
          raw[x.row0 + st] = ((c4[0] + c4[KT]) + (c4[2 * KT] + c4[3 * KT])) * inv_rows;
        }
        ++it;
      }
    } else if (do_attn) {
      const int q4 = warp & 3;                         // TMEM lane quadrant this warp may access
      const int row = q4 * 32 + lane;
      const int rep = row / rows_rep;                  // warp-uniform
      const uint32_t lane_addr = tmem_base + ((uint32_t)(q4 * 32) << 16);
      const int chunk_keys = KT / R;                   // key slice of a tile owned by this replica
      int it = 0;
      bool ok = true;
      for (int t = t_begin; t < t_end && ok; ++t) {
        const Tile x = tile_of(t, tiles1, KT, KT2, n1, n2);
        if (x.nv == 0) continue;
        const int s = it % NS, sb = it & 1;
        // columns of this tile owned by this replica; a warp whose 32 accumulator rows all lie beyond the valid rows of
        // its replica owns nothing
        const bool idle = q4 * 32 - rep * rows_rep >= M_rt;
        const int c_lo = idle ? x.nv : min(rep * chunk_keys, x.nv), c_hi = min((rep + 1) * chunk_keys, x.nv);
        if (!wait_bar_warp(BAR(S_FULL + sb), (it >> 1) & 1, abort_flag, p.status, 9, p.wait_cycles)) { ok = false; break; }
        tc_fence_after();
        const uint32_t s_addr = lane_addr + (uint32_t)sb * S_STRIDE;
        // ---- the owned part of the S row. Chunks of 32 columns that are owned and valid as a whole go through the
        //      unrolled register path, all their loads in flight together; the one chunk the end of the slice may cut
        //      (cp) takes a small predicated path of its own, so the common code stays short ----
        const int cf_lo = c_lo >> 5, cf_hi = c_hi >> 5;          // full chunks [cf_lo, cf_hi); c_lo is a multiple of 32
        const int cp = (c_hi & 31) && c_lo < c_hi ? cf_hi : -1;  // partial chunk, if any
        uint32_t sv[NCH][32];
#pragma unroll
        for (int c = 0; c < NCH; ++c)
          if (c >= cf_lo && c < cf_hi) tmem_ld32(s_addr + c * 32, sv[c]);
        uint32_t tv[32];
        if (cp >= 0) tmem_ld32(s_addr + cp * 32, tv);
        tc_wait_ld();
        float mx = -INFINITY;
#pragma unroll
        for (int c = 0; c < NCH; ++c)
          if (c >= cf_lo && c < cf_hi) {
            float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int i = 0; i < 32; ++i) m4[i & 3] = fmaxf(m4[i & 3], __uint_as_float(sv[c][i]));
            mx = fmaxf(mx, fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3])));
          }
        if (cp >= 0) {
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (cp * 32 + i >= c_lo && cp * 32 + i < c_hi) mx = fmaxf(mx, __uint_as_float(tv[i]));
        }
        // ---- running maximum: O (in TMEM) and l are rescaled only when the maximum grows by more than 2^8, so P stays
        //      below 2^8 and the accumulator is touched on very few tiles ----
        const float m_new = fmaxf(m_run, mx * p.scale_log2);
        const bool grow = m_new > m_run + 8.f;          // also true on the first finite maximum
        float alpha = 1.f;
        if (grow) {
          alpha = fast_exp2(m_run - m_new);             // 0 when m_run is -inf
          m_run = m_new;
          l_run *= alpha;
        }
        if (it > 0 && __any_sync(0xffffffffu, grow)) {
          // every PV issued so far must have landed before the rows are rewritten; PV of this tile waits for our arrive
          if (!wait_bar_warp(BAR(PV_DONE + ((it - 1) & 1)), ((it - 1) >> 1) & 1, abort_flag, p.status, 8, p.wait_cycles)) { ok = false; break; }
          tc_fence_after();
#pragma unroll 1
          for (int c = 0; c < D / 16; ++c) {
            uint32_t ov[16];
            tmem_ld16(lane_addr + O_COL + c * 16, ov);
            tc_wait_ld();
#pragma unroll
            for (int i = 0; i < 16; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * alpha);
            tmem_st16(lane_addr + O_COL + c * 16, ov);
          }
        }
        const float mu = (m_run == -INFINITY) ? 0.f : m_run;
        // ---- P = exp2(S * scale_log2 - mu) as bf16 over the S columns; zero outside the owned slice ----
        float psum = 0.f;
#pragma unroll
        for (int c = 0; c < NCH; ++c)
          if (c >= cf_lo && c < cf_hi) {
            uint32_t pk[16];
            float ps4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float e0 = fast_exp2(fmaf(__uint_as_float(sv[c][2 * i]), p.scale_log2, -mu));
              const float e1 = fast_exp2(fmaf(__uint_as_float(sv[c][2 * i + 1]), p.scale_log2, -mu));
              ps4[i & 3] += e0 + e1;
              pk[i] = pack_bf16(e0, e1);
            }
            psum += (ps4[0] + ps4[1]) + (ps4[2] + ps4[3]);
            tmem_st16(s_addr + c * 16, pk);
          }
        if (cp >= 0) {
          uint32_t pk[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const int j0 = cp * 32 + 2 * i;
            const float e0 = (j0 >= c_lo && j0 < c_hi) ? fast_exp2(fmaf(__uint_as_float(tv[2 * i]), p.scale_log2, -mu)) : 0.f;
            const float e1 = (j0 + 1 >= c_lo && j0 + 1 < c_hi) ? fast_exp2(fmaf(__uint_as_float(tv[2 * i + 1]), p.scale_log2, -mu)) : 0.f;
            psum += e0 + e1;
            pk[i] = pack_bf16(e0, e1);
          }
          tmem_st16(s_addr + cp * 16, pk);
        }
        if (R > 1) {                                    // the other replicas' slices of this tile read as zero
          uint32_t zz[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) zz[i] = 0u;
#pragma unroll 1
          for (int c = 0; c * 32 < x.n_mma; ++c)
            if (!(c >= cf_lo && c < cf_hi) && c != cp) tmem_st16(s_addr + c * 16, zz);
        }
        l_run += psum;
        // ---- V rows past the source's count may hold anything: zero them so that 0 * V stays 0 ----
        if (x.nv < x.n_mma) {
          if (!wait_bar_warp(BAR(FULL_V + s), (it / NS) & 1, abort_flag, p.status, 10, p.wait_cycles)) { ok = false; break; }
          unsigned char* vs = stage0 + (size_t)s * stage_bytes + kv_bytes;
          const int nz = (x.n_mma - x.nv) * H * 8;     // 16-byte chunks to clear
          for (int i = (warp - 2) * 32 + lane; i < nz; i += 128) {
            const int rr = x.nv + i / (H * 8), c = i % (H * 8);
            *reinterpret_cast<uint4*>(vs + (c >> 3) * half_bytes + rr * 128 + (((c & 7) ^ (rr & 7)) << 4)) = make_uint4(0u, 0u, 0u, 0u);
          }
          fence_proxy_async();
        }
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(BAR(P_FULL + sb));
        ++it;
      }
      sm_ok = ok; sm_tiles = it;
    }
  } else {
    // ======================================= saliency warps (refresh) =======================================
    if (do_scores) {
      // qbar <- Mean(Q_b) over the b*G rows of the KV head, fp32, fixed order
      for (int d = tid - 192; d < D; d += 64) {
        float acc = 0.f;
        for (int hg = 0; hg < p.G; ++hg) {
          const __nv_bfloat16* qh = reinterpret_cast<const __nv_bfloat16*>(p.q) + (int64_t)bi * p.q_stride[0] +
                                    (int64_t)(g * p.G + hg) * p.q_stride[1];
          for (int i = 0; i < p.b; ++i) acc += __bfloat162float(qh[(int64_t)i * p.q_stride[2] + d]);
        }
        qbar_s[d] = acc / (float)p.M;
      }
      asm volatile("bar.sync 1, 64;\n" ::: "memory");
      float qb[DUAL ? 8 : D];                            // the whole mean query in registers (DUAL: read per use)
      if constexpr (!DUAL) {
#pragma unroll
        for (int d = 0; d < D; d += 4) {
          const float4 v4 = *reinterpret_cast<const float4*>(qbar_s + d);
          qb[d] = v4.x; qb[d + 1] = v4.y; qb[d + 2] = v4.z; qb[d + 3] = v4.w;
        }
      }
      int it = 0;
      for (int t = t_begin; t < t_end; ++t) {
        const Tile x = tile_of(t, tiles1, KT, KT2, n1, n2);
        if (x.nv == 0) continue;
        const int s = it % NS;
        if (!wait_bar_warp(BAR(FULL_K + s), (it / NS) & 1, abort_flag, p.status, 11, p.wait_cycles)) break;
        if (x.src1) {
          // one key per lane: a_j = scale * <qbar, k_j>; the 128-byte swizzle keeps 32 consecutive rows conflict-free
          const unsigned char* kst = stage0 + (size_t)s * stage_bytes;
          if constexpr (DUAL) {
            for (int kk = (warp - 6) * 32 + lane; kk < x.nv; kk += 64) {
              float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll 2
              for (int c = 0; c < H * 8; ++c) {
                const uint4 raw = *reinterpret_cast<const uint4*>(kst + (c >> 3) * half_bytes + kk * 128 + (((c & 7) ^ (kk & 7)) << 4));
                const float4 qa = *reinterpret_cast<const float4*>(qbar_s + c * 8), qc = *reinterpret_cast<const float4*>(qbar_s + c * 8 + 4);
                a0 = fmaf(qa.x, __uint_as_float(raw.x << 16), a0);
                a1 = fmaf(qa.y, __uint_as_float(raw.x & 0xffff0000u), a1);
                a2 = fmaf(qa.z, __uint_as_float(raw.y << 16), a2);
                a3 = fmaf(qa.w, __uint_as_float(raw.y & 0xffff0000u), a3);
                a0 = fmaf(qc.x, __uint_as_float(raw.z << 16), a0);
                a1 = fmaf(qc.y, __uint_as_float(raw.z & 0xffff0000u), a1);
                a2 = fmaf(qc.z, __uint_as_float(raw.w << 16), a2);
                a3 = fmaf(qc.w, __uint_as_float(raw.w & 0xffff0000u), a3);
              }
              p.raw_scores[(int64_t)(bi * p.Hkv + g) * p.n1_max + x.row0 + kk] = ((a0 + a1) + (a2 + a3)) * p.scale;
            }
          } else {
            for (int kk = (warp - 6) * 32 + lane; kk < x.nv; kk += 64) {
              float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
              for (int c = 0; c < H * 8; ++c) {
                const uint4 raw = *reinterpret_cast<const uint4*>(kst + (c >> 3) * half_bytes + kk * 128 + (((c & 7) ^ (kk & 7)) << 4));
                a0 = fmaf(qb[c * 8 + 0], __uint_as_float(raw.x << 16), a0);
                a1 = fmaf(qb[c * 8 + 1], __uint_as_float(raw.x & 0xffff0000u), a1);
                a2 = fmaf(qb[c * 8 + 2], __uint_as_float(raw.y << 16), a2);
                a3 = fmaf(qb[c * 8 + 3], __uint_as_float(raw.y & 0xffff0000u), a3);
                a0 = fmaf(qb[c * 8 + 4], __uint_as_float(raw.z << 16), a0);
                a1 = fmaf(qb[c * 8 + 5], __uint_as_float(raw.z & 0xffff0000u), a1);
                a2 = fmaf(qb[c * 8 + 6], __uint_as_float(raw.w << 16), a2);
                a3 = fmaf(qb[c * 8 + 7], __uint_as_float(raw.w & 0xffff0000u), a3);
              }
              p.raw_scores[(int64_t)(bi * p.Hkv + g) * p.n1_max + x.row0 + kk] = ((a0 + a1) + (a2 + a3)) * p.scale;
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(BAR(EMPTY_K + s));
        ++it;
      }
      // the softmax warps reuse the ring as scratch once they are done: tell them the K tiles are no longer read
      if (do_attn) asm volatile("bar.sync 3, 192;\n" ::: "memory");
    }
  }

  // ======================================= epilogue =======================================
  // The ring is idle now (every load was consumed), so it serves as scratch for the way out of TMEM:
  //   o_s [128][D] fp32, the float4 index XOR-swizzled by the row; ml_s [128]; lm_s [rows_rep].
  // Each accumulator row is weighted for the merge of the R replicas while it moves from TMEM to shared memory;
  // then consecutive threads store consecutive float4 of a row, so every global store is coalesced.
  const int64_t unit = (int64_t)(bi * p.Hkv + g) * up.row_tiles + rt;      // (sequence, KV head, row tile)
  if (do_attn && warp >= 2 && warp < 6) {
    constexpr int D4 = D / 4;
    const int q4 = warp & 3;
    const int row = q4 * 32 + lane;
    const int rep = row / rows_rep, m_local = row - rep * rows_rep;
    float* o_s = reinterpret_cast<float*>(stage0);
    float2* ml_s = reinterpret_cast<float2*>(DUAL ? smem + 1024 : stage0 + 128 * D * 4);   // DUAL: the ring is all o_s
    float2* lm_s = ml_s + 128;
    if (do_scores) asm volatile("bar.sync 3, 192;\n" ::: "memory");      // the saliency warps have left the ring
    ml_s[row] = make_float2(m_run, l_run);
    asm volatile("bar.sync 2, 128;\n" ::: "memory");
    float mstar = -INFINITY;
    for (int r2 = 0; r2 < R; ++r2) {
      const float2 x = ml_s[r2 * rows_rep + m_local];
      if (x.y > 0.f) mstar = fmaxf(mstar, x.x);
    }
    float lsum = 0.f;
    for (int r2 = 0; r2 < R; ++r2) {
      const float2 x = ml_s[r2 * rows_rep + m_local];
      if (x.y > 0.f) lsum = fmaf(x.y, fast_exp2(x.x - mstar), lsum);
    }
    const float w = l_run > 0.f ? fast_exp2(m_run - mstar) : 0.f;       // this replica's weight in the merged row
    if (rep == 0) lm_s[m_local] = make_float2(mstar, lsum);
    // the finished accumulator row: TMEM -> weight -> shared memory, 32 columns at a time
    const bool have_o = sm_ok && sm_tiles > 0 &&
                        wait_bar_warp(BAR(PV_DONE + ((sm_tiles - 1) & 1)), ((sm_tiles - 1) >> 1) & 1, abort_flag, p.status, 6, p.wait_cycles);
    tc_fence_after();
#pragma unroll 1
    for (int c = 0; c < D / 32; ++c) {
      uint32_t ov[32];
      if (have_o) {
        tmem_ld32(tmem_base + ((uint32_t)(q4 * 32) << 16) + O_COL + c * 32, ov);
        tc_wait_ld();
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) ov[i] = 0u;
      }
#pragma unroll
      for (int j = 0; j < 8; ++j)
        *reinterpret_cast<float4*>(o_s + row * D + (((c * 8 + j) ^ (row & (D4 - 1))) << 2)) =
            make_float4(__uint_as_float(ov[4 * j]) * w, __uint_as_float(ov[4 * j + 1]) * w, __uint_as_float(ov[4 * j + 2]) * w,
                        __uint_as_float(ov[4 * j + 3]) * w);
    }
  }
  if (do_attn) {
    // all eight warps share the stores: consecutive threads take consecutive float4 of a row; a thread keeps its column
    // and walks down the rows, four rows per step with all their shared-memory reads in flight together
    constexpr int D4 = D / 4;
    const float* o_s = reinterpret_cast<const float*>(stage0);
    const float2* lm_s = reinterpret_cast<const float2*>(DUAL ? smem + 1024 : stage0 + 128 * D * 4) + 128;
    __syncthreads();
    const int st = tid;
    if (!*abort_flag) {
      const int d4 = st % D4, r_first = st / D4, r_step = UM_THREADS / D4;
      const int m_first = rt * 128;
      for (int mb = r_first; mb < M_rt; mb += 4 * r_step) {
        float4 acc[4];
        float2 x[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int ml = min(mb + u * r_step, M_rt - 1);
          acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
          x[u] = lm_s[ml];
          for (int r2 = 0; r2 < R; ++r2) {
            const int rr = r2 * rows_rep + ml;
            const float4 o = *reinterpret_cast<const float4*>(o_s + rr * D + ((d4 ^ (rr & (D4 - 1))) << 2));
            acc[u].x += o.x; acc[u].y += o.y; acc[u].z += o.z; acc[u].w += o.w;
          }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int ml = mb + u * r_step;
          if (ml >= M_rt) break;
          const int m = m_first + ml;                  // row within the KV head: m = head_in_group * b + i
          const int hg = m / p.b, i = m - hg * p.b;
          if (p.splits == 1) {
            const float inv = x[u].y > 0.f ? 1.f / x[u].y : 0.f;
            __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(p.out) + (int64_t)bi * p.o_stride[0] +
                               (int64_t)(g * p.G + hg) * p.o_stride[1] + (int64_t)i * p.o_stride[2] + d4 * 4;
            uint2 w2;
            w2.x = pack_bf16(acc[u].x * inv, acc[u].y * inv);
            w2.y = pack_bf16(acc[u].z * inv, acc[u].w * inv);
            *reinterpret_cast<uint2*>(o) = w2;
            if (d4 == 0 && p.lse) p.lse[((int64_t)bi * p.Hq + g * p.G + hg) * p.b + i] = (x[u].x + log2f(x[u].y)) * kLn2;
          } else if (up.cluster > 1) {
            // this split's partial stays on chip: pm_s [M_rt][D] next to lm_s, read by the cluster peers below
            *reinterpret_cast<float4*>(reinterpret_cast<float*>(stage0 + 128 * D * 4 + 2048) + ml * D + d4 * 4) = acc[u];
          } else {
            const int64_t prow = (unit * p.splits + split) * min(p.M, 128) + ml;
            *reinterpret_cast<float4*>(p.part_o + prow * D + d4 * 4) = acc[u];
            if (d4 == 0) reinterpret_cast<float2*>(p.part_ml)[prow] = x[u];
          }
        }
      }
    }
  }

  // ---- fused tail: the last CTA of the unit merges the key splits and pools the saliency; nobody waits ----
  const bool tail_merge = do_attn && p.splits > 1;
  const bool tail_pool = (do_scores || prob_pass) && p.pooled != nullptr;
  // who counts: the key splits of a unit; in the probability pass all row tiles of the head as well (its pooling
  // needs every row tile's column sums), on the counter of the head's first unit
  const int expected = prob_pass ? p.splits * up.row_tiles : p.splits;
  int32_t* counter = p.counters + (prob_pass ? unit - rt : unit);
  if (up.cluster > 1) {
    // ---- cluster tail: the key splits of the unit are the CTAs of one cluster. After a cluster barrier every split's
    //      partial (in its shared memory) and raw saliency (in global memory) is visible to all of them; each CTA then
    //      merges a share of the rows straight out of its peers' shared memory and pools a share of the positions.
    //      No partial touches global memory, no counter, no CTA is left to do the whole tail alone. ----
    constexpr int D4 = D / 4;
    const int S = up.cluster;
    __threadfence();
    __syncthreads();                     // also brings the lanes of the producer and MMA warps back together
    cluster_sync_all();
    if (tail_merge && !*abort_flag) {
      const uint32_t lm_a = smem_u32(stage0 + 128 * D * 4) + 128 * 8;      // lm_s
      const uint32_t pm_a = smem_u32(stage0 + 128 * D * 4 + 2048);         // pm_s
      const int r_lo = (int)(((long long)split * M_rt) / S), r_hi = (int)(((long long)(split + 1) * M_rt) / S);
      for (int slot = tid; slot < (r_hi - r_lo) * D4; slot += UM_THREADS) {
        const int ml = r_lo + slot / D4, d4 = slot % D4;
        float2 x[8];
        float4 o[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const uint32_t peer = (uint32_t)min(c, S - 1);
          x[c] = ld_cluster_f2(map_to_cta(lm_a + ml * 8, peer));
          o[c] = ld_cluster_f4(map_to_cta(pm_a + (uint32_t)(ml * D + d4 * 4) * 4u, peer));
        }
        float mstar = -INFINITY;
#pragma unroll
        for (int c = 0; c < 8; ++c)
          if (c < S && x[c].y > 0.f) mstar = fmaxf(mstar, x[c].x);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float l = 0.f;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          if (c >= S || !(x[c].y > 0.f)) continue;
          const float w = fast_exp2(x[c].x - mstar);
          l = fmaf(x[c].y, w, l);
          acc.x = fmaf(o[c].x, w, acc.x); acc.y = fmaf(o[c].y, w, acc.y); acc.z = fmaf(o[c].z, w, acc.z); acc.w = fmaf(o[c].w, w, acc.w);
        }
        const float inv = l > 0.f ? 1.f / l : 0.f;
        const int m = rt * 128 + ml;
        const int hg = m / p.b, i = m - hg * p.b;
        __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(p.out) + (int64_t)bi * p.o_stride[0] +
                             (int64_t)(g * p.G + hg) * p.o_stride[1] + (int64_t)i * p.o_stride[2] + d4 * 4;
        uint2 w2;
        w2.x = pack_bf16(acc.x * inv, acc.y * inv);
        w2.y = pack_bf16(acc.z * inv, acc.w * inv);
        *reinterpret_cast<uint2*>(out) = w2;
        if (d4 == 0 && p.lse) p.lse[((int64_t)bi * p.Hq + g * p.G + hg) * p.b + i] = (mstar + log2f(l)) * kLn2;
      }
    }
    if (tail_pool && !*abort_flag) {
      const float* a = p.raw_scores + (int64_t)(bi * p.Hkv + g) * p.n1_max;
      const int p_lo = (int)(((long long)split * p.n1_max) / S), p_hi = (int)(((long long)(split + 1) * p.n1_max) / S);
      for (int pos = p_lo + tid; pos < p_hi; pos += UM_THREADS)
        p.pooled[(int64_t)(bi * p.Hkv + g) * p.n1_max + pos] = pool_at_ldcg(p, a, n1, p.block_off[bi], pos);
    }
    cluster_sync_all();                  // nobody leaves while a peer may still read its shared memory
  } else if (up.fused_tail && (tail_merge || tail_pool)) {
    __threadfence();
    __syncthreads();
    bool last = true;
    if (expected > 1) {
      if (tid == 0) {
        const int old = atomicAdd(counter, 1);
        *last_flag = (old == expected - 1) ? 1 : 0;
      }
      __syncthreads();
      last = *last_flag != 0;
    }
    if (last && !*abort_flag) {
      __threadfence();
      if (tail_merge)
        for (int s0 = tid; s0 < M_rt * (D / 4); s0 += 4 * UM_THREADS) {
          int four[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) four[u] = s0 + u * UM_THREADS < M_rt * (D / 4) ? s0 + u * UM_THREADS : -1;
          merge_slots<D, 4, 4>(p, unit, bi, g, rt, four);
        }
      if (tail_pool) {
        // stage the head's raw saliency in shared memory (the ring is free), then pool from there
        float* a_s = reinterpret_cast<float*>(stage0);
        const float* a = p.raw_scores + (int64_t)(bi * p.Hkv + g) * p.n1_max;
        const int n_arr = prob_pass ? up.row_tiles : 1;          // the probability pass left one array per row tile
        for (int i = tid; i < n1; i += UM_THREADS) {
          float x = 0.f;
          for (int r2 = 0; r2 < n_arr; ++r2) x += __ldcg(a + (int64_t)r2 * p.B * p.Hkv * p.n1_max + i);
          a_s[i] = x;
        }
        __syncthreads();
        for (int pos = tid; pos < p.n1_max; pos += UM_THREADS)
          p.pooled[(int64_t)(bi * p.Hkv + g) * p.n1_max + pos] = pool_at(p, a_s, n1, p.block_off[bi], pos);
      }
    }
    // ready for the next call, whether or not this one gave up: a counter left at its final value would keep every
    // later call on this workspace from ever finding its last CTA
    if (last && expected > 1 && tid == 0) *counter = 0;
  }

  // ---- free the tensor memory ----
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// ---------------------------------------------------------------------------------------------------------
// Host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess)
      f = nullptr;
    return reinterpret_cast<EncodeTiledFn>(f);
  }();
  return fn;
}

// 4-D bf16 tensor (D, rows, heads, batch) with element strides for the three outer axes; box = (64, box_rows, box_heads, 1),
// 128-byte swizzle, out-of-range rows read as zero.
bool make_map(CUtensorMap* m, const void* base, int D, int rows, int heads, int batch, const int64_t* stride_bhr, int box_rows,
              int box_heads) {
  EncodeTiledFn enc = encode_fn();
  if (!enc || rows < 1) return false;
  const cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)rows, (cuuint64_t)heads, (cuuint64_t)batch};
  auto st = [&](int64_t s) { return (cuuint64_t)(s > 0 ? s * 2 : (int64_t)D * 2); };   // unused strides stay legal
  const cuuint64_t strides[3] = {st(stride_bhr[2]), st(stride_bhr[1]), st(stride_bhr[0])};
  const cuuint32_t box[4] = {64u, (cuuint32_t)box_rows, (cuuint32_t)box_heads, 1u};
  const cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

size_t umma_smem_bytes(int D, int KT, bool dual) {
  const size_t H = D / 64;
  if (dual) return 1024 /*alignment slack*/ + 4096 /*control block*/ + H * 128 * 128 + (size_t)2 * 2 * H * 64 * 128;
  const size_t need = 1024 /*alignment slack*/ + 1024 /*barriers, qbar*/ + H * 128 * 128 + (size_t)UM_STAGES * 2 * H * KT * 128;
  // every CTA allocates all 512 TMEM columns, so two CTAs must never share an SM: ask for more than half its shared memory
  return need > 120 * 1024 ? need : 120 * 1024;
}

template <int D, bool PROB, bool DUAL>
cudaError_t launch_umma_d(const UmmaMaps& tm, const UmmaParams& up, const AttnPlan& pl, bool pdl, cudaStream_t st) {
  auto kern = attn_umma_bf16_kernel<D, PROB, DUAL>;
  static SmemConfig configured;
  cudaError_t e = configure_smem(reinterpret_cast<const void*>(kern), pl.smem_bytes, configured, true);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(pl.splits, up.a.Hkv * up.row_tiles, up.a.B);
  cfg.blockDim = dim3(UM_THREADS);
  cfg.dynamicSmemBytes = pl.smem_bytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  int na = 0;
  if (pdl) {
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  if (up.cluster > 1) {                      // the key splits (grid x) of a unit form one cluster
    attr[na].id = cudaLaunchAttributeClusterDimension;
    attr[na].val.clusterDim.x = up.cluster; attr[na].val.clusterDim.y = 1; attr[na].val.clusterDim.z = 1;
    ++na;
  }
  cfg.attrs = attr; cfg.numAttrs = na;
  return cudaLaunchKernelEx(&cfg, kern, tm, up);
}

}  // namespace

bool umma_make_map(CUtensorMap* m, const void* base, int D, int rows, int heads, int batch, const int64_t* stride_bhr, int box_rows,
                   int box_heads) {
  return make_map(m, base, D, rows, heads, batch, stride_bhr, box_rows, box_heads);
}

// Whether the tcgen05 kernel covers a shape: bf16, D in {64, 128}, block length a multiple of 16 that either keeps all
// b*G rows inside one 128-row tile or divides 128.
bool umma_supported(int dtype, int D, int M, int b) {
  if (dtype != SDLLM_BF16 || (D != 64 && D != 128) || encode_fn() == nullptr) return false;
  if (b % 16 != 0 || b > 128) return false;
  return M <= 128 || 128 % b == 0;
}

// The last CTA of a unit does the tail itself while that is a small job; otherwise a second launch spreads it over
// the whole GPU.
bool umma_tail_is_fused(const AttnPlan& pl, int D, int M, int n1_max, bool pool, bool merge) {
  const size_t merge_bytes = merge && pl.splits > 1 ? (size_t)pl.splits * (M < 128 ? M : 128) * D * 4 : 0;
  // (a merge of full 128-row partials by the last CTA alone lost to the second launch at every split count measured,
  // 16.2 against 22.6 us with four splits: the last CTA does it only for small partials)
  bool fused = merge_bytes <= 32 * 1024 && (!pool || n1_max <= 8192);
  const int forced = tuning().fused_tail;
  if (forced >= 0) fused = forced == 1 && (!pool || n1_max <= 8192);
  return fused;
}

AttnPlan plan_attention_umma(int D, int M, int b, int B, int Hkv, int n1_max, int n2, const Tuning& tn) {
  AttnPlan pl{};
  pl.kind = 2; pl.tma = true; pl.cluster = 1; pl.fused_tail = true;
  pl.threads = UM_THREADS; pl.stages = UM_STAGES;
  const int sms = sm_count();
  const int G = M / b;
  pl.row_tiles = M <= 128 ? 1 : (G + 128 / b - 1) / (128 / b);
  pl.rep = M <= 32 ? 4 : (M <= 64 ? 2 : 1);
  const long long units = (long long)B * Hkv * pl.row_tiles;
  // Several waves of CTAs: the small-footprint variant puts two of them on an SM, so that one's set-up and way out
  // overlap the other's streaming. It works on 64-key tiles, which leaves room for two replicas of the rows at most.
  pl.dual = units >= 2 * sms && n2 > 0;              // measured: pays for the reuse step, not for the refresh step
  if (tn.dual >= 0) pl.dual = tn.dual == 1;
  if (pl.dual && pl.rep > 2) pl.rep = 2;
  long long want = sms / units;
  if (want < 1) want = 1;
  // 8 units: sixteen splits (128 CTAs) measured 5 % ahead of eighteen (144) at every length tried, refresh and reuse
  if (want > 16 && want < 24) want = 16;
  if (tn.splits > 0) want = tn.splits;
  // Reuse step with replicated rows (few query rows per head, so a tile costs a softmax warp little): a CTA works
  // best on about four 128-key tiles. With fewer, the set-up of the CTAs and the merge of their partials weigh more
  // than the streaming they save.
  if (n2 > 0 && pl.rep > 1 && !pl.dual && tn.splits <= 0) {
    const long long cap = ((n1_max + 127) / 128 + 1 + 3) / 4;
    if (want > cap) want = cap;
  }
  // Full 128-row tiles (nothing replicated), from the same sweep as the cluster note below: with at most 24 tiles per
  // head eight splits beat sixteen (11.4 against 13.7 us at 1024 keys, 13.1 against 14.2 at 2048); with 32 units or more
  // and at most five tiles per head no split at all beats four (13.1 against 20.8 us at 256 keys, 32 units).
  // Nine splits (16 units) lost 6 % to eight wherever measured.
  if (pl.rep == 1 && !pl.dual && tn.splits <= 0) {
    const int t128 = (n1_max + 127) / 128 + (n2 > 0 ? 1 : 0);
    if (want > 8 && (t128 <= 24 || want < 16)) want = 8;
    if (n2 > 0 && units >= 32 && t128 <= 5) want = 1;
  }
  const int kt2 = n2 > 0 ? (n2 < 128 ? n2 : 128) : 0;
  pl.key_tile = 128;
  if (pl.rep <= 2 && (n1_max + 127) / 128 + (n2 > 0 ? 1 : 0) < want) pl.key_tile = 64;
  if (tn.key_tile == 64 && pl.rep <= 2) pl.key_tile = 64;
  if (tn.key_tile == 128) pl.key_tile = 128;
  if (pl.dual) { pl.key_tile = 64; pl.stages = 2; }
  // A reuse step with few heads and a short cache: rather than many one-tile splits whose merge needs a second launch,
  // take at most eight splits of 128-key tiles, which one cluster merges on chip.
  const int tiles128 = (n1_max + 127) / 128 + (n2 > 0 ? 1 : 0);
  // The cluster tail of this kernel (every split pulls its share of the rows out of its peers' shared memory between two
  // cluster barriers) measured slower than partials in the workspace at every shape of a sweep over 1 to 8 sequences x
  // 256 to 4096 cached keys of 4 KV heads x 7 query heads (10 to 80 %: 11.5 against 12.6 us at 1024 keys, 13.1 against
  // 23.7 us with two sequences), so it is taken only on request (Tuning::cluster = 2); the key-row kernel's push-style
  // merge is the cluster path that pays.
  const bool no_cluster = tn.cluster != 2 || tn.fused_tail == 0;
  if (!pl.dual && !no_cluster && tn.splits <= 0 && tn.key_tile == 0 && n2 > 0 && want > 8 && tiles128 <= 16) {
    pl.key_tile = 128;
    want = tiles128 < 8 ? tiles128 : 8;
  }
  pl.key_tile2 = kt2 > 0 ? (kt2 < pl.key_tile ? kt2 : pl.key_tile) : pl.key_tile;
  const int tiles = (n1_max + pl.key_tile - 1) / pl.key_tile + (n2 > 0 ? (n2 + pl.key_tile2 - 1) / pl.key_tile2 : 0);
  if (want > tiles) want = tiles;
  if (want > kMaxSplits) want = kMaxSplits;
  if (want < 1) want = 1;
  pl.splits = (int)want;
  pl.parts = pl.splits;                 // replicas are merged inside the CTA
  pl.rows_rep = 128 / pl.rep;
  pl.part_rows = pl.splits > 1 ? (size_t)pl.row_tiles * pl.splits * (M < 128 ? M : 128) : 0;
  pl.n_counters = (size_t)B * Hkv * pl.row_tiles;
  pl.smem_bytes = umma_smem_bytes(D, pl.key_tile, pl.dual);
  // Few key splits of a small problem: make them one thread-block cluster, so that they merge through distributed shared
  // memory instead of the workspace. Only where the whole grid is one wave (a cluster needs all its SMs at once).
  // Several row tiles only at the reuse step: the probability pass of the refresh step pools over all row tiles of a
  // head, which one cluster does not span.
  if (!no_cluster && pl.splits >= 2 && pl.splits <= 8 && (pl.row_tiles == 1 || n2 > 0) && pl.key_tile == 128 &&
      units * pl.splits <= sms && n1_max <= 8192)
    pl.cluster = pl.splits;
  return pl;
}

cudaError_t launch_attn_umma(const AttnParams& p, const AttnPlan& pl, int D, cudaStream_t st) {
  const Tuning tn = tuning();
  UmmaMaps tm;
  UmmaParams up{};
  up.a = p;
  up.a.splits = pl.splits;
  up.a.wait_cycles = tn.wait_cycles;
  up.KT = pl.key_tile; up.KT2 = pl.key_tile2; up.R = pl.rep; up.row_tiles = pl.row_tiles;
  up.heads_rt = pl.row_tiles == 1 ? p.G : 128 / p.b;
  const bool pool = p.want_scores && p.pooled != nullptr;
  up.early_src1 = (p.n2 > 0 && p.n1_max > 0 && tn.early_loads != 0) ? 1 : 0;
  up.prob_pass = p.prob_pass;
  up.cluster = pl.cluster;
  {
    const long long ctas = (long long)pl.splits * p.Hkv * pl.row_tiles * p.B;
    up.lpt = (p.n1_per_seq != nullptr && p.B >= 4 && p.B <= 64 && ctas > sm_count()) ? 1 : 0;
    if (tn.lpt >= 0) up.lpt = (tn.lpt == 1 && p.n1_per_seq != nullptr && p.B >= 2 && p.B <= 64) ? 1 : 0;
  }
  up.fused_tail = (pl.cluster > 1 || umma_tail_is_fused(pl, D, p.M, p.n1_max, pool || p.prob_pass, p.out != nullptr && !p.prob_pass)) ? 1 : 0;
  memset(&tm, 0, sizeof(tm));
  bool ok = true;
  if (p.out != nullptr || p.prob_pass) ok = make_map(&tm.q, p.q, D, p.b, p.Hq, p.B, p.q_stride, p.b, up.heads_rt);
  if (p.n1_max > 0) {
    ok = ok && make_map(&tm.k1, p.k1, D, p.n1_max, p.Hkv, p.B, p.k1_stride, pl.key_tile, 1);
    ok = ok && make_map(&tm.v1, p.v1, D, p.n1_max, p.Hkv, p.B, p.k1_stride, pl.key_tile, 1);
  }
  if (p.n2 > 0) {
    ok = ok && make_map(&tm.k2, p.k2, D, p.n2, p.Hkv, p.B, p.k2_stride, pl.key_tile2, 1);
    ok = ok && make_map(&tm.v2, p.v2, D, p.n2, p.Hkv, p.B, p.k2_stride, pl.key_tile2, 1);
    if (p.n1_max <= 0) { tm.k1 = tm.k2; tm.v1 = tm.v2; }
  } else {
    tm.k2 = tm.k1; tm.v2 = tm.v1;
  }
  if (!ok) return cudaErrorInvalidValue;
  cudaError_t err;
  const bool pdl = tn.pdl != 0;
  if (pl.dual) {
    if (up.prob_pass) err = D == 128 ? launch_umma_d<128, true, true>(tm, up, pl, pdl, st) : launch_umma_d<64, true, true>(tm, up, pl, pdl, st);
    else err = D == 128 ? launch_umma_d<128, false, true>(tm, up, pl, pdl, st) : launch_umma_d<64, false, true>(tm, up, pl, pdl, st);
  } else {
    if (up.prob_pass) err = D == 128 ? launch_umma_d<128, true, false>(tm, up, pl, pdl, st) : launch_umma_d<64, true, false>(tm, up, pl, pdl, st);
    else err = D == 128 ? launch_umma_d<128, false, false>(tm, up, pl, pdl, st) : launch_umma_d<64, false, false>(tm, up, pl, pdl, st);
  }
  if (err != cudaSuccess || up.fused_tail) return err;
  const bool merge = p.out != nullptr && !p.prob_pass && pl.splits > 1;
  const bool pool_tail = pool || (p.prob_pass && p.pooled != nullptr);
  if (!merge && !pool_tail) return cudaSuccess;
  const long long merge_threads = merge ? (long long)p.B * p.Hkv * pl.row_tiles * 128 * (D / 4) : 0;
  const long long pool_threads = pool_tail ? (long long)p.B * p.Hkv * p.n1_max : 0;
  const int merge_blocks = (int)((merge_threads + 255) / 256);
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)(merge_blocks + (pool_threads + 255) / 256));
  cfg.blockDim = dim3(256);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  int na = 0;
  if (pdl) {
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  cfg.attrs = attr; cfg.numAttrs = na;
  return D == 128 ? cudaLaunchKernelEx(&cfg, umma_tail_kernel<128>, up, merge_blocks)
                  : cudaLaunchKernelEx(&cfg, umma_tail_kernel<64>, up, merge_blocks);
}

// ---------------------------------------------------------------------------------------------------------
// Dispatch between the kernel families
AttnPlan plan_attention_legacy(int dtype, int D, int M, int B, int Hkv, int n_keys_max, const Tuning& tn);
cudaError_t launch_attn_legacy(const AttnParams& p, const AttnPlan& plan, int dtype, int D, cudaStream_t st);
bool kt_supported(int dtype, int D, int M, int b);
bool kt_preferred(int M, int B, int Hkv, int n1_max, int n2);
AttnPlan plan_attention_kt(int D, int M, int b, int B, int Hkv, int n1_max, int n2, const Tuning& tn);
cudaError_t launch_attn_kt(const AttnParams& p, const AttnPlan& pl, int D, cudaStream_t st);

AttnPlan plan_attention(int dtype, int D, int M, int b, int B, int Hkv, int n1_max, int n2, bool prob_scores) {
  // bf16 goes to the tcgen05 kernels wherever they apply: heads with at most 128 query rows to the kernel that puts the
  // keys on the accumulator rows (it has no softmax-probability saliency pass) unless its cluster limit would leave most
  // SMs idle, the rest to the one that puts the queries there; fp32 and the remaining bf16 shapes go to the cp.async
  // kernels. Tuning::kernel forces a family.
  const Tuning tn = tuning();
  const bool kt_ok = kt_supported(dtype, D, M, b) && !prob_scores;
  if (kt_ok && (tn.kernel == 3 || (tn.kernel == 0 && kt_preferred(M, B, Hkv, n1_max, n2))))
    return plan_attention_kt(D, M, b, B, Hkv, n1_max, n2, tn);
  if (tn.kernel != 1 && umma_supported(dtype, D, M, b)) return plan_attention_umma(D, M, b, B, Hkv, n1_max, n2, tn);
  AttnPlan pl = plan_attention_legacy(dtype, D, M, B, Hkv, n1_max + n2, tn);
  pl.tma = false; pl.cluster = 1; pl.warp_keys = 32; pl.kind = 0;
  pl.part_rows = pl.splits > 1 ? (size_t)pl.splits * M : 0;      // partial rows the kernels leave per (sequence, KV head)
  pl.n_counters = 0; pl.fused_tail = false;
  pl.rep = 1; pl.row_tiles = 1; pl.parts = pl.splits; pl.rows_rep = M; pl.key_tile2 = pl.key_tile;
  return pl;
}

cudaError_t launch_attn_partial(const AttnParams& p, const AttnPlan& plan, int dtype, int D, cudaStream_t st) {
  if (plan.kind == 3) return launch_attn_kt(p, plan, D, st);
  if (plan.kind == 2) return launch_attn_umma(p, plan, D, st);
  return launch_attn_legacy(p, plan, dtype, D, st);
}

}  // namespace sdllm
