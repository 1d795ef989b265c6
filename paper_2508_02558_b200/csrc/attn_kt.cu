// bf16 block-query attention with the KEYS on the accumulator rows (tcgen05, sm_100a), for heads with few query rows.
//
// When a KV head has N = b*G <= 64 query rows (multi-head attention with a block of 32: N = 32), putting the queries on
// the 128 accumulator rows wastes three quarters of every MMA and forces the rows to be replicated and merged again.
// Here the score tile is transposed instead:
//     S^T [128 keys x N queries] = K_tile [128 x D] . Q^T            (A = K tile, B = Q, both K-major in shared memory)
//     O^T [D x N queries]       += V_tile^T [D x keys] . P^T [keys x N]   (A = V tile read MN-major, B = P^T MN-major)
// so one thread of the four softmax warps owns one KEY of the tile (a TMEM lane) and sees that key's logits against all
// N queries. What this buys:
//   * nothing is replicated and nothing is merged inside the CTA; both MMAs are N/128 of the row-major ones;
//   * the mean-query saliency of Algorithm 1 ("qbar <- Mean(Q_b)", "A <- MatMul(qbar, K_f^T)") is, by linearity, the
//     mean of the key's N logits: the thread that owns the key already holds them, no separate pass over K;
//   * the finished O^T has one head dimension per thread and N columns: key splits are merged column by column.
// The softmax needs one reference value per query (column) that all keys share. It is taken once, from the column
// maxima of the CTA's first tile (warp reductions and a shared-memory max), and afterwards only checked: a tile
// whose logits exceed a reference by more than 2^8 makes the softmax threads raise the references and rescale O^T and
// the partial sums (rare). P is bf16, whose exponent range is that of fp32, so a reference within 2^8 of the true
// maximum loses nothing.
//
// The key axis is  [source 1 rows 0..n1) ++ [source 2 rows 0..n2)  cut into groups of 32 rows; a CTA takes a contiguous
// range of groups and walks it in tiles of up to four groups (128 keys), so a tile may mix the two sources.
//   refresh step : source 1 = the full K/V of the sequence, no source 2;
//   reuse step   : source 1 = the compacted cache, source 2 = the block's fresh rows (Algorithm 3, Concat(K_c, K_n)).
// The S key splits of a (sequence, KV head) are the CTAs of one thread-block cluster. Each split pushes, for every
// query column, its un-normalised O^T column and its (reference, sum) pair into the shared memory of the CTA that owns
// the column (st.shared::cluster); after ONE cluster barrier every CTA merges and stores the columns it owns and, at
// the refresh step, pools its share of the head's saliency (Algorithm 1, MaxPool1D). Nothing goes through global
// memory, there is no counter and no second launch.
// Warp roles (192 threads): warp 0 TMA producer, warp 1 MMA issuer and TMEM owner, warps 2-5 softmax.
// With N <= 32 a CTA needs about 110 KB of shared memory and 128 TMEM columns, so two CTAs share an SM and, with
// programmatic dependent launch, the next call's CTAs load their first tiles while this call's CTAs finish.
//
// Every wait on an mbarrier is bounded. On expiry the thread sets an abort flag that all other waits poll, records a
// code in the status word and the CTA runs to its end, still taking part in the cluster barriers (no peer is left
// waiting) and freeing its TMEM; the outputs of that call are then invalid.
#include <cuda.h>
#include <string.h>

#include <mutex>

#include "attn_device.cuh"
#include "kt_params.cuh"
#include "tuning.cuh"
#include "umma_host.cuh"

namespace sdllm {
using namespace dev;
namespace {

constexpr int KT_MAX_STAGES = 3;

#include "kt_common.cuh"

// WG = 2: two softmax warpgroups take the tiles in turn, each with its own accumulator and references (32 query columns).
// CG > 1: CG softmax warpgroups share every tile, each owning 32 of the 32 * CG query columns (one accumulator).
template <int D, int WG, int CG>
__global__ void __launch_bounds__(64 + 128 * WG * CG, (WG == 1 && CG == 1) ? 2 : 1) attn_kt_kernel(const __grid_constant__ KtMaps tm, const KtParams kp) {
  static_assert(WG == 1 || CG == 1, "tile-alternating warpgroups only with one column group");
  constexpr int NG = WG * CG;                // softmax warpgroups
  constexpr int NTHREADS = 64 + 128 * NG;
  constexpr int H = D / 64;                  // 128-byte column halves of a K/V row
  constexpr int NP = 32;                     // query columns of one softmax thread
  constexpr int NPT = 32 * CG;               // query columns of the tile (padded)
  constexpr int PHALVES = (CG + 1) / 2;      // 64-column halves of a P^T row (CG > 1: 128-byte rows, 128-byte swizzle)
  constexpr int PBUF = CG == 1 ? 128 * 64 : PHALVES * 128 * 128;   // one P^T buffer: 128 key rows (CG = 1: 64-byte rows, 64-byte swizzle)
  constexpr uint32_t O_COL = 2 * NPT;        // TMEM columns: two S^T buffers of NPT, then one O^T of NPT per tile-alternating warpgroup
  constexpr uint32_t TMEM_NEED = 2 * NPT + NPT * WG;
  constexpr int MS = 8;                      // largest cluster (key splits of one unit)
  constexpr uint32_t TMEM_COLS = TMEM_NEED <= 128 ? 128 : (TMEM_NEED <= 256 ? 256 : 512);
  constexpr int KT_CTRL = KT_CTRL0 + NG * KT_GRP;
  extern __shared__ unsigned char smem_raw[];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int NS = kp.NS, S = kp.S, N = kp.N;
  const AttnParams& p = kp.a;
  constexpr int GPT = 4;                     // groups of 32 keys per tile (compile-time: the address arithmetic of the hot loops hangs on it)
  constexpr int HALF = GPT * 32 * 128;       // bytes of one 64-column half of a tile
  constexpr int KV_BYTES = H * HALF;         // one K (or V) tile
  constexpr int SLOT = 2 * KV_BYTES;
  const int g = blockIdx.y, split = blockIdx.x;
  // Which sequence: grid z itself, or, for ragged batches that take several waves, the sequence of that rank when the
  // batch is ordered from the longest to the shortest - CTAs are handed out in grid order, so the long ones start first
  // and the short ones fill the tail. Every warp ranks the (at most 64) lengths on its own: no shared memory, no barrier.
  int bi = blockIdx.z;
  if (kp.lpt) {
    if (!kp.early_src1) grid_dependency_wait();        // the lengths may come from the kernel in front
    const int l0 = lane < p.B ? p.n1_per_seq[lane] : -1, l1 = lane + 32 < p.B ? p.n1_per_seq[lane + 32] : -1;
    int r0 = 0, r1 = 0;                                // how many sequences come before mine (longer, or equal and earlier)
    for (int i = 0; i < p.B; ++i) {
      const int li = __shfl_sync(0xffffffffu, i < 32 ? l0 : l1, i & 31);
      r0 += (li > l0 || (li == l0 && i < lane)) ? 1 : 0;
      r1 += (li > l1 || (li == l1 && i < lane + 32)) ? 1 : 0;
    }
    const unsigned hit0 = __ballot_sync(0xffffffffu, lane < p.B && r0 == (int)blockIdx.z);
    const unsigned hit1 = __ballot_sync(0xffffffffu, lane + 32 < p.B && r1 == (int)blockIdx.z);
    bi = hit0 ? __ffs(hit0) - 1 : (hit1 ? __ffs(hit1) + 31 : (int)blockIdx.z);
  }
  const int n2 = p.n2;
  const long long wlim = kp.wait_cycles;
  // The count of source 1 is read ahead of the grid dependency only at the reuse step (it is older than any kernel that
  // may still run); the load is issued first so that its latency hides behind the set-up.
  // The line is asked to stay in L2 (evict-last): every reuse step of the block reads it again, first thing, while the
  // K/V streams of a whole model pass through L2 in between.
  int n1_early = p.n1_max;
  if (kp.early_src1 && p.n1_per_seq) {
    uint64_t keep;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;\n" : "=l"(keep));
    asm volatile("ld.global.L2::cache_hint.s32 %0, [%1], %2;\n" : "=r"(n1_early) : "l"(p.n1_per_seq + bi), "l"(keep) : "memory");
  }

  // ---- shared memory carve-up (1024-byte aligned for the 128-byte swizzle; identical in every CTA of the cluster) ----
  const uint32_t raw_addr = smem_u32(smem_raw);
  unsigned char* smem = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
  const uint32_t bars = smem_u32(smem);
  auto BAR = [&](int i) { return bars + 8u * (uint32_t)i; };
  constexpr int Q_FULL = 0, FULL_K = 1, FULL_V = 1 + KT_MAX_STAGES, EMPTY_K = 1 + 2 * KT_MAX_STAGES, EMPTY_V = 1 + 3 * KT_MAX_STAGES;
  constexpr int S_FULL = 1 + 4 * KT_MAX_STAGES, P_FULL = S_FULL + 2, PV_DONE = S_FULL + 4, DRAIN = S_FULL + 6, MERGE = S_FULL + 7;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + 256);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + 260);
  // per softmax warpgroup: its index, and which tiles / columns it takes
  const int grp = (NG > 1 && warp >= 2) ? (warp - 2) >> 2 : 0;
  const int wg = WG == 2 ? grp : 0;        // tile parity it works on
  const int cg = CG > 1 ? grp : 0;         // column group it owns
  unsigned char* gblk = smem + KT_CTRL0 + grp * KT_GRP;
  float* m_ref = reinterpret_cast<float*>(gblk);                    // [32] references of the group's columns (log2 units)
  uint32_t* enc = reinterpret_cast<uint32_t*>(gblk + 256);          // [32] scratch of a raise: column maxima, order-preserving codes
  float* l_tot = reinterpret_cast<float*>(gblk + 512);              // [32] sums of this split
  float* delta_s = reinterpret_cast<float*>(gblk + 768);            // [32] by how much a raise lifts each reference
  float* l_w = reinterpret_cast<float*>(gblk + 1024);               // [4][32] per-warp sums
  float* sal_s = reinterpret_cast<float*>(gblk + 1536);             // [2][128] this group's share of the keys' logit sums (CG > 1)
  const int bar_id = 1 + grp;              // (a compile-time constant with one warpgroup)
  unsigned char* q_s = smem + KT_CTRL;                              // [H][NPT rows][128 B]
  unsigned char* p_s = q_s + H * NPT * 128;                         // [PB][P^T buffer]
  unsigned char* ring = p_s + kp.PB * PBUF;                         // [NS][K tile | V tile]
  // Cluster merge: what the S splits push into this CTA (it owns DL head dimensions of every column). With one column
  // group the area is its own; with several it would not fit beside the ring, so it lies over the ring and is written
  // only after a cluster barrier behind every CTA's last PV.
  float* recv = reinterpret_cast<float*>(CG == 1 ? ring + (size_t)NS * SLOT : ring);   // [S][NPT/4][DL] float4: un-normalised O^T, four columns of one owned head dimension
  float2* ml_recv = reinterpret_cast<float2*>(recv + (size_t)S * kp.DL * NPT);  // [S][NPT] (reference, sum) of every column
  float* w_s = reinterpret_cast<float*>(ml_recv + (size_t)S * NPT); // [S][NPT] merge weights, normalisation folded in

  // ---- this CTA's share of the key axis, in groups of 32 rows ----
  int n1 = 0, g1 = 0, gb = 0, ge = 0, T = 0;
  auto set_counts = [&](int n1_raw) {
    n1 = min(max(n1_raw, 0), p.n1_max);
    g1 = (n1 + 31) >> 5;
    const int gt = g1 + ((n2 + 31) >> 5);
    gb = (int)(((long long)split * gt) / S);
    ge = (int)(((long long)(split + 1) * gt) / S);
    T = (ge - gb + GPT - 1) / GPT;
  };
  auto read_counts = [&]() { set_counts(p.n1_per_seq ? p.n1_per_seq[bi] : p.n1_max); };

  // ---- the producer lane (thread 0) ----
  int t_next = 0, k_issued = 0, v_issued = 0;        // next tile to load; tiles whose K / V loads are on their way
  auto tile_groups = [&](int t, int& gi0) { gi0 = gb + GPT * t; return min(GPT, ge - gi0); };
  auto issue_tile = [&](int t) -> bool {
    const int s = t % NS;
    const uint32_t ph = ((t / NS) - 1) & 1;
    int gi0;
    const int ng = tile_groups(t, gi0);
    const bool whole = 4 * ng >= 3 * GPT && gi0 + ng <= g1;   // (nearly) full tile of source 1: one box per 64-column half
    uint32_t bytes = 0;
    if (whole) bytes = (uint32_t)KV_BYTES;
    else for (int j = 0; j < ng; ++j) bytes += (uint32_t)(H * 128 * (gi0 + j < g1 ? 32 : kp.gr2));
    const uint32_t kdst = smem_u32(ring + (size_t)s * SLOT), vdst = kdst + KV_BYTES;
    for (int kv = 0; kv < 2; ++kv) {
      const int full = kv == 0 ? FULL_K : FULL_V, empty = kv == 0 ? EMPTY_K : EMPTY_V;
      if (t >= NS && !wait_bar(BAR(empty + s), ph, abort_flag, p.status, 1 + kv, wlim)) return false;
      mbar_expect_tx(BAR(full + s), bytes);
      if (whole) {
        for (int h = 0; h < H; ++h)
          tma_load_4d((kv == 0 ? kdst : vdst) + (uint32_t)(h * HALF), kv == 0 ? &tm.k1t : &tm.v1t, BAR(full + s), h * 64, gi0 * 32, g, bi);
      } else {
        for (int j = 0; j < ng; ++j) {
          const Group x = group_of(gi0 + j, g1, n1, n2);
          const CUtensorMap* m = kv == 0 ? (x.src1 ? &tm.k1 : &tm.k2) : (x.src1 ? &tm.v1 : &tm.v2);
          for (int h = 0; h < H; ++h)
            tma_load_4d((kv == 0 ? kdst : vdst) + (uint32_t)(h * HALF + j * 4096), m, BAR(full + s), h * 64, x.row0, g, bi);
        }
      }
      if (kv == 0) k_issued = t + 1; else v_issued = t + 1;
    }
    return true;
  };

  if (tid == 0) {                        // the descriptors live in the kernel parameters: fetch them while the CTA sets up
    prefetch_tmap(&tm.k1t); prefetch_tmap(&tm.v1t); prefetch_tmap(&tm.k1); prefetch_tmap(&tm.v1);
    if (n2 > 0) { prefetch_tmap(&tm.k2); prefetch_tmap(&tm.v2); }
    prefetch_tmap(&tm.q);
    mbar_init(BAR(Q_FULL), 1);
    for (int s = 0; s < KT_MAX_STAGES; ++s) {
      mbar_init(BAR(FULL_K + s), 1);
      mbar_init(BAR(FULL_V + s), 1);
      mbar_init(BAR(EMPTY_K + s), 1);
      mbar_init(BAR(EMPTY_V + s), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(BAR(S_FULL + i), 1);
      mbar_init(BAR(P_FULL + i), 4 * CG);
      mbar_init(BAR(PV_DONE + i), 1);
    }
    mbar_init(BAR(DRAIN), 1);
    mbar_init(BAR(MERGE), 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    if (S > 1) {
      // what the S splits will push into this CTA: the O^T rows of the head dimensions it owns, and every column's pair
      const int rows = min(((split + 1) * D + S - 1) / S, D) - (split * D + S - 1) / S;
      mbar_expect_tx(BAR(MERGE), (uint32_t)(S * (rows * NPT * 4 + N * 8)));
    }
    // Ahead of everything else, and of the kernels in front of this one: Q on its way into L2 and, at the reuse step,
    // the first tiles of the compacted cache straight into the ring - they need nothing but the barriers above. Tiles that would turn the ring, or hold rows of source 2, wait for the dependency.
    for (int h = 0; h < H; ++h) tma_prefetch_l2(&tm.q, h * 64, 0, g * p.G, bi);
    if (kp.early_src1) {
      set_counts(n1_early);
      int gi0;
      while (t_next < T && t_next < NS && tile_groups(t_next, gi0) + gi0 <= g1) issue_tile(t_next++);
      if (ge > g1)                                   // this split holds the block's fresh rows
        for (int h = 0; h < H; ++h) { tma_prefetch_l2(&tm.k2, h * 64, 0, g, bi); tma_prefetch_l2(&tm.v2, h * 64, 0, g, bi); }
    }
  }
  // query rows past N (N not a multiple of 32) take part in the MMAs: they must be finite
  if (N < NPT)
    for (int i = tid; i < H * (NPT - N) * 8; i += NTHREADS) {
      const int h = i / ((NPT - N) * 8), r = i % ((NPT - N) * 8);
      reinterpret_cast<uint4*>(q_s + h * NPT * 128 + N * 128)[r] = make_uint4(0u, 0u, 0u, 0u);
    }
  if (warp == 1) {                       // the MMA warp owns the tensor memory
    tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
    tmem_relinquish();
  }
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // The next kernel in the stream may start its own set-up now; before it touches anything this kernel writes it
  // waits for this grid to complete (griddepcontrol.wait, in that kernel).
  if (kp.early_trigger) grid_launch_dependents();
  // the one cluster barrier: "this CTA runs, its barriers are set up" (their initialisation was released to the cluster by
  // the fence above); waited for before the pushes
  if (S > 1) cluster_arrive_relaxed();

  if (kp.early_src1 && tid != 0) set_counts(n1_early);
  // Everything else comes after the kernels in front of this one: the threads read the counts, write global memory, or
  // depend on Q. (All lanes of the producer warp take the wait together: a warp blocks in it as a whole.)
  grid_dependency_wait();
  if (!kp.early_trigger) grid_launch_dependents();
  if (!kp.early_src1) read_counts();

  float l_lane = 0.f;                    // softmax warps: the sum over this warp's 32 key rows of column `lane` of its group
  bool dead = false;                     // softmax warps: a wait gave up; the warp keeps meeting the others at every barrier

  if (warp == 0) {
    // ======================================= TMA producer =======================================
    if (lane == 0) {
      mbar_expect_tx(BAR(Q_FULL), (uint32_t)(H * N * 128));
      for (int h = 0; h < H; ++h) tma_load_4d(smem_u32(q_s + h * NPT * 128), &tm.q, BAR(Q_FULL), h * 64, 0, g * p.G, bi);
      while (t_next < T && issue_tile(t_next)) ++t_next;
      if (*abort_flag) {
        // let the copies that were issued land before the CTA retires
        for (int j = max(k_issued - NS, 0); j < k_issued; ++j) drain_bar(BAR(FULL_K + j % NS), (j / NS) & 1);
        for (int j = max(v_issued - NS, 0); j < v_issued; ++j) drain_bar(BAR(FULL_V + j % NS), (j / NS) & 1);
        drain_bar(BAR(Q_FULL), 0);
      }
    }
  } else if (warp == 1) {
    // ======================================= MMA issuer =======================================
    if (lane == 0) {
      const uint32_t idesc_s = kt_idesc(NPT, false, false);
      const uint32_t idesc_pv = kt_idesc(NPT, true, true);
      const uint32_t qsm = smem_u32(q_s);
      bool ok = wait_bar(BAR(Q_FULL), 0, abort_flag, p.status, 3, wlim);
      const uint32_t ring_a = smem_u32(ring), p_a = smem_u32(p_s);
      const bool two_p = kp.PB == 2;
      auto issue_pv = [&](int j, int s, uint32_t par) -> bool {       // tile j lives in ring slot s, in its use of parity par
        const int pb = j & 1;
        const int ng = min(GPT, ge - (gb + GPT * j));
        if (!wait_bar(BAR(P_FULL + pb), (j >> 1) & 1, abort_flag, p.status, 4, wlim)) return false;
        if (!wait_bar(BAR(FULL_V + s), par, abort_flag, p.status, 5, wlim)) return false;
        tc_fence_after();
        const uint32_t vsm = ring_a + (uint32_t)s * SLOT + KV_BYTES;
        const uint32_t psm = p_a + ((two_p && pb) ? (uint32_t)PBUF : 0u);
        // O^T += V^T P^T, 16 keys per instruction. A: the V tile read MN-major (the head dimension runs along M; its two
        // 64-element halves lie HALF bytes apart; with D = 64 both halves alias the same data and rows 64..127 of O^T
        // are duplicates nobody reads). B: P^T, MN-major, 8 keys per swizzle atom; its 64-column halves lie 16 KB apart.
        for (int ks = 0; ks < 2 * ng; ++ks)
          mma_ss(tmem_base + O_COL + (uint32_t)(j % WG) * NPT, smem_desc(vsm + ks * 2048, H == 2 ? (uint32_t)HALF : 0u, 1024u),
                 CG > 1 ? smem_desc(psm + ks * 2048, 128u * 128u, 1024u) : smem_desc_sw64(psm + ks * 1024, (uint32_t)PBUF, 512u),
                 idesc_pv, (j >= WG || ks > 0) ? 1u : 0u);
        tc_commit(BAR(PV_DONE + pb));    // two alternating barriers: a waiter is never a whole phase ahead of either
        tc_commit(BAR(EMPTY_V + s));
        return true;
      };
      int s = 0, s_prev = 0;               // ring slot of tile t and of tile t - 1, and the parities of their uses
      uint32_t par = 0, par_prev = 0;
      for (int t = 0; t < T && ok; ++t) {
        const int sb = t & 1;
        if (!wait_bar(BAR(FULL_K + s), par, abort_flag, p.status, 7, wlim)) { ok = false; break; }
        tc_fence_after();
        const uint32_t ksm = ring_a + (uint32_t)s * SLOT;
        const uint32_t d_t = tmem_base + (uint32_t)sb * NPT;
        // S^T = K_tile Q^T: the S^T buffer of tile t - 2 is free, its softmax arrived before PV(t - 2) was issued
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint32_t hk = (ks >> 2) * HALF + (ks & 3) * 32;
          const uint32_t hq = (ks >> 2) * (NPT * 128) + (ks & 3) * 32;
          mma_ss(d_t, smem_desc(ksm + hk, 16u, 1024u), smem_desc(qsm + hq, 16u, 1024u), idesc_s, ks > 0 ? 1u : 0u);
        }
        tc_commit(BAR(S_FULL + sb));
        tc_commit(BAR(EMPTY_K + s));
        if (t > 0 && !issue_pv(t - 1, s_prev, par_prev)) { ok = false; break; }
        s_prev = s; par_prev = par;
        if (++s == NS) { s = 0; par ^= 1u; }
      }
      if (ok && T > 0) ok = issue_pv(T - 1, s_prev, par_prev);
      if (*abort_flag) {                 // wait for the tensor pipe to finish what was issued before TMEM is freed
        tc_commit(BAR(DRAIN));
        drain_bar(BAR(DRAIN), 0);
      }
    }
  } else {
    // ======================================= softmax warps =======================================
    // A warp whose wait gave up (`dead`) keeps walking the tiles without touching data, so that the four warps meet at
    // every named barrier below; the barrier pattern depends only on values all four warps share.
    const int q4 = warp & 3;                           // TMEM lane quadrant this warp may access = its group of the tile
    const int row = q4 * 32 + lane;                    // key row of the tile
    const uint32_t lane_addr = tmem_base + ((uint32_t)(q4 * 32) << 16);
    const float sl2 = p.scale_log2;
    const bool scores = p.want_scores != 0;
    const int st = (tid - 64) & 127;                   // index inside the warpgroup
    const uint32_t o_col = O_COL + (uint32_t)wg * NPT + (uint32_t)cg * 32;   // this warpgroup's accumulator (columns)
    const int n_mine = min(max(N - 32 * cg, 0), 32);   // real query columns among this group's 32
    const bool two_p = kp.PB == 2;
    for (int t = wg; t < T; t += WG) {
      const int sb = t & 1;
      const int gi0 = gb + GPT * t, ng = min(GPT, ge - gi0);
      const bool active = q4 < ng;                     // warp-uniform: this warp's group exists in the tile
      Group x{1, 0, 0};
      if (active) x = group_of(gi0 + q4, g1, n1, n2);
      const bool valid = lane < x.nv;                  // this thread's row is a real key
      if (!dead && !wait_bar_warp(BAR(S_FULL + sb), (t >> 1) & 1, abort_flag, p.status, 9, wlim)) dead = true;
      tc_fence_after();
      const bool work = active && !dead;
      float sv[NP];                                    // this key's logits against the N queries, then their scaled distance to the references
      if (work) {
        tmem_ld32(lane_addr + (uint32_t)sb * NPT + (uint32_t)cg * 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[0]));
        tc_wait_ld();
      } else {
#pragma unroll
        for (int c = 0; c < NP; ++c) sv[c] = 0.f;
      }
      // ---- saliency of this key (refresh step): scale * mean of its N logits ----
      if (scores) {
        float a4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int c = 0; c < NP; ++c)
          if (c < n_mine) a4[c & 3] += sv[c];
        float a = (a4[0] + a4[1]) + (a4[2] + a4[3]);
        if constexpr (CG > 1) {
          // the key's logits are spread over the column groups: their sums meet in shared memory (two buffers in turn,
          // so the next tile never overwrites what the first group is still adding up)
          sal_s[(t & 1) * 128 + row] = a;
          softmax_barrier_all<NG>();
          if (cg == 0) {
#pragma unroll
            for (int c2 = 1; c2 < CG; ++c2) a += reinterpret_cast<const float*>(gblk + c2 * KT_GRP + 1536)[(t & 1) * 128 + row];
          }
        }
        if (cg == 0 && work && valid && x.src1)
          p.raw_scores[(int64_t)(bi * p.Hkv + g) * p.n1_max + x.row0 + lane] = a * (p.scale / (float)N);
      }
      // ---- the references. The first key of the CTA's first tile lends its logits: it is part of the softmax, so sums
      //      never vanish, and exp2 of anything up to 2^64 above it is still an ordinary bf16 / fp32 number. Every tile is
      //      only checked against the references; one that exceeds them by more than 64 raises them (rare). ----
      if (t < WG) {
        if (row == 0 && work) {
#pragma unroll
          for (int c = 0; c < NP; c += 4)
            *reinterpret_cast<float4*>(m_ref + c) = make_float4(sv[c] * sl2, sv[c + 1] * sl2, sv[c + 2] * sl2, sv[c + 3] * sl2);
        }
        softmax_barrier(bar_id);
      }
      float far0 = -INFINITY, far1 = -INFINITY;        // the largest distance above a reference
#pragma unroll
      for (int c = 0; c < NP; c += 4) {
        const float4 m4 = *reinterpret_cast<const float4*>(m_ref + c);
        sv[c] = fmaf(sv[c], sl2, -m4.x); sv[c + 1] = fmaf(sv[c + 1], sl2, -m4.y);
        sv[c + 2] = fmaf(sv[c + 2], sl2, -m4.z); sv[c + 3] = fmaf(sv[c + 3], sl2, -m4.w);
        far0 = fmaxf(far0, fmaxf(sv[c], sv[c + 1])); far1 = fmaxf(far1, fmaxf(sv[c + 2], sv[c + 3]));
      }
      const bool over = fmaxf(far0, far1) > 64.f;
      if (softmax_barrier_or(bar_id, over && work && valid)) {
        // ---- raise the references by the tile's column maxima (where positive) and rescale what has been accumulated.
        //      Every PV issued so far must have landed before O^T is rewritten; the PV of this tile waits for our arrive. ----
        if (t >= WG && !dead && !wait_bar_warp(BAR(PV_DONE + ((t - WG) & 1)), ((t - WG) >> 1) & 1, abort_flag, p.status, 8, wlim)) dead = true;
        tc_fence_after();
        if (st < NP) enc[st] = f2ord(0.f);
        softmax_barrier(bar_id);
        if (work) {
          float mine = 0.f;
#pragma unroll
          for (int c = 0; c < NP; ++c) {
            const float r = warp_max_f32(valid ? sv[c] : -INFINITY);
            if (c == lane) mine = r;
          }
          atomicMax(enc + lane, f2ord(mine));
        }
        softmax_barrier(bar_id);
        if (st < NP) {
          const float dlt = ord2f(enc[st]);            // >= 0
          delta_s[st] = dlt;
          m_ref[st] += dlt;
        }
        softmax_barrier(bar_id);
#pragma unroll
        for (int c = 0; c < NP; ++c) sv[c] -= delta_s[c];
        l_lane *= fast_exp2(-delta_s[lane]);
        if (t >= WG && !dead) {
          // this thread's TMEM lane is a head dimension of O^T here, not a key: all four warps rescale their lanes
          uint32_t o32[32];
          tmem_ld32(lane_addr + o_col, o32);
          tc_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) o32[i] = __float_as_uint(__uint_as_float(o32[i]) * fast_exp2(-delta_s[i]));
          tmem_st16(lane_addr + o_col, *reinterpret_cast<uint32_t(*)[16]>(&o32[0]));
          tmem_st16(lane_addr + o_col + 16, *reinterpret_cast<uint32_t(*)[16]>(&o32[16]));
          tc_wait_st();
        }
        softmax_barrier(bar_id);         // delta_s and m_ref are stable again before the next tile reads them
      }
      // ---- P^T = exp2(distance to the reference) as bf16, one 128-byte row per key (128-byte swizzle) ----
      // the P^T buffer is free once the PV that read it has completed
      const int tp = two_p ? t - 2 : t - 1;            // the tile whose PV read this buffer last
      if (!dead && tp >= 0 && !wait_bar_warp(BAR(PV_DONE + (tp & 1)), (tp >> 1) & 1, abort_flag, p.status, 6, wlim)) dead = true;
      if (active && !dead) {
        // CG = 1: rows of 64 bytes, 64-byte swizzle; CG > 1: 128-byte rows per 64-column half, this group's 32 columns
        // are chunks 4 * (cg & 1) .. of half cg / 2; the 16-byte chunk index is XORed with address bits 7.. of the row
        unsigned char* prow = p_s + ((two_p && sb) ? PBUF : 0) + (CG == 1 ? row * 64 : (cg >> 1) * (128 * 128) + row * 128);
        const int swz = CG == 1 ? ((row >> 1) & 3) : (row & 7);
        const int cbase = CG == 1 ? 0 : 4 * (cg & 1);
        if (x.nv < 32) {                               // ragged group (warp-uniform): rows past the count contribute nothing
#pragma unroll
          for (int c = 0; c < NP; ++c) sv[c] = valid ? sv[c] : -INFINITY;
        }
#pragma unroll
        for (int c8 = 0; c8 < NP / 8; ++c8) {
          uint32_t pk[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int c = c8 * 8 + 2 * i;
            const float e0 = fast_exp2(sv[c]);
            const float e1 = fast_exp2(sv[c + 1]);
            sv[c] = e0; sv[c + 1] = e1;
            pk[i] = pack_bf16(e0, e1);
          }
          *reinterpret_cast<uint4*>(prow + (((cbase + c8) ^ swz) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
        // ---- V rows of this group past its count may hold anything: zero them so that 0 * V stays 0 ----
        if (x.nv < 32 && cg == 0) {
          const int s = t % NS;
          if (!wait_bar_warp(BAR(FULL_V + s), (t / NS) & 1, abort_flag, p.status, 10, wlim)) dead = true;
          unsigned char* vs = ring + (size_t)s * SLOT + KV_BYTES;
          const int nz = dead ? 0 : (32 - x.nv) * H * 8;          // 16-byte chunks to clear
          for (int i = lane; i < nz; i += 32) {
            const int rr = q4 * 32 + x.nv + i / (H * 8), c = i % (H * 8);
            *reinterpret_cast<uint4*>(vs + (c >> 3) * HALF + rr * 128 + (((c & 7) ^ (rr & 7)) << 4)) = make_uint4(0u, 0u, 0u, 0u);
          }
        }
        fence_proxy_async();
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0 && !dead) mbar_arrive(BAR(P_FULL + sb));
      // ---- column sums, off the critical path (the MMA warp already has P^T): shuffle transpose over the warp's 32 key
      //      rows, lane i ends up with the sum of column i ----
      if (active && !dead) {
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
          const bool up_half = (lane & off) != 0;
#pragma unroll
          for (int k = 0; k < off; ++k) {
            const float send = up_half ? sv[k] : sv[k + off];
            const float keep = up_half ? sv[k + off] : sv[k];
            sv[k] = keep + __shfl_xor_sync(0xffffffffu, send, off);
          }
        }
        l_lane += sv[0];
      }
    }
  }

  // ======================================= epilogue =======================================
  const bool do_attn = p.out != nullptr;
  const int DL = kp.DL;                  // head dimensions a CTA owns in the merge: ceil(D / S)
  uint32_t ov[NP];                       // softmax threads: this thread's head dimension of O^T, its group's 32 columns
  float l_mine = 0.f, m_mine = -INFINITY;// softmax thread st < 32: sum and reference of column 32 * cg + st
  const bool carry = warp >= 2 && (WG == 1 || grp == 0);      // the threads that carry the result out
  if (warp >= 2) {
    const int q4 = warp & 3;
    const int row = q4 * 32 + lane;      // from here on: a head dimension of O^T
    const int st = (tid - 64) & 127;     // index inside the warpgroup
    // ---- column sums over the 128 key rows: the four warps' sums in a fixed order ----
    l_w[((warp - 2) & 3) * 32 + lane] = l_lane;
    if (S > 1 && p.want_scores) __threadfence();       // this thread's raw saliency, ahead of the pushes that tell the peers
    softmax_barrier(bar_id);
    if (st < NP) {
      l_mine = (l_w[st] + l_w[32 + st]) + (l_w[64 + st] + l_w[96 + st]);
      m_mine = T > wg ? m_ref[st] : -INFINITY;
    }
    // ---- two tile-alternating warpgroups: the second one's partial (reference, sum, accumulator rows) is folded into the first one's ----
    const bool fold = WG == 2 && T >= 2;
    const float* m_a = reinterpret_cast<const float*>(smem + KT_CTRL0); const float* m_b = m_a + KT_GRP / 4;
    const float* l_a = m_a + 128; const float* l_b = l_a + KT_GRP / 4;
    if (fold) {
      if (st < NP) l_tot[st] = l_mine;
      softmax_barrier_all<NG>();         // both warpgroups' references and sums are posted
      if (wg == 0 && st < NP) {
        const float mb = m_b[st], lb = l_b[st];
        const bool ha = l_mine > 0.f, hb = lb > 0.f;
        const float ms = fmaxf(ha ? m_mine : -INFINITY, hb ? mb : -INFINITY);
        l_mine = (ha ? l_mine * fast_exp2(m_mine - ms) : 0.f) + (hb ? lb * fast_exp2(mb - ms) : 0.f);
        m_mine = ms;
      }
    }
    if (CG == 1 && carry && S > 1) {
      // every split's (reference, sum) of every column goes to every CTA of the cluster, ahead of the accumulator rows
      cluster_wait_acquire();            // every CTA of the cluster runs: its shared memory and barriers may be written
      if (st < N) {
        const uint32_t ml_a = smem_u32(ml_recv + split * NPT + st);
        for (int r = 0; r < S; ++r) st_async_f2(map_to_cta(ml_a, (uint32_t)r), map_to_cta(BAR(MERGE), (uint32_t)r), m_mine, l_mine);
      }
    }
    // ---- the finished accumulator row of this thread (its group's columns of its warpgroup's accumulator) ----
    const int t_last = T > wg ? wg + ((T - 1 - wg) / WG) * WG : 0;      // the warpgroup's last tile
    const bool pv_ok = !dead && T > wg && wait_bar_warp(BAR(PV_DONE + (t_last & 1)), (t_last >> 1) & 1, abort_flag, p.status, 6, wlim);
    const bool have_o = do_attn && pv_ok;
    tc_fence_after();
    if (have_o) {
      tmem_ld32(tmem_base + ((uint32_t)(q4 * 32) << 16) + O_COL + (uint32_t)wg * NPT + (uint32_t)cg * 32, ov);
      tc_wait_ld();
    } else {
#pragma unroll
      for (int c = 0; c < NP; ++c) ov[c] = 0u;
    }
    if (fold) {
      // The rows cross in the first ring slot, once both warpgroups have seen their last PV complete. Every thread scales
      // its own row to the common references; the factors are recomputed from the posted references and sums.
      float4* xch = reinterpret_cast<float4*>(ring);                // [NP / 4][128 rows]
      softmax_barrier_all<NG>();
#pragma unroll
      for (int c4 = 0; c4 < NP / 4; ++c4) {
        const float4 ma = *reinterpret_cast<const float4*>(m_a + 4 * c4), mb = *reinterpret_cast<const float4*>(m_b + 4 * c4);
        const float4 la = *reinterpret_cast<const float4*>(l_a + 4 * c4), lb = *reinterpret_cast<const float4*>(l_b + 4 * c4);
        const float mav[4] = {ma.x, ma.y, ma.z, ma.w}, mbv[4] = {mb.x, mb.y, mb.z, mb.w};
        const float lav[4] = {la.x, la.y, la.z, la.w}, lbv[4] = {lb.x, lb.y, lb.z, lb.w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const bool ha = lav[u] > 0.f, hb = lbv[u] > 0.f;
          const float ms = fmaxf(ha ? mav[u] : -INFINITY, hb ? mbv[u] : -INFINITY);
          const float f = wg == 0 ? (ha ? fast_exp2(mav[u] - ms) : 0.f) : (hb ? fast_exp2(mbv[u] - ms) : 0.f);
          ov[4 * c4 + u] = __float_as_uint(__uint_as_float(ov[4 * c4 + u]) * f);
        }
        if (wg == 1)
          xch[c4 * 128 + row] = make_float4(__uint_as_float(ov[4 * c4]), __uint_as_float(ov[4 * c4 + 1]), __uint_as_float(ov[4 * c4 + 2]),
                                            __uint_as_float(ov[4 * c4 + 3]));
      }
      softmax_barrier_all<NG>();
      if (wg == 0) {
#pragma unroll
        for (int c4 = 0; c4 < NP / 4; ++c4) {
          const float4 x = xch[c4 * 128 + row];
          ov[4 * c4] = __float_as_uint(__uint_as_float(ov[4 * c4]) + x.x); ov[4 * c4 + 1] = __float_as_uint(__uint_as_float(ov[4 * c4 + 1]) + x.y);
          ov[4 * c4 + 2] = __float_as_uint(__uint_as_float(ov[4 * c4 + 2]) + x.z); ov[4 * c4 + 3] = __float_as_uint(__uint_as_float(ov[4 * c4 + 3]) + x.w);
        }
      }
    }
  }
  if (CG > 1 && S > 1) {
    // Several column groups: the merge area lies over the ring. Every thread of every CTA of the cluster passes one more
    // cluster barrier; the softmax threads arrive at it only behind their last PV, so behind it no CTA's ring is in use.
    cluster_wait_acquire();              // (the barrier taken at the start: every CTA runs, its mbarriers are set up)
    cluster_arrive_release();
    cluster_wait_acquire();
  }
  if (carry) {
    const int q4 = warp & 3;
    const int row = q4 * 32 + lane;
    const int st = (tid - 64) & 127;
    const int c_first = 32 * cg;         // first query column of this group
    if (S == 1) {
      if (st < NP) l_tot[st] = l_mine > 0.f ? 1.f / l_mine : 0.f;       // one split: the normaliser itself
      softmax_barrier(bar_id);
      if (do_attn && !*abort_flag) {
        // one split: normalise and store; a warp writes 32 consecutive bf16 of one output row per column
        if (row < D) {
          // column c is row c % b of head c / b of the group: the pointer walks the rows and hops to the next head
          const int hg0 = c_first / p.b;
          int i = c_first - hg0 * p.b;
          __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(p.out) + (int64_t)bi * p.o_stride[0] + (int64_t)(g * p.G + hg0) * p.o_stride[1] +
                             (int64_t)i * p.o_stride[2] + row;
          const int64_t hop = p.o_stride[1] - (int64_t)(p.b - 1) * p.o_stride[2];
#pragma unroll
          for (int c = 0; c < NP; c += 4) {
            if (c_first + c >= N) break;
            const float4 inv = *reinterpret_cast<const float4*>(l_tot + c);
            const float iv[4] = {inv.x, inv.y, inv.z, inv.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              *o = __float2bfloat16_rn(__uint_as_float(ov[c + u]) * iv[u]);
              if (++i == p.b) { i = 0; o += hop; } else o += p.o_stride[2];
            }
          }
        }
        if (p.lse && st < NP && c_first + st < N) {
          const int c = c_first + st;
          const int hg = c / p.b, i = c - hg * p.b;
          p.lse[((int64_t)bi * p.Hq + g * p.G + hg) * p.b + i] = (m_mine + log2f(l_mine)) * kLn2;
        }
      }
    } else {
      if (CG > 1 && st < NP && c_first + st < N) {     // (one column group: pushed ahead of the accumulator rows, above)
        const uint32_t ml_a = smem_u32(ml_recv + split * NPT + c_first + st);
        for (int r = 0; r < S; ++r) st_async_f2(map_to_cta(ml_a, (uint32_t)r), map_to_cta(BAR(MERGE), (uint32_t)r), m_mine, l_mine);
      }
      if (row < D) {
        // ---- this head dimension's row of O^T goes to the CTA that owns the dimension, 16 bytes at a time (always, also
        //      when this CTA is aborting: the owner counts the bytes) ----
        const int owner = row * S / D;
        const int dl = row - (owner * D + S - 1) / S;
        const uint32_t dst = map_to_cta(smem_u32(recv + ((size_t)(split * (NPT / 4) + 8 * cg) * DL + dl) * 4), (uint32_t)owner);
        const uint32_t mb = map_to_cta(BAR(MERGE), (uint32_t)owner);
#pragma unroll
        for (int c4 = 0; c4 < NP / 4; ++c4)          // consecutive lanes (head dimensions) write consecutive 16-byte units
          st_async_f4(dst + (uint32_t)(c4 * DL * 16), mb, __uint_as_float(ov[4 * c4]), __uint_as_float(ov[4 * c4 + 1]),
                      __uint_as_float(ov[4 * c4 + 2]), __uint_as_float(ov[4 * c4 + 3]));
      }
    }
  }

  if (S > 1) {
    // ---- cluster merge: once everything owed to this CTA has landed, it merges and stores the head dimensions it owns ----
    if (CG == 1 && !carry) cluster_wait_acquire();     // (the carrying threads passed the cluster barrier before their pushes)
    wait_merge(BAR(MERGE), abort_flag, p.status, wlim);
    const bool live = do_attn && !*abort_flag;
    if (carry) {
      const int st = (tid - 64) & 127;
      const int c_mine = 32 * cg + st;   // the column whose weights this thread computes (st < 32)
      // weights of the S splits for that column, the normalisation folded in
      if (live && st < NP && c_mine < N) {
        float2 x[MS];
#pragma unroll
        for (int s2 = 0; s2 < MS; ++s2) x[s2] = ml_recv[min(s2, S - 1) * NPT + c_mine];
        float mstar = -INFINITY;
#pragma unroll
        for (int s2 = 0; s2 < MS; ++s2)
          if (s2 < S && x[s2].y > 0.f) mstar = fmaxf(mstar, x[s2].x);
        float w[MS], l = 0.f;
#pragma unroll
        for (int s2 = 0; s2 < MS; ++s2) {
          w[s2] = (s2 < S && x[s2].y > 0.f) ? fast_exp2(x[s2].x - mstar) : 0.f;
          l = fmaf(x[s2].y, w[s2], l);
        }
        const float inv = l > 0.f ? 1.f / l : 0.f;
#pragma unroll
        for (int s2 = 0; s2 < MS; ++s2)
          if (s2 < S) w_s[s2 * NPT + c_mine] = w[s2] * inv;
        if (split == 0 && p.lse) {
          const int hg = c_mine / p.b, i = c_mine - hg * p.b;
          p.lse[((int64_t)bi * p.Hq + g * p.G + hg) * p.b + i] = (mstar + log2f(l)) * kLn2;
        }
      }
      if constexpr (CG > 1) softmax_barrier_all<NG>(); else softmax_barrier(1);
      // thread -> (owned head dimension, chunk of columns); all loads of a group of four columns are in flight together
      const int d_lo = (split * D + S - 1) / S, d_hi = min(((split + 1) * D + S - 1) / S, D);
      const int sa = 128 * cg + st;      // index among all carrying threads
      const int dl = sa % DL, qc = sa / DL;
      const int cpt = kp.cpt;            // columns per thread, a multiple of 4
      if (live && d_lo + dl < d_hi) {
        for (int c0 = qc * cpt; c0 < min((qc + 1) * cpt, N); c0 += 4) {
          float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
          float4 r4[MS], w4[MS];                         // all splits' loads in flight together
#pragma unroll
          for (int s2 = 0; s2 < MS; ++s2) {
            const int sc = min(s2, S - 1);
            r4[s2] = *reinterpret_cast<const float4*>(recv + ((size_t)(sc * (NPT / 4) + (c0 >> 2)) * DL + dl) * 4);
            w4[s2] = *reinterpret_cast<const float4*>(w_s + sc * NPT + c0);
          }
#pragma unroll
          for (int s2 = 0; s2 < MS; ++s2)
            if (s2 < S) {
              acc.x = fmaf(r4[s2].x, w4[s2].x, acc.x); acc.y = fmaf(r4[s2].y, w4[s2].y, acc.y);
              acc.z = fmaf(r4[s2].z, w4[s2].z, acc.z); acc.w = fmaf(r4[s2].w, w4[s2].w, acc.w);
            }
          const float a[4] = {acc.x, acc.y, acc.z, acc.w};
          const int hg = c0 / p.b, i0 = c0 - hg * p.b;    // b is a multiple of 16: the four columns are rows of one head
          __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(p.out) + (int64_t)bi * p.o_stride[0] +
                             (int64_t)(g * p.G + hg) * p.o_stride[1] + (int64_t)i0 * p.o_stride[2] + d_lo + dl;
#pragma unroll
          for (int i4 = 0; i4 < 4; ++i4) o[(int64_t)i4 * p.o_stride[2]] = __float2bfloat16_rn(a[i4]);
        }
      }
    }
  } else {
    __syncthreads();                     // the raw saliency of the whole head is visible to this CTA
  }

  // ---- pooling of the head's saliency (refresh step): this CTA's share of the positions ----
  if (p.want_scores && p.pooled != nullptr && !*abort_flag) {
    const float* a = p.raw_scores + (int64_t)(bi * p.Hkv + g) * p.n1_max;
    const int p_lo = (int)(((long long)split * p.n1_max) / S), p_hi = (int)(((long long)(split + 1) * p.n1_max) / S);
    const int o = p.block_off[bi];
    kt_pool_span(p, a, p.pooled + (int64_t)(bi * p.Hkv + g) * p.n1_max, n1, o, p_lo, p_hi, tid, NTHREADS);
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
size_t kt_smem_bytes(int D, int CG, int WG, int NS, int PB, int S) {
  const size_t H = D / 64, NPT = 32 * CG, NG = (size_t)CG * WG;
  const size_t DL = (D + S - 1) / S;
  const size_t pbuf = CG == 1 ? 128 * 64 : (size_t)((CG + 1) / 2) * 128 * 128;
  const size_t ring = (size_t)NS * 2 * H * 128 * 128;
  const size_t merge = S > 1 ? (size_t)S * DL * NPT * 4 /*recv*/ + (size_t)S * NPT * 12 /*ml_recv, w_s*/ : 0;
  // one column group: the merge area follows the ring; several: it lies over the ring (which must be large enough)
  const size_t tail = CG == 1 ? ring + merge : (ring > merge ? ring : merge);
  return 1024 /*alignment slack*/ + KT_CTRL0 + NG * KT_GRP + H * NPT * 128 + (size_t)PB * pbuf + tail;
}

// what has been set as the kernel's dynamic shared memory limit, per device (one record per kernel: launch and
// occupancy query both raise it, neither may lower it behind the other's back)
template <int D, int WG, int CG>
SmemConfig& kt_smem_config() {
  static SmemConfig configured;
  return configured;
}

template <int D, int WG, int CG>
cudaError_t launch_kt_d(const KtMaps& tm, const KtParams& kp, const AttnPlan& pl, bool pdl, cudaStream_t st) {
  auto kern = attn_kt_kernel<D, WG, CG>;
  cudaError_t e = configure_smem(reinterpret_cast<const void*>(kern), pl.smem_bytes, kt_smem_config<D, WG, CG>(), true);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(kp.S, kp.a.Hkv, kp.a.B);
  cfg.blockDim = dim3(64 + 128 * WG * CG);
  cfg.dynamicSmemBytes = pl.smem_bytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  int na = 0;
  if (pdl) {
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  if (kp.S > 1) {                            // the key splits (grid x) of a unit form one cluster
    attr[na].id = cudaLaunchAttributeClusterDimension;
    attr[na].val.clusterDim.x = kp.S; attr[na].val.clusterDim.y = 1; attr[na].val.clusterDim.z = 1;
    ++na;
  }
  cfg.attrs = attr; cfg.numAttrs = na;
  return cudaLaunchKernelEx(&cfg, kern, tm, kp);
}

template <int D>
cudaError_t launch_kt_shape(const KtMaps& tm, const KtParams& kp, const AttnPlan& pl, int WG, int CG, bool pdl, cudaStream_t st) {
  if (WG == 2) return launch_kt_d<D, 2, 1>(tm, kp, pl, pdl, st);
  switch (CG) {
    case 1: return launch_kt_d<D, 1, 1>(tm, kp, pl, pdl, st);
    case 2: return launch_kt_d<D, 1, 2>(tm, kp, pl, pdl, st);
    case 3: return launch_kt_d<D, 1, 3>(tm, kp, pl, pdl, st);
    default: return launch_kt_d<D, 1, 4>(tm, kp, pl, pdl, st);
  }
}

// How many clusters of S whole-SM CTAs (several column groups: footprint (c)) the current device keeps resident at once:
// cudaOccupancyMaxActiveClusters, asked once per (head dimension, column groups, cluster size) and device. -1: no answer.
template <int D, int WG, int CG>
int kt_query_clusters(int S) {
  auto kern = attn_kt_kernel<D, WG, CG>;
  const size_t smem = 200 * 1024;        // any footprint above half an SM: one CTA per SM
  if (configure_smem(reinterpret_cast<const void*>(kern), 226 * 1024, kt_smem_config<D, WG, CG>(), true) != cudaSuccess) return -1;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(S, 1, 1);
  cfg.blockDim = dim3(64 + 128 * WG * CG);
  cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = S; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) { (void)cudaGetLastError(); return -1; }
  return n;
}
// (CG = 1 stands for footprint (b): two tile-alternating softmax warpgroups on one column group)
int kt_resident_clusters(int D, int CG, int S) {
  static std::mutex mu;
  static int cache[kMaxDevices][2][5][9];          // [device][D == 128][CG][S]: 0 = not asked yet, else answer + 2
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { (void)cudaGetLastError(); return -1; }
  if (CG < 1 || CG > 4 || S < 2 || S > 8) return -1;
  std::lock_guard<std::mutex> lock(mu);
  int& c = cache[dev][D == 128 ? 1 : 0][CG][S];
  if (c == 0) {
    int n = -1;
    if (D == 128) n = CG == 1 ? kt_query_clusters<128, 2, 1>(S) : (CG == 2 ? kt_query_clusters<128, 1, 2>(S) : (CG == 3 ? kt_query_clusters<128, 1, 3>(S) : kt_query_clusters<128, 1, 4>(S)));
    else n = CG == 1 ? kt_query_clusters<64, 2, 1>(S) : (CG == 2 ? kt_query_clusters<64, 1, 2>(S) : (CG == 3 ? kt_query_clusters<64, 1, 3>(S) : kt_query_clusters<64, 1, 4>(S)));
    c = n + 2;
  }
  return c - 2;
}

}  // namespace

// Whether the key-row kernel covers a shape: bf16, D in {64, 128}, at most 128 query rows per KV head, block length a
// multiple of 16.
bool kt_supported(int dtype, int D, int M, int b) {
  return umma_supported(dtype, D, M, b) && M <= 128;
}

// Whether the planner picks it among the shapes it covers. A unit's key splits are the CTAs of one cluster, eight at
// most. With up to 32 query rows that is enough everywhere. With more, a CTA takes a whole SM, and a few units with
// long key ranges (8 KV heads, one sequence, 16k keys: 64 CTAs) would leave most SMs idle; the query-row kernel splits
// those further through its workspace and measured faster there (25 against 38 us), slower with 64 units and more.
// Short walks are latency chains whatever the number of CTAs, and this kernel's chain is the shorter one: up to six
// tiles per CTA at 64 query columns (8 KV heads x 1024 keys: 8.1 against 14.5 us; x 4096: 12.2 against 15.2), up to two
// with more columns (12.1 against 13.0 us at 128 columns x 1024 keys; at 4096 keys the query-row kernel is ahead).
bool kt_preferred(int M, int B, int Hkv, int n1_max, int n2) {
  if (M <= 32) return true;
  const long long units = (long long)B * Hkv;
  const int sms = sm_count();
  long long S = sms / units;
  const long long by_tiles = ((n1_max + 31) / 32 + (n2 + 31) / 32 + 3) / 4;
  if (S > by_tiles) S = by_tiles;
  if (S > 8) S = 8;
  if (S < 1) S = 1;
  const long long tiles_cta = (by_tiles + S - 1) / S;
  // (three or four column groups walk a tile in 2 us, the query-row kernel in 1.5: long walks go there even when the
  // SMs are filled - 32 units x 128 tiles: 70.7 against 79.6 us)
  // (with 16 to 24 units the query-row kernel, which can use more CTAs, is ahead from five tiles per CTA on: 19.7 against
  // 22.3 us at 16 units x 33 tiles)
  if (units * S * 4 >= (long long)sms * 3) return M <= 64 || tiles_cta <= (units >= 32 ? 16 : 4);
  return tiles_cta <= (M <= 64 ? 6 : 2);
}

AttnPlan plan_attention_kt(int D, int M, int b, int B, int Hkv, int n1_max, int n2, const Tuning& tn) {
  (void)b;
  AttnPlan pl{};
  pl.kind = 3; pl.tma = true; pl.fused_tail = true;
  pl.key_tile = 128; pl.key_tile2 = n2 < 32 ? n2 : 32;
  pl.rep = 1; pl.row_tiles = 1; pl.rows_rep = M;
  const int CG = (M + 31) / 32;          // column groups of 32 query columns: one softmax warpgroup each
  const int groups = (n1_max + 31) / 32 + (n2 + 31) / 32;
  const long long units = (long long)B * Hkv;
  const int sms = sm_count();
  // Key splits: enough CTAs to fill the SMs (two per SM with one column group), but at least one full 128-key tile
  // per CTA, and at most eight (one cluster).
  long long want = (CG == 1 ? 2 : 1) * (long long)sms / units;
  const long long by_tiles = (groups + 3) / 4;
  if (want > by_tiles) want = by_tiles;
  // Six groups of 32 keys at most (two tiles, the second one short): one CTA walks both rather than two CTAs one each -
  // a short second tile costs less than the cluster merge (124 cached keys, 32 heads: 6.0 against 6.9 us; with eight
  // groups four splits are ahead again, 6.7 against 7.3 us).
  if (groups <= 6) want = 1;
  // More than half as many units as SMs, each with a walk of five tiles or more: one whole-SM CTA per unit (footprint
  // (b) below) beats two splits per unit at two CTAs per SM - the same share of the SMs is busy and nothing is merged
  // (128 units x 17 tiles: 29.6 against 32.8 us; 96 units x 5 tiles: 12.3 against 19.3 us with clusters of three; at
  // 128 units x 5 tiles the two are equal).
  if (CG == 1 && D == 128 && units * 2 > sms && units <= sms && groups >= 20) want = 1;
  if (tn.splits > 0) want = tn.splits;
  if (want > 8) want = 8;
  if (want < 1) want = 1;
  // Clusters of 3, 5 or 7 measured slower than the next even size (7.4 / 7.6 / 7.9 us against 6.8 / 7.2 / 7.8 us per
  // reuse call of 32 heads at 9, 17 and 25 groups): uneven shares of the head dimensions in the merge, and clusters that
  // pack the SMs of a GPC badly.
  // Where the next even size would leave the one-wave budget, the one below is taken.
  if (tn.splits <= 0 && want >= 3 && (want & 1))
    want += (want + 1 <= groups && units * (want + 1) <= (CG == 1 ? 2 : 1) * (long long)sms) ? 1 : -1;
  if (CG > 1 && tn.splits <= 0) {
    // Whole-SM CTAs: a cluster needs its SMs inside one GPC, so fewer clusters are resident than SMs / S suggests (16
    // clusters of eight do not fit a B200, 16 of six do, 24 of six do not, 32 of four do). A grid whose clusters do not
    // all fit runs in two waves: 15.9 against 9.3 us for 16 units x 1024 keys. The device is asked; without an answer
    // the numbers above stand in.
    if (by_tiles <= 3 && units >= 24) want = 1;          // (short walks of many units: no split, 7.7 against 9.6 us)
    while (want > 1) {
      const int fit = kt_resident_clusters(D, CG, (int)want);
      const long long room = fit >= 0 ? fit : (want >= 7 ? 12 : (want >= 5 ? 20 : (want >= 3 ? 36 : 74)));
      if (units <= room) break;
      want = want > 2 ? ((want - 1) & ~1LL) : 1;
    }
  }
  // ... and the same for footprints (a) and (b) below: where the clusters would not all be resident the cluster size goes
  // down until they are (48 units: clusters of six at two CTAs per SM ran in two waves, 17.8 against 11.4 us with four).
  auto is_small = [&](long long s_) {
    const long long gc = (groups + s_ - 1) / s_;
    return CG == 1 && (D == 64 || gc <= 8 || (units * s_ > sms && units * s_ <= 2 * sms) || (units > sms && groups < (n2 > 0 ? 20 : 28)));
  };
  while (CG == 1 && tn.splits <= 0 && tn.dual < 0 && want > 1) {
    long long room;
    if (is_small(want)) {
      // (two CTAs per SM: the occupancy query is too careful here - it would turn away 32 clusters of six, which do run
      // together - so the rule is the measured one: clusters of three or more fill at most nine tenths of the slots)
      room = want >= 3 ? (2LL * sms * 9 / 10) / want : units;
    } else {
      const int fit = kt_resident_clusters(D, 1, (int)want);
      room = fit >= 0 ? fit : (want >= 7 ? 12 : (want >= 5 ? 20 : (want >= 3 ? 36 : 74)));
    }
    if (units <= room) break;
    want = want > 2 ? ((want - 1) & ~1LL) : 1;
  }
  const int S = (int)want;
  // Footprint, ring depth, P^T buffers and softmax warpgroups:
  // (a) one column group and either at most two full tiles per CTA or a grid that fits the GPU only at two CTAs per
  //     SM: the footprint is kept below half an SM, so that two CTAs are resident and the next call's CTAs can start
  //     loading while this call's finish;
  // (b) one column group and longer walks: the CTA takes what one SM has, and two softmax warpgroups take the tiles in
  //     turn (one warp per scheduler cannot hide its own latencies; two tiles in flight can);
  // (c) 33 to 128 query columns: one CTA per SM, one softmax warpgroup per 32 columns, all on the same tile.
  const int groups_cta = (groups + S - 1) / S;
  const size_t half_sm = 113 * 1024;     // two CTAs of this size, each with its 1 KB system share, fit one SM
  // (more units than SMs with walks of less than seven tiles at the refresh step, five at the reuse step: two small CTAs per SM overlap their set-up and way out
  // better than the resident walk of (d), whose cost per unit is about three tiles' worth: 38 against 45 us for 512
  // units of four tiles)
  // (head dimension 64: a tile is half the bytes for the same softmax, so the softmax warps are what is short: always two
  // CTAs per SM - 97.5 against 140 us for 512 units x 4352 keys, 30.2 against 41.1 us for 128 units)
  bool small = CG == 1 && (D == 64 || groups_cta <= 8 || (units * S > sms && units * S <= 2 * sms) || (units > sms && groups < (n2 > 0 ? 20 : 28)));
  int WG = (CG == 1 && !small) ? 2 : 1;
  if (tn.dual == 1) { small = CG == 1; WG = 1; }       // force (a) / (b) where they apply
  if (tn.dual == 0 && CG == 1) { small = false; WG = 2; }
  const int tiles_cta = (groups_cta + 3) / 4;
  int NS = 1, PB = WG == 2 ? 2 : 1;
  // Batches of four or more sequences whose units fit the GPU only at two CTAs per SM, with walks of twelve tiles or
  // more: the single ring slot of footprint (a) makes a CTA wait for every tile, which two CTAs per SM hide from each
  // other only while both have work. Serving batches are ragged: the long units are soon alone on their SMs and the call
  // lasts as long as the longest crawls. One softmax warpgroup with the whole SM's shared memory for a ring of three
  // slots, one CTA per SM, longest sequences first, in two waves: 62 against 81 us (refresh) and 30 against 40 us
  // (reuse) on a ragged batch of six sequences of 512 to 4096 tokens, 71 / 35 against 86 / 42 us with eight; at
  // uniform lengths it costs 4 to 11 %. (The plan is a function of the description alone, so it cannot look at the lengths.)
  const bool deep_ring = CG == 1 && S == 1 && D == 128 && small && units > sms && units <= 2 * sms && B >= 4 && tiles_cta >= 12 &&
                         tn.dual < 0;
  const size_t limit = (small && !deep_ring) ? half_sm : 226 * 1024;
  if (!small && kt_smem_bytes(D, CG, WG, 1, 2, S) <= limit) PB = 2;
  while (NS < KT_MAX_STAGES && NS < tiles_cta && kt_smem_bytes(D, CG, WG, NS + 1, PB, S) <= limit) ++NS;
  if (!small && PB == 2 && WG == 1 && NS < 2 && tiles_cta >= 2 && kt_smem_bytes(D, CG, WG, 2, 1, S) <= limit) { PB = 1; NS = 2; }   // a second ring slot is worth more than a second P^T buffer
  if (tn.stages > 0) {
    NS = tn.stages > KT_MAX_STAGES ? KT_MAX_STAGES : tn.stages;
    while (NS > 1 && kt_smem_bytes(D, CG, WG, NS, PB, S) > 226 * 1024) --NS;
  }
  pl.splits = 1;                        // nothing is left in the workspace: the splits merge inside their cluster
  pl.parts = 1;
  pl.cluster = S;
  pl.stages = NS;
  pl.m_warps = PB;                      // (field reused: P^T buffers)
  pl.c_warps = WG;                      // (field reused: tile-alternating softmax warpgroups)
  pl.warp_keys = CG;                    // (field reused: column groups)
  pl.threads = 64 + 128 * WG * CG;
  pl.part_rows = 0;
  pl.n_counters = 0;
  pl.smem_bytes = kt_smem_bytes(D, CG, WG, NS, PB, S);
  // (d) as (b), but with more units than SMs: the CTAs would run in waves, each paying its set-up and its way out with
  //     the SM's memory pipe idle; one resident CTA per SM walks the units as one sequence of tiles instead.
  pl.persistent = CG == 1 && S == 1 && WG == 2 && units > sms;
  if (tn.persist == 0) pl.persistent = false;
  if (tn.persist >= 1) pl.persistent = CG == 1 && S == 1;
  if (pl.persistent) {
    pl.stages = 3; pl.m_warps = 2; pl.c_warps = 2; pl.threads = 64 + 2 * 128;
    pl.smem_bytes = kt_stream_smem_bytes(D);
    pl.n_counters = 2;                  // the next unit to hand out, and the CTAs that have finished
  }
  return pl;
}

cudaError_t launch_attn_kt(const AttnParams& p, const AttnPlan& pl, int D, cudaStream_t st) {
  const Tuning tn = tuning();
  KtMaps tm;
  KtParams kp{};
  const int CG = (p.M + 31) / 32, WG = pl.c_warps;
  kp.a = p;
  kp.a.wait_cycles = tn.wait_cycles;
  kp.N = p.M; kp.S = pl.cluster; kp.NS = pl.stages; kp.PB = pl.m_warps;
  kp.DL = (D + kp.S - 1) / kp.S;
  {
    const int chunks = 128 * CG / kp.DL;                 // carrying threads that share one owned head dimension
    kp.cpt = ((32 * CG + chunks - 1) / chunks + 3) / 4 * 4;
  }
  kp.gr2 = p.n2 < 32 ? p.n2 : 32;
  kp.early_src1 = (p.n2 > 0 && p.n1_max > 0 && tn.early_loads != 0) ? 1 : 0;
  kp.early_trigger = tn.trigger != 0 ? 1 : 0;
  {
    const long long ctas = (long long)kp.S * p.Hkv * p.B;
    kp.lpt = (p.n1_per_seq != nullptr && p.B >= 4 && p.B <= 64 && ctas > sm_count()) ? 1 : 0;
    if (tn.lpt >= 0) kp.lpt = (tn.lpt == 1 && p.n1_per_seq != nullptr && p.B >= 2 && p.B <= 64) ? 1 : 0;
  }
  kp.wait_cycles = tn.wait_cycles;
  memset(&tm, 0, sizeof(tm));
  bool ok = umma_make_map(&tm.q, p.q, D, p.b, p.Hq, p.B, p.q_stride, p.b, p.G);
  if (p.n1_max > 0) {
    ok = ok && umma_make_map(&tm.k1, p.k1, D, p.n1_max, p.Hkv, p.B, p.k1_stride, 32, 1);
    ok = ok && umma_make_map(&tm.v1, p.v1, D, p.n1_max, p.Hkv, p.B, p.k1_stride, 32, 1);
    ok = ok && umma_make_map(&tm.k1t, p.k1, D, p.n1_max, p.Hkv, p.B, p.k1_stride, 128, 1);
    ok = ok && umma_make_map(&tm.v1t, p.v1, D, p.n1_max, p.Hkv, p.B, p.k1_stride, 128, 1);
  }
  if (p.n2 > 0) {
    ok = ok && umma_make_map(&tm.k2, p.k2, D, p.n2, p.Hkv, p.B, p.k2_stride, kp.gr2, 1);
    ok = ok && umma_make_map(&tm.v2, p.v2, D, p.n2, p.Hkv, p.B, p.k2_stride, kp.gr2, 1);
    if (p.n1_max <= 0) { tm.k1 = tm.k2; tm.v1 = tm.v2; tm.k1t = tm.k2; tm.v1t = tm.v2; }
  } else {
    tm.k2 = tm.k1; tm.v2 = tm.v1;
  }
  if (!ok) return cudaErrorInvalidValue;
  const bool pdl = tn.pdl != 0;
  if (pl.persistent) {
    kp.lpt = (p.n1_per_seq != nullptr && p.B <= 64 && tn.lpt != 0) ? 1 : 0;      // the walk starts with the longest sequences
    return launch_kt_stream(tm, kp, D, pl.smem_bytes, pdl, st);
  }
  return D == 128 ? launch_kt_shape<128>(tm, kp, pl, WG, CG, pdl, st) : launch_kt_shape<64>(tm, kp, pl, WG, CG, pdl, st);
}

}  // namespace sdllm
