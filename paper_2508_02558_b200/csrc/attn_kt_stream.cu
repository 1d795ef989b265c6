// bf16 block-query attention with the keys on the accumulator rows, streaming variant for large batches.
//
// attn_kt.cu gives every (sequence, KV head) unit its own CTA (or cluster). With several hundred units and long key
// ranges each CTA takes a whole SM, so the units run in waves, and what a CTA does before its first tile arrives and
// after its last one (barriers, tensor memory, the Q load, the first K/V tiles' latency, the way out of TMEM) is paid
// once per unit with the SM's memory pipe idle. Here one CTA per SM stays resident and takes unit after unit from a
// counter in the workspace (units ordered from the longest sequence to the shortest, so the short ones fill the end),
// as ONE sequence of 128-key tiles: the producer runs ahead into the next unit's tiles while the softmax warps finish the
// current one, the barriers' phases simply continue, and nothing is set up twice.
//
// Shape: up to 32 query rows per KV head (one column group), one split per unit, two softmax warpgroups that take the
// tiles in turn (even / odd tiles of the CTA's sequence), each with its own references and accumulator; at the end of
// a unit warpgroup 0 reads both accumulators from tensor memory, folds them and stores the output rows.
//   warp 0      TMA producer: K and V tiles into a three-slot ring, Q of the next unit once the last S^T = K Q^T of the
//               current one has completed
//   warp 1      tcgen05.mma issuer: S^T = K_tile Q^T, O^T_w += V_tile^T P^T
//   warps 2-5   softmax warpgroup 0 (even tiles), carries every unit's result out
//   warps 6-9   softmax warpgroup 1 (odd tiles)
// Algorithm 3 (reuse step, Concat(K_c, K_n)) and Algorithm 1 (refresh step: attention over the full K/V plus the mean
// logit of every key and its max-pooling) as in attn_kt.cu; every mbarrier wait is bounded in the same way.
#include <cuda.h>
#include <string.h>

#include "attn_device.cuh"
#include "kt_params.cuh"
#include "tuning.cuh"
#include "umma_host.cuh"

namespace sdllm {
using namespace dev;
namespace {

#include "kt_common.cuh"

constexpr int KS_NS = 3;                 // ring slots
constexpr int KS_THREADS = 64 + 2 * 128;
constexpr int KS_CTRL = KT_CTRL0 + 2 * KT_GRP;

// asymmetric named barriers between the two softmax warpgroups (256 threads): one side only announces, the other waits
__device__ __forceinline__ void pair_arrive(int id) { asm volatile("bar.arrive %0, 256;\n" ::"r"(id) : "memory"); }
__device__ __forceinline__ void pair_sync(int id) { asm volatile("bar.sync %0, 256;\n" ::"r"(id) : "memory"); }

template <int D>
__global__ void __launch_bounds__(KS_THREADS, 1) attn_kt_stream_kernel(const __grid_constant__ KtMaps tm, const KtParams kp) {
  constexpr int NS = KS_NS;
  constexpr int H = D / 64;                  // 128-byte column halves of a K/V row
  constexpr int NP = 32;                     // query columns (padded)
  constexpr int GPT = 4;                     // groups of 32 keys per tile
  constexpr int HALF = GPT * 32 * 128;       // bytes of one 64-column half of a tile
  constexpr int KV_BYTES = H * HALF;
  constexpr int SLOT = 2 * KV_BYTES;
  constexpr int PBUF = 128 * 64;             // one P^T buffer: 128 key rows of 64 bytes (64-byte swizzle)
  constexpr uint32_t O_COL = 2 * NP;         // TMEM columns: S^T buffers at 0 and 32, O^T of warpgroup 0 at 64, of warpgroup 1 at 96
  constexpr uint32_t TMEM_COLS = 128;
  extern __shared__ unsigned char smem_raw[];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const AttnParams& p = kp.a;
  const int N = kp.N, n2 = p.n2;
  const long long wlim = kp.wait_cycles;
  const int n_units = p.B * p.Hkv;

  // ---- shared memory carve-up (1024-byte aligned for the 128-byte swizzle) ----
  const uint32_t raw_addr = smem_u32(smem_raw);
  unsigned char* smem = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
  const uint32_t bars = smem_u32(smem);
  auto BAR = [&](int i) { return bars + 8u * (uint32_t)i; };
  constexpr int Q_FULL = 0, Q_EMPTY = 1, FULL_K = 2, FULL_V = 2 + NS, EMPTY_K = 2 + 2 * NS, EMPTY_V = 2 + 3 * NS;
  constexpr int S_FULL = 2 + 4 * NS, P_FULL = S_FULL + 2, PV_DONE = S_FULL + 4, DRAIN = S_FULL + 6;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + 256);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + 260);
  volatile int* unit_list = reinterpret_cast<volatile int*>(smem + 320);   // [16] the units this CTA took, in order (-1: no more)
  volatile int* n_pub = reinterpret_cast<volatile int*>(smem + 384);       // entries of the list published so far
  volatile int* n_done = reinterpret_cast<volatile int*>(smem + 388);      // units whose results have been stored
  int* seq_of_rank = reinterpret_cast<int*>(smem + 512);            // [64] sequence with the r-th longest source 1
  int* n1_of_rank = reinterpret_cast<int*>(smem + 768);             // [64] its clamped count
  const int grp = warp >= 6 ? 1 : 0;       // softmax warpgroup = parity of the tiles it takes
  unsigned char* gblk = smem + KT_CTRL0 + grp * KT_GRP;
  float* m_ref = reinterpret_cast<float*>(gblk);                    // [32] references of the columns (log2 units)
  uint32_t* enc = reinterpret_cast<uint32_t*>(gblk + 256);          // [32] scratch of a raise
  float* l_tot = reinterpret_cast<float*>(gblk + 512);              // [32] warpgroup 0: weights of its own accumulator
  float* delta_s = reinterpret_cast<float*>(gblk + 768);            // [32] by how much a raise lifts each reference
  float* l_w = reinterpret_cast<float*>(gblk + 1024);               // [4][32] per-warp sums
  float* post = reinterpret_cast<float*>(gblk + 1536);              // [2 unit parities][64]: references, then sums, as posted at the end of a unit
  float* w_other = reinterpret_cast<float*>(gblk + 2048);           // [32] warpgroup 0: weights of the other accumulator
  const int bar_id = 1 + grp;
  unsigned char* q_s = smem + KS_CTRL;                              // [H][32 rows][128 B]
  unsigned char* p_s = q_s + H * NP * 128;                          // [2][P^T buffer]
  unsigned char* ring = p_s + 2 * PBUF;                             // [NS][K tile | V tile]

  if (tid == 0) {
    prefetch_tmap(&tm.k1t); prefetch_tmap(&tm.v1t); prefetch_tmap(&tm.k1); prefetch_tmap(&tm.v1);
    if (n2 > 0) { prefetch_tmap(&tm.k2); prefetch_tmap(&tm.v2); }
    prefetch_tmap(&tm.q);
    mbar_init(BAR(Q_FULL), 1);
    mbar_init(BAR(Q_EMPTY), 1);
    for (int s = 0; s < NS; ++s) {
      mbar_init(BAR(FULL_K + s), 1);
      mbar_init(BAR(FULL_V + s), 1);
      mbar_init(BAR(EMPTY_K + s), 1);
      mbar_init(BAR(EMPTY_V + s), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(BAR(S_FULL + i), 1);
      mbar_init(BAR(P_FULL + i), 4);
      mbar_init(BAR(PV_DONE + i), 1);
    }
    mbar_init(BAR(DRAIN), 1);
    *abort_flag = 0;
    *n_pub = 0;
    *n_done = 0;
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  // query rows past N take part in the MMAs: they must be finite (the Q loads never touch them)
  if (N < NP)
    for (int i = tid; i < H * (NP - N) * 8; i += KS_THREADS) {
      const int h = i / ((NP - N) * 8), r = i % ((NP - N) * 8);
      reinterpret_cast<uint4*>(q_s + h * NP * 128 + N * 128)[r] = make_uint4(0u, 0u, 0u, 0u);
    }
  if (warp == 1) {                       // the MMA warp owns the tensor memory
    tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
    tmem_relinquish();
  }
  if (kp.early_trigger) grid_launch_dependents();
  grid_dependency_wait();                // the counts, Q and the block's fresh rows come from the kernels in front
  if (!kp.early_trigger) grid_launch_dependents();
  // ---- the order of the units: sequences from the longest source 1 to the shortest (ties: lower index first), so the
  //      long ones start first and the short ones fill the end. Warp 2 ranks the (at most 64) lengths. ----
  if (warp == 2) {
    for (int i = lane; i < 64; i += 32) { seq_of_rank[i] = i; n1_of_rank[i] = 0; }
    __syncwarp();
    auto count_of = [&](int i) { return i < p.B ? min(max(p.n1_per_seq ? p.n1_per_seq[i] : p.n1_max, 0), p.n1_max) : -1; };
    if (kp.lpt) {
      const int l0 = count_of(lane), l1 = count_of(lane + 32);
      int r0 = 0, r1 = 0;                // how many sequences come before mine (longer, or equal and earlier)
      for (int i = 0; i < p.B; ++i) {
        const int li = __shfl_sync(0xffffffffu, i < 32 ? l0 : l1, i & 31);
        r0 += (li > l0 || (li == l0 && i < lane)) ? 1 : 0;
        r1 += (li > l1 || (li == l1 && i < lane + 32)) ? 1 : 0;
      }
      if (lane < p.B) { seq_of_rank[r0] = lane; n1_of_rank[r0] = l0; }
      if (lane + 32 < p.B) { seq_of_rank[r1] = lane + 32; n1_of_rank[r1] = l1; }
    }
  }
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // One unit of the walk: which sequence and head, and its share of the key axis in groups of 32 rows.
  struct Unit { int bi, g, n1, g1, ge, T; };
  auto unit_of = [&](int u) {
    Unit x;
    const int rank = u / p.Hkv;
    x.g = u - rank * p.Hkv;
    if (kp.lpt) { x.bi = seq_of_rank[rank]; x.n1 = n1_of_rank[rank]; }
    else { x.bi = rank; x.n1 = min(max(p.n1_per_seq ? p.n1_per_seq[rank] : p.n1_max, 0), p.n1_max); }
    x.g1 = (x.n1 + 31) >> 5;
    x.ge = x.g1 + ((n2 + 31) >> 5);
    x.T = (x.ge + GPT - 1) / GPT;
    return x;
  };

  // The k-th unit of this CTA, as published by the producer lane (-1: no more). The answer depends on the list alone,
  // never on the abort flag or on a clock: all softmax warps must take the same units, or they would miss one another at
  // the named barriers. The producer lane publishes an end mark as soon as one of its own (bounded) waits gives up, so
  // this wait ends shortly after; its own limit is far beyond that and only guards against a producer that is gone.
  auto unit_at = [&](int k) -> int {
    if (*n_pub <= k) {
      const long long lim = 4 * (wlim > kDrainCycles ? wlim : kDrainCycles);
      const long long t0 = clock64();
      while (*n_pub <= k) {
        if (clock64() - t0 > lim) { *abort_flag = 1; atomicExch(p.status, 14); return -1; }
      }
    }
    return unit_list[k & 15];
  };

  if (warp == 0) {
    // ======================================= TMA producer =======================================
    if (lane == 0) {
      int G = 0;                         // tiles whose K and V loads are both issued (all units of this CTA)
      int k_issued = 0;                  // tiles whose K load is issued
      int qn = 0;                        // Q loads issued so far (units with at least one tile)
      bool ok = true;
      int n_listed = 0;                  // entries of the unit list written so far
      bool ended = false;                // ... the last of them being the end mark
      // The counter is asked one unit ahead: the answer for unit k + 1 travels (an L2 round trip under full load) while
      // unit k's loads are issued, instead of holding up the first loads of unit k + 1.
      int u_ahead = atomicAdd(p.counters, 1);
      for (int k = 0; ok; ++k) {
        // The next unit: whoever asks first gets the longest one left. The list in shared memory has 16 places; the
        // producer never runs more than eight units ahead of the stores (it could, through units without keys).
        if (*n_done + 8 <= k) {
          const long long t0 = clock64();
          while (*n_done + 8 <= k && ok) {
            if (*abort_flag) ok = false;
            else if (clock64() - t0 > wlim) { *abort_flag = 1; atomicExch(p.status, 15); ok = false; }
          }
        }
        int u = ok ? u_ahead : -1;
        if (u >= n_units) u = -1;
        if (u >= 0) u_ahead = atomicAdd(p.counters, 1);
        unit_list[k & 15] = u;
        __threadfence_block();
        *n_pub = k + 1;
        n_listed = k + 1;
        if (u < 0) { ended = true; break; }
        const Unit x = unit_of(u);
        if (x.T > 0)
          for (int h = 0; h < H; ++h) tma_prefetch_l2(&tm.q, h * 64, 0, x.g * p.G, x.bi);
        for (int t = 0; t <= x.T && ok; ++t) {
          if (t == min(2, x.T) && x.T > 0) {
            // Q of this unit, behind its first tiles: the buffer is free once the last S^T of the previous unit is done
            if (qn > 0 && !wait_bar(BAR(Q_EMPTY), (uint32_t)(qn - 1) & 1u, abort_flag, p.status, 11, wlim)) { ok = false; break; }
            mbar_expect_tx(BAR(Q_FULL), (uint32_t)(H * N * 128));
            for (int h = 0; h < H; ++h) tma_load_4d(smem_u32(q_s + h * NP * 128), &tm.q, BAR(Q_FULL), h * 64, 0, x.g * p.G, x.bi);
            ++qn;
          }
          if (t == x.T) break;
          const int s = G % NS;
          const uint32_t ph = (uint32_t)((G / NS) - 1) & 1u;
          const int gi0 = GPT * t, ng = min(GPT, x.ge - gi0);
          const bool whole = 4 * ng >= 3 * GPT && gi0 + ng <= x.g1;   // (nearly) full tile of source 1: one box per 64-column half
          uint32_t bytes = 0;
          if (whole) bytes = (uint32_t)KV_BYTES;
          else for (int j = 0; j < ng; ++j) bytes += (uint32_t)(H * 128 * (gi0 + j < x.g1 ? 32 : kp.gr2));
          const uint32_t kdst = smem_u32(ring + (size_t)s * SLOT), vdst = kdst + KV_BYTES;
          for (int kv = 0; kv < 2; ++kv) {
            const int full = kv == 0 ? FULL_K : FULL_V, empty = kv == 0 ? EMPTY_K : EMPTY_V;
            if (G >= NS && !wait_bar(BAR(empty + s), ph, abort_flag, p.status, 1 + kv, wlim)) { ok = false; break; }
            mbar_expect_tx(BAR(full + s), bytes);
            if (whole) {
              for (int h = 0; h < H; ++h)
                tma_load_4d((kv == 0 ? kdst : vdst) + (uint32_t)(h * HALF), kv == 0 ? &tm.k1t : &tm.v1t, BAR(full + s), h * 64, gi0 * 32, x.g, x.bi);
            } else {
              for (int j = 0; j < ng; ++j) {
                const Group gr = group_of(gi0 + j, x.g1, x.n1, n2);
                const CUtensorMap* m = kv == 0 ? (gr.src1 ? &tm.k1 : &tm.k2) : (gr.src1 ? &tm.v1 : &tm.v2);
                for (int h = 0; h < H; ++h)
                  tma_load_4d((kv == 0 ? kdst : vdst) + (uint32_t)(h * HALF + j * 4096), m, BAR(full + s), h * 64, gr.row0, x.g, x.bi);
              }
            }
            if (kv == 0) k_issued = G + 1; else ++G;
          }
        }
      }
      if (!ended) {                      // a wait gave up: tell the other warps that no unit follows
        unit_list[n_listed & 15] = -1;
        __threadfence_block();
        *n_pub = n_listed + 1;
      }
      if (*abort_flag) {
        // let the copies that were issued land before the CTA retires
        for (int j = max(k_issued - NS, 0); j < k_issued; ++j) drain_bar(BAR(FULL_K + j % NS), (uint32_t)(j / NS) & 1u);
        for (int j = max(G - NS, 0); j < G; ++j) drain_bar(BAR(FULL_V + j % NS), (uint32_t)(j / NS) & 1u);
        if (qn > 0) drain_bar(BAR(Q_FULL), (uint32_t)(qn - 1) & 1u);
      }
    }
  } else if (warp == 1) {
    // ======================================= MMA issuer =======================================
    if (lane == 0) {
      const uint32_t idesc_s = kt_idesc(NP, false, false);
      const uint32_t idesc_pv = kt_idesc(NP, true, true);
      const uint32_t qsm = smem_u32(q_s), ring_a = smem_u32(ring), p_a = smem_u32(p_s);
      int G = 0, qn = 0;
      bool ok = true;
      // the tile whose PV comes next: its index in the CTA's sequence, its groups, whether it starts its warpgroup's accumulator
      int pv_G = -1, pv_ng = 0; bool pv_first = false;
      auto issue_pv = [&]() -> bool {
        const int j = pv_G, pb = j & 1, s = j % NS;
        if (!wait_bar(BAR(P_FULL + pb), (uint32_t)(j >> 1) & 1u, abort_flag, p.status, 4, wlim)) return false;
        if (!wait_bar(BAR(FULL_V + s), (uint32_t)(j / NS) & 1u, abort_flag, p.status, 5, wlim)) return false;
        tc_fence_after();
        const uint32_t vsm = ring_a + (uint32_t)s * SLOT + KV_BYTES;
        const uint32_t psm = p_a + (pb ? (uint32_t)PBUF : 0u);
        // O^T_w += V^T P^T, 16 keys per instruction. A: the V tile read MN-major (its two 64-element halves lie HALF bytes
        // apart; with D = 64 both halves alias the same data and rows 64..127 of O^T are duplicates nobody reads).
        // B: P^T, MN-major, 64-byte rows, 8 keys per swizzle atom.
        for (int ks = 0; ks < 2 * pv_ng; ++ks)
          mma_ss(tmem_base + O_COL + (uint32_t)pb * NP, smem_desc(vsm + ks * 2048, H == 2 ? (uint32_t)HALF : 0u, 1024u),
                 smem_desc_sw64(psm + ks * 1024, (uint32_t)PBUF, 512u), idesc_pv, (!pv_first || ks > 0) ? 1u : 0u);
        tc_commit(BAR(PV_DONE + pb));
        tc_commit(BAR(EMPTY_V + s));
        return true;
      };
      for (int k = 0; ok; ++k) {
        const int u = unit_at(k);
        if (u < 0) break;
        const Unit x = unit_of(u);
        if (x.T == 0) continue;
        if (!wait_bar(BAR(Q_FULL), (uint32_t)qn & 1u, abort_flag, p.status, 3, wlim)) { ok = false; break; }
        ++qn;
        for (int t = 0; t < x.T && ok; ++t, ++G) {
          const int s = G % NS, sb = G & 1;
          if (!wait_bar(BAR(FULL_K + s), (uint32_t)(G / NS) & 1u, abort_flag, p.status, 7, wlim)) { ok = false; break; }
          tc_fence_after();
          const uint32_t ksm = ring_a + (uint32_t)s * SLOT;
          const uint32_t d_t = tmem_base + (uint32_t)sb * NP;
          // S^T = K_tile Q^T: the S^T buffer of tile G - 2 is free, its softmax arrived before PV(G - 2) was issued
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks) {
            const uint32_t hk = (ks >> 2) * HALF + (ks & 3) * 32;
            const uint32_t hq = (ks >> 2) * (NP * 128) + (ks & 3) * 32;
            mma_ss(d_t, smem_desc(ksm + hk, 16u, 1024u), smem_desc(qsm + hq, 16u, 1024u), idesc_s, ks > 0 ? 1u : 0u);
          }
          tc_commit(BAR(S_FULL + sb));
          tc_commit(BAR(EMPTY_K + s));
          if (t == x.T - 1) tc_commit(BAR(Q_EMPTY));   // the unit's last use of Q
          if (pv_G >= 0 && !issue_pv()) { ok = false; break; }
          pv_G = G; pv_ng = min(GPT, x.ge - GPT * t); pv_first = t < 2;
        }
      }
      if (ok && pv_G >= 0) ok = issue_pv();
      if (*abort_flag) {                 // wait for the tensor pipe to finish what was issued before TMEM is freed
        tc_commit(BAR(DRAIN));
        drain_bar(BAR(DRAIN), 0);
      }
    }
  } else {
    // ======================================= softmax warps =======================================
    // Warpgroup w takes the tiles of even (w = 0) or odd (w = 1) index in the CTA's sequence, so it alone ever waits on
    // the barriers of S^T buffer w, P^T buffer w and accumulator w, one phase per tile. A warp whose wait gave up (`dead`)
    // keeps walking tiles and units without touching data, so that all named barriers below are met.
    const int w = grp;
    const int q4 = warp & 3;                           // TMEM lane quadrant this warp may access = its group of 32 keys of a tile
    const int wq = (warp - 2) & 3;                     // index of the warp inside its warpgroup
    const int row = q4 * 32 + lane;                    // key row of a tile; head dimension of O^T at the end of a unit
    const uint32_t lane_addr = tmem_base + ((uint32_t)(q4 * 32) << 16);
    const float sl2 = p.scale_log2;
    const bool scores = p.want_scores != 0;
    const bool do_attn = p.out != nullptr;
    const int st = (tid - 64) & 127;                   // index inside the warpgroup
    const uint32_t o_col = O_COL + (uint32_t)w * NP;
    const int n_mine = min(N, NP);
    unsigned char* p_mine = p_s + (w ? PBUF : 0);
    const float* post_other = reinterpret_cast<const float*>(smem + KT_CTRL0 + KT_GRP + 1536);   // what warpgroup 1 posts
    bool dead = false;
    bool owe_sync = false;                             // warpgroup 1: warpgroup 0 has not yet confirmed the previous unit
    int Gbase = 0;                                     // tiles of the units walked so far
    for (int k = 0;; ++k) {                            // units walked so far
      const int u = __shfl_sync(0xffffffffu, unit_at(k), 0);       // (one answer per warp; all warps read the same list)
      if (u < 0) break;
      const Unit x = unit_of(u);
      const int bi = x.bi, g = x.g;
      float l_lane = 0.f;                              // sum over this warp's key rows of column `lane`
      const int t0 = ((Gbase & 1) == w) ? 0 : 1;       // this warpgroup's first tile of the unit
      int G_last = -1;
      for (int t = t0; t < x.T; t += 2) {
        const int G = Gbase + t;                       // (G & 1) == w
        G_last = G;
        const uint32_t par = (uint32_t)(G >> 1) & 1u;
        const int gi0 = GPT * t, ng = min(GPT, x.ge - gi0);
        const bool active = q4 < ng;                   // warp-uniform: this warp's group exists in the tile
        Group gr{1, 0, 0};
        if (active) gr = group_of(gi0 + q4, x.g1, x.n1, n2);
        const bool valid = lane < gr.nv;
        if (!dead && !wait_bar_warp(BAR(S_FULL + w), par, abort_flag, p.status, 9, wlim)) dead = true;
        tc_fence_after();
        const bool work = active && !dead;
        float sv[NP];
        if (work) {
          tmem_ld32(lane_addr + (uint32_t)w * NP, *reinterpret_cast<uint32_t(*)[32]>(&sv[0]));
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
          const float a = (a4[0] + a4[1]) + (a4[2] + a4[3]);
          if (work && valid && gr.src1)
            p.raw_scores[(int64_t)(bi * p.Hkv + g) * p.n1_max + gr.row0 + lane] = a * (p.scale / (float)N);
        }
        // ---- the references: the first key of the warpgroup's first tile of the unit lends its logits ----
        if (t == t0) {
          if (row == 0 && work) {
#pragma unroll
            for (int c = 0; c < NP; c += 4)
              *reinterpret_cast<float4*>(m_ref + c) = make_float4(sv[c] * sl2, sv[c + 1] * sl2, sv[c + 2] * sl2, sv[c + 3] * sl2);
          }
          softmax_barrier(bar_id);
        }
        float far0 = -INFINITY, far1 = -INFINITY;      // the largest distance above a reference
#pragma unroll
        for (int c = 0; c < NP; c += 4) {
          const float4 m4 = *reinterpret_cast<const float4*>(m_ref + c);
          sv[c] = fmaf(sv[c], sl2, -m4.x); sv[c + 1] = fmaf(sv[c + 1], sl2, -m4.y);
          sv[c + 2] = fmaf(sv[c + 2], sl2, -m4.z); sv[c + 3] = fmaf(sv[c + 3], sl2, -m4.w);
          far0 = fmaxf(far0, fmaxf(sv[c], sv[c + 1])); far1 = fmaxf(far1, fmaxf(sv[c + 2], sv[c + 3]));
        }
        const bool over = fmaxf(far0, far1) > 64.f;
        if (softmax_barrier_or(bar_id, over && work && valid)) {
          // ---- raise the references by the tile's column maxima (where positive) and rescale what has been accumulated:
          //      the warpgroup's previous PV of this unit must have landed before O^T_w is rewritten ----
          if (t > t0 && !dead && !wait_bar_warp(BAR(PV_DONE + w), (uint32_t)((G - 2) >> 1) & 1u, abort_flag, p.status, 8, wlim)) dead = true;
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
            const float dlt = ord2f(enc[st]);          // >= 0
            delta_s[st] = dlt;
            m_ref[st] += dlt;
          }
          softmax_barrier(bar_id);
#pragma unroll
          for (int c = 0; c < NP; ++c) sv[c] -= delta_s[c];
          l_lane *= fast_exp2(-delta_s[lane]);
          if (t > t0 && !dead) {
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
          softmax_barrier(bar_id);       // delta_s and m_ref are stable again before the next tile reads them
        }
        // ---- P^T = exp2(distance to the reference) as bf16, one 64-byte row per key (64-byte swizzle); the buffer is
        //      free once the PV of the warpgroup's previous tile (this unit's or the one before) has completed ----
        if (!dead && G >= 2 && !wait_bar_warp(BAR(PV_DONE + w), (uint32_t)((G - 2) >> 1) & 1u, abort_flag, p.status, 6, wlim)) dead = true;
        if (active && !dead) {
          unsigned char* prow = p_mine + row * 64;
          const int swz = (row >> 1) & 3;
          if (gr.nv < 32) {                            // ragged group (warp-uniform): rows past the count contribute nothing
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
            *reinterpret_cast<uint4*>(prow + ((c8 ^ swz) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
          }
          // ---- V rows of this group past its count may hold anything: zero them so that 0 * V stays 0 ----
          if (gr.nv < 32) {
            const int s = G % NS;
            if (!wait_bar_warp(BAR(FULL_V + s), (uint32_t)(G / NS) & 1u, abort_flag, p.status, 10, wlim)) dead = true;
            unsigned char* vs = ring + (size_t)s * SLOT + KV_BYTES;
            const int nz = dead ? 0 : (32 - gr.nv) * H * 8;          // 16-byte chunks to clear
            for (int i = lane; i < nz; i += 32) {
              const int rr = q4 * 32 + gr.nv + i / (H * 8), c = i % (H * 8);
              *reinterpret_cast<uint4*>(vs + (c >> 3) * HALF + rr * 128 + (((c & 7) ^ (rr & 7)) << 4)) = make_uint4(0u, 0u, 0u, 0u);
            }
          }
          fence_proxy_async();
        }
        // Warpgroup 1's first PV of a unit overwrites accumulator 1, which warpgroup 0 reads at the end of the unit
        // before: it must have confirmed that (this is the first arrive of warpgroup 1 since then).
        if (owe_sync) { pair_sync(6); owe_sync = false; }
        tc_fence_before();
        __syncwarp();
        if (lane == 0 && !dead) mbar_arrive(BAR(P_FULL + w));
        // ---- column sums, off the critical path: shuffle transpose over the warp's 32 key rows ----
        if (active && !dead) {
#pragma unroll
          for (int off = 16; off >= 1; off >>= 1) {
            const bool up_half = (lane & off) != 0;
#pragma unroll
            for (int kk = 0; kk < off; ++kk) {
              const float send = up_half ? sv[kk] : sv[kk + off];
              const float keep = up_half ? sv[kk + off] : sv[kk];
              sv[kk] = keep + __shfl_xor_sync(0xffffffffu, send, off);
            }
          }
          l_lane += sv[0];
        }
      }

      // ======================================= end of the unit =======================================
      // ---- refresh step: pooling of the head's saliency, once both warpgroups' raw values are in L2 ----
      if (scores) {
        __threadfence_block();                         // writers and readers of the unit's raw saliency are this CTA's threads
        asm volatile("bar.sync 5, 256;\n" ::: "memory");
        if (p.pooled != nullptr && !*abort_flag) {
          const float* a = p.raw_scores + (int64_t)(bi * p.Hkv + g) * p.n1_max;
          const int o = p.block_off[bi];
          kt_pool_span(p, a, p.pooled + (int64_t)(bi * p.Hkv + g) * p.n1_max, x.n1, o, 0, p.n1_max, tid - 64, 256);
        }
      }
      // ---- this warpgroup's sums of the 32 columns ----
      l_w[wq * 32 + lane] = l_lane;
      softmax_barrier(bar_id);
      float l_mine = 0.f, m_mine = -INFINITY;          // st < 32: sum and reference of column st
      if (st < NP) {
        l_mine = (l_w[st] + l_w[32 + st]) + (l_w[64 + st] + l_w[96 + st]);
        m_mine = G_last >= 0 ? m_ref[st] : -INFINITY;
      }
      if (w == 1) {
        // post them for warpgroup 0 and go on (warpgroup 0 has confirmed the unit before this one, so the slot of the
        // unit before that one, which this post overwrites, is no longer read)
        if (owe_sync) { pair_sync(6); owe_sync = false; }
        if (st < NP) { post[(k & 1) * 64 + st] = m_mine; post[(k & 1) * 64 + 32 + st] = l_mine; }
        __threadfence_block();
        pair_arrive(7);
        owe_sync = true;
        softmax_barrier(bar_id);                       // the references and per-warp sums are read: the next unit may overwrite them
      } else {
        pair_sync(7);                                  // warpgroup 1 has posted this unit's references and sums
        if (st < NP) {
          const float mb = post_other[(k & 1) * 64 + st], lb = post_other[(k & 1) * 64 + 32 + st];
          const bool ha = l_mine > 0.f, hb = lb > 0.f;
          const float ms = fmaxf(ha ? m_mine : -INFINITY, hb ? mb : -INFINITY);
          const float fa = ha ? fast_exp2(m_mine - ms) : 0.f, fb = hb ? fast_exp2(mb - ms) : 0.f;
          const float l = l_mine * fa + lb * fb;
          const float inv = l > 0.f ? 1.f / l : 0.f;
          l_tot[st] = fa * inv;
          w_other[st] = fb * inv;
          if (p.lse && st < N && !*abort_flag) {
            const int hg = st / p.b, i = st - hg * p.b;
            p.lse[((int64_t)bi * p.Hq + g * p.G + hg) * p.b + i] = (ms + log2f(l)) * kLn2;
          }
        }
        // ---- both accumulators, once the last PV of either warpgroup has landed ----
        const int G_end = Gbase + x.T - 1;             // the unit's last tile
        const int G_other = x.T >= 1 ? (((G_end & 1) == 1) ? G_end : (x.T >= 2 ? G_end - 1 : -1)) : -1;   // warpgroup 1's last tile of the unit
        const bool have0 = !dead && G_last >= 0 && wait_bar_warp(BAR(PV_DONE + 0), (uint32_t)(G_last >> 1) & 1u, abort_flag, p.status, 6, wlim);
        const bool have1 = !dead && G_other >= 0 && wait_bar_warp(BAR(PV_DONE + 1), (uint32_t)(G_other >> 1) & 1u, abort_flag, p.status, 6, wlim);
        tc_fence_after();
        uint32_t ov0[NP], ov1[NP];
        if (have0) tmem_ld32(lane_addr + O_COL, ov0);
        if (have1) tmem_ld32(lane_addr + O_COL + NP, ov1);
        tc_wait_ld();
        if (!have0) {
#pragma unroll
          for (int c = 0; c < NP; ++c) ov0[c] = 0u;
        }
        if (!have1) {
#pragma unroll
          for (int c = 0; c < NP; ++c) ov1[c] = 0u;
        }
        tc_fence_before();
        pair_arrive(6);                                // accumulator 1 and the posted values are no longer needed
        softmax_barrier(bar_id);                       // the weights are visible
        if (do_attn && !*abort_flag && row < D) {
          // normalise, fold and store; a warp writes 32 consecutive bf16 of one output row per column. Column c is row
          // c % b of head c / b of the group: the pointer walks the rows and hops to the next head.
          int i = 0;
          __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(p.out) + (int64_t)bi * p.o_stride[0] + (int64_t)(g * p.G) * p.o_stride[1] + row;
          const int64_t hop = p.o_stride[1] - (int64_t)(p.b - 1) * p.o_stride[2];
#pragma unroll
          for (int c = 0; c < NP; c += 4) {
            if (c >= N) break;
            const float4 wa = *reinterpret_cast<const float4*>(l_tot + c), wb = *reinterpret_cast<const float4*>(w_other + c);
            const float av[4] = {wa.x, wa.y, wa.z, wa.w}, bv[4] = {wb.x, wb.y, wb.z, wb.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              *o = __float2bfloat16_rn(fmaf(__uint_as_float(ov0[c + q]), av[q], __uint_as_float(ov1[c + q]) * bv[q]));
              if (++i == p.b) { i = 0; o += hop; } else o += p.o_stride[2];
            }
          }
        }
        // (the next writes of the weights, references and per-warp sums all lie behind the barriers above or behind the
        // next unit's barrier in front of its sums)
        if (st == 0) *n_done = k + 1;
      }
      Gbase += x.T;
    }
    if (owe_sync) pair_sync(6);                        // warpgroup 0's last confirmation
  }

  // ---- free the tensor memory ----
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
  // The last CTA to get here puts both counters back to zero for the next call: by then every CTA has taken its last
  // unit (the next kernel in the stream reads the counter only behind its grid dependency, i.e. after this grid).
  if (tid == 0 && atomicAdd(p.counters + 1, 1) == (int)gridDim.x - 1) {
    p.counters[0] = 0;
    p.counters[1] = 0;
  }
}

template <int D>
cudaError_t launch_kt_stream_d(const KtMaps& tm, const KtParams& kp, size_t smem_bytes, bool pdl, cudaStream_t st) {
  auto kern = attn_kt_stream_kernel<D>;
  static SmemConfig configured;
  cudaError_t e = configure_smem(reinterpret_cast<const void*>(kern), smem_bytes, configured, true);
  if (e != cudaSuccess) return e;
  const long long units = (long long)kp.a.B * kp.a.Hkv;
  long long ctas = sm_count();           // one resident CTA per SM (Tuning::persist >= 2 caps their number)
  const int cap = tuning().persist;
  if (cap >= 2 && cap < ctas) ctas = cap;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)(units < ctas ? units : ctas));
  cfg.blockDim = dim3(KS_THREADS);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  int na = 0;
  if (pdl) {
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  cfg.attrs = attr; cfg.numAttrs = na;
  return cudaLaunchKernelEx(&cfg, kern, tm, kp);
}

}  // namespace

size_t kt_stream_smem_bytes(int D) {
  const size_t H = D / 64;
  return 1024 /*alignment slack*/ + KS_CTRL + H * 32 * 128 + 2 * 128 * 64 + (size_t)KS_NS * 2 * H * 128 * 128;
}

cudaError_t launch_kt_stream(const KtMaps& tm, const KtParams& kp, int D, size_t smem_bytes, bool pdl, cudaStream_t st) {
  return D == 128 ? launch_kt_stream_d<128>(tm, kp, smem_bytes, pdl, st) : launch_kt_stream_d<64>(tm, kp, smem_bytes, pdl, st);
}

}  // namespace sdllm
