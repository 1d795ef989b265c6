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
//   warps 2-5   softmax: each thread owns one of the 128 accumulator rows (TMEM lane), reads S with tcgen05.ld,
//               keeps the running max / sum, writes P (bf16) over S in TMEM, and accumulates O in registers
//   warps 6-7   refresh only: mean-query saliency of every streamed key (Algorithm 1, "qbar <- Mean(Q_b)",
//               "A <- MatMul(qbar, K_f^T)") from the K tile in shared memory, fp32
// When b*G <= 64 the query rows are replicated R = 2 or 4 times along the 128 accumulator rows and every replica
// takes its own slice of each key tile, so all four softmax warps work; the replicas are merged like key splits.
// Key splits (and replicas) leave (max, sum, O) partials in the workspace; the last CTA of a (sequence, KV head,
// row tile) to finish - found with one atomic counter, nobody waits - merges them, writes the output and, at the
// refresh step, pools the head's saliency along the key axis (Algorithm 1, MaxPool1D).
//
// Every wait on an mbarrier is bounded. On expiry the thread sets an abort flag that all other waits poll, records a
// code in the status word and the CTA runs to its end (freeing its TMEM); the outputs of that call are then invalid.
#include <cuda.h>
#include <stdlib.h>
#include <string.h>

#include "attn_device.cuh"

namespace sdllm {
using namespace dev;
namespace {

constexpr int UM_THREADS = 256;
constexpr int UM_STAGES = 3;
constexpr long long kWaitCycles = 400000000LL;   // ~0.2 s

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
  int parts;         // partials per (sequence, KV head, row tile) = splits * R
};

// ---------------------------------------------------------------------------------------------------------
// PTX wrappers
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int x, int y, int z, int w) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];\n"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* tm) {
  asm volatile("prefetch.tensormap [%0];\n" ::"l"(tm) : "memory");
}
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}\n"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// 32 lanes x 32 consecutive 32-bit columns: thread i of the warp receives lane (base lane + i)
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};\n"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) : "memory");
}
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}

// Shared-memory matrix descriptor of tcgen05.mma: 128-byte swizzle, start address / leading / stride offsets in
// 16-byte units, descriptor version 1 in bits 46-47, swizzle mode 2 (128 B) in bits 61-63.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
// Instruction descriptor, kind::f16: fp32 accumulator, bf16 A and B, M = 128, N = n, A K-major, B K- or MN-major.
__device__ __forceinline__ uint32_t instr_desc(int n, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(n >> 3) << 17) | ((128u >> 4) << 24);
}

// Which tile (source, first row, valid rows, MMA width) a CTA-local ordinal refers to.
struct Tile {
  int src1;      // 1: source 1, 0: source 2
  int row0;      // first row inside its source
  int nv;        // valid rows (0: skip the tile)
  int n_mma;     // nv rounded up to 16
};
__device__ __forceinline__ Tile tile_of(int t, int tiles1, int KT, int KT2, int n1, int n2) {
  Tile x;
  if (t < tiles1) { x.src1 = 1; x.row0 = t * KT; x.nv = min(max(n1 - x.row0, 0), KT); }
  else { x.src1 = 0; x.row0 = (t - tiles1) * KT2; x.nv = min(max(n2 - x.row0, 0), KT2); }
  x.n_mma = (x.nv + 15) & ~15;
  return x;
}

// Bounded wait on an mbarrier phase. Returns false when the CTA is aborting (this wait or another one expired).
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status, int code) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > kWaitCycles) {
      *abort_flag = 1;
      atomicExch(status, code);
      return false;
    }
  }
}
// The same for a whole warp: every lane takes the same decision, so warp-synchronous instructions stay converged.
__device__ __forceinline__ bool wait_bar_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status, int code) {
  return __all_sync(0xffffffffu, wait_bar(bar, parity, abort_flag, status, code)) != 0;
}
// Bounded wait that ignores the abort flag (used while draining in-flight work on the way out).
__device__ __forceinline__ void drain_bar(uint32_t bar, uint32_t parity) {
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > kWaitCycles) return;
  }
}

template <int D>
__global__ void __launch_bounds__(UM_THREADS, 1) attn_umma_bf16_kernel(const __grid_constant__ UmmaMaps tm, const UmmaParams up) {
  constexpr int H = D / 64;            // 128-byte column halves of a row
  constexpr int NS = UM_STAGES;
  const AttnParams& p = up.a;
  extern __shared__ unsigned char smem_raw[];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int KT = up.KT, KT2 = up.KT2, R = up.R;
  const int rows_rep = 128 / R;
  const int bi = blockIdx.z;
  const int g = blockIdx.y / up.row_tiles, rt = blockIdx.y - g * up.row_tiles;
  const int split = blockIdx.x;
  const int tiles1 = (p.n1_max + KT - 1) / KT;
  const int tiles2 = (p.n2 + KT2 - 1) / KT2;
  const int tiles_all = tiles1 + tiles2;
  const int t_begin = (int)(((long long)split * tiles_all) / p.splits);
  const int t_end = (int)(((long long)(split + 1) * tiles_all) / p.splits);
  const int M_rt = min(p.M - rt * 128, 128);          // valid query rows of this row tile (<= rows_rep when R > 1)
  const bool do_attn = p.out != nullptr;
  const bool do_scores = p.want_scores && rt == 0;

  // ---- shared memory carve-up (1024-byte aligned for the 128-byte swizzle) ----
  const uint32_t raw_addr = smem_u32(smem_raw);
  unsigned char* smem = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
  const uint32_t bars = smem_u32(smem);
  auto BAR = [&](int i) { return bars + 8u * (uint32_t)i; };
  const int Q_FULL = 0, FULL_K = 1, FULL_V = 1 + NS, EMPTY_K = 1 + 2 * NS, EMPTY_V = 1 + 3 * NS;
  const int S_FULL = 1 + 4 * NS, P_FULL = S_FULL + 2, O_FULL = S_FULL + 4, O_FREE = S_FULL + 6, DRAIN = S_FULL + 8;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + 256);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + 260);
  int* last_flag = reinterpret_cast<int*>(smem + 264);
  float* qbar_s = reinterpret_cast<float*>(smem + 512);
  unsigned char* q_s = smem + 1024;
  unsigned char* stage0 = q_s + H * 128 * 128;
  const int half_bytes = KT * 128;                     // one 64-column half of a K or V tile
  const int kv_bytes = H * half_bytes;                 // a whole K (or V) tile
  const int stage_bytes = 2 * kv_bytes;

  if (tid == 0) {
    mbar_init(BAR(Q_FULL), 1);
    for (int s = 0; s < NS; ++s) {
      mbar_init(BAR(FULL_K + s), 1);
      mbar_init(BAR(FULL_V + s), 1);
      mbar_init(BAR(EMPTY_K + s), max((do_attn ? 1 : 0) + (do_scores ? 2 : 0), 1));
      mbar_init(BAR(EMPTY_V + s), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(BAR(S_FULL + i), 1);
      mbar_init(BAR(P_FULL + i), 4);
      mbar_init(BAR(O_FULL + i), 1);
      mbar_init(BAR(O_FREE + i), 4);
    }
    mbar_init(BAR(DRAIN), 1);
    *abort_flag = 0;
    *last_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  // Q rows that no TMA box covers must not hold non-finite garbage: clear the tile first
  if (do_attn)
    for (int i = tid; i < H * 128 * 128 / 16; i += UM_THREADS) reinterpret_cast<uint4*>(q_s)[i] = make_uint4(0u, 0u, 0u, 0u);
  if (warp == 0) {
    tmem_alloc(smem_u32(tmem_slot), 512);
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
  const int n2 = p.n2;

  // per-thread softmax state (softmax warps only)
  float o_reg[D];
  float m_run = -INFINITY, l_run = 0.f;

  if (warp == 0) {
    // ======================================= TMA producer =======================================
    if (lane == 0) {
      prefetch_tmap(&tm.k1); prefetch_tmap(&tm.v1);
      if (n2 > 0) { prefetch_tmap(&tm.k2); prefetch_tmap(&tm.v2); }
      if (do_attn) {
        prefetch_tmap(&tm.q);
        mbar_expect_tx(BAR(Q_FULL), (uint32_t)(R * H * p.b * up.heads_rt * 128));
        for (int rep = 0; rep < R; ++rep)
          for (int h = 0; h < H; ++h)
            tma_load_4d(smem_u32(q_s + h * 128 * 128 + rep * rows_rep * 128), &tm.q, BAR(Q_FULL), h * 64, 0,
                        g * p.G + rt * up.heads_rt, bi);
      }
      int it = 0;
      bool ok = true;
      for (int t = t_begin; t < t_end && ok && (do_attn || do_scores); ++t) {
        const Tile x = tile_of(t, tiles1, KT, KT2, n1, n2);
        if (x.nv == 0) continue;
        const int s = it % NS;
        const uint32_t ph = ((it / NS) - 1) & 1;
        const uint32_t kdst = smem_u32(stage0 + (size_t)s * stage_bytes), vdst = kdst + kv_bytes;
        const CUtensorMap* mk = x.src1 ? &tm.k1 : &tm.k2;
        const CUtensorMap* mv = x.src1 ? &tm.v1 : &tm.v2;
        const int box_rows = x.src1 ? KT : KT2;
        const uint32_t tile_tx = (uint32_t)(H * box_rows * 128);
        if (it >= NS && !wait_bar(BAR(EMPTY_K + s), ph, abort_flag, p.status, 1)) { ok = false; break; }
        mbar_expect_tx(BAR(FULL_K + s), tile_tx);
        for (int h = 0; h < H; ++h) tma_load_4d(kdst + h * half_bytes, mk, BAR(FULL_K + s), h * 64, x.row0, g, bi);
        if (do_attn) {
          if (it >= NS && !wait_bar(BAR(EMPTY_V + s), ph, abort_flag, p.status, 2)) { ok = false; break; }
          mbar_expect_tx(BAR(FULL_V + s), tile_tx);
          for (int h = 0; h < H; ++h) tma_load_4d(vdst + h * half_bytes, mv, BAR(FULL_V + s), h * 64, x.row0, g, bi);
        }
        ++it;
      }
      if (*abort_flag) {
        // let the copies that were issued land before the CTA retires
        for (int j = max(it - NS, 0); j < it; ++j) {
          drain_bar(BAR(FULL_K + j % NS), (j / NS) & 1);
          if (do_attn) drain_bar(BAR(FULL_V + j % NS), (j / NS) & 1);
        }
      }
    }
  } else if (warp == 1) {
    // ======================================= MMA issuer =======================================
    if (lane == 0 && do_attn) {
      const uint32_t idesc_pv = instr_desc(D, true);
      bool ok = wait_bar(BAR(Q_FULL), 0, abort_flag, p.status, 3);
      int it = 0;
      Tile prev{}; int prev_it = -1;
      auto issue_pv = [&](const Tile& x, int j) -> bool {
        const int s = j % NS, pb = j & 1;
        if (!wait_bar(BAR(P_FULL + pb), (j >> 1) & 1, abort_flag, p.status, 4)) return false;
        if (!wait_bar(BAR(FULL_V + s), (j / NS) & 1, abort_flag, p.status, 5)) return false;
        if (j >= 2 && !wait_bar(BAR(O_FREE + pb), ((j >> 1) - 1) & 1, abort_flag, p.status, 6)) return false;
        tc_fence_after();
        const uint32_t vsm = smem_u32(stage0 + (size_t)s * stage_bytes) + kv_bytes;
        const uint32_t d_t = tmem_base + 256u + (uint32_t)pb * 128u;
        const uint32_t a_t = tmem_base + (uint32_t)pb * 128u;
        for (int ks = 0; ks < x.n_mma / 16; ++ks)
          mma_ts(d_t, a_t + ks * 8, smem_desc(vsm + ks * 2048, (uint32_t)half_bytes, 1024u), idesc_pv, ks > 0 ? 1u : 0u);
        tc_commit(BAR(O_FULL + pb));
        tc_commit(BAR(EMPTY_V + s));
        return true;
      };
      for (int t = t_begin; t < t_end && ok; ++t) {
        const Tile x = tile_of(t, tiles1, KT, KT2, n1, n2);
        if (x.nv == 0) continue;
        const int s = it % NS, sb = it & 1;
        if (!wait_bar(BAR(FULL_K + s), (it / NS) & 1, abort_flag, p.status, 7)) { ok = false; break; }
        tc_fence_after();
        const uint32_t ksm = smem_u32(stage0 + (size_t)s * stage_bytes);
        const uint32_t qsm = smem_u32(q_s);
        const uint32_t idesc_s = instr_desc(x.n_mma, false);
        const uint32_t d_t = tmem_base + (uint32_t)sb * 128u;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint32_t hq = (ks >> 2) * (128 * 128) + (ks & 3) * 32;
          const uint32_t hk = (ks >> 2) * half_bytes + (ks & 3) * 32;
          mma_ss(d_t, smem_desc(qsm + hq, 16u, 1024u), smem_desc(ksm + hk, 16u, 1024u), idesc_s, ks > 0 ? 1u : 0u);
        }
        tc_commit(BAR(S_FULL + sb));
        tc_commit(BAR(EMPTY_K + s));
        if (prev_it >= 0 && !issue_pv(prev, prev_it)) { ok = false; break; }
        prev = x; prev_it = it;
        ++it;
      }
      if (ok && prev_it >= 0) ok = issue_pv(prev, prev_it);
      if (*abort_flag) {               // wait for the tensor pipe to finish what was issued before TMEM is freed
        tc_commit(BAR(DRAIN));
        drain_bar(BAR(DRAIN), 0);
      }
    }
  } else if (warp < 6) {
