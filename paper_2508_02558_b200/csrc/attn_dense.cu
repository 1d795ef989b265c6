// Full-sequence bf16 attention on tcgen05 (the dense step: every row of a sequence over all of its keys).
//
// A dense contraction, bound by the tensor pipe and, in front of it, by the softmax. One CTA owns TWO 128-row query
// tiles of one query head and streams the head's K/V once for both:
//   warp 0      TMA producer: the two Q tiles, then K and V tiles (128 keys, 128-byte swizzle) into a two-slot ring
//   warp 1      one thread issues tcgen05.mma. Per key tile j:  S0 = Q0 K_j^T,  O1 += P1(j-1) V_(j-1),  S1 = Q1 K_j^T,
//               O0 += P0(j) V_j  -  while the softmax warps of one query tile work, the tensor pipe serves the other
//   warps 2-5   softmax of query tile 0, warps 6-9 of query tile 1: a thread owns one accumulator row (TMEM lane),
//               reads its S row, keeps the running max / sum and writes P (bf16) over S in TMEM; O accumulates in
//               TMEM and is rescaled in place only when the row's maximum grows by more than 2^8
// Tensor memory (512 columns): S0 | S1 | O0 | O1, 128 columns each (D = 64 uses half of an O region).
// The finished rows go from TMEM through registers straight to global memory (bf16), normalised by the row sum.
// Every wait on an mbarrier is bounded; on expiry the CTA sets an abort flag, records a code in the status word and
// runs to its end (freeing its TMEM); the outputs of that call are then invalid.
#include <cuda.h>
#include <string.h>

#include "attn_device.cuh"
#include "tuning.cuh"
#include "umma_host.cuh"

namespace sdllm {
using namespace dev;
namespace {

constexpr int DN_THREADS = 320;
constexpr int DN_STAGES = 2;

struct DenseMaps {
  CUtensorMap q, k, v;
};

struct DenseParams {
  const int32_t* seq_len;   // [B], nullable -> L
  void* out;                // [B, Hq, L, D] bf16 with o_stride
  float* lse;               // [B, Hq, L], nullable
  int32_t* status;          // device status word
  int B, Hq, G, L;
  float scale_log2;         // softmax scale * log2(e)
  int64_t o_stride[3];
  long long wait_cycles;    // limit of every abortable mbarrier wait
};

#include "umma_ptx.cuh"

template <int D>
__global__ void __launch_bounds__(DN_THREADS, 1) dense_attn_bf16_kernel(const __grid_constant__ DenseMaps tm, const DenseParams p) {
  extern __shared__ unsigned char smem_raw[];
  constexpr int H = D / 64;                 // 64-column halves of a row (128 bytes each: one swizzle atom wide)
  constexpr int KT = 128;                   // keys per tile
  constexpr int NS = DN_STAGES;
  constexpr int HALF = KT * 128;            // bytes of one 64-column half of a 128-row tile
  constexpr int TILE = H * HALF;            // bytes of a Q, K or V tile
  constexpr uint32_t S_COL0 = 0, O_COL0 = 256, T_STRIDE = 128;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int bi = blockIdx.z, h = blockIdx.y, g = h / p.G, jp = blockIdx.x;

  grid_dependency_wait();                   // everything this kernel reads may come from the kernel in front of it
  grid_launch_dependents();
  int n = p.seq_len ? p.seq_len[bi] : p.L;
  n = min(max(n, 0), p.L);
  const int row00 = 2 * jp * 128;           // first row of query tile 0; query tile 1 starts 128 rows further
  if (row00 >= n) return;                   // both query tiles lie past the sequence's end (whole CTA, before any set-up)
  const bool act1 = row00 + 128 < n;
  const int nt = (n + KT - 1) / KT;         // key tiles

  const uint32_t raw_addr = smem_u32(smem_raw);
  unsigned char* smem = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
  const uint32_t bars = smem_u32(smem);
  auto BAR = [&](int i) { return bars + 8u * (uint32_t)i; };
  const int Q_FULL = 0, FULL_K = 1, FULL_V = 1 + NS, EMPTY_K = 1 + 2 * NS, EMPTY_V = 1 + 3 * NS;
  const int S_FULL = 1 + 4 * NS, P_FULL = S_FULL + 2, PV_DONE = S_FULL + 4, DRAIN = S_FULL + 6;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + 256);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + 260);
  unsigned char* q_s = smem + 1024;
  unsigned char* stage0 = q_s + 2 * TILE;

  if (tid == 0) {
    prefetch_tmap(&tm.q); prefetch_tmap(&tm.k); prefetch_tmap(&tm.v);
    mbar_init(BAR(Q_FULL), 1);
    for (int i = 0; i < NS; ++i) {
      mbar_init(BAR(FULL_K + i), 1); mbar_init(BAR(FULL_V + i), 1);
      mbar_init(BAR(EMPTY_K + i), 1); mbar_init(BAR(EMPTY_V + i), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(BAR(S_FULL + i), 1);
      mbar_init(BAR(P_FULL + i), 4);       // the four softmax warps of a query tile
      mbar_init(BAR(PV_DONE + i), 1);
    }
    mbar_init(BAR(DRAIN), 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if (warp == 1) {                          // the MMA warp owns the tensor memory
    tmem_alloc(smem_u32(tmem_slot), 512);
    tmem_relinquish();
  }
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  auto tile_nv = [&](int j) { return min(n - j * KT, KT); };     // valid keys of tile j (> 0 for j < nt)

  if (warp == 0) {
    // ======================================= TMA producer =======================================
    if (lane == 0) {
      mbar_expect_tx(BAR(Q_FULL), (uint32_t)((act1 ? 2 : 1) * TILE));
      for (int t = 0; t < (act1 ? 2 : 1); ++t)
        for (int hh = 0; hh < H; ++hh)
          tma_load_4d(smem_u32(q_s + t * TILE + hh * HALF), &tm.q, BAR(Q_FULL), hh * 64, row00 + t * 128, h, bi);
      int issued = 0;
      bool ok = true;
      for (int j = 0; j < nt && ok; ++j) {
        const int s = j % NS;
        const uint32_t ph = ((j / NS) - 1) & 1;
        const uint32_t kdst = smem_u32(stage0 + (size_t)s * 2 * TILE), vdst = kdst + TILE;
        if (j >= NS && !wait_bar(BAR(EMPTY_K + s), ph, abort_flag, p.status, 21, p.wait_cycles)) { ok = false; break; }
        mbar_expect_tx(BAR(FULL_K + s), (uint32_t)TILE);
        for (int hh = 0; hh < H; ++hh) tma_load_4d(kdst + hh * HALF, &tm.k, BAR(FULL_K + s), hh * 64, j * KT, g, bi);
        if (j >= NS && !wait_bar(BAR(EMPTY_V + s), ph, abort_flag, p.status, 22, p.wait_cycles)) {
          drain_bar(BAR(FULL_K + s), (j / NS) & 1);                 // the K half of this slot is already on its way
          ok = false; break;
        }
        mbar_expect_tx(BAR(FULL_V + s), (uint32_t)TILE);
        for (int hh = 0; hh < H; ++hh) tma_load_4d(vdst + hh * HALF, &tm.v, BAR(FULL_V + s), hh * 64, j * KT, g, bi);
        issued = j + 1;
      }
      if (*abort_flag) {                    // let the copies that were issued land before the CTA retires
        for (int j = max(issued - NS, 0); j < issued; ++j) {
          drain_bar(BAR(FULL_K + j % NS), (j / NS) & 1);
          drain_bar(BAR(FULL_V + j % NS), (j / NS) & 1);
        }
        drain_bar(BAR(Q_FULL), 0);
      }
    }
  } else if (warp == 1) {
    // ======================================= MMA issuer =======================================
    if (lane == 0) {
      const uint32_t idesc_pv = instr_desc(D, true);
      const uint32_t qsm = smem_u32(q_s);
      bool ok = wait_bar(BAR(Q_FULL), 0, abort_flag, p.status, 23, p.wait_cycles);
      // S_t = Q_t K_j^T into the S region of query tile t
      auto issue_s = [&](int t, int j) {
        const uint32_t ksm = smem_u32(stage0 + (size_t)(j % NS) * 2 * TILE);
        const uint32_t idesc_s = instr_desc((tile_nv(j) + 15) & ~15, false);
        const uint32_t d_t = tmem_base + S_COL0 + (uint32_t)t * T_STRIDE;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint32_t off = (ks >> 2) * HALF + (ks & 3) * 32;
          mma_ss(d_t, smem_desc(qsm + t * TILE + off, 16u, 1024u), smem_desc(ksm + off, 16u, 1024u), idesc_s, ks > 0 ? 1u : 0u);
        }
        tc_commit(BAR(S_FULL + t));
      };
      // O_t += P_t V_j once the softmax warps of query tile t have written P_t; `release` frees the V slot afterwards
      auto issue_pv = [&](int t, int j, bool release) -> bool {
        const int s = j % NS;
        if (!wait_bar(BAR(P_FULL + t), j & 1, abort_flag, p.status, 24, p.wait_cycles)) return false;
        if (!wait_bar(BAR(FULL_V + s), (j / NS) & 1, abort_flag, p.status, 25, p.wait_cycles)) return false;
        tc_fence_after();
        const uint32_t vsm = smem_u32(stage0 + (size_t)s * 2 * TILE) + TILE;
        const uint32_t a_t = tmem_base + S_COL0 + (uint32_t)t * T_STRIDE;
        const int n_mma = (tile_nv(j) + 15) & ~15;
        for (int ks = 0; ks < n_mma / 16; ++ks)
          mma_ts(tmem_base + O_COL0 + (uint32_t)t * T_STRIDE, a_t + ks * 8, smem_desc(vsm + ks * 2048, (uint32_t)HALF, 1024u), idesc_pv,
                 (j > 0 || ks > 0) ? 1u : 0u);
        tc_commit(BAR(PV_DONE + t));
        if (release) tc_commit(BAR(EMPTY_V + s));
        return true;
      };
      for (int j = 0; j < nt && ok; ++j) {
        const int s = j % NS;
        if (!wait_bar(BAR(FULL_K + s), (j / NS) & 1, abort_flag, p.status, 26, p.wait_cycles)) { ok = false; break; }
        tc_fence_after();
        issue_s(0, j);
        if (act1) {
          if (j > 0 && !issue_pv(1, j - 1, true)) { ok = false; break; }
          issue_s(1, j);
        }
        tc_commit(BAR(EMPTY_K + s));
        if (!issue_pv(0, j, !act1)) { ok = false; break; }
      }
      if (ok && act1) ok = issue_pv(1, nt - 1, true);
      if (*abort_flag) {                    // wait for the tensor pipe to finish what was issued before TMEM is freed
        tc_commit(BAR(DRAIN));
        drain_bar(BAR(DRAIN), 0);
      }
    }
  } else {
    // ======================================= softmax warps =======================================
    const int t = (warp - 2) >> 2;                     // query tile of this warp
    const int q4 = warp & 3;                           // TMEM lane quadrant this warp may access
    const int row = q4 * 32 + lane;
    if (t == 0 || act1) {
      const uint32_t lane_addr = tmem_base + ((uint32_t)(q4 * 32) << 16);
      const uint32_t s_addr = lane_addr + S_COL0 + (uint32_t)t * T_STRIDE;
      const uint32_t o_addr = lane_addr + O_COL0 + (uint32_t)t * T_STRIDE;
      float m_run = -INFINITY, l_run = 0.f;
      bool ok = true;
      for (int j = 0; j < nt && ok; ++j) {
        const int nv = tile_nv(j);
        if (!wait_bar_warp(BAR(S_FULL + t), j & 1, abort_flag, p.status, 27, p.wait_cycles)) { ok = false; break; }
        tc_fence_after();
        uint32_t sv[4][32];
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_ld32(s_addr + c * 32, sv[c]);
        tc_wait_ld();
        if (nv < KT) {                                   // the ragged last tile: keys past the end count as -inf
#pragma unroll
          for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (c * 32 + i >= nv) sv[c][i] = __float_as_uint(-INFINITY);
        }
        float mx = -INFINITY;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int i = 0; i < 32; ++i) m4[i & 3] = fmaxf(m4[i & 3], __uint_as_float(sv[c][i]));
          mx = fmaxf(mx, fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3])));
        }
        // running maximum: O (in TMEM) and l are rescaled only when the maximum grows by more than 2^8
        const float m_new = fmaxf(m_run, mx * p.scale_log2);
        const bool grow = m_new > m_run + 8.f;          // also true on the first finite maximum
        float alpha = 1.f;
        if (grow) {
          alpha = fast_exp2(m_run - m_new);             // 0 when m_run is -inf
          m_run = m_new;
          l_run *= alpha;
        }
        if (j > 0 && __any_sync(0xffffffffu, grow)) {
          // every PV of this query tile issued so far must have landed before its rows are rewritten
          if (!wait_bar_warp(BAR(PV_DONE + t), (j - 1) & 1, abort_flag, p.status, 28, p.wait_cycles)) { ok = false; break; }
          tc_fence_after();
#pragma unroll 1
          for (int c = 0; c < D / 16; ++c) {
            uint32_t ov[16];
            tmem_ld16(o_addr + c * 16, ov);
            tc_wait_ld();
#pragma unroll
            for (int i = 0; i < 16; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * alpha);
            tmem_st16(o_addr + c * 16, ov);
          }
        }
        const float mu = (m_run == -INFINITY) ? 0.f : m_run;
        // P = exp2(S * scale_log2 - mu) as bf16 over the first 64 columns of the S region
        float psum = 0.f;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
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
        l_run += psum;
        // V rows past the sequence's end may hold anything: query tile 0 zeroes them so that 0 * V stays 0
        const int n_mma = (nv + 15) & ~15;
        if (t == 0 && nv < n_mma) {
          const int s = j % NS;
          if (!wait_bar_warp(BAR(FULL_V + s), (j / NS) & 1, abort_flag, p.status, 29, p.wait_cycles)) { ok = false; break; }
          unsigned char* vs = stage0 + (size_t)s * 2 * TILE + TILE;
          const int nz = (n_mma - nv) * H * 8;           // 16-byte chunks to clear
          for (int i = (warp - 2) * 32 + lane; i < nz; i += 128) {
            const int rr = nv + i / (H * 8), c = i % (H * 8);
            *reinterpret_cast<uint4*>(vs + (c >> 3) * HALF + rr * 128 + (((c & 7) ^ (rr & 7)) << 4)) = make_uint4(0u, 0u, 0u, 0u);
          }
          fence_proxy_async();
        }
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(BAR(P_FULL + t));
      }
      // ---- the finished row: TMEM -> registers -> normalise -> bf16 -> global memory ----
      if (ok) ok = wait_bar_warp(BAR(PV_DONE + t), (nt - 1) & 1, abort_flag, p.status, 30, p.wait_cycles);
      tc_fence_after();
      const int r_glob = row00 + t * 128 + row;
      if (ok) {
        const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
        __nv_bfloat16* orow = reinterpret_cast<__nv_bfloat16*>(p.out) + (int64_t)bi * p.o_stride[0] + (int64_t)h * p.o_stride[1] +
                              (int64_t)r_glob * p.o_stride[2];
#pragma unroll 1
        for (int c = 0; c < D / 32; ++c) {
          uint32_t ov[32];
          tmem_ld32(o_addr + c * 32, ov);               // warp-wide: every lane takes part, valid row or not
          tc_wait_ld();
          if (r_glob < n) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              uint4 w4;
              w4.x = pack_bf16(__uint_as_float(ov[8 * i]) * inv, __uint_as_float(ov[8 * i + 1]) * inv);
              w4.y = pack_bf16(__uint_as_float(ov[8 * i + 2]) * inv, __uint_as_float(ov[8 * i + 3]) * inv);
              w4.z = pack_bf16(__uint_as_float(ov[8 * i + 4]) * inv, __uint_as_float(ov[8 * i + 5]) * inv);
              w4.w = pack_bf16(__uint_as_float(ov[8 * i + 6]) * inv, __uint_as_float(ov[8 * i + 7]) * inv);
              *reinterpret_cast<uint4*>(orow + c * 32 + i * 8) = w4;
            }
          }
        }
        if (r_glob < n && p.lse) p.lse[((int64_t)bi * p.Hq + h) * p.L + r_glob] = (m_run + log2f(l_run)) * kLn2;
      }
    }
  }

  // ---- teardown ----
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

size_t dense_smem_bytes(int D) {
  const size_t tile = (size_t)(D / 64) * 128 * 128;
  return 1024 /*alignment slack*/ + 1024 /*barriers*/ + 2 * tile + (size_t)DN_STAGES * 2 * tile;
}

template <int D>
cudaError_t launch_dense_d(const DenseMaps& tm, const DenseParams& p, int nqb, cudaStream_t st) {
  auto kern = dense_attn_bf16_kernel<D>;
  static SmemConfig configured;
  const size_t smem = dense_smem_bytes(D);
  const cudaError_t ce = configure_smem(reinterpret_cast<const void*>(kern), smem, configured, true);
  if (ce != cudaSuccess) return ce;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((nqb + 1) / 2, p.Hq, p.B);
  cfg.blockDim = dim3(DN_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  int na = 0;
  if (tuning().pdl != 0) {
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  cfg.attrs = attr; cfg.numAttrs = na;
  return cudaLaunchKernelEx(&cfg, kern, tm, p);
}

}  // namespace

cudaError_t launch_dense_pair(const void* q, const int64_t* q_stride, const void* k, const void* v, const int64_t* kv_stride,
                              const int32_t* seq_len, void* out, const int64_t* o_stride, float* lse, int32_t* status, int B, int Hq,
                              int Hkv, int L, int D, float scale, cudaStream_t st) {
  if (Hq > 65535 || B > 65535) return cudaErrorInvalidValue;
  DenseMaps tm;
  memset(&tm, 0, sizeof(tm));
  bool ok = umma_make_map(&tm.q, q, D, L, Hq, B, q_stride, 128, 1);
  ok = ok && umma_make_map(&tm.k, k, D, L, Hkv, B, kv_stride, 128, 1);
  ok = ok && umma_make_map(&tm.v, v, D, L, Hkv, B, kv_stride, 128, 1);
  if (!ok) return cudaErrorInvalidValue;
  DenseParams p{};
  p.seq_len = seq_len; p.out = out; p.lse = lse; p.status = status;
  p.B = B; p.Hq = Hq; p.G = Hq / Hkv; p.L = L;
  p.scale_log2 = scale * kLog2e;
  p.wait_cycles = tuning().wait_cycles;
  for (int i = 0; i < 3; ++i) p.o_stride[i] = o_stride[i];
  const int nqb = (L + 127) / 128;
  return D == 128 ? launch_dense_d<128>(tm, p, nqb, st) : launch_dense_d<64>(tm, p, nqb, st);
}

}  // namespace sdllm
