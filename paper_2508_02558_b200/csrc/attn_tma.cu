// bf16 block-query attention for sm_100a: TMA-fed shared-memory ring, one producer warp, tensor-core consumers,
// and a merge of the key splits through distributed shared memory inside a thread-block cluster.
//
// One CTA owns (sequence, KV head, key split). The key axis is a fixed tile grid over
//   [source 1 padded to n1_max rows] ++ [source 2]
// (refresh: the full K/V; reuse: the compacted cache followed by the block's fresh rows, Algorithm 3
// "K <- Concat(K_c, K_n)"), so which tile a CTA loads never depends on a value read from device memory; rows at or
// beyond the sequence's own count are masked after the fact and whole tiles beyond it are skipped once the count is
// known. K and V tiles arrive through cp.async.bulk.tensor (128-byte swizzle) into a ring guarded by full/empty
// mbarriers; consumer warps run QK^T and PV with mma.sync m16n8k16 (fp32 accumulate) and an online softmax. The
// CTAs of a cluster then combine their (max, sum, O) partials by reading each other's shared memory, so for the
// common case no partial ever touches global memory and no second kernel runs.
// At the refresh step the same pass emits the mean-query saliency of every streamed key (Algorithm 1,
// "qbar <- Mean(Q_b)", "A <- MatMul(qbar, K_f^T)").
//
// Every wait on an mbarrier is bounded: on expiry the thread records a code in the status word, stops waiting and
// runs to the end (the output of that call is then invalid), so a protocol error cannot hang the device.
#include <cuda.h>
#include <stdlib.h>

#include "attn_device.cuh"

namespace sdllm {
using namespace dev;

size_t attn_legacy_smem_bytes(int dtype, int D, const AttnPlan& plan);
AttnPlan plan_attention_legacy(int dtype, int D, int M, int B, int Hkv, int n_keys_max);
cudaError_t launch_attn_legacy(const AttnParams& p, const AttnPlan& plan, int dtype, int D, cudaStream_t st);
bool umma_supported(int dtype, int D, int M, int b);
AttnPlan plan_attention_umma(int D, int M, int b, int B, int Hkv, int n1_max, int n2);
cudaError_t launch_attn_umma(const AttnParams& p, const AttnPlan& pl, int D, cudaStream_t st);

namespace {

struct TmaMaps {
  CUtensorMap q, k1, v1, k2, v2;
};

constexpr long long kWaitCycles = 400000000LL;   // ~0.2 s at 2 GHz

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
// Bounded wait. Returns false when the limit expired (the caller then stops waiting for good).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > kWaitCycles) return false;
  }
  return true;
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int x, int y, int z, int w) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];\n"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* tm) {
  asm volatile("prefetch.tensormap [%0];\n" ::"l"(tm) : "memory");
}
__device__ __forceinline__ void consumer_bar(int nthreads) { asm volatile("bar.sync 1, %0;\n" ::"r"(nthreads) : "memory"); }
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;\n" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;\n" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(r) : "r"(local_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ float4 ld_cluster_f4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];\n" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ float2 ld_cluster_f2(uint32_t addr) {
  float2 v;
  asm volatile("ld.shared::cluster.v2.f32 {%0,%1}, [%2];\n" : "=f"(v.x), "=f"(v.y) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }

// Which tiles of its range a CTA processes: the first STAGES ones always (their loads are issued before the
// sequence's key count is known), later ones only while they still hold valid source-1 rows or belong to source 2.
__device__ __forceinline__ bool tile_is_processed(int ordinal, int t, int tiles1, int key_tile, int n1, int uncond) {
  return ordinal < uncond || t >= tiles1 || t * key_tile < n1;
}

template <int D, int WK, int STAGES, int NT_MAX, bool QREG>
__global__ void __launch_bounds__(NT_MAX) attn_tma_bf16_kernel(const __grid_constant__ TmaMaps tm, const AttnParams p,
                                                                 const int m_warps, const int c_warps, const int cluster) {
  constexpr int H = D / 64;          // 128-byte column halves of a row
  constexpr int KS = D / 16;         // k-steps of QK^T
  constexpr int DN = D / 8;          // n-tiles of PV
  constexpr int NT = WK / 8;         // n-tiles of S per warp
  constexpr int KK = WK / 16;        // k-steps of PV per warp
  extern __shared__ unsigned char smem_raw[];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_cons = m_warps * c_warps;
  const int n_cons_threads = n_cons * 32;
  const bool is_producer = warp == n_cons;
  const int KT = c_warps * WK;
  const int Mpad = m_warps * 16;
  const int bi = blockIdx.z, g = blockIdx.y;
  const int tiles1 = (p.n1_max + KT - 1) / KT;
  const int tiles_all = tiles1 + (p.n2 + KT - 1) / KT;
  const int t_begin = (int)(((long long)blockIdx.x * tiles_all) / p.splits_total);
  const int t_end = (int)(((long long)(blockIdx.x + 1) * tiles_all) / p.splits_total);
  CtaRange r;                        // geometry for the shared store helpers
  r.bi = bi; r.g = g; r.split = blockIdx.x / cluster; r.t_begin = t_begin; r.t_end = t_end;

  // ---- shared memory carve-up (1024-byte aligned for the 128-byte swizzle) ----
  const uint32_t raw_addr = smem_u32(smem_raw);
  unsigned char* smem = smem_raw + (((raw_addr + 1023u) & ~1023u) - raw_addr);
  const uint32_t bars = smem_u32(smem);                 // full[STAGES], empty[STAGES], q_full
  float* qbar_s = reinterpret_cast<float*>(smem + 128);
  unsigned char* q_s = smem + 1024;
  unsigned char* stage0 = q_s + H * Mpad * 128;
  const int half_bytes = KT * 128;
  const int stage_bytes = 2 * H * half_bytes;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
  const uint32_t q_bar = bars + 8u * (2 * STAGES);

  if (tid == 0) {
#pragma unroll
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), n_cons); }
    mbar_init(q_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  __syncthreads();
  grid_dependency_wait();            // everything below may read what the previous kernel in the stream wrote
  grid_launch_dependents();

  bool dead = false;                 // set when a bounded wait expired
  float oacc[DN][4];
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  const int rw = warp / c_warps, cw = warp - rw * c_warps;
  const int r0 = rw * 16;
  const int g8 = lane >> 2, t4 = lane & 3;

  if (is_producer) {
    // =============================== producer warp: one lane issues every TMA load ===============================
    if (lane == 0) {
      prefetch_tmap(&tm.q); prefetch_tmap(&tm.k1); prefetch_tmap(&tm.v1);
      if (p.n2 > 0) { prefetch_tmap(&tm.k2); prefetch_tmap(&tm.v2); }
      if (p.out != nullptr && t_begin < t_end) {
        mbar_expect_tx(q_bar, (uint32_t)(H * p.M * 128));
#pragma unroll
        for (int h = 0; h < H; ++h) tma_load_4d(smem_u32(q_s + h * Mpad * 128), &tm.q, q_bar, h * 64, 0, g * p.G, bi);
      }
      int n1 = -1, it = 0;
      for (int t = t_begin; t < t_end && !dead; ++t) {
        if (t - t_begin >= STAGES) {
          if (n1 < 0) { n1 = p.n1_per_seq ? p.n1_per_seq[bi] : p.n1_max; n1 = min(max(n1, 0), p.n1_max); }
          if (!tile_is_processed(t - t_begin, t, tiles1, KT, n1, STAGES)) continue;
        }
        const int s = it % STAGES;
        if (it >= STAGES && !mbar_wait(empty_bar(s), ((it / STAGES) - 1) & 1)) { dead = true; atomicExch(p.status, 1); break; }
        mbar_expect_tx(full_bar(s), (uint32_t)stage_bytes);
        const uint32_t kdst = smem_u32(stage0 + (size_t)s * stage_bytes), vdst = kdst + H * half_bytes;
        const bool src1 = t < tiles1;
        const CUtensorMap* mk = src1 ? &tm.k1 : &tm.k2;
        const CUtensorMap* mv = src1 ? &tm.v1 : &tm.v2;
        const int row = (src1 ? t : t - tiles1) * KT;
#pragma unroll
        for (int h = 0; h < H; ++h) {
          tma_load_4d(kdst + h * half_bytes, mk, full_bar(s), h * 64, row, g, bi);
          tma_load_4d(vdst + h * half_bytes, mv, full_bar(s), h * 64, row, g, bi);
        }
        ++it;
      }
    }
  } else {
    // =============================== consumer warps ===============================
    int n1 = p.n1_per_seq ? p.n1_per_seq[bi] : p.n1_max;
    n1 = min(max(n1, 0), p.n1_max);
    r.n1 = n1; r.N = n1 + p.n2;
#pragma unroll
    for (int i = 0; i < DN; ++i) { oacc[i][0] = 0.f; oacc[i][1] = 0.f; oacc[i][2] = 0.f; oacc[i][3] = 0.f; }

    if (p.want_scores) {
      for (int d = tid; d < D; d += n_cons_threads) {
        float acc = 0.f;
        for (int hg = 0; hg < p.G; ++hg) {
          const __nv_bfloat16* qh = reinterpret_cast<const __nv_bfloat16*>(p.q) + (int64_t)bi * p.q_stride[0] +
                                    (int64_t)(g * p.G + hg) * p.q_stride[1];
          for (int i = 0; i < p.b; ++i) acc += __bfloat162float(qh[(int64_t)i * p.q_stride[2] + d]);
        }
        qbar_s[d] = acc / (float)p.M;
      }
      consumer_bar(n_cons_threads);
    }

    uint32_t qf[QREG ? KS : 1][4];
    const int q_row = r0 + (lane & 7) + ((lane >> 3) & 1) * 8;
    const uint32_t q_addr_row = smem_u32(q_s) + q_row * 128;
    const int q_sw = q_row & 7, q_cadd = lane >> 4;
    auto q_frag_addr = [&](int ks) {
      const int c = ks * 2 + q_cadd;                       // 16-byte chunk of the row
      return q_addr_row + (c >> 3) * (Mpad * 128) + (((c & 7) ^ q_sw) << 4);
    };
    if (p.out != nullptr && t_begin < t_end) {
      if (!mbar_wait(q_bar, 0)) { dead = true; atomicExch(p.status, 2); }
      if (QREG) {
#pragma unroll
        for (int ks = 0; ks < KS; ++ks)
          ldsm_x4(q_frag_addr(ks), qf[QREG ? ks : 0][0], qf[QREG ? ks : 0][1], qf[QREG ? ks : 0][2], qf[QREG ? ks : 0][3]);
      }
    }

    int it = 0;
    for (int t = t_begin; t < t_end; ++t) {
      if (!tile_is_processed(t - t_begin, t, tiles1, KT, n1, STAGES)) continue;
      const int s = it % STAGES;
      if (!dead && !mbar_wait(full_bar(s), (it / STAGES) & 1)) { dead = true; atomicExch(p.status, 3); }
      const unsigned char* kst = stage0 + (size_t)s * stage_bytes;
      const uint32_t ks_base = smem_u32(kst);
      const uint32_t vs_base = ks_base + H * half_bytes;
      const bool src1 = t < tiles1;
      const int j0 = (src1 ? t : t - tiles1) * KT;        // first row of the tile within its source
      const int n_src = src1 ? n1 : p.n2;                 // valid rows of that source

      // ---- saliency of this tile's keys (source 1 only): a_j = scale * <qbar, k_j>, 8 lanes per key ----
      if (p.want_scores && src1) {
        const int l8 = lane & 7;
        for (int kk = warp * 4 + (lane >> 3); kk < KT; kk += n_cons * 4) {
          float acc = 0.f;
#pragma unroll
          for (int h = 0; h < H; ++h) {
            const uint4 raw = *reinterpret_cast<const uint4*>(kst + h * half_bytes + kk * 128 + ((l8 ^ (kk & 7)) << 4));
            const float4 qa = *reinterpret_cast<const float4*>(qbar_s + h * 64 + l8 * 8);
            const float4 qb = *reinterpret_cast<const float4*>(qbar_s + h * 64 + l8 * 8 + 4);
            const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
            float2 f;
            f = __bfloat1622float2(h2[0]); acc = fmaf(qa.x, f.x, acc); acc = fmaf(qa.y, f.y, acc);
            f = __bfloat1622float2(h2[1]); acc = fmaf(qa.z, f.x, acc); acc = fmaf(qa.w, f.y, acc);
            f = __bfloat1622float2(h2[2]); acc = fmaf(qb.x, f.x, acc); acc = fmaf(qb.y, f.y, acc);
            f = __bfloat1622float2(h2[3]); acc = fmaf(qb.z, f.x, acc); acc = fmaf(qb.w, f.y, acc);
          }
          acc += __shfl_xor_sync(0xffffffffu, acc, 1);
          acc += __shfl_xor_sync(0xffffffffu, acc, 2);
          acc += __shfl_xor_sync(0xffffffffu, acc, 4);
          const int j = j0 + kk;
          if (l8 == 0 && j < n1) p.raw_scores[(int64_t)(bi * p.Hkv + g) * p.n1_max + j] = acc * p.scale;
        }
      }

      if (p.out != nullptr) {
        // ---- S = Q K^T for this warp's 16 rows x WK keys ----
        float sacc[NT][4];
#pragma unroll
        for (int i = 0; i < NT; ++i) { sacc[i][0] = 0.f; sacc[i][1] = 0.f; sacc[i][2] = 0.f; sacc[i][3] = 0.f; }
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
          uint32_t a[4];
          if (QREG) {
            a[0] = qf[QREG ? ks : 0][0]; a[1] = qf[QREG ? ks : 0][1]; a[2] = qf[QREG ? ks : 0][2]; a[3] = qf[QREG ? ks : 0][3];
          } else {
            ldsm_x4(q_frag_addr(ks), a[0], a[1], a[2], a[3]);
          }
          const int c = ks * 2 + ((lane >> 3) & 1);
          const uint32_t kh = ks_base + (c >> 3) * half_bytes;
#pragma unroll
          for (int nt2 = 0; nt2 < NT / 2; ++nt2) {
            const int row = cw * WK + nt2 * 16 + (lane & 7) + ((lane >> 4) << 3);
            uint32_t b0, b1, b2, b3;
            ldsm_x4(kh + row * 128 + (((c & 7) ^ (row & 7)) << 4), b0, b1, b2, b3);
            mma_bf16(sacc[2 * nt2], a, b0, b1);
            mma_bf16(sacc[2 * nt2 + 1], a, b2, b3);
          }
        }
        // ---- mask rows at or beyond the source's count, online softmax in log2 units ----
        const int jw = j0 + cw * WK;
        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const int j = jw + nt * 8 + 2 * t4;
          if (j >= n_src) { sacc[nt][0] = -INFINITY; sacc[nt][2] = -INFINITY; }
          if (j + 1 >= n_src) { sacc[nt][1] = -INFINITY; sacc[nt][3] = -INFINITY; }
          mx0 = fmaxf(mx0, fmaxf(sacc[nt][0], sacc[nt][1]));
          mx1 = fmaxf(mx1, fmaxf(sacc[nt][2], sacc[nt][3]));
        }
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
        const float mn0 = fmaxf(m_run[0], mx0 * p.scale_log2), mn1 = fmaxf(m_run[1], mx1 * p.scale_log2);
        const float mu0 = (mn0 == -INFINITY) ? 0.f : mn0, mu1 = (mn1 == -INFINITY) ? 0.f : mn1;
        const float al0 = exp2f(m_run[0] - mu0), al1 = exp2f(m_run[1] - mu1);
        m_run[0] = mn0; m_run[1] = mn1;
        float ps0 = 0.f, ps1 = 0.f;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          sacc[nt][0] = exp2f(fmaf(sacc[nt][0], p.scale_log2, -mu0));
          sacc[nt][1] = exp2f(fmaf(sacc[nt][1], p.scale_log2, -mu0));
          sacc[nt][2] = exp2f(fmaf(sacc[nt][2], p.scale_log2, -mu1));
          sacc[nt][3] = exp2f(fmaf(sacc[nt][3], p.scale_log2, -mu1));
          ps0 += sacc[nt][0] + sacc[nt][1];
          ps1 += sacc[nt][2] + sacc[nt][3];
        }
        l_run[0] = fmaf(l_run[0], al0, ps0);
        l_run[1] = fmaf(l_run[1], al1, ps1);
#pragma unroll
        for (int dn = 0; dn < DN; ++dn) { oacc[dn][0] *= al0; oacc[dn][1] *= al0; oacc[dn][2] *= al1; oacc[dn][3] *= al1; }

        // ---- rows of V past the count may hold anything (padding): zero this warp's slice of them so that 0 * V stays 0 ----
        if (jw + WK > n_src) {
          const int first = max(n_src - jw, 0);              // first invalid row inside the warp's slice
          for (int idx = lane; idx < (WK - first) * H * 8; idx += 32) {
            const int rr = first + idx / (H * 8), c = idx % (H * 8);
            const int row = cw * WK + rr;
            *reinterpret_cast<uint4*>(const_cast<unsigned char*>(kst) + H * half_bytes + (c >> 3) * half_bytes + row * 128 +
                                      (((c & 7) ^ (row & 7)) << 4)) = make_uint4(0u, 0u, 0u, 0u);
          }
          asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
          __syncwarp();
        }
        // ---- O += P V ----
#pragma unroll
        for (int kk = 0; kk < KK; ++kk) {
          uint32_t pa[4];
          pa[0] = pack_bf16(sacc[2 * kk][0], sacc[2 * kk][1]);
          pa[1] = pack_bf16(sacc[2 * kk][2], sacc[2 * kk][3]);
          pa[2] = pack_bf16(sacc[2 * kk + 1][0], sacc[2 * kk + 1][1]);
          pa[3] = pack_bf16(sacc[2 * kk + 1][2], sacc[2 * kk + 1][3]);
          const int row = cw * WK + kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
          const uint32_t v_row = vs_base + row * 128;
          const int sw = row & 7;
#pragma unroll
          for (int dn2 = 0; dn2 < DN / 2; ++dn2) {
            const int c = dn2 * 2 + (lane >> 4);
            uint32_t b0, b1, b2, b3;
            ldsm_x4_trans(v_row + (c >> 3) * half_bytes + (((c & 7) ^ sw) << 4), b0, b1, b2, b3);
            mma_bf16(oacc[2 * dn2], pa, b0, b1);
            mma_bf16(oacc[2 * dn2 + 1], pa, b2, b3);
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty_bar(s));
      ++it;
    }
  }

  if (p.out == nullptr) return;      // scores only: uniform over the grid, no cluster barrier was entered

  const bool direct = c_warps == 1 && cluster == 1;
  float* scr = reinterpret_cast<float*>(stage0);           // per-warp partials, then the CTA-level partial
  const int per_warp = 16 * D + 32;
  float* red = scr + (c_warps > 1 ? (size_t)n_cons * per_warp : 0);   // [Mpad][D] then [Mpad][2]
  float* red_ml = red + (size_t)Mpad * D;

  if (!is_producer) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 1);
      l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 2);
    }
    if (direct) {
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int m = r0 + g8 + h * 8;
        if (m >= p.M) continue;
        if (p.splits == 1) {
          const float inv = l_run[h] > 0.f ? 1.f / l_run[h] : 0.f;
          __nv_bfloat16* o = out_row_ptr<__nv_bfloat16>(p, r, m);
#pragma unroll
          for (int dn = 0; dn < DN; ++dn) store_out2(o + dn * 8 + 2 * t4, oacc[dn][2 * h] * inv, oacc[dn][2 * h + 1] * inv);
        } else {
          float* o = p.part_o + part_row(p, r, m) * D;
#pragma unroll
          for (int dn = 0; dn < DN; ++dn) *reinterpret_cast<float2*>(o + dn * 8 + 2 * t4) = make_float2(oacc[dn][2 * h], oacc[dn][2 * h + 1]);
        }
        if (t4 == 0) store_ml(p, r, m, m_run[h], l_run[h]);
      }
    } else if (c_warps == 1) {
      // ---- each warp owns its 16 rows outright: park them as the CTA-level partial for the cluster merge ----
      consumer_bar(n_cons_threads);                        // the ring is idle from here on
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int m = r0 + g8 + h * 8;
#pragma unroll
        for (int dn = 0; dn < DN; ++dn)
          *reinterpret_cast<float2*>(red + (size_t)m * D + dn * 8 + 2 * t4) = make_float2(oacc[dn][2 * h], oacc[dn][2 * h + 1]);
        if (t4 == 0) *reinterpret_cast<float2*>(red_ml + m * 2) = make_float2(m_run[h], l_run[h]);
      }
    } else {
      // ---- phase A: every consumer warp parks its partial in shared memory (the ring is idle now) ----
      consumer_bar(n_cons_threads);
      float* mine = scr + (size_t)warp * per_warp;
#pragma unroll
      for (int dn = 0; dn < DN; ++dn) {
        *reinterpret_cast<float2*>(mine + g8 * D + dn * 8 + 2 * t4) = make_float2(oacc[dn][0], oacc[dn][1]);
        *reinterpret_cast<float2*>(mine + (g8 + 8) * D + dn * 8 + 2 * t4) = make_float2(oacc[dn][2], oacc[dn][3]);
      }
      if (t4 == 0) {
        mine[16 * D + g8 * 2] = m_run[0]; mine[16 * D + g8 * 2 + 1] = l_run[0];
        mine[16 * D + (g8 + 8) * 2] = m_run[1]; mine[16 * D + (g8 + 8) * 2 + 1] = l_run[1];
      }
      consumer_bar(n_cons_threads);
      // ---- phase B: merge the c_warps key slices of every row inside the CTA ----
      const int total = Mpad * (D / 4);
      for (int idx = tid; idx < total; idx += n_cons_threads) {
        const int m = idx / (D / 4), d4 = idx - m * (D / 4);
        if (m >= p.M) continue;
        const int band = m >> 4, rr = m & 15;
        const float* w0 = scr + (size_t)(band * c_warps) * per_warp;
        float mstar = -INFINITY;
        for (int c = 0; c < c_warps; ++c) mstar = fmaxf(mstar, w0[(size_t)c * per_warp + 16 * D + rr * 2]);
        const float mu = (mstar == -INFINITY) ? 0.f : mstar;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float l = 0.f;
        for (int c = 0; c < c_warps; ++c) {
          const float* wc = w0 + (size_t)c * per_warp;
          const float w = exp2f(wc[16 * D + rr * 2] - mu);
          l = fmaf(wc[16 * D + rr * 2 + 1], w, l);
          const float4 o = *reinterpret_cast<const float4*>(wc + rr * D + d4 * 4);
          acc.x = fmaf(o.x, w, acc.x); acc.y = fmaf(o.y, w, acc.y); acc.z = fmaf(o.z, w, acc.z); acc.w = fmaf(o.w, w, acc.w);
        }
        if (cluster > 1) {
          *reinterpret_cast<float4*>(red + (size_t)m * D + d4 * 4) = acc;
          if (d4 == 0) *reinterpret_cast<float2*>(red_ml + m * 2) = make_float2(mstar, l);
        } else if (p.splits == 1) {
          const float inv = l > 0.f ? 1.f / l : 0.f;
          __nv_bfloat16* o = out_row_ptr<__nv_bfloat16>(p, r, m) + d4 * 4;
          store_out2(o, acc.x * inv, acc.y * inv);
          store_out2(o + 2, acc.z * inv, acc.w * inv);
          if (d4 == 0) store_ml(p, r, m, mstar, l);
        } else {
          *reinterpret_cast<float4*>(p.part_o + part_row(p, r, m) * D + d4 * 4) = acc;
          if (d4 == 0) store_ml(p, r, m, mstar, l);
        }
      }
    }
  }

  if (cluster > 1) {
    // ---- phase C: the CTAs of the cluster combine their partials through distributed shared memory ----
    cluster_sync_all();
    if (!is_producer) {
      const int rank = (int)cluster_ctarank();
      const int m_lo = (int)(((long long)rank * p.M) / cluster), m_hi = (int)(((long long)(rank + 1) * p.M) / cluster);
      const uint32_t red_a = smem_u32(red), ml_a = smem_u32(red_ml);
      const int total = (m_hi - m_lo) * (D / 4);
      for (int idx = tid; idx < total; idx += n_cons_threads) {
        const int m = m_lo + idx / (D / 4), d4 = idx % (D / 4);
        float2 ml[8];
        float mstar = -INFINITY;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          ml[c] = make_float2(-INFINITY, 0.f);
          if (c < cluster) {
            ml[c] = ld_cluster_f2(map_to_cta(ml_a + m * 8, c));
            if (ml[c].y > 0.f) mstar = fmaxf(mstar, ml[c].x);
          }
        }
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float l = 0.f;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          if (c >= cluster || !(ml[c].y > 0.f)) continue;
          const float w = exp2f(ml[c].x - mstar);
          l = fmaf(ml[c].y, w, l);
          const float4 o = ld_cluster_f4(map_to_cta(red_a + (uint32_t)(m * D + d4 * 4) * 4u, c));
          acc.x = fmaf(o.x, w, acc.x); acc.y = fmaf(o.y, w, acc.y); acc.z = fmaf(o.z, w, acc.z); acc.w = fmaf(o.w, w, acc.w);
        }
        if (p.splits == 1) {
          const float inv = l > 0.f ? 1.f / l : 0.f;
          __nv_bfloat16* o = out_row_ptr<__nv_bfloat16>(p, r, m) + d4 * 4;
          store_out2(o, acc.x * inv, acc.y * inv);
          store_out2(o + 2, acc.z * inv, acc.w * inv);
        } else {
          *reinterpret_cast<float4*>(p.part_o + part_row(p, r, m) * D + d4 * 4) = acc;
        }
        if (d4 == 0) store_ml(p, r, m, mstar, l);
      }
    }
    cluster_sync_all();                // nobody leaves while a peer may still read its shared memory
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

// 4-D bf16 tensor (D, rows, heads, batch) with element strides for the three outer axes; box = (64, box_rows, box_heads, 1).
bool make_map(CUtensorMap* m, const void* base, int D, int rows, int heads, int batch, const int64_t* stride_bhr, int box_rows,
              int box_heads) {
  EncodeTiledFn enc = encode_fn();
  if (!enc || rows < 1) return false;
  const cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)rows, (cuuint64_t)heads, (cuuint64_t)batch};
  // a stride of an axis of extent 1 is never used; keep it a legal value
  auto st = [&](int64_t s) { return (cuuint64_t)(s > 0 ? s * 2 : (int64_t)D * 2); };
  const cuuint64_t strides[3] = {st(stride_bhr[2]), st(stride_bhr[1]), st(stride_bhr[0])};
  const cuuint32_t box[4] = {64u, (cuuint32_t)box_rows, (cuuint32_t)box_heads, 1u};
  const cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

size_t tma_smem_bytes(int D, const AttnPlan& pl) {
  const size_t H = D / 64, Mpad = (size_t)pl.m_warps * 16;
  size_t ring = (size_t)pl.stages * 2 * H * pl.key_tile * 128;
  const size_t n_cons = (size_t)pl.m_warps * pl.c_warps;
  const bool direct = pl.c_warps == 1 && pl.cluster == 1;
  const size_t scratch = direct ? 0 : ((pl.c_warps > 1 ? n_cons * (16 * D + 32) : 0) + Mpad * (D + 2)) * 4;
  if (scratch > ring) ring = scratch;
  return 1024 /*alignment slack*/ + 1024 /*barriers, qbar*/ + H * Mpad * 128 + ring;
}

bool pdl_enabled() {   // SDLLM_PDL=0 turns programmatic dependent launch off (tuning and test aid)
  const char* e = getenv("SDLLM_PDL");
  return !(e && e[0] == '0');
}

template <int D, int WK, int STAGES, int NT_MAX, bool QREG>
cudaError_t launch_inst(const TmaMaps& tm, const AttnParams& p, const AttnPlan& pl, cudaStream_t st) {
  auto kern = attn_tma_bf16_kernel<D, WK, STAGES, NT_MAX, QREG>;
  static size_t configured = 0;
  if (pl.smem_bytes > configured) {
    const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem_bytes);
    if (e != cudaSuccess) return e;
    // ask for the largest shared-memory carve-out so that two CTAs of the small-row shapes fit on one SM
    (void)cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    configured = pl.smem_bytes;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(pl.cluster * pl.splits, p.Hkv, p.B);
  cfg.blockDim = dim3(pl.threads);
  cfg.dynamicSmemBytes = pl.smem_bytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  int na = 0;
  attr[na].id = cudaLaunchAttributeClusterDimension;
  attr[na].val.clusterDim.x = pl.cluster; attr[na].val.clusterDim.y = 1; attr[na].val.clusterDim.z = 1;
  ++na;
  if (pdl_enabled()) {
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  cfg.attrs = attr; cfg.numAttrs = na;
  return cudaLaunchKernelEx(&cfg, kern, tm, p, pl.m_warps, pl.c_warps, pl.cluster);
}

template <int D, int WK, int NT_MAX, bool QREG>
cudaError_t launch_stages(const TmaMaps& tm, const AttnParams& p, const AttnPlan& pl, cudaStream_t st) {
  switch (pl.stages) {
    case 2: return launch_inst<D, WK, 2, NT_MAX, QREG>(tm, p, pl, st);
    case 3: return launch_inst<D, WK, 3, NT_MAX, QREG>(tm, p, pl, st);
    default: return launch_inst<D, WK, 4, NT_MAX, QREG>(tm, p, pl, st);
  }
}

template <int D>
cudaError_t launch_tma_d(const TmaMaps& tm, const AttnParams& p, const AttnPlan& pl, cudaStream_t st) {
  // (warp_keys, thread bound) pairs the planner produces
  if (pl.warp_keys == 16 && pl.threads <= 160) return launch_stages<D, 16, 160, true>(tm, p, pl, st);
  if (pl.warp_keys == 16) return launch_stages<D, 16, 288, true>(tm, p, pl, st);
  if (pl.warp_keys == 32 && pl.threads <= 288) return launch_stages<D, 32, 288, true>(tm, p, pl, st);
  if (pl.warp_keys == 32) return launch_stages<D, 32, 544, false>(tm, p, pl, st);
  return launch_stages<D, 64, 288, true>(tm, p, pl, st);
}

}  // namespace

// Partial rows the mma.sync kernels leave per (sequence, KV head).
static void finish_plan(AttnPlan& pl, int M) {
  pl.part_rows = pl.splits > 1 ? (size_t)pl.splits * M : 0;
  pl.n_counters = 0; pl.fused_tail = false;
  pl.rep = 1; pl.row_tiles = 1; pl.parts = pl.splits; pl.rows_rep = M; pl.key_tile2 = pl.key_tile;
}

AttnPlan plan_attention(int dtype, int D, int M, int b, int B, int Hkv, int n1_max, int n2) {
  // SDLLM_KERNEL = cpasync | tma | umma picks a kernel family for bf16 (tuning and test aid); default: tcgen05 where it applies
  const char* kern = getenv("SDLLM_KERNEL");
  const char* no_tma = getenv("SDLLM_NO_TMA");
  const bool want_cpasync = (no_tma && no_tma[0] == '1') || (kern && kern[0] == 'c');
  const bool want_tma = kern && kern[0] == 't';
  if (dtype != SDLLM_BF16 || want_cpasync || encode_fn() == nullptr) {
    AttnPlan pl = plan_attention_legacy(dtype, D, M, B, Hkv, n1_max + n2);
    pl.tma = false; pl.cluster = 1; pl.warp_keys = 32; pl.kind = 0;
    finish_plan(pl, M);
    return pl;
  }
  if (!want_tma && umma_supported(dtype, D, M, b)) return plan_attention_umma(D, M, b, B, Hkv, n1_max, n2);
  AttnPlan pl{};
  pl.tma = true; pl.kind = 1;
  pl.m_warps = (M + 15) / 16;
  if (pl.m_warps <= 2) { pl.c_warps = 8 / pl.m_warps; pl.warp_keys = 16; }        // 8 warps, 64- or 128-key tiles
  else if (pl.m_warps <= 4) { pl.c_warps = 2; pl.warp_keys = 32; }                // 6-8 warps, 64-key tiles
  else if (pl.m_warps <= 8) { pl.c_warps = 1; pl.warp_keys = 64; }                // 5-8 warps, 64-key tiles
  else { pl.c_warps = 1; pl.warp_keys = 32; }                                     // 9-16 warps, 32-key tiles
  if (pl.m_warps == 1) { pl.c_warps = 4; }
  pl.key_tile = pl.c_warps * pl.warp_keys;
  pl.threads = (pl.m_warps * pl.c_warps + 1) * 32;
  pl.cluster = 1;
  const size_t budget = pl.m_warps <= 4 ? 112 * 1024 : 220 * 1024;              // two CTAs per SM for the small-row shapes
  pl.stages = 4;
  while (pl.stages > 2 && tma_smem_bytes(D, pl) > budget) --pl.stages;

  const int tiles = (n1_max + pl.key_tile - 1) / pl.key_tile + (n2 + pl.key_tile - 1) / pl.key_tile;
  const long long base = (long long)B * Hkv;
  const bool two_per_sm = tma_smem_bytes(D, pl) <= 112 * 1024;
  long long total = two_per_sm ? (kNumSMs + base - 1) / base : kNumSMs / base;
  if (const char* e = getenv("SDLLM_SPLITS")) { if (atoi(e) >= 1) total = atoi(e); }   // tuning aid
  if (total > tiles) total = tiles;
  if (total < 1) total = 1;
  if (total > 8 * kMaxSplits) total = 8 * kMaxSplits;
  int max_cluster = 1;   // merging through the workspace measured faster than cluster launches on every shape tried
  if (const char* e = getenv("SDLLM_CLUSTER")) { if (atoi(e) >= 1 && atoi(e) <= 8) max_cluster = atoi(e); }
  const int outer = (int)((total + max_cluster - 1) / max_cluster);
  pl.cluster = (int)((total + outer - 1) / outer);
  pl.splits = outer;
  pl.smem_bytes = tma_smem_bytes(D, pl);
  finish_plan(pl, M);
  return pl;
}

cudaError_t launch_attn_partial(const AttnParams& p_in, const AttnPlan& plan, int dtype, int D, cudaStream_t st) {
  if (plan.kind == 2) return launch_attn_umma(p_in, plan, D, st);
  if (!plan.tma) return launch_attn_legacy(p_in, plan, dtype, D, st);
  AttnParams p = p_in;
  TmaMaps tm;
  bool ok = make_map(&tm.q, p.q, D, p.b, p.Hq, p.B, p.q_stride, p.b, p.G);
  if (p.n1_max > 0) {
    ok = ok && make_map(&tm.k1, p.k1, D, p.n1_max, p.Hkv, p.B, p.k1_stride, plan.key_tile, 1);
    ok = ok && make_map(&tm.v1, p.v1, D, p.n1_max, p.Hkv, p.B, p.k1_stride, plan.key_tile, 1);
  }
  if (p.n2 > 0) {
    ok = ok && make_map(&tm.k2, p.k2, D, p.n2, p.Hkv, p.B, p.k2_stride, plan.key_tile, 1);
    ok = ok && make_map(&tm.v2, p.v2, D, p.n2, p.Hkv, p.B, p.k2_stride, plan.key_tile, 1);
    if (p.n1_max <= 0) { tm.k1 = tm.k2; tm.v1 = tm.v2; }
  } else {
    tm.k2 = tm.k1; tm.v2 = tm.v1;
  }
  if (!ok) return cudaErrorInvalidValue;
  p.splits = plan.splits;
  p.splits_total = plan.splits * plan.cluster;
  return D == 128 ? launch_tma_d<128>(tm, p, plan, st) : launch_tma_d<64>(tm, p, plan, st);
}

}  // namespace sdllm
