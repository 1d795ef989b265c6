// Block-query attention over a streamed key axis, split along the keys (flash-decoding style).
//
// One CTA owns (sequence, KV head, key split): it streams its share of K/V rows once through a
// cp.async shared-memory ring (16-byte coalesced loads, XOR-swizzled rows), keeps the b*G query rows
// of the KV head on chip, runs an online softmax, and leaves an unnormalised partial (running max,
// running sum, O) in the workspace; a small second kernel merges the splits. At the refresh step the
// same pass also produces the mean-query saliency of every streamed key (Algorithm 1, "qbar <- Mean(Q_b)",
// "A <- MatMul(qbar, K_f^T)"), so the L x b probability matrix and the logit matrix never exist in memory.
//
// bf16: QK^T and PV run on the tensor cores (mma.sync m16n8k16, fp32 accumulate); fp32: plain FMA.

#include "attn_device.cuh"
#include "tuning.cuh"

namespace sdllm {
using namespace dev;
namespace {

// ---------------------------------------------------------------------------------------------------------
// bf16 tensor-core kernel
constexpr int WK = 32;  // keys per warp per tile

template <int D, int STAGES, int NT_MAX, bool QREG>
__global__ void __launch_bounds__(NT_MAX) attn_partial_bf16_kernel(const AttnParams p, const int m_warps, const int c_warps) {
  constexpr int RB = D * 2;        // bytes per row
  constexpr int CH = RB / 16;      // 16-byte chunks per row
  constexpr int KS = D / 16;       // k-steps of QK^T
  constexpr int DN = D / 8;        // n-tiles of PV
  extern __shared__ __align__(128) unsigned char smem[];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nthreads = blockDim.x, nwarps = nthreads >> 5;
  const int KT = c_warps * WK;
  const CtaRange r = cta_range(p, blockIdx.x, KT);
  const int Mpad = m_warps * 16;

  unsigned char* q_s = smem;
  float* qbar_s = reinterpret_cast<float*>(q_s + Mpad * RB);
  unsigned char* stage0 = reinterpret_cast<unsigned char*>(qbar_s + D);
  const int stage_bytes = 2 * KT * RB;

  const __nv_bfloat16* qg = reinterpret_cast<const __nv_bfloat16*>(p.q);
  const __nv_bfloat16* k1 = reinterpret_cast<const __nv_bfloat16*>(p.k1);
  const __nv_bfloat16* v1 = reinterpret_cast<const __nv_bfloat16*>(p.v1);
  const __nv_bfloat16* k2 = reinterpret_cast<const __nv_bfloat16*>(p.k2);
  const __nv_bfloat16* v2 = reinterpret_cast<const __nv_bfloat16*>(p.v2);
  const int64_t k1_base = (int64_t)r.bi * p.k1_stride[0] + (int64_t)r.g * p.k1_stride[1];
  const int64_t k2_base = (int64_t)r.bi * p.k2_stride[0] + (int64_t)r.g * p.k2_stride[1];

  // ---- Q tile (rows beyond M are zero) ----
  for (int idx = tid; idx < Mpad * CH; idx += nthreads) {
    const int row = idx / CH, c = idx % CH;
    const __nv_bfloat16* src = qg;
    int bytes = 0;
    if (row < p.M) {
      const int hg = row / p.b, i = row - hg * p.b;
      src = qg + (int64_t)r.bi * p.q_stride[0] + (int64_t)(r.g * p.G + hg) * p.q_stride[1] + (int64_t)i * p.q_stride[2] + c * 8;
      bytes = 16;
    }
    cp_async16(smem_u32(q_s) + row * RB + ((c ^ (row & 7)) << 4), src, bytes);
  }
  cp_async_commit();

  auto load_tile = [&](int t, int buf) {
    const uint32_t ks = smem_u32(stage0 + (size_t)buf * stage_bytes);
    const uint32_t vs = ks + KT * RB;
    const int j0 = t * KT;
    for (int idx = tid; idx < KT * CH; idx += nthreads) {
      const int row = idx / CH, c = idx % CH;
      const int j = j0 + row;
      const __nv_bfloat16 *ksrc = k1, *vsrc = v1;
      int bytes = 0;
      if (j < r.n1) {
        const int64_t off = k1_base + (int64_t)j * p.k1_stride[2] + c * 8;
        ksrc = k1 + off; vsrc = v1 + off; bytes = 16;
      } else if (j < r.N) {
        const int64_t off = k2_base + (int64_t)(j - r.n1) * p.k2_stride[2] + c * 8;
        ksrc = k2 + off; vsrc = v2 + off; bytes = 16;
      }
      const uint32_t d = row * RB + ((c ^ (row & 7)) << 4);
      cp_async16(ks + d, ksrc, bytes);
      cp_async16(vs + d, vsrc, bytes);
    }
  };

  // ---- prologue: STAGES-1 tiles in flight ----
#pragma unroll
  for (int s = 0; s < STAGES - 1; ++s) {
    if (r.t_begin + s < r.t_end) load_tile(r.t_begin + s, s);
    cp_async_commit();
  }
  if (p.want_scores) compute_qbar<__nv_bfloat16>(p, r, D, qbar_s);

  const int rw = warp / c_warps, cw = warp - rw * c_warps;
  const int r0 = rw * 16;
  const int g8 = lane >> 2, t4 = lane & 3;

  uint32_t qf[QREG ? KS : 1][4];
  float oacc[DN][4];
#pragma unroll
  for (int i = 0; i < DN; ++i) { oacc[i][0] = 0.f; oacc[i][1] = 0.f; oacc[i][2] = 0.f; oacc[i][3] = 0.f; }
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};

  const int q_row = r0 + (lane & 7) + ((lane >> 3) & 1) * 8;
  const uint32_t q_addr_row = smem_u32(q_s) + q_row * RB;
  const int q_sw = q_row & 7, q_cadd = lane >> 4;

  for (int t = r.t_begin; t < r.t_end; ++t) {
    const int it = t - r.t_begin;
    cp_async_wait<STAGES - 2>();
    __syncthreads();
    {  // refill the buffer that was consumed in the previous iteration
      const int tn = t + STAGES - 1;
      if (tn < r.t_end) load_tile(tn, (it + STAGES - 1) % STAGES);
      cp_async_commit();
    }
    if (QREG && it == 0) {
#pragma unroll
      for (int ks = 0; ks < KS; ++ks)
        ldsm_x4(q_addr_row + (((ks * 2 + q_cadd) ^ q_sw) << 4), qf[QREG ? ks : 0][0], qf[QREG ? ks : 0][1], qf[QREG ? ks : 0][2], qf[QREG ? ks : 0][3]);
    }
    const unsigned char* kst = stage0 + (size_t)(it % STAGES) * stage_bytes;
    const uint32_t ks_base = smem_u32(kst);
    const uint32_t vs_base = ks_base + KT * RB;
    const int j0 = t * KT;

    // ---- saliency of this tile's keys: a_j = scale * <qbar, k_j>, 8 lanes per key ----
    if (p.want_scores) {
      const int l8 = lane & 7;
      for (int kk = warp * 4 + (lane >> 3); kk < KT; kk += nwarps * 4) {
        float acc = 0.f;
#pragma unroll
        for (int h = 0; h < CH / 8; ++h) {
          const int c = l8 + h * 8;
          const uint4 raw = *reinterpret_cast<const uint4*>(kst + kk * RB + ((c ^ (kk & 7)) << 4));
          const float4 qa = *reinterpret_cast<const float4*>(qbar_s + c * 8);
          const float4 qb = *reinterpret_cast<const float4*>(qbar_s + c * 8 + 4);
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
        if (l8 == 0 && j < r.n1) p.raw_scores[(int64_t)(r.bi * p.Hkv + r.g) * p.n1_max + j] = acc * p.scale;
      }
    }

    if (p.out != nullptr) {
      // ---- S = Q K^T for this warp's 16 rows x 32 keys ----
      float sacc[WK / 8][4];
#pragma unroll
      for (int i = 0; i < WK / 8; ++i) { sacc[i][0] = 0.f; sacc[i][1] = 0.f; sacc[i][2] = 0.f; sacc[i][3] = 0.f; }
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        uint32_t a[4];
        if (QREG) {
          a[0] = qf[QREG ? ks : 0][0]; a[1] = qf[QREG ? ks : 0][1]; a[2] = qf[QREG ? ks : 0][2]; a[3] = qf[QREG ? ks : 0][3];
        } else {
          ldsm_x4(q_addr_row + (((ks * 2 + q_cadd) ^ q_sw) << 4), a[0], a[1], a[2], a[3]);
        }
#pragma unroll
        for (int nt2 = 0; nt2 < WK / 16; ++nt2) {
          const int row = cw * WK + nt2 * 16 + (lane & 7) + ((lane >> 4) << 3);
          const int c = ks * 2 + ((lane >> 3) & 1);
          uint32_t b0, b1, b2, b3;
          ldsm_x4(ks_base + row * RB + ((c ^ (row & 7)) << 4), b0, b1, b2, b3);
          mma_bf16(sacc[2 * nt2], a, b0, b1);
          mma_bf16(sacc[2 * nt2 + 1], a, b2, b3);
        }
      }
      // ---- mask the ragged tail, online softmax in log2 units ----
      const int jw = j0 + cw * WK;
      float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < WK / 8; ++nt) {
        const int j = jw + nt * 8 + 2 * t4;
        if (j >= r.N) { sacc[nt][0] = -INFINITY; sacc[nt][2] = -INFINITY; }
        if (j + 1 >= r.N) { sacc[nt][1] = -INFINITY; sacc[nt][3] = -INFINITY; }
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
      for (int nt = 0; nt < WK / 8; ++nt) {
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
      // ---- O += P V ----
#pragma unroll
      for (int kk = 0; kk < WK / 16; ++kk) {
        uint32_t pa[4];
        pa[0] = pack_bf16(sacc[2 * kk][0], sacc[2 * kk][1]);
        pa[1] = pack_bf16(sacc[2 * kk][2], sacc[2 * kk][3]);
        pa[2] = pack_bf16(sacc[2 * kk + 1][0], sacc[2 * kk + 1][1]);
        pa[3] = pack_bf16(sacc[2 * kk + 1][2], sacc[2 * kk + 1][3]);
        const int row = cw * WK + kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
        const uint32_t v_row = vs_base + row * RB;
        const int sw = row & 7;
#pragma unroll
        for (int dn2 = 0; dn2 < DN / 2; ++dn2) {
          const int c = dn2 * 2 + (lane >> 4);
          uint32_t b0, b1, b2, b3;
          ldsm_x4_trans(v_row + ((c ^ sw) << 4), b0, b1, b2, b3);
          mma_bf16(oacc[2 * dn2], pa, b0, b1);
          mma_bf16(oacc[2 * dn2 + 1], pa, b2, b3);
        }
      }
    }
  }
  cp_async_wait<0>();
  __syncthreads();
  if (p.out == nullptr) return;

  // ---- row sums live per thread; finish them across the quad ----
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 1);
    l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 2);
  }

  if (c_warps > 1) {
    // merge the c_warps key slices of every 16-row band through shared memory (the ring is idle now)
    float* scr = reinterpret_cast<float*>(stage0);
    const int per_warp = 16 * D + 32;
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
    __syncthreads();
    const int total = Mpad * (D / 4);
    for (int idx = tid; idx < total; idx += nthreads) {
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
  } else {
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
  }
}

// ---------------------------------------------------------------------------------------------------------
// fp32 kernel: 256 threads own 32 query rows; thread (r = tid/8, c8 = tid%8).
constexpr int F32_KT = 64;

template <int D>
__global__ void __launch_bounds__(256) attn_partial_f32_kernel(const AttnParams p, const int row_chunks) {
  constexpr int RS = D + 4;        // padded row stride in floats
  constexpr int CH = D / 4;        // 16-byte chunks per row
  constexpr int KT = F32_KT;
  extern __shared__ __align__(128) unsigned char smem[];
  float* q_s = reinterpret_cast<float*>(smem);          // [32][RS]
  float* p_s = q_s + 32 * RS;                           // [32][KT + 1]
  float* qbar_s = p_s + 32 * (KT + 1);                  // 32 * 65 floats keeps 16-byte alignment
  float* stage0 = qbar_s + D;                           // 2 x { K[KT][RS], V[KT][RS] }
  constexpr int stage_floats = 2 * KT * RS;

  const int tid = threadIdx.x;
  const int split = blockIdx.x / row_chunks, rc = blockIdx.x - split * row_chunks;
  const CtaRange r = cta_range(p, split, KT);
  const int rr = tid >> 3, c8 = tid & 7;
  const int m = rc * 32 + rr;
  const bool score_cta = p.want_scores && rc == 0;

  const float* qg = reinterpret_cast<const float*>(p.q);
  const float* k1 = reinterpret_cast<const float*>(p.k1);
  const float* v1 = reinterpret_cast<const float*>(p.v1);
  const float* k2 = reinterpret_cast<const float*>(p.k2);
  const float* v2 = reinterpret_cast<const float*>(p.v2);
  const int64_t k1_base = (int64_t)r.bi * p.k1_stride[0] + (int64_t)r.g * p.k1_stride[1];
  const int64_t k2_base = (int64_t)r.bi * p.k2_stride[0] + (int64_t)r.g * p.k2_stride[1];

  for (int idx = tid; idx < 32 * CH; idx += 256) {
    const int row = idx / CH, c = idx % CH;
    const int mm = rc * 32 + row;
    const float* src = qg;
    int bytes = 0;
    if (mm < p.M) {
      const int hg = mm / p.b, i = mm - hg * p.b;
      src = qg + (int64_t)r.bi * p.q_stride[0] + (int64_t)(r.g * p.G + hg) * p.q_stride[1] + (int64_t)i * p.q_stride[2] + c * 4;
      bytes = 16;
    }
    cp_async16(smem_u32(q_s + row * RS + c * 4), src, bytes);
  }
  cp_async_commit();

  auto load_tile = [&](int t, int buf) {
    float* ks = stage0 + (size_t)buf * stage_floats;
    float* vs = ks + KT * RS;
    const int j0 = t * KT;
    for (int idx = tid; idx < KT * CH; idx += 256) {
      const int row = idx / CH, c = idx % CH;
      const int j = j0 + row;
      const float *ksrc = k1, *vsrc = v1;
      int bytes = 0;
      if (j < r.n1) {
        const int64_t off = k1_base + (int64_t)j * p.k1_stride[2] + c * 4;
        ksrc = k1 + off; vsrc = v1 + off; bytes = 16;
      } else if (j < r.N) {
        const int64_t off = k2_base + (int64_t)(j - r.n1) * p.k2_stride[2] + c * 4;
        ksrc = k2 + off; vsrc = v2 + off; bytes = 16;
      }
      cp_async16(smem_u32(ks + row * RS + c * 4), ksrc, bytes);
      cp_async16(smem_u32(vs + row * RS + c * 4), vsrc, bytes);
    }
  };

  if (r.t_begin < r.t_end) load_tile(r.t_begin, 0);
  cp_async_commit();
  if (score_cta) compute_qbar<float>(p, r, D, qbar_s);

  float4 acc[D / 32];
#pragma unroll
  for (int i = 0; i < D / 32; ++i) acc[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  float m_run = -INFINITY, l_run = 0.f;

  for (int t = r.t_begin; t < r.t_end; ++t) {
    const int it = t - r.t_begin;
    if (t + 1 < r.t_end) load_tile(t + 1, (it + 1) & 1);
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();
    const float* ks = stage0 + (size_t)(it & 1) * stage_floats;
    const float* vs = ks + KT * RS;
    const int j0 = t * KT;

    if (score_cta) {
      const int lane = tid & 31, warp = tid >> 5, l8 = lane & 7;
      for (int kk = warp * 4 + (lane >> 3); kk < KT; kk += 8 * 4) {
        float a = 0.f;
#pragma unroll
        for (int h = 0; h < D / 32; ++h) {
          const int d = (l8 + 8 * h) * 4;
          const float4 kv4 = *reinterpret_cast<const float4*>(ks + kk * RS + d);
          const float4 q4 = *reinterpret_cast<const float4*>(qbar_s + d);
          a = fmaf(q4.x, kv4.x, a); a = fmaf(q4.y, kv4.y, a); a = fmaf(q4.z, kv4.z, a); a = fmaf(q4.w, kv4.w, a);
        }
        a += __shfl_xor_sync(0xffffffffu, a, 1);
        a += __shfl_xor_sync(0xffffffffu, a, 2);
        a += __shfl_xor_sync(0xffffffffu, a, 4);
        const int j = j0 + kk;
        if (l8 == 0 && j < r.n1) p.raw_scores[(int64_t)(r.bi * p.Hkv + r.g) * p.n1_max + j] = a * p.scale;
      }
    }

    if (p.out != nullptr) {
      float s[KT / 8];
#pragma unroll
      for (int jj = 0; jj < KT / 8; ++jj) s[jj] = 0.f;
      for (int d = 0; d < D; d += 4) {
        const float4 q4 = *reinterpret_cast<const float4*>(q_s + rr * RS + d);
#pragma unroll
        for (int jj = 0; jj < KT / 8; ++jj) {
          const float4 k4 = *reinterpret_cast<const float4*>(ks + (c8 + 8 * jj) * RS + d);
          s[jj] = fmaf(q4.x, k4.x, s[jj]); s[jj] = fmaf(q4.y, k4.y, s[jj]);
          s[jj] = fmaf(q4.z, k4.z, s[jj]); s[jj] = fmaf(q4.w, k4.w, s[jj]);
        }
      }
      float mx = -INFINITY;
#pragma unroll
      for (int jj = 0; jj < KT / 8; ++jj) {
        if (j0 + c8 + 8 * jj >= r.N) s[jj] = -INFINITY;
        mx = fmaxf(mx, s[jj]);
      }
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
      const float mn = fmaxf(m_run, mx * p.scale_log2);
      const float mu = (mn == -INFINITY) ? 0.f : mn;
      const float al = exp2f(m_run - mu);
      m_run = mn;
      float ps = 0.f;
#pragma unroll
      for (int jj = 0; jj < KT / 8; ++jj) {
        const float e = exp2f(fmaf(s[jj], p.scale_log2, -mu));
        ps += e;
        p_s[rr * (KT + 1) + c8 + 8 * jj] = e;
      }
      ps += __shfl_xor_sync(0xffffffffu, ps, 1);
      ps += __shfl_xor_sync(0xffffffffu, ps, 2);
      ps += __shfl_xor_sync(0xffffffffu, ps, 4);
      l_run = fmaf(l_run, al, ps);
#pragma unroll
      for (int i = 0; i < D / 32; ++i) { acc[i].x *= al; acc[i].y *= al; acc[i].z *= al; acc[i].w *= al; }
      __syncwarp();
      for (int j = 0; j < KT; ++j) {
        const float pj = p_s[rr * (KT + 1) + j];
#pragma unroll
        for (int i = 0; i < D / 32; ++i) {
          const float4 v4 = *reinterpret_cast<const float4*>(vs + j * RS + (c8 + 8 * i) * 4);
          acc[i].x = fmaf(pj, v4.x, acc[i].x); acc[i].y = fmaf(pj, v4.y, acc[i].y);
          acc[i].z = fmaf(pj, v4.z, acc[i].z); acc[i].w = fmaf(pj, v4.w, acc[i].w);
        }
      }
    }
    __syncthreads();
  }
  cp_async_wait<0>();
  if (p.out == nullptr || m >= p.M) return;

  if (p.splits == 1) {
    const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
    float* o = out_row_ptr<float>(p, r, m);
#pragma unroll
    for (int i = 0; i < D / 32; ++i)
      *reinterpret_cast<float4*>(o + (c8 + 8 * i) * 4) = make_float4(acc[i].x * inv, acc[i].y * inv, acc[i].z * inv, acc[i].w * inv);
  } else {
    float* o = p.part_o + part_row(p, r, m) * D;
#pragma unroll
    for (int i = 0; i < D / 32; ++i) *reinterpret_cast<float4*>(o + (c8 + 8 * i) * 4) = acc[i];
  }
  if (c8 == 0) store_ml(p, r, m, m_run, l_run);
}

// ---------------------------------------------------------------------------------------------------------
// Split merge + key-axis pooling (Algorithm 1, MaxPool1D) in one launch.
__global__ void __launch_bounds__(256) merge_pool_kernel(const MergeParams p) {
  const int tid = threadIdx.x;
  if ((int)blockIdx.x < p.merge_blocks) {
    const int D4 = p.D / 4;
    const int64_t idx = (int64_t)blockIdx.x * 256 + tid;
    const int64_t total = (int64_t)p.B * p.Hq * p.b * D4;
    if (idx >= total) return;
    const int d4 = (int)(idx % D4);
    const int64_t row = idx / D4;
    const int i = (int)(row % p.b);
    const int hq = (int)((row / p.b) % p.Hq);
    const int bi = (int)(row / ((int64_t)p.b * p.Hq));
    const int g = hq / p.G, m = (hq - g * p.G) * p.b + i;
    const int64_t base = (int64_t)(bi * p.Hkv + g) * p.splits;
    const float2* ml = reinterpret_cast<const float2*>(p.part_ml);
    float mstar = -INFINITY;
    for (int s = 0; s < p.splits; ++s) {
      const float2 x = ml[(base + s) * p.M + m];
      if (x.y > 0.f) mstar = fmaxf(mstar, x.x);
    }
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float l = 0.f;
    for (int s = 0; s < p.splits; ++s) {
      const float2 x = ml[(base + s) * p.M + m];
      if (!(x.y > 0.f)) continue;
      const float w = exp2f(x.x - mstar);
      l = fmaf(x.y, w, l);
      const float4 o = *reinterpret_cast<const float4*>(p.part_o + ((base + s) * p.M + m) * p.D + d4 * 4);
      acc.x = fmaf(o.x, w, acc.x); acc.y = fmaf(o.y, w, acc.y); acc.z = fmaf(o.z, w, acc.z); acc.w = fmaf(o.w, w, acc.w);
    }
    const float inv = l > 0.f ? 1.f / l : 0.f;
    const int64_t off = (int64_t)bi * p.o_stride[0] + (int64_t)hq * p.o_stride[1] + (int64_t)i * p.o_stride[2] + d4 * 4;
    if (p.dtype == SDLLM_BF16) {
      __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(p.out) + off;
      store_out2(o, acc.x * inv, acc.y * inv);
      store_out2(o + 2, acc.z * inv, acc.w * inv);
    } else {
      *reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + off) = make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
    }
    if (d4 == 0 && p.lse) p.lse[((int64_t)bi * p.Hq + hq) * p.b + i] = (mstar + log2f(l)) * kLn2;
    return;
  }
  // ---- pooling: one thread per absolute position ----
  const int64_t idx = (int64_t)(blockIdx.x - p.merge_blocks) * 256 + tid;
  const int64_t total = (int64_t)p.B * p.Hkv * p.Lmax;
  if (idx >= total) return;
  const int pos = (int)(idx % p.Lmax);
  const int64_t bh = idx / p.Lmax;
  const int bi = (int)(bh / p.Hkv);
  int L = p.seq_len ? p.seq_len[bi] : p.Lmax;
  L = min(max(L, 0), p.Lmax);
  const int o = p.block_off[bi], b = p.b;
  float outv = -INFINITY;
  if (pos < L && (pos < o || pos >= o + b)) {
    const int C = L - b;
    const int c = pos < o ? pos : pos - b;
    int lo = 0, hi = C;
    if (p.per_region) { if (c < o) hi = o; else lo = o; }
    const int w = (p.window - 1) / 2;
    const float* a = p.raw_scores + bh * p.Lmax;
    float mx = -INFINITY, sum = 0.f;
    for (int t = c - w; t <= c + w; ++t) {
      if (t < lo || t >= hi) continue;
      const float x = a[t < o ? t : t + b];
      mx = fmaxf(mx, x);
      sum += x;
    }
    outv = p.pool_kind == SDLLM_POOL_MAX ? mx : sum / (float)p.window;
  }
  p.pooled[idx] = outv;
}

// Raise the dynamic shared-memory limit of a kernel once per (kernel, device, size high-water mark).
template <typename K>
cudaError_t set_smem(K kernel, size_t bytes, SmemConfig* configured) {
  return configure_smem(reinterpret_cast<const void*>(kernel), bytes, *configured, false);
}

template <int D, int STAGES>
cudaError_t launch_bf16(const AttnParams& p, const AttnPlan& plan, cudaStream_t st) {
  const dim3 grid(plan.splits, p.Hkv, p.B), block(plan.threads);
  cudaError_t e;
#define SDLLM_LAUNCH(NT, QR)                                                                          \
  do {                                                                                                \
    auto kern = attn_partial_bf16_kernel<D, STAGES, NT, QR>;                                          \
    static SmemConfig configured;                                                                     \
    if ((e = set_smem(kern, plan.smem_bytes, &configured)) != cudaSuccess) return e;                  \
    kern<<<grid, block, plan.smem_bytes, st>>>(p, plan.m_warps, plan.c_warps);                        \
  } while (0)
  if (plan.threads <= 128) SDLLM_LAUNCH(128, true);
  else if (plan.threads <= 256) SDLLM_LAUNCH(256, true);
  else SDLLM_LAUNCH(512, false);
#undef SDLLM_LAUNCH
  return cudaGetLastError();
}

}  // namespace

size_t attn_legacy_smem_bytes(int dtype, int D, const AttnPlan& plan) {
  if (dtype == SDLLM_BF16) {
    const size_t rb = (size_t)D * 2;
    size_t ring = (size_t)plan.stages * 2 * plan.key_tile * rb;
    // the ring doubles as the scratch of the in-CTA merge across the key-slice warps
    const size_t scratch = plan.c_warps > 1 ? (size_t)plan.m_warps * plan.c_warps * (16 * D + 32) * 4 : 0;
    if (scratch > ring) ring = scratch;
    return (size_t)plan.m_warps * 16 * rb + (size_t)D * 4 + ring;
  }
  const size_t rs = (size_t)D + 4;
  return (32 * rs + 32 * (F32_KT + 1) + D + 2 * 2 * F32_KT * rs) * 4;
}

AttnPlan plan_attention_legacy(int dtype, int D, int M, int B, int Hkv, int n_keys_max, const Tuning& tn) {
  AttnPlan pl{};
  pl.cluster = 1; pl.warp_keys = 32; pl.tma = false;
  const long long base = (long long)B * Hkv;
  if (dtype == SDLLM_BF16) {
    pl.m_warps = (M + 15) / 16;
    pl.c_warps = pl.m_warps <= 1 ? 4 : (pl.m_warps <= 4 ? 2 : 1);
    pl.key_tile = pl.c_warps * WK;
    pl.threads = pl.m_warps * pl.c_warps * 32;
    pl.stages = 4;
    // keep room for two CTAs per SM when the tile is small enough
    while (pl.stages > 2 && attn_legacy_smem_bytes(dtype, D, pl) > 110 * 1024) --pl.stages;
  } else {
    pl.m_warps = (M + 31) / 32;
    pl.c_warps = 1;
    pl.key_tile = F32_KT;
    pl.threads = 256;
    pl.stages = 2;
  }
  pl.smem_bytes = attn_legacy_smem_bytes(dtype, D, pl);
  const int n_tiles = (n_keys_max + pl.key_tile - 1) / pl.key_tile;
  const int sms = sm_count();
  long long want = (sms + base - 1) / base;
  if (dtype != SDLLM_BF16) want = (want + pl.m_warps - 1) / pl.m_warps;
  long long splits = want < 1 ? 1 : want;
  if (tn.splits > 0) splits = tn.splits;
  if (splits > n_tiles) splits = n_tiles;
  if (splits > kMaxSplits) splits = kMaxSplits;
  if (splits < 1) splits = 1;
  pl.splits = (int)splits;
  return pl;
}

cudaError_t launch_attn_legacy(const AttnParams& p, const AttnPlan& plan, int dtype, int D, cudaStream_t st) {
  if (dtype == SDLLM_BF16) {
    if (D == 128) {
      if (plan.stages == 4) return launch_bf16<128, 4>(p, plan, st);
      if (plan.stages == 3) return launch_bf16<128, 3>(p, plan, st);
      return launch_bf16<128, 2>(p, plan, st);
    }
    if (plan.stages == 4) return launch_bf16<64, 4>(p, plan, st);
    if (plan.stages == 3) return launch_bf16<64, 3>(p, plan, st);
    return launch_bf16<64, 2>(p, plan, st);
  }
  const dim3 grid(plan.splits * plan.m_warps, p.Hkv, p.B), block(256);
  cudaError_t e;
  static SmemConfig configured128, configured64;
  if (D == 128) {
    if ((e = set_smem(attn_partial_f32_kernel<128>, plan.smem_bytes, &configured128)) != cudaSuccess) return e;
    attn_partial_f32_kernel<128><<<grid, block, plan.smem_bytes, st>>>(p, plan.m_warps);
  } else {
    if ((e = set_smem(attn_partial_f32_kernel<64>, plan.smem_bytes, &configured64)) != cudaSuccess) return e;
    attn_partial_f32_kernel<64><<<grid, block, plan.smem_bytes, st>>>(p, plan.m_warps);
  }
  return cudaGetLastError();
}

cudaError_t launch_merge_pool(const MergeParams& p, cudaStream_t st) {
  const long long merge_threads = p.part_o ? (long long)p.B * p.Hq * p.b * (p.D / 4) : 0;
  const long long pool_threads = p.pooled ? (long long)p.B * p.Hkv * p.Lmax : 0;
  MergeParams q = p;
  q.merge_blocks = (int)((merge_threads + 255) / 256);
  const long long blocks = q.merge_blocks + (pool_threads + 255) / 256;
  if (blocks == 0) return cudaSuccess;
  merge_pool_kernel<<<(unsigned)blocks, 256, 0, st>>>(q);
  return cudaGetLastError();
}

}  // namespace sdllm
