// Device helpers shared by the attention kernels: async copies, ldmatrix / mma.sync wrappers, the split geometry
// and the row stores.
#pragma once
#include "common.cuh"

namespace sdllm {
namespace dev {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// ---------------------------------------------------------------------------------------------------------
// Geometry shared by both kernels
struct CtaRange {
  int bi, g, split, n1, N, t_begin, t_end;
};
__device__ __forceinline__ CtaRange cta_range(const AttnParams& p, int split, int key_tile) {
  CtaRange r;
  r.split = split; r.g = blockIdx.y; r.bi = blockIdx.z;
  int n1 = p.n1_per_seq ? p.n1_per_seq[r.bi] : p.n1_max;
  r.n1 = min(max(n1, 0), p.n1_max);
  r.N = r.n1 + p.n2;
  const int n_tiles = (r.N + key_tile - 1) / key_tile;
  r.t_begin = (int)(((long long)split * n_tiles) / p.splits_total);
  r.t_end = (int)(((long long)(split + 1) * n_tiles) / p.splits_total);
  return r;
}

// Store one finished row slice: either the final normalised output (single split) or the partial.
template <typename T>
__device__ __forceinline__ void store_out2(T* out, float a, float b);
template <>
__device__ __forceinline__ void store_out2<float>(float* out, float a, float b) { *reinterpret_cast<float2*>(out) = make_float2(a, b); }
template <>
__device__ __forceinline__ void store_out2<__nv_bfloat16>(__nv_bfloat16* out, float a, float b) {
  *reinterpret_cast<__nv_bfloat162*>(out) = __floats2bfloat162_rn(a, b);
}

template <typename T>
__device__ __forceinline__ T* out_row_ptr(const AttnParams& p, const CtaRange& r, int m) {
  const int hg = m / p.b, i = m - hg * p.b;
  return reinterpret_cast<T*>(p.out) + (int64_t)r.bi * p.o_stride[0] + (int64_t)(r.g * p.G + hg) * p.o_stride[1] +
         (int64_t)i * p.o_stride[2];
}
__device__ __forceinline__ int64_t part_row(const AttnParams& p, const CtaRange& r, int m) {
  return ((int64_t)(r.bi * p.Hkv + r.g) * p.splits + r.split) * p.M + m;
}
__device__ __forceinline__ void store_ml(const AttnParams& p, const CtaRange& r, int m, float mx, float l) {
  if (p.splits == 1) {
    if (p.lse) {
      const int hg = m / p.b, i = m - hg * p.b;
      p.lse[((int64_t)r.bi * p.Hq + r.g * p.G + hg) * p.b + i] = (mx + log2f(l)) * kLn2;
    }
  } else {
    reinterpret_cast<float2*>(p.part_ml)[part_row(p, r, m)] = make_float2(mx, l);
  }
}

// Mean block query of the KV head, Algorithm 1 "qbar <- Mean(Q_b)": fp32 sum over the b*G rows in a fixed order.
template <typename T>
__device__ __forceinline__ float to_f32(T x);
template <>
__device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T>
__device__ __forceinline__ void compute_qbar(const AttnParams& p, const CtaRange& r, int D, float* qbar_s) {
  for (int d = threadIdx.x; d < D; d += blockDim.x) {
    float acc = 0.f;
    for (int hg = 0; hg < p.G; ++hg) {
      const T* qh = reinterpret_cast<const T*>(p.q) + (int64_t)r.bi * p.q_stride[0] + (int64_t)(r.g * p.G + hg) * p.q_stride[1];
      for (int i = 0; i < p.b; ++i) acc += to_f32<T>(qh[(int64_t)i * p.q_stride[2] + d]);
    }
    qbar_s[d] = acc / (float)p.M;
  }
}


}  // namespace dev
}  // namespace sdllm
