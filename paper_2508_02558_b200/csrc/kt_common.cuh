// Device helpers shared by the two kernels that put the keys on the accumulator rows (attn_kt.cu, attn_kt_stream.cu).
// Included inside namespace sdllm { namespace { ... } } of each of them, after kt_params.cuh.
#pragma once

constexpr int KT_GRP = 3072;             // control block, per softmax warpgroup: references, raise scratch, sums, saliency partials
constexpr int KT_CTRL0 = 1024;           // control block, common part: barriers and flags

#include "umma_ptx.cuh"

__device__ __forceinline__ void cluster_arrive_relaxed() { asm volatile("barrier.cluster.arrive.relaxed;\n" ::: "memory"); }
__device__ __forceinline__ void cluster_arrive_release() { asm volatile("barrier.cluster.arrive.release;\n" ::: "memory"); }
__device__ __forceinline__ void cluster_wait_acquire() { asm volatile("barrier.cluster.wait.acquire;\n" ::: "memory"); }
// Asynchronous stores into the shared memory of a CTA of the cluster; each one reports its bytes to an mbarrier of that
// CTA (complete_tx, release at cluster scope), so the receiver waits for exactly the data it is owed and for nothing else.
__device__ __forceinline__ void st_async_f4(uint32_t addr, uint32_t mbar, float x, float y, float z, float w) {
  asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.v4.f32 [%0], {%1, %2, %3, %4}, [%5];\n"
               ::"r"(addr), "f"(x), "f"(y), "f"(z), "f"(w), "r"(mbar) : "memory");
}
__device__ __forceinline__ void st_async_f2(uint32_t addr, uint32_t mbar, float x, float y) {
  asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.v2.f32 [%0], {%1, %2}, [%3];\n"
               ::"r"(addr), "f"(x), "f"(y), "r"(mbar) : "memory");
}
// Bounded wait on an mbarrier that remote CTAs complete: acquire at cluster scope.
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool wait_merge(uint32_t bar, volatile int* abort_flag, int32_t* status, long long limit) {
  if (mbar_try_wait_cluster(bar, 0)) return true;
  const long long t0 = clock64();
  for (;;) {
    if (mbar_try_wait_cluster(bar, 0)) return true;
    const bool aborting = *abort_flag != 0;
    // an aborting CTA still lets its peers' pushes land before it retires (drain limit)
    if (clock64() - t0 > (aborting ? kDrainCycles : limit)) {
      if (!aborting) { *abort_flag = 1; atomicExch(status, 13); }
      else return false;
    }
  }
}
// Pulls one box of a tensor into L2 without waiting for it. L2 is the point of coherence, so this is safe for data a
// kernel in front of this one may still be writing: the later copy into shared memory reads what L2 holds then.
__device__ __forceinline__ void tma_prefetch_l2(const CUtensorMap* tm, int x, int y, int z, int w) {
  asm volatile("cp.async.bulk.prefetch.tensor.4d.L2.global.tile [%0, {%1, %2, %3, %4}];\n" ::"l"(tm), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
__device__ __forceinline__ float warp_max_f32(float v) {
  float r;
  asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;\n" : "=f"(r) : "f"(v));
  return r;
}
// barrier of the 128 softmax threads that also ORs a predicate over them
__device__ __forceinline__ bool softmax_barrier_or(int id, bool pred) {
  uint32_t r;
  asm volatile(
      "{\n .reg .pred p, q;\n setp.ne.u32 q, %1, 0;\n bar.red.or.pred p, %2, 128, q;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(r) : "r"((uint32_t)pred), "r"(id) : "memory");
  return r != 0;
}
// barrier of one softmax warpgroup (ids 1 to 4), and of all of them (id 5)
__device__ __forceinline__ void softmax_barrier(int id) { asm volatile("bar.sync %0, 128;\n" ::"r"(id) : "memory"); }
template <int NG>
__device__ __forceinline__ void softmax_barrier_all() { asm volatile("bar.sync 5, %0;\n" ::"n"(128 * NG) : "memory"); }

// order-preserving fp32 <-> u32 (larger float <=> larger code), for the shared-memory max of the references
__device__ __forceinline__ uint32_t f2ord(float x) {
  const uint32_t u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float ord2f(uint32_t k) { return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k); }

// Shared-memory matrix descriptor with the 64-byte swizzle (mode 4 in bits 61-63): rows of 64 bytes, 8 rows per atom.
__device__ __forceinline__ uint64_t smem_desc_sw64(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
         (1ull << 46) | (4ull << 61);
}
// Instruction descriptor, kind::f16: fp32 accumulator, bf16 A and B, M = 128, N = n; A and B K-major or MN-major.
__device__ __forceinline__ uint32_t kt_idesc(int n, bool a_mn, bool b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) | ((uint32_t)(n >> 3) << 17) |
         ((128u >> 4) << 24);
}

// One group of 32 key rows: where it comes from and how many of its rows are real keys.
struct Group {
  int src1;     // 1: source 1, 0: source 2
  int row0;     // first row inside its source
  int nv;       // valid rows, 1..32
};
__device__ __forceinline__ Group group_of(int gi, int g1, int n1, int n2) {
  Group x;
  if (gi < g1) { x.src1 = 1; x.row0 = gi * 32; x.nv = min(n1 - x.row0, 32); }
  else { x.src1 = 0; x.row0 = (gi - g1) * 32; x.nv = min(n2 - x.row0, 32); }
  return x;
}

// Importance of one absolute position: Algorithm 1, MaxPool1D(A, kernel_size = s, padding = s/2) over the candidate
// axis Concat(prefix, suffix) (AvgPool for the ablation); block positions and padding get -inf. `a` is the raw
// saliency by absolute position in global memory, written by other CTAs during this launch (read through L2).
__device__ __forceinline__ float kt_pool_at(const AttnParams& p, const float* a, int L, int o_in, int pos) {
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
// kt_pool_at for windows of at most 2 W + 1 with a fixed trip count: the window's loads are independent of one another and
// go out together (the loop of kt_pool_at waits for each before it issues the next: three L2 round trips for a window
// of three, on the critical path of a call that lasts 12 us). Same values, same order of the sum.
template <int W>
__device__ __forceinline__ float kt_pool_at_w(const AttnParams& p, const float* a, int L, int o_in, int pos) {
  const int b = p.b;
  const int o = min(max(o_in, 0), max(L - b, 0));
  if (pos >= L || (pos >= o && pos < o + b)) return -INFINITY;
  const int C = max(L - b, 0), w = (p.window - 1) / 2;
  const int c = pos < o ? pos : pos - b;
  int lo = 0, hi = C;
  if (p.per_region) { if (c < o) hi = o; else lo = o; }
  float x[2 * W + 1];
  bool ok[2 * W + 1];
#pragma unroll
  for (int k = -W; k <= W; ++k) {
    const int t = c + k;
    ok[k + W] = k >= -w && k <= w && t >= lo && t < hi;
    const int tt = ok[k + W] ? t : c;                  // (c itself is always a valid candidate)
    x[k + W] = __ldcg(a + (tt < o ? tt : tt + b));
  }
  float mx = -INFINITY, sum = 0.f;
#pragma unroll
  for (int i = 0; i < 2 * W + 1; ++i) {
    mx = ok[i] ? fmaxf(mx, x[i]) : mx;
    sum += ok[i] ? x[i] : 0.f;
  }
  return p.pool_kind == SDLLM_POOL_MAX ? mx : sum / (float)p.window;
}

// Pools the absolute positions [p_lo, p_hi) of one head with `nthreads` threads (this one is `tid`): `out` and `a` are the
// head's rows of the pooled and of the raw scores. A thread takes sixteen consecutive candidates at a time: their windows
// overlap, so 24 loads (all of them issued together: fixed count, clamped addresses) serve sixteen outputs, and the window
// logic runs on registers. Same values and the same order of the sums as kt_pool_at, which the wider windows still use.
// (One position at a time, each with its own loop of dependent L2 round trips, cost 16 us per 4352 positions.)
__device__ __forceinline__ void kt_pool_span(const AttnParams& p, const float* a, float* out, int L, int o_in, int p_lo, int p_hi,
                                             int tid, int nthreads) {
  const int b = p.b;
  const int o = min(max(o_in, 0), max(L - b, 0));
  const int C = max(L - b, 0), w = (p.window - 1) / 2;
  for (int pos = p_lo + tid; pos < p_hi; pos += nthreads)       // the block's own positions and the padding
    if (pos >= L || (pos >= o && pos < o + b)) out[pos] = -INFINITY;
  auto below = [&](int x) {                                     // candidates whose position lies below x
    const int c = x <= o ? x : (x <= o + b ? o : x - b);
    return min(max(c, 0), C);
  };
  const int cl = below(p_lo), ch = below(p_hi);
  if (w > 4 || ch - cl <= 4 * nthreads) {                     // (a few positions per thread: batching does not pay yet)
    for (int c = cl + tid; c < ch; c += nthreads) {
      const int pos = c < o ? c : c + b;
      out[pos] = w <= 1 ? kt_pool_at_w<1>(p, a, L, o_in, pos) : (w <= 2 ? kt_pool_at_w<2>(p, a, L, o_in, pos) : kt_pool_at(p, a, L, o_in, pos));
    }
    return;
  }
  constexpr int K = 16;
  const bool is_max = p.pool_kind == SDLLM_POOL_MAX;
  for (int c0 = cl + tid * K; c0 < ch; c0 += nthreads * K) {
    float v[K + 8];
#pragma unroll
    for (int i = 0; i < K + 8; ++i) {
      const int c = min(max(c0 - 4 + i, 0), C - 1);             // (C >= 1 here: the range is not empty)
      v[i] = __ldcg(a + (c < o ? c : c + b));
    }
#pragma unroll
    for (int u = 0; u < K; ++u) {
      const int c = c0 + u;
      if (c < ch) {
        int lo = 0, hi = C;
        if (p.per_region) { if (c < o) hi = o; else lo = o; }
        float mx = -INFINITY, sum = 0.f;
#pragma unroll
        for (int k = -4; k <= 4; ++k) {
          const int t = c + k;
          const bool ok = k >= -w && k <= w && t >= lo && t < hi;
          const float x = v[u + 4 + k];
          mx = ok ? fmaxf(mx, x) : mx;
          sum += ok ? x : 0.f;
        }
        out[c < o ? c : c + b] = is_max ? mx : sum / (float)p.window;
      }
    }
  }
}
