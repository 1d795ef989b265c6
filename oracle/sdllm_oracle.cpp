// CPU oracle for the Sparse-dLLM cache-refresh / sparse-block-attention path.
//
// TEST INFRASTRUCTURE ONLY. This file is a plain, slow, double-precision restatement of what
// the paper's method computes, written from the paper's equations and algorithms. It exists so
// that the CUDA library can be checked against something that is easy to verify by eye. It shares
// no code with the CUDA library, and nothing in the product path may call it: only the tests, the
// smoke check and the benchmark's CPU-baseline leg do.
//
// Every routine works on ONE sequence of ONE layer. Arrays are dense row-major doubles:
//   q      [Hq ][b ][D]   block queries Q_b
//   k, v   [Hkv][nk][D]   keys / values
// Query head h reads KV head h / G with G = Hq / Hkv (grouped-query attention).
// Loops over heads run under OpenMP; the arithmetic inside a head is strictly sequential.
//
// Parity pins (see tests): textbook attention by brute force and closed forms; linearity of the
// mean-query score; pooling as a dilation and against a library max-pool; full stable sort for the
// selection; r = 1 reproducing dense attention. Readings of the paper that nothing in it fixes
// (score kind, per-KV-head selection under GQA, joint-vs-per-region policy, ascending order of the
// kept rows) are "parity unpinned": they are fixed by this project's design notes only.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <numeric>
#include <vector>

namespace {
const double kNegInf = -std::numeric_limits<double>::infinity();
}

extern "C" {

// Softmax attention of the block queries over nk keys (Section 3.3 / Appendix A.2: the refresh step
// still performs bidirectional attention; Algorithm 3 at cache_state 2 attends over Concat(K_c, K_n)).
//   S_ij = scale * <q_i, k_j>,  P = row-softmax(S),  out_i = sum_j P_ij v_j,  lse_i = log sum_j exp(S_ij)
// out [Hq][b][D]; lse [Hq][b] (nullable); probs [Hq][b][nk] (nullable).
int orc_attention(const double* q, const double* k, const double* v, int Hq, int Hkv, int b, int nk, int D,
                  double scale, double* out, double* lse, double* probs) {
  if (Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || b <= 0 || nk <= 0 || D <= 0) return 1;
  const int G = Hq / Hkv;
#pragma omp parallel for schedule(dynamic)
  for (int h = 0; h < Hq; ++h) {
    const int g = h / G;
    std::vector<double> s(nk);
    for (int i = 0; i < b; ++i) {
      const double* qi = q + ((size_t)h * b + i) * D;
      double mx = kNegInf;
      for (int j = 0; j < nk; ++j) {
        const double* kj = k + ((size_t)g * nk + j) * D;
        double dot = 0.0;
        for (int d = 0; d < D; ++d) dot += qi[d] * kj[d];
        s[j] = scale * dot;
        mx = std::max(mx, s[j]);
      }
      double denom = 0.0;
      for (int j = 0; j < nk; ++j) { s[j] = std::exp(s[j] - mx); denom += s[j]; }
      double* oi = out + ((size_t)h * b + i) * D;
      for (int d = 0; d < D; ++d) oi[d] = 0.0;
      for (int j = 0; j < nk; ++j) {
        const double p = s[j] / denom;
        if (probs) probs[((size_t)h * b + i) * nk + j] = p;
        const double* vj = v + ((size_t)g * nk + j) * D;
        for (int d = 0; d < D; ++d) oi[d] += p * vj[d];
      }
      if (lse) lse[(size_t)h * b + i] = mx + std::log(denom);
    }
  }
  return 0;
}

// Candidate position map of Algorithm 1 ("extract the candidates"): K_f = Concat(K[:o], K[o+b:]); candidate c sits at
// absolute position c (prefix) or c + b (suffix).
int orc_candidate_pos(int c, int o, int b) { return c < o ? c : c + b; }

// Saliency of Algorithm 1 ("Mean(Q_b)", "MatMul(qbar, K_f^T)") with the 1/sqrt(d_k) of the body's attention-score equation:
//   qbar_g = Mean over the b*G block queries of KV head g;   a[g][c] = scale * <qbar_g, K_f[g][c]>
// k is the full-sequence K [Hkv][L][D]; a is [Hkv][L-b].
int orc_scores_logit_mean(const double* q, const double* k, int Hq, int Hkv, int b, int L, int D, int o,
                          double scale, double* a) {
  if (Hq % Hkv != 0 || o < 0 || o + b > L) return 1;
  const int G = Hq / Hkv, C = L - b;
#pragma omp parallel for schedule(dynamic)
  for (int g = 0; g < Hkv; ++g) {
    std::vector<double> qbar(D, 0.0);
    for (int hh = 0; hh < G; ++hh)
      for (int i = 0; i < b; ++i)
        for (int d = 0; d < D; ++d) qbar[d] += q[(((size_t)g * G + hh) * b + i) * D + d];
    for (int d = 0; d < D; ++d) qbar[d] /= (double)(G * b);
    for (int c = 0; c < C; ++c) {
      const double* kc = k + ((size_t)g * L + orc_candidate_pos(c, o, b)) * D;
      double dot = 0.0;
      for (int d = 0; d < D; ++d) dot += qbar[d] * kc[d];
      a[(size_t)g * C + c] = scale * dot;
    }
  }
  return 0;
}

// The same saliency evaluated the way the body's equation writes it: the full b x (L-b) logit matrix
// A = scale * Q_b K_f^T per query head, then the mean over the group's rows. Equal to
// orc_scores_logit_mean in exact arithmetic (linearity); kept as a separate evaluation order.
int orc_scores_logit_matrix_mean(const double* q, const double* k, int Hq, int Hkv, int b, int L, int D, int o,
                                 double scale, double* a) {
  if (Hq % Hkv != 0 || o < 0 || o + b > L) return 1;
  const int G = Hq / Hkv, C = L - b;
  for (int g = 0; g < Hkv; ++g)
    for (int c = 0; c < C; ++c) {
      const double* kc = k + ((size_t)g * L + orc_candidate_pos(c, o, b)) * D;
      double acc = 0.0;
      for (int hh = 0; hh < G; ++hh)
        for (int i = 0; i < b; ++i) {
          const double* qi = q + (((size_t)g * G + hh) * b + i) * D;
          double dot = 0.0;
          for (int d = 0; d < D; ++d) dot += qi[d] * kc[d];
          acc += scale * dot;
        }
      a[(size_t)g * C + c] = acc / (double)(G * b);
    }
  return 0;
}

// Softmax-probability variant of the saliency (SnapKV-style reading of "average attention scores"):
// a[g][c] = mean over the group's b*G rows of P[row][pos(c)], P normalised over all L keys.
// probs is [Hq][b][L] as produced by orc_attention.
int orc_scores_prob_mean(const double* probs, int Hq, int Hkv, int b, int L, int o, double* a) {
  if (Hq % Hkv != 0 || o < 0 || o + b > L) return 1;
  const int G = Hq / Hkv, C = L - b;
  for (int g = 0; g < Hkv; ++g)
    for (int c = 0; c < C; ++c) {
      const int pos = orc_candidate_pos(c, o, b);
      double acc = 0.0;
      for (int hh = 0; hh < G; ++hh)
        for (int i = 0; i < b; ++i) acc += probs[(((size_t)g * G + hh) * b + i) * L + pos];
      a[(size_t)g * C + c] = acc / (double)(G * b);
    }
  return 0;
}

// Algorithm 1, pooling step: I = Pool1D(A, kernel_size = s, padding = s/2), stride 1, odd s, so |I| = |A|.
// kind 0: max pooling, padding acts as -inf. kind 1: average pooling, padding counts as zeros and the
// divisor is always s (the default behaviour of a framework AvgPool1d).
// seam < 0: one window axis over all C candidates (the literal Concat reading: the last prefix key and the
// first suffix key are neighbours). seam >= 0: pooled separately inside [0, seam) and [seam, C).
int orc_pool(const double* a, int Hkv, int C, int s, int kind, int seam, double* out) {
  if (s < 1 || s % 2 == 0 || (kind != 0 && kind != 1)) return 1;
  const int w = (s - 1) / 2;
  for (int g = 0; g < Hkv; ++g)
    for (int c = 0; c < C; ++c) {
      int lo = 0, hi = C;
      if (seam >= 0) { if (c < seam) hi = seam; else lo = seam; }
      double mx = kNegInf, sum = 0.0;
      for (int t = c - w; t <= c + w; ++t) {
        if (t < lo || t >= hi) continue;
        const double x = a[(size_t)g * C + t];
        mx = std::max(mx, x);
        sum += x;
      }
      out[(size_t)g * C + c] = kind == 0 ? mx : sum / (double)s;
    }
  return 0;
}

// Algorithm 1, count step (n = floor(|I| * r)) and the two other counting policies.
//   mode 0 joint     : n_total = floor((L-b) * r); quotas are data dependent (-1).
//   mode 1 per region: ceil(r * o) from the prefix, ceil(r * (L-o-b)) from the suffix.
//   mode 2 prefix only (Algorithm 5): floor(o * r) from the prefix, the whole suffix.
// All products are taken in IEEE double; results clamped to the region sizes.
int orc_keep_count(int L, int b, int o, double r, int mode, int* n_total, int* n_prefix, int* n_suffix) {
  if (o < 0 || b < 0 || o + b > L || !(r >= 0.0 && r <= 1.0)) return 1;
  const int pre = o, suf = L - o - b;
  auto clampi = [](long long x, int hi) { return (int)std::max<long long>(0, std::min<long long>(x, hi)); };
  if (mode == 0) {
    *n_total = clampi((long long)std::floor((double)(pre + suf) * r), pre + suf);
    *n_prefix = -1; *n_suffix = -1;
  } else if (mode == 1) {
    *n_prefix = clampi((long long)std::ceil((double)pre * r), pre);
    *n_suffix = clampi((long long)std::ceil((double)suf * r), suf);
    *n_total = *n_prefix + *n_suffix;
  } else if (mode == 2) {
    *n_prefix = clampi((long long)std::floor((double)pre * r), pre);
    *n_suffix = suf;
    *n_total = *n_prefix + *n_suffix;
  } else {
    return 1;
  }
  return 0;
}

// Algorithm 1, selection step: TopKIndices(I, n) on one head's scores x[0..C). Ties go to the lowest index; the
// result is returned in ascending index order. Done as a full stable sort by descending score.
int orc_select_topk(const double* x, int C, int n, int32_t* idx_out) {
  if (n < 0 || n > C) return 1;
  std::vector<int32_t> order(C);
  std::iota(order.begin(), order.end(), 0);
  std::stable_sort(order.begin(), order.end(), [&](int32_t u, int32_t w) { return x[u] > x[w]; });
  std::vector<int32_t> kept(order.begin(), order.begin() + n);
  std::sort(kept.begin(), kept.end());
  std::copy(kept.begin(), kept.end(), idx_out);
  return 0;
}

// Algorithm 1, Select and cache store: K_c = Select(K, idx) for one tensor; src [Hkv][L][D], idx [Hkv][n] absolute
// positions, dst [Hkv][n][D]. Element size is given in bytes so the copy is bit-exact for any dtype.
int orc_gather_rows(const void* src, const int32_t* idx, int Hkv, int L, int n, size_t row_bytes, void* dst) {
  for (int g = 0; g < Hkv; ++g)
    for (int i = 0; i < n; ++i) {
      const int32_t p = idx[(size_t)g * n + i];
      if (p < 0 || p >= L) return 1;
      std::memcpy((char*)dst + ((size_t)g * n + i) * row_bytes, (const char*)src + ((size_t)g * L + p) * row_bytes,
                  row_bytes);
    }
  return 0;
}

// Algorithm 2 (x = 1) and Algorithm 4 (general delay x): 0 = dense step, 1 = refresh, 2 = reuse.
int orc_cache_state(int i, int x) { return i > x ? 2 : (i == x ? 1 : 0); }

}  // extern "C"
