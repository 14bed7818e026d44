// LRSA oracle: a plain, slow, fp64 CPU statement of Lag-Relative Sparse Attention.
//
// TEST INFRASTRUCTURE ONLY. This file is the checker the CUDA library is compared
// against. It shares no code, header, table or helper with the CUDA path, and the
// product never calls it. Only the tests, the smoke check and the benchmark's
// cpu-baseline leg may load it.
//
// Everything is written in the order and notation of the paper:
//   * Section 3.2, Eq. 4-8  : LagKV score  (min/max of the NEXT window, normalise,
//                             Std over channels, Softmax over the window, K+V sum)
//   * Section 3.2 (text after Eq. 8): sink of size S, windows of lag size L, keep the
//                             top r*L = K tokens of each window
//   * Section 3.2, Attn-Fill 1 / Attn-Fill 2 : which keys a query chunk may see
//   * Section 3.1, Eq. 3    : A = softmax(Q K^T / sqrt(d_h) + M), output A V
//   * backward              : the textbook gradient of Eq. 3 with M held constant
//
// Inputs are bf16 bit patterns (uint16), converted exactly to double. There is no
// blocking, fusion or reordering: every function is a direct loop over its definition.
//
// Readings of the paper where it is silent (each is a parameter or stated here):
//   - previous window is seen uncompressed (n_dense_prev = 1); 0 gives the variant in
//     which it is already compressed when its follower is a full window
//   - Std is over the d channels of one token, divisor d - ddof (ddof = 1 default)
//   - a channel whose reference range is zero contributes normalised value 0
//   - only windows followed by a FULL window are scored; a tail shorter than L is an
//     ordinary query chunk, never compressed, never a reference
//   - ties in the score go to the lower position; kept positions listed ascending
//   - selection is a constant in the backward pass
//
// Parity pins (tests/test_oracle_*.py): dense-causal special case against a library
// softmax + autograd, brute-force explicit mask on tiny inputs, finite differences,
// a hand-enumerated mask, a hand-worked score, score invariants.  Choices the paper
// does not fix (ddof, zero range, tail handling, tie order) are "parity unpinned"
// beyond those checks.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <numeric>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

struct Params {
  int32_t B, Hq, Hkv, N, d, L, K, S, n_dense_prev, ddof;
  double scale;  // softmax scale of Eq. 3 (1/sqrt(d_h))
};

struct Geo {
  int W;     // full windows:   floor((N-S)/L)
  int T;     // tail tokens:    N - S - W*L
  int C;     // query chunks:   W + [T>0]
  int Wsel;  // scored windows: those with a full follower = max(W-1,0)
};

Geo geometry(const Params& p) {
  Geo g;
  g.W = (p.N >= p.S) ? (p.N - p.S) / p.L : 0;
  g.T = (p.N >= p.S) ? (p.N - p.S - g.W * p.L) : 0;
  g.C = g.W + (g.T > 0 ? 1 : 0);
  g.Wsel = std::max(g.W - 1, 0);
  return g;
}

// Element load: bf16 bit pattern (exact) or double (used by the finite-difference pin,
// which needs perturbations that bf16 cannot hold).
inline double ld(uint16_t h) {
  uint32_t u = static_cast<uint32_t>(h) << 16;
  float f;
  std::memcpy(&f, &u, sizeof f);
  return static_cast<double>(f);
}
inline double ld(double x) { return x; }

// element (b, h, t, c) of a [B, H, N, d] tensor
inline size_t at(const Params& p, int H, int b, int h, int t) {
  return ((static_cast<size_t>(b) * H + h) * p.N + t) * static_cast<size_t>(p.d);
}

// Number of leading windows that query chunk c sees only through their kept tokens.
// Attn-Fill 1/2: with the previous window kept as a sliding window (n_dense_prev = 1),
// chunk c sees windows 0..c-2 compressed.  Only scored windows can be compressed.
inline int n_compressed_for_chunk(const Params& p, const Geo& g, int c) {
  return std::min(std::max(c - p.n_dense_prev, 0), g.Wsel);
}

// May query position t attend key position j?  kept[j] != 0 iff j survived selection.
inline bool visible(const Params& p, const Geo& g, const uint8_t* kept, int t, int j) {
  if (j > t) return false;            // causal (Section 3.1)
  if (t < p.S) return true;           // sink queries: causal among the sinks
  if (j < p.S) return true;           // sinks are always seen
  const int c = (t - p.S) / p.L;      // chunk of the query
  const int w = (j - p.S) / p.L;      // window of the key
  if (w >= n_compressed_for_chunk(p, g, c)) return true;  // sliding window + own chunk
  return kept[j] != 0;                // compressed window: kept tokens only
}

void kept_mask(const Params& p, const Geo& g, const int32_t* idx, int b, int hkv,
               std::vector<uint8_t>& kept) {
  kept.assign(p.N, 0);
  const int32_t* ix = idx + (static_cast<size_t>(b) * p.Hkv + hkv) * g.Wsel * p.K;
  for (int i = 0; i < g.Wsel * p.K; ++i) kept[ix[i]] = 1;
}

// Eq. 3 for one query row: returns LSE, fills O[d].
template <class E>
double forward_row(const Params& p, const Geo& g, const E* Q, const E* K,
                   const E* V, const uint8_t* kept, int b, int hq, int t, double* O) {
  const int G = p.Hq / p.Hkv, hkv = hq / G, d = p.d;
  const E* q = Q + at(p, p.Hq, b, hq, t);
  std::vector<double> s(t + 1);
  std::vector<uint8_t> vis(t + 1);
  double m = -INFINITY;
  for (int j = 0; j <= t; ++j) {
    vis[j] = visible(p, g, kept, t, j);
    if (!vis[j]) continue;
    const E* k = K + at(p, p.Hkv, b, hkv, j);
    double acc = 0.0;
    for (int c = 0; c < d; ++c) acc += ld(q[c]) * ld(k[c]);
    s[j] = acc * p.scale;
    m = std::max(m, s[j]);
  }
  double denom = 0.0;
  for (int j = 0; j <= t; ++j)
    if (vis[j]) denom += std::exp(s[j] - m);
  const double lse = m + std::log(denom);
  for (int c = 0; c < d; ++c) O[c] = 0.0;
  for (int j = 0; j <= t; ++j) {
    if (!vis[j]) continue;
    const double a = std::exp(s[j] - lse);  // A_tj of Eq. 3
    const E* v = V + at(p, p.Hkv, b, hkv, j);
    for (int c = 0; c < d; ++c) O[c] += a * ld(v[c]);
  }
  return lse;
}

}  // namespace


// out = {W, T, C, Wsel}
extern "C" void lrsa_oracle_geometry(const Params* p, int32_t* out) {
  Geo g = geometry(*p);
  out[0] = g.W; out[1] = g.T; out[2] = g.C; out[3] = g.Wsel;
}

// Eq. 4-8.  Kt, Vt: bf16 bits [B,Hkv,N,d].  score: double [B,Hkv,Wsel,L].
// If score_k / score_v are non-null they receive the two terms of Eq. 8 separately.
template <class E>
static void score_impl(const Params* pp, const E* Kt, const E* Vt, double* score,
                       double* score_k, double* score_v) {
  const Params p = *pp;
  const Geo g = geometry(p);
  const int d = p.d, L = p.L;
#pragma omp parallel for collapse(3) schedule(dynamic)
  for (int b = 0; b < p.B; ++b)
    for (int h = 0; h < p.Hkv; ++h)
      for (int w = 0; w < g.Wsel; ++w) {
        const size_t out = ((static_cast<size_t>(b) * p.Hkv + h) * g.Wsel + w) * L;
        std::vector<double> mn(d), mx(d), spread(L), part(L);
        for (int which = 0; which < 2; ++which) {
          const E* Z = which == 0 ? Kt : Vt;
          // Eq. 4, Eq. 5: per-channel min / max over the sequence axis of window w+1
          for (int c = 0; c < d; ++c) { mn[c] = INFINITY; mx[c] = -INFINITY; }
          for (int t = p.S + (w + 1) * L; t < p.S + (w + 2) * L; ++t) {
            const E* z = Z + at(p, p.Hkv, b, h, t);
            for (int c = 0; c < d; ++c) {
              const double x = ld(z[c]);
              mn[c] = std::min(mn[c], x);
              mx[c] = std::max(mx[c], x);
            }
          }
          // Eq. 6 then Std over the channels of each token of window w
          for (int i = 0; i < L; ++i) {
            const E* z = Z + at(p, p.Hkv, b, h, p.S + w * L + i);
            std::vector<double> zb(d);
            double mean = 0.0;
            for (int c = 0; c < d; ++c) {
              const double range = mx[c] - mn[c];
              zb[c] = range == 0.0 ? 0.0 : (ld(z[c]) - mn[c]) / range;
              mean += zb[c];
            }
            mean /= d;
            double ss = 0.0;
            for (int c = 0; c < d; ++c) ss += (zb[c] - mean) * (zb[c] - mean);
            spread[i] = std::sqrt(ss / (d - p.ddof));
          }
          // Eq. 7: Softmax over the L tokens of the window
          double m = -INFINITY, denom = 0.0;
          for (int i = 0; i < L; ++i) m = std::max(m, spread[i]);
          for (int i = 0; i < L; ++i) denom += std::exp(spread[i] - m);
          for (int i = 0; i < L; ++i) part[i] = std::exp(spread[i] - m) / denom;
          double* side = which == 0 ? score_k : score_v;
          if (side) for (int i = 0; i < L; ++i) side[out + i] = part[i];
          // Eq. 8
          for (int i = 0; i < L; ++i) score[out + i] = (which == 0 ? 0.0 : score[out + i]) + part[i];
        }
      }
}

// Keep the K highest-scoring tokens of each scored window (text after Eq. 8).
// idx: int32 [B,Hkv,Wsel,K], absolute positions, ascending. Ties -> lower position.
extern "C" void lrsa_oracle_select(const Params* pp, const double* score, int32_t* idx) {
  const Params p = *pp;
  const Geo g = geometry(p);
  const int L = p.L;
  const long units = static_cast<long>(p.B) * p.Hkv * g.Wsel;
#pragma omp parallel for schedule(dynamic)
  for (long u = 0; u < units; ++u) {
    const int w = static_cast<int>(u % g.Wsel);
    const double* sc = score + u * L;
    std::vector<int> order(L);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return sc[a] > sc[b]; });
    std::vector<int> keep(order.begin(), order.begin() + p.K);
    std::sort(keep.begin(), keep.end());
    for (int i = 0; i < p.K; ++i) idx[u * p.K + i] = p.S + w * L + keep[i];
  }
}

// visibility of key j for query t of kv head (b,hkv): out[j] in {0,1}, j in [0,N)
extern "C" void lrsa_oracle_visible_row(const Params* pp, const int32_t* idx, int b, int hkv, int t,
                             uint8_t* out) {
  const Params p = *pp;
  const Geo g = geometry(p);
  std::vector<uint8_t> kept;
  kept_mask(p, g, idx, b, hkv, kept);
  for (int j = 0; j < p.N; ++j) out[j] = visible(p, g, kept.data(), t, j) ? 1 : 0;
}

// Forward (Eq. 3) for listed query rows. rows: int32 [n,3] = (b, hq, t).
// O: double [n,d]; LSE: double [n] (natural log).
template <class E>
static void fwd_rows_impl(const Params* pp, const E* Q, const E* K, const E* V,
                          const int32_t* idx, long n, const int32_t* rows, double* O, double* LSE) {
  const Params p = *pp;
  const Geo g = geometry(p);
  const int G = p.Hq / p.Hkv;
  std::vector<std::vector<uint8_t>> kept(static_cast<size_t>(p.B) * p.Hkv);
  for (int b = 0; b < p.B; ++b)
    for (int h = 0; h < p.Hkv; ++h) kept_mask(p, g, idx, b, h, kept[b * p.Hkv + h]);
#pragma omp parallel for schedule(dynamic, 4)
  for (long r = 0; r < n; ++r) {
    const int b = rows[3 * r], hq = rows[3 * r + 1], t = rows[3 * r + 2];
    LSE[r] = forward_row(p, g, Q, K, V, kept[b * p.Hkv + hq / G].data(), b, hq, t, O + r * p.d);
  }
}

// dQ for listed query rows. The row's own O and LSE are recomputed in fp64.
//   D_t = dO_t . O_t ;  P_tj = exp(s_tj - LSE_t) ;  dS_tj = P_tj (dO_t . v_j - D_t)
//   dQ_t = scale * sum_j dS_tj k_j
template <class E>
static void bwd_rows_impl(const Params* pp, const E* Q, const E* K, const E* V,
                          const E* dO, const int32_t* idx, long n, const int32_t* rows,
                          double* dQ) {
  const Params p = *pp;
  const Geo g = geometry(p);
  const int G = p.Hq / p.Hkv, d = p.d;
  std::vector<std::vector<uint8_t>> kept(static_cast<size_t>(p.B) * p.Hkv);
  for (int b = 0; b < p.B; ++b)
    for (int h = 0; h < p.Hkv; ++h) kept_mask(p, g, idx, b, h, kept[b * p.Hkv + h]);
#pragma omp parallel for schedule(dynamic, 4)
  for (long r = 0; r < n; ++r) {
    const int b = rows[3 * r], hq = rows[3 * r + 1], t = rows[3 * r + 2], hkv = hq / G;
    const uint8_t* kp = kept[b * p.Hkv + hkv].data();
    std::vector<double> O(d);
    const double lse = forward_row(p, g, Q, K, V, kp, b, hq, t, O.data());
    const E* q = Q + at(p, p.Hq, b, hq, t);
    const E* go = dO + at(p, p.Hq, b, hq, t);
    double D = 0.0;
    for (int c = 0; c < d; ++c) D += ld(go[c]) * O[c];
    double* out = dQ + r * d;
    for (int c = 0; c < d; ++c) out[c] = 0.0;
    for (int j = 0; j <= t; ++j) {
      if (!visible(p, g, kp, t, j)) continue;
      const E* k = K + at(p, p.Hkv, b, hkv, j);
      const E* v = V + at(p, p.Hkv, b, hkv, j);
      double s = 0.0, dP = 0.0;
      for (int c = 0; c < d; ++c) {
        s += ld(q[c]) * ld(k[c]);
        dP += ld(go[c]) * ld(v[c]);
      }
      const double P = std::exp(s * p.scale - lse);
      const double dS = P * (dP - D);
      for (int c = 0; c < d; ++c) out[c] += p.scale * dS * ld(k[c]);
    }
  }
}

// dK, dV for listed keys. keys: int32 [n,3] = (b, hkv, j).  dK, dV: double [n,d].
//   dV_j = sum_t P_tj dO_t ;  dK_j = scale * sum_t dS_tj q_t
// summed over every query head of the group and every query t that sees j.
template <class E>
static void bwd_keys_impl(const Params* pp, const E* Q, const E* K, const E* V,
                          const E* dO, const int32_t* idx, long n, const int32_t* keys,
                          double* dK, double* dV) {
  const Params p = *pp;
  const Geo g = geometry(p);
  const int G = p.Hq / p.Hkv, d = p.d;
  for (long r = 0; r < n * d; ++r) { dK[r] = 0.0; dV[r] = 0.0; }
  for (int b = 0; b < p.B; ++b)
    for (int hkv = 0; hkv < p.Hkv; ++hkv) {
      std::vector<long> mine;
      for (long r = 0; r < n; ++r)
        if (keys[3 * r] == b && keys[3 * r + 1] == hkv) mine.push_back(r);
      if (mine.empty()) continue;
      std::vector<uint8_t> kept;
      kept_mask(p, g, idx, b, hkv, kept);
      // which queries see at least one listed key
      std::vector<uint8_t> need(p.N, 0);
      for (long r : mine)
        for (int t = keys[3 * r + 2]; t < p.N; ++t)
          if (visible(p, g, kept.data(), t, keys[3 * r + 2])) need[t] = 1;
      // pass 1: LSE_t and D_t of those queries, for each head of the group
      std::vector<double> lse(static_cast<size_t>(G) * p.N, 0.0), Dt(static_cast<size_t>(G) * p.N, 0.0);
#pragma omp parallel for collapse(2) schedule(dynamic, 4)
      for (int gq = 0; gq < G; ++gq)
        for (int t = 0; t < p.N; ++t) {
          if (!need[t]) continue;
          const int hq = hkv * G + gq;
          std::vector<double> O(d);
          lse[static_cast<size_t>(gq) * p.N + t] = forward_row(p, g, Q, K, V, kept.data(), b, hq, t, O.data());
          const E* go = dO + at(p, p.Hq, b, hq, t);
          double D = 0.0;
          for (int c = 0; c < d; ++c) D += ld(go[c]) * O[c];
          Dt[static_cast<size_t>(gq) * p.N + t] = D;
        }
      // pass 2: one key at a time
#pragma omp parallel for schedule(dynamic, 1)
      for (size_t m = 0; m < mine.size(); ++m) {
        const long r = mine[m];
        const int j = keys[3 * r + 2];
        const E* k = K + at(p, p.Hkv, b, hkv, j);
        const E* v = V + at(p, p.Hkv, b, hkv, j);
        for (int gq = 0; gq < G; ++gq) {
          const int hq = hkv * G + gq;
          for (int t = j; t < p.N; ++t) {
            if (!visible(p, g, kept.data(), t, j)) continue;
            const E* q = Q + at(p, p.Hq, b, hq, t);
            const E* go = dO + at(p, p.Hq, b, hq, t);
            double s = 0.0, dP = 0.0;
            for (int c = 0; c < d; ++c) {
              s += ld(q[c]) * ld(k[c]);
              dP += ld(go[c]) * ld(v[c]);
            }
            const double P = std::exp(s * p.scale - lse[static_cast<size_t>(gq) * p.N + t]);
            const double dS = P * (dP - Dt[static_cast<size_t>(gq) * p.N + t]);
            for (int c = 0; c < d; ++c) {
              dV[r * d + c] += P * ld(go[c]);
              dK[r * d + c] += p.scale * dS * ld(q[c]);
            }
          }
        }
      }
    }
}

extern "C" int lrsa_oracle_num_threads() {
  int n = 1;
#pragma omp parallel
  {
#pragma omp single
    n =
#ifdef _OPENMP
        omp_get_num_threads();
#else
        1;
#endif
  }
  return n;
}


// C entry points: bf16-bit inputs (the parity path) and, suffixed _f64, double inputs.
#define LRSA_ORACLE_ENTRY(SUF, E)                                                                   \
  extern "C" void lrsa_oracle_score##SUF(const Params* p, const E* K, const E* V, double* score,    \
                                         double* sk, double* sv) {                                  \
    score_impl<E>(p, K, V, score, sk, sv);                                                          \
  }                                                                                                 \
  extern "C" void lrsa_oracle_fwd_rows##SUF(const Params* p, const E* Q, const E* K, const E* V,    \
                                            const int32_t* idx, long n, const int32_t* rows,        \
                                            double* O, double* LSE) {                               \
    fwd_rows_impl<E>(p, Q, K, V, idx, n, rows, O, LSE);                                             \
  }                                                                                                 \
  extern "C" void lrsa_oracle_bwd_rows##SUF(const Params* p, const E* Q, const E* K, const E* V,    \
                                            const E* dO, const int32_t* idx, long n,                \
                                            const int32_t* rows, double* dQ) {                      \
    bwd_rows_impl<E>(p, Q, K, V, dO, idx, n, rows, dQ);                                             \
  }                                                                                                 \
  extern "C" void lrsa_oracle_bwd_keys##SUF(const Params* p, const E* Q, const E* K, const E* V,    \
                                            const E* dO, const int32_t* idx, long n,                \
                                            const int32_t* keys, double* dK, double* dV) {          \
    bwd_keys_impl<E>(p, Q, K, V, dO, idx, n, keys, dK, dV);                                         \
  }
LRSA_ORACLE_ENTRY(, uint16_t)
LRSA_ORACLE_ENTRY(_f64, double)
