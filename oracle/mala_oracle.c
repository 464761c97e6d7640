/*
 * MALA reference oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, fp64 CPU statement of what the MassAlloc Attention (MALA) hot path
 * computes, written from the paper's Methodology section (Eqs. 1-4), Algorithm 1
 * (forward), Algorithm 2 (backward), the "Fused decoding execution" paragraph of the
 * appendix (split-KV decode) and Proposition 1.  It shares no code with the CUDA path and
 * is imported only by the tests, by the smoke check and by the benchmark's CPU-baseline
 * leg.  Nothing here is blocked, fused or reordered beyond what the algorithms state.
 *
 * Notation follows the paper for ONE query head and its key/value head:
 *   Q [N_q, d], K, V [N_k, d] row-major doubles (bf16 inputs widened exactly by the caller),
 *   s_qk = scale * <Q_q, K_k>  (the paper absorbs the scale into Q; here it multiplies the
 *   fp64 dot product), natural exp/log, blocks I_i of B_q query rows, J_j of B_k keys,
 *   L_q = q + 1 for equal-length causal attention (zero-based q), L = N_k otherwise,
 *   theta_q = log(tau / L_q)  (-inf when tau = 0, so nothing is ever skipped).
 *
 * Mask byte per tile: 0 = not legal (never visited, not counted), 1 = legal and skipped,
 * 2 = legal and retained.  crit holds the tile criterion C (skip iff C < 0), NaN if illegal.
 *
 * Readings of points the paper leaves open (each also listed in the design notes):
 *   - strict '<' in Eq. 3 / Eq. 4: C == 0 retains;
 *   - a row with no legal key in the tile does not constrain it (text after Eq. 3);
 *   - a row with a legal key and an empty retained set has log-ratio +inf (text after Eq. 3);
 *   - the test uses the state left by the previously retained tile (Alg. 1 line order);
 *   - a retained tile updates every row of the block;  exp(-inf - (-inf)) := 0;
 *   - backward follows Algorithm 2 literally with the saved lse and D = rowsum(O o dO); it is
 *     not the derivative of the forward result;
 *   - decode: rows of the tile are the query heads that share the KV head, L = N_k,
 *     num_splits contiguous tile-aligned chunks, tiles visited newest to oldest in a split.
 *
 * Pins (tests/test_oracle_pins.py): brute force from Eqs. 1-2 with explicit key sets,
 * textbook softmax, finite differences of the dense forward, closed forms (Q = 0, one boosted
 * key), single tile == dense, B_q = B_k = 1, Proposition 1, nesting, tau-monotonicity,
 * split-merge == unsplit at tau = 0.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define MASK_ILLEGAL 0
#define MASK_SKIPPED 1
#define MASK_RETAINED 2

int mala_oracle_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

static double dot(const double* a, const double* b, int d) {
  double s = 0.0;
  for (int c = 0; c < d; ++c) s += a[c] * b[c];
  return s;
}

int mala_oracle_decode_merge(const double* o_part, const double* lse_part, int num_splits, int R, int d,
                             double* o, double* lse);

/* Visible-key count L_q (Section 2.1): the number of keys the query may attend to.  Causal: the queries are
 * the LAST N_q of N_k positions (off = N_k - N_q >= 0), query row q sits at position q + off and sees the keys
 * 0 .. q + off, so L_q = q + 1 + off (q + 1 for equal lengths, N_k for the single decode query); otherwise N_k. */
static double visible_count(int q, int Nk, int causal, int off) { return causal ? (double)(q + 1 + off) : (double)Nk; }

/* theta_q = log(tau / L_q); tau = 0 gives -inf. */
static double log_threshold(double tau, double L) { return tau > 0.0 ? log(tau / L) : -INFINITY; }

/* ------------------------------------------------------------------------------------------
 * FullAttn, the plain definition: p = softmax over legal keys, o = sum p v, lse = log sum exp s.
 * Rows q_begin <= q < q_end of one head.  (Section 2.3: tau -> 0 recovers this.)
 * ---------------------------------------------------------------------------------------- */
int mala_oracle_dense_fwd(const double* Q, const double* K, const double* V, int Nq, int Nk, int d,
                          double scale, int causal, int q_begin, int q_end, double* O, double* lse) {
  if (causal && Nq > Nk) return -1;
#pragma omp parallel for schedule(dynamic, 16)
  for (int q = q_begin; q < q_end; ++q) {
    int kmax = causal ? q + 1 + (Nk - Nq) : Nk;
    double* s = (double*)malloc(sizeof(double) * (size_t)kmax);
    double m = -INFINITY;
    for (int k = 0; k < kmax; ++k) {
      s[k] = scale * dot(Q + (size_t)q * d, K + (size_t)k * d, d);
      if (s[k] > m) m = s[k];
    }
    double Z = 0.0;
    for (int k = 0; k < kmax; ++k) Z += exp(s[k] - m);
    double* o = O + (size_t)q * d;
    for (int c = 0; c < d; ++c) o[c] = 0.0;
    for (int k = 0; k < kmax; ++k) {
      double p = exp(s[k] - m) / Z;
      for (int c = 0; c < d; ++c) o[c] += p * V[(size_t)k * d + c];
    }
    lse[q] = m + log(Z);
    free(s);
  }
  return 0;
}

/* FullAttn backward, closed forms row by row:
 *   dV = P^T dO, dP = dO V^T, D_q = <o_q, do_q>, dS = P o (dP - D), dQ = scale dS K, dK = scale dS^T Q.
 * Serial over q (dK, dV are accumulated); meant for small shapes. */
int mala_oracle_dense_bwd(const double* Q, const double* K, const double* V, const double* dO, int N, int d,
                          double scale, int causal, double* dQ, double* dK, double* dV) {
  double* O = (double*)malloc(sizeof(double) * (size_t)N * d);
  double* lse = (double*)malloc(sizeof(double) * (size_t)N);
  mala_oracle_dense_fwd(Q, K, V, N, N, d, scale, causal, 0, N, O, lse);
  memset(dQ, 0, sizeof(double) * (size_t)N * d);
  memset(dK, 0, sizeof(double) * (size_t)N * d);
  memset(dV, 0, sizeof(double) * (size_t)N * d);
  for (int q = 0; q < N; ++q) {
    int kmax = causal ? q + 1 : N;
    double D = dot(O + (size_t)q * d, dO + (size_t)q * d, d);
    for (int k = 0; k < kmax; ++k) {
      double s = scale * dot(Q + (size_t)q * d, K + (size_t)k * d, d);
      double p = exp(s - lse[q]);
      double dP = dot(dO + (size_t)q * d, V + (size_t)k * d, d);
      double dS = p * (dP - D);
      for (int c = 0; c < d; ++c) {
        dV[(size_t)k * d + c] += p * dO[(size_t)q * d + c];
        dQ[(size_t)q * d + c] += scale * dS * K[(size_t)k * d + c];
        dK[(size_t)k * d + c] += scale * dS * Q[(size_t)q * d + c];
      }
    }
  }
  free(O);
  free(lse);
  return 0;
}

/* ------------------------------------------------------------------------------------------
 * Algorithm 1 (forward): the key blocks j_hi, j_hi - 1, ..., j_lo of query block i, in that order, on the
 * running state m, l, acc (rows of the block).  S, mt: scratch.  mask, crit: [Tr*Tc] or NULL.
 * ---------------------------------------------------------------------------------------- */
static void fwd_block_range(const double* Q, const double* K, const double* V, int N, int Nk, int d, double scale,
                            double tau, int Bq, int Bk, int causal, int shift, int i, int j_lo, int j_hi, int Tc,
                            double* m, double* l, double* acc, double* S, double* mt, uint8_t* mask, double* crit) {
  const int off = Nk - N; /* N queries (the last N positions) against Nk keys */
  /* query block i holds the rows q with i*Bq <= q + shift < (i+1)*Bq (shift = 0: blocks count from the first row) */
  const int q0 = (i * Bq - shift > 0 ? i * Bq - shift : 0);
  const int q1 = ((i + 1) * Bq - shift < N ? (i + 1) * Bq - shift : N), rows = q1 - q0;
  for (int j = j_hi; j >= j_lo; --j) { /* descending from the diagonal toward earlier keys */
    const int k0 = j * Bk, cols = (k0 + Bk <= Nk ? Bk : Nk - k0);
    /* a tile with no legal key for any row is not visited */
    if (causal && k0 > q0 + rows - 1 + off) {
      if (mask) mask[(size_t)i * Tc + j] = MASK_ILLEGAL;
      if (crit) crit[(size_t)i * Tc + j] = NAN;
      continue;
    }
    /* S_ij = Q_i K_j^T with the causal mask (-inf) */
    double C = -INFINITY;
    for (int r = 0; r < rows; ++r) {
      const int q = q0 + r;
      double mrow = -INFINITY;
      int legal = 0;
      for (int c = 0; c < cols; ++c) {
        const int k = k0 + c;
        double s = -INFINITY;
        if (!causal || k <= q + off) { s = scale * dot(Q + (size_t)q * d, K + (size_t)k * d, d); legal = 1; }
        S[(size_t)r * Bk + c] = s;
        if (s > mrow) mrow = s;
      }
      mt[r] = mrow; /* rowmax(S_ij) */
      /* row criterion: rowmax - m - log l - log(tau/L), state BEFORE this tile (Eq. 3) */
      double cq;
      if (!legal) cq = -INFINITY;             /* does not constrain retention */
      else if (l[r] == 0.0) cq = INFINITY;    /* nothing retained yet: log-ratio is +inf */
      else cq = mrow - (m[r] + log(l[r])) - log_threshold(tau, visible_count(q, Nk, causal, off));
      if (cq > C) C = cq;
    }
    const int retain = !(C < 0.0); /* skip only if every relevant row is strictly below */
    if (mask) mask[(size_t)i * Tc + j] = retain ? MASK_RETAINED : MASK_SKIPPED;
    if (crit) crit[(size_t)i * Tc + j] = C;
    if (!retain) continue; /* m, l, O unchanged */
    /* online-softmax update of every row of the block (Alg. 1, retained branch) */
    for (int r = 0; r < rows; ++r) {
      const double mnew = (m[r] > mt[r] ? m[r] : mt[r]);
      if (mnew == -INFINITY) continue; /* still empty: stays (-inf, 0, 0) */
      const double alpha = (m[r] == -INFINITY ? 0.0 : exp(m[r] - mnew));
      double lt = 0.0;
      for (int c = 0; c < d; ++c) acc[(size_t)r * d + c] *= alpha;
      for (int c = 0; c < cols; ++c) {
        const double s = S[(size_t)r * Bk + c];
        if (s == -INFINITY) continue;
        const double p = exp(s - mnew);
        lt += p;
        const double* v = V + (size_t)(k0 + c) * d;
        for (int e = 0; e < d; ++e) acc[(size_t)r * d + e] += p * v[e];
      }
      l[r] = alpha * l[r] + lt;
      m[r] = mnew;
    }
  }
}

/* Algorithm 1 for the listed query blocks of one head (blocks == NULL: all).
 * O [N,d], lse [N]: rows of the listed blocks are written.  mask, crit: [Tr*Tc], rows of the
 * listed blocks are written (may be NULL).
 * shift (0 <= shift < Bq): the query blocks are laid out as if shift more rows preceded the first one, i.e. block i
 * holds the rows q with i*Bq <= q + shift < (i+1)*Bq and there are ceil((N + shift)/Bq) blocks.  With
 * shift = (Nk - N) mod Bq the blocks of a chunk of queries coincide with the blocks those rows have in the
 * equal-length problem over all Nk positions (the result depends on the partition).
 * num_splits > 1: the key blocks are cut into num_splits contiguous ranges of ceil(Tc / num_splits) blocks; every
 * range runs the rule on its own running state (its test sees the range's PARTIAL normalizer, as in "Fused decoding
 * execution") and the ranges' results (o_s, lse_s) are merged by lse = log sum_s exp(lse_s),
 * o = sum_s exp(lse_s - lse) o_s.  A range that holds no legal key of a row contributes nothing to it. */
int mala_oracle_fwd_split(const double* Q, const double* K, const double* V, int N, int Nk, int d, double scale,
                          double tau, int Bq, int Bk, int causal, int num_splits, int shift, int n_blocks,
                          const int* blocks, double* O, double* lse, uint8_t* mask, double* crit) {
  if (N <= 0 || (causal && Nk < N) || d <= 0 || Bq <= 0 || Bk <= 0 || num_splits <= 0 || !(tau >= 0.0)) return -1;
  if (shift < 0 || shift >= Bq) return -1;
  const int Tr = (N + shift + Bq - 1) / Bq, Tc = (Nk + Bk - 1) / Bk;
  const int tps = (Tc + num_splits - 1) / num_splits;
  const int nb = blocks ? n_blocks : Tr;
#pragma omp parallel for schedule(dynamic, 1)
  for (int u = 0; u < nb; ++u) {
    const int i = blocks ? blocks[u] : (Tr - 1 - u); /* long blocks first when running all */
    const int q0 = (i * Bq - shift > 0 ? i * Bq - shift : 0);
    const int q1 = ((i + 1) * Bq - shift < N ? (i + 1) * Bq - shift : N), rows = q1 - q0;
    /* Alg. 1: O_i = 0, l_i = 0, m_i = -inf; L_i from positions */
    double* m = (double*)malloc(sizeof(double) * rows);
    double* l = (double*)malloc(sizeof(double) * rows);
    double* acc = (double*)malloc(sizeof(double) * (size_t)rows * d);
    double* S = (double*)malloc(sizeof(double) * (size_t)rows * Bk);
    double* mt = (double*)malloc(sizeof(double) * rows);
    double* o_s = (double*)malloc(sizeof(double) * (size_t)num_splits * rows * d);
    double* lse_s = (double*)malloc(sizeof(double) * (size_t)num_splits * rows);
    for (int s = 0; s < num_splits; ++s) {
      for (int r = 0; r < rows; ++r) { m[r] = -INFINITY; l[r] = 0.0; }
      memset(acc, 0, sizeof(double) * (size_t)rows * d);
      const int j_lo = s * tps, j_hi = ((s + 1) * tps < Tc ? (s + 1) * tps : Tc) - 1;
      fwd_block_range(Q, K, V, N, Nk, d, scale, tau, Bq, Bk, causal, shift, i, j_lo, j_hi, Tc, m, l, acc, S, mt, mask,
                      crit);
      /* O_i <- diag(l)^-1 O_i,  l_i <- m_i + log l_i */
      for (int r = 0; r < rows; ++r) {
        lse_s[(size_t)s * rows + r] = (l[r] == 0.0 ? -INFINITY : m[r] + log(l[r]));
        for (int c = 0; c < d; ++c)
          o_s[((size_t)s * rows + r) * d + c] = (l[r] == 0.0 ? 0.0 : acc[(size_t)r * d + c] / l[r]);
      }
    }
    if (num_splits == 1) {
      for (int r = 0; r < rows; ++r) {
        for (int c = 0; c < d; ++c) O[(size_t)(q0 + r) * d + c] = acc[(size_t)r * d + c] / l[r];
        lse[q0 + r] = m[r] + log(l[r]);
      }
    } else {
      mala_oracle_decode_merge(o_s, lse_s, num_splits, rows, d, O + (size_t)q0 * d, lse + q0);
    }
    free(m); free(l); free(acc); free(S); free(mt); free(o_s); free(lse_s);
  }
  return 0;
}

int mala_oracle_fwd(const double* Q, const double* K, const double* V, int N, int Nk, int d, double scale, double tau,
                    int Bq, int Bk, int causal, int n_blocks, const int* blocks, double* O, double* lse,
                    uint8_t* mask, double* crit) {
  return mala_oracle_fwd_split(Q, K, V, N, Nk, d, scale, tau, Bq, Bk, causal, 1, 0, n_blocks, blocks, O, lse, mask,
                               crit);
}

/* D = rowsum(O o dO) (Alg. 2, the term subtracted from dP). */
int mala_oracle_bwd_D(const double* O, const double* dO, int N, int d, double* D) {
  for (int q = 0; q < N; ++q) D[q] = dot(O + (size_t)q * d, dO + (size_t)q * d, d);
  return 0;
}

/* One backward tile (key block j, query block i) of Algorithm 2.  Computes S_ji = K_j Q_i^T with
 * the causal mask, the offline test of Eq. 4 against the saved lse, and, if retained, P and dS
 * (both [Bk x Bq], row = key, column b = query q0 + b).  Returns 1 if retained; *C_out is the tile
 * criterion max over valid causal entries of (s - lse_q - theta_q).
 * shift: query block i holds the rows q with i*Bq <= q + shift < (i+1)*Bq, as in the forward pass. */
static int bwd_tile(const double* Q, const double* K, const double* V, const double* dO, const double* lse,
                    const double* D, int N, int Nk, int d, double scale, double tau, int Bq, int Bk, int causal, int shift,
                    int j, int i, double* S, double* P, double* dS, double* C_out) {
  const int off = Nk - N;
  const int k0 = j * Bk, cols_k = (k0 + Bk <= Nk ? Bk : Nk - k0);
  const int q0 = (i * Bq - shift > 0 ? i * Bq - shift : 0);
  const int q1 = ((i + 1) * Bq - shift < N ? (i + 1) * Bq - shift : N), cols_q = q1 - q0;
  double C = -INFINITY;
  for (int a = 0; a < cols_k; ++a) {
    const int k = k0 + a;
    for (int b = 0; b < cols_q; ++b) {
      const int q = q0 + b;
      double s = -INFINITY;
      if (!causal || k <= q + off) {
        s = scale * dot(K + (size_t)k * d, Q + (size_t)q * d, d);
        const double c = s - lse[q] - log_threshold(tau, visible_count(q, Nk, causal, off));
        if (c > C) C = c;
      }
      S[(size_t)a * Bq + b] = s;
    }
  }
  *C_out = C;
  if (C < 0.0) return 0; /* every valid entry strictly below: skip (the diagonal tile may be skipped) */
  for (int a = 0; a < cols_k; ++a) {
    const int k = k0 + a;
    for (int b = 0; b < cols_q; ++b) {
      const int q = q0 + b;
      const double s = S[(size_t)a * Bq + b];
      if (s == -INFINITY) { P[(size_t)a * Bq + b] = 0.0; dS[(size_t)a * Bq + b] = 0.0; continue; }
      const double p = exp(s - lse[q]);                                   /* P_ji = exp(S_ji - lse^T) */
      const double dP = dot(V + (size_t)k * d, dO + (size_t)q * d, d);     /* dP_ji = V_j dO_i^T */
      P[(size_t)a * Bq + b] = p;
      dS[(size_t)a * Bq + b] = p * (dP - D[q]);                            /* dS = P o (dP - D^T) */
    }
  }
  return 1;
}

/* Algorithm 2 for the listed key blocks of one query head (key_blocks == NULL: all).
 * dK, dV [N,d]: rows of the listed key blocks are overwritten with this head's contribution.
 * dQ [N,d] or NULL: contributions of the listed key blocks are ADDED (atomically).
 * mask, crit [Tc*Tr] indexed [j*Tr + i] (may be NULL); Tr = ceil((N + shift)/Bq), shift as in the
 * forward pass (0 <= shift < Bq). */
int mala_oracle_bwd(const double* Q, const double* K, const double* V, const double* dO, const double* lse,
                    const double* D, int N, int Nk, int d, double scale, double tau, int Bq, int Bk, int causal,
                    int shift, int n_blocks, const int* key_blocks, double* dQ, double* dK, double* dV, uint8_t* mask,
                    double* crit) {
  if (N <= 0 || (causal && Nk < N) || d <= 0 || Bq <= 0 || Bk <= 0 || !(tau >= 0.0)) return -1;
  if (shift < 0 || shift >= Bq) return -1;
  const int off = Nk - N;
  const int Tr = (N + shift + Bq - 1) / Bq, Tc = (Nk + Bk - 1) / Bk;
  const int nb = key_blocks ? n_blocks : Tc;
#pragma omp parallel for schedule(dynamic, 1)
  for (int u = 0; u < nb; ++u) {
    const int j = key_blocks ? key_blocks[u] : u;
    const int k0 = j * Bk, cols_k = (k0 + Bk <= Nk ? Bk : Nk - k0);
    double* S = (double*)malloc(sizeof(double) * (size_t)Bk * Bq);
    double* P = (double*)malloc(sizeof(double) * (size_t)Bk * Bq);
    double* dS = (double*)malloc(sizeof(double) * (size_t)Bk * Bq);
    /* dK_j = 0, dV_j = 0 */
    for (int a = 0; a < cols_k; ++a)
      for (int c = 0; c < d; ++c) { dK[(size_t)(k0 + a) * d + c] = 0.0; dV[(size_t)(k0 + a) * d + c] = 0.0; }
    for (int i = 0; i < Tr; ++i) { /* ascending; legal tiles start at the diagonal */
      const int q0 = (i * Bq - shift > 0 ? i * Bq - shift : 0);
      const int q1 = ((i + 1) * Bq - shift < N ? (i + 1) * Bq - shift : N), cols_q = q1 - q0;
      if (causal && k0 > q0 + cols_q - 1 + off) { /* no valid causal entry */
        if (mask) mask[(size_t)j * Tr + i] = MASK_ILLEGAL;
        if (crit) crit[(size_t)j * Tr + i] = NAN;
        continue;
      }
      double C;
      const int retain = bwd_tile(Q, K, V, dO, lse, D, N, Nk, d, scale, tau, Bq, Bk, causal, shift, j, i, S, P, dS, &C);
      if (mask) mask[(size_t)j * Tr + i] = retain ? MASK_RETAINED : MASK_SKIPPED;
      if (crit) crit[(size_t)j * Tr + i] = C;
      if (!retain) continue;
      for (int a = 0; a < cols_k; ++a) {
        for (int b = 0; b < cols_q; ++b) {
          const double p = P[(size_t)a * Bq + b], ds = dS[(size_t)a * Bq + b];
          if (p == 0.0 && ds == 0.0) continue;
          const double* doq = dO + (size_t)(q0 + b) * d;
          const double* qq = Q + (size_t)(q0 + b) * d;
          for (int c = 0; c < d; ++c) {
            dV[(size_t)(k0 + a) * d + c] += p * doq[c];          /* dV_j += P_ji dO_i */
            dK[(size_t)(k0 + a) * d + c] += scale * ds * qq[c];  /* dK_j += dS_ji Q_i (scale un-absorbed) */
          }
          if (dQ) {
            const double* kk = K + (size_t)(k0 + a) * d;
            for (int c = 0; c < d; ++c) {
              const double add = scale * ds * kk[c];             /* dQ_i += dS_ji^T K_j */
#pragma omp atomic
              dQ[(size_t)(q0 + b) * d + c] += add;
            }
          }
        }
      }
    }
    free(S); free(P); free(dS);
  }
  return 0;
}

/* dQ rows of the listed query blocks of one head: the same tiles as Algorithm 2, gathered per
 * query block (all legal key blocks j), so that sampled blocks can be checked at full size. */
int mala_oracle_bwd_dq(const double* Q, const double* K, const double* V, const double* dO, const double* lse,
                       const double* D, int N, int Nk, int d, double scale, double tau, int Bq, int Bk, int causal,
                       int shift, int n_blocks, const int* query_blocks, double* dQ) {
  if (N <= 0 || (causal && Nk < N) || d <= 0 || Bq <= 0 || Bk <= 0 || !(tau >= 0.0)) return -1;
  if (shift < 0 || shift >= Bq) return -1;
  const int off = Nk - N;
  const int Tr = (N + shift + Bq - 1) / Bq, Tc = (Nk + Bk - 1) / Bk;
  const int nb = query_blocks ? n_blocks : Tr;
#pragma omp parallel for schedule(dynamic, 1)
  for (int u = 0; u < nb; ++u) {
    const int i = query_blocks ? query_blocks[u] : (Tr - 1 - u);
    const int q0 = (i * Bq - shift > 0 ? i * Bq - shift : 0);
    const int q1 = ((i + 1) * Bq - shift < N ? (i + 1) * Bq - shift : N), cols_q = q1 - q0;
    double* S = (double*)malloc(sizeof(double) * (size_t)Bk * Bq);
    double* P = (double*)malloc(sizeof(double) * (size_t)Bk * Bq);
    double* dS = (double*)malloc(sizeof(double) * (size_t)Bk * Bq);
    for (int b = 0; b < cols_q; ++b)
      for (int c = 0; c < d; ++c) dQ[(size_t)(q0 + b) * d + c] = 0.0;
    for (int j = 0; j < Tc; ++j) {
      const int k0 = j * Bk, cols_k = (k0 + Bk <= Nk ? Bk : Nk - k0);
      if (causal && k0 > q0 + cols_q - 1 + off) continue;
      double C;
      if (!bwd_tile(Q, K, V, dO, lse, D, N, Nk, d, scale, tau, Bq, Bk, causal, shift, j, i, S, P, dS, &C)) continue;
      for (int a = 0; a < cols_k; ++a)
        for (int b = 0; b < cols_q; ++b) {
          const double ds = dS[(size_t)a * Bq + b];
          if (ds == 0.0) continue;
          const double* kk = K + (size_t)(k0 + a) * d;
          for (int c = 0; c < d; ++c) dQ[(size_t)(q0 + b) * d + c] += scale * ds * kk[c];
        }
    }
    free(S); free(P); free(dS);
  }
  return 0;
}

/* ------------------------------------------------------------------------------------------
 * Split-KV decode ("Fused decoding execution"): R query rows (the query heads sharing this KV
 * head; one new token each) against N_k cached keys.  L = N_k for every row, every key legal.
 * The key range is cut into num_splits contiguous chunks of chunk = ceil(ceil(N_k/S)/B_k)*B_k
 * keys; each split runs the forward rule on its chunk, newest tile first, with its own m, l,
 * testing against its PARTIAL normalizer.  o_part [S][R][d] (normalized per split),
 * lse_part [S][R] (-inf for an empty split), mask/crit [S][tiles_per_split].
 * ---------------------------------------------------------------------------------------- */
int mala_oracle_decode_tiles_per_split(int Nk, int num_splits, int Bk) {
  const int per = (Nk + num_splits - 1) / num_splits;
  return (per + Bk - 1) / Bk;
}

/* The same with the chunk length given (tps tiles of B_k keys per split) instead of derived from N_k: a batch
 * of sequences of different lengths shares one layout of splits over the key positions, and a sequence shorter
 * than a split's first position leaves that split empty.  N_k = 0 is allowed (every split empty). */
int mala_oracle_decode_splits_rows(const double* Q, const double* K, const double* V, int R, int Nk, int d,
                                   double scale, double tau, int num_splits, int tps, int Bk, const int* vis,
                                   double* o_part, double* lse_part, uint8_t* mask, double* crit);

int mala_oracle_decode_splits_tps(const double* Q, const double* K, const double* V, int R, int Nk, int d,
                                  double scale, double tau, int num_splits, int tps, int Bk, double* o_part,
                                  double* lse_part, uint8_t* mask, double* crit) {
  return mala_oracle_decode_splits_rows(Q, K, V, R, Nk, d, scale, tau, num_splits, tps, Bk, NULL, o_part, lse_part,
                                        mask, crit);
}

/* The general form: row r sees the keys 0 .. vis[r]-1 only and has L = vis[r] (vis == NULL: every row sees all
 * N_k keys).  This is a decode step with several new tokens per sequence, whose keys already sit at the end of the
 * cache: the token at position x sees x + 1 keys.  A row that sees no key of a tile does not constrain it
 * (Section 2.2, as for the causal diagonal); a row that has seen no key at all stays (0, -inf). */
int mala_oracle_decode_splits_rows(const double* Q, const double* K, const double* V, int R, int Nk, int d,
                                   double scale, double tau, int num_splits, int tps, int Bk, const int* vis,
                                   double* o_part, double* lse_part, uint8_t* mask, double* crit) {
  if (R <= 0 || Nk < 0 || d <= 0 || num_splits <= 0 || tps <= 0 || Bk <= 0 || !(tau >= 0.0)) return -1;
  const int chunk = tps * Bk;
#pragma omp parallel for schedule(dynamic, 1)
  for (int s = 0; s < num_splits; ++s) {
    const int lo = s * chunk, hi = (lo + chunk <= Nk ? lo + chunk : Nk);
    double* m = (double*)malloc(sizeof(double) * R);
    double* l = (double*)malloc(sizeof(double) * R);
    double* acc = (double*)calloc((size_t)R * d, sizeof(double));
    double* S = (double*)malloc(sizeof(double) * (size_t)R * Bk);
    double* mt = (double*)malloc(sizeof(double) * R);
    for (int r = 0; r < R; ++r) { m[r] = -INFINITY; l[r] = 0.0; }
    for (int t = tps - 1; t >= 0; --t) {
      const int k0 = lo + t * Bk;
      if (k0 >= hi) { /* tile beyond the end of the cache: not legal */
        if (mask) mask[(size_t)s * tps + t] = MASK_ILLEGAL;
        if (crit) crit[(size_t)s * tps + t] = NAN;
        continue;
      }
      const int cols = (k0 + Bk <= hi ? Bk : hi - k0);
      double C = -INFINITY;
      for (int r = 0; r < R; ++r) {
        const int seen = vis ? vis[r] : Nk; /* keys visible to this row = its L */
        double mrow = -INFINITY;
        int legal = 0;
        for (int c = 0; c < cols; ++c) {
          double sc = -INFINITY;
          if (k0 + c < seen) { sc = scale * dot(Q + (size_t)r * d, K + (size_t)(k0 + c) * d, d); legal = 1; }
          S[(size_t)r * Bk + c] = sc;
          if (sc > mrow) mrow = sc;
        }
        mt[r] = mrow;
        double cq;
        if (!legal) cq = -INFINITY;
        else if (l[r] == 0.0) cq = INFINITY;
        else cq = mrow - (m[r] + log(l[r])) - log_threshold(tau, (double)seen);
        if (cq > C) C = cq;
      }
      const int retain = !(C < 0.0);
      if (mask) mask[(size_t)s * tps + t] = retain ? MASK_RETAINED : MASK_SKIPPED;
      if (crit) crit[(size_t)s * tps + t] = C;
      if (!retain) continue;
      for (int r = 0; r < R; ++r) {
        const double mnew = (m[r] > mt[r] ? m[r] : mt[r]);
        if (mnew == -INFINITY) continue; /* has seen no key yet */
        const double alpha = (m[r] == -INFINITY ? 0.0 : exp(m[r] - mnew));
        double lt = 0.0;
        for (int e = 0; e < d; ++e) acc[(size_t)r * d + e] *= alpha;
        for (int c = 0; c < cols; ++c) {
          if (S[(size_t)r * Bk + c] == -INFINITY) continue;
          const double p = exp(S[(size_t)r * Bk + c] - mnew);
          lt += p;
          const double* v = V + (size_t)(k0 + c) * d;
          for (int e = 0; e < d; ++e) acc[(size_t)r * d + e] += p * v[e];
        }
        l[r] = alpha * l[r] + lt;
        m[r] = mnew;
      }
    }
    for (int r = 0; r < R; ++r) {
      if (l[r] == 0.0) { /* empty split */
        for (int e = 0; e < d; ++e) o_part[((size_t)s * R + r) * d + e] = 0.0;
        lse_part[(size_t)s * R + r] = -INFINITY;
      } else {
        for (int e = 0; e < d; ++e) o_part[((size_t)s * R + r) * d + e] = acc[(size_t)r * d + e] / l[r];
        lse_part[(size_t)s * R + r] = m[r] + log(l[r]);
      }
    }
    free(m); free(l); free(acc); free(S); free(mt);
  }
  return 0;
}

int mala_oracle_decode_splits(const double* Q, const double* K, const double* V, int R, int Nk, int d,
                              double scale, double tau, int num_splits, int Bk, double* o_part,
                              double* lse_part, uint8_t* mask, double* crit) {
  if (Nk <= 0 || num_splits <= 0 || Bk <= 0) return -1;
  return mala_oracle_decode_splits_tps(Q, K, V, R, Nk, d, scale, tau, num_splits,
                                       mala_oracle_decode_tiles_per_split(Nk, num_splits, Bk), Bk, o_part, lse_part,
                                       mask, crit);
}

/* Normalizer-aware reduction of the split partials:
 *   lse = log sum_s exp(lse_s),  o = sum_s exp(lse_s - lse) o_s. */
int mala_oracle_decode_merge(const double* o_part, const double* lse_part, int num_splits, int R, int d,
                             double* o, double* lse) {
  for (int r = 0; r < R; ++r) {
    double mx = -INFINITY;
    for (int s = 0; s < num_splits; ++s)
      if (lse_part[(size_t)s * R + r] > mx) mx = lse_part[(size_t)s * R + r];
    double Z = 0.0;
    for (int s = 0; s < num_splits; ++s)
      if (lse_part[(size_t)s * R + r] != -INFINITY) Z += exp(lse_part[(size_t)s * R + r] - mx);
    lse[r] = mx + log(Z);
    for (int e = 0; e < d; ++e) o[(size_t)r * d + e] = 0.0;
    for (int s = 0; s < num_splits; ++s) {
      if (lse_part[(size_t)s * R + r] == -INFINITY) continue;
      const double w = exp(lse_part[(size_t)s * R + r] - lse[r]);
      for (int e = 0; e < d; ++e) o[(size_t)r * d + e] += w * o_part[((size_t)s * R + r) * d + e];
    }
  }
  return 0;
}
