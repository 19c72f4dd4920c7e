/*
 * BlossomRec block-level fused sparse attention -- fp64 CPU ORACLE.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, obviously-correct
 * restatement of the paper's equations that the CUDA library is checked
 * against.  It shares no code, header, table or helper with the CUDA path and
 * must never be called from the product path (only from tests, the smoke
 * check and the benchmark's cpu_baseline / reference arm).
 *
 * What it computes, per (batch n, head h), all in double precision, in the
 * paper's order (section "Block-Level Fused Sparse Attention Mechanism"):
 *
 *   block splitting      Eq. 8  with l = s = l' = Bk (non-overlapping blocks,
 *                               0-based half-open, ragged last block kept)
 *   block compression    Eq. 9  with phi := mean over the valid keys of a block, or a learnable
 *                               softmax pooling over the block's positions (phi_weight)
 *   importance scoring   Eq. 10 softmax over the strictly-past live blocks,
 *                               logits scaled by sm_scale
 *   score sharing        Eq. 12 rule (sum of the probabilities of everyone who
 *                               shares one selection) applied to the queries
 *                               of a query block
 *   top-k selection      Eq. 13 own block always kept, ties -> lower index; per query block
 *                               (summed probabilities) or per query position (as printed:
 *                               blossom_oracle_select_pq)
 *   overlapping blocks   Eq. 8 with l, s != Bk and the score remap of Eq. 11
 *                               (blossom_oracle_select_cmp; per query position:
 *                               blossom_oracle_select_pq_cmp)
 *   selected-KV attention Eq. 14 + Eq. 16 (via Eq. 1 with the causal mask)
 *   window attention     Eq. 15 first case (|i-j| < w), causal side, Eq. 17
 *   power-law mask       Eq. 15 all three cases (stis_mode 1), causal side:
 *                               window, block-index distance a power of two,
 *                               the last blk positions
 *   gate combine         Eq. 19 with alpha_h = sigmoid(a[h][0] - a[h][1]), or Eq. 18's
 *                               input-dependent gate with a one-layer F_o (gate_mode 1)
 *   backward             chain rule through Eq. 19, Eq. 16/17 and Eq. 1 with
 *                        the selection frozen (top-k is piecewise constant)
 *
 * Parity pins (tests/test_oracle_*.py): explicit dense-mask evaluation of
 * Eq. 1, softmax/causality invariants, reductions to dense causal attention,
 * constructed selections with known answers, an independent numpy scorer,
 * finite differences, and Table 5's key-budget closed form.  The readings of
 * the paper that no printed value pins (selection per query block, phi = mean
 * or a softmax pooling, scalar gate or one-layer F_o, own block always
 * selected, which compression blocks a position may score) are "parity
 * unpinned by the paper": the pins above fix the arithmetic of each reading,
 * not the choice of the reading.
 *
 * Layout: q, k, v, out*, dout, dq, dk, dv are contiguous [B][H][L][D] doubles;
 * lse is [2][B][H][L] (0 = long-term branch, 1 = short-term branch), natural
 * log of the sum of exp(sm_scale * q.k); gate is [H][2]; idx is
 * [B][H][M][topk] int32 ascending, -1 padded; scores is [B][H][M][M].
 * seq_lens[n] = number of valid (right-aligned) positions; NULL = all valid.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

static int n_blocks(int L, int Bk) { return (L + Bk - 1) / Bk; }
static int imin(int a, int b) { return a < b ? a : b; }
static int imax(int a, int b) { return a > b ? a : b; }

int blossom_oracle_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* Eq. 9's learnable summary, in the one-layer form this oracle takes: a softmax pooling over the
 * positions of a block, k~ = sum_i w_i k_i / sum_i w_i over the block's valid keys with
 * w_i = exp(phi[i]), i the position inside the block.  phi == NULL (or all zeros) is the mean. */
static double phi_weight(const double *phi, int i) { return phi ? exp(phi[i]) : 1.0; }

/* ---- selection for one (n,h) unit: Eq. 8-10, 12, 13 --------------------- */
/* causal = 1: the candidates of query block b are the live blocks before it; causal = 0 (a
 * bidirectional encoder): every live block but b itself.  The own block is always kept. */
static void select_unit(int L, int D, int Bk, int topk, double scale, int pad0, int causal,
                        const double *q, const double *k, const double *phi, int32_t *idx,
                        double *scores /* [M][M] or NULL */) {
  const int M = n_blocks(L, Bk);
  double *ktil = (double *)calloc((size_t)M * D, sizeof(double));
  int *live = (int *)calloc((size_t)M, sizeof(int));
  double *S = (double *)malloc(sizeof(double) * (size_t)M);
  double *z = (double *)malloc(sizeof(double) * (size_t)M);
  char *taken = (char *)malloc((size_t)M);
  int *chosen = (int *)malloc(sizeof(int) * (size_t)(topk + 1));

  /* Eq. 8 + Eq. 9: block j = [j*Bk, min((j+1)*Bk, L)), summary = mean of its valid keys */
  for (int j = 0; j < M; ++j) {
    int lo = imax(j * Bk, pad0), hi = imin((j + 1) * Bk, L), cnt = 0;
    double wsum = 0.0;
    for (int p = lo; p < hi; ++p) {
      const double w = phi_weight(phi, p - j * Bk);
      for (int c = 0; c < D; ++c) ktil[(size_t)j * D + c] += w * k[(size_t)p * D + c];
      wsum += w;
      ++cnt;
    }
    live[j] = cnt > 0;
    if (cnt > 0)
      for (int c = 0; c < D; ++c) ktil[(size_t)j * D + c] /= wsum;
  }

  for (int b = 0; b < M; ++b) {
    int32_t *row = idx + (size_t)b * topk;
    for (int s = 0; s < topk; ++s) row[s] = -1;
    if (scores)
      for (int j = 0; j < M; ++j) scores[(size_t)b * M + j] = 0.0;
    int qlo = imax(b * Bk, pad0), qhi = imin((b + 1) * Bk, L);
    if (qlo >= qhi) continue; /* query block holds only padding */

    const int hi = causal ? b : M; /* candidates: j < hi, j != b */
    int ncand = 0;
    for (int j = 0; j < hi; ++j) {
      S[j] = 0.0;
      if (j != b) ncand += live[j];
    }
    /* Eq. 10 per query, summed over the queries that share the selection (Eq. 12's rule) */
    if (ncand > 0) {
      for (int t = qlo; t < qhi; ++t) {
        double mx = -INFINITY;
        for (int j = 0; j < hi; ++j) {
          if (!live[j] || j == b) continue;
          double acc = 0.0;
          for (int c = 0; c < D; ++c) acc += q[(size_t)t * D + c] * ktil[(size_t)j * D + c];
          z[j] = scale * acc;
          if (z[j] > mx) mx = z[j];
        }
        double den = 0.0;
        for (int j = 0; j < hi; ++j)
          if (live[j] && j != b) den += exp(z[j] - mx);
        for (int j = 0; j < hi; ++j)
          if (live[j] && j != b) S[j] += exp(z[j] - mx) / den;
      }
    }
    if (scores)
      for (int j = 0; j < hi; ++j)
        if (live[j] && j != b) scores[(size_t)b * M + j] = S[j];

    /* Eq. 13: the own block plus the (topk-1) best candidates, ties to the lower index */
    int want = imin(topk - 1, ncand), nch = 0;
    memset(taken, 0, (size_t)M);
    for (int s = 0; s < want; ++s) {
      int best = -1;
      for (int j = 0; j < hi; ++j) {
        if (!live[j] || j == b || taken[j]) continue;
        if (best < 0 || S[j] > S[best]) best = j; /* strict > keeps the lower index on ties */
      }
      taken[best] = 1;
      chosen[nch++] = best;
    }
    /* ascending order: walk the flags, the own block in its place */
    taken[b] = 1;
    int s = 0;
    for (int j = 0; j < M; ++j)
      if (taken[j]) row[s++] = j;
  }
  free(ktil); free(live); free(S); free(z); free(taken); free(chosen);
}

int blossom_oracle_select(int B, int H, int L, int D, int Bk, int topk, int causal, double scale,
                          const double *q, const double *k, const int32_t *seq_lens,
                          const double *phi /* [Bk] or NULL */, int32_t *idx, double *scores) {
  if (B < 1 || H < 1 || L < 1 || D < 1 || Bk < 1 || topk < 1) return 1;
  const int M = n_blocks(L, Bk);
#pragma omp parallel for collapse(2) schedule(dynamic)
  for (int n = 0; n < B; ++n)
    for (int h = 0; h < H; ++h) {
      size_t u = (size_t)n * H + h;
      int len = seq_lens ? seq_lens[n] : L;
      if (len < 0) len = 0;
      if (len > L) len = L;
      select_unit(L, D, Bk, topk, scale, L - len, causal, q + u * L * D, k + u * L * D, phi,
                  idx + u * M * topk, scores ? scores + u * M * M : NULL);
    }
  return 0;
}

/* ---- selection per query position for one (n,h) unit: Eq. 8-10, 13 as printed -----------
 * The paper selects for each query position: query t (in query block b = t / Bk) takes the softmax
 * of Eq. 10 over the live blocks j < b (strictly-past blocks, whose summaries hold no key after
 * t) and keeps the top_k - 1 largest probabilities, ties to the lower index, plus its own block b.
 * idx is [L][topk] (one row per position, -1 rows for padding), probs [L][M] optional. */
static void select_unit_pq(int L, int D, int Bk, int topk, double scale, int pad0,
                           const double *q, const double *k, const double *phi, int32_t *idx, double *probs) {
  const int M = n_blocks(L, Bk);
  double *ktil = (double *)calloc((size_t)M * D, sizeof(double));
  int *live = (int *)calloc((size_t)M, sizeof(int));
  double *P = (double *)malloc(sizeof(double) * (size_t)M);
  char *taken = (char *)malloc((size_t)M);
  for (int j = 0; j < M; ++j) { /* Eq. 8 + Eq. 9 */
    int lo = imax(j * Bk, pad0), hi = imin((j + 1) * Bk, L), cnt = 0;
    double wsum = 0.0;
    for (int p = lo; p < hi; ++p) {
      const double w = phi_weight(phi, p - j * Bk);
      for (int c = 0; c < D; ++c) ktil[(size_t)j * D + c] += w * k[(size_t)p * D + c];
      wsum += w;
      ++cnt;
    }
    live[j] = cnt > 0;
    if (cnt > 0)
      for (int c = 0; c < D; ++c) ktil[(size_t)j * D + c] /= wsum;
  }
  for (int t = 0; t < L; ++t) {
    int32_t *row = idx + (size_t)t * topk;
    for (int s = 0; s < topk; ++s) row[s] = -1;
    if (probs)
      for (int j = 0; j < M; ++j) probs[(size_t)t * M + j] = 0.0;
    if (t < pad0) continue;
    const int b = t / Bk;
    int ncand = 0;
    double mx = -INFINITY;
    for (int j = 0; j < b; ++j) {
      P[j] = 0.0;
      if (!live[j]) continue;
      ++ncand;
      double acc = 0.0;
      for (int c = 0; c < D; ++c) acc += q[(size_t)t * D + c] * ktil[(size_t)j * D + c];
      P[j] = scale * acc;
      if (P[j] > mx) mx = P[j];
    }
    double den = 0.0;
    for (int j = 0; j < b; ++j)
      if (live[j]) den += exp(P[j] - mx);
    for (int j = 0; j < b; ++j) /* Eq. 10 */
      P[j] = live[j] ? exp(P[j] - mx) / den : 0.0;
    if (probs)
      for (int j = 0; j < b; ++j) probs[(size_t)t * M + j] = P[j];
    int want = imin(topk - 1, ncand); /* Eq. 13 */
    memset(taken, 0, (size_t)M);
    for (int s = 0; s < want; ++s) {
      int best = -1;
      for (int j = 0; j < b; ++j) {
        if (!live[j] || taken[j]) continue;
        if (best < 0 || P[j] > P[best]) best = j;
      }
      taken[best] = 1;
    }
    int s = 0;
    for (int j = 0; j < b; ++j)
      if (taken[j]) row[s++] = j;
    row[s++] = b;
  }
  free(ktil); free(live); free(P); free(taken);
}

int blossom_oracle_select_pq(int B, int H, int L, int D, int Bk, int topk, double scale,
                             const double *q, const double *k, const int32_t *seq_lens,
                             const double *phi /* [Bk] or NULL */, int32_t *idx, double *probs) {
  if (B < 1 || H < 1 || L < 1 || D < 1 || Bk < 1 || topk < 1) return 1;
  const int M = n_blocks(L, Bk);
#pragma omp parallel for collapse(2) schedule(dynamic)
  for (int n = 0; n < B; ++n)
    for (int h = 0; h < H; ++h) {
      size_t u = (size_t)n * H + h;
      int len = seq_lens ? seq_lens[n] : L;
      if (len < 0) len = 0;
      if (len > L) len = L;
      select_unit_pq(L, D, Bk, topk, scale, L - len, q + u * L * D, k + u * L * D, phi,
                     idx + u * L * topk, probs ? probs + u * L * M : NULL);
    }
  return 0;
}

/* ---- selection with overlapping compression blocks for one (n,h) unit: Eq. 8-11, 13 -------
 * Compression blocks K_i = positions [s i, s i + l), i = 0 .. Mc-1, Mc = floor((L - l)/s) + 1
 * (Eq. 8, 0-based; none if L < l), summarised by the mean of their valid keys (Eq. 9 with
 * phi := mean).  For query block b (selection blocks of lp = Bk positions) the candidates are the
 * live compression blocks that end before the query block starts, s i + l <= lp b; Eq. 10 per
 * query over the candidates, summed over the block's valid queries (Eq. 12's rule).  Eq. 11 maps
 * the compression scores to selection blocks j < b,
 *   S_ltis[j] = sum_{m < lp/s} sum_{n < l/s} S_cmp[(lp/s) j - m - n],
 * terms whose index is out of range or not a candidate being zero.  Eq. 13 as in select_unit.
 * scores_cmp [M][Mc] and scores [M][M] are optional outputs. */
static void select_unit_cmp(int L, int D, int Bk, int topk, int l, int s, double scale, int pad0,
                            const double *q, const double *k, const double *phi, int32_t *idx,
                            double *scores, double *scores_cmp) {
  const int M = n_blocks(L, Bk);
  const int Mc = L >= l ? (L - l) / s + 1 : 0;
  const int rs = Bk / s, rl = l / s;
  double *ktil = (double *)calloc((size_t)(Mc > 0 ? Mc : 1) * D, sizeof(double));
  int *livec = (int *)calloc((size_t)(Mc > 0 ? Mc : 1), sizeof(int));
  double *Sc = (double *)malloc(sizeof(double) * (size_t)(Mc > 0 ? Mc : 1));
  double *z = (double *)malloc(sizeof(double) * (size_t)(Mc > 0 ? Mc : 1));
  double *S = (double *)malloc(sizeof(double) * (size_t)M);
  char *taken = (char *)malloc((size_t)M);

  for (int i = 0; i < Mc; ++i) { /* Eq. 8 + Eq. 9 */
    int lo = imax(i * s, pad0), hi = i * s + l, cnt = 0;
    double wsum = 0.0;
    for (int p = lo; p < hi; ++p) {
      const double w = phi_weight(phi, p - i * s);
      for (int c = 0; c < D; ++c) ktil[(size_t)i * D + c] += w * k[(size_t)p * D + c];
      wsum += w;
      ++cnt;
    }
    livec[i] = cnt > 0;
    if (cnt > 0)
      for (int c = 0; c < D; ++c) ktil[(size_t)i * D + c] /= wsum;
  }

  for (int b = 0; b < M; ++b) {
    int32_t *row = idx + (size_t)b * topk;
    for (int e = 0; e < topk; ++e) row[e] = -1;
    if (scores)
      for (int j = 0; j < M; ++j) scores[(size_t)b * M + j] = 0.0;
    if (scores_cmp)
      for (int i = 0; i < Mc; ++i) scores_cmp[(size_t)b * Mc + i] = 0.0;
    int qlo = imax(b * Bk, pad0), qhi = imin((b + 1) * Bk, L);
    if (qlo >= qhi) continue; /* query block holds only padding */

    /* candidates: compression blocks 0 .. nc-1 end before the query block starts */
    int nc = 0;
    while (nc < Mc && nc * s + l <= b * Bk) ++nc;
    int ncand = 0;
    for (int i = 0; i < nc; ++i) {
      Sc[i] = 0.0;
      ncand += livec[i];
    }
    if (ncand > 0) { /* Eq. 10 per query, summed over the block's valid queries */
      for (int t = qlo; t < qhi; ++t) {
        double mx = -INFINITY;
        for (int i = 0; i < nc; ++i) {
          if (!livec[i]) continue;
          double acc = 0.0;
          for (int c = 0; c < D; ++c) acc += q[(size_t)t * D + c] * ktil[(size_t)i * D + c];
          z[i] = scale * acc;
          if (z[i] > mx) mx = z[i];
        }
        double den = 0.0;
        for (int i = 0; i < nc; ++i)
          if (livec[i]) den += exp(z[i] - mx);
        for (int i = 0; i < nc; ++i)
          if (livec[i]) Sc[i] += exp(z[i] - mx) / den;
      }
    }
    if (scores_cmp)
      for (int i = 0; i < nc; ++i)
        if (livec[i]) scores_cmp[(size_t)b * Mc + i] = Sc[i];

    /* Eq. 11, and which past selection blocks hold a valid key */
    int nlive = 0;
    for (int j = 0; j < b; ++j) {
      double acc = 0.0;
      for (int m = 0; m < rs; ++m)
        for (int n = 0; n < rl; ++n) {
          int i = rs * j - m - n;
          if (i >= 0 && i < nc && livec[i]) acc += Sc[i];
        }
      S[j] = acc;
      taken[j] = 0;
      if (imin((j + 1) * Bk, L) > imax(j * Bk, pad0)) {
        ++nlive;
        if (scores) scores[(size_t)b * M + j] = acc;
      } else {
        taken[j] = 2; /* not selectable */
      }
    }
    /* Eq. 13: the own block plus the (topk-1) best past blocks, ties to the lower index */
    int want = imin(topk - 1, nlive);
    for (int e = 0; e < want; ++e) {
      int best = -1;
      for (int j = 0; j < b; ++j) {
        if (taken[j]) continue;
        if (best < 0 || S[j] > S[best]) best = j;
      }
      taken[best] = 1;
    }
    int e = 0;
    for (int j = 0; j < b; ++j)
      if (taken[j] == 1) row[e++] = j;
    row[e++] = b;
  }
  free(ktil); free(livec); free(Sc); free(z); free(S); free(taken);
}

int blossom_oracle_select_cmp(int B, int H, int L, int D, int Bk, int topk, int l, int s,
                              double scale, const double *q, const double *k,
                              const int32_t *seq_lens, const double *phi /* [l] or NULL */,
                              int32_t *idx, double *scores, double *scores_cmp) {
  if (B < 1 || H < 1 || L < 1 || D < 1 || Bk < 1 || topk < 1) return 1;
  if (l < 1 || s < 1 || l % s || Bk % s) return 1;
  const int M = n_blocks(L, Bk);
  const int Mc = L >= l ? (L - l) / s + 1 : 0;
#pragma omp parallel for collapse(2) schedule(dynamic)
  for (int n = 0; n < B; ++n)
    for (int h = 0; h < H; ++h) {
      size_t u = (size_t)n * H + h;
      int len = seq_lens ? seq_lens[n] : L;
      if (len < 0) len = 0;
      if (len > L) len = L;
      select_unit_cmp(L, D, Bk, topk, l, s, scale, L - len, q + u * L * D, k + u * L * D, phi,
                      idx + u * M * topk, scores ? scores + u * M * M : NULL,
                      scores_cmp ? scores_cmp + u * M * Mc : NULL);
    }
  return 0;
}

/* ---- selection per query position through overlapping compression blocks ---- */
/* Eq. 8-11 and Eq. 13 as printed (one selection per position): position t, in selection block
 * b = t / Bk, scores the live compression blocks that end before its block starts (the rule of
 * the per-block selection above, so no summary holds a key the position must not see), takes its
 * own softmax over them (Eq. 10), maps the probabilities onto the selection blocks j < b with
 * Eq. 11, and keeps its own block plus the top-(k-1) selectable past blocks, ties to the lower
 * index.  scores, if given, receives the mapped scores [L][M] (zero where not selectable). */
static void select_unit_pq_cmp(int L, int D, int Bk, int topk, int l, int s, double scale, int pad0,
                               const double *q, const double *k, const double *phi, int32_t *idx,
                               double *scores) {
  const int M = n_blocks(L, Bk);
  const int Mc = L >= l ? (L - l) / s + 1 : 0;
  const int rs = Bk / s, rl = l / s;
  double *ktil = (double *)calloc((size_t)(Mc > 0 ? Mc : 1) * D, sizeof(double));
  int *livec = (int *)calloc((size_t)(Mc > 0 ? Mc : 1), sizeof(int));
  double *P = (double *)malloc(sizeof(double) * (size_t)(Mc > 0 ? Mc : 1));
  double *S = (double *)malloc(sizeof(double) * (size_t)M);
  char *taken = (char *)malloc((size_t)M);
  for (int i = 0; i < Mc; ++i) { /* Eq. 8 + Eq. 9 */
    int lo = imax(i * s, pad0), hi = i * s + l, cnt = 0;
    double wsum = 0.0;
    for (int p = lo; p < hi; ++p) {
      const double w = phi_weight(phi, p - i * s);
      for (int c = 0; c < D; ++c) ktil[(size_t)i * D + c] += w * k[(size_t)p * D + c];
      wsum += w;
      ++cnt;
    }
    livec[i] = cnt > 0;
    if (cnt > 0)
      for (int c = 0; c < D; ++c) ktil[(size_t)i * D + c] /= wsum;
  }
  for (int t = 0; t < L; ++t) {
    int32_t *row = idx + (size_t)t * topk;
    for (int e = 0; e < topk; ++e) row[e] = -1;
    if (scores)
      for (int j = 0; j < M; ++j) scores[(size_t)t * M + j] = 0.0;
    if (t < pad0) continue;
    const int b = t / Bk;
    int nc = 0; /* compression blocks 0 .. nc-1 end before block b starts */
    while (nc < Mc && nc * s + l <= b * Bk) ++nc;
    double mx = -INFINITY;
    int ncand = 0;
    for (int i = 0; i < nc; ++i) {
      P[i] = 0.0;
      if (!livec[i]) continue;
      ++ncand;
      double acc = 0.0;
      for (int c = 0; c < D; ++c) acc += q[(size_t)t * D + c] * ktil[(size_t)i * D + c];
      P[i] = scale * acc;
      if (P[i] > mx) mx = P[i];
    }
    if (ncand > 0) { /* Eq. 10 */
      double den = 0.0;
      for (int i = 0; i < nc; ++i)
        if (livec[i]) den += exp(P[i] - mx);
      for (int i = 0; i < nc; ++i) P[i] = livec[i] ? exp(P[i] - mx) / den : 0.0;
    }
    int nlive = 0;
    for (int j = 0; j < b; ++j) { /* Eq. 11 */
      double acc = 0.0;
      for (int m = 0; m < rs; ++m)
        for (int n = 0; n < rl; ++n) {
          int i = rs * j - m - n;
          if (i >= 0 && i < nc && livec[i]) acc += P[i];
        }
      S[j] = acc;
      taken[j] = 0;
      if (imin((j + 1) * Bk, L) > imax(j * Bk, pad0)) {
        ++nlive;
        if (scores) scores[(size_t)t * M + j] = acc;
      } else {
        taken[j] = 2; /* not selectable */
      }
    }
    int want = imin(topk - 1, nlive); /* Eq. 13 */
    for (int e = 0; e < want; ++e) {
      int best = -1;
      for (int j = 0; j < b; ++j) {
        if (taken[j]) continue;
        if (best < 0 || S[j] > S[best]) best = j;
      }
      taken[best] = 1;
    }
    int e = 0;
    for (int j = 0; j < b; ++j)
      if (taken[j] == 1) row[e++] = j;
    row[e++] = b;
  }
  free(ktil); free(livec); free(P); free(S); free(taken);
}

int blossom_oracle_select_pq_cmp(int B, int H, int L, int D, int Bk, int topk, int l, int s,
                                 double scale, const double *q, const double *k,
                                 const int32_t *seq_lens, const double *phi /* [l] or NULL */,
                                 int32_t *idx /* [B][H][L][topk] */, double *scores /* [B][H][L][M] or NULL */) {
  if (B < 1 || H < 1 || L < 1 || D < 1 || Bk < 1 || topk < 1) return 1;
  if (l < 1 || s < 1 || l % s || Bk % s) return 1;
  const int M = n_blocks(L, Bk);
#pragma omp parallel for collapse(2) schedule(dynamic)
  for (int n = 0; n < B; ++n)
    for (int h = 0; h < H; ++h) {
      size_t u = (size_t)n * H + h;
      int len = seq_lens ? seq_lens[n] : L;
      if (len < 0) len = 0;
      if (len > L) len = L;
      select_unit_pq_cmp(L, D, Bk, topk, l, s, scale, L - len, q + u * L * D, k + u * L * D, phi,
                         idx + u * (size_t)L * topk, scores ? scores + u * (size_t)L * M : NULL);
    }
  return 0;
}

/* ---- one softmax-attention row over an explicit key list: Eq. 1 ---------- */
/* keys[0..nk) are key positions; writes out[D], returns lse (0 and zeros if nk == 0) */
static double attend_row(int D, double scale, const double *qt, const double *k, const double *v,
                         const int *keys, int nk, double *sbuf, double *out) {
  for (int c = 0; c < D; ++c) out[c] = 0.0;
  if (nk == 0) return 0.0;
  double mx = -INFINITY;
  for (int i = 0; i < nk; ++i) {
    const double *kp = k + (size_t)keys[i] * D;
    double acc = 0.0;
    for (int c = 0; c < D; ++c) acc += qt[c] * kp[c];
    sbuf[i] = scale * acc;
    if (sbuf[i] > mx) mx = sbuf[i];
  }
  double den = 0.0;
  for (int i = 0; i < nk; ++i) den += exp(sbuf[i] - mx);
  for (int i = 0; i < nk; ++i) {
    double p = exp(sbuf[i] - mx) / den;
    const double *vp = v + (size_t)keys[i] * D;
    for (int c = 0; c < D; ++c) out[c] += p * vp[c];
  }
  return mx + log(den);
}

/* key list of the long-term branch for query t (Eq. 14 + causal mask): valid p <= t inside the
 * selected blocks of t's query block */
static int ltis_keys(int L, int Bk, int topk, int pad0, int causal, const int32_t *row, int t, int *keys) {
  int nk = 0;
  const int M = n_blocks(L, Bk);
  for (int s = 0; s < topk; ++s) {
    int j = row[s];
    if (j < 0 || j >= M) continue;
    int lo = imax(j * Bk, pad0), hi = imin((j + 1) * Bk, L);
    if (causal) hi = imin(hi, t + 1);
    for (int p = lo; p < hi; ++p) keys[nk++] = p;
  }
  return nk;
}

/* Eq. 15, one (query i, key j) pair: 1 if the short-term branch lets i attend to j.
 *   mode 0: the window alone, |i - j| < w;
 *   mode 1: the paper's power-law mask: the window, or the block-index distance
 *           |floor(i/blk) - floor(j/blk)| is 2^r for some integer r >= 0, or j is one of
 *           the last blk positions of the sequence array. */
static int stis_mask(int mode, int w, int blk, int L, int i, int j) {
  int d = i > j ? i - j : j - i;
  if (d < w) return 1;
  if (mode == 0) return 0;
  int bd = i / blk - j / blk;
  if (bd < 0) bd = -bd;
  if (bd >= 1 && (bd & (bd - 1)) == 0) return 1; /* a power of two */
  if (j >= L - blk) return 1;
  return 0;
}

/* key list of the short-term branch: Eq. 15 restricted to the causal side (p <= t) and to the
 * valid (non-padding) positions */
static int stis_keys(int mode, int w, int blk, int L, int pad0, int causal, int t, int *keys) {
  int nk = 0;
  for (int p = pad0; p <= (causal ? t : L - 1); ++p)
    if (stis_mask(mode, w, blk, L, t, p)) keys[nk++] = p;
  return nk;
}

static double sigmoid(double x) { return 1.0 / (1.0 + exp(-x)); }

/* per_query = 0: idx is [B][H][M][topk], one row per query block; 1: [B][H][L][topk], one row per
 * query position (Eq. 13 as printed) */
/* gate_mode = 0: gate is [H][2], alpha_h = sigmoid(a[h][0] - a[h][1]) for the whole head;
 * 1: the input-dependent gate of Eq. 18 with a one-layer F_o: gate is [H][2 D + 1] = (w_lt[D],
 * w_st[D], b) and alpha_t = sigmoid(<w_lt, O_lt,t> + <w_st, O_st,t> + b), one weight per token
 * and head, broadcast over the head's channels in Eq. 19 */
int blossom_oracle_forward(int B, int H, int L, int D, int Bk, int topk, int window, int stis_mode,
                           int stis_blk, int per_query, int gate_mode, int causal, double scale,
                           const double *q, const double *k, const double *v, const double *gate,
                           const int32_t *seq_lens, const int32_t *idx, double *out,
                           double *out_lt, double *out_st, double *lse) {
  if (B < 1 || H < 1 || L < 1 || D < 1 || Bk < 1 || topk < 1 || window < 1) return 1;
  if (stis_mode < 0 || stis_mode > 1 || stis_blk < 1) return 1;
  const int M = n_blocks(L, Bk);
  const size_t BHL = (size_t)B * H * L;
#pragma omp parallel for collapse(2) schedule(dynamic)
  for (int n = 0; n < B; ++n)
    for (int h = 0; h < H; ++h) {
      size_t u = (size_t)n * H + h;
      int len = seq_lens ? seq_lens[n] : L;
      if (len < 0) len = 0;
      if (len > L) len = L;
      const int pad0 = L - len;
      const double *qu = q + u * L * D, *ku = k + u * L * D, *vu = v + u * L * D;
      const int GW = 2 * D + 1;
      const double alpha_h = gate_mode ? 0.0 : sigmoid(gate[h * 2 + 0] - gate[h * 2 + 1]); /* Eq. 18 reduced to a scalar */
      int *keys = (int *)malloc(sizeof(int) * (size_t)(L + 1));
      double *sbuf = (double *)malloc(sizeof(double) * (size_t)(L + 1));
      double *oL = (double *)malloc(sizeof(double) * (size_t)D);
      double *oS = (double *)malloc(sizeof(double) * (size_t)D);
      for (int t = 0; t < L; ++t) {
        size_t ro = (u * L + t) * (size_t)D;
        double lL = 0.0, lS = 0.0;
        if (t < pad0) {
          for (int c = 0; c < D; ++c) oL[c] = oS[c] = 0.0;
        } else {
          const int32_t *row = per_query ? idx + (u * L + (size_t)t) * topk
                                         : idx + (u * M + (size_t)(t / Bk)) * topk;
          int nk = ltis_keys(L, Bk, topk, pad0, causal, row, t, keys);
          lL = attend_row(D, scale, qu + (size_t)t * D, ku, vu, keys, nk, sbuf, oL); /* Eq. 16 */
          nk = stis_keys(stis_mode, window, stis_blk, L, pad0, causal, t, keys);
          lS = attend_row(D, scale, qu + (size_t)t * D, ku, vu, keys, nk, sbuf, oS); /* Eq. 17 */
        }
        double alpha = alpha_h;
        if (gate_mode) { /* Eq. 18: F_o of the concatenated branch outputs, then the sigmoid */
          double a = gate[h * GW + 2 * D];
          for (int c = 0; c < D; ++c) a += gate[h * GW + c] * oL[c] + gate[h * GW + D + c] * oS[c];
          alpha = sigmoid(a);
        }
        for (int c = 0; c < D; ++c) {
          if (out_lt) out_lt[ro + c] = oL[c];
          if (out_st) out_st[ro + c] = oS[c];
          out[ro + c] = alpha * oL[c] + (1.0 - alpha) * oS[c]; /* Eq. 19 */
        }
        if (lse) {
          lse[u * L + t] = lL;
          lse[BHL + u * L + t] = lS;
        }
      }
      free(keys); free(sbuf); free(oL); free(oS);
    }
  return 0;
}

/* gradient of one softmax-attention row (Eq. 1) given upstream g = dL/d(out row):
 *   P = exp(s - lse); dV_p += P g; dP = <g, v_p>; delta = <g, o>; dS = P (dP - delta);
 *   dq += scale dS k_p; dK_p += scale dS q */
static void attend_row_bwd(int D, double scale, const double *qt, const double *k, const double *v,
                           const int *keys, int nk, double lse, const double *o, const double *g,
                           double *dqt, double *dk, double *dv) {
  if (nk == 0) return;
  double delta = 0.0;
  for (int c = 0; c < D; ++c) delta += g[c] * o[c];
  for (int i = 0; i < nk; ++i) {
    const size_t p = (size_t)keys[i];
    const double *kp = k + p * D, *vp = v + p * D;
    double acc = 0.0, dP = 0.0;
    for (int c = 0; c < D; ++c) {
      acc += qt[c] * kp[c];
      dP += g[c] * vp[c];
    }
    double P = exp(scale * acc - lse);
    double dS = P * (dP - delta);
    for (int c = 0; c < D; ++c) {
      dv[p * D + c] += P * g[c];
      dqt[c] += scale * dS * kp[c];
      dk[p * D + c] += scale * dS * qt[c];
    }
  }
}

int blossom_oracle_backward(int B, int H, int L, int D, int Bk, int topk, int window, int stis_mode,
                            int stis_blk, int per_query, int gate_mode, int causal, double scale,
                            const double *q, const double *k, const double *v, const double *gate,
                            const int32_t *seq_lens, const int32_t *idx, const double *out_lt,
                            const double *out_st, const double *lse, const double *dout,
                            double *dq, double *dk, double *dv, double *dgate) {
  if (B < 1 || H < 1 || L < 1 || D < 1 || Bk < 1 || topk < 1 || window < 1) return 1;
  if (stis_mode < 0 || stis_mode > 1 || stis_blk < 1) return 1;
  const int M = n_blocks(L, Bk);
  const size_t BHL = (size_t)B * H * L;
  const int GW = 2 * D + 1;
  /* per (n, h): d alpha (scalar gate) or the gradient of (w_lt, w_st, b) (input-dependent gate) */
  double *dalpha_unit = (double *)calloc((size_t)B * H * (gate_mode ? GW : 1), sizeof(double));
  memset(dq, 0, sizeof(double) * BHL * D);
  memset(dk, 0, sizeof(double) * BHL * D);
  memset(dv, 0, sizeof(double) * BHL * D);
#pragma omp parallel for collapse(2) schedule(dynamic)
  for (int n = 0; n < B; ++n)
    for (int h = 0; h < H; ++h) {
      size_t u = (size_t)n * H + h;
      int len = seq_lens ? seq_lens[n] : L;
      if (len < 0) len = 0;
      if (len > L) len = L;
      const int pad0 = L - len;
      const double *qu = q + u * L * D, *ku = k + u * L * D, *vu = v + u * L * D;
      double *dqu = dq + u * L * D, *dku = dk + u * L * D, *dvu = dv + u * L * D;
      const double alpha_h = gate_mode ? 0.0 : sigmoid(gate[h * 2 + 0] - gate[h * 2 + 1]);
      int *keys = (int *)malloc(sizeof(int) * (size_t)(L + 1));
      double *gL = (double *)malloc(sizeof(double) * (size_t)D);
      double *gS = (double *)malloc(sizeof(double) * (size_t)D);
      double dalpha = 0.0;
      double *dw = gate_mode ? dalpha_unit + u * GW : NULL;
      for (int t = pad0; t < L; ++t) {
        size_t ro = (u * L + t) * (size_t)D;
        double alpha = alpha_h, da_t = 0.0; /* d loss / d alpha of this row */
        for (int c = 0; c < D; ++c) da_t += dout[ro + c] * (out_lt[ro + c] - out_st[ro + c]); /* Eq. 19 */
        dalpha += da_t;
        double cpre = 0.0; /* d loss / d (pre-activation of the gate) of this row */
        if (gate_mode) {
          double a = gate[h * GW + 2 * D];
          for (int c = 0; c < D; ++c)
            a += gate[h * GW + c] * out_lt[ro + c] + gate[h * GW + D + c] * out_st[ro + c];
          alpha = sigmoid(a);
          cpre = alpha * (1.0 - alpha) * da_t;
          for (int c = 0; c < D; ++c) { /* F_o's parameters */
            dw[c] += cpre * out_lt[ro + c];
            dw[D + c] += cpre * out_st[ro + c];
          }
          dw[2 * D] += cpre;
        }
        for (int c = 0; c < D; ++c) {
          /* through Eq. 19 directly and, with the input-dependent gate, through alpha as well */
          gL[c] = alpha * dout[ro + c] + (gate_mode ? cpre * gate[h * GW + c] : 0.0);
          gS[c] = (1.0 - alpha) * dout[ro + c] + (gate_mode ? cpre * gate[h * GW + D + c] : 0.0);
        }
        const int32_t *row = per_query ? idx + (u * L + (size_t)t) * topk
                                       : idx + (u * M + (size_t)(t / Bk)) * topk;
        int nk = ltis_keys(L, Bk, topk, pad0, causal, row, t, keys);
        attend_row_bwd(D, scale, qu + (size_t)t * D, ku, vu, keys, nk, lse[u * L + t],
                       out_lt + ro, gL, dqu + (size_t)t * D, dku, dvu);
        nk = stis_keys(stis_mode, window, stis_blk, L, pad0, causal, t, keys);
        attend_row_bwd(D, scale, qu + (size_t)t * D, ku, vu, keys, nk, lse[BHL + u * L + t],
                       out_st + ro, gS, dqu + (size_t)t * D, dku, dvu);
      }
      if (!gate_mode) dalpha_unit[u] = dalpha;
      free(keys); free(gL); free(gS);
    }
  if (gate_mode) { /* sum the parameter gradients over the batch, in batch order */
    for (int h = 0; h < H; ++h)
      for (int c = 0; c < GW; ++c) {
        double a = 0.0;
        for (int n = 0; n < B; ++n) a += dalpha_unit[((size_t)n * H + h) * GW + c];
        dgate[h * GW + c] = a;
      }
    free(dalpha_unit);
    return 0;
  }
  /* gate logits: alpha = sigmoid(a0 - a1)  =>  d a0 = alpha (1 - alpha) d alpha = - d a1 */
  for (int h = 0; h < H; ++h) {
    double da = 0.0;
    for (int n = 0; n < B; ++n) da += dalpha_unit[(size_t)n * H + h];
    const double alpha = sigmoid(gate[h * 2 + 0] - gate[h * 2 + 1]);
    dgate[h * 2 + 0] = alpha * (1.0 - alpha) * da;
    dgate[h * 2 + 1] = -dgate[h * 2 + 0];
  }
  free(dalpha_unit);
  return 0;
}
