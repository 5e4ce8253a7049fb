/*
 * Float64 CPU oracle for Stochastic Attention (SA).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * CUDA library must compute.  It shares no code, header, table or constant
 * generator with the CUDA path and is never called by it.  Only the tests, the
 * smoke check and the CPU-baseline leg of the benchmark may load it.
 *
 * What each function follows (paper = "Stochastic Attention", Sec. 3, App. A/B):
 *   - visible():            Eq. 3 (window in shuffled space, circular distance of
 *                           Sec. 3.1) intersected with the causal rule of App. B
 *                           "Stochastic attention mask" (pos(q) >= pos(k)).
 *   - swa_visible():        Sec. 3.1 and its footnote (one-sided causal window).
 *   - oracle_forward():     Eq. 1 evaluated on the neighbourhood of Eq. 3; equal
 *                           to Alg. 1 (permute, SWA, un-permute) and to Eq. 4.
 *   - oracle_forward_dense: Eq. 4 literally: full n x n mask, dense softmax.
 *   - oracle_gated_forward: Eq. 5 with one scalar logit per head and branch
 *                           (independent sigmoids, Sec. 3.4).
 *   - oracle_backward():    textbook derivative of Eq. 1 / Eq. 5 (the paper only
 *                           times the backward pass, Sec. 4.3).
 *   - oracle_coverage():    reachable set R_l of Prop. 2 and the mask row counts
 *                           used in the proof of Prop. 1.
 *   - oracle_make_perm():   Alg. 1 line 1 ("sample sigma uniformly").  The paper
 *                           fixes only the distribution; the generator here is
 *                           Philox4x32-10 (Salmon et al., SC'11) sort keys and a
 *                           stable sort, which is this library's definition.
 *
 * Pins (see tests/test_oracle_*.py): Philox known-answer vectors, permutation
 * bijection/uniformity, closed-form mask counts, Prop. 1 by exhaustion, identity
 * permutation == independently written SWA, w >= n+1 == dense attention, Alg. 1
 * three-stage form, uniform-attention mean, w = 1 gives Y = V, finite differences
 * for every gradient, closed-form SWA reach; the selected-row variants
 * (oracle_forward_rows, oracle_backward_rows) on every row index of small cases against
 * the whole-tensor functions and against dense numpy attention.  No function here is
 * unpinned.
 *
 * Layout: all tensors contiguous, q/y/dq [B,Hq,n,d], k/v/dk/dv [B,Hkv,n,d],
 * perm/inv [B,n], lse [B,Hq,n]; everything in ORIGINAL token order.
 * perm[b][p] = token in slot p; inv[b][i] = slot of token i (the paper's sigma(i)).
 * Query head hq uses KV head hq / (Hq/Hkv).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_CAUSAL 1u         /* causality in original order (App. B)        */
#define ORACLE_LINEAR_WINDOW 2u  /* plain |a-b| instead of circular |a-b|_n     */
#define ORACLE_SWA_ONE_SIDED 4u  /* SWA branch: 0 <= i-j <= w-1 (Sec. 3.1 fn.)  */

/* ------------------------------------------------------------------ Philox */

/* One Philox4x32 round (Salmon et al. 2011, Sec. 3.3): two 32x32->64 multiplies,
 * the high halves are xored with the other counter words and the round key.   */
static void philox_round(uint32_t c[4], const uint32_t k[2]) {
  const uint64_t p0 = (uint64_t)0xD2511F53u * c[0];
  const uint64_t p1 = (uint64_t)0xCD9E8D57u * c[2];
  const uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
  const uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
  const uint32_t n0 = hi1 ^ c[1] ^ k[0];
  const uint32_t n1 = lo1;
  const uint32_t n2 = hi0 ^ c[3] ^ k[1];
  const uint32_t n3 = lo0;
  c[0] = n0; c[1] = n1; c[2] = n2; c[3] = n3;
}

void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c[4] = {ctr[0], ctr[1], ctr[2], ctr[3]};
  uint32_t k[2] = {key[0], key[1]};
  for (int r = 0; r < 10; ++r) {
    if (r > 0) { k[0] += 0x9E3779B9u; k[1] += 0xBB67AE85u; } /* Weyl key schedule */
    philox_round(c, k);
  }
  memcpy(out, c, sizeof c);
}

/* 64-bit sort key of token i of sequence b at a layer: counter (i, b, layer, 0),
 * key (seed low, seed high); the first two output words, high word first.      */
uint64_t oracle_sort_key(uint64_t seed, uint32_t layer, uint32_t b, uint32_t i) {
  const uint32_t ctr[4] = {i, b, layer, 0u};
  const uint32_t key[2] = {(uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32)};
  uint32_t r[4];
  oracle_philox4x32_10(ctr, key, r);
  return ((uint64_t)r[0] << 32) | (uint64_t)r[1];
}

typedef struct { uint64_t key; int32_t idx; } keyed;

static int keyed_less(const void* a, const void* b) {
  const keyed* x = (const keyed*)a; const keyed* y = (const keyed*)b;
  if (x->key != y->key) return x->key < y->key ? -1 : 1;
  return (x->idx > y->idx) - (x->idx < y->idx);   /* ties: smaller token first */
}

/* perm = tokens sorted ascending by (key, token); inv[perm[p]] = p.            */
void oracle_make_perm(uint64_t seed, uint32_t layer, int32_t B, int32_t n,
                      int32_t* perm, int32_t* inv) {
  keyed* a = (keyed*)malloc(sizeof(keyed) * (size_t)(n > 0 ? n : 1));
  for (int32_t b = 0; b < B; ++b) {
    for (int32_t i = 0; i < n; ++i) {
      a[i].key = oracle_sort_key(seed, layer, (uint32_t)b, (uint32_t)i);
      a[i].idx = i;
    }
    qsort(a, (size_t)n, sizeof(keyed), keyed_less);  /* total order => unique result */
    for (int32_t p = 0; p < n; ++p) {
      perm[(size_t)b * n + p] = a[p].idx;
      inv[(size_t)b * n + a[p].idx] = p;
    }
  }
  free(a);
}

/* -------------------------------------------------------------------- mask */

static int64_t iabs64(int64_t x) { return x < 0 ? -x : x; }

/* SA predicate: may query token i see key token j?  inv is one sequence's
 * token->slot map (NULL = identity).  Window test in exact integers: the
 * printed |.|_n < w/2 is 2*dist < w.                                           */
int oracle_visible(int32_t n, int32_t w, uint32_t flags, const int32_t* inv,
                   int32_t i, int32_t j) {
  const int64_t si = inv ? inv[i] : i, sj = inv ? inv[j] : j;
  int64_t dist = iabs64(si - sj);
  if (!(flags & ORACLE_LINEAR_WINDOW)) {
    const int64_t wrap = (int64_t)n - dist;
    if (wrap < dist) dist = wrap;
  }
  if (!(2 * dist < (int64_t)w)) return 0;
  if ((flags & ORACLE_CAUSAL) && j > i) return 0;
  return 1;
}

/* Predicate of the plain SWA branch: the one-sided causal window of the Sec. 3.1
 * footnote when ORACLE_SWA_ONE_SIDED is set, otherwise the SA predicate under
 * the identity permutation.                                                    */
int oracle_swa_visible(int32_t n, int32_t w, uint32_t flags, int32_t i, int32_t j) {
  if (flags & ORACLE_SWA_ONE_SIDED) {
    const int64_t back = (int64_t)i - (int64_t)j;
    return back >= 0 && back <= (int64_t)w - 1;
  }
  return oracle_visible(n, w, flags, NULL, i, j);
}

static int branch_visible(int swa, int32_t n, int32_t w, uint32_t flags,
                          const int32_t* inv, int32_t i, int32_t j) {
  return swa ? oracle_swa_visible(n, w, flags, i, j)
             : oracle_visible(n, w, flags, inv, i, j);
}

/* ----------------------------------------------------------------- forward */

/* One query row: scores over the candidate keys cand[0..nc), softmax, output.
 * Returns lse; writes y_row[d] and, when p_out != NULL, the probabilities.     */
static double attend_row(int32_t d, double scale, const double* q_row,
                         const double* k_head, const double* v_head,
                         const int32_t* cand, int32_t nc, double* s_buf,
                         double* y_row) {
  double m = -INFINITY;
  for (int32_t t = 0; t < nc; ++t) {
    const double* kr = k_head + (size_t)cand[t] * d;
    double acc = 0.0;
    for (int32_t c = 0; c < d; ++c) acc += q_row[c] * kr[c];
    s_buf[t] = acc * scale;
    if (s_buf[t] > m) m = s_buf[t];
  }
  double l = 0.0;
  for (int32_t t = 0; t < nc; ++t) { s_buf[t] = exp(s_buf[t] - m); l += s_buf[t]; }
  for (int32_t c = 0; c < d; ++c) y_row[c] = 0.0;
  for (int32_t t = 0; t < nc; ++t) {
    const double* vr = v_head + (size_t)cand[t] * d;
    const double p = s_buf[t] / l;
    s_buf[t] = p;
    for (int32_t c = 0; c < d; ++c) y_row[c] += p * vr[c];
  }
  return m + log(l);
}

/* Visible keys of query token i, in increasing token order.  dense != 0 tests
 * every token j (Eq. 4's full mask); otherwise only the tokens that sit in the
 * slots within reach of the window are tested (same predicate, fewer tests).   */
static int32_t collect_visible(int swa, int dense, int32_t n, int32_t w, uint32_t flags,
                               const int32_t* perm, const int32_t* inv, int32_t i,
                               int32_t* cand) {
  int32_t nc = 0;
  const int64_t h = ((int64_t)w + 1) / 2 - 1;      /* 2*dist < w  <=>  dist <= h */
  const int one_sided = swa && (flags & ORACLE_SWA_ONE_SIDED);
  const int64_t reach = one_sided ? (int64_t)w - 1 : h;
  if (dense || 2 * reach + 1 >= (int64_t)n) {
    for (int32_t j = 0; j < n; ++j)
      if (branch_visible(swa, n, w, flags, inv, i, j)) cand[nc++] = j;
    return nc;
  }
  const int64_t s = (swa || !inv) ? i : inv[i];
  for (int64_t off = -reach; off <= reach; ++off) {
    int64_t slot = s + off;
    if (flags & ORACLE_LINEAR_WINDOW || one_sided) {
      if (slot < 0 || slot >= n) continue;
    } else {
      slot = ((slot % n) + n) % n;
    }
    const int32_t j = (swa || !perm) ? (int32_t)slot : perm[slot];
    if (branch_visible(swa, n, w, flags, inv, i, j)) cand[nc++] = j;
  }
  /* increasing token order, so both forms add the terms in the same order */
  for (int32_t a = 1; a < nc; ++a) {
    const int32_t x = cand[a]; int32_t b = a - 1;
    while (b >= 0 && cand[b] > x) { cand[b + 1] = cand[b]; --b; }
    cand[b + 1] = x;
  }
  return nc;
}

static void forward_impl(int swa, int dense, int32_t B, int32_t Hq, int32_t Hkv,
                         int32_t n, int32_t d, int32_t w, uint32_t flags, double scale,
                         const double* q, const double* k, const double* v,
                         const int32_t* perm, const int32_t* inv, double* y, double* lse) {
  const int32_t G = Hq / Hkv;
  const int64_t rows = (int64_t)B * Hq * n;
#pragma omp parallel
  {
    int32_t* cand = (int32_t*)malloc(sizeof(int32_t) * (size_t)n);
    double* s_buf = (double*)malloc(sizeof(double) * (size_t)n);
#pragma omp for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
      const int32_t i = (int32_t)(r % n);
      const int32_t hq = (int32_t)((r / n) % Hq);
      const int32_t b = (int32_t)(r / ((int64_t)n * Hq));
      const int32_t hk = hq / G;
      const int32_t* pb = perm ? perm + (size_t)b * n : NULL;
      const int32_t* ib = inv ? inv + (size_t)b * n : NULL;
      const int32_t nc = collect_visible(swa, dense, n, w, flags, pb, ib, i, cand);
      const double* kh = k + ((size_t)b * Hkv + hk) * n * d;
      const double* vh = v + ((size_t)b * Hkv + hk) * n * d;
      const double l = attend_row(d, scale, q + (size_t)r * d, kh, vh, cand, nc, s_buf,
                                  y + (size_t)r * d);
      if (lse) lse[r] = l;
    }
    free(cand); free(s_buf);
  }
}

/* SA forward: perm/inv [B,n].  SWA forward: pass swa=1 (perm/inv ignored).     */
void oracle_forward(int32_t swa, int32_t B, int32_t Hq, int32_t Hkv, int32_t n, int32_t d,
                    int32_t w, uint32_t flags, double scale, const double* q,
                    const double* k, const double* v, const int32_t* perm,
                    const int32_t* inv, double* y, double* lse) {
  forward_impl(swa, 0, B, Hq, Hkv, n, d, w, flags, scale, q, k, v, perm, inv, y, lse);
}

/* Eq. 4: every (i, j) pair is tested against the mask.  O(n^2 d); small n only. */
void oracle_forward_dense(int32_t swa, int32_t B, int32_t Hq, int32_t Hkv, int32_t n,
                          int32_t d, int32_t w, uint32_t flags, double scale,
                          const double* q, const double* k, const double* v,
                          const int32_t* perm, const int32_t* inv, double* y, double* lse) {
  forward_impl(swa, 1, B, Hq, Hkv, n, d, w, flags, scale, q, k, v, perm, inv, y, lse);
}

static double sigmoid(double x) { return 1.0 / (1.0 + exp(-x)); }

/* Eq. 5 with per-head scalar gates: y = sig(l[0][hq]) y_sa + sig(l[1][hq]) y_swa.
 * gate_logits [2,Hq]: row 0 = SA branch, row 1 = SWA branch.                   */
void oracle_gated_forward(int32_t B, int32_t Hq, int32_t Hkv, int32_t n, int32_t d,
                          int32_t w, uint32_t flags, double scale, const double* q,
                          const double* k, const double* v, const int32_t* perm,
                          const int32_t* inv, const double* gate_logits, double* y,
                          double* y_sa, double* y_swa, double* lse_sa, double* lse_swa) {
  forward_impl(0, 0, B, Hq, Hkv, n, d, w, flags, scale, q, k, v, perm, inv, y_sa, lse_sa);
  forward_impl(1, 0, B, Hq, Hkv, n, d, w, flags, scale, q, k, v, NULL, NULL, y_swa, lse_swa);
  for (int32_t b = 0; b < B; ++b)
    for (int32_t hq = 0; hq < Hq; ++hq) {
      const double g_sa = sigmoid(gate_logits[hq]), g_swa = sigmoid(gate_logits[Hq + hq]);
      const size_t base = ((size_t)b * Hq + hq) * n * d;
      for (size_t e = 0; e < (size_t)n * d; ++e)
        y[base + e] = g_sa * y_sa[base + e] + g_swa * y_swa[base + e];
    }
}

/* ---------------------------------------------------------------- backward */

/* Gradients of L = sum(dy * y).  gate_logits == NULL: ungated SA only (y = y_sa,
 * dgate untouched).  Otherwise both branches through Eq. 5.  The forward pass is
 * recomputed here in float64; nothing saved by another implementation is used.
 * Per branch x with upstream dY_x = g_x dY:  P_ij = softmax row;
 * D_i = dY_x[i].Y_x[i];  dV_j += P_ij dY_x[i];  dS_ij = P_ij (dY_x[i].V_j - D_i);
 * dQ_i += scale dS_ij K_j;  dK_j += scale dS_ij Q_i;
 * dlogit[x][hq] = g_x (1-g_x) sum_{b,i,c} dY[b,hq,i,c] Y_x[b,hq,i,c].          */
void oracle_backward(int32_t B, int32_t Hq, int32_t Hkv, int32_t n, int32_t d, int32_t w,
                     uint32_t flags, double scale, const double* q, const double* k,
                     const double* v, const int32_t* perm, const int32_t* inv,
                     const double* gate_logits, const double* dy, double* dq, double* dk,
                     double* dv, double* dgate_logits) {
  const int32_t G = Hq / Hkv;
  const int32_t nbranch = gate_logits ? 2 : 1;
  memset(dq, 0, sizeof(double) * (size_t)B * Hq * n * d);
  memset(dk, 0, sizeof(double) * (size_t)B * Hkv * n * d);
  memset(dv, 0, sizeof(double) * (size_t)B * Hkv * n * d);
  double* dot_yx = (double*)calloc((size_t)B * 2 * Hq, sizeof(double));
  const int64_t units = (int64_t)B * Hkv;      /* a unit owns dk/dv of one (b, hk) */
#pragma omp parallel
  {
    int32_t* cand = (int32_t*)malloc(sizeof(int32_t) * (size_t)n);
    double* p = (double*)malloc(sizeof(double) * (size_t)n);
    double* yx = (double*)malloc(sizeof(double) * (size_t)d);
    double* dyx = (double*)malloc(sizeof(double) * (size_t)d);
#pragma omp for schedule(dynamic, 1)
    for (int64_t u = 0; u < units; ++u) {
      const int32_t b = (int32_t)(u / Hkv), hk = (int32_t)(u % Hkv);
      const int32_t* pb = perm ? perm + (size_t)b * n : NULL;
      const int32_t* ib = inv ? inv + (size_t)b * n : NULL;
      const double* kh = k + ((size_t)b * Hkv + hk) * n * d;
      const double* vh = v + ((size_t)b * Hkv + hk) * n * d;
      double* dkh = dk + ((size_t)b * Hkv + hk) * n * d;
      double* dvh = dv + ((size_t)b * Hkv + hk) * n * d;
      for (int32_t hq = hk * G; hq < (hk + 1) * G; ++hq)
        for (int32_t x = 0; x < nbranch; ++x) {
          const double g = gate_logits ? sigmoid(gate_logits[x * Hq + hq]) : 1.0;
          for (int32_t i = 0; i < n; ++i) {
            const size_t r = ((size_t)b * Hq + hq) * n + i;
            const double* qr = q + r * d;
            const int32_t nc = collect_visible(x == 1, 0, n, w, flags, pb, ib, i, cand);
            attend_row(d, scale, qr, kh, vh, cand, nc, p, yx);   /* p = probabilities */
            double D = 0.0, dotg = 0.0;
            for (int32_t c = 0; c < d; ++c) {
              dyx[c] = g * dy[r * d + c];
              D += dyx[c] * yx[c];
              dotg += dy[r * d + c] * yx[c];
            }
            dot_yx[((size_t)b * 2 + x) * Hq + hq] += dotg;
            for (int32_t t = 0; t < nc; ++t) {
              const int32_t j = cand[t];
              double dp = 0.0;
              for (int32_t c = 0; c < d; ++c) dp += dyx[c] * vh[(size_t)j * d + c];
              const double ds = p[t] * (dp - D);
              for (int32_t c = 0; c < d; ++c) {
                dvh[(size_t)j * d + c] += p[t] * dyx[c];
                dq[r * d + c] += scale * ds * kh[(size_t)j * d + c];
                dkh[(size_t)j * d + c] += scale * ds * qr[c];
              }
            }
          }
        }
    }
    free(cand); free(p); free(yx); free(dyx);
  }
  if (gate_logits && dgate_logits)
    for (int32_t x = 0; x < 2; ++x)
      for (int32_t hq = 0; hq < Hq; ++hq) {
        const double g = sigmoid(gate_logits[x * Hq + hq]);
        double s = 0.0;
        for (int32_t b = 0; b < B; ++b) s += dot_yx[((size_t)b * 2 + x) * Hq + hq];
        dgate_logits[x * Hq + hq] = g * (1.0 - g) * s;
      }
  free(dot_yx);
}

/* ---------------------------------------------------------------- coverage */

/* L layers, each with its own permutation perm/inv [L,n] (NULL = identity, i.e.
 * plain SWA with the SA predicate).  Per layer: row_count[l][i] = number of keys
 * visible to query i; nnz[l] = their sum.  Reach (Prop. 2): R_0 = {src};
 * R_l = union over q in R_{l-1} of {k : visible_l(q, k)}; reach[l-1] = |R_l|.   */
void oracle_coverage(int32_t L, int32_t n, int32_t w, uint32_t flags, const int32_t* perm,
                     const int32_t* inv, int32_t src, int64_t* nnz, int32_t* row_count,
                     int32_t* reach) {
  uint8_t* cur = (uint8_t*)calloc((size_t)n, 1);
  uint8_t* nxt = (uint8_t*)calloc((size_t)n, 1);
  if (src >= 0 && src < n) cur[src] = 1;
  for (int32_t l = 0; l < L; ++l) {
    const int32_t* il = inv ? inv + (size_t)l * n : NULL;
    (void)perm;
    int64_t total = 0;
    memset(nxt, 0, (size_t)n);
    for (int32_t i = 0; i < n; ++i) {
      int32_t cnt = 0;
      for (int32_t j = 0; j < n; ++j)
        if (oracle_visible(n, w, flags, il, i, j)) { ++cnt; if (cur[i]) nxt[j] = 1; }
      if (row_count) row_count[(size_t)l * n + i] = cnt;
      total += cnt;
    }
    if (nnz) nnz[l] = total;
    int32_t sz = 0;
    for (int32_t j = 0; j < n; ++j) sz += nxt[j];
    if (reach) reach[l] = sz;
    uint8_t* t = cur; cur = nxt; nxt = t;
  }
  free(cur); free(nxt);
}

/* Selected rows only: rows[t] is a flat (b*Hq + hq)*n + i index; y_rows [n_rows,d],
 * lse_rows [n_rows].  Same arithmetic as oracle_forward, for spot checks at sizes where
 * the whole tensor would take hours.                                             */
void oracle_forward_rows(int32_t swa, int32_t B, int32_t Hq, int32_t Hkv, int32_t n, int32_t d,
                         int32_t w, uint32_t flags, double scale, const double* q,
                         const double* k, const double* v, const int32_t* perm,
                         const int32_t* inv, int64_t n_rows, const int64_t* rows,
                         double* y_rows, double* lse_rows) {
  const int32_t G = Hq / Hkv;
  (void)B;
#pragma omp parallel
  {
    int32_t* cand = (int32_t*)malloc(sizeof(int32_t) * (size_t)n);
    double* s_buf = (double*)malloc(sizeof(double) * (size_t)n);
#pragma omp for schedule(dynamic, 16)
    for (int64_t t = 0; t < n_rows; ++t) {
      const int64_t r = rows[t];
      const int32_t i = (int32_t)(r % n);
      const int32_t hq = (int32_t)((r / n) % Hq);
      const int32_t b = (int32_t)(r / ((int64_t)n * Hq));
      const int32_t hk = hq / G;
      const int32_t* pb = perm ? perm + (size_t)b * n : NULL;
      const int32_t* ib = inv ? inv + (size_t)b * n : NULL;
      const int32_t nc = collect_visible(swa, 0, n, w, flags, pb, ib, i, cand);
      const double* kh = k + ((size_t)b * Hkv + hk) * n * d;
      const double* vh = v + ((size_t)b * Hkv + hk) * n * d;
      const double l = attend_row(d, scale, q + (size_t)r * d, kh, vh, cand, nc, s_buf,
                                  y_rows + (size_t)t * d);
      if (lse_rows) lse_rows[t] = l;
    }
    free(cand); free(s_buf);
  }
}

/* Selected gradient rows only, for spot checks at sizes where oracle_backward would take
 * days.  Same formulas as oracle_backward (textbook derivative of Eq. 1 / Eq. 5), written
 * per requested row:
 *   q_rows[t] = flat (b*Hq + hq)*n + i   ->  dq_rows[t][d]: sum over the branches x and the
 *               keys j visible to query i of scale * dS_ij * K_j;
 *   kv_rows[t] = flat (b*Hkv + hk)*n + j ->  dk_rows[t][d], dv_rows[t][d]: sum over the query
 *               heads of the group, the branches and EVERY query token i that sees key j
 *               (all n tokens are tested with the branch's predicate) of scale * dS_ij * Q_i
 *               and P_ij * dY_x[i].
 * Each query's softmax row is recomputed in full, as in oracle_backward.  gate_logits ==
 * NULL: ungated SA only.                                                               */
void oracle_backward_rows(int32_t B, int32_t Hq, int32_t Hkv, int32_t n, int32_t d, int32_t w,
                          uint32_t flags, double scale, const double* q, const double* k,
                          const double* v, const int32_t* perm, const int32_t* inv,
                          const double* gate_logits, const double* dy,
                          int64_t n_q_rows, const int64_t* q_rows, double* dq_rows,
                          int64_t n_kv_rows, const int64_t* kv_rows, double* dk_rows,
                          double* dv_rows) {
  const int32_t G = Hq / Hkv;
  const int32_t nbranch = gate_logits ? 2 : 1;
  (void)B;
#pragma omp parallel
  {
    int32_t* cand = (int32_t*)malloc(sizeof(int32_t) * (size_t)n);
    double* p = (double*)malloc(sizeof(double) * (size_t)n);
    double* yx = (double*)malloc(sizeof(double) * (size_t)d);
    double* dyx = (double*)malloc(sizeof(double) * (size_t)d);
#pragma omp for schedule(dynamic, 4)
    for (int64_t t = 0; t < n_q_rows; ++t) {
      const int64_t r = q_rows[t];
      const int32_t i = (int32_t)(r % n);
      const int32_t hq = (int32_t)((r / n) % Hq);
      const int32_t b = (int32_t)(r / ((int64_t)n * Hq));
      const int32_t hk = hq / G;
      const int32_t* pb = perm ? perm + (size_t)b * n : NULL;
      const int32_t* ib = inv ? inv + (size_t)b * n : NULL;
      const double* kh = k + ((size_t)b * Hkv + hk) * n * d;
      const double* vh = v + ((size_t)b * Hkv + hk) * n * d;
      const double* qr = q + (size_t)r * d;
      double* out = dq_rows + (size_t)t * d;
      for (int32_t c = 0; c < d; ++c) out[c] = 0.0;
      for (int32_t x = 0; x < nbranch; ++x) {
        const double g = gate_logits ? sigmoid(gate_logits[x * Hq + hq]) : 1.0;
        const int32_t nc = collect_visible(x == 1, 0, n, w, flags, pb, ib, i, cand);
        attend_row(d, scale, qr, kh, vh, cand, nc, p, yx);
        double D = 0.0;
        for (int32_t c = 0; c < d; ++c) { dyx[c] = g * dy[(size_t)r * d + c]; D += dyx[c] * yx[c]; }
        for (int32_t u = 0; u < nc; ++u) {
          const int32_t j = cand[u];
          double dp = 0.0;
          for (int32_t c = 0; c < d; ++c) dp += dyx[c] * vh[(size_t)j * d + c];
          const double ds = p[u] * (dp - D);
          for (int32_t c = 0; c < d; ++c) out[c] += scale * ds * kh[(size_t)j * d + c];
        }
      }
    }
#pragma omp for schedule(dynamic, 1)
    for (int64_t t = 0; t < n_kv_rows; ++t) {
      const int64_t r = kv_rows[t];
      const int32_t j = (int32_t)(r % n);
      const int32_t hk = (int32_t)((r / n) % Hkv);
      const int32_t b = (int32_t)(r / ((int64_t)n * Hkv));
      const int32_t* pb = perm ? perm + (size_t)b * n : NULL;
      const int32_t* ib = inv ? inv + (size_t)b * n : NULL;
      const double* kh = k + ((size_t)b * Hkv + hk) * n * d;
      const double* vh = v + ((size_t)b * Hkv + hk) * n * d;
      double* odk = dk_rows + (size_t)t * d;
      double* odv = dv_rows + (size_t)t * d;
      for (int32_t c = 0; c < d; ++c) { odk[c] = 0.0; odv[c] = 0.0; }
      for (int32_t hq = hk * G; hq < (hk + 1) * G; ++hq)
        for (int32_t x = 0; x < nbranch; ++x) {
          const double g = gate_logits ? sigmoid(gate_logits[x * Hq + hq]) : 1.0;
          for (int32_t i = 0; i < n; ++i) {
            if (!branch_visible(x == 1, n, w, flags, ib, i, j)) continue;
            const size_t qi = ((size_t)b * Hq + hq) * n + i;
            const double* qr = q + qi * d;
            const int32_t nc = collect_visible(x == 1, 0, n, w, flags, pb, ib, i, cand);
            attend_row(d, scale, qr, kh, vh, cand, nc, p, yx);
            int32_t at = -1;
            for (int32_t u = 0; u < nc; ++u) if (cand[u] == j) { at = u; break; }
            if (at < 0) continue;   /* cannot happen: j passed the same predicate */
            double D = 0.0, dp = 0.0;
            for (int32_t c = 0; c < d; ++c) {
              dyx[c] = g * dy[qi * d + c];
              D += dyx[c] * yx[c];
              dp += dyx[c] * vh[(size_t)j * d + c];
            }
            const double ds = p[at] * (dp - D);
            for (int32_t c = 0; c < d; ++c) {
              odv[c] += p[at] * dyx[c];
              odk[c] += scale * ds * qr[c];
            }
          }
        }
    }
    free(cand); free(p); free(yx); free(dyx);
  }
}
