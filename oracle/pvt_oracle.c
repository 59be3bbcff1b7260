/*
 * CPU checker for the discrete V step of PV-Tuning.  TEST INFRASTRUCTURE ONLY:
 * it defines what the GPU library must compute, it is deliberately plain and
 * slow, and it shares no code with the CUDA path.  Only the tests, the smoke
 * check and the benchmark's CPU-baseline leg may call it.
 *
 * Every function follows one passage of the paper:
 *   - group update norm and arg-top-tau choice: the selection step of
 *     Algorithm 2, Section 3.4 (ranking by update size, matrix by matrix),
 *     choose_subspace of Algorithm 3;
 *   - target of the search: Eq. (8), y - (1/L) Z(grad phi(y)), in the scaled
 *     space of the codebooks (Appendix J: one trainable scale per channel);
 *   - M = 1 search: Appendix C / Appendix J (all codewords are tried and the
 *     one with the smallest squared error is taken);
 *   - M >= 2 search: Appendix C / Appendix J (beam search, beam size 8, target =
 *     gradient-updated dequantised weight), greedy residual form;
 *   - untouched codes outside the subspace: Section 3.3 (x+_i = y_i for i not
 *     in S^k);
 *   - dequantisation: dequantize_weights of Algorithm 3.
 *
 * Arithmetic: the norm, the target and the dequantised weight are sequences of
 * single IEEE binary32 operations (stated at each function) so that a GPU can
 * reproduce them bit for bit; every distance is accumulated in binary64.
 * Build with -O2 -ffp-contract=off: no operation may be fused except the
 * explicit fmaf calls.
 *
 * Pins (tests marked "not gpu"): the paper's two printed assignment examples,
 * brute-force enumeration of every code tuple on tiny inputs, a library
 * nearest-centroid routine (the V step with phi = ||x - z||^2 is the K-means
 * assignment step, Section 3.1), the expansion ||x-B||^2 = ||x||^2 - 2<x,B> +
 * ||B||^2 (Appendix D), beam >= K equals exhaustive search, beam = 1 equals
 * greedy residual quantisation (two, three and four codebooks), narrow beams
 * over three and four codebooks against an independent stage-by-stage search
 * (tuples and distances equal, exact ties among partial tuples included), zero
 * second codebook reduces to M = 1,
 * monotonicity (Lemma 3.3), locality, fixed point, full-sort selection with
 * crafted ties, closed-form dequantisation.  No end-to-end V-step result on a
 * real layer is printed in the paper, so beyond these pins parity is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define PVT_ORACLE_MAX_M 4
#define PVT_ORACLE_MAX_BEAM 4096

int pvt_oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

void pvt_oracle_set_num_threads(int n) {
#ifdef _OPENMP
  if (n > 0) omp_set_num_threads(n);
#else
  (void)n;
#endif
}

/* Squared norm of the update eta*g of every weight group (Algorithm 2; Section
 * 3.4).  binary32: u_i = eta*g_i rounded once; acc = fmaf(u_i, u_i, acc) for i
 * in index order starting from 0. */
void pvt_oracle_group_norms(const float* g, int64_t rows, int64_t cols, int32_t dg, float eta,
                            float* norms) {
  const int64_t gpr = cols / dg;
#pragma omp parallel for schedule(static)
  for (int64_t j = 0; j < rows * gpr; ++j) {
    const int64_t r = j / gpr, c = j % gpr;
    const float* gj = g + r * cols + c * dg;
    float acc = 0.0f;
    for (int32_t i = 0; i < dg; ++i) {
      const float u = eta * gj[i];
      acc = fmaf(u, u, acc);
    }
    norms[j] = acc;
  }
}

typedef struct {
  float n;
  uint32_t j;
} norm_entry;

static int by_norm_desc_then_index(const void* a, const void* b) {
  const norm_entry* x = (const norm_entry*)a;
  const norm_entry* y = (const norm_entry*)b;
  if (x->n > y->n) return -1;
  if (x->n < y->n) return 1;
  if (x->j < y->j) return -1;
  if (x->j > y->j) return 1;
  return 0;
}

static int by_u32(const void* a, const void* b) {
  const uint32_t x = *(const uint32_t*)a, y = *(const uint32_t*)b;
  return (x > y) - (x < y);
}

/* arg top-k (Algorithm 2): order all groups by (norm descending, index
 * ascending), keep the first k, return them in ascending index order.
 * Returns 0, or -1 on a bad argument / non-finite norm. */
int pvt_oracle_select(const float* norms, int64_t G, int64_t k, uint32_t* idx_out) {
  if (k < 1 || k > G || G >= ((int64_t)1 << 32)) return -1;
  norm_entry* e = (norm_entry*)malloc((size_t)G * sizeof(norm_entry));
  if (!e) return -1;
  for (int64_t j = 0; j < G; ++j) {
    if (!isfinite(norms[j]) || norms[j] < 0.0f) {
      free(e);
      return -1;
    }
    e[j].n = norms[j];
    e[j].j = (uint32_t)j;
  }
  qsort(e, (size_t)G, sizeof(norm_entry), by_norm_desc_then_index);
  for (int64_t i = 0; i < k; ++i) idx_out[i] = e[i].j;
  free(e);
  qsort(idx_out, (size_t)k, sizeof(uint32_t), by_u32);
  return 0;
}

/* Target of the search for the selected groups (Eq. 8, scaled space):
 * t_i = (W_i - eta*g_i) / s_row, binary32: one fmaf(-eta, g_i, W_i), one
 * division. */
void pvt_oracle_targets(const float* W, const float* g, const float* scale, int64_t rows,
                        int64_t cols, int32_t dg, float eta, const uint32_t* idx, int64_t k,
                        float* t_out) {
  (void)rows;
  const int64_t gpr = cols / dg;
#pragma omp parallel for schedule(static)
  for (int64_t n = 0; n < k; ++n) {
    const int64_t j = idx[n], r = j / gpr, c = j % gpr;
    const float* Wj = W + r * cols + c * dg;
    const float* gj = g + r * cols + c * dg;
    for (int32_t i = 0; i < dg; ++i) t_out[n * dg + i] = fmaf(-eta, gj[i], Wj[i]) / scale[r];
  }
}

/* ||r - c||^2 in binary64, terms added in index order. */
static double sqdist(const double* r, const float* c, int32_t dg) {
  double d = 0.0;
  for (int32_t i = 0; i < dg; ++i) {
    const double e = r[i] - (double)c[i];
    d = d + e * e;
  }
  return d;
}

typedef struct {
  double d;                       /* ||t - sum of chosen codewords||^2 */
  int32_t code[PVT_ORACLE_MAX_M]; /* chosen codeword per codebook so far */
} beam_entry;

/* (distance, code tuple) lexicographic order over the first m codes */
static int entry_less(const beam_entry* a, const beam_entry* b, int32_t m) {
  if (a->d < b->d) return 1;
  if (a->d > b->d) return 0;
  for (int32_t i = 0; i < m; ++i) {
    if (a->code[i] < b->code[i]) return 1;
    if (a->code[i] > b->code[i]) return 0;
  }
  return 0;
}

static void residual_of(const float* t, const float* books, int32_t dg, int32_t K,
                        const int32_t* code, int32_t m, double* r) {
  for (int32_t i = 0; i < dg; ++i) r[i] = (double)t[i];
  for (int32_t q = 0; q < m; ++q) {
    const float* c = books + ((int64_t)q * K + code[q]) * dg;
    for (int32_t i = 0; i < dg; ++i) r[i] = r[i] - (double)c[i];
  }
}

/* M = 1 (Appendix C / Appendix J): every codeword of the codebook is tried;
 * the result is the argmin of (||t - c||^2, code).  *d2 receives the smallest
 * distance over the other codewords. */
static void search_single(const float* t, int32_t dg, int32_t K, const float* book, int32_t* code,
                          double* d1, double* d2) {
  double r[64];
  for (int32_t i = 0; i < dg; ++i) r[i] = (double)t[i];
  int32_t arg = 0;
  double best = sqdist(r, book, dg), second = INFINITY;
  for (int32_t q = 1; q < K; ++q) {
    const double d = sqdist(r, book + (int64_t)q * dg, dg);
    if (d < best) { /* strict: equal distances keep the lower code */
      second = best;
      best = d;
      arg = q;
    } else if (d < second) {
      second = d;
    }
  }
  *code = arg;
  *d1 = best;
  *d2 = (K > 1) ? second : best;
}

/* M >= 2 (Appendix C / Appendix J: beam search, target = gradient-updated
 * dequantised weight), greedy residual form.  Stage m extends each kept partial
 * tuple by every codeword of codebook m and scores ||t - c^1 - ... - c^m||^2 with
 * the residual carried in binary64.  After stages 1..M-1 the `beam` best partial
 * tuples under (distance, tuple) are kept.  The final pool is every extension
 * made at the last stage plus the previous tuple, so the result is never worse
 * than the previous code (Lemma 3.3); result = argmin of (distance, tuple).
 * Returns 0, -1 on allocation failure or an out-of-range previous code. */
static int search_beam(const float* t, int32_t dg, int32_t M, int32_t K, const float* books,
                       int32_t beam, const int32_t* prev, int32_t* code, double* d1, double* d2,
                       double* gap_in, double* gap_out) {
  double r[64];
  int have_gap = 0;
  int64_t nkept = 1; /* the single empty tuple */
  beam_entry* kept = (beam_entry*)calloc(1, sizeof(beam_entry));
  beam_entry* cand = NULL;
  if (!kept) return -1;
  for (int32_t m = 0; m < M; ++m) {
    const int64_t ncand = nkept * K;
    cand = (beam_entry*)malloc((size_t)ncand * sizeof(beam_entry));
    if (!cand) {
      free(kept);
      return -1;
    }
    for (int64_t b = 0; b < nkept; ++b) {
      residual_of(t, books, dg, K, kept[b].code, m, r);
      for (int32_t q = 0; q < K; ++q) {
        beam_entry* e = &cand[b * K + q];
        *e = kept[b];
        e->code[m] = q;
        e->d = sqdist(r, books + ((int64_t)m * K + q) * dg, dg);
      }
    }
    free(kept);
    kept = NULL;
    if (m == M - 1) break;
    /* keep the `beam` best: selection by repeated minimum, one extra round to
     * learn the first dropped tuple */
    const int64_t nkeep = ncand < beam ? ncand : beam;
    kept = (beam_entry*)malloc((size_t)(nkeep + 1) * sizeof(beam_entry));
    if (!kept) {
      free(cand);
      return -1;
    }
    for (int64_t s = 0; s <= nkeep && s < ncand; ++s) {
      int64_t arg = s;
      for (int64_t c = s + 1; c < ncand; ++c)
        if (entry_less(&cand[c], &cand[arg], m + 1)) arg = c;
      const beam_entry tmp = cand[s];
      cand[s] = cand[arg];
      cand[arg] = tmp;
      kept[s] = cand[s];
    }
    if (nkeep < ncand) {
      const double din = kept[nkeep - 1].d, dout = kept[nkeep].d;
      if (!have_gap || (dout - din) * (*gap_out) < (*gap_out - *gap_in) * dout) {
        *gap_in = din;
        *gap_out = dout;
        have_gap = 1;
      }
    }
    nkept = nkeep;
    free(cand);
    cand = NULL;
  }

  /* final pool */
  const int64_t npool = nkept * K;
  beam_entry best = cand[0], second = cand[0];
  int have_second = 0;
  for (int64_t c = 1; c < npool; ++c) {
    if (entry_less(&cand[c], &best, M)) {
      second = best;
      have_second = 1;
      best = cand[c];
    } else if (!have_second || entry_less(&cand[c], &second, M)) {
      second = cand[c];
      have_second = 1;
    }
  }
  beam_entry p;
  memset(&p, 0, sizeof p);
  int in_pool = 0, ok = 1;
  for (int32_t q = 0; q < M; ++q) {
    p.code[q] = prev[q];
    if (prev[q] < 0 || prev[q] >= K) ok = 0;
  }
  if (ok) {
    for (int64_t c = 0; c < npool && !in_pool; ++c) {
      int same = 1;
      for (int32_t q = 0; q < M; ++q) same = same && cand[c].code[q] == p.code[q];
      in_pool = same;
    }
    if (!in_pool) {
      residual_of(t, books, dg, K, p.code, M - 1, r);
      p.d = sqdist(r, books + ((int64_t)(M - 1) * K + p.code[M - 1]) * dg, dg);
      if (entry_less(&p, &best, M)) {
        second = best;
        have_second = 1;
        best = p;
      } else if (!have_second || entry_less(&p, &second, M)) {
        second = p;
        have_second = 1;
      }
    }
  }
  free(cand);
  if (!ok) return -1;
  for (int32_t q = 0; q < M; ++q) code[q] = best.code[q];
  *d1 = best.d;
  *d2 = have_second ? second.d : best.d;
  if (!have_gap) {
    *gap_in = best.d;
    *gap_out = best.d;
  }
  return 0;
}

/* Nearest-codeword search for k targets t [k][dg].
 * books: [M][K][dg] binary32 (fp16 codebooks widened exactly by the caller).
 * prev, codes_out: [k][M].  d_best/d_second: smallest and second-smallest
 * distance over the final pool (second: over pool members other than the
 * winner).  bd_in/bd_out (may be NULL): distances of the last kept and the first
 * dropped partial tuple at the beam stage where their gap is relatively
 * smallest (both d_best when nothing is dropped).
 * Returns 0, or -1 on bad arguments. */
int pvt_oracle_encode(const float* t, int64_t k, int32_t dg, int32_t M, int32_t K,
                      const float* books, int32_t beam, const int32_t* prev, int32_t* codes_out,
                      double* d_best, double* d_second, double* bd_in, double* bd_out) {
  if (M < 1 || M > PVT_ORACLE_MAX_M || K < 1 || dg < 1 || dg > 64) return -1;
  if (M > 1 && (beam < 1 || beam > PVT_ORACLE_MAX_BEAM)) return -1;
  int bad = 0;
#pragma omp parallel for schedule(dynamic, 16)
  for (int64_t n = 0; n < k; ++n) {
    double gi = 0.0, go = 0.0;
    if (M == 1) {
      search_single(t + n * dg, dg, K, books, &codes_out[n], &d_best[n], &d_second[n]);
      gi = go = d_best[n];
    } else if (search_beam(t + n * dg, dg, M, K, books, beam, prev + n * M, codes_out + n * M,
                           &d_best[n], &d_second[n], &gi, &go) != 0) {
      bad = 1;
    }
    if (bd_in) bd_in[n] = gi;
    if (bd_out) bd_out[n] = go;
  }
  return bad ? -1 : 0;
}

/* Squared error ||t - sum_m C_m[code_m]||^2 in binary64 for given code tuples
 * (the same accumulation order as the search). */
void pvt_oracle_tuple_error(const float* t, int64_t k, int32_t dg, int32_t M, int32_t K,
                            const float* books, const int32_t* codes, double* d_out) {
#pragma omp parallel for schedule(static)
  for (int64_t n = 0; n < k; ++n) {
    double r[64];
    residual_of(t + n * dg, books, dg, K, codes + n * M, M - 1, r);
    d_out[n] = sqdist(r, books + ((int64_t)(M - 1) * K + codes[n * M + M - 1]) * dg, dg);
  }
}

/* W_hat = s_row * sum_m C_m[b_m] (Algorithm 3, dequantize_weights).  binary32:
 * codewords added left to right, each addition rounded once, then one
 * multiplication by the row scale. */
void pvt_oracle_dequant(const int32_t* codes, const float* books, const float* scale, int64_t rows,
                        int64_t cols, int32_t dg, int32_t M, int32_t K, float* W_hat) {
  const int64_t gpr = cols / dg;
#pragma omp parallel for schedule(static)
  for (int64_t j = 0; j < rows * gpr; ++j) {
    const int64_t r = j / gpr, c = j % gpr;
    for (int32_t i = 0; i < dg; ++i) {
      float v = books[((int64_t)0 * K + codes[j * M]) * dg + i];
      for (int32_t q = 1; q < M; ++q) v = v + books[((int64_t)q * K + codes[j * M + q]) * dg + i];
      W_hat[r * cols + c * dg + i] = scale[r] * v;
    }
  }
}

/* ---- P step, the part that shares its inputs with the V step ---------------------------------------------
 * Algorithm 3, P-step lines: grad_codebooks = backprop(grad_phi); codebooks = adam(grad_codebooks)
 * (Section 3.4: adaptive learning rates for the P step; Appendix J: beta1 = 0.9, beta2 = 0.95; codebooks and
 * per-channel scales are the trainable continuous parameters of the representation).
 *
 * backprop is the chain rule through dequantize_weights, W_hat[r, dg*c + i] = s_r * v_{j,i},
 * v_j = sum_m C_m[b_{j,m}] (the binary32 sum that dequantisation forms):
 *     grad_codebooks[m][kappa][i] = sum over groups j with b_{j,m} = kappa of  s_{r(j)} * g[j][i]
 *     grad_scale[r]               = sum over groups j of row r and over i of   g[j][i] * v_{j,i}
 * Each product of two binary32 numbers is exact in binary64; the sums run in group order in binary64.
 * Pins: automatic differentiation of the same forward map in a library, central finite differences of a
 * quadratic phi, linearity in g, and the case of a single shared code (the gradient is the plain sum).
 */
void pvt_oracle_pstep_grad(const float* g, const float* scale, const int32_t* codes, const float* books,
                           int64_t rows, int64_t cols, int32_t dg, int32_t M, int32_t K, double* grad_books,
                           double* grad_scale) {
  const int64_t gpr = cols / dg;
  memset(grad_books, 0, sizeof(double) * (size_t)M * K * dg);
  memset(grad_scale, 0, sizeof(double) * (size_t)rows);
  for (int64_t j = 0; j < rows * gpr; ++j) {
    const int64_t r = j / gpr, c = j % gpr;
    const float* gj = g + r * cols + c * dg;
    for (int32_t i = 0; i < dg; ++i) {
      float v = books[((int64_t)0 * K + codes[j * M]) * dg + i];
      for (int32_t q = 1; q < M; ++q) v = v + books[((int64_t)q * K + codes[j * M + q]) * dg + i];
      grad_scale[r] += (double)gj[i] * (double)v;
      for (int32_t q = 0; q < M; ++q)
        grad_books[((int64_t)q * K + codes[j * M + q]) * dg + i] += (double)scale[r] * (double)gj[i];
    }
  }
}

/* One Adam update of n binary32 parameters (Kingma & Ba; the codebook update of Algorithm 3's P step).  The
 * gradient arrives in binary64 and is rounded once to binary32; then, all in binary32, each operation
 * rounded once, in this order:
 *     m = fmaf(beta1, m, (1 - beta1) * gr)          v = fmaf(beta2, v, ((1 - beta2) * gr) * gr)
 *     p = p - (lr * (m / bias1)) / (sqrtf(v / bias2) + eps)
 * bias1 = 1 - beta1^t and bias2 = 1 - beta2^t are passed in (binary32) by the caller.
 * Pins: a library Adam, and the closed form of the first step, lr * gr / (|gr| + eps). */
void pvt_oracle_adam(float* param, const double* grad, float* exp_avg, float* exp_avg_sq, int64_t n, float lr,
                     float beta1, float beta2, float eps, float bias1, float bias2) {
  const float omb1 = 1.0f - beta1, omb2 = 1.0f - beta2;
  for (int64_t i = 0; i < n; ++i) {
    const float gr = (float)grad[i];
    const float m = fmaf(beta1, exp_avg[i], omb1 * gr);
    const float v = fmaf(beta2, exp_avg_sq[i], (omb2 * gr) * gr);
    exp_avg[i] = m;
    exp_avg_sq[i] = v;
    const float num = lr * (m / bias1);
    const float den = sqrtf(v / bias2) + eps;
    param[i] = param[i] - num / den;
  }
}

/* Update direction of the V step as the paper runs it (Section 3.4: grad phi(y) in Eq. 8 is replaced by a single
 * Adam update; the update line of Algorithm 3's V step; the subspace is then chosen by the
 * magnitude of this update).  Moments as in Adam; the direction is the bias-corrected ratio, all in binary32,
 * every operation rounded once:
 *     m = fmaf(beta1, m, (1 - beta1) * g)        v = fmaf(beta2, v, ((1 - beta2) * g) * g)
 *     u = (m / bias1) / (sqrtf(v / bias2) + eps)
 * The V step then runs on (W, u, eta = learning rate of the codes).
 * Pins: the first step's closed form g / (|g| + eps), and a library Adam with learning rate 1 started at 0,
 * whose parameter is minus the accumulated directions. */
void pvt_oracle_adam_direction(const float* grad, float* exp_avg, float* exp_avg_sq, float* dir, int64_t n,
                               float beta1, float beta2, float eps, float bias1, float bias2) {
  const float omb1 = 1.0f - beta1, omb2 = 1.0f - beta2;
  for (int64_t i = 0; i < n; ++i) {
    const float gr = grad[i];
    const float m = fmaf(beta1, exp_avg[i], omb1 * gr);
    const float v = fmaf(beta2, exp_avg_sq[i], (omb2 * gr) * gr);
    exp_avg[i] = m;
    exp_avg_sq[i] = v;
    dir[i] = (m / bias1) / (sqrtf(v / bias2) + eps);
  }
}

/* ---- subspace size from a trust ratio (Section 4.3; Appendix J, hyper-parameter paragraph) --------------------
 * The experiments behind Tables 1-2 do not fix tau: they take the largest number of weights, in the order of
 * decreasing update norm, whose re-encoding keeps ||x_new - x_old|| / ||x_old|| below 0.01, x being the
 * dequantised weights of one matrix.  The procedure the appendix describes -- re-encode a hundredth of the
 * weights at a time until the change exceeds the bound, then put back codes from the end of the last portion
 * until it holds again, always letting one change through -- is driven from pvt_oracle.py; the two functions
 * below supply its arithmetic.
 * Pins: a six-weight example worked by hand (bound met exactly, broken by the first change, never reached),
 * the bound and its maximality recomputed from the dequantised matrices before and after, the longest-prefix
 * form computed from one V step over all groups (which also shows the result does not depend on the portion
 * size), ratio = 0 (one change) and a huge ratio (the plain V step).
 */

/* The order the portions are taken in: the first k groups by (norm descending, index ascending), NOT re-sorted. */
int pvt_oracle_rank(const float* norms, int64_t G, int64_t k, uint32_t* rank_out) {
  if (k < 1 || k > G || G >= ((int64_t)1 << 32)) return -1;
  norm_entry* e = (norm_entry*)malloc((size_t)G * sizeof(norm_entry));
  if (!e) return -1;
  for (int64_t j = 0; j < G; ++j) {
    if (!isfinite(norms[j]) || norms[j] < 0.0f) {
      free(e);
      return -1;
    }
    e[j].n = norms[j];
    e[j].j = (uint32_t)j;
  }
  qsort(e, (size_t)G, sizeof(norm_entry), by_norm_desc_then_index);
  for (int64_t i = 0; i < k; ++i) rank_out[i] = e[i].j;
  free(e);
  return 0;
}

/* Squared change of the dequantised weights of each listed group when its code tuple goes from codes_old to
 * codes_new (both [k][M], one row per listed group): sum over the dg elements, in element order, of
 * (w_new - w_old)^2 with w = s_row * (C_1[b_1] + ... ) formed in binary32 exactly as dequantisation forms it,
 * the difference, the square and the sum in binary64.  sq_old (optional) receives sum w_old^2 of the same groups. */
void pvt_oracle_group_change(const int32_t* codes_old, const int32_t* codes_new, const float* books,
                             const float* scale, int64_t cols, int32_t dg, int32_t M, int32_t K,
                             const uint32_t* idx, int64_t k, double* change_out, double* sq_old) {
  const int64_t gpr = cols / dg;
  for (int64_t n = 0; n < k; ++n) {
    const int64_t r = (int64_t)idx[n] / gpr;
    double acc = 0.0, own = 0.0;
    for (int32_t i = 0; i < dg; ++i) {
      float vo = books[((int64_t)0 * K + codes_old[n * M]) * dg + i];
      float vn = books[((int64_t)0 * K + codes_new[n * M]) * dg + i];
      for (int32_t q = 1; q < M; ++q) {
        vo = vo + books[((int64_t)q * K + codes_old[n * M + q]) * dg + i];
        vn = vn + books[((int64_t)q * K + codes_new[n * M + q]) * dg + i];
      }
      const float wo = scale[r] * vo, wn = scale[r] * vn;
      const double diff = (double)wn - (double)wo;
      acc = acc + diff * diff;
      own = own + (double)wo * (double)wo;
    }
    change_out[n] = acc;
    if (sq_old) sq_old[n] = own;
  }
}

/* ---- local search over single-index changes (Appendix D) ---------------------------------------------------
 * Appendix D's neighbourhood N_1 holds every assignment that differs from the current one in exactly one
 * index, and its local search moves to the best neighbour while that lowers the squared error.  The error is
 * a sum over weight groups, so the search separates: for one group with code tuple (b_1..b_M) the neighbours
 * are the M*(K-1) tuples that differ in one code.  One move = the neighbour that is smallest under
 * (error, tuple), taken only if its error is strictly below the current one; at most max_moves moves.
 * Errors are evaluated exactly as everywhere else in this file (residual carried in binary64 through the
 * codebooks in order), so a run started from the beam search's result can only improve on it.
 * Pins: a two-codebook scalar example worked by hand (two moves to the optimum; a start that is stuck in a
 * local optimum), Appendix D's difference formula hat_x^2 - x^2 - 2 (hat_x - x) B for the scalar case,
 * M = 1 (one move reaches the exhaustive optimum), enumeration of all neighbours by an independent routine
 * (the result has no better neighbour), monotonicity.
 */
int pvt_oracle_local_search(const float* t, int64_t k, int32_t dg, int32_t M, int32_t K, const float* books,
                            int32_t* codes, int32_t max_moves, double* d_out, int32_t* moves_out) {
  if (M < 1 || M > PVT_ORACLE_MAX_M || K < 1 || dg < 1 || dg > 64 || max_moves < 0) return -1;
  int bad = 0;
#pragma omp parallel for schedule(dynamic, 16)
  for (int64_t n = 0; n < k; ++n) {
    beam_entry cur;
    memset(&cur, 0, sizeof cur);
    int ok = 1;
    for (int32_t q = 0; q < M; ++q) {
      cur.code[q] = codes[n * M + q];
      if (cur.code[q] < 0 || cur.code[q] >= K) ok = 0;
    }
    if (!ok) {
      bad = 1;
      continue;
    }
    double r[64];
    residual_of(t + n * dg, books, dg, K, cur.code, M - 1, r);
    cur.d = sqdist(r, books + ((int64_t)(M - 1) * K + cur.code[M - 1]) * dg, dg);
    int32_t moves = 0;
    while (moves < max_moves) {
      beam_entry best = cur;
      int found = 0;
      for (int32_t m = 0; m < M; ++m) {
        for (int32_t q = 0; q < K; ++q) {
          if (q == cur.code[m]) continue;
          beam_entry e = cur;
          e.code[m] = q;
          residual_of(t + n * dg, books, dg, K, e.code, M - 1, r);
          e.d = sqdist(r, books + ((int64_t)(M - 1) * K + e.code[M - 1]) * dg, dg);
          if (!found || entry_less(&e, &best, M)) {
            best = e;
            found = 1;
          }
        }
      }
      if (!found || !(best.d < cur.d)) break;
      cur = best;
      ++moves;
    }
    for (int32_t q = 0; q < M; ++q) codes[n * M + q] = cur.code[q];
    if (d_out) d_out[n] = cur.d;
    if (moves_out) moves_out[n] = moves;
  }
  return bad ? -1 : 0;
}

/* ---- straight-through buffer (Appendix E; Section 3.4 and the "PV + STE" rows of Table 1) -------------------
 * Straight-through estimation keeps an auxiliary, non-quantised copy of the weights.  Every step moves it by the
 * update computed at the quantised weights, and the codes are then chosen to approximate the buffer: updates that
 * are too small to change a code are not lost but add up in the buffer until the stored code stops being the
 * nearest one.  Combined with the subspace V step (the reading taken here): the buffer takes the step of every
 * weight, the subspace is still chosen by the size of this step's update, and the chosen groups are re-encoded
 * against the buffer (the V step's search with W := buffer and a zero step).
 *     buffer_i = fmaf(-eta, g_i, buffer_i)        binary32, one fused operation per weight
 * Pins: a scalar example worked by hand in which four equal small updates flip a code that the plain V step
 * (which restarts from the dequantised weight every time) never flips; eta = 0 leaves the buffer bit for bit;
 * exact rationals for single elements.
 */
void pvt_oracle_ste_accumulate(float* buffer, const float* g, int64_t n, float eta) {
  for (int64_t i = 0; i < n; ++i) buffer[i] = fmaf(-eta, g[i], buffer[i]);
}

/* ---- random subspaces (appendix on small-scale experiments: besides the greedy choice, subspaces drawn
 * uniformly at random, or at random in proportion to the size of the gradient entries) ----------------------
 * Every group j gets a 32-bit random word from a counter-based generator, Philox-4x32 with 10 rounds (Salmon,
 * Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3", SC 2011): counter (j mod 2^32, j div 2^32,
 * 0, 0), key (seed mod 2^32, seed div 2^32), first output word r_j.  The k groups with the largest sampling key
 * are taken, ties towards the lowest index (the same selection rule as the greedy choice):
 *   uniform:       key_j = (float)(r_j >> 8)                  (24 random bits, exact in binary32): a uniformly
 *                  random k-subset.
 *   proportional:  key_j = (float)(w_j / E_j),  E_j = -ln u_j,  u_j = (r_j + 1/2) 2^-32,  w_j = the group's
 *                  squared update norm: the groups with the k earliest arrivals of independent exponential
 *                  clocks of rates w_j, i.e. k draws without replacement, each in proportion to w among the
 *                  groups not yet drawn (Efraimidis and Spirakis, "Weighted random sampling with a reservoir",
 *                  2006).  Groups of weight 0 get key 0.
 * -ln u is evaluated by a fixed sequence of binary64 operations so that it can be reproduced bit for bit:
 *   x = r + 1/2 = m 2^e with m in [1, 2); if m > sqrt 2: m = m/2, e = e + 1;  z = (m - 1)/(m + 1);
 *   p = 1 + z^2/3 + ... + z^20/21 by Horner's rule in z^2 with one fused operation per coefficient;
 *   E = fma(32 - e, ln 2, -(2z * p)).
 * Pins: the generator's published known-answer vectors; E against the C library's logarithm; a k-subset of
 * distinct indices for every k; k = G; inclusion frequencies over many seeds against k/G (uniform) and against
 * w_j / sum w for k = 1 (proportional) within binomial bounds; zero weights never drawn; equal weights behave
 * like the uniform rule in distribution.
 */
void pvt_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3], k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    const uint64_t p0 = (uint64_t)0xD2511F53u * c0, p1 = (uint64_t)0xCD9E8D57u * c2;
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0, n1 = (uint32_t)p1;
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1, n3 = (uint32_t)p0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* -ln((r + 1/2) 2^-32), the fixed binary64 sequence described above */
double pvt_oracle_neglog_u32(uint32_t r) {
  int e = -1;
  if (r) {
    e = 31;
    while (!(r >> e)) --e;
  }
  double m = ldexp((double)r + 0.5, -e); /* exact: in [1, 2) */
  if (m > 1.4142135623730951) {
    m = m * 0.5;
    e = e + 1;
  }
  const double z = (m - 1.0) / (m + 1.0), z2 = z * z;
  double p = 1.0 / 21.0;
  for (int d = 19; d >= 1; d -= 2) p = fma(p, z2, 1.0 / (double)d);
  const double lnm = (2.0 * z) * p;
  return fma((double)(32 - e), 0.6931471805599453, -lnm);
}

/* Sampling keys of all G groups.  mode 0: uniform; mode 1: proportional to norms[j] (binary32, >= 0). */
int pvt_oracle_sample_keys(const float* norms, int64_t G, int32_t mode, uint64_t seed, float* keys_out) {
  if (mode != 0 && mode != 1) return -1;
  if (mode == 1 && !norms) return -1;
  const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  for (int64_t j = 0; j < G; ++j) {
    const uint32_t ctr[4] = {(uint32_t)j, (uint32_t)((uint64_t)j >> 32), 0u, 0u};
    uint32_t out[4];
    pvt_oracle_philox4x32_10(ctr, key, out);
    if (mode == 0) {
      keys_out[j] = (float)(out[0] >> 8);
    } else {
      const float w = norms[j];
      if (!(w >= 0.0f) || !isfinite(w)) return -1;
      keys_out[j] = w > 0.0f ? (float)((double)w / pvt_oracle_neglog_u32(out[0])) : 0.0f;
    }
  }
  return 0;
}
