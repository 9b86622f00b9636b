/*
 * TurboBoA reference oracle (TEST INFRASTRUCTURE, not a product path).
 *
 * Plain, slow, float64 CPU restatement of the out-channel-group quantization
 * loop of TurboBoA (Algorithm 1), its GPTAQ column sweep (Algorithm 2), the
 * joint error-compensation rules (Propositions 3.1 and 3.2) and the
 * coordinate-descent scale refinement (Proposition 3.3 / Algorithm 3).
 *
 * Only tests, the smoke check and the CPU-baseline leg of the benchmark may
 * call this file.  It shares no code with the CUDA library and includes none
 * of its headers.
 *
 * Conventions
 *   W      [d_out][d_in] row-major, row = out-channel; heads are contiguous
 *          blocks of d_head rows (Algorithm 1, input W in R^{H x d_h x d}).
 *   H_in   [n_hin][d_in][d_in]  (n_hin = 1: shared by all heads; = n_heads:
 *          one per head, the W_V row of Table 1).  U_in, R, P, C likewise.
 *   H_out  [n_heads][d_head][d_head], U_out likewise; NULL = identity, i.e.
 *          the GPTQ / GPTAQ row of Table 1 (all rows quantized at once).
 *   U      upper triangular with H^{-1} = U^T U (Eq. 2).
 *   R      alpha * (X - Xfp) X^T, already scaled (Algorithm 1, deviation step).
 *
 * Readings of points the paper leaves open (stated once here, used below):
 *   - integer zero-point z per (row, column group): q = clamp(rne(w/s + z)),
 *     Q = s (q - z).  Every formula of the paper holds with W_int replaced by
 *     Wbar = W_int - z.
 *   - the scale search of Algorithm 1 (grid step) is a search over n_cand clipped
 *     min-max grids, p_k = 1 - k/32, scored by e H_in[G,G] e^T with
 *     round-to-nearest codes, lowest k on ties.
 *   - column groups of quant_group columns each own a (s, z) pair; the score
 *     uses the diagonal block of H_in of that group.
 *   - rounding is round-half-to-even of x = w/s + z.
 *   - by default the grid of a row is fixed before its sweep starts (Algorithm 1
 *     hands the scales to the sweep).  Variant TBO_F_DYNAMIC_GRID: the (s, z) of a
 *     column group is searched when the sweep ARRIVES at the group's first column,
 *     from the group's current values, i.e. after the error feedback of all earlier
 *     columns of the row; same candidates, same score, same tie rule.
 *
 * Loop order: Algorithm 2 walks columns for all rows at once; rows never
 * interact inside the sweep, so this file walks one row at a time (the row
 * loop is the only thing threads are spread over).  No blocking or fusion.
 *
 * Guided comparison: integer decisions (codes, zero-points, grid candidate)
 * are chaotic under error feedback, so a caller comparing another
 * implementation may pass that implementation's decisions as hints.  A hint
 * is adopted only where this oracle's own pre-rounding value lies within
 * `band` of the decision boundary (codes, zeros) or the hinted candidate's
 * score is within cand_tol (relative) of the best score; every adoption is
 * counted.  With NULL hints the oracle decides everything itself.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>

#define TBO_F_ADAPTIVE_GRID 1u
#define TBO_F_CD_REFINE 2u
#define TBO_F_DYNAMIC_GRID 4u /* variant of the reading on column groups: see sweep_row */

typedef struct {
  int d_out, d_in;
  int n_heads, d_head;
  int n_hin;
  int bits;
  int quant_group; /* 0 = one group spanning the whole row */
  int out_block;   /* N of Algorithm 1 */
  int n_cand;
  int cd_iters;
  unsigned flags;
} tbo_desc;

typedef struct {
  long long near_tie_codes; /* own x within band of a boundary that matters */
  long long adopted_codes;
  long long adopted_zeros;
  long long adopted_cands;
} tbo_counters;

static double rne(double x) { return nearbyint(x); } /* default mode: half-to-even */

static double clampd(double v, double lo, double hi) { return v < lo ? lo : (v > hi ? hi : v); }

/* ------------------------------------------------------------------------- */
/* Grid for one row segment (Algorithm 1, grid step).                         */
/* w: n weights; H: the n x n diagonal block of H_in (leading dimension ldh). */
/* Returns chosen candidate; writes s, z and (optionally) all scores.         */
/* ------------------------------------------------------------------------- */
static int grid_segment(const double *w, int n, const double *H, int ldh, int maxq, int n_cand,
                        double band, double cand_tol, int hint_cand, int hint_zero,
                        double *s_out, int *z_out, double *scores, tbo_counters *cnt) {
  double mn = 0.0, mx = 0.0;
  for (int a = 0; a < n; ++a) {
    if (w[a] < mn) mn = w[a];
    if (w[a] > mx) mx = w[a];
  }
  double *e = (double *)malloc(sizeof(double) * (size_t)n);
  double best_J = 0.0, best_s = 1.0;
  int best_k = -1, best_z = 0;
  double hint_J = 0.0, hint_s = 1.0;
  int hint_z = 0, hint_ok = 0;
  for (int k = 0; k < n_cand; ++k) {
    double p = 1.0 - (double)k / 32.0;
    double lo = p * mn, hi = p * mx;
    double s, z;
    int z_adopted = 0;
    if (hi == lo) {
      s = 1.0;
      z = 0.0;
    } else {
      s = (hi - lo) / (double)maxq;
      double xz = -lo / s;
      z = clampd(rne(xz), 0.0, (double)maxq);
      /* zero-point near-tie: adopt the hinted neighbour inside the band */
      if (hint_zero >= 0 && k == hint_cand && (double)hint_zero != z) {
        double fl = floor(xz);
        if (fabs(xz - (fl + 0.5)) < band) {
          double a0 = clampd(fl, 0.0, (double)maxq), a1 = clampd(fl + 1.0, 0.0, (double)maxq);
          if ((double)hint_zero == a0 || (double)hint_zero == a1) {
            z = (double)hint_zero;
            z_adopted = 1;
          }
        }
      }
    }
    for (int a = 0; a < n; ++a) {
      double c = clampd(rne(w[a] / s + z), 0.0, (double)maxq);
      e[a] = w[a] - s * (c - z);
    }
    double J = 0.0;
    for (int a = 0; a < n; ++a) {
      double t = 0.0;
      for (int b = 0; b < n; ++b) t += H[(size_t)a * ldh + b] * e[b];
      J += e[a] * t;
    }
    if (scores) scores[k] = J;
    if (best_k < 0 || J < best_J) { /* strict <: lowest k wins ties */
      best_J = J;
      best_k = k;
      best_s = s;
      best_z = (int)z;
    }
    if (k == hint_cand) {
      hint_J = J;
      hint_s = s;
      hint_z = (int)z;
      hint_ok = 1;
      if (z_adopted) hint_ok = 2; /* counted below, only if this candidate is used */
    }
  }
  free(e);
  int use_k = best_k;
  double use_s = best_s;
  int use_z = best_z;
  if (hint_ok && hint_cand != best_k) {
    double tol = cand_tol * fabs(best_J);
    if (hint_J - best_J <= tol) {
      use_k = hint_cand;
      use_s = hint_s;
      use_z = hint_z;
      if (cnt) {
#pragma omp atomic
        cnt->adopted_cands++;
      }
    }
  }
  if (hint_ok == 2 && use_k == hint_cand && cnt) {
#pragma omp atomic
    cnt->adopted_zeros++;
  }
  *s_out = use_s;
  *z_out = use_z;
  return use_k;
}

/* Grid for one full row: one segment per column group. */
static void grid_row(const double *w, int d, int gq, const double *Hin, int maxq, int n_cand,
                     double band, double cand_tol, const unsigned char *hint_cand,
                     const int *hint_zero, double *s, int *z, unsigned char *cand,
                     tbo_counters *cnt) {
  int seg = gq > 0 ? gq : d;
  int ng = d / seg;
  for (int g = 0; g < ng; ++g) {
    int c0 = g * seg;
    int hc = hint_cand ? (int)hint_cand[g] : -1;
    int hz = hint_zero ? hint_zero[g] : -1;
    int k = grid_segment(w + c0, seg, Hin + (size_t)c0 * d + c0, d, maxq, n_cand, band, cand_tol,
                         hc, hz, &s[g], &z[g], NULL, cnt);
    if (cand) cand[g] = (unsigned char)k;
  }
}

/* ------------------------------------------------------------------------- */
/* GPTAQ sweep of one row (Algorithm 2, its column loop).                     */
/* w: working copy, overwritten (on return w[j] is NOT meaningful).           */
/* U: upper factor of H_in^{-1}; P: strictly upper correction or NULL.        */
/* ------------------------------------------------------------------------- */
typedef struct { /* dynamic-grid variant: what the in-sweep search needs (Hin NULL = grid fixed beforehand) */
  const double *Hin;
  int n_cand;
  double cand_tol;
  const unsigned char *hint_cand;
  const int *hint_zero;
  unsigned char *cand;
} tbo_dyn;

static void sweep_row(double *w, int d, int gq, const double *U, const double *P, double *s, int *z,
                      int maxq, double band, const unsigned char *hint, unsigned char *codes,
                      double *Q, double *err, tbo_counters *cnt, const tbo_dyn *dyn) {
  int seg = gq > 0 ? gq : d;
  long long near = 0, adopted = 0;
  for (int j = 0; j < d; ++j) {
    int g = j / seg;
    if (dyn && dyn->Hin && j % seg == 0) {
      /* the group's grid from its values on arrival (all earlier columns' feedback applied) */
      int k = grid_segment(w + j, seg, dyn->Hin + (size_t)j * d + j, d, maxq, dyn->n_cand, band,
                           dyn->cand_tol, dyn->hint_cand ? (int)dyn->hint_cand[g] : -1,
                           dyn->hint_zero ? dyn->hint_zero[g] : -1, &s[g], &z[g], NULL, cnt);
      if (dyn->cand) dyn->cand[g] = (unsigned char)k;
    }
    double sj = s[g], zj = (double)z[g];
    double wj = w[j]; /* value on arrival at column j */
    double x = wj / sj + zj;
    double q = clampd(rne(x), 0.0, (double)maxq);
    double fl = floor(x);
    if (fabs(x - (fl + 0.5)) < band) {
      double a0 = clampd(fl, 0.0, (double)maxq), a1 = clampd(fl + 1.0, 0.0, (double)maxq);
      if (a0 != a1) {
        near++;
        if (hint && (double)hint[j] != q && ((double)hint[j] == a0 || (double)hint[j] == a1)) {
          q = (double)hint[j];
          adopted++;
        }
      }
    }
    double Qj = sj * (q - zj);
    double ej = (wj - Qj) / U[(size_t)j * d + j];
    codes[j] = (unsigned char)q;
    Q[j] = Qj;
    if (err) err[j] = ej;
    const double *Uj = U + (size_t)j * d;
    if (P) {
      const double *Pj = P + (size_t)j * d;
      for (int k = j + 1; k < d; ++k) w[k] = w[k] - ej * Uj[k] - wj * Pj[k];
    } else {
      for (int k = j + 1; k < d; ++k) w[k] = w[k] - ej * Uj[k];
    }
  }
  if (cnt) {
#pragma omp atomic
    cnt->near_tie_codes += near;
#pragma omp atomic
    cnt->adopted_codes += adopted;
  }
}

/* ------------------------------------------------------------------------- */
/* T = [U_out^T]_{rem,B} ([U_out^T]_{B,B})^{-1}  (Propositions 3.1 / 3.2).    */
/* Uo: d_head x d_head upper factor; B = {i0..i0+nb-1}; rem = {i0+nb..dh-1}.  */
/* T: [n_rem][nb].                                                            */
/* ------------------------------------------------------------------------- */
static void comp_matrix(const double *Uo, int dh, int i0, int nb, double *T) {
  int r0 = i0 + nb, nrem = dh - r0;
  /* A = U_out^T is lower triangular: A[a][b] = Uo[b][a].  Solve T A_BB = A_remB
     column by column, last column first. */
  for (int r = 0; r < nrem; ++r) {
    double *Tr = T + (size_t)r * nb;
    for (int c = nb - 1; c >= 0; --c) {
      double v = Uo[(size_t)(i0 + c) * dh + (r0 + r)]; /* A[rem r][B c] */
      for (int c2 = c + 1; c2 < nb; ++c2)
        v -= Tr[c2] * Uo[(size_t)(i0 + c) * dh + (i0 + c2)]; /* A[B c2][B c] */
      Tr[c] = v / Uo[(size_t)(i0 + c) * dh + (i0 + c)];
    }
  }
}

/* ------------------------------------------------------------------------- */
/* Group loop of Algorithm 1 for one head.                                    */
/* Wt: [dh][d] working weights W-tilde (in: original rows; out: Q rows).      */
/* ------------------------------------------------------------------------- */
static void group_loop_head(const tbo_desc *D, double *Wt, const double *Hin, const double *Uin,
                            const double *Uo /* NULL = identity */, const double *P,
                            const double *C, double band, double cand_tol,
                            const unsigned char *hint_codes, const int *hint_zeros,
                            const unsigned char *hint_cand, unsigned char *codes, double *scales,
                            int *zeros, unsigned char *cand, double *Q, double *Wcomp,
                            double *trace /* [n_steps][dh][d] W-tilde after each step, or NULL */,
                            tbo_counters *cnt) {
  const int dh = D->d_head, d = D->d_in, gq = D->quant_group;
  const int seg = gq > 0 ? gq : d, ng = d / seg;
  const int maxq = (1 << D->bits) - 1;
  const int dynamic = (D->flags & TBO_F_DYNAMIC_GRID) != 0;
  const int adaptive = (D->flags & TBO_F_ADAPTIVE_GRID) != 0 && !dynamic;
  const int N = Uo ? D->out_block : dh; /* H_out = I: every row at once */

  if (!adaptive && !dynamic) {
    /* fixed grid: computed once from the original weights, all rows */
#pragma omp parallel for schedule(dynamic)
    for (int r = 0; r < dh; ++r)
      grid_row(Wt + (size_t)r * d, d, gq, Hin, maxq, D->n_cand, band, cand_tol,
               hint_cand ? hint_cand + (size_t)r * ng : NULL,
               hint_zeros ? hint_zeros + (size_t)r * ng : NULL, scales + (size_t)r * ng,
               zeros + (size_t)r * ng, cand ? cand + (size_t)r * ng : NULL, cnt);
  }

  for (int i0 = 0; i0 < dh; i0 += N) {
    int nb = (i0 + N <= dh) ? N : dh - i0;
    int r0 = i0 + nb, nrem = dh - r0;
    double *E = (double *)malloc(sizeof(double) * (size_t)nb * d);
    /* rows of B: grid, sweep, error E = W0 - Q (minus W0 C with the R term) */
#pragma omp parallel for schedule(dynamic)
    for (int b = 0; b < nb; ++b) {
      int r = i0 + b;
      double *w0 = Wt + (size_t)r * d; /* snapshot W^(i) row */
      if (Wcomp) memcpy(Wcomp + (size_t)r * d, w0, sizeof(double) * (size_t)d);
      if (adaptive)
        grid_row(w0, d, gq, Hin, maxq, D->n_cand, band, cand_tol,
                 hint_cand ? hint_cand + (size_t)r * ng : NULL,
                 hint_zeros ? hint_zeros + (size_t)r * ng : NULL, scales + (size_t)r * ng,
                 zeros + (size_t)r * ng, cand ? cand + (size_t)r * ng : NULL, cnt);
      double *w = (double *)malloc(sizeof(double) * (size_t)d);
      memcpy(w, w0, sizeof(double) * (size_t)d);
      tbo_dyn dyn = {dynamic ? Hin : NULL, D->n_cand, cand_tol,
                     hint_cand ? hint_cand + (size_t)r * ng : NULL,
                     hint_zeros ? hint_zeros + (size_t)r * ng : NULL,
                     cand ? cand + (size_t)r * ng : NULL};
      sweep_row(w, d, gq, Uin, P, scales + (size_t)r * ng, zeros + (size_t)r * ng, maxq, band,
                hint_codes ? hint_codes + (size_t)r * d : NULL, codes + (size_t)r * d,
                Q + (size_t)r * d, NULL, cnt, &dyn);
      free(w);
      double *Er = E + (size_t)b * d;
      for (int k = 0; k < d; ++k) Er[k] = w0[k] - Q[(size_t)r * d + k];
      if (C) { /* propagated-error term: E <- E - W0 (R H_in^{-1}) */
        for (int a = 0; a < d; ++a) {
          double wa = w0[a];
          const double *Ca = C + (size_t)a * d;
          for (int k = 0; k < d; ++k) Er[k] -= wa * Ca[k];
        }
      }
    }
    if (Uo && nrem > 0) {
      double *T = (double *)malloc(sizeof(double) * (size_t)nrem * nb);
      comp_matrix(Uo, dh, i0, nb, T);
#pragma omp parallel for schedule(static)
      for (int r = 0; r < nrem; ++r) {
        double *wr = Wt + (size_t)(r0 + r) * d;
        for (int b = 0; b < nb; ++b) {
          double t = T[(size_t)r * nb + b];
          const double *Eb = E + (size_t)b * d;
          for (int k = 0; k < d; ++k) wr[k] -= t * Eb[k];
        }
      }
      free(T);
    }
    for (int b = 0; b < nb; ++b)
      memcpy(Wt + (size_t)(i0 + b) * d, Q + (size_t)(i0 + b) * d, sizeof(double) * (size_t)d);
    free(E);
    if (trace) memcpy(trace + (size_t)(i0 / N) * dh * d, Wt, sizeof(double) * (size_t)dh * d);
  }
}

/* ------------------------------------------------------------------------- */
/* Coordinate-descent scale refinement for one head (Algorithm 3).            */
/* The numerator needs row j of Hout ((Q - W) Hin + W R).  The inner product  */
/* Dm = (Q - W) Hin + W R is kept current: when Q's row changes by            */
/* delta * Wbar[j,G], row j of Dm changes by delta * Wbar[j,G] Hin[G,:]       */
/* (that is the weight-update step of Algorithm 3, carried                     */
/* through the product).                                                      */
/* ------------------------------------------------------------------------- */
static void cd_head(const tbo_desc *D, const double *W, const unsigned char *codes,
                    const int *zeros, double *scales, const double *Hin, const double *Hout,
                    const double *R) {
  const int dh = D->d_head, d = D->d_in, gq = D->quant_group;
  const int seg = gq > 0 ? gq : d, ng = d / seg;
  double *Wb = (double *)malloc(sizeof(double) * (size_t)dh * d);
  double *Dm = (double *)calloc((size_t)dh * d, sizeof(double));
#pragma omp parallel for schedule(static)
  for (int r = 0; r < dh; ++r) {
    double *dr = Dm + (size_t)r * d;
    for (int a = 0; a < d; ++a) {
      int g = a / seg;
      double wb = (double)codes[(size_t)r * d + a] - (double)zeros[(size_t)r * ng + g];
      Wb[(size_t)r * d + a] = wb;
      double diff = scales[(size_t)r * ng + g] * wb - W[(size_t)r * d + a];
      const double *Ha = Hin + (size_t)a * d;
      for (int k = 0; k < d; ++k) dr[k] += diff * Ha[k];
      if (R) {
        double wa = W[(size_t)r * d + a];
        const double *Ra = R + (size_t)a * d;
        for (int k = 0; k < d; ++k) dr[k] += wa * Ra[k];
      }
    }
  }
  for (int it = 0; it < D->cd_iters; ++it) {
    for (int j = 0; j < dh; ++j) {
      const double *wbj = Wb + (size_t)j * d;
      for (int g = 0; g < ng; ++g) {
        int c0 = g * seg;
        double num = 0.0;
        for (int a = c0; a < c0 + seg; ++a) {
          double Gja = 0.0; /* [Hout Dm]_{j,a} */
          if (Hout) {
            for (int i = 0; i < dh; ++i) Gja += Hout[(size_t)j * dh + i] * Dm[(size_t)i * d + a];
          } else {
            Gja = Dm[(size_t)j * d + a];
          }
          num += wbj[a] * Gja;
        }
        double quad = 0.0;
        for (int a = c0; a < c0 + seg; ++a) {
          double t = 0.0;
          for (int b = c0; b < c0 + seg; ++b) t += Hin[(size_t)a * d + b] * wbj[b];
          quad += wbj[a] * t;
        }
        double hjj = Hout ? Hout[(size_t)j * dh + j] : 1.0;
        double den = quad * hjj;
        if (den == 0.0) continue;
        double delta = -num / den;
        scales[(size_t)j * ng + g] += delta;
        double *dj = Dm + (size_t)j * d;
        for (int a = c0; a < c0 + seg; ++a) {
          double c = delta * wbj[a];
          if (c == 0.0) continue;
          const double *Ha = Hin + (size_t)a * d;
          for (int k = 0; k < d; ++k) dj[k] += c * Ha[k];
        }
      }
    }
  }
  free(Wb);
  free(Dm);
}

/* ------------------------------------------------------------------------- */
/* Loss of one head: tr(dW Hin dW^T Hout) + 2 tr(Hout W R dW^T), dW = Q - W   */
/* (first line of the Lagrangian in the proof of Proposition 3.1; expansion   */
/* at the start of the proof of Proposition 3.2).                             */
/* ------------------------------------------------------------------------- */
static double loss_head(int dh, int d, const double *W, const double *Q, const double *Hin,
                        const double *Hout, const double *R) {
  double *Z = (double *)calloc((size_t)dh * d, sizeof(double)); /* dW Hin + W R */
  double *dW = (double *)malloc(sizeof(double) * (size_t)dh * d);
#pragma omp parallel for schedule(static)
  for (int r = 0; r < dh; ++r) {
    double *zr = Z + (size_t)r * d;
    for (int a = 0; a < d; ++a) {
      double dw = Q[(size_t)r * d + a] - W[(size_t)r * d + a];
      dW[(size_t)r * d + a] = dw;
      const double *Ha = Hin + (size_t)a * d;
      for (int k = 0; k < d; ++k) zr[k] += dw * Ha[k];
      if (R) {
        double wa = 2.0 * W[(size_t)r * d + a];
        const double *Ra = R + (size_t)a * d;
        for (int k = 0; k < d; ++k) zr[k] += wa * Ra[k];
      }
    }
  }
  double total = 0.0;
#pragma omp parallel for schedule(static) reduction(+ : total)
  for (int j = 0; j < dh; ++j) {
    for (int i = 0; i < dh; ++i) {
      double h = Hout ? Hout[(size_t)j * dh + i] : (i == j ? 1.0 : 0.0);
      if (h == 0.0) continue;
      double dot = 0.0;
      for (int k = 0; k < d; ++k) dot += Z[(size_t)i * d + k] * dW[(size_t)j * d + k];
      total += h * dot;
    }
  }
  free(Z);
  free(dW);
  return total;
}

/* ------------------------------------------------------------------------- */
/* Entry points                                                               */
/* ------------------------------------------------------------------------- */

/* Full per-projection procedure (Algorithm 1 for one W).
 * Returns 0, or a negative number for an invalid description.
 * scales_pre (optional) receives the scales before CD refinement. */
int tbo_quantize_layer(const tbo_desc *D, const double *W, const double *Hin, const double *Uin,
                       const double *Hout, const double *Uout, const double *R, const double *P,
                       const double *C, double band, double cand_tol,
                       const unsigned char *hint_codes, const int *hint_zeros,
                       const unsigned char *hint_cand, unsigned char *codes, double *scales,
                       int *zeros, unsigned char *cand, double *What, double *Wcomp,
                       double *scales_pre, double *loss, tbo_counters *cnt) {
  const int dh = D->d_head, d = D->d_in, H = D->n_heads;
  if (D->d_out != H * dh || d <= 0 || D->bits < 1 || D->bits > 8) return -1;
  const int seg = D->quant_group > 0 ? D->quant_group : d;
  if (d % seg) return -2;
  if (D->n_hin != 1 && D->n_hin != H) return -3;
  if (D->out_block < 1) return -4;
  const int ng = d / seg;
  const size_t dd = (size_t)d * d;
  if (cnt) memset(cnt, 0, sizeof(*cnt));
  double *Wt = (double *)malloc(sizeof(double) * (size_t)dh * d);
  double *Q = (double *)malloc(sizeof(double) * (size_t)dh * d);
  for (int h = 0; h < H; ++h) {
    size_t ro = (size_t)h * dh;
    size_t io = D->n_hin == 1 ? 0 : (size_t)h * dd;
    const double *Wh = W + ro * d;
    const double *Hin_h = Hin + io, *Uin_h = Uin + io;
    const double *Rh = R ? R + io : NULL, *Ph = R ? P + io : NULL, *Ch = R ? C + io : NULL;
    const double *Ho = Hout ? Hout + (size_t)h * dh * dh : NULL;
    const double *Uo = Hout ? Uout + (size_t)h * dh * dh : NULL;
    memcpy(Wt, Wh, sizeof(double) * (size_t)dh * d);
    group_loop_head(D, Wt, Hin_h, Uin_h, Uo, Ph, Ch, band, cand_tol,
                    hint_codes ? hint_codes + ro * d : NULL, hint_zeros ? hint_zeros + ro * ng : NULL,
                    hint_cand ? hint_cand + ro * ng : NULL, codes + ro * d, scales + ro * ng,
                    zeros + ro * ng, cand ? cand + ro * ng : NULL, Q,
                    Wcomp ? Wcomp + ro * d : NULL, NULL, cnt);
    if (scales_pre) memcpy(scales_pre + ro * ng, scales + ro * ng, sizeof(double) * (size_t)dh * ng);
    if ((D->flags & TBO_F_CD_REFINE) && D->cd_iters > 0)
      cd_head(D, Wh, codes + ro * d, zeros + ro * ng, scales + ro * ng, Hin_h, Ho, Rh);
    /* Q <- diag(s) W_int (Algorithm 1, final step) */
    for (int r = 0; r < dh; ++r)
      for (int a = 0; a < d; ++a) {
        int g = a / seg;
        double wb = (double)codes[(ro + r) * d + a] - (double)zeros[(ro + r) * ng + g];
        Q[(size_t)r * d + a] = scales[(ro + r) * ng + g] * wb;
      }
    memcpy(What + ro * d, Q, sizeof(double) * (size_t)dh * d);
    if (loss) loss[h] = loss_head(dh, d, Wh, Q, Hin_h, Ho, Rh);
  }
  free(Wt);
  free(Q);
  return 0;
}

/* Stand-alone pieces, exported so that tests can pin each one. */

/* Group loop of one head with W-tilde recorded after every step.
 * Wt [dh][d] in: original rows, out: quantized rows. */
void tbo_group_loop_trace(const tbo_desc *D, double *Wt, const double *Hin, const double *Uin,
                          const double *Uout, const double *P, const double *C,
                          unsigned char *codes, double *scales, int *zeros, double *Q,
                          double *Wcomp, double *trace) {
  group_loop_head(D, Wt, Hin, Uin, Uout, P, C, 0.0, 0.0, NULL, NULL, NULL, codes, scales, zeros,
                  NULL, Q, Wcomp, trace, NULL);
}

void tbo_grid_rows(const double *W0, int m, int d, int gq, const double *Hin, int bits, int n_cand,
                   double *s, int *z, unsigned char *cand, double *scores /* [m][ng][n_cand] or NULL */) {
  int seg = gq > 0 ? gq : d, ng = d / seg, maxq = (1 << bits) - 1;
#pragma omp parallel for schedule(dynamic)
  for (int r = 0; r < m; ++r)
    for (int g = 0; g < ng; ++g) {
      int c0 = g * seg;
      int k = grid_segment(W0 + (size_t)r * d + c0, seg, Hin + (size_t)c0 * d + c0, d, maxq, n_cand,
                           0.0, 0.0, -1, -1, &s[(size_t)r * ng + g], &z[(size_t)r * ng + g],
                           scores ? scores + ((size_t)r * ng + g) * n_cand : NULL, NULL);
      if (cand) cand[(size_t)r * ng + g] = (unsigned char)k;
    }
}

/* Hin_dyn != NULL selects the dynamic-grid variant: s and z are then outputs. */
void tbo_sweep_rows(const double *W0, int m, int d, int gq, const double *Uin, const double *P,
                    double *s, int *z, int bits, double band, const unsigned char *hint_codes,
                    unsigned char *codes, double *Q, double *err, tbo_counters *cnt,
                    const double *Hin_dyn, int n_cand) {
  int seg = gq > 0 ? gq : d, ng = d / seg, maxq = (1 << bits) - 1;
  if (cnt) memset(cnt, 0, sizeof(*cnt));
#pragma omp parallel for schedule(dynamic)
  for (int r = 0; r < m; ++r) {
    double *w = (double *)malloc(sizeof(double) * (size_t)d);
    memcpy(w, W0 + (size_t)r * d, sizeof(double) * (size_t)d);
    tbo_dyn dyn = {Hin_dyn, n_cand, 0.0, NULL, NULL, NULL};
    sweep_row(w, d, gq, Uin, P, s + (size_t)r * ng, z + (size_t)r * ng, maxq, band,
              hint_codes ? hint_codes + (size_t)r * d : NULL, codes + (size_t)r * d,
              Q + (size_t)r * d, err ? err + (size_t)r * d : NULL, cnt, &dyn);
    free(w);
  }
}

void tbo_comp_matrix(const double *Uo, int dh, int i0, int nb, double *T) {
  comp_matrix(Uo, dh, i0, nb, T);
}

void tbo_cd_refine(const tbo_desc *D, const double *W, const unsigned char *codes, const int *zeros,
                   double *scales, const double *Hin, const double *Hout, const double *R) {
  cd_head(D, W, codes, zeros, scales, Hin, Hout, R);
}

double tbo_loss_head(int dh, int d, const double *W, const double *Q, const double *Hin,
                     const double *Hout, const double *R) {
  return loss_head(dh, d, W, Q, Hin, Hout, R);
}

int tbo_num_threads(void) {
#ifdef _OPENMP
  extern int omp_get_max_threads(void);
  return omp_get_max_threads();
#else
  return 1;
#endif
}
