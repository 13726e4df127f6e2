/*
 * TEST INFRASTRUCTURE -- NOT PART OF THE PRODUCT PATH.
 *
 * Plain fp64 CPU oracle for alpha-entmax / ASEntmax attention, written from the paper's
 * definitions.  Only the tests, the smoke check and the CPU-baseline leg of the benchmark may
 * call it.  It shares no code, header, table or constant with the CUDA library.
 *
 * What each function follows:
 *   oracle_entmax_row          Eq. 1 (alpha-entmax map) and App. A ("alpha-entmax computation"):
 *                              order-based exact threshold for alpha = 2 (sparsemax) and
 *                              alpha = 1.5, bisection inside the bracket of Eq. "bounds_entmax"
 *                              for any other alpha.
 *   oracle_asentmax_scale      Eq. "asentmax": c = delta + beta * (log n)^gamma.
 *   oracle_attn_fwd_rows       Sec. 2.1: z_ij = <q_i,k_j>/sqrt(d) (+ the ALiBi term m (j - i) of App. B when a
 *                              slope is given), causal j <= i, output sum_j p_ij v_j, with the ASEntmax scale
 *                              applied to the whole logit.
 *   oracle_attn_bwd_head       Jacobian of Eq. 1 by implicit differentiation:
 *                              dp_j/ds_k = u_j (delta_jk - u_k / sum u), u = p^(2-alpha).
 *   oracle_attn_bwd_scale_head chain rule through Eq. "asentmax": gradients of the per-row scale c_i and of
 *                              the head's beta, gamma, delta.
 *   oracle_scale_projection(_bwd)  Sec. 4.1: the content-dependent scale, beta = softplus(X w_beta),
 *                              gamma = s tanh(X w_gamma) per query and head, c = delta + beta (log n)^gamma, and the
 *                              chain rule back to w_beta, w_gamma, delta and X.
 *
 * Pins (tests that do not use this file's own arithmetic): the paper's worked sparsemax example,
 * the two-level closed form of Lemma 2, brute-force enumeration of supports for n <= 8, the
 * finite-n scalar equation of the representational-collapse construction, the softmax limit,
 * the Tsallis variational objective, shift/append invariances and central finite differences
 * for the backward pass.  Parity unpinned: none of the row-level functions; the support sizes on
 * the large synthetic workloads have no value printed in the paper to compare against.
 *
 * Conventions: tau is Eq. 1's threshold, i.e. p_j = max((alpha-1) s_j - tau, 0)^(1/(alpha-1)).
 * A logit with (alpha-1) s_j <= tau gets exactly 0 and is outside the support.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_METHOD_AUTO 0
#define ORACLE_METHOD_BISECT 1
#define ORACLE_METHOD_SORT 2

static int cmp_desc(const void* a, const void* b) {
  double x = *(const double*)a, y = *(const double*)b;
  return (x < y) - (x > y);
}

/* y^e for y > 0, with the three exponents that are integers done by multiplication. */
static double pow_pos(double y, double e) {
  if (e == 1.0) return y;
  if (e == 2.0) return y * y;
  if (e == 4.0) { double t = y * y; return t * t; }
  return exp(e * log(y));
}

/* sum_j max(x_j - tau, 0)^e  (x already multiplied by alpha-1) */
static double mass(const double* x, int n, double tau, double e) {
  double acc = 0.0;
  for (int j = 0; j < n; ++j) {
    double y = x[j] - tau;
    if (y > 0.0) acc += pow_pos(y, e);
  }
  return acc;
}

/* App. A: bisection on f(tau) = sum_j [x_j - tau]_+^(1/(alpha-1)) - 1.  The paper states the bracket for
 * logits normalised by their maximum; the caller passes x already shifted so that max x = 0, which turns
 * it into [-1, -n^(1-alpha)] (p_max lies in [1/n, 1]).  Halving stops at an interval of 1e-12; for
 * alpha > 2 it goes on until the interval no longer shrinks in double precision, because there
 * p = y^(1/(alpha-1)) is not Lipschitz at y = 0 and sum p = 1 needs tau at the spacing of doubles near 1
 * (this is also why the search runs on the shifted logits: the spacing near |x_max| would be coarser). */
static double tau_bisect(const double* x, int n, double alpha) {
  double e = 1.0 / (alpha - 1.0);
  double lo = -1.0;
  double hi = -pow((double)n, 1.0 - alpha);
  double tol = alpha > 2.0 ? 0.0 : 1e-12;
  for (int it = 0; it < 200 && (hi - lo) > tol; ++it) {
    double mid = 0.5 * (lo + hi);
    if (!(mid > lo && mid < hi)) break;
    if (mass(x, n, mid, e) >= 1.0) lo = mid; else hi = mid;
  }
  return alpha > 2.0 ? lo : 0.5 * (lo + hi);
}

/* alpha = 2 (sparsemax): sort descending, k* = max{k : 1 + k x_(k) > sum_{l<=k} x_(l)},
 * tau = (sum_{l<=k*} x_(l) - 1) / k*.  x = (alpha-1) z = z. */
static double tau_sort_sparsemax(const double* x, int n, double* scratch) {
  memcpy(scratch, x, sizeof(double) * (size_t)n);
  qsort(scratch, (size_t)n, sizeof(double), cmp_desc);
  double top = scratch[0];
  double csum = 0.0, tau = 0.0;
  for (int k = 1; k <= n; ++k) {
    double xk = scratch[k - 1] - top; /* shifted so that the largest is 0: keeps sums small */
    csum += xk;
    if (1.0 + k * xk > csum) tau = (csum - 1.0) / k; else break;
  }
  return tau + top;
}

/* alpha = 1.5: p_j = (x_j - tau)^2 with x = z/2.  For the k largest, sum (x_(l) - tau)^2 = 1 has
 * the smaller root tau_k = mean_k - sqrt((1 - ss_k)/k), ss_k = sum (x_(l) - mean_k)^2.  The
 * support size is the largest k with tau_k <= x_(k). */
static double tau_sort_15(const double* x, int n, double* scratch) {
  memcpy(scratch, x, sizeof(double) * (size_t)n);
  qsort(scratch, (size_t)n, sizeof(double), cmp_desc);
  double top = scratch[0];
  double s1 = 0.0, s2 = 0.0, tau = -1.0;
  for (int k = 1; k <= n; ++k) {
    double xk = scratch[k - 1] - top;
    s1 += xk;
    s2 += xk * xk;
    double mean = s1 / k;
    double ss = s2 - k * mean * mean;
    double rad = (1.0 - ss) / k;
    if (rad < 0.0) rad = 0.0;
    double tk = mean - sqrt(rad);
    if (tk <= xk) tau = tk; else break;
  }
  return tau + top;
}

/* Eq. 1 on one row of logits z (any real values).  Returns the support size.
 * p may be NULL.  method: ORACLE_METHOD_*. */
int oracle_entmax_row(const double* z, int n, double alpha, int method, double* p, double* tau_out) {
  if (n <= 0 || !(alpha > 1.0)) return -1;
  double* x = (double*)malloc(sizeof(double) * (size_t)n * 2);
  if (!x) return -2;
  double* scratch = x + n;
  double am1 = alpha - 1.0;
  /* x = (alpha-1) z, shifted so that its maximum is 0 (App. A normalises the logits the same way): the
   * threshold of the shifted row lies in [-1, 0), and tau = that threshold + the maximum. */
  double xmax = am1 * z[0];
  for (int j = 1; j < n; ++j) if (am1 * z[j] > xmax) xmax = am1 * z[j];
  for (int j = 0; j < n; ++j) x[j] = am1 * z[j] - xmax;
  double tau;
  int use_sort = (method == ORACLE_METHOD_SORT) ||
                 (method == ORACLE_METHOD_AUTO && (alpha == 2.0 || alpha == 1.5));
  if (use_sort && alpha == 2.0) tau = tau_sort_sparsemax(x, n, scratch);
  else if (use_sort && alpha == 1.5) tau = tau_sort_15(x, n, scratch);
  else tau = tau_bisect(x, n, alpha);
  double e = 1.0 / am1;
  int support = 0;
  for (int j = 0; j < n; ++j) {
    double y = x[j] - tau;
    double pj = 0.0;
    if (y > 0.0) { pj = pow_pos(y, e); ++support; }
    if (p) p[j] = pj;
  }
  if (tau_out) *tau_out = tau + xmax;
  free(x);
  return support;
}

/* Eq. "asentmax": c = delta + beta (log n)^gamma, natural log.  A single visible key (n = 1)
 * has log n = 0, where 0^gamma is undefined for gamma <= 0: the row is one-hot whatever the scale
 * is, and the reading taken is c = delta. */
double oracle_asentmax_scale(double beta, double gamma, double delta, long n) {
  if (n <= 1) return delta;
  return delta + beta * pow(log((double)n), gamma);
}

static long visible_keys(long i, long N, int causal) { return causal ? i + 1 : N; }

/* ALiBi positional term of the logits (App. B "Positional encodings"): z_ij = <q_i,k_j>/sqrt(d) + m (j - i)
 * for j <= i, a penalty linear in the distance; for keys after the query (non-causal use) the same penalty
 * by distance, -m |j - i|.  m = 0 is NoPE. */
static double alibi_bias(double slope, long i, long j) {
  long dist = j <= i ? i - j : j - i;
  return -slope * (double)dist;
}

/* Forward for selected query rows of ONE head.
 *   q,k,v        [N,d] row-major, float (bf16- or fp32-rounded values, converted exactly)
 *   use_scale    0: c_i = 1 (fixed temperature); 1: c_i from beta,gamma,delta
 *   n_mode       0: n_i = number of visible keys of row i; 1: n_i = N
 *   rows         nrows query indices
 *   tau_out      [nrows]; o_out [nrows,d]; p_out NULL or [nrows,N] (zeros where masked)
 *   supp_out     NULL or [nrows] support sizes
 */
int oracle_attn_fwd_rows(const float* q, const float* k, const float* v, long N, int d,
                         double alpha, double sm_scale, int causal, int n_mode, int use_scale,
                         double beta, double gamma, double delta, double alibi_slope,
                         const int64_t* rows, long nrows,
                         double* tau_out, double* o_out, double* p_out, int64_t* supp_out) {
  if (N <= 0 || d <= 0 || !(alpha > 1.0)) return -1;
  int err = 0;
#pragma omp parallel
  {
    double* s = (double*)malloc(sizeof(double) * (size_t)N);
    double* p = (double*)malloc(sizeof(double) * (size_t)N);
    if (!s || !p) {
#pragma omp atomic write
      err = -2;
    } else {
#pragma omp for schedule(dynamic, 4)
      for (long r = 0; r < nrows; ++r) {
        long i = rows[r];
        long nv = visible_keys(i, N, causal);
        long n_i = n_mode ? N : nv;
        double c = use_scale ? oracle_asentmax_scale(beta, gamma, delta, n_i) : 1.0;
        const float* qi = q + (size_t)i * d;
        for (long j = 0; j < nv; ++j) {
          const float* kj = k + (size_t)j * d;
          double dot = 0.0;
          for (int t = 0; t < d; ++t) dot += (double)qi[t] * (double)kj[t];
          s[j] = c * (dot * sm_scale + alibi_bias(alibi_slope, i, j));
        }
        double tau;
        int supp = oracle_entmax_row(s, (int)nv, alpha, ORACLE_METHOD_AUTO, p, &tau);
        tau_out[r] = tau;
        if (supp_out) supp_out[r] = supp;
        double* o = o_out + (size_t)r * d;
        for (int t = 0; t < d; ++t) o[t] = 0.0;
        for (long j = 0; j < nv; ++j) {
          if (p[j] > 0.0) {
            const float* vj = v + (size_t)j * d;
            for (int t = 0; t < d; ++t) o[t] += p[j] * (double)vj[t];
          }
        }
        if (p_out) {
          double* pr = p_out + (size_t)r * N;
          for (long j = 0; j < nv; ++j) pr[j] = p[j];
          for (long j = nv; j < N; ++j) pr[j] = 0.0;
        }
      }
    }
    free(s);
    free(p);
  }
  return err;
}

/* Backward for ONE head, all query rows (dK and dV need every row).
 *   d_o [N,d] float; outputs dq,dk,dv [N,d] double (overwritten).
 * dP_ij = <dO_i, v_j>; u_ij = p_ij^(2-alpha) on the support, 0 off it (alpha = 2: u = 1 there);
 * dS_ij = u_ij (dP_ij - sum_l u_il dP_il / sum_l u_il);
 * dQ_i = g_i sum_j dS_ij k_j, dK_j = sum_i g_i dS_ij q_i with g_i = c_i * sm_scale;
 * dV_j = sum_i p_ij dO_i. */
int oracle_attn_bwd_head(const float* q, const float* k, const float* v, const float* d_o,
                         long N, int d, double alpha, double sm_scale, int causal, int n_mode,
                         int use_scale, double beta, double gamma, double delta, double alibi_slope,
                         double* dq, double* dk, double* dv) {
  if (N <= 0 || d <= 0 || !(alpha > 1.0)) return -1;
  size_t nd = (size_t)N * d;
  memset(dq, 0, sizeof(double) * nd);
  memset(dk, 0, sizeof(double) * nd);
  memset(dv, 0, sizeof(double) * nd);
  int err = 0;
#pragma omp parallel
  {
    double* s = (double*)malloc(sizeof(double) * (size_t)N);
    double* p = (double*)malloc(sizeof(double) * (size_t)N);
    double* dkl = (double*)calloc(nd, sizeof(double));
    double* dvl = (double*)calloc(nd, sizeof(double));
    if (!s || !p || !dkl || !dvl) {
#pragma omp atomic write
      err = -2;
    } else {
#pragma omp for schedule(dynamic, 4)
      for (long i = 0; i < N; ++i) {
        long nv = visible_keys(i, N, causal);
        long n_i = n_mode ? N : nv;
        double c = use_scale ? oracle_asentmax_scale(beta, gamma, delta, n_i) : 1.0;
        double g = c * sm_scale;
        const float* qi = q + (size_t)i * d;
        const float* doi = d_o + (size_t)i * d;
        for (long j = 0; j < nv; ++j) {
          const float* kj = k + (size_t)j * d;
          double dot = 0.0;
          for (int t = 0; t < d; ++t) dot += (double)qi[t] * (double)kj[t];
          s[j] = c * (dot * sm_scale + alibi_bias(alibi_slope, i, j));
        }
        double tau;
        oracle_entmax_row(s, (int)nv, alpha, ORACLE_METHOD_AUTO, p, &tau);
        /* first sweep: sum u and <u, dP>; dP kept in s[] (scores no longer needed) */
        double su = 0.0, sud = 0.0;
        for (long j = 0; j < nv; ++j) {
          if (p[j] > 0.0) {
            const float* vj = v + (size_t)j * d;
            double dp = 0.0;
            for (int t = 0; t < d; ++t) dp += (double)doi[t] * (double)vj[t];
            double u = (alpha == 2.0) ? 1.0 : pow(p[j], 2.0 - alpha);
            s[j] = dp;
            su += u;
            sud += u * dp;
          }
        }
        double rho = sud / su;
        double* dqi = dq + (size_t)i * d;
        for (long j = 0; j < nv; ++j) {
          if (p[j] > 0.0) {
            double u = (alpha == 2.0) ? 1.0 : pow(p[j], 2.0 - alpha);
            double ds = u * (s[j] - rho);
            const float* kj = k + (size_t)j * d;
            double* dkj = dkl + (size_t)j * d;
            double* dvj = dvl + (size_t)j * d;
            for (int t = 0; t < d; ++t) {
              dqi[t] += g * ds * (double)kj[t];
              dkj[t] += g * ds * (double)qi[t];
              dvj[t] += p[j] * (double)doi[t];
            }
          }
        }
      }
#pragma omp critical
      {
        for (size_t t = 0; t < nd; ++t) { dk[t] += dkl[t]; dv[t] += dvl[t]; }
      }
    }
    free(s); free(p); free(dkl); free(dvl);
  }
  return err;
}

/* Row-local part of the backward pass (dQ_i and dS_i) for selected rows of one head.
 * ds_out NULL or [nrows,N]. */
int oracle_attn_bwd_rows(const float* q, const float* k, const float* v, const float* d_o,
                         long N, int d, double alpha, double sm_scale, int causal, int n_mode,
                         int use_scale, double beta, double gamma, double delta, double alibi_slope,
                         const int64_t* rows, long nrows, double* dq_out, double* ds_out) {
  if (N <= 0 || d <= 0 || !(alpha > 1.0)) return -1;
  int err = 0;
#pragma omp parallel
  {
    double* s = (double*)malloc(sizeof(double) * (size_t)N);
    double* p = (double*)malloc(sizeof(double) * (size_t)N);
    if (!s || !p) {
#pragma omp atomic write
      err = -2;
    } else {
#pragma omp for schedule(dynamic, 4)
      for (long r = 0; r < nrows; ++r) {
        long i = rows[r];
        long nv = visible_keys(i, N, causal);
        long n_i = n_mode ? N : nv;
        double c = use_scale ? oracle_asentmax_scale(beta, gamma, delta, n_i) : 1.0;
        double g = c * sm_scale;
        const float* qi = q + (size_t)i * d;
        const float* doi = d_o + (size_t)i * d;
        for (long j = 0; j < nv; ++j) {
          const float* kj = k + (size_t)j * d;
          double dot = 0.0;
          for (int t = 0; t < d; ++t) dot += (double)qi[t] * (double)kj[t];
          s[j] = c * (dot * sm_scale + alibi_bias(alibi_slope, i, j));
        }
        double tau;
        oracle_entmax_row(s, (int)nv, alpha, ORACLE_METHOD_AUTO, p, &tau);
        double su = 0.0, sud = 0.0;
        for (long j = 0; j < nv; ++j) {
          if (p[j] > 0.0) {
            const float* vj = v + (size_t)j * d;
            double dp = 0.0;
            for (int t = 0; t < d; ++t) dp += (double)doi[t] * (double)vj[t];
            double u = (alpha == 2.0) ? 1.0 : pow(p[j], 2.0 - alpha);
            s[j] = dp;
            su += u;
            sud += u * dp;
          }
        }
        double rho = sud / su;
        double* dqi = dq_out + (size_t)r * d;
        for (int t = 0; t < d; ++t) dqi[t] = 0.0;
        if (ds_out) for (long j = 0; j < N; ++j) ds_out[(size_t)r * N + j] = 0.0;
        for (long j = 0; j < nv; ++j) {
          if (p[j] > 0.0) {
            double u = (alpha == 2.0) ? 1.0 : pow(p[j], 2.0 - alpha);
            double ds = u * (s[j] - rho);
            const float* kj = k + (size_t)j * d;
            for (int t = 0; t < d; ++t) dqi[t] += g * ds * (double)kj[t];
            if (ds_out) ds_out[(size_t)r * N + j] = ds;
          }
        }
      }
    }
    free(s); free(p);
  }
  return err;
}

/* Gradients with respect to the ASEntmax scale, ONE head, all query rows.
 * The logits are s_ij = c_i z_ij with z_ij = <q_i,k_j> * sm_scale (Sec. 2.1) and
 * c_i = delta + beta (log n_i)^gamma (Eq. "asentmax"), so by the chain rule
 *   dL/dc_i     = sum_j dS_ij z_ij                       (dc_out [N])
 *   dL/ddelta   = sum_i dL/dc_i
 *   dL/dbeta    = sum_{i: n_i > 1} dL/dc_i (log n_i)^gamma
 *   dL/dgamma   = sum_{i: n_i > 1} dL/dc_i beta (log n_i)^gamma log(log n_i)
 * (rows with n_i = 1 have c_i = delta).  dS as in oracle_attn_bwd_head.  grads_out = {dbeta, dgamma, ddelta}. */
int oracle_attn_bwd_scale_head(const float* q, const float* k, const float* v, const float* d_o,
                               long N, int d, double alpha, double sm_scale, int causal, int n_mode,
                               int use_scale, double beta, double gamma, double delta, double alibi_slope,
                               double* dc_out, double* grads_out) {
  if (N <= 0 || d <= 0 || !(alpha > 1.0)) return -1;
  int err = 0;
#pragma omp parallel
  {
    double* z = (double*)malloc(sizeof(double) * (size_t)N);
    double* s = (double*)malloc(sizeof(double) * (size_t)N);
    double* p = (double*)malloc(sizeof(double) * (size_t)N);
    if (!z || !s || !p) {
#pragma omp atomic write
      err = -2;
    } else {
#pragma omp for schedule(dynamic, 4)
      for (long i = 0; i < N; ++i) {
        long nv = visible_keys(i, N, causal);
        long n_i = n_mode ? N : nv;
        double c = use_scale ? oracle_asentmax_scale(beta, gamma, delta, n_i) : 1.0;
        const float* qi = q + (size_t)i * d;
        const float* doi = d_o + (size_t)i * d;
        for (long j = 0; j < nv; ++j) {
          const float* kj = k + (size_t)j * d;
          double dot = 0.0;
          for (int t = 0; t < d; ++t) dot += (double)qi[t] * (double)kj[t];
          z[j] = dot * sm_scale + alibi_bias(alibi_slope, i, j);
          s[j] = c * z[j];
        }
        double tau;
        oracle_entmax_row(s, (int)nv, alpha, ORACLE_METHOD_AUTO, p, &tau);
        double su = 0.0, sud = 0.0;
        for (long j = 0; j < nv; ++j) {
          if (p[j] > 0.0) {
            const float* vj = v + (size_t)j * d;
            double dp = 0.0;
            for (int t = 0; t < d; ++t) dp += (double)doi[t] * (double)vj[t];
            double u = (alpha == 2.0) ? 1.0 : pow(p[j], 2.0 - alpha);
            s[j] = dp;
            su += u;
            sud += u * dp;
          }
        }
        double rho = sud / su;
        double dc = 0.0;
        for (long j = 0; j < nv; ++j) {
          if (p[j] > 0.0) {
            double u = (alpha == 2.0) ? 1.0 : pow(p[j], 2.0 - alpha);
            dc += u * (s[j] - rho) * z[j];
          }
        }
        dc_out[i] = dc;
      }
    }
    free(z); free(s); free(p);
  }
  if (err) return err;
  double gb = 0.0, gg = 0.0, gd = 0.0;
  for (long i = 0; i < N; ++i) {
    long nv = visible_keys(i, N, causal);
    long n_i = n_mode ? N : nv;
    gd += dc_out[i];
    if (n_i > 1) {
      double L = log((double)n_i);
      double Lg = pow(L, gamma);
      gb += dc_out[i] * Lg;
      gg += dc_out[i] * beta * Lg * log(L);
    }
  }
  grads_out[0] = gb; grads_out[1] = gg; grads_out[2] = gd;
  return 0;
}

/* Sec. 4.1: ASEntmax's scale from the layer input.  For token i of batch element b and head h
 *   beta = softplus(<x_bi, w_beta_h>),  gamma = s tanh(<x_bi, w_gamma_h>),  c = delta_h + beta (log n_i)^gamma
 * (c = delta_h when n_i = 1), n_i = i + 1 under the causal mask, N otherwise or with n_mode = 1.
 *   x [B,N,dm], w_beta, w_gamma [H,dm], delta [H]; outputs c, beta_out, gamma_out [B,H,N] (the last two may be NULL). */
int oracle_scale_projection(const double* x, const double* w_beta, const double* w_gamma, const double* delta,
                            long B, long H, long N, long dm, double s, int causal, int n_mode,
                            double* c, double* beta_out, double* gamma_out) {
  if (B <= 0 || H <= 0 || N <= 0 || dm <= 0) return -1;
  for (long b = 0; b < B; ++b)
    for (long h = 0; h < H; ++h)
      for (long i = 0; i < N; ++i) {
        const double* xi = x + ((size_t)b * N + i) * dm;
        double pb = 0.0, pg = 0.0;
        for (long t = 0; t < dm; ++t) { pb += xi[t] * w_beta[h * dm + t]; pg += xi[t] * w_gamma[h * dm + t]; }
        double beta = pb > 0.0 ? pb + log1p(exp(-pb)) : log1p(exp(pb));   /* softplus, written for both signs */
        double gamma = s * tanh(pg);
        long n_i = (n_mode || !causal) ? N : i + 1;
        size_t at = ((size_t)b * H + h) * N + i;
        c[at] = oracle_asentmax_scale(beta, gamma, delta[h], n_i);
        if (beta_out) beta_out[at] = beta;
        if (gamma_out) gamma_out[at] = gamma;
      }
  return 0;
}

/* Chain rule of the above: given dc = dL/dc [B,H,N],
 *   dL/ddelta_h = sum dc;  with L = log n_i (rows with n_i > 1 only):
 *   dL/dbeta = dc L^gamma,  dL/dgamma = dc beta L^gamma log L,
 *   d beta / d pre_beta = sigmoid(pre_beta),  d gamma / d pre_gamma = s (1 - tanh^2(pre_gamma)),
 *   dL/dw_beta_h = sum_{b,i} g_beta x_bi,  dL/dw_gamma_h likewise,  dL/dx_bi = sum_h (g_beta w_beta_h + g_gamma w_gamma_h).
 * Outputs dw_beta, dw_gamma [H,dm], ddelta [H], dx [B,N,dm] (overwritten). */
int oracle_scale_projection_bwd(const double* x, const double* w_beta, const double* w_gamma, const double* dc,
                                long B, long H, long N, long dm, double s, int causal, int n_mode,
                                double* dw_beta, double* dw_gamma, double* ddelta, double* dx) {
  if (B <= 0 || H <= 0 || N <= 0 || dm <= 0) return -1;
  memset(dw_beta, 0, sizeof(double) * (size_t)H * dm);
  memset(dw_gamma, 0, sizeof(double) * (size_t)H * dm);
  memset(ddelta, 0, sizeof(double) * (size_t)H);
  memset(dx, 0, sizeof(double) * (size_t)B * N * dm);
  for (long b = 0; b < B; ++b)
    for (long h = 0; h < H; ++h)
      for (long i = 0; i < N; ++i) {
        const double* xi = x + ((size_t)b * N + i) * dm;
        double* dxi = dx + ((size_t)b * N + i) * dm;
        double pb = 0.0, pg = 0.0;
        for (long t = 0; t < dm; ++t) { pb += xi[t] * w_beta[h * dm + t]; pg += xi[t] * w_gamma[h * dm + t]; }
        double g = dc[((size_t)b * H + h) * N + i];
        ddelta[h] += g;
        long n_i = (n_mode || !causal) ? N : i + 1;
        if (n_i <= 1) continue;
        double beta = pb > 0.0 ? pb + log1p(exp(-pb)) : log1p(exp(pb));
        double th = tanh(pg);
        double gamma = s * th;
        double L = log((double)n_i), Lg = pow(L, gamma);
        double gb = g * Lg * (1.0 / (1.0 + exp(-pb)));
        double gg = g * beta * Lg * log(L) * s * (1.0 - th * th);
        for (long t = 0; t < dm; ++t) {
          dw_beta[h * dm + t] += gb * xi[t];
          dw_gamma[h * dm + t] += gg * xi[t];
          dxi[t] += gb * w_beta[h * dm + t] + gg * w_gamma[h * dm + t];
        }
      }
  return 0;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

void oracle_set_num_threads(int n) {
#ifdef _OPENMP
  if (n > 0) omp_set_num_threads(n);
#else
  (void)n;
#endif
}
