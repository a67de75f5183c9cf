/*
 * CPU oracle for causal linear attention with per-head exponential decay.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, fp64 statement of
 * what the method computes.  It shares no code, header, table or constant with
 * the CUDA library and must never be called from the product path; only the
 * tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * The method reaches exactly (up to rounding order) a result with a plain
 * definition, so every routine here is that definition written out:
 *
 *   masked quadratic form (Section 3.2.1, "Lightning Attention"; Algorithms 3/4)
 *       O = (Q K^T (.) M) V,   M_ts = lambda^(t-s) for t >= s, else 0
 *   token recurrence (Algorithm 2, "Robust Inference")
 *       kv_t = lambda kv_{t-1} + k_t v_t^T,   o_t = kv_t^T q_t,   kv_0 = 0
 *   prescaled recurrence (Algorithm 1, "Origin Inference"), kept only to show
 *       where it loses precision and overflows.
 *   normalisation and gate that follow the attention product in the token mixer
 *       (Eq. 3 "Gated Linear Attention" with Eq. 8 "SimpleRMSNorm"), per row of
 *       e values:  y = o / (||o||_2 / sqrt(e)) (.) u,  and its gradients.
 *
 * Layout: q,k [B,H,N,d], v,o,dO [B,H,N,e], states [B,H,d,e] with
 * kv[i][j] = sum_s lambda^(t-s) k_s[i] v_s[j]; everything row-major contiguous.
 * Inputs are fp32 containers holding the exact input values (bf16 widens to
 * fp32 exactly); all arithmetic and all outputs are fp64.  lambda is per head.
 *
 * Gradients are those of L = <O, dO> (+ <kv_out, grad_kv_out> when a state is
 * handed over).  lambda is not learnable (Section 3.1.1), so it has no gradient.
 *
 * Readings of the paper taken here:
 *   - the diagonal term s = t is included (Algorithm 2 adds k_t v_t^T before
 *     reading o_t), so M_tt = 1;
 *   - no 1/sqrt(d) scaling and no softmax (Section 3.1.4);
 *   - Algorithm 4's update lines are read as dK_j += dA_ij^T Q_i and
 *     dQ_i += dA_ij K_j (the printed right-hand sides do not type-check), and
 *     O is not an input of the backward pass;
 *   - the state starts at zero unless kv_in is given; kv_out is the state after
 *     the last token with no extra decay;
 *   - SimpleRMSNorm is applied to each head's e output values of a token (the
 *     model-parallel form of Eq. 3 normalises each rank's heads on their own);
 *     Eq. 8 has no epsilon, so a row with ||o||_2 = 0 is given y = 0 and zero
 *     gradients;
 *   - Eq. 1's rotation (LRPE-d): theta is one learnable angle per head and per
 *     feature, the score is the real part of the complex expression,
 *       a_ts = lambda^(t-s) sum_i q_t[i] k_s[i] cos(theta[h][i] (t - s)),  s <= t
 *     (the paper prints a bare theta; the cited LRPE work uses one angle per
 *     feature, and a single angle is the special case of equal entries).
 *
 * Every routine is pinned by tests that do not call it twice: closed forms,
 * a hand-worked example, numpy prefix sums for lambda = 1, brute force on tiny
 * inputs, finite differences for the gradients, and form-against-form checks.
 */
#include <math.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_OK 0
#define ORC_ERR 1

int orc_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* lambda^n for integer n >= 0: the mask entry M_ts with n = t - s. */
static double mask_entry(double lambda, long n) { return pow(lambda, (double)n); }

/* ------------------------------------------------------------------------- */
/* Token recurrence, forward (Algorithm 2).                                    */
/* ------------------------------------------------------------------------- */
int orc_fwd_rec(const float* q, const float* k, const float* v, const double* lambda,
                const double* kv_in, int B, int H, int N, int d, int e,
                double* o, double* kv_out) {
  if (B < 0 || H < 0 || N < 0 || d < 1 || e < 1) return ORC_ERR;
  const long BH = (long)B * H;
  int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
  for (long bh = 0; bh < BH; ++bh) {
    const double lam = lambda[bh % H];
    double* kv = (double*)malloc(sizeof(double) * d * e);
    if (!kv) { failed = 1; continue; }
    if (kv_in) memcpy(kv, kv_in + bh * d * e, sizeof(double) * d * e);
    else memset(kv, 0, sizeof(double) * d * e);
    for (long t = 0; t < N; ++t) {
      const float* qt = q + (bh * N + t) * d;
      const float* kt = k + (bh * N + t) * d;
      const float* vt = v + (bh * N + t) * e;
      double* ot = o + (bh * N + t) * e;
      /* kv_t = lambda kv_{t-1} + k_t v_t^T */
      for (int i = 0; i < d; ++i)
        for (int j = 0; j < e; ++j)
          kv[i * e + j] = lam * kv[i * e + j] + (double)kt[i] * (double)vt[j];
      /* o_t = kv_t^T q_t */
      for (int j = 0; j < e; ++j) ot[j] = 0.0;
      for (int i = 0; i < d; ++i)
        for (int j = 0; j < e; ++j) ot[j] += kv[i * e + j] * (double)qt[i];
    }
    if (kv_out) memcpy(kv_out + bh * d * e, kv, sizeof(double) * d * e);
    free(kv);
  }
  return failed ? ORC_ERR : ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* Token recurrence, backward.                                                 */
/* Chain rule through Algorithm 2:                                             */
/*   dq_t = kv_t do_t                       (forward-running state)            */
/*   R_s  = sum_{t>=s} lambda^(t-s) q_t do_t^T = lambda R_{s+1} + q_s do_s^T   */
/*   dk_s = R_s v_s,  dv_s = R_s^T k_s      (reverse-running state)            */
/* With a handed-over state: R starts from grad_kv_out, and                    */
/*   grad_kv_in = lambda R_0 (the gradient w.r.t. the state before token 0).   */
/* ------------------------------------------------------------------------- */
int orc_bwd_rec(const float* q, const float* k, const float* v, const float* d_o,
                const double* lambda, const double* kv_in, const double* grad_kv_out,
                int B, int H, int N, int d, int e,
                double* dq, double* dk, double* dv, double* grad_kv_in) {
  if (B < 0 || H < 0 || N < 0 || d < 1 || e < 1) return ORC_ERR;
  const long BH = (long)B * H;
  int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
  for (long bh = 0; bh < BH; ++bh) {
    const double lam = lambda[bh % H];
    double* kv = (double*)malloc(sizeof(double) * d * e);
    double* R = (double*)malloc(sizeof(double) * d * e);
    if (!kv || !R) { failed = 1; free(kv); free(R); continue; }
    if (kv_in) memcpy(kv, kv_in + bh * d * e, sizeof(double) * d * e);
    else memset(kv, 0, sizeof(double) * d * e);
    for (long t = 0; t < N; ++t) {
      const float* kt = k + (bh * N + t) * d;
      const float* vt = v + (bh * N + t) * e;
      const float* dot = d_o + (bh * N + t) * e;
      double* dqt = dq + (bh * N + t) * d;
      for (int i = 0; i < d; ++i)
        for (int j = 0; j < e; ++j)
          kv[i * e + j] = lam * kv[i * e + j] + (double)kt[i] * (double)vt[j];
      for (int i = 0; i < d; ++i) {
        double acc = 0.0;
        for (int j = 0; j < e; ++j) acc += kv[i * e + j] * (double)dot[j];
        dqt[i] = acc;
      }
    }
    if (grad_kv_out) memcpy(R, grad_kv_out + bh * d * e, sizeof(double) * d * e);
    else memset(R, 0, sizeof(double) * d * e);
    for (long t = (long)N - 1; t >= 0; --t) {
      const float* qt = q + (bh * N + t) * d;
      const float* kt = k + (bh * N + t) * d;
      const float* vt = v + (bh * N + t) * e;
      const float* dot = d_o + (bh * N + t) * e;
      double* dkt = dk + (bh * N + t) * d;
      double* dvt = dv + (bh * N + t) * e;
      /* R_t = (decayed carry) + q_t do_t^T */
      for (int i = 0; i < d; ++i)
        for (int j = 0; j < e; ++j) R[i * e + j] += (double)qt[i] * (double)dot[j];
      for (int i = 0; i < d; ++i) {
        double acc = 0.0;
        for (int j = 0; j < e; ++j) acc += R[i * e + j] * (double)vt[j];
        dkt[i] = acc;
      }
      for (int j = 0; j < e; ++j) dvt[j] = 0.0;
      for (int i = 0; i < d; ++i)
        for (int j = 0; j < e; ++j) dvt[j] += R[i * e + j] * (double)kt[i];
      /* carry to token t-1 */
      for (int i = 0; i < d * e; ++i) R[i] *= lam;
    }
    if (grad_kv_in) memcpy(grad_kv_in + bh * d * e, R, sizeof(double) * d * e);
    free(kv);
    free(R);
  }
  return failed ? ORC_ERR : ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* Masked quadratic form, forward: O = (Q K^T (.) M) V, materialising A.       */
/* ------------------------------------------------------------------------- */
int orc_fwd_quad(const float* q, const float* k, const float* v, const double* lambda,
                 int B, int H, int N, int d, int e, double* o) {
  if (B < 0 || H < 0 || N < 0 || d < 1 || e < 1) return ORC_ERR;
  if ((double)N * (double)N > 2.0e8) return ORC_ERR; /* A is N x N doubles per thread */
  const long BH = (long)B * H;
  int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
  for (long bh = 0; bh < BH; ++bh) {
    const double lam = lambda[bh % H];
    double* A = (double*)malloc(sizeof(double) * (size_t)N * N);
    if (!A) { failed = 1; continue; }
    for (long t = 0; t < N; ++t)
      for (long s = 0; s < N; ++s) {
        double a = 0.0;
        if (t >= s) {
          for (int i = 0; i < d; ++i)
            a += (double)q[(bh * N + t) * d + i] * (double)k[(bh * N + s) * d + i];
          a *= mask_entry(lam, t - s);
        }
        A[t * N + s] = a;
      }
    for (long t = 0; t < N; ++t)
      for (int j = 0; j < e; ++j) {
        double acc = 0.0;
        for (long s = 0; s < N; ++s) acc += A[t * N + s] * (double)v[(bh * N + s) * e + j];
        o[(bh * N + t) * e + j] = acc;
      }
    free(A);
  }
  return failed ? ORC_ERR : ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* Masked quadratic form, backward (Algorithm 4 without the tiling):           */
/*   A = (Q K^T) (.) M,  dA = (dO V^T) (.) M,                                  */
/*   dQ = dA K,  dK = dA^T Q,  dV = A^T dO.                                    */
/* ------------------------------------------------------------------------- */
int orc_bwd_quad(const float* q, const float* k, const float* v, const float* d_o,
                 const double* lambda, int B, int H, int N, int d, int e,
                 double* dq, double* dk, double* dv) {
  if (B < 0 || H < 0 || N < 0 || d < 1 || e < 1) return ORC_ERR;
  if ((double)N * (double)N > 1.0e8) return ORC_ERR;
  const long BH = (long)B * H;
  int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
  for (long bh = 0; bh < BH; ++bh) {
    const double lam = lambda[bh % H];
    double* A = (double*)malloc(sizeof(double) * (size_t)N * N);
    double* dA = (double*)malloc(sizeof(double) * (size_t)N * N);
    if (!A || !dA) { failed = 1; free(A); free(dA); continue; }
    for (long t = 0; t < N; ++t)
      for (long s = 0; s < N; ++s) {
        double a = 0.0, da = 0.0;
        if (t >= s) {
          const double m = mask_entry(lam, t - s);
          for (int i = 0; i < d; ++i)
            a += (double)q[(bh * N + t) * d + i] * (double)k[(bh * N + s) * d + i];
          for (int j = 0; j < e; ++j)
            da += (double)d_o[(bh * N + t) * e + j] * (double)v[(bh * N + s) * e + j];
          a *= m;
          da *= m;
        }
        A[t * N + s] = a;
        dA[t * N + s] = da;
      }
    for (long t = 0; t < N; ++t)
      for (int i = 0; i < d; ++i) {
        double acc = 0.0;
        for (long s = 0; s < N; ++s) acc += dA[t * N + s] * (double)k[(bh * N + s) * d + i];
        dq[(bh * N + t) * d + i] = acc;
      }
    for (long s = 0; s < N; ++s)
      for (int i = 0; i < d; ++i) {
        double acc = 0.0;
        for (long t = 0; t < N; ++t) acc += dA[t * N + s] * (double)q[(bh * N + t) * d + i];
        dk[(bh * N + s) * d + i] = acc;
      }
    for (long s = 0; s < N; ++s)
      for (int j = 0; j < e; ++j) {
        double acc = 0.0;
        for (long t = 0; t < N; ++t) acc += A[t * N + s] * (double)d_o[(bh * N + t) * e + j];
        dv[(bh * N + s) * e + j] = acc;
      }
    free(A);
    free(dA);
  }
  return failed ? ORC_ERR : ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* Sampled rows of the masked quadratic form, for sizes where N x N is too     */
/* slow.  Row r is (bh[r], t[r]); kind selects the tensor:                     */
/*   0: o_t  = sum_{s<=t} M_ts (q_t.k_s) v_s          -> out[r, 0..e)          */
/*   1: dq_t = sum_{s<=t} M_ts (do_t.v_s) k_s         -> out[r, 0..d)          */
/*   2: dk_s = sum_{t>=s} M_ts (do_t.v_s) q_t         -> out[r, 0..d)          */
/*   3: dv_s = sum_{t>=s} M_ts (q_t.k_s) do_t         -> out[r, 0..e)          */
/* d_o may be NULL for kind 0.                                                 */
/* ------------------------------------------------------------------------- */
int orc_rows(int kind, const float* q, const float* k, const float* v, const float* d_o,
             const double* lambda, int B, int H, int N, int d, int e,
             int nrows, const int* bh_idx, const int* t_idx, double* out) {
  if (kind < 0 || kind > 3 || (kind != 0 && !d_o)) return ORC_ERR;
  const int w = (kind == 0 || kind == 3) ? e : d;
  for (int r = 0; r < nrows; ++r)
    if (bh_idx[r] < 0 || bh_idx[r] >= B * H || t_idx[r] < 0 || t_idx[r] >= N) return ORC_ERR;
#pragma omp parallel for schedule(dynamic, 1)
  for (int r = 0; r < nrows; ++r) {
    const long bh = bh_idx[r];
    const long x = t_idx[r];
    const double lam = lambda[bh % H];
    double* row = out + (size_t)r * w;
    for (int c = 0; c < w; ++c) row[c] = 0.0;
    if (kind == 0 || kind == 1) {
      const long t = x;
      for (long s = 0; s <= t; ++s) {
        const double m = mask_entry(lam, t - s);
        double dot = 0.0;
        if (kind == 0) {
          for (int i = 0; i < d; ++i)
            dot += (double)q[(bh * N + t) * d + i] * (double)k[(bh * N + s) * d + i];
          for (int j = 0; j < e; ++j) row[j] += m * dot * (double)v[(bh * N + s) * e + j];
        } else {
          for (int j = 0; j < e; ++j)
            dot += (double)d_o[(bh * N + t) * e + j] * (double)v[(bh * N + s) * e + j];
          for (int i = 0; i < d; ++i) row[i] += m * dot * (double)k[(bh * N + s) * d + i];
        }
      }
    } else {
      const long s = x;
      for (long t = s; t < N; ++t) {
        const double m = mask_entry(lam, t - s);
        double dot = 0.0;
        if (kind == 2) {
          for (int j = 0; j < e; ++j)
            dot += (double)d_o[(bh * N + t) * e + j] * (double)v[(bh * N + s) * e + j];
          for (int i = 0; i < d; ++i) row[i] += m * dot * (double)q[(bh * N + t) * d + i];
        } else {
          for (int i = 0; i < d; ++i)
            dot += (double)q[(bh * N + t) * d + i] * (double)k[(bh * N + s) * d + i];
          for (int j = 0; j < e; ++j) row[j] += m * dot * (double)d_o[(bh * N + t) * e + j];
        }
      }
    }
  }
  return ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* One recurrent decode step (one iteration of Algorithm 2), state in place.   */
/* q,k [B,H,d], v [B,H,e], kv [B,H,d,e] (fp64, updated), o [B,H,e].            */
/* ------------------------------------------------------------------------- */
int orc_decode_step(const float* q, const float* k, const float* v, const double* lambda,
                    double* kv, int B, int H, int d, int e, double* o) {
  if (B < 0 || H < 0 || d < 1 || e < 1) return ORC_ERR;
  const long BH = (long)B * H;
#pragma omp parallel for schedule(static)
  for (long bh = 0; bh < BH; ++bh) {
    const double lam = lambda[bh % H];
    double* S = kv + bh * d * e;
    for (int i = 0; i < d; ++i)
      for (int j = 0; j < e; ++j)
        S[i * e + j] = lam * S[i * e + j] + (double)k[bh * d + i] * (double)v[bh * e + j];
    for (int j = 0; j < e; ++j) o[bh * e + j] = 0.0;
    for (int i = 0; i < d; ++i)
      for (int j = 0; j < e; ++j) o[bh * e + j] += S[i * e + j] * (double)q[bh * d + i];
  }
  return ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* Prescaled recurrence (Algorithm 1), tokens numbered t = 1..n as printed:    */
/*   kv_t = kv_{t-1} + (k_t lambda^-t) v_t^T,   o_t = (q_t lambda^t) kv_t.     */
/* Equal to Algorithm 2 in exact arithmetic (Appendix C); in floating point    */
/* lambda^-t overflows and lambda^t underflows, which the tests demonstrate.   */
/* ------------------------------------------------------------------------- */
int orc_fwd_origin(const float* q, const float* k, const float* v, const double* lambda,
                   int B, int H, int N, int d, int e, double* o) {
  if (B < 0 || H < 0 || N < 0 || d < 1 || e < 1) return ORC_ERR;
  const long BH = (long)B * H;
  int failed = 0;
  for (long bh = 0; bh < BH; ++bh) {
    const double lam = lambda[bh % H];
    double* kv = (double*)calloc((size_t)d * e, sizeof(double));
    if (!kv) { failed = 1; continue; }
    for (long t = 1; t <= N; ++t) {
      const float* qt = q + (bh * N + (t - 1)) * d;
      const float* kt = k + (bh * N + (t - 1)) * d;
      const float* vt = v + (bh * N + (t - 1)) * e;
      double* ot = o + (bh * N + (t - 1)) * e;
      const double up = pow(lam, -(double)t);
      const double down = pow(lam, (double)t);
      for (int i = 0; i < d; ++i)
        for (int j = 0; j < e; ++j) kv[i * e + j] += ((double)kt[i] * up) * (double)vt[j];
      for (int j = 0; j < e; ++j) ot[j] = 0.0;
      for (int i = 0; i < d; ++i)
        for (int j = 0; j < e; ++j) ot[j] += ((double)qt[i] * down) * kv[i * e + j];
    }
    free(kv);
  }
  return failed ? ORC_ERR : ORC_OK;
}

/*
 * Eq. 3 with Eq. 8: y = SRMSNorm(o) (.) u per row of e values, SRMSNorm(x) = x / (||x||_2 / sqrt(e)).
 * o [rows, e] fp64 (the attention output), u [rows, e] (exact input values), y [rows, e] fp64,
 * rstd [rows] = sqrt(e) / ||o||_2 (0 for a zero row), or NULL.
 */
int orc_norm_gate_fwd(const double* o, const float* u, long rows, int e, double* y, double* rstd) {
  if (!o || !u || !y || rows < 0 || e < 1) return ORC_ERR;
#pragma omp parallel for schedule(static)
  for (long r = 0; r < rows; ++r) {
    const double* orow = o + r * e;
    double ss = 0.0;
    for (int j = 0; j < e; ++j) ss += orow[j] * orow[j];
    const double s = ss > 0.0 ? sqrt((double)e) / sqrt(ss) : 0.0;
    if (rstd) rstd[r] = s;
    for (int j = 0; j < e; ++j) y[r * e + j] = orow[j] * s * (double)u[r * e + j];
  }
  return ORC_OK;
}

/*
 * Gradients of L = <y, dy> with respect to o and u.  With n = o s, s = sqrt(e) / ||o||_2 and g = dy (.) u:
 *   du = dy (.) n,     do = s (g - n (n . g) / e)
 * (the second from d(o / ||o||) = (I - o o^T / ||o||^2) / ||o||; it is orthogonal to o because the norm
 * removes the scale of o).
 */
int orc_norm_gate_bwd(const double* o, const float* u, const float* dy, long rows, int e, double* d_o,
                      double* d_u) {
  if (!o || !u || !dy || !d_o || !d_u || rows < 0 || e < 1) return ORC_ERR;
#pragma omp parallel for schedule(static)
  for (long r = 0; r < rows; ++r) {
    const double* orow = o + r * e;
    double ss = 0.0;
    for (int j = 0; j < e; ++j) ss += orow[j] * orow[j];
    const double s = ss > 0.0 ? sqrt((double)e) / sqrt(ss) : 0.0;
    double ng = 0.0;
    for (int j = 0; j < e; ++j) ng += (orow[j] * s) * ((double)dy[r * e + j] * (double)u[r * e + j]);
    for (int j = 0; j < e; ++j) {
      const double n = orow[j] * s, g = (double)dy[r * e + j] * (double)u[r * e + j];
      d_u[r * e + j] = (double)dy[r * e + j] * n;
      d_o[r * e + j] = s * (g - n * ng / (double)e);
    }
  }
  return ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* LRPE-d (Eq. 1): decay and a learnable rotation of the relative position.    */
/*   a_ts = lambda^(t-s) sum_i q_t[i] k_s[i] cos(theta_i (t-s))   (s <= t)     */
/*   o_t  = sum_{s<=t} a_ts v_s                                                */
/* theta [H, d] fp64.  The N x N matrix is materialised as in orc_fwd_quad.    */
/* ------------------------------------------------------------------------- */
int orc_lrpe_fwd_quad(const float* q, const float* k, const float* v, const double* lambda,
                      const double* theta, int B, int H, int N, int d, int e, double* o) {
  if (B < 0 || H < 0 || N < 0 || d < 1 || e < 1) return ORC_ERR;
  if ((double)N * (double)N > 2.0e8) return ORC_ERR;
  const long BH = (long)B * H;
  int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
  for (long bh = 0; bh < BH; ++bh) {
    const double lam = lambda[bh % H];
    const double* th = theta + (size_t)(bh % H) * d;
    double* A = (double*)malloc(sizeof(double) * (size_t)N * N);
    if (!A) { failed = 1; continue; }
    for (long t = 0; t < N; ++t)
      for (long s = 0; s < N; ++s) {
        double a = 0.0;
        if (t >= s) {
          for (int i = 0; i < d; ++i)
            a += (double)q[(bh * N + t) * d + i] * (double)k[(bh * N + s) * d + i] * cos(th[i] * (double)(t - s));
          a *= mask_entry(lam, t - s);
        }
        A[t * N + s] = a;
      }
    for (long t = 0; t < N; ++t)
      for (int j = 0; j < e; ++j) {
        double acc = 0.0;
        for (long s = 0; s < N; ++s) acc += A[t * N + s] * (double)v[(bh * N + s) * e + j];
        o[(bh * N + t) * e + j] = acc;
      }
    free(A);
  }
  return failed ? ORC_ERR : ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* Gradients of L = <O, dO> for LRPE-d.  With dA_ts = lambda^(t-s) do_t.v_s:   */
/*   dq_t[i]   =  sum_{s<=t} dA_ts k_s[i] cos(theta_i (t-s))                   */
/*   dk_s[i]   =  sum_{t>=s} dA_ts q_t[i] cos(theta_i (t-s))                   */
/*   dv_s      =  sum_{t>=s} a_ts do_t                                         */
/*   dtheta_i  = -sum_{b} sum_{s<=t} dA_ts q_t[i] k_s[i] (t-s) sin(theta_i (t-s))   (theta is shared by the batch) */
/* dtheta [H, d].                                                              */
/* ------------------------------------------------------------------------- */
int orc_lrpe_bwd_quad(const float* q, const float* k, const float* v, const float* d_o,
                      const double* lambda, const double* theta, int B, int H, int N, int d, int e,
                      double* dq, double* dk, double* dv, double* dtheta) {
  if (B < 0 || H < 0 || N < 0 || d < 1 || e < 1) return ORC_ERR;
  if ((double)N * (double)N > 1.0e8) return ORC_ERR;
  const long BH = (long)B * H;
  int failed = 0;
  double* dth_part = (double*)calloc((size_t)(BH > 0 ? BH : 1) * d, sizeof(double)); /* one row per (b,h) */
  if (!dth_part) return ORC_ERR;
#pragma omp parallel for schedule(dynamic, 1)
  for (long bh = 0; bh < BH; ++bh) {
    const double lam = lambda[bh % H];
    const double* th = theta + (size_t)(bh % H) * d;
    double* A = (double*)malloc(sizeof(double) * (size_t)N * N);
    double* dA = (double*)malloc(sizeof(double) * (size_t)N * N);
    if (!A || !dA) { failed = 1; free(A); free(dA); continue; }
    for (long t = 0; t < N; ++t)
      for (long s = 0; s < N; ++s) {
        double a = 0.0, da = 0.0;
        if (t >= s) {
          const double m = mask_entry(lam, t - s);
          for (int i = 0; i < d; ++i)
            a += (double)q[(bh * N + t) * d + i] * (double)k[(bh * N + s) * d + i] * cos(th[i] * (double)(t - s));
          for (int j = 0; j < e; ++j)
            da += (double)d_o[(bh * N + t) * e + j] * (double)v[(bh * N + s) * e + j];
          a *= m;
          da *= m;
        }
        A[t * N + s] = a;
        dA[t * N + s] = da;
      }
    for (long t = 0; t < N; ++t)
      for (int i = 0; i < d; ++i) {
        double acc = 0.0;
        for (long s = 0; s <= t; ++s)
          acc += dA[t * N + s] * (double)k[(bh * N + s) * d + i] * cos(th[i] * (double)(t - s));
        dq[(bh * N + t) * d + i] = acc;
      }
    for (long s = 0; s < N; ++s)
      for (int i = 0; i < d; ++i) {
        double acc = 0.0;
        for (long t = s; t < N; ++t)
          acc += dA[t * N + s] * (double)q[(bh * N + t) * d + i] * cos(th[i] * (double)(t - s));
        dk[(bh * N + s) * d + i] = acc;
      }
    for (long s = 0; s < N; ++s)
      for (int j = 0; j < e; ++j) {
        double acc = 0.0;
        for (long t = 0; t < N; ++t) acc += A[t * N + s] * (double)d_o[(bh * N + t) * e + j];
        dv[(bh * N + s) * e + j] = acc;
      }
    for (int i = 0; i < d; ++i) {
      double acc = 0.0;
      for (long t = 0; t < N; ++t)
        for (long s = 0; s <= t; ++s)
          acc -= dA[t * N + s] * (double)q[(bh * N + t) * d + i] * (double)k[(bh * N + s) * d + i] *
                 (double)(t - s) * sin(th[i] * (double)(t - s));
      dth_part[bh * d + i] = acc;
    }
    free(A);
    free(dA);
  }
  for (long hi = 0; hi < (long)H * d; ++hi) dtheta[hi] = 0.0;
  for (long bh = 0; bh < BH; ++bh)
    for (int i = 0; i < d; ++i) dtheta[(bh % H) * d + i] += dth_part[bh * d + i];
  free(dth_part);
  return failed ? ORC_ERR : ORC_OK;
}
