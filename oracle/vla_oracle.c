/*
 * vla_oracle.c -- CPU oracle for the Variational Linear Attention forward scan.
 *
 * TEST INFRASTRUCTURE ONLY (see vla_oracle.h).  Plain C, fp64, one token at a
 * time: the recurrence of Section 3.3 (Eqs. "sm", "s-update", "output") taken in the
 * order Algorithm 1 takes its steps, one helper per equation, with three stated
 * departures from Algorithm 1:
 *   - the projections W_k, W_q, W_v, W_u are not applied: q, k, v (and u when
 *     given) arrive already projected;
 *   - the periodic identity refresh (A += eta*I every 20 steps) is off unless the
 *     caller asks for it, because it contradicts A_t = M_t^{-1} (Section 1.2,
 *     Eq. "A-covariance"); when on it sits where Algorithm 1 puts it, between the
 *     Sherman-Morrison step and the write direction;
 *   - both norms are guarded as x / max(||x||, eps) (Section 5.3: "eps for
 *     all denominators").
 * No blocking, fusion or reordering: every matrix-vector product is a double
 * loop, every rank-1 update a double loop.
 *
 * What pins it (tests/test_oracle_*.py, all independent of this file):
 *   A-chain      brute-force inverse of M_t = lambda*I + sum u u^T; trace and
 *                eigenvalue invariants; delta in [1, 1 + 1/lambda].
 *   alpha_hat    unit norm; parallel to inv(M_t) k_hat (post-update A_t).
 *   S-chain      closed forms (first step, orthonormal keys, repeated key),
 *                the u = 0 reduction to the normalised delta rule written
 *                separately, the corrected associative (R, G) composition of
 *                Section 3.4, Proposition 1's norm identities.
 *   readout      S_t q_t from dumped states; denominator from a direct sum.
 *   state carry  split invariance; segments stitched through a transfer scan
 *                (S_end = S_start P + G) with A at the cuts from matrix inverses.
 *   refresh      u = 0 closed form, step-by-step brute force with matrix inverses,
 *                split invariance with the carried step offset.
 *   additive     (linear attention, Eq. "linear-attn") direct double sums over s <= t.
 * Absolute output values on random data are otherwise fixed by nothing the
 * paper prints ("parity unpinned" beyond the pins above): this file is the
 * definition the CUDA path is compared with.
 */
#include "vla_oracle.h"

#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* phi(x) = ELU(x) + 1  (Section 3.3, below Eq. "output") */
static double phi(double x) { return x > 0.0 ? x + 1.0 : exp(x); }

/* exact widening of one stored element */
static double load_elem(const void* base, size_t idx, int dtype) {
  if (dtype == VLA_ORACLE_F64) return ((const double*)base)[idx];
  if (dtype == VLA_ORACLE_F32) return (double)((const float*)base)[idx];
  /* bfloat16: the upper 16 bits of an IEEE binary32 */
  uint32_t bits = (uint32_t)((const uint16_t*)base)[idx] << 16;
  float f;
  memcpy(&f, &bits, sizeof f);
  return (double)f;
}

static double dot(const double* a, const double* b, int n) {
  double s = 0.0;
  for (int i = 0; i < n; ++i) s += a[i] * b[i];
  return s;
}

/* ---- the steps of one token, one helper per equation of Section 3.3 ---- */

/* Feature map and unit key: key_map = phi(k_t) (Algorithm 1) or k_t itself (Section 3.1),
   key_unit = key_map / max(||key_map||, eps). */
static void make_unit_key(const void* k, size_t row, int dtype, int identity, double eps, int dk,
                          double* key_map, double* key_unit) {
  for (int j = 0; j < dk; ++j) {
    double raw = load_elem(k, row + j, dtype);
    key_map[j] = identity ? raw : phi(raw);
  }
  double len = sqrt(dot(key_map, key_map, dk));
  double guard = len > eps ? len : eps;
  for (int j = 0; j < dk; ++j) key_unit[j] = key_map[j] / guard;
}

/* Eq. "sm": rank-1 downdate of the inverse penalty by the direction pen.  gain receives
   A_{t-1} pen; returns delta (clamped at eps as Algorithm 1 does; it is >= 1 for A > 0). */
static double inverse_penalty_step(double* A, const double* pen, double* gain, int dk, double eps) {
  for (int i = 0; i < dk; ++i) gain[i] = dot(A + (size_t)i * dk, pen, dk);
  double delta = 1.0 + dot(pen, gain, dk);
  if (delta < eps) delta = eps;
  for (int i = 0; i < dk; ++i)
    for (int j = 0; j < dk; ++j) A[(size_t)i * dk + j] -= gain[i] * gain[j] / delta;
  return delta;
}

/* Eq. "s-update", first half: unit write direction from the POST-update A_t. */
static void unit_write_direction(const double* A, const double* key_unit, double* write_dir, int dk,
                                 double eps) {
  for (int i = 0; i < dk; ++i) write_dir[i] = dot(A + (size_t)i * dk, key_unit, dk);
  double len = sqrt(dot(write_dir, write_dir, dk));
  double guard = len > eps ? len : eps;
  for (int i = 0; i < dk; ++i) write_dir[i] /= guard;
}

/* Eq. "s-update", second half: resid = v_t - S_{t-1} key_unit, then S += resid write_dir^T. */
static void residual_write(double* S, const void* v, size_t row_v, int dtype, const double* key_unit,
                           const double* write_dir, double* resid, int dk, int dv) {
  for (int i = 0; i < dv; ++i)
    resid[i] = load_elem(v, row_v + i, dtype) - dot(S + (size_t)i * dk, key_unit, dk);
  for (int i = 0; i < dv; ++i)
    for (int j = 0; j < dk; ++j) S[(size_t)i * dk + j] += resid[i] * write_dir[j];
}

/* Eq. "linear-attn" (Section 2): the additive write S += v_t phi(k_t)^T of linear attention, the
   comparison mode (no penalty, no residual; the state stores value (x) key, as S does here). */
static void additive_write(double* S, const void* v, size_t row_v, int dtype, const double* key_map,
                           double* resid, int dk, int dv) {
  for (int i = 0; i < dv; ++i) {
    resid[i] = load_elem(v, row_v + i, dtype);
    for (int j = 0; j < dk; ++j) S[(size_t)i * dk + j] += resid[i] * key_map[j];
  }
}

/* Eq. "output": o_t = S_t phi(q_t) / max(phi(q_t) . z_t, eps) with z_t the key sum INCLUDING token
   t; with the identity map o_t = S_t q_t.  Returns the denominator used. */
static double read_out(const double* S, const void* q, size_t row_q, int dtype, int identity, double eps,
                       const double* key_map, double* key_sum, double* qry_map, double* o, int dk, int dv) {
  double den = 1.0;
  for (int j = 0; j < dk; ++j) {
    double raw = load_elem(q, row_q + j, dtype);
    qry_map[j] = identity ? raw : phi(raw);
  }
  if (!identity) {
    for (int j = 0; j < dk; ++j) key_sum[j] += key_map[j];
    den = dot(key_sum, qry_map, dk);
    if (den < eps) den = eps;
  }
  for (int i = 0; i < dv; ++i) o[i] = dot(S + (size_t)i * dk, qry_map, dk) / den;
  return den;
}

/*
 * One (b, h) unit.  q,k,u point at this unit's [T, d_k] block, v at [T, d_v].
 * S [d_v*d_k], A [d_k*d_k], key_sum [d_k] hold the incoming state and are updated
 * in place; out is [T, d_v].
 */
static void scan_unit(const void* q, const void* k, const void* v, const void* u_in,
                      size_t qk_off, size_t v_off, int dtype, int T, int dk, int dv,
                      unsigned flags, double eps, double* S, double* A, double* key_sum,
                      double* out, const vla_oracle_trace_t* tr,
                      const vla_oracle_refresh_t* rf) {
  const int identity = (flags & VLA_ORACLE_IDENTITY_MAP) != 0;
  const int additive = (flags & VLA_ORACLE_LINEAR_ATTENTION) != 0;
  double* key_map = (double*)malloc(sizeof(double) * (size_t)dk);
  double* key_unit = (double*)malloc(sizeof(double) * (size_t)dk);
  double* pen = (double*)malloc(sizeof(double) * (size_t)dk);
  double* gain = (double*)malloc(sizeof(double) * (size_t)dk);
  double* write_dir = (double*)malloc(sizeof(double) * (size_t)dk);
  double* qry_map = (double*)malloc(sizeof(double) * (size_t)dk);
  double* resid = (double*)malloc(sizeof(double) * (size_t)dv);

  for (int t = 0; t < T; ++t) {
    const size_t row_k = qk_off + (size_t)t * (size_t)dk;
    const size_t row_v = v_off + (size_t)t * (size_t)dv;
    double delta = 1.0;

    make_unit_key(k, row_k, dtype, identity, eps, dk, key_map, key_unit);
    if (additive) {
      /* comparison mode: A is not touched, nothing is normalised */
      for (int j = 0; j < dk; ++j) { pen[j] = 0.0; write_dir[j] = key_map[j]; }
      additive_write(S, v, row_v, dtype, key_map, resid, dk, dv);
    } else {
      /* penalty direction: supplied verbatim, else the unit key (Section 7.1) */
      for (int j = 0; j < dk; ++j)
        pen[j] = u_in ? load_elem(u_in, row_k + j, dtype) : key_unit[j];
      delta = inverse_penalty_step(A, pen, gain, dk, eps);
      /* periodic refresh of Section 5.3, placed as Algorithm 1 places it: after the downdate of
         every period-th token of the whole sequence, before the write direction */
      if (rf && rf->period > 0 && (rf->step_offset + t + 1) % rf->period == 0)
        for (int i = 0; i < dk; ++i) A[(size_t)i * dk + i] += rf->eta;
      unit_write_direction(A, key_unit, write_dir, dk, eps);
      residual_write(S, v, row_v, dtype, key_unit, write_dir, resid, dk, dv);
    }
    double den = read_out(S, q, row_k, dtype, identity, eps, key_map, key_sum, qry_map,
                          out + (size_t)t * dv, dk, dv);

    if (tr) {
      if (tr->A) memcpy(tr->A + (size_t)t * dk * dk, A, sizeof(double) * (size_t)dk * dk);
      if (tr->S) memcpy(tr->S + (size_t)t * dv * dk, S, sizeof(double) * (size_t)dv * dk);
      if (tr->khat) memcpy(tr->khat + (size_t)t * dk, key_unit, sizeof(double) * (size_t)dk);
      if (tr->u) memcpy(tr->u + (size_t)t * dk, pen, sizeof(double) * (size_t)dk);
      if (tr->alpha) memcpy(tr->alpha + (size_t)t * dk, write_dir, sizeof(double) * (size_t)dk);
      if (tr->e) memcpy(tr->e + (size_t)t * dv, resid, sizeof(double) * (size_t)dv);
      if (tr->delta) tr->delta[t] = delta;
      if (tr->den) tr->den[t] = den;
    }
  }
  free(key_map); free(key_unit); free(pen); free(gain); free(write_dir); free(qry_map); free(resid);
}

typedef struct {
  const void *q, *k, *v, *u;
  int dtype, T, dk, dv;
  double lambda, eps;
  unsigned flags;
  const double *S0, *A0, *z0;
  double *out, *S_T, *A_T, *z_T;
  const vla_oracle_trace_t* tr;
  const vla_oracle_refresh_t* rf;
  long unit_begin, unit_end;
} job_t;

static void* run_units(void* arg) {
  const job_t* jb = (const job_t*)arg;
  const size_t dk = (size_t)jb->dk, dv = (size_t)jb->dv, T = (size_t)jb->T;
  double* S = (double*)malloc(sizeof(double) * dv * dk);
  double* A = (double*)malloc(sizeof(double) * dk * dk);
  double* zk = (double*)malloc(sizeof(double) * dk);
  for (long n = jb->unit_begin; n < jb->unit_end; ++n) {
    /* initial state: S_0 = 0, A_0 = I/lambda_0, z = 0 unless carried in */
    if (jb->S0) memcpy(S, jb->S0 + (size_t)n * dv * dk, sizeof(double) * dv * dk);
    else memset(S, 0, sizeof(double) * dv * dk);
    if (jb->A0) memcpy(A, jb->A0 + (size_t)n * dk * dk, sizeof(double) * dk * dk);
    else {
      memset(A, 0, sizeof(double) * dk * dk);
      for (size_t i = 0; i < dk; ++i) A[i * dk + i] = 1.0 / jb->lambda;
    }
    if (jb->z0) memcpy(zk, jb->z0 + (size_t)n * dk, sizeof(double) * dk);
    else memset(zk, 0, sizeof(double) * dk);

    scan_unit(jb->q, jb->k, jb->v, jb->u, (size_t)n * T * dk, (size_t)n * T * dv, jb->dtype,
              jb->T, jb->dk, jb->dv, jb->flags, jb->eps, S, A, zk,
              jb->out + (size_t)n * T * dv, jb->tr, jb->rf);

    if (jb->S_T) memcpy(jb->S_T + (size_t)n * dv * dk, S, sizeof(double) * dv * dk);
    if (jb->A_T) memcpy(jb->A_T + (size_t)n * dk * dk, A, sizeof(double) * dk * dk);
    if (jb->z_T) memcpy(jb->z_T + (size_t)n * dk, zk, sizeof(double) * dk);
  }
  free(S); free(A); free(zk);
  return NULL;
}

static int check_args(const void* q, const void* k, const void* v, int in_dtype, double lambda,
                      long units, int T, int dk, int dv, const double* A0, double eps,
                      const double* out) {
  if (units < 0 || T < 0 || dk <= 0 || dv <= 0) return -1;
  if (in_dtype != VLA_ORACLE_F32 && in_dtype != VLA_ORACLE_BF16 && in_dtype != VLA_ORACLE_F64)
    return -1;
  if (!A0 && !(lambda > 0.0)) return -1;
  if (!(eps > 0.0)) return -1;
  if (units > 0 && T > 0 && (!q || !k || !v || !out)) return -1;
  return 0;
}

int vla_oracle_forward(const void* q, const void* k, const void* v, const void* u,
                       int in_dtype, double lambda, int B, int H, int T, int d_k, int d_v,
                       const double* S0, const double* A0, const double* z0, unsigned flags,
                       double eps, double* out, double* S_T, double* A_T, double* z_T,
                       int n_threads, const vla_oracle_refresh_t* refresh) {
  if (B < 0 || H < 0) return -1;
  const long units = (long)B * (long)H;
  if (check_args(q, k, v, in_dtype, lambda, units, T, d_k, d_v, A0, eps, out)) return -1;
  if (units == 0) return 0;
  if (n_threads < 1) n_threads = 1;
  if (n_threads > units) n_threads = (int)units;

  job_t base = {q, k, v, u, in_dtype, T, d_k, d_v, lambda, eps, flags,
                S0, A0, z0, out, S_T, A_T, z_T, NULL, refresh, 0, 0};
  if (n_threads == 1) {
    base.unit_begin = 0;
    base.unit_end = units;
    run_units(&base);
    return 0;
  }
  pthread_t* th = (pthread_t*)malloc(sizeof(pthread_t) * (size_t)n_threads);
  job_t* jobs = (job_t*)malloc(sizeof(job_t) * (size_t)n_threads);
  for (int i = 0; i < n_threads; ++i) {
    jobs[i] = base;
    jobs[i].unit_begin = units * i / n_threads;
    jobs[i].unit_end = units * (i + 1) / n_threads;
    pthread_create(&th[i], NULL, run_units, &jobs[i]);
  }
  for (int i = 0; i < n_threads; ++i) pthread_join(th[i], NULL);
  free(th); free(jobs);
  return 0;
}

int vla_oracle_forward_trace(const void* q, const void* k, const void* v, const void* u,
                             int in_dtype, double lambda, int T, int d_k, int d_v,
                             const double* S0, const double* A0, const double* z0,
                             unsigned flags, double eps, double* out, double* S_T,
                             double* A_T, double* z_T, const vla_oracle_trace_t* trace,
                             const vla_oracle_refresh_t* refresh) {
  if (check_args(q, k, v, in_dtype, lambda, 1, T, d_k, d_v, A0, eps, out)) return -1;
  job_t jb = {q, k, v, u, in_dtype, T, d_k, d_v, lambda, eps, flags,
              S0, A0, z0, out, S_T, A_T, z_T, trace, refresh, 0, 1};
  run_units(&jb);
  return 0;
}
