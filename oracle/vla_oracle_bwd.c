/*
 * vla_oracle_bwd.c -- CPU oracle for the BACKWARD pass of the Variational Linear Attention
 * forward scan (the gradients the paper's Corollary on gradient flow, Section 4, is about).
 *
 * TEST INFRASTRUCTURE ONLY.  Plain C, fp64, one token at a time.  The paper gives no
 * backward algorithm: this file is reverse-mode differentiation, written out by hand, of
 * exactly the forward recurrence that vla_oracle.c computes (Algorithm 1 without the
 * projections; Eqs. "sm", "s-update", "output"; the optional periodic refresh), in the same
 * notation.  It shares no code with the CUDA library.
 *
 * What pins it (tests/test_oracle_bwd_pins.py, independent of this file): central finite
 * differences of vla_oracle_forward for a random linear functional of (o, S_T, A_T, z_T), for
 * every input (q, k, v, u, S0, A0, z0), both feature-map modes, with and without an explicit u,
 * with the refresh; linearity in the incoming gradients; closed forms for one token; planted
 * mistakes in a copy of this file.  Parity of anything compared with it is otherwise unpinned by
 * the paper.
 *
 * Per token the forward computes (S, A, zk the incoming state):
 *   kf = phi(k) | k            nk = max(||kf||, eps)        k_hat = kf / nk
 *   u  = given | k_hat
 *   z  = A u                   delta = max(1 + u.z, eps)    A' = A - z z^T / delta  [+ eta I]
 *   a  = A' k_hat              na = max(||a||, eps)         alpha = a / na
 *   e  = v - S k_hat           S' = S + e alpha^T
 *   qf = phi(q) | q            zk' = zk + kf                den = max(zk'.qf, eps) | 1
 *   o  = S' qf / den
 * and the reverse sweep below undoes the state updates token by token (S = S' - e alpha^T,
 * A = A' [- eta I] + z z^T / delta) instead of storing every state.
 */
#include "vla_oracle_bwd.h"

#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double phi(double x) { return x > 0.0 ? x + 1.0 : exp(x); }
static double dphi(double x) { return x > 0.0 ? 1.0 : exp(x); }

static double load_elem(const void* base, size_t idx, int dtype) {
  if (dtype == VLA_ORACLE_F64) return ((const double*)base)[idx];
  if (dtype == VLA_ORACLE_F32) return (double)((const float*)base)[idx];
  {
    uint32_t bits = ((uint32_t)((const uint16_t*)base)[idx]) << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
  }
}

static double dot(const double* a, const double* b, int n) {
  double s = 0.0;
  for (int i = 0; i < n; ++i) s += a[i] * b[i];
  return s;
}

typedef struct {
  const void *q, *k, *v, *u;
  int dtype, T, dk, dv;
  unsigned flags;
  double lambda, eps;
  const double *S0, *A0, *z0;          /* this unit's blocks or NULL */
  const double *d_out, *dS_T, *dA_T, *dz_T;
  double *dq, *dk_, *dv_, *du, *dS0, *dA0, *dz0;
  size_t qk_off, v_off;                /* element offsets of this unit in q/k/u and v */
  const vla_oracle_refresh_t* rf;
} unit_job;

static void backward_unit(const unit_job* J) {
  const int T = J->T, dk = J->dk, dv = J->dv;
  const int identity = (J->flags & VLA_ORACLE_IDENTITY_MAP) != 0;
  const double eps = J->eps;
  const size_t nkk = (size_t)dk * dk, nvk = (size_t)dv * dk;
#define VEC(name, n) double* name = (double*)calloc((size_t)(n) * (size_t)T + 1, sizeof(double))
  VEC(kraw, dk); VEC(qraw, dk); VEC(kf, dk); VEC(khat, dk); VEC(uu, dk); VEC(z, dk);
  VEC(a, dk); VEC(alpha, dk); VEC(qf, dk); VEC(e, dv);
  VEC(nk, 1); VEC(delta, 1); VEC(dclamp, 1); VEC(na, 1); VEC(den, 1); VEC(denclamp, 1);
  VEC(refreshed, 1);
#undef VEC
  double* S = (double*)calloc(nvk, sizeof(double));
  double* A = (double*)calloc(nkk, sizeof(double));
  double* zk = (double*)calloc((size_t)dk, sizeof(double));
  if (J->S0) memcpy(S, J->S0, nvk * sizeof(double));
  if (J->A0) memcpy(A, J->A0, nkk * sizeof(double));
  else for (int i = 0; i < dk; ++i) A[(size_t)i * dk + i] = 1.0 / J->lambda;
  if (J->z0) memcpy(zk, J->z0, (size_t)dk * sizeof(double));

  /* ---------------- forward sweep, keeping the per-token vectors ---------------- */
  for (int t = 0; t < T; ++t) {
    const size_t rk = J->qk_off + (size_t)t * dk, rv = J->v_off + (size_t)t * dv;
    double *kr = kraw + (size_t)t * dk, *qr = qraw + (size_t)t * dk, *kft = kf + (size_t)t * dk;
    double *kh = khat + (size_t)t * dk, *ut = uu + (size_t)t * dk, *zt = z + (size_t)t * dk;
    double *at = a + (size_t)t * dk, *al = alpha + (size_t)t * dk, *qft = qf + (size_t)t * dk;
    double* et = e + (size_t)t * dv;
    for (int j = 0; j < dk; ++j) {
      kr[j] = load_elem(J->k, rk + j, J->dtype);
      qr[j] = load_elem(J->q, rk + j, J->dtype);
      kft[j] = identity ? kr[j] : phi(kr[j]);
      qft[j] = identity ? qr[j] : phi(qr[j]);
    }
    {
      double n = sqrt(dot(kft, kft, dk));
      nk[t] = n > eps ? n : eps;
      for (int j = 0; j < dk; ++j) kh[j] = kft[j] / nk[t];
    }
    for (int j = 0; j < dk; ++j) ut[j] = J->u ? load_elem(J->u, rk + j, J->dtype) : kh[j];
    for (int i = 0; i < dk; ++i) zt[i] = dot(A + (size_t)i * dk, ut, dk);
    {
      double d = 1.0 + dot(ut, zt, dk);
      dclamp[t] = d < eps ? 1.0 : 0.0;
      delta[t] = d < eps ? eps : d;
    }
    for (int i = 0; i < dk; ++i)
      for (int j = 0; j < dk; ++j) A[(size_t)i * dk + j] -= zt[i] * zt[j] / delta[t];
    if (J->rf && J->rf->period > 0 && (J->rf->step_offset + t + 1) % J->rf->period == 0) {
      refreshed[t] = 1.0;
      for (int i = 0; i < dk; ++i) A[(size_t)i * dk + i] += J->rf->eta;
    }
    for (int i = 0; i < dk; ++i) at[i] = dot(A + (size_t)i * dk, kh, dk);
    {
      double n = sqrt(dot(at, at, dk));
      na[t] = n > eps ? n : eps;
      for (int i = 0; i < dk; ++i) al[i] = at[i] / na[t];
    }
    for (int i = 0; i < dv; ++i)
      et[i] = load_elem(J->v, rv + i, J->dtype) - dot(S + (size_t)i * dk, kh, dk);
    for (int i = 0; i < dv; ++i)
      for (int j = 0; j < dk; ++j) S[(size_t)i * dk + j] += et[i] * al[j];
    den[t] = 1.0;
    if (!identity) {
      for (int j = 0; j < dk; ++j) zk[j] += kft[j];
      double d = dot(zk, qft, dk);
      denclamp[t] = d < eps ? 1.0 : 0.0;
      den[t] = d < eps ? eps : d;
    }
  }

  /* ---------------- reverse sweep ---------------- */
  double* GS = (double*)calloc(nvk, sizeof(double));   /* dL/dS' */
  double* GA = (double*)calloc(nkk, sizeof(double));   /* dL/dA' */
  double* gz = (double*)calloc((size_t)dk, sizeof(double));  /* dL/dzk' */
  if (J->dS_T) memcpy(GS, J->dS_T, nvk * sizeof(double));
  if (J->dA_T) memcpy(GA, J->dA_T, nkk * sizeof(double));
  if (J->dz_T) memcpy(gz, J->dz_T, (size_t)dk * sizeof(double));   /* identity mode: z_T = z0 */
  double* dy = (double*)malloc(sizeof(double) * (size_t)dv);
  double* de = (double*)malloc(sizeof(double) * (size_t)dv);
  double* dqf = (double*)malloc(sizeof(double) * (size_t)dk);
  double* dkf = (double*)malloc(sizeof(double) * (size_t)dk);
  double* dkh = (double*)malloc(sizeof(double) * (size_t)dk);
  double* dal = (double*)malloc(sizeof(double) * (size_t)dk);
  double* da = (double*)malloc(sizeof(double) * (size_t)dk);
  double* dz = (double*)malloc(sizeof(double) * (size_t)dk);
  double* duv = (double*)malloc(sizeof(double) * (size_t)dk);

  for (int t = T - 1; t >= 0; --t) {
    const size_t ok = (size_t)t * dk, ov = (size_t)t * dv;
    const double *kr = kraw + ok, *qr = qraw + ok, *kft = kf + ok, *kh = khat + ok, *ut = uu + ok;
    const double *zt = z + ok, *at = a + ok, *al = alpha + ok, *qft = qf + ok, *et = e + ov;
    const double* go = J->d_out + (J->v_off + ov);
    (void)at;

    /* o = S' qf / den */
    double odo = 0.0;   /* (S' qf) . do */
    for (int i = 0; i < dv; ++i) {
      dy[i] = go[i] / den[t];
      odo += dot(S + (size_t)i * dk, qft, dk) * go[i];
    }
    double dden = (identity || denclamp[t] != 0.0) ? 0.0 : -odo / (den[t] * den[t]);
    for (int j = 0; j < dk; ++j) {
      double s = 0.0;
      for (int i = 0; i < dv; ++i) s += S[(size_t)i * dk + j] * dy[i];
      dqf[j] = s + dden * zk[j];
      dkf[j] = 0.0;
      dkh[j] = 0.0;
    }
    for (int i = 0; i < dv; ++i)
      for (int j = 0; j < dk; ++j) GS[(size_t)i * dk + j] += dy[i] * qft[j];
    if (!identity) {
      /* den = zk'.qf ; zk' = zk + kf */
      for (int j = 0; j < dk; ++j) gz[j] += dden * qft[j];
      for (int j = 0; j < dk; ++j) dkf[j] += gz[j];
      for (int j = 0; j < dk; ++j) zk[j] -= kft[j];            /* back to zk */
    }
    /* S' = S + e alpha^T */
    for (int i = 0; i < dv; ++i) de[i] = dot(GS + (size_t)i * dk, al, dk);
    for (int j = 0; j < dk; ++j) {
      double s = 0.0;
      for (int i = 0; i < dv; ++i) s += GS[(size_t)i * dk + j] * et[i];
      dal[j] = s;
    }
    for (int i = 0; i < dv; ++i)
      for (int j = 0; j < dk; ++j) S[(size_t)i * dk + j] -= et[i] * al[j];   /* back to S */
    /* e = v - S k_hat */
    for (int i = 0; i < dv; ++i) J->dv_[J->v_off + ov + i] = de[i];
    for (int j = 0; j < dk; ++j) {
      double s = 0.0;
      for (int i = 0; i < dv; ++i) s += S[(size_t)i * dk + j] * de[i];
      dkh[j] -= s;
    }
    for (int i = 0; i < dv; ++i)
      for (int j = 0; j < dk; ++j) GS[(size_t)i * dk + j] -= de[i] * kh[j];
    /* alpha = a / na */
    {
      double n2 = sqrt(dot(at, at, dk));
      if (n2 > eps) {
        double ad = dot(al, dal, dk);
        for (int j = 0; j < dk; ++j) da[j] = (dal[j] - al[j] * ad) / na[t];
      } else {
        for (int j = 0; j < dk; ++j) da[j] = dal[j] / eps;
      }
    }
    /* a = A' k_hat  (A holds A' here) */
    for (int j = 0; j < dk; ++j) {
      double s = 0.0;
      for (int i = 0; i < dk; ++i) s += A[(size_t)i * dk + j] * da[i];
      dkh[j] += s;
    }
    for (int i = 0; i < dk; ++i)
      for (int j = 0; j < dk; ++j) GA[(size_t)i * dk + j] += da[i] * kh[j];
    /* refresh: A' = A'' + eta I passes the gradient through */
    if (refreshed[t] != 0.0)
      for (int i = 0; i < dk; ++i) A[(size_t)i * dk + i] -= J->rf->eta;
    /* A'' = A - z z^T / delta */
    double ddelta = 0.0;
    for (int i = 0; i < dk; ++i) {
      double s = 0.0;
      for (int j = 0; j < dk; ++j) {
        s += (GA[(size_t)i * dk + j] + GA[(size_t)j * dk + i]) * zt[j];
        ddelta += GA[(size_t)i * dk + j] * zt[i] * zt[j];
      }
      dz[i] = -s / delta[t];
    }
    ddelta /= delta[t] * delta[t];
    if (dclamp[t] != 0.0) ddelta = 0.0;
    for (int i = 0; i < dk; ++i)
      for (int j = 0; j < dk; ++j) A[(size_t)i * dk + j] += zt[i] * zt[j] / delta[t];   /* back to A */
    /* delta = 1 + u.z */
    for (int j = 0; j < dk; ++j) {
      duv[j] = ddelta * zt[j];
      dz[j] += ddelta * ut[j];
    }
    /* z = A u */
    for (int j = 0; j < dk; ++j) {
      double s = 0.0;
      for (int i = 0; i < dk; ++i) s += A[(size_t)i * dk + j] * dz[i];
      duv[j] += s;
    }
    for (int i = 0; i < dk; ++i)
      for (int j = 0; j < dk; ++j) GA[(size_t)i * dk + j] += dz[i] * ut[j];
    if (J->u) {
      if (J->du) for (int j = 0; j < dk; ++j) J->du[J->qk_off + ok + j] = duv[j];
    } else {
      for (int j = 0; j < dk; ++j) dkh[j] += duv[j];
    }
    /* k_hat = kf / nk */
    {
      double n = sqrt(dot(kft, kft, dk));
      if (n > eps) {
        double kd = dot(kh, dkh, dk);
        for (int j = 0; j < dk; ++j) dkf[j] += (dkh[j] - kh[j] * kd) / nk[t];
      } else {
        for (int j = 0; j < dk; ++j) dkf[j] += dkh[j] / eps;
      }
    }
    for (int j = 0; j < dk; ++j) {
      J->dk_[J->qk_off + ok + j] = identity ? dkf[j] : dkf[j] * dphi(kr[j]);
      J->dq[J->qk_off + ok + j] = identity ? dqf[j] : dqf[j] * dphi(qr[j]);
    }
  }
  if (J->dS0) memcpy(J->dS0, GS, nvk * sizeof(double));
  if (J->dA0) memcpy(J->dA0, GA, nkk * sizeof(double));
  if (J->dz0) memcpy(J->dz0, gz, (size_t)dk * sizeof(double));

  free(kraw); free(qraw); free(kf); free(khat); free(uu); free(z); free(a); free(alpha); free(qf);
  free(e); free(nk); free(delta); free(dclamp); free(na); free(den); free(denclamp); free(refreshed);
  free(S); free(A); free(zk); free(GS); free(GA); free(gz);
  free(dy); free(de); free(dqf); free(dkf); free(dkh); free(dal); free(da); free(dz); free(duv);
}

typedef struct {
  const unit_job* jobs;
  int lo, hi;
} thread_arg;

static void* run_units(void* arg) {
  const thread_arg* a = (const thread_arg*)arg;
  for (int n = a->lo; n < a->hi; ++n) backward_unit(&a->jobs[n]);
  return NULL;
}

int vla_oracle_backward(const void* q, const void* k, const void* v, const void* u, int in_dtype,
                        double lambda, int B, int H, int T, int d_k, int d_v, const double* S0,
                        const double* A0, const double* z0, unsigned flags, double eps,
                        const double* d_out, const double* dS_T, const double* dA_T,
                        const double* dz_T, double* dq, double* dk, double* dv, double* du,
                        double* dS0, double* dA0, double* dz0, int n_threads,
                        const vla_oracle_refresh_t* refresh) {
  if (B < 0 || H < 0 || T < 0 || d_k <= 0 || d_v <= 0) return -1;
  if (in_dtype != VLA_ORACLE_F32 && in_dtype != VLA_ORACLE_BF16 && in_dtype != VLA_ORACLE_F64) return -1;
  if (!A0 && !(lambda > 0.0)) return -1;
  if (!(eps > 0.0)) return -1;
  const int units = B * H;
  if (units == 0) return 0;
  if (T > 0 && (!q || !k || !v || !d_out || !dq || !dk || !dv)) return -1;
  unit_job* jobs = (unit_job*)calloc((size_t)units, sizeof(unit_job));
  const size_t nkk = (size_t)d_k * d_k, nvk = (size_t)d_v * d_k;
  for (int n = 0; n < units; ++n) {
    unit_job* J = &jobs[n];
    J->q = q; J->k = k; J->v = v; J->u = u;
    J->dtype = in_dtype; J->T = T; J->dk = d_k; J->dv = d_v;
    J->flags = flags; J->lambda = lambda; J->eps = eps;
    J->S0 = S0 ? S0 + (size_t)n * nvk : NULL;
    J->A0 = A0 ? A0 + (size_t)n * nkk : NULL;
    J->z0 = z0 ? z0 + (size_t)n * d_k : NULL;
    J->d_out = d_out;
    J->dS_T = dS_T ? dS_T + (size_t)n * nvk : NULL;
    J->dA_T = dA_T ? dA_T + (size_t)n * nkk : NULL;
    J->dz_T = dz_T ? dz_T + (size_t)n * d_k : NULL;
    J->dq = dq; J->dk_ = dk; J->dv_ = dv; J->du = du;
    J->dS0 = dS0 ? dS0 + (size_t)n * nvk : NULL;
    J->dA0 = dA0 ? dA0 + (size_t)n * nkk : NULL;
    J->dz0 = dz0 ? dz0 + (size_t)n * d_k : NULL;
    J->qk_off = (size_t)n * (size_t)T * d_k;
    J->v_off = (size_t)n * (size_t)T * d_v;
    J->rf = refresh;
  }
  if (n_threads < 1) n_threads = 1;
  if (n_threads > units) n_threads = units;
  if (n_threads == 1) {
    thread_arg a = {jobs, 0, units};
    run_units(&a);
  } else {
    pthread_t* th = (pthread_t*)malloc(sizeof(pthread_t) * (size_t)n_threads);
    thread_arg* args = (thread_arg*)malloc(sizeof(thread_arg) * (size_t)n_threads);
    for (int i = 0; i < n_threads; ++i) {
      args[i].jobs = jobs;
      args[i].lo = (int)((long)units * i / n_threads);
      args[i].hi = (int)((long)units * (i + 1) / n_threads);
      pthread_create(&th[i], NULL, run_units, &args[i]);
    }
    for (int i = 0; i < n_threads; ++i) pthread_join(th[i], NULL);
    free(th);
    free(args);
  }
  free(jobs);
  return 0;
}
