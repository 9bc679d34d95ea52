/*
 * vla_oracle_bwd.h -- CPU oracle for the backward pass of the VLA forward scan.
 *
 * TEST INFRASTRUCTURE ONLY (see vla_oracle.h): hand-written reverse-mode differentiation, in
 * fp64, of the recurrence that vla_oracle_forward computes.  Pinned by central finite
 * differences of vla_oracle_forward; parity status in the header comment of vla_oracle_bwd.c.
 *
 * All pointers are HOST pointers owned by the caller; layouts as in vla_oracle.h.  Gradients
 * are fp64 with the shape of the quantity they belong to.
 */
#ifndef VLA_ORACLE_BWD_H
#define VLA_ORACLE_BWD_H

#include "vla_oracle.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Given dL/d(out) [B,H,T,d_v] and, optionally, dL/dS_T, dL/dA_T, dL/dz_T (NULL = zero), returns
 * dL/dq, dL/dk [B,H,T,d_k], dL/dv [B,H,T,d_v], dL/du (only when u is given; may be NULL) and,
 * when asked for (non-NULL), dL/dS0, dL/dA0, dL/dz0.  The forward is recomputed inside from
 * q, k, v, u, S0, A0, z0 exactly as vla_oracle_forward computes it.  In identity-map mode
 * z_T = z0, so dL/dz0 = dL/dz_T.  Returns 0, or -1 on an invalid argument.
 */
int vla_oracle_backward(const void* q, const void* k, const void* v, const void* u, int in_dtype,
                        double lambda, int B, int H, int T, int d_k, int d_v, const double* S0,
                        const double* A0, const double* z0, unsigned flags, double eps,
                        const double* d_out, const double* dS_T, const double* dA_T,
                        const double* dz_T, double* dq, double* dk, double* dv, double* du,
                        double* dS0, double* dA0, double* dz0, int n_threads,
                        const vla_oracle_refresh_t* refresh);

#ifdef __cplusplus
}
#endif
#endif
