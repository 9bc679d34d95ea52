/*
 * vla_oracle.h -- CPU oracle for the Variational Linear Attention forward scan.
 *
 * TEST INFRASTRUCTURE ONLY.  This is a plain, slow, fp64 restatement of the
 * paper's sequential forward pass (Algorithm 1 without the projections, its
 * periodic refresh optional; Eqs. "sm", "s-update", "output" of Section 3.3).
 * It shares no code with the CUDA library and the CUDA library never calls it.
 * Only the tests, the smoke check and the CPU-baseline leg of the benchmark
 * may load it.
 *
 * Parity status of each part is listed in the header comment of vla_oracle.c.
 *
 * All pointers are HOST pointers owned by the caller.  Tensors are contiguous,
 * row-major:
 *   q, k, u : [B, H, T, d_k]     v : [B, H, T, d_v]     (storage dtype in_dtype)
 *   S0, S_T : [B, H, d_v, d_k]   fp64, row = value index (S k_hat predicts v)
 *   A0, A_T : [B, H, d_k, d_k]   fp64
 *   z0, z_T : [B, H, d_k]        fp64, running sum of phi(k) (paper mode only)
 *   out     : [B, H, T, d_v]     fp64
 */
#ifndef VLA_ORACLE_H
#define VLA_ORACLE_H

#ifdef __cplusplus
extern "C" {
#endif

/* storage type of q, k, v, u; every value is widened exactly to fp64 */
enum { VLA_ORACLE_F32 = 0, VLA_ORACLE_BF16 = 1, VLA_ORACLE_F64 = 2 };

/* flags */
enum {
  /* Section 3.1 reading: k_hat = k/||k||, o_t = S_t q_t (no feature map, no
     normaliser).  Without it: Algorithm 1 (phi = ELU+1 on k and q, Eq. "output"). */
  VLA_ORACLE_IDENTITY_MAP = 1u << 0,
  /* Comparison mode, Section 2, Eq. "linear-attn": S_t = S_{t-1} + v_t phi(k_t)^T (additive write,
     no penalty matrix, no residual); readout as Eq. "output".  A is passed through untouched;
     u and the refresh are ignored. */
  VLA_ORACLE_LINEAR_ATTENTION = 1u << 1
};

/* Algorithm 1's periodic identity refresh: after the Sherman-Morrison step of the token whose
   1-based position in the whole sequence is a multiple of `period`, A += eta * I.  The paper
   uses period 20, eta 1e-3 (Section 5.3).  `step_offset` = tokens of the sequence processed
   before this call (for carried state).  NULL or period <= 0: no refresh. */
typedef struct {
  int period;
  double eta;
  long step_offset;
} vla_oracle_refresh_t;

/* Optional per-step dump of one unit (any pointer may be NULL). */
typedef struct {
  double* A;      /* [T, d_k, d_k]  A_t after the Sherman-Morrison step            */
  double* S;      /* [T, d_v, d_k]  S_t after the residual update                  */
  double* khat;   /* [T, d_k]                                                       */
  double* u;      /* [T, d_k]       the penalty direction actually used            */
  double* alpha;  /* [T, d_k]       unit write direction                           */
  double* e;      /* [T, d_v]       prediction residual                            */
  double* delta;  /* [T]                                                            */
  double* den;    /* [T]            readout denominator (1 in identity mode)       */
} vla_oracle_trace_t;

/*
 * Runs all B*H units.  u may be NULL (then u_t = k_hat_t, the special case of
 * Section 7.1).  S0/A0/z0 may be NULL (zero / I/lambda / zero).  S_T/A_T/z_T may
 * be NULL.  n_threads <= 1 runs serially; otherwise units are split in
 * contiguous blocks over that many pthreads (units are independent).
 * Returns 0, or -1 on an invalid argument.
 */
int vla_oracle_forward(const void* q, const void* k, const void* v, const void* u,
                       int in_dtype, double lambda,
                       int B, int H, int T, int d_k, int d_v,
                       const double* S0, const double* A0, const double* z0,
                       unsigned flags, double eps,
                       double* out, double* S_T, double* A_T, double* z_T,
                       int n_threads, const vla_oracle_refresh_t* refresh);

/* Same recurrence for ONE unit (B = H = 1) with a per-step trace. */
int vla_oracle_forward_trace(const void* q, const void* k, const void* v, const void* u,
                             int in_dtype, double lambda, int T, int d_k, int d_v,
                             const double* S0, const double* A0, const double* z0,
                             unsigned flags, double eps,
                             double* out, double* S_T, double* A_T, double* z_T,
                             const vla_oracle_trace_t* trace,
                             const vla_oracle_refresh_t* refresh);

#ifdef __cplusplus
}
#endif
#endif
