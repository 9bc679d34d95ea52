/*
 * vla.h -- C ABI of the B200 (sm_100a) Variational Linear Attention forward scan.
 *
 * One call runs, for every (batch, head) unit independently, the causal scan of
 * the paper's Section 3.3 (Eqs. "sm", "s-update", "output"; Algorithm 1 without
 * the projections; its periodic refresh is an option, see vla_opts_t).  Per token t:
 *
 *     k_hat = kf / max(||kf||, eps)        kf = phi(k_t)  (phi = ELU+1, Algorithm 1)
 *                                          kf = k_t       (VLA_FLAG_IDENTITY_MAP, Section 3.1)
 *     u     = u_t as given, or k_hat when no u is supplied          (Eq. "penalty")
 *     z     = A_{t-1} u ;  delta = max(1 + u.z, eps) ;  A_t = A_{t-1} - z z^T / delta   (Eq. "sm")
 *     alpha = A_t k_hat / max(||A_t k_hat||, eps)                   (Eq. "s-update", post-update A_t)
 *     e     = v_t - S_{t-1} k_hat ;  S_t = S_{t-1} + e alpha^T      (Eq. "s-update")
 *     o_t   = S_t phi(q_t) / max(phi(q_t).zkey_t, eps),  zkey_t = zkey_{t-1} + phi(k_t)   (Eq. "output")
 *     o_t   = S_t q_t                                               (VLA_FLAG_IDENTITY_MAP)
 *
 * All state arithmetic is fp32 on the GPU.  There is no CPU fallback: a shape
 * the kernels do not cover returns VLA_ERR_UNSUPPORTED.
 *
 * Memory: unless a function says otherwise every pointer is a DEVICE pointer owned by
 * the caller, tensors are contiguous and row-major, and base pointers are 16-byte
 * aligned (else VLA_ERR_ALIGNMENT).  The device-pointer calls allocate no memory and never
 * synchronise the device; work is enqueued on `stream`.
 *
 * State the library keeps for the life of the process (none of it carries results from one
 * call to the next):
 *   - a launch counter and, per device, 16 slots of hand-over flags (device memory inside the
 *     library, about 256 KB per kernel variant) for launches that cut units across CTAs; a
 *     slot is reused only once the launch that held it last has finished (one CUDA event per
 *     slot, created on first use), otherwise the launch runs one CTA per unit;
 *   - VLA_STATIC_SCRATCH_BYTES of device memory per GPU for vla_forward_host_static, and its
 *     device address once looked up;
 *   - per host thread, a note of the last kernel launched (vla_last_launch).
 * vla_forward_host creates and destroys its short-lived streams and events per call.
 */
#ifndef VLA_H
#define VLA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  VLA_OK = 0,
  VLA_ERR_INVALID_ARG = -1,    /* null/negative/ill-formed argument (host-side check)        */
  VLA_ERR_UNSUPPORTED = -2,    /* shape/dtype/flag combination without a kernel              */
  VLA_ERR_ALIGNMENT = -3,      /* a base pointer is not 16-byte aligned                      */
  VLA_ERR_CUDA = -4,           /* a CUDA runtime call or the launch failed                   */
  VLA_ERR_DEVICE_TIMEOUT = -5, /* written to opts->status: a bounded device-side wait ran out */
  VLA_ERR_NONFINITE = -6,      /* written to opts->status: non-finite delta / norm seen       */
  VLA_ERR_TOO_LARGE = -7       /* vla_forward_host_static: the built-in buffer is too small   */
} vla_status_t;

typedef enum { VLA_F32 = 0, VLA_BF16 = 1 } vla_dtype_t;

enum {
  VLA_FLAG_IDENTITY_MAP = 1u << 0, /* Section 3.1: k_hat = k/||k||, o_t = S_t q_t              */
  VLA_FLAG_CHECK_FINITE = 1u << 1, /* report non-finite delta or ||A_t k_hat|| in opts->status */
  VLA_FLAG_TOKEN_MAJOR = 1u << 2,  /* q, k, v, u and out are [B,T,H,d] (the layout projections write)
                                      instead of [B,H,T,d] (in vla_backward also d_out and the
                                      gradients of q, k, v, u); the states stay [B,H,d,d].
                                      vla_forward, the host-buffer calls (which then cut large
                                      batches by batch index), vla_backward (d >= 32);
                                      VLA_ERR_UNSUPPORTED elsewhere */
  VLA_FLAG_LINEAR_ATTENTION = 1u << 3 /* comparison mode, Section 2, Eq. "linear-attn": the additive
                                      write S_t = S_{t-1} + v_t phi(k_t)^T of linear attention (no
                                      penalty matrix, no residual), readout as Eq. "output"; with
                                      VLA_FLAG_IDENTITY_MAP phi is the identity and o_t = S_t q_t.
                                      A0 is passed through to A_T.  vla_forward and the host-buffer
                                      calls, every d, on the token kernel; not with opts->u, the
                                      refresh, or a forced chunk / decode kernel
                                      (VLA_ERR_UNSUPPORTED) */
};

/* Which scan kernel runs.  AUTO picks by shape; the others force one (tests, benchmarks). */
typedef enum {
  VLA_KERNEL_AUTO = 0,
  VLA_KERNEL_TOKEN = 1, /* one CTA per unit, one state pass per token; every shape, explicit u */
  VLA_KERNEL_CHUNK = 2, /* 16 tokens per state pass (exact Woodbury form) on the fp32 FMA pipe; d >= 32,
                           every option; VLA_ERR_UNSUPPORTED for d = 16 */
  VLA_KERNEL_DECODE = 3, /* one step (T = 1) with S0, A0, S_T, A_T all given, u = k_hat, no refresh,
                           d >= 32: the states stream through shared memory once (HBM-bound);
                           VLA_ERR_UNSUPPORTED otherwise.  AUTO picks it when it applies */
  VLA_KERNEL_CHUNK_TC = 4 /* the chunk algebra on the tensor cores (Section 3.4: the chunked recurrence
                           is a chain of dense products): states in tensor memory, TF32 products in
                           hi/lo pairs with fp32 accumulation.  d = 128, u = k_hat, no refresh,
                           [B,H,T,d] or [B,T,H,d] tensors, T >= 1; VLA_ERR_UNSUPPORTED otherwise.  AUTO picks it
                           where it applies (and VLA_KERNEL_CHUNK then forces the fp32-FMA form) */
} vla_kernel_t;

typedef struct {
  uint32_t struct_size;  /* = sizeof(vla_opts_t); lets the struct grow without breaking callers */
  int32_t qkv_dtype;     /* vla_dtype_t of q, k, v, u.  Default VLA_F32                          */
  const void* u;         /* [B,H,T,d_k] penalty directions, used verbatim (the caller applies
                            f_theta, the L2 norm and any 1/sqrt(d_h)); NULL => u_t = k_hat_t    */
  uint32_t flags;        /* VLA_FLAG_*; 0 = Algorithm 1                                         */
  float eps;             /* stability floor of every denominator; <= 0 => 1e-4 (Section 5.3)    */
  const float* z0;       /* [B,H,d_k] running sum of phi(k) carried in;  NULL => 0              */
  float* zT;             /* [B,H,d_k] the same after T tokens;           NULL => not written    */
  int32_t* status;       /* device int32, 0 on entry; set to a negative vla_status_t on a
                            device-side problem.  Read it after synchronising.  NULL allowed    */
  int32_t kernel;        /* vla_kernel_t                                                        */
  /* Algorithm 1's periodic identity refresh (Section 5.3: every 20 steps, + 1e-3 I): after
     the Sherman-Morrison step of each token whose 1-based position in the whole sequence
     (step_offset + t + 1) is a multiple of refresh_period, A += refresh_eta * I.  Off when
     refresh_period <= 0 (the default: it breaks A_t = M_t^-1).  Both kernels implement it.   */
  int32_t refresh_period;
  float refresh_eta;
  int64_t step_offset;   /* tokens of this sequence processed by earlier calls (state carry)     */
  float* du;             /* vla_backward with explicit u: [B,H,T,d_k] fp32 gradient of u (required
                            when u is given there; ignored by the forward calls)                 */
  void* workspace;       /* vla_forward (not the host-buffer calls), kernel AUTO: optional DEVICE scratch.  When the problem has
                            too few units to fill the device and the library would cut its sequences
                            (vla_seqpar_segments(...) > 1) and this holds at least
                            vla_seqpar_workspace_bytes(B, H, T, d_k, that many) bytes, the call runs as
                            vla_forward_seqpar; otherwise it is not touched.  NULL: never            */
  size_t workspace_bytes;
  uint32_t wait_probe_limit; /* a device-side wait (on a copy, on another warp group, on the CTA that
                            hands a unit over) gives up after this many failed probes and sets
                            VLA_ERR_DEVICE_TIMEOUT in *status; 0 = the default (about a second) */
} vla_opts_t;

/*
 * vla_forward -- Section 3.3 / Algorithm 1, all B*H units, T tokens each.
 *   q, k : [B,H,T,d_k]   v : [B,H,T,d_v]   in opts->qkv_dtype (fp32 default, bf16 widened in-kernel)
 *          (with VLA_FLAG_TOKEN_MAJOR: q, k, opts->u [B,T,H,d_k], v and out [B,T,H,d_v])
 *   lambda_ : lambda_0 of Eq. "penalty"; A_0 = I/lambda_ when A0 == NULL (must then be > 0)
 *   S0 : [B,H,d_v,d_k] fp32, row = value index (S k_hat predicts v); NULL => 0
 *   A0 : [B,H,d_k,d_k] fp32, symmetric positive definite;           NULL => I/lambda_
 *   out: [B,H,T,d_v] fp32
 *   S_T, A_T: final states, fp32, same layouts; NULL => not written.  They may alias S0/A0.
 *   out must not overlap any input.  T == 0 is legal and copies the state through.
 *   Supported: d_k == d_v in {16, 32, 64, 128}.
 * Returns VLA_OK once the work is enqueued on `stream` (a cudaStream_t; NULL = default
 * stream), or a negative vla_status_t from host-side validation / launch.  Device-side
 * problems are reported through opts->status.
 */
int vla_forward(const void* q, const void* k, const void* v, float lambda_,
                int B, int H, int T, int d_k, int d_v,
                const float* S0, const float* A0,
                float* out, float* S_T, float* A_T,
                const vla_opts_t* opts, void* stream);

/*
 * vla_forward_host -- the same computation for callers whose tensors live in HOST memory.
 * q, k, v, opts->u, S0, A0, opts->z0, out, S_T, A_T, opts->zT are HOST pointers (pinned
 * memory makes the copies asynchronous); `workspace` is a DEVICE buffer of at least
 * vla_host_workspace_bytes(...) bytes, 256-byte aligned, owned by the caller.  The call
 * enqueues host->device copies, the scan and device->host copies and returns without
 * synchronising; everything is ordered after the work already in `stream`, and `stream`
 * completes only after all of it, so outputs are valid once `stream` has been synchronised.
 * Batches that move at least 64 MB are pipelined in up to 32 slices of whole units over
 * short-lived internal streams (one for every copy-in, one for every copy-out, four for the
 * scans), so that what stays exposed is the first copy-in and the last scan and copy-out.
 * opts->status, when given, stays a DEVICE pointer.
 */
int vla_forward_host(const void* q, const void* k, const void* v, float lambda_,
                     int B, int H, int T, int d_k, int d_v,
                     const float* S0, const float* A0,
                     float* out, float* S_T, float* A_T,
                     const vla_opts_t* opts, void* workspace, size_t workspace_bytes,
                     void* stream);

/*
 * vla_forward_host_static -- vla_forward_host for callers that cannot hand over a device
 * workspace.  (The paper has no counterpart; this is a convenience of the library.)
 *
 * Who needs it: code that has host buffers and a stream but no way to obtain device
 * memory at the point of the call -- a plug-in inside a host application that gave the
 * whole device to another memory pool, a process running against a hard device-memory
 * cap that is already committed, or a latency-critical loop that must not pay
 * cudaMalloc's cost and implicit synchronisation.  For them the staging memory that
 * vla_forward_host takes as `workspace` is built into the library instead: a fixed array
 * of VLA_STATIC_SCRATCH_BYTES in device memory, present on every GPU that loads the
 * library until the process exits.  The call allocates and frees nothing.
 *
 * Arguments and results are exactly those of vla_forward_host without `workspace`.
 * Limits and rules:
 *   - vla_host_workspace_bytes(...) for the problem must not exceed
 *     VLA_STATIC_SCRATCH_BYTES, else VLA_ERR_TOO_LARGE is returned and nothing is enqueued.
 *   - The first call on each device looks up the array's device address (a one-time
 *     set-up for that device); make that first call before starting any stream capture
 *     (a first call on a capturing stream returns VLA_ERR_INVALID_ARG and enqueues nothing).
 *   - All calls on a device share the one array, and it keeps whatever the last call left
 *     in it.  Two calls whose work can overlap on the GPU (different streams without an
 *     ordering between them) race on it: order them, or use vla_forward_host with
 *     separate workspaces.
 */
#define VLA_STATIC_SCRATCH_BYTES (32u << 20)
int vla_forward_host_static(const void* q, const void* k, const void* v, float lambda_,
                            int B, int H, int T, int d_k, int d_v,
                            const float* S0, const float* A0,
                            float* out, float* S_T, float* A_T,
                            const vla_opts_t* opts, void* stream);

/*
 * vla_forward_seqpar -- the same forward scan with each unit's sequence cut into `segments`
 * equal pieces that are scanned at the same time (for long sequences with few (batch, head)
 * units, where one CTA per unit leaves most of the GPU idle).  It follows the parallel form
 * of Section 3.4 with the composition written as the recurrence needs it: the memory map
 * acts on the right, S_t = S_{t-1} (I - k_hat_t alpha_t^T) + v_t alpha_t^T, so a segment
 * composes to S_end = S_start P + G; and A at a segment start is the inverse of
 * lambda I + sum of u u^T over the earlier tokens (Eq. "penalty"), formed in fp64.  Results
 * equal vla_forward's up to rounding.
 *
 * Arguments as vla_forward, with these differences: a carried-in A0 must be symmetric positive
 * definite (it is inverted in fp64 to recover the penalty matrix the earlier tokens left);
 * the periodic refresh, VLA_FLAG_TOKEN_MAJOR and VLA_KERNEL_TOKEN are not available
 * (VLA_ERR_UNSUPPORTED), nor is d = 16; `segments` must divide T/16 (T a multiple of 16), else VLA_ERR_INVALID_ARG;
 * segments <= 0 lets the library choose (vla_seqpar_segments), and a choice of 1 runs
 * vla_forward.  `workspace` is a DEVICE buffer of at least
 * vla_seqpar_workspace_bytes(B, H, T, d_k, segments) bytes (any alignment; with
 * segments <= 0 size it for vla_seqpar_segments(...)), owned by the caller and free for
 * reuse once the work enqueued on `stream` has completed.
 */
int vla_forward_seqpar(const void* q, const void* k, const void* v, float lambda_,
                       int B, int H, int T, int d_k, int d_v,
                       const float* S0, const float* A0,
                       float* out, float* S_T, float* A_T,
                       const vla_opts_t* opts, int segments,
                       void* workspace, size_t workspace_bytes, void* stream);

/* Segments per unit that vla_forward_seqpar picks on the current device for this problem:
   enough to fill the GPU with 2 * B * H * segments concurrent scans, at least 256 tokens each;
   1 when cutting does not pay (or the shape is not covered). */
int vla_seqpar_segments(int B, int H, int T, int d_k, int qkv_dtype);

/* Device bytes vla_forward_seqpar needs for `segments` >= 1 (0 on a bad argument). */
size_t vla_seqpar_workspace_bytes(int B, int H, int T, int d_k, int segments);

/*
 * vla_backward -- gradients of the forward scan.  The
 * paper gives no backward algorithm; this is reverse-mode differentiation of exactly the
 * recurrence vla_forward computes (Algorithm 1 without projections; Eqs. "sm", "s-update",
 * "output"), the gradients its Corollary on gradient flow (Section 4) is about.
 *
 * Inputs as vla_forward (q, k, v, lambda_, S0, A0, opts->z0, opts->flags, opts->eps,
 * opts->qkv_dtype) plus the incoming gradients d_out [B,H,T,d_v] and, optionally, dS_T, dA_T
 * [B,H,d,d], dz_T [B,H,d_k] (NULL = zero); all gradients are fp32.  Outputs dq, dk [B,H,T,d_k],
 * dv [B,H,T,d_v] and, when non-NULL, dS0, dA0, dz0.  The forward is recomputed inside; no
 * state of the forward call is needed.  In identity-map mode z_T = z0, so dz0 = dz_T.
 *
 * Covered: u = k_hat (opts->u NULL; d_k = d_v in {16, 32, 64, 128}) or explicit penalty
 * directions (opts->u given, used verbatim as in vla_forward; their gradient goes to opts->du,
 * which must then be non-NULL; d in {32, 64, 128}); the periodic refresh of opts (d in
 * {32, 64, 128}); VLA_FLAG_TOKEN_MAJOR (d in {32, 64, 128}); anything else returns
 * VLA_ERR_UNSUPPORTED.  `workspace` is a
 * DEVICE buffer of at least vla_backward_workspace_bytes(B, H, T, d_k) bytes (per token: z_t,
 * e_t, delta_t of the forward and three vectors the two reverse scans exchange; the final
 * states), owned by the caller and free for reuse once the work enqueued on `stream` has completed.
 */
int vla_backward(const void* q, const void* k, const void* v, float lambda_,
                 int B, int H, int T, int d_k, int d_v,
                 const float* S0, const float* A0,
                 const float* d_out, const float* dS_T, const float* dA_T, const float* dz_T,
                 float* dq, float* dk, float* dv, float* dS0, float* dA0, float* dz0,
                 const vla_opts_t* opts, void* workspace, size_t workspace_bytes, void* stream);

size_t vla_backward_workspace_bytes(int B, int H, int T, int d_k);

/*
 * vla_make_u -- the penalty directions of Algorithm 1 from a projection (its step
 * "u_t = L2norm(W_u k_t) / sqrt(d_h)", Section 3.2 "learned penalty"):
 *
 *     y_t = W_u[h] k_t,     u_t = scale * y_t / max(||y_t||_2, eps)
 *
 * for every token of every (b, h), to fp32 accuracy on the device (d_k = 128: on the tensor cores,
 * TF32 products in hi/lo pairs with fp32 accumulation; below that on the fp32 pipe).  k [B,H,T,d_k] (k_dtype, the raw keys:
 * no feature map is applied), W_u [H,d_k,d_k] fp32 row-major (one matrix per head; y = W k),
 * u [B,H,T,d_k] (u_dtype: VLA_F32, or VLA_BF16 rounded to nearest even) -- the buffer a later
 * vla_forward takes as opts->u (with opts->qkv_dtype == u_dtype).  scale is used as given
 * (Algorithm 1: 1/sqrt(d_k); Eq. "penalty": 1); eps <= 0 => 1e-4.  All DEVICE pointers, 16-byte
 * aligned, caller-owned; asynchronous on `stream`; nothing allocated.  d_k in {16,32,64,128},
 * else VLA_ERR_UNSUPPORTED.  A zero y_t gives u_t = 0 (no penalty for that token).
 */
int vla_make_u(const void* k, const float* W_u, int B, int H, int T, int d_k, int k_dtype, int u_dtype,
               float scale, float eps, void* u, void* stream);

/*
 * vla_probe_fp32_fma -- measurement helper (the paper has no counterpart): enqueues a
 * register-only loop of fp32 FMAs on every SM (2048 threads per SM, 16 independent chains per
 * thread, `iters` x 128 FMAs per thread) and reports the floating-point operations launched in
 * *flops (HOST pointer, may be NULL).  Timed with events by the caller it gives the fp32
 * FMA rate this device sustains at its current clocks -- the "alu" roofline the scan kernels
 * are measured against.  `sink` is a DEVICE float the kernel never actually writes.
 */
int vla_probe_fp32_fma(int iters, float* sink, double* flops, void* stream);

/*
 * vla_selftest_wait_timeout -- test helper (the paper has no counterpart): enqueues a one-warp
 * kernel that waits, with the scan kernels' bounded wait and `probe_limit` probes, on a barrier
 * that cannot complete.  When the probes run out the kernel writes VLA_ERR_DEVICE_TIMEOUT to
 * *status (DEVICE int32, 0 on entry) and returns normally; nothing traps and the context stays
 * usable.  probe_limit must be > 0 (a few thousand probes take well under a millisecond).
 */
int vla_selftest_wait_timeout(uint32_t probe_limit, int32_t* status, void* stream);

/*
 * vla_last_launch -- which kernel the calling host thread's last library call launched last,
 * as text ("vla_scan_chunk_kernel<128,bf16> grid=148 balanced"); empty before the first launch.
 * For benchmarks and logs: the name comes from the launch itself, not from the shape.
 */
int vla_last_launch(char* buf, size_t len);

/* Device bytes vla_forward_host needs for these sizes (0 on invalid sizes). */
size_t vla_host_workspace_bytes(int B, int H, int T, int d_k, int d_v, int qkv_dtype, int has_u);

/* VLA_OK when a kernel covers (d_k, d_v, dtype, flags), else VLA_ERR_UNSUPPORTED. */
int vla_query_support(int d_k, int d_v, int qkv_dtype, uint32_t flags);

/* Static, NUL-terminated description of a vla_status_t value. */
const char* vla_status_string(int status);

/* major*10000 + minor*100 + patch */
int vla_version(void);

#ifdef __cplusplus
}
#endif
#endif /* VLA_H */
