"""fp64 CPU oracle of the penalty directions formed from a projection.

TEST INFRASTRUCTURE ONLY (tests, the smoke check, the benchmark's CPU-baseline leg): the CUDA
package never imports this.

Algorithm 1, the step that forms u_t from the raw key, with the norm guarded like every other
denominator of the method (Section 5.3):

    y_t = W_u[h] k_t          (k_t: the raw key of head h, no feature map)
    u_t = scale * y_t / max(||y_t||_2, eps)

Algorithm 1 prints scale = 1/sqrt(d_h); Eq. "penalty" has a unit vector (scale = 1).  The stored
keys (fp32, or bf16 bit patterns) are widened exactly; everything else is float64.  numpy's
matmul is the one library step.
"""
import numpy as np

F32, BF16, F64 = 0, 1, 2


def widen(a, in_dtype):
    """Stored values as float64, exactly."""
    if in_dtype == BF16:
        bits = np.ascontiguousarray(a, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
        return bits.view(np.float32).astype(np.float64)
    return np.asarray(a).astype(np.float64)


def make_u(k, W_u, scale, eps=1e-4, in_dtype=F32):
    """k [B,H,T,d] stored keys, W_u [H,d,d] (y = W k) -> u [B,H,T,d] float64."""
    kk = widen(k, in_dtype)
    W = np.asarray(W_u, dtype=np.float64)
    B, H, T, d = kk.shape
    assert W.shape == (H, d, d)
    u = np.empty((B, H, T, d), dtype=np.float64)
    for b in range(B):
        for h in range(H):
            y = kk[b, h] @ W[h].T                      # row t: W[h] k_t
            nrm = np.sqrt((y * y).sum(axis=1))
            u[b, h] = scale * y / np.maximum(nrm, eps)[:, None]
    return u
