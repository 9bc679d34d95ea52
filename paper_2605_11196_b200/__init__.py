"""B200 (sm_100a) Variational Linear Attention forward scan: a C-ABI CUDA library
(``libvla.so``, declared in ``include/vla.h``) and this thin binding.

The library is loaded on first use; a missing build raises (no fallback path).
"""
from .binding import (VLA_BF16, VLA_ERR_ALIGNMENT, VLA_ERR_CUDA, VLA_ERR_DEVICE_TIMEOUT,  # noqa: F401
                      VLA_ERR_INVALID_ARG, VLA_ERR_NONFINITE, VLA_ERR_UNSUPPORTED, VLA_F32,
                      VLA_FLAG_CHECK_FINITE, VLA_FLAG_IDENTITY_MAP, VLA_FLAG_TOKEN_MAJOR, VLA_FLAG_LINEAR_ATTENTION, VLA_KERNEL_AUTO,
                      VLA_KERNEL_CHUNK, VLA_KERNEL_CHUNK_TC, VLA_KERNEL_DECODE, VLA_KERNEL_TOKEN, VLA_OK, VlaError, VlaOpts, VlaResult, library_path,
                      load_library, status_string, vla_forward, vla_forward_host,
                      vla_forward_host_static, VLA_ERR_TOO_LARGE, VLA_STATIC_SCRATCH_BYTES,
                      vla_host_workspace_bytes, vla_query_support, vla_version,
                      vla_forward_seqpar, seqpar_segments, seqpar_workspace_bytes,
                      measure_fp32_fma_tflops, vla_backward, VlaGrads,
                      backward_workspace_bytes, vla_make_u, last_launch,
                      selftest_wait_timeout)
from .autograd import vla_scan, check_status  # noqa: F401,E402
