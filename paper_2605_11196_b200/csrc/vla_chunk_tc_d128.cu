// Tensor-core chunk kernel, d = 128, fp32 and bf16 inputs.
#include "vla.h"
#include "vla_launch.h"
#include "vla_scan_tc.cuh"

namespace vla {

int launch_chunk_tc(int d, int dtype, const ScanParams& p, cudaStream_t st) {
  if (d != 128) return VLA_ERR_UNSUPPORTED;
  if (p.flags & VLA_FLAG_TOKEN_MAJOR)
    return dtype == VLA_F32 ? launch_chunk_tc_t<float, true>(p, st) : launch_chunk_tc_t<uint16_t, true>(p, st);
  return dtype == VLA_F32 ? launch_chunk_tc_t<float, false>(p, st) : launch_chunk_tc_t<uint16_t, false>(p, st);
}

// The same as the forward of a backward pass (u = k_hat, no refresh): leaves z_t, e_t, delta_t per
// token and the key sum per chunk (p.stash_*, always [units, T, d]).
int launch_chunk_tc_stash(int d, int dtype, const ScanParams& p, cudaStream_t st) {
  if (d != 128) return VLA_ERR_UNSUPPORTED;
  if (p.flags & VLA_FLAG_TOKEN_MAJOR)
    return dtype == VLA_F32 ? launch_chunk_tc_t<float, true, true>(p, st) : launch_chunk_tc_t<uint16_t, true, true>(p, st);
  return dtype == VLA_F32 ? launch_chunk_tc_t<float, false, true>(p, st) : launch_chunk_tc_t<uint16_t, false, true>(p, st);
}

}  // namespace vla
