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

}  // namespace vla
