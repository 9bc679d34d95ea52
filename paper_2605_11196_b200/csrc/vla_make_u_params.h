// Arguments of the kernel that forms penalty directions from a projection (see vla_make_u.cuh).
#pragma once

namespace vla {

struct MakeUParams {
  const void* k;     // [units, T, D], TIn
  const float* W;    // [heads, D, D] row-major: y = W k
  void* u;           // [units, T, D], TOut
  float scale;
  float eps;
  int T;
  int units;
  int heads;
};

}  // namespace vla
