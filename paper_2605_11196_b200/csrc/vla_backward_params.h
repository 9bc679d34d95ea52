// Arguments of the backward kernel (see vla_backward.cuh).
#pragma once

#include <cstdint>

namespace vla {

struct BackwardParams {
  const void* q;        // [units, T, D]
  const void* k;
  const void* v;
  const float* S0;      // [units, D, D] or nullptr
  const float* A0;      // [units, D, D] or nullptr
  const float* z0;      // [units, D] or nullptr
  const float* d_out;   // [units, T, D]
  const float* dS_T;    // [units, D, D] or nullptr
  const float* dA_T;
  const float* dz_T;    // [units, D] or nullptr
  float* dq;            // [units, T, D]
  float* dk;
  float* dv;
  float* dS0;           // [units, D, D] or nullptr
  float* dA0;
  float* dz0;           // [units, D] or nullptr
  float* zst;           // workspace [units, T, D]  z_t
  float* est;           // workspace [units, T, D]  e_t
  float* dst;           // workspace [units, T]     delta_t
  int* status;
  float lambda;
  float eps;
  int T;
  int units;
  uint32_t flags;
};

}  // namespace vla
