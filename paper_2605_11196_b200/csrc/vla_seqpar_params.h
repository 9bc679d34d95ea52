// Arguments of the sequence-parallel helper kernels (see vla_seqpar.cuh).
#pragma once

#include <cstdint>

namespace vla {

// CTAs that share the Gram matrix of one segment (they add into it atomically)
constexpr int kGramSplit = 4;

struct SeqParParams {
  const void* k;        // [units, T, D] raw keys
  const void* u;        // [units, T, D] explicit penalty directions or nullptr
  const float* S0;      // [units, D, D] or nullptr
  const float* A0;      // [units, D, D] symmetric positive definite, or nullptr (I / lambda)
  double* M0;           // [units, D, D] A0^-1 (only with A0)
  const float* z0;      // [units, D] or nullptr
  float* out;           // [units, T, D] o0 on entry of `correct`, o on exit
  float* S_T;           // [units, D, D] or nullptr
  double* Gd;           // [N, D, D]  segment Gram matrices, zero on entry (N = units * P)
  float* zsum;          // [N, D]     segment sums of phi(k), zero on entry
  float* Astart;        // [N, D, D]
  float* zstart;        // [N, D]
  const float* ST2;     // [2N, D, D]  G_j, then P_j
  const float* wn;      // [N, Ls, D]  transfer readouts
  float* Sstart;        // [N, D, D]
  float lambda;
  float eps;
  int T;                // tokens per unit
  int P;                // segments per unit
  int units;
  uint32_t flags;
};

}  // namespace vla
