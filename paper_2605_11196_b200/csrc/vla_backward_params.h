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
  float* zkc;           // workspace [units, ceil(T / 16), D]  key sum after each 16 tokens
  int* status;
  float lambda;
  float eps;
  int T;
  int units;
  uint32_t flags;
};

// Arguments of the two reverse scans (see vla_backward_split.cuh).
struct BackwardSplitParams {
  const void* q;        // [units, T, D]
  const void* k;
  const void* u;        // [units, T, D] explicit penalty directions, or nullptr (u = k_hat)
  const float* ast;     // [units, T, D] a_t = A_t k_hat_t of the forward (explicit u only)
  float* du;            // [units, T, D] gradient of u (explicit u only)
  const float* z0;      // unused by the sweeps (the forward consumed it)
  const float* d_out;   // [units, T, D]
  const float* dS_T;    // [units, D, D] or nullptr
  const float* dA_T;
  const float* dz_T;    // [units, D] or nullptr
  const float* ST;      // [units, D, D] final states of the forward (workspace)
  const float* AT;
  const float* zT;      // [units, D]
  const float* zst;     // [units, T, D] z_t
  const float* est;     // [units, T, D] e_t
  const float* dst;     // [units, T]    delta_t
  const float* zkc;     // [units, ceil(T / 16), D] key sum after each 16 tokens (paper mode)
  const float* ost;     // the forward's readout o_t, laid out like q (so that S_t qf_t = den_t o_t needs no product)
  float* dal;           // [units, T, D] S side -> A side: dL/d alpha_t
  float* dkS;           // [units, T, D] S side -> A side: S-side part of dL/d k_hat_t
  float* gzt;           // [units, T, D] S side -> A side: dL/d(key sum) seen by token t
  float* dq;            // [units, T, D]
  float* dk;
  float* dv;
  float* dS0;           // [units, D, D] or nullptr
  float* dA0;
  float* dz0;           // [units, D] or nullptr
  int* progress;             // [units + 1], zero on entry: per unit the tokens (from the end) whose S-side
                             // vectors are out; the last word hands out the CTAs' tickets
  int* status;
  float eps;
  int T;
  int units;
  uint32_t flags;
  int heads;                 // H, for [B, T, H, d] tensors (VLA_FLAG_TOKEN_MAJOR): unit = b * H + h
  int general;               // the general path: explicit u and / or the periodic refresh
  int refresh_period;        // <= 0: none
  float refresh_eta;
  long long step_offset;
};

}  // namespace vla
