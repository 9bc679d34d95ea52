// Penalty directions from a projection (Algorithm 1, the step u_t = L2norm(W_u k_t) / sqrt(d_h)):
//   y_t = W_u[h] k_t,   u_t = scale * y_t / max(||y_t||, eps)
// for every token of every (batch, head) unit, written in the layout and element type the scan
// kernels read explicit directions in.  A dense [tokens, d] x [d, d] product per head.  This
// file: the fp32-FMA form, used for d < 128 (d = 128 runs on the tensor cores, vla_make_u_tc.cuh):
// u feeds the recurrence, whose 1e-4 bound leaves no room for a reduced-precision product, and
// it is 2 d^2 of the scan's ~12 d^2 flops per token.
//
// One CTA of 256 threads takes kTokensPerCta consecutive tokens of one unit, W_u[h]^T staged
// once in shared memory; per tile of 64 tokens thread (ty, tx) of a 16 x 16 grid forms 4
// tokens x d/16 columns, the row norms are summed over the 16 lanes that share the tokens.
#pragma once

#include "vla_common.cuh"
#include "vla_make_u_params.h"

namespace vla {

constexpr int kMakeUTile = 64;
constexpr int kMakeUTokensPerCta = 1024;

template <int D>
struct MakeUCfg {
  static constexpr int WS = D + 4;   // padded rows keep 16-byte alignment and spread the banks
  static constexpr size_t smem_bytes = sizeof(float) * (size_t(D) * WS + size_t(kMakeUTile) * WS);
};

__device__ __forceinline__ float2 make_u_ffma2(float2 a, float2 b, float2 c) {
  uint64_t ra, rb, rc, rd;
  asm("mov.b64 %0, {%1, %2};" : "=l"(ra) : "f"(a.x), "f"(a.y));
  asm("mov.b64 %0, {%1, %2};" : "=l"(rb) : "f"(b.x), "f"(b.y));
  asm("mov.b64 %0, {%1, %2};" : "=l"(rc) : "f"(c.x), "f"(c.y));
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(rd) : "l"(ra), "l"(rb), "l"(rc));
  float2 d;
  asm("mov.b64 {%0, %1}, %2;" : "=f"(d.x), "=f"(d.y) : "l"(rd));
  return d;
}

__device__ __forceinline__ void store_u(float* p, float x) { *p = x; }
__device__ __forceinline__ void store_u(uint16_t* p, float x) {   // bf16, round to nearest even
  uint32_t b = __float_as_uint(x);
  b += 0x7fffu + ((b >> 16) & 1u);
  *p = uint16_t(b >> 16);
}

template <int D, typename TIn, typename TOut>
__global__ void __launch_bounds__(256) vla_make_u_kernel(const MakeUParams p) {
  using Cfg = MakeUCfg<D>;
  constexpr int WS = Cfg::WS;
  constexpr int CPT = D / 16;   // columns per thread
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* Wt = reinterpret_cast<float*>(smem_raw);   // Wt[j][c] = W[c][j]
  float* Ks = Wt + size_t(D) * WS;                  // Ks[token][j]
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int tiles_per_unit = (p.T + kMakeUTokensPerCta - 1) / kMakeUTokensPerCta;
  const int unit = blockIdx.x / tiles_per_unit;
  const int t_first = (blockIdx.x % tiles_per_unit) * kMakeUTokensPerCta;
  const int t_last = min(p.T, t_first + kMakeUTokensPerCta);
  const int head = unit % p.heads;
  const float* W = p.W + size_t(head) * D * D;
  for (int i = tid; i < D * D; i += 256) {
    const int c = i / D, j = i % D;
    Wt[j * WS + c] = W[i];
  }
  const TIn* gk = static_cast<const TIn*>(p.k) + size_t(unit) * size_t(p.T) * D;
  TOut* gu = static_cast<TOut*>(p.u) + size_t(unit) * size_t(p.T) * D;
  for (int t0 = t_first; t0 < t_last; t0 += kMakeUTile) {
    const int n = min(kMakeUTile, t_last - t0);
    __syncthreads();   // the previous tile has been read (and, first time, Wt is complete below)
    for (int i = tid; i < kMakeUTile * D; i += 256) {
      const int tk = i / D, j = i % D;
      Ks[tk * WS + j] = tk < n ? load1<TIn>(gk, size_t(t0 + tk) * D + j) : 0.0f;
    }
    __syncthreads();
    float acc[4][CPT];
    if constexpr (CPT % 2 == 0) {
      // column pairs: packed fp32 FMAs (half the issue slots of the scalar form)
      float2 acc2[4][CPT / 2];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int c = 0; c < CPT / 2; ++c) acc2[i][c] = make_float2(0.0f, 0.0f);
#pragma unroll 2
      for (int j = 0; j < D; j += 4) {
        float a[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float4 x = *reinterpret_cast<const float4*>(Ks + (ty * 4 + i) * WS + j);
          a[i][0] = x.x; a[i][1] = x.y; a[i][2] = x.z; a[i][3] = x.w;
        }
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
          float2 b[CPT / 2];
          if constexpr (CPT >= 4) {
            // this thread's columns come in groups of four, 64 apart: a warp's 16-byte reads of
            // one group are adjacent (no bank conflicts)
#pragma unroll
            for (int g4 = 0; g4 < CPT / 4; ++g4) {
              const float4 x = *reinterpret_cast<const float4*>(Wt + (j + jj) * WS + g4 * 64 + tx * 4);
              b[2 * g4] = make_float2(x.x, x.y);
              b[2 * g4 + 1] = make_float2(x.z, x.w);
            }
          } else {
#pragma unroll
            for (int c = 0; c < CPT / 2; ++c)
              b[c] = *reinterpret_cast<const float2*>(Wt + (j + jj) * WS + tx * CPT + 2 * c);
          }
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float2 aa = make_float2(a[i][jj], a[i][jj]);
#pragma unroll
            for (int c = 0; c < CPT / 2; ++c) acc2[i][c] = make_u_ffma2(aa, b[c], acc2[i][c]);
          }
        }
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int c = 0; c < CPT / 2; ++c) { acc[i][2 * c] = acc2[i][c].x; acc[i][2 * c + 1] = acc2[i][c].y; }
    } else {
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int c = 0; c < CPT; ++c) acc[i][c] = 0.0f;
#pragma unroll 2
      for (int j = 0; j < D; j += 4) {
        float a[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float4 x = *reinterpret_cast<const float4*>(Ks + (ty * 4 + i) * WS + j);
          a[i][0] = x.x; a[i][1] = x.y; a[i][2] = x.z; a[i][3] = x.w;
        }
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
          float b[CPT];
#pragma unroll
          for (int c = 0; c < CPT; ++c) b[c] = Wt[(j + jj) * WS + tx * CPT + c];
#pragma unroll
          for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int c = 0; c < CPT; ++c) acc[i][c] = fmaf(a[i][jj], b[c], acc[i][c]);
        }
      }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float ss = 0.0f;
#pragma unroll
      for (int c = 0; c < CPT; ++c) ss = fmaf(acc[i][c], acc[i][c], ss);
#pragma unroll
      for (int off = 8; off >= 1; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
      const float f = p.scale / fmaxf(sqrtf(ss), p.eps);
      const int tk = ty * 4 + i;
      if (tk < n) {
#pragma unroll
        for (int c = 0; c < CPT; ++c) {
          const int col = CPT >= 4 ? (c / 4) * 64 + tx * 4 + (c % 4) : tx * CPT + c;
          store_u(gu + size_t(t0 + tk) * D + col, acc[i][c] * f);
        }
      }
    }
  }
}

}  // namespace vla
