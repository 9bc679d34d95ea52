// Sequence-parallel VLA forward: the helper kernels around the chunk kernel.
//
// Section 3.4 writes the memory recurrence as a composition of per-token maps.  With the map
// acting on the right (S_t = S_{t-1} R_t + G_t, R_t = I - k_hat_t alpha_t^T, G_t = v_t alpha_t^T)
// a segment of tokens composes to S_end = S_start P + G with P = prod R_t and G the state the
// segment reaches from S = 0.  The penalty side needs no composition at all: A before token t
// is the inverse of M = lambda I + sum_{s<t} u_s u_s^T (Eq. "penalty"), a prefix SUM, so A at a
// segment start comes from a Gram matrix and one inversion.  A unit's sequence is therefore cut
// into P equal segments that are scanned at the same time:
//
//   1. gram     G_j = sum_{t in segment j} u_t u_t^T  (fp32 products, fp64 accumulation) and
//               the segment's sum of phi(k)
//   2. invert   A_start_j = (lambda I + sum_{i<j} G_i)^-1 in fp64 (Gauss-Jordan, no pivoting:
//               the matrix is symmetric positive definite), running key sum at the start;
//               with a carried-in A0, lambda I is replaced by A0^-1 (also formed in fp64)
//   3. scan     the chunk kernel over 2 * units * P virtual units: segment j from S = 0
//               (readout o0_t, final state G_j) and its transfer scan from S = I with v = 0
//               (readout w_t = P_t q_t / den_t, final state P_j)
//   4. combine  per unit, in order: S_start_{j+1} = S_start_j P_j + G_j
//   5. correct  o_t = o0_t + S_start_j w_t
//
// All of it is exact algebra; it costs about twice the arithmetic of the plain scan and
// makes P times as many CTAs, which is what a long sequence with few (batch, head) units needs.
#pragma once

#include "vla_common.cuh"
#include "vla_seqpar_params.h"

namespace vla {


__device__ __forceinline__ float seqpar_phi(float x) { return x > 0.0f ? x + 1.0f : __expf(x); }

// ---- 1. Gram matrix and key sum of one slice of a segment.  Grid (units * P, kGramSplit): a
// segment's tokens are divided among kGramSplit CTAs of 256 threads, which add their results
// into the segment's (zeroed) matrix; the last segment of a unit needs neither and is skipped.
// Input rows: 8 lanes per token, 32 tokens per block, every load of a block in flight at once.
// Thread (ty, tx) of a 16 x 16 grid owns an R x R block of the D x D result, R = D / 16.

template <int D, typename TIn>
__global__ void __launch_bounds__(256) seqpar_gram_kernel(const SeqParParams p) {
  constexpr int R = D / 16;
  constexpr int TB = 32;          // tokens per shared-memory block (one fp32 partial sum)
  constexpr int EPL = D / 8;      // elements per lane of a token row (8 lanes per token)
  constexpr int LDU = D + 4;
  __shared__ __align__(16) float U[TB][LDU];
  __shared__ float zpart[TB][D];
  const int vu = blockIdx.x, unit = vu / p.P, j = vu % p.P;
  if (j == p.P - 1) return;
  const int Ls = p.T / p.P;
  // this CTA's tokens of the segment: [tlo, thi), whole 32-token blocks except at the end
  const int nblk = (Ls + TB - 1) / TB;
  const int tlo = int((long long)nblk * blockIdx.y / kGramSplit) * TB;
  const int thi = min(Ls, int((long long)nblk * (blockIdx.y + 1) / kGramSplit) * TB);
  const int tid = threadIdx.x;
  const int ty = tid >> 4, tx = tid & 15;
  const int tok = tid >> 3, pl = tid & 7;      // input stage: token of the block, lane of the token
  const bool ident = (p.flags & VLA_FLAG_IDENTITY_MAP) != 0;
  const TIn* kk = static_cast<const TIn*>(p.k) + (size_t(unit) * p.T + size_t(j) * Ls) * D;
  const TIn* uu = p.u ? static_cast<const TIn*>(p.u) + (size_t(unit) * p.T + size_t(j) * Ls) * D : nullptr;

  double accd[R][R];
#pragma unroll
  for (int a = 0; a < R; ++a)
#pragma unroll
    for (int b = 0; b < R; ++b) accd[a][b] = 0.0;
  float zs[EPL];
#pragma unroll
  for (int e = 0; e < EPL; ++e) zs[e] = 0.0f;

  for (int t0 = tlo; t0 < thi; t0 += TB) {
    // rows u_t of this block: k_hat = phi(k)/||phi(k)|| (or k/||k||), or the given u verbatim
    {
      const int t = t0 + tok;
      const bool act = t < thi;
      float x[EPL];
      float ss = 0.0f;
#pragma unroll
      for (int f = 0; f < EPL / 4; ++f) {
        float4 k4 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (act) k4 = load4(kk + size_t(t) * D, f * 8 + pl);
        if (act && !ident) {
          k4.x = seqpar_phi(k4.x); k4.y = seqpar_phi(k4.y);
          k4.z = seqpar_phi(k4.z); k4.w = seqpar_phi(k4.w);
        }
        x[4 * f + 0] = k4.x; x[4 * f + 1] = k4.y; x[4 * f + 2] = k4.z; x[4 * f + 3] = k4.w;
      }
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        zs[e] += x[e];
        ss = fmaf(x[e], x[e], ss);
      }
#pragma unroll
      for (int off = 4; off >= 1; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
      const float inv = 1.0f / fmaxf(sqrtf(ss), p.eps);
#pragma unroll
      for (int f = 0; f < EPL / 4; ++f) {
        float4 v4 = make_float4(x[4 * f] * inv, x[4 * f + 1] * inv, x[4 * f + 2] * inv, x[4 * f + 3] * inv);
        if (uu) v4 = act ? load4(uu + size_t(t) * D, f * 8 + pl) : make_float4(0.f, 0.f, 0.f, 0.f);
        *reinterpret_cast<float4*>(&U[tok][(f * 8 + pl) * 4]) = v4;
      }
    }
    __syncthreads();
    float acc[R][R];
#pragma unroll
    for (int a = 0; a < R; ++a)
#pragma unroll
      for (int b = 0; b < R; ++b) acc[a][b] = 0.0f;
#pragma unroll 4
    for (int tt = 0; tt < TB; ++tt) {
      float ra[R], cb[R];
#pragma unroll
      for (int a = 0; a < R; ++a) { ra[a] = U[tt][ty * R + a]; cb[a] = U[tt][tx * R + a]; }
#pragma unroll
      for (int a = 0; a < R; ++a)
#pragma unroll
        for (int b = 0; b < R; ++b) acc[a][b] = fmaf(ra[a], cb[b], acc[a][b]);
    }
#pragma unroll
    for (int a = 0; a < R; ++a)
#pragma unroll
      for (int b = 0; b < R; ++b) accd[a][b] += double(acc[a][b]);
    __syncthreads();
  }
  // the kGramSplit CTAs of a segment add into one matrix (zeroed by the host before the
  // launch): fp64 additions are scarce on this part, the inversion kernel should not repeat them
  double* G = p.Gd + size_t(vu) * D * D;
#pragma unroll
  for (int a = 0; a < R; ++a)
#pragma unroll
    for (int b = 0; b < R; ++b) atomicAdd(&G[(ty * R + a) * D + tx * R + b], accd[a][b]);
  // key sum: this thread's columns are (f * 8 + pl) * 4 + i; add over the 32 token slots
#pragma unroll
  for (int e = 0; e < EPL; ++e) zpart[tok][((e / 4) * 8 + pl) * 4 + (e & 3)] = zs[e];
  __syncthreads();
  for (int c = tid; c < D; c += 256) {
    float s = 0.0f;
#pragma unroll
    for (int w = 0; w < TB; ++w) s += zpart[w][c];
    atomicAdd(&p.zsum[size_t(vu) * D + c], s);
  }
}

// In-place Gauss-Jordan inversion of a symmetric positive definite D x D matrix held in
// registers by 256 threads (thread: row r, columns c0 .. c0 + EC - 1); no pivoting.  fp64
// arithmetic is scarce on this part: one FMA per element and pivot, the pivot's reciprocal
// folded into the column factor.
template <int D, int EC>
__device__ __forceinline__ void seqpar_gauss_jordan(double (&m)[EC], int r, int c0, double* rowraw,
                                                    double* colp) {
#pragma unroll 1
  for (int pv = 0; pv < D; ++pv) {
    if (r == pv) {
#pragma unroll
      for (int e = 0; e < EC; ++e) rowraw[c0 + e] = m[e];
    }
    if (pv >= c0 && pv < c0 + EC) {
      double x = 0.0;
#pragma unroll
      for (int e = 0; e < EC; ++e)
        if (c0 + e == pv) x = m[e];
      colp[r] = x;
    }
    __syncthreads();
    const double d = 1.0 / rowraw[pv];
    const double ncrd = -colp[r] * d;
    if (r == pv) {
#pragma unroll
      for (int e = 0; e < EC; ++e) m[e] = (c0 + e == pv) ? d : rowraw[c0 + e] * d;
    } else {
#pragma unroll
      for (int e = 0; e < EC; ++e) m[e] = (c0 + e == pv) ? ncrd : fma(ncrd, rowraw[c0 + e], m[e]);
    }
    __syncthreads();
  }
}

// ---- 2a. With a carried-in A0: M0 = A0^-1 per unit in fp64 (the penalty matrix the earlier
// tokens left behind).  One CTA of 256 threads per unit.
template <int D>
__global__ void __launch_bounds__(256) seqpar_m0_kernel(const SeqParParams p) {
  constexpr int EC = D * D / 256, TPR = D / EC;
  __shared__ double rowraw[D];
  __shared__ double colp[D];
  const int unit = blockIdx.x, tid = threadIdx.x;
  const int r = tid / TPR, c0 = (tid % TPR) * EC;
  double m[EC];
#pragma unroll
  for (int e = 0; e < EC; ++e) m[e] = double(p.A0[(size_t(unit) * D + r) * D + c0 + e]);
  seqpar_gauss_jordan<D, EC>(m, r, c0, rowraw, colp);
#pragma unroll
  for (int e = 0; e < EC; ++e) p.M0[(size_t(unit) * D + r) * D + c0 + e] = m[e];
}

// ---- 2. A at the start of segment j, and the running key sum there.  One CTA of 256
// threads per (unit, segment).  The matrix stays in registers: thread t owns D*D/256
// consecutive elements of one row; a pivot step exchanges only the pivot row and column
// through shared memory.
template <int D>
__global__ void __launch_bounds__(256) seqpar_invert_kernel(const SeqParParams p) {
  constexpr int EC = D * D / 256;     // elements per thread
  constexpr int TPR = D / EC;         // threads per row
  __shared__ double rowraw[D];        // pivot row before scaling
  __shared__ double colp[D];          // pivot column
  const int vu = blockIdx.x, unit = vu / p.P, j = vu % p.P;
  const int tid = threadIdx.x;
  const int r = tid / TPR, c0 = (tid % TPR) * EC;
  float* A = p.Astart + size_t(vu) * D * D;
  for (int c = tid; c < D; c += 256) {
    double s = p.z0 ? double(p.z0[size_t(unit) * D + c]) : 0.0;
    // the identity-map reading has no readout normaliser: the key sum is carried through
    if (!(p.flags & VLA_FLAG_IDENTITY_MAP))
      for (int i = 0; i < j; ++i) s += double(p.zsum[(size_t(unit) * p.P + i) * D + c]);
    p.zstart[size_t(vu) * D + c] = float(s);
  }
  if (j == 0) {
    const float dg = 1.0f / p.lambda;
#pragma unroll
    for (int e = 0; e < EC; ++e)
      A[r * D + c0 + e] = p.A0 ? p.A0[(size_t(unit) * D + r) * D + c0 + e] : ((c0 + e == r) ? dg : 0.0f);
    return;
  }
  // M = lambda I (or the carried-in A0^-1) + the Gram matrices of the earlier segments
  double m[EC];
#pragma unroll
  for (int e = 0; e < EC; ++e)
    m[e] = p.A0 ? p.M0[(size_t(unit) * D + r) * D + c0 + e] : ((c0 + e == r) ? double(p.lambda) : 0.0);
  for (int i = 0; i < j; ++i) {
    const double* G = p.Gd + (size_t(unit) * p.P + i) * D * D + r * D + c0;
#pragma unroll
    for (int e = 0; e < EC; ++e) m[e] += G[e];
  }
  seqpar_gauss_jordan<D, EC>(m, r, c0, rowraw, colp);
#pragma unroll
  for (int e = 0; e < EC; ++e) A[r * D + c0 + e] = float(m[e]);
}

// ---- 4. states at the segment starts, in order: S_start_{j+1} = S_start_j P_j + G_j.  The rows
// of S do not mix, so a unit is spread over D / 16 CTAs of 16 rows each: grid (units, D / 16),
// 256 threads (thread = one row of the block, D / 16 columns); dynamic shared memory:
// (16 + D) * (D + 1) floats.
template <int D>
__global__ void __launch_bounds__(256) seqpar_combine_kernel(const SeqParParams p) {
  extern __shared__ __align__(16) unsigned char seqpar_smem[];
  constexpr int LD = D + 1, R = D / 16, RB = 16;
  float* Sc = reinterpret_cast<float*>(seqpar_smem);   // [RB][LD] current rows of S_start
  float* Pj = Sc + RB * LD;                            // [D][LD]
  const int unit = blockIdx.x, row0 = blockIdx.y * RB, tid = threadIdx.x;
  const int ty = tid >> 4, tx = tid & 15;
  const size_t N = size_t(p.units) * p.P;
  for (int idx = tid; idx < RB * D; idx += 256)
    Sc[(idx / D) * LD + idx % D] = p.S0 ? p.S0[(size_t(unit) * D + row0) * D + idx] : 0.0f;
  __syncthreads();
  for (int j = 0; j < p.P; ++j) {
    const size_t vu = size_t(unit) * p.P + j;
    const float* G = p.ST2 + (vu * D + row0) * D;
    const float* Pg = p.ST2 + (N + vu) * D * D;
    float* Ss = p.Sstart + (vu * D + row0) * D;
    for (int idx = tid; idx < RB * D; idx += 256) Ss[idx] = Sc[(idx / D) * LD + idx % D];
    for (int idx = tid; idx < D * D; idx += 256) Pj[(idx / D) * LD + idx % D] = Pg[idx];
    __syncthreads();
    float acc[R];
#pragma unroll
    for (int b = 0; b < R; ++b) acc[b] = G[ty * D + tx * R + b];
#pragma unroll 4
    for (int m = 0; m < D; ++m) {
      const float sa = Sc[ty * LD + m];
#pragma unroll
      for (int b = 0; b < R; ++b) acc[b] = fmaf(sa, Pj[m * LD + tx * R + b], acc[b]);
    }
    __syncthreads();
#pragma unroll
    for (int b = 0; b < R; ++b) Sc[ty * LD + tx * R + b] = acc[b];
    __syncthreads();
  }
  if (p.S_T)
    for (int idx = tid; idx < RB * D; idx += 256)
      p.S_T[(size_t(unit) * D + row0) * D + idx] = Sc[(idx / D) * LD + idx % D];
}

// ---- 5. o_t = o0_t + S_start_j w_t.  Grid (units * P, ceil(Ls / 256)): a CTA keeps S_start_j
// in shared memory and walks four 64-token tiles of its segment; dynamic shared memory:
// D * (D + 4) + 64 * (D + 4) floats.
constexpr int kCorrectTile = 64;     // tokens per shared-memory tile
constexpr int kCorrectTiles = 4;     // tiles per CTA

template <int D>
__global__ void __launch_bounds__(256) seqpar_correct_kernel(const SeqParParams p) {
  extern __shared__ __align__(16) unsigned char seqpar_smem[];
  constexpr int LD = D + 4, TBK = kCorrectTile;
  constexpr int RW = D >= 64 ? 4 : 2;          // rows per thread: tr, tr + TRW, ...
  constexpr int TRW = D / RW;                  // threads along the rows
  constexpr int TTK = 256 / TRW;               // threads along the tokens
  constexpr int TT = TBK / TTK;                // tokens per thread
  float* Ss = reinterpret_cast<float*>(seqpar_smem);   // [D][LD]
  float* Wb = Ss + D * LD;                              // [TBK][LD]
  const int vu = blockIdx.x, j = vu % p.P;
  if (j == 0 && !p.S0) return;                 // S_start = 0: nothing to add
  const int Ls = p.T / p.P;
  const int tid = threadIdx.x;
  const int tr = tid % TRW, tk = tid / TRW;
  const float4* Sg = reinterpret_cast<const float4*>(p.Sstart + size_t(vu) * D * D);
  for (int idx = tid; idx < D * D / 4; idx += 256)
    *reinterpret_cast<float4*>(&Ss[(idx / (D / 4)) * LD + (idx % (D / 4)) * 4]) = Sg[idx];
  for (int tile = 0; tile < kCorrectTiles; ++tile) {
    const int t0 = (blockIdx.y * kCorrectTiles + tile) * TBK;
    if (t0 >= Ls) break;                       // uniform over the CTA
    const int nt = min(TBK, Ls - t0);
    __syncthreads();                           // the previous tile has been consumed
    const float4* wg = reinterpret_cast<const float4*>(p.wn + (size_t(vu) * Ls + t0) * D);
    for (int idx = tid; idx < TBK * D / 4; idx += 256) {
      const int t = idx / (D / 4);
      *reinterpret_cast<float4*>(&Wb[t * LD + (idx % (D / 4)) * 4]) =
          t < nt ? wg[idx] : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    __syncthreads();
    float acc[TT][RW];
#pragma unroll
    for (int a = 0; a < TT; ++a)
#pragma unroll
      for (int b = 0; b < RW; ++b) acc[a][b] = 0.0f;
#pragma unroll 2
    for (int m = 0; m < D; m += 4) {
      float4 sv[RW], wv[TT];
#pragma unroll
      for (int b = 0; b < RW; ++b) sv[b] = *reinterpret_cast<const float4*>(&Ss[(tr + b * TRW) * LD + m]);
#pragma unroll
      for (int a = 0; a < TT; ++a) wv[a] = *reinterpret_cast<const float4*>(&Wb[(tk * TT + a) * LD + m]);
#pragma unroll
      for (int a = 0; a < TT; ++a)
#pragma unroll
        for (int b = 0; b < RW; ++b) {
          acc[a][b] = fmaf(wv[a].x, sv[b].x, acc[a][b]);
          acc[a][b] = fmaf(wv[a].y, sv[b].y, acc[a][b]);
          acc[a][b] = fmaf(wv[a].z, sv[b].z, acc[a][b]);
          acc[a][b] = fmaf(wv[a].w, sv[b].w, acc[a][b]);
        }
    }
    float* og = p.out + (size_t(vu) * Ls + t0) * D;
#pragma unroll
    for (int a = 0; a < TT; ++a) {
      const int t = tk * TT + a;
      if (t < nt) {
#pragma unroll
        for (int b = 0; b < RW; ++b) og[size_t(t) * D + tr + b * TRW] += acc[a][b];
      }
    }
  }
}

}  // namespace vla
