// VLA forward scan, "chunk" kernel (u = k_hat): the recurrence of Section 3.3 evaluated
// C = 16 tokens at a time in exact algebra, so that the fp32 FMA pipe works on rank-16
// updates instead of a chain of rank-1 steps.  One CTA per (batch, head) unit, two warp
// groups of D threads each:
//
//   group A holds A (the inverse penalty matrix) in registers, thread tile TR x TW;
//   group S holds S (the memory state) in registers, same tiling.
//
// For a chunk with keys K (rows k_hat_t), queries Q (rows q_f,t), values V, and the states
// A, S at the chunk start (Eqs. "sm", "s-update", "output"):
//
//   Z0 = A K^T                          W = K Z0 = K A K^T
//   I + W = L diag(delta) L^T           delta_t is Eq. "sm"'s 1 + u.z, L[t,s] = (z_s.k_t)/delta_s
//   Z  = Z0 L^-T                        column t is z_t = A_{t-1} k_hat_t
//   alpha_t = sc_t z_t,  sc_t = (1/delta_t) / max(||z_t||/delta_t, eps)      (A_t k_hat_t = z_t/delta_t)
//   A <- A - Z diag(1/delta) Z^T        (Woodbury form of 16 Sherman-Morrison steps)
//   B  = V^T - S K^T                    E = B (I + Gu)^-1,  Gu[s,t] = alpha_s.k_hat_t (s < t)
//   E' = E diag(sc) = B T2'             O[:,t] = (S q_t + sum_{s<=t} e'_s (z_s.q_t)) / den_t
//   S <- S + E' Z^T
//
// Group A runs ahead of group S; Z and T2' travel through a two-slot shared-memory ring
// guarded by mbarriers.  q/k/v arrive through a ring of 1-D bulk-async (TMA) copies; each
// group widens and normalises what it needs.  Every mbarrier wait is bounded: if one runs
// out the CTA records VLA_ERR_DEVICE_TIMEOUT, stops waiting and runs to its end.
#pragma once

#include "vla_common.cuh"

namespace vla {

// ---- packed fp32x2 arithmetic (one instruction, two FMAs on the fp32 pipe)
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) {
  unsigned long long ra, rb, rc, rd;
  ra = *reinterpret_cast<unsigned long long*>(&a);
  rb = *reinterpret_cast<unsigned long long*>(&b);
  rc = *reinterpret_cast<unsigned long long*>(&c);
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(rd) : "l"(ra), "l"(rb), "l"(rc));
  return *reinterpret_cast<float2*>(&rd);
}

__device__ __forceinline__ void group_bar(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

template <int D>
struct ChunkTile {
  static constexpr int TW = (D >= 64) ? 16 : 8;  // state columns per thread
  static constexpr int TR = D / TW;              // state rows per thread (= lanes per row block)
};

template <int D, typename TIn>
struct ChunkCfg {
  static constexpr int C = 16;                   // tokens per chunk
  static constexpr int TW = ChunkTile<D>::TW;
  static constexpr int TR = ChunkTile<D>::TR;
  static constexpr int LPR = D / TW;             // lanes that share a row block (== TR)
  static constexpr int NV = TW / 4;              // float4 operand groups per thread
  static constexpr int NG = D;                   // threads per warp group
  static constexpr int NT = 2 * D;               // threads per CTA
  static constexpr int NWG = D / 32;             // warps per group
  static constexpr int NSTAGE = sizeof(TIn) == 2 ? 4 : 3;
  static constexpr int RING = 2;
  static constexpr int TOK_LANES = D / 4;        // prep: threads per token
  static constexpr int TOK_PER_PASS = NG / TOK_LANES;  // = 4
  static constexpr int CP = C + 4;               // padded row of the small C x C matrices

  // shared memory layout (floats unless noted)
  static constexpr size_t raw_bytes = size_t(NSTAGE) * 3 * C * D * sizeof(TIn);
  static constexpr size_t slot_floats = size_t(C) * D + C * CP;       // Zs, T2p
  static constexpr size_t a_floats = size_t(3) * C * D + 2 * C * CP + NWG * C + 2 * C;
  //   KhA, Z0s, ZDs | Ws, T1s | N2p | delta, inv_delta
  static constexpr size_t s_floats = size_t(5) * C * D + 2 * C * D + C * CP + NWG * C + 2 * C;
  //   KhS, QfS, VS(B), R0s, Eps | ostage[2] | Hs | denp | nrm, inv_den
  static constexpr size_t smem_bytes = raw_bytes +
      (RING * slot_floats + a_floats + s_floats) * sizeof(float) +
      (2 * NSTAGE + 2 * RING) * sizeof(uint64_t) + 16 + 128;
};

// Reduce-scatter of N = LPR values over LPR consecutive lanes: on return v[0] is the sum,
// over those lanes, of the element whose index equals the lane's position in the group.
template <int LPR>
__device__ __forceinline__ float reduce_scatter(float (&v)[LPR], int cg) {
#pragma unroll
  for (int off = LPR / 2; off >= 1; off >>= 1) {
    const bool up = (cg & off) != 0;
#pragma unroll
    for (int i = 0; i < off; ++i) {
      const float send = up ? v[i] : v[i + off];
      const float keep = up ? v[i + off] : v[i];
      v[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
    }
  }
  return v[0];
}

// Reduce-scatter of 16 values over a full warp: lanes 2t and 2t+1 end with the sum of v[t].
__device__ __forceinline__ float warp_reduce_scatter16(float (&v)[16], int lane) {
#pragma unroll
  for (int off = 16; off >= 2; off >>= 1) {
    const int n = off / 2;  // values kept after this step
    const bool up = (lane & off) != 0;
#pragma unroll
    for (int i = 0; i < n; ++i) {
      const float send = up ? v[i] : v[i + n];
      const float keep = up ? v[i + n] : v[i];
      v[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
    }
  }
  v[0] += __shfl_xor_sync(0xffffffffu, v[0], 1);
  return v[0];  // token index = lane >> 1, with bits taken from lane bits 4..1
}

template <int D, typename TIn>
__global__ void __launch_bounds__(2 * D, 1) vla_scan_chunk_kernel(const ScanParams p) {
  using Cfg = ChunkCfg<D, TIn>;
  constexpr int C = Cfg::C, TW = Cfg::TW, TR = Cfg::TR, LPR = Cfg::LPR, NV = Cfg::NV;
  constexpr int NG = Cfg::NG, NWG = Cfg::NWG, NSTAGE = Cfg::NSTAGE, RING = Cfg::RING;
  constexpr int TOK_LANES = Cfg::TOK_LANES, TOK_PER_PASS = Cfg::TOK_PER_PASS, CP = Cfg::CP;
  static_assert(TR == LPR, "row ownership after the reduce-scatter needs TR == D/TW");
  static_assert(C == 16, "the small-matrix code is written for 16-token chunks");

  extern __shared__ __align__(128) unsigned char smem[];
  TIn* raw = reinterpret_cast<TIn*>(smem);
  float* fbase = reinterpret_cast<float*>(smem + Cfg::raw_bytes);
  // ring slots
  float* ringZ[RING];
  float* ringT2[RING];
#pragma unroll
  for (int r = 0; r < RING; ++r) {
    ringZ[r] = fbase + size_t(r) * Cfg::slot_floats;
    ringT2[r] = ringZ[r] + C * D;
  }
  float* abase = fbase + RING * Cfg::slot_floats;
  float* KhA = abase;
  float* Z0s = KhA + C * D;
  float* ZDs = Z0s + C * D;
  float* Ws = ZDs + C * D;      // [C][CP]
  float* T1s = Ws + C * CP;     // [C][CP]
  float* N2p = T1s + C * CP;    // [NWG][C]
  float* dlt = N2p + NWG * C;   // [C]
  float* idl = dlt + C;         // [C]
  float* sbase = abase + Cfg::a_floats;
  float* KhS = sbase;
  float* QfS = KhS + C * D;
  float* VS = QfS + C * D;      // becomes B = V - S K^T in place
  float* R0s = VS + C * D;
  float* Eps = R0s + C * D;
  float* ostage = Eps + C * D;  // [2][C*D]
  float* Hs = ostage + 2 * C * D;  // [C][CP]
  float* denp = Hs + C * CP;       // [NWG][C]
  float* nrm = denp + NWG * C;     // [C]
  float* inv_den = nrm + C;        // [C]
  uint64_t* bars = reinterpret_cast<uint64_t*>(
      (reinterpret_cast<uintptr_t>(sbase + Cfg::s_floats) + 15) & ~uintptr_t(15));
  uint64_t* full = bars;                    // [NSTAGE] raw stage filled by TMA
  uint64_t* empty = full + NSTAGE;          // [NSTAGE] both groups done with the raw stage
  uint64_t* ring_full = empty + NSTAGE;     // [RING] group A published Z, T2'
  uint64_t* ring_empty = ring_full + RING;  // [RING] group S is done with the slot
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ring_empty + RING);

  const int tid = threadIdx.x;
  const bool is_A = tid < NG;
  const int g = is_A ? tid : tid - NG;   // thread within its group; also the row it owns
  const int lane = g & 31, gw = g >> 5;
  const int cg = g % LPR;                // column group
  const int rb = g / LPR;                // row block: rows rb*TR .. rb*TR+TR-1
  const int unit = blockIdx.x;
  const int T = p.T;
  const bool ident = (p.flags & VLA_FLAG_IDENTITY_MAP) != 0;
  const float eps = p.eps;
  const int nchunks = (T + C - 1) / C;

  const size_t tok_base = size_t(unit) * size_t(T);
  const TIn* gq = static_cast<const TIn*>(p.q) + tok_base * D;
  const TIn* gk = static_cast<const TIn*>(p.k) + tok_base * D;
  const TIn* gv = static_cast<const TIn*>(p.v) + tok_base * D;
  float* gout = p.out + tok_base * D;

  auto issue = [&](int c) {
    const int s = c % NSTAGE;
    const int n = min(C, T - c * C);
    const uint32_t bytes = uint32_t(n) * D * sizeof(TIn);
    TIn* dst = raw + size_t(s) * 3 * C * D;
    const size_t off = size_t(c) * C * D;
    mbar_arrive_expect_tx(&full[s], 3 * bytes);
    bulk_load(dst + 0 * C * D, gq + off, bytes, &full[s]);
    bulk_load(dst + 1 * C * D, gk + off, bytes, &full[s]);
    bulk_load(dst + 2 * C * D, gv + off, bytes, &full[s]);
  };
  // Bounded wait shared by every mbarrier in this kernel.
  auto wait = [&](uint64_t* bar, uint32_t parity) {
    if (*abort_flag) return;
    if (!mbar_wait_bounded(bar, parity)) {
      *abort_flag = 1;
      if (p.status) atomicCAS(p.status, 0, int(VLA_ERR_DEVICE_TIMEOUT));
    }
  };

  if (tid == 0) {
    for (int s = 0; s < NSTAGE; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 2); }
    for (int r = 0; r < RING; ++r) { mbar_init(&ring_full[r], 1); mbar_init(&ring_empty[r], 1); }
    *abort_flag = 0;
    mbar_init_fence();
  }
  __syncthreads();
  if (tid == NG) {  // thread 0 of group S is the TMA producer
    for (int c = 0; c < NSTAGE && c < nchunks; ++c) issue(c);
  }

  // ---- a0: this thread's TR x TW tile of A (group A) or S (group S), as column pairs
  float2 st[TR][TW / 2];
  {
    const float* src = is_A ? p.A0 : p.S0;
#pragma unroll
    for (int r = 0; r < TR; ++r) {
      const int row = rb * TR + r;
#pragma unroll
      for (int m = 0; m < NV; ++m) {
        const int c4 = m * LPR + cg;
        float4 x;
        if (src) {
          x = reinterpret_cast<const float4*>(src + (size_t(unit) * D + row) * D)[c4];
        } else {
          const float dg = is_A ? 1.0f / p.lambda : 0.0f;
          x.x = (c4 * 4 + 0 == row) ? dg : 0.0f;
          x.y = (c4 * 4 + 1 == row) ? dg : 0.0f;
          x.z = (c4 * 4 + 2 == row) ? dg : 0.0f;
          x.w = (c4 * 4 + 3 == row) ? dg : 0.0f;
        }
        st[r][2 * m] = make_float2(x.x, x.y);
        st[r][2 * m + 1] = make_float2(x.z, x.w);
      }
    }
  }

  const int ptok0 = g / TOK_LANES;  // prep: first token of this thread (then +4, +8, +12)
  const int pc4 = g % TOK_LANES;    // prep: float4 column group

#ifdef VLA_SECTION_TIMERS
  long long tsec[12];
  for (int i = 0; i < 12; ++i) tsec[i] = 0;
  long long tlast = clock64();
#define VLA_MARK(i) { long long now_ = clock64(); tsec[i] += now_ - tlast; tlast = now_; }
#else
#define VLA_MARK(i)
#endif

  if (is_A) {
    // =====================================================================  group A
    for (int c = 0; c < nchunks; ++c) {
      const int s = c % NSTAGE;
      const int n = min(C, T - c * C);
      const int slot = c % RING;
      wait(&full[s], (c / NSTAGE) & 1);
      VLA_MARK(0)

      // ---- prep: k_hat rows of this chunk (zero rows past the end of the sequence)
      {
        const TIn* rk = raw + (size_t(s) * 3 + 1) * C * D;
#pragma unroll
        for (int it = 0; it < C / TOK_PER_PASS; ++it) {
          const int tt = it * TOK_PER_PASS + ptok0;
          const bool act = tt < n;
          float4 kf = make_float4(0.f, 0.f, 0.f, 0.f);
          if (act) {
            kf = load4(rk + tt * D, pc4);
            if (!ident) {
              kf.x = phi_elu1(kf.x); kf.y = phi_elu1(kf.y);
              kf.z = phi_elu1(kf.z); kf.w = phi_elu1(kf.w);
            }
          }
          float ss = kf.x * kf.x + kf.y * kf.y + kf.z * kf.z + kf.w * kf.w;
#pragma unroll
          for (int off = TOK_LANES / 2; off >= 1; off >>= 1)
            ss += __shfl_xor_sync(0xffffffffu, ss, off);
          const float inv = 1.0f / fmaxf(sqrtf(ss), eps);
          reinterpret_cast<float4*>(KhA + tt * D)[pc4] =
              make_float4(kf.x * inv, kf.y * inv, kf.z * inv, kf.w * inv);
        }
      }
      group_bar(1, NG);
      VLA_MARK(1)
      if (g == 0) mbar_arrive(&empty[s]);

      // ---- Z0 = A K^T: per token one pass over the tile, reduce-scatter over the row block
#pragma unroll 2
      for (int t = 0; t < C; ++t) {
        float2 acc[TR];
#pragma unroll
        for (int r = 0; r < TR; ++r) acc[r] = make_float2(0.f, 0.f);
#pragma unroll
        for (int m = 0; m < NV; ++m) {
          const float4 k4 = reinterpret_cast<const float4*>(KhA + t * D)[m * LPR + cg];
          const float2 k01 = make_float2(k4.x, k4.y), k23 = make_float2(k4.z, k4.w);
#pragma unroll
          for (int r = 0; r < TR; ++r) {
            acc[r] = ffma2(st[r][2 * m], k01, acc[r]);
            acc[r] = ffma2(st[r][2 * m + 1], k23, acc[r]);
          }
        }
        float v[TR];
#pragma unroll
        for (int r = 0; r < TR; ++r) v[r] = acc[r].x + acc[r].y;
        Z0s[t * D + g] = reduce_scatter<LPR>(v, cg);
      }
      group_bar(1, NG);
      VLA_MARK(2)

      // ---- W = K Z0 (C x C), 4x4 output tiles, D/16 threads per tile over the d index
      {
        constexpr int P = NG / 16;  // threads per output tile
        const int tile = g / P, part = g % P;
        const int s0 = (tile >> 2) * 4, t0 = (tile & 3) * 4;
        float w[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) w[i] = 0.f;
#pragma unroll
        for (int step = 0; step < D / (4 * P); ++step) {
          const int f = step * P + part;
          float4 a[4], b[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            a[i] = reinterpret_cast<const float4*>(KhA + (s0 + i) * D)[f];
            b[i] = reinterpret_cast<const float4*>(Z0s + (t0 + i) * D)[f];
          }
#pragma unroll
          for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              w[4 * i + j] = fmaf(a[i].x, b[j].x, w[4 * i + j]);
              w[4 * i + j] = fmaf(a[i].y, b[j].y, w[4 * i + j]);
              w[4 * i + j] = fmaf(a[i].z, b[j].z, w[4 * i + j]);
              w[4 * i + j] = fmaf(a[i].w, b[j].w, w[4 * i + j]);
            }
        }
        // sum over the P threads of the tile (consecutive lanes)
#pragma unroll
        for (int off = P / 2; off >= 1; off >>= 1)
#pragma unroll
          for (int i = 0; i < 16; ++i) w[i] += __shfl_xor_sync(0xffffffffu, w[i], off);
        if (part == 0) {
#pragma unroll
          for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) Ws[(s0 + i) * CP + t0 + j] = w[4 * i + j];
        }
      }
      group_bar(1, NG);
      VLA_MARK(3)

      // ---- warp 0: I + W = L diag(delta) L^T, then T1 = L^-T (Z = Z0 T1)
      if (gw == 0) {
        // lane l holds row r = l & 15, columns h*8 .. h*8+7 (h = l >> 4) of M = I + W
        const int r = lane & 15, h = lane >> 4;
        float m[8], lrow[16];
#pragma unroll
        for (int j = 0; j < 8; ++j) m[j] = Ws[r * CP + h * 8 + j] + ((h * 8 + j == r) ? 1.0f : 0.0f);
#pragma unroll
        for (int s2 = 0; s2 < 16; ++s2) {
          const int hs = s2 >> 3, js = s2 & 7;
          const float piv = fmaxf(__shfl_sync(0xffffffffu, m[js], s2 + 16 * hs), eps);
          const float mrs = __shfl_sync(0xffffffffu, m[js], r + 16 * hs);
          const float ipiv = 1.0f / piv;
          const float l = (r > s2) ? mrs * ipiv : 0.0f;
          lrow[s2] = l;  // L[r][s2]
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float msj = __shfl_sync(0xffffffffu, m[j], s2 + 16 * h);
            m[j] = fmaf(-l, msj, m[j]);
          }
          if (lane == 0) { dlt[s2] = piv; idl[s2] = ipiv; }
        }
        // T1[:, t] = e_t - sum_{s<t} L[t][s] T1[:, s]; lane r (< 16) keeps row r of T1
        float t1[16];
#pragma unroll
        for (int t = 0; t < 16; ++t) {
          float a0 = (r == t) ? 1.0f : 0.0f, a1 = 0.0f;
#pragma unroll
          for (int s2 = 0; s2 < t; ++s2) {
            const float lts = __shfl_sync(0xffffffffu, lrow[s2], t);  // L[t][s2]
            if (s2 & 1) a1 = fmaf(-lts, t1[s2], a1); else a0 = fmaf(-lts, t1[s2], a0);
          }
          t1[t] = a0 + a1;
        }
        if (h == 0) {
#pragma unroll
          for (int t = 0; t < 16; ++t) T1s[r * CP + t] = t1[t];
        } else {
          // upper half keeps L for the T2' step: Ws is free now, store L there (row r)
#pragma unroll
          for (int s2 = 0; s2 < 16; ++s2) Ws[r * CP + s2] = lrow[s2];
        }
      }
      group_bar(1, NG);
      VLA_MARK(4)

      // the ring slot must have been released by group S (chunk c - RING)
      if (c >= RING) wait(&ring_empty[slot], ((c / RING) + 1) & 1);
      VLA_MARK(5)

      // ---- Z = Z0 T1 (row g), published as Zs; ZD = Z / delta; partial ||z_t||^2
      {
        float z0[16], z[16];
#pragma unroll
        for (int t = 0; t < 16; ++t) z0[t] = Z0s[t * D + g];
#pragma unroll
        for (int t = 0; t < 16; ++t) z[t] = 0.f;
#pragma unroll
        for (int s2 = 0; s2 < 16; ++s2) {
#pragma unroll
          for (int t4 = s2 / 4; t4 < 4; ++t4) {
            const float4 tt = reinterpret_cast<const float4*>(T1s + s2 * CP)[t4];
            if (4 * t4 + 0 >= s2) z[4 * t4 + 0] = fmaf(z0[s2], tt.x, z[4 * t4 + 0]);
            if (4 * t4 + 1 >= s2) z[4 * t4 + 1] = fmaf(z0[s2], tt.y, z[4 * t4 + 1]);
            if (4 * t4 + 2 >= s2) z[4 * t4 + 2] = fmaf(z0[s2], tt.z, z[4 * t4 + 2]);
            if (4 * t4 + 3 >= s2) z[4 * t4 + 3] = fmaf(z0[s2], tt.w, z[4 * t4 + 3]);
          }
        }
        float* Zs = ringZ[slot];
        float sq[16];
#pragma unroll
        for (int t = 0; t < 16; ++t) {
          Zs[t * D + g] = z[t];
          ZDs[t * D + g] = z[t] * idl[t];
          sq[t] = z[t] * z[t];
        }
        const float tot = warp_reduce_scatter16(sq, lane);
        // lane bits 4..1 select the token: bit 4 <-> token bit 3, ..., bit 1 <-> token bit 0
        if ((lane & 1) == 0) N2p[gw * C + (lane >> 1)] = tot;
      }
      group_bar(1, NG);
      VLA_MARK(6)

      // ---- warp 1 (or 0 when the group has one warp): sc, Gu, T2' = (I + Gu)^-1 diag(sc)
      if (gw == (NWG > 1 ? 1 : 0)) {
        const int r = lane & 15;
        float n2 = 0.f;
#pragma unroll
        for (int w2 = 0; w2 < NWG; ++w2) n2 += N2p[w2 * C + r];
        const float id_r = idl[r], d_r = dlt[r];
        const float sc_r = id_r / fmaxf(sqrtf(n2) * id_r, eps);  // alpha_r = sc_r z_r
        if ((p.flags & VLA_FLAG_CHECK_FINITE) && p.status && !isfinite(n2 + d_r))
          atomicCAS(p.status, 0, int(VLA_ERR_NONFINITE));
        // lane r keeps row r of T2 and the column r of Gu: Gu[s][t] = sc_s delta_s L[t][s]
        // T2[:, t] = e_t - sum_{s<t} Gu[s][t] T2[:, s]
        const float scd = sc_r * d_r;
        float t2[16];
#pragma unroll
        for (int t = 0; t < 16; ++t) {
          float a0 = (r == t) ? 1.0f : 0.0f, a1 = 0.0f;
#pragma unroll
          for (int s2 = 0; s2 < t; ++s2) {
            // Gu[s2][t] = sc_{s2} delta_{s2} L[t][s2]
            const float gst = __shfl_sync(0xffffffffu, scd, s2) * Ws[t * CP + s2];
            if (s2 & 1) a1 = fmaf(-gst, t2[s2], a1); else a0 = fmaf(-gst, t2[s2], a0);
          }
          t2[t] = a0 + a1;
        }
        float* T2p = ringT2[slot];
        if (lane < 16) {
#pragma unroll
          for (int t = 0; t < 16; ++t)
            T2p[r * CP + t] = t2[t] * __shfl_sync(0x0000ffffu, sc_r, t);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&ring_full[slot]);
      }

      VLA_MARK(7)
      // ---- A <- A - Z diag(1/delta) Z^T
      {
        const float* Zs = ringZ[slot];
#pragma unroll 2
        for (int s2 = 0; s2 < C; ++s2) {
          float zd[TR];
#pragma unroll
          for (int r4 = 0; r4 < TR / 4; ++r4) {
            const float4 x = reinterpret_cast<const float4*>(ZDs + s2 * D + rb * TR)[r4];
            zd[4 * r4 + 0] = -x.x; zd[4 * r4 + 1] = -x.y; zd[4 * r4 + 2] = -x.z; zd[4 * r4 + 3] = -x.w;
          }
#pragma unroll
          for (int m = 0; m < NV; ++m) {
            const float4 z4 = reinterpret_cast<const float4*>(Zs + s2 * D)[m * LPR + cg];
            const float2 z01 = make_float2(z4.x, z4.y), z23 = make_float2(z4.z, z4.w);
#pragma unroll
            for (int r = 0; r < TR; ++r) {
              const float2 zz = make_float2(zd[r], zd[r]);
              st[r][2 * m] = ffma2(zz, z01, st[r][2 * m]);
              st[r][2 * m + 1] = ffma2(zz, z23, st[r][2 * m + 1]);
            }
          }
        }
      }
      group_bar(1, NG);  // ZDs, Ws, N2p may be rewritten by the next chunk
      VLA_MARK(8)
    }
    // final A
    if (p.A_T) {
#pragma unroll
      for (int r = 0; r < TR; ++r) {
        const int row = rb * TR + r;
#pragma unroll
        for (int m = 0; m < NV; ++m)
          reinterpret_cast<float4*>(p.A_T + (size_t(unit) * D + row) * D)[m * LPR + cg] =
              make_float4(st[r][2 * m].x, st[r][2 * m].y, st[r][2 * m + 1].x, st[r][2 * m + 1].y);
      }
    }
  } else {
    // =====================================================================  group S
    float zk = 0.0f;  // running sum of phi(k), column g
    if (p.z0) zk = p.z0[size_t(unit) * D + g];
    if (g < C) inv_den[g] = 1.0f;

    for (int c = 0; c < nchunks; ++c) {
      const int s = c % NSTAGE;
      const int n = min(C, T - c * C);
      const int slot = c % RING;
      wait(&full[s], (c / NSTAGE) & 1);
      VLA_MARK(0)
      if (g == 0) bulk_wait_read<1>();  // the out stage of chunk c-2 has left shared memory

      // ---- prep: k_hat, ||phi(k)||, q_f, v (zero rows past the end of the sequence)
      {
        const TIn* rq = raw + (size_t(s) * 3 + 0) * C * D;
        const TIn* rk = raw + (size_t(s) * 3 + 1) * C * D;
        const TIn* rv = raw + (size_t(s) * 3 + 2) * C * D;
#pragma unroll
        for (int it = 0; it < C / TOK_PER_PASS; ++it) {
          const int tt = it * TOK_PER_PASS + ptok0;
          const bool act = tt < n;
          float4 kf = make_float4(0.f, 0.f, 0.f, 0.f), qf = kf, vv = kf;
          if (act) {
            kf = load4(rk + tt * D, pc4);
            qf = load4(rq + tt * D, pc4);
            vv = load4(rv + tt * D, pc4);
            if (!ident) {
              kf.x = phi_elu1(kf.x); kf.y = phi_elu1(kf.y);
              kf.z = phi_elu1(kf.z); kf.w = phi_elu1(kf.w);
              qf.x = phi_elu1(qf.x); qf.y = phi_elu1(qf.y);
              qf.z = phi_elu1(qf.z); qf.w = phi_elu1(qf.w);
            }
          }
          float ss = kf.x * kf.x + kf.y * kf.y + kf.z * kf.z + kf.w * kf.w;
#pragma unroll
          for (int off = TOK_LANES / 2; off >= 1; off >>= 1)
            ss += __shfl_xor_sync(0xffffffffu, ss, off);
          const float nr = sqrtf(ss);
          const float inv = 1.0f / fmaxf(nr, eps);
          reinterpret_cast<float4*>(KhS + tt * D)[pc4] =
              make_float4(kf.x * inv, kf.y * inv, kf.z * inv, kf.w * inv);
          reinterpret_cast<float4*>(QfS + tt * D)[pc4] = qf;
          reinterpret_cast<float4*>(VS + tt * D)[pc4] = vv;
          // phi(k) = k_hat * mult (mult = max(||phi(k)||, eps) unless the floor was active)
          if (pc4 == 0) nrm[tt] = act ? fmaxf(nr, eps) : 0.0f;
        }
      }
      group_bar(2, NG);
      VLA_MARK(1)
      if (g == 0) {
        mbar_arrive(&empty[s]);
        if (c + NSTAGE < nchunks) {  // refill the stage once group A has left it too
          wait(&empty[s], (c / NSTAGE) & 1);
          issue(c + NSTAGE);
        }
      }

      // ---- running key sum and readout denominators (thread = column g)
      if (!ident) {
        float pr[16];
#pragma unroll
        for (int t = 0; t < 16; ++t) {
          zk = fmaf(KhS[t * D + g], nrm[t], zk);
          pr[t] = zk * QfS[t * D + g];
        }
        const float tot = warp_reduce_scatter16(pr, lane);
        if ((lane & 1) == 0) denp[gw * C + (lane >> 1)] = tot;
      }

      // ---- P0 = S K^T, R0 = S Q^T; B = V^T - P0 (in place over V)
#pragma unroll 2
      for (int t = 0; t < C; ++t) {
        float2 ap[TR], ar[TR];
#pragma unroll
        for (int r = 0; r < TR; ++r) { ap[r] = make_float2(0.f, 0.f); ar[r] = make_float2(0.f, 0.f); }
#pragma unroll
        for (int m = 0; m < NV; ++m) {
          const float4 k4 = reinterpret_cast<const float4*>(KhS + t * D)[m * LPR + cg];
          const float4 q4 = reinterpret_cast<const float4*>(QfS + t * D)[m * LPR + cg];
          const float2 k01 = make_float2(k4.x, k4.y), k23 = make_float2(k4.z, k4.w);
          const float2 q01 = make_float2(q4.x, q4.y), q23 = make_float2(q4.z, q4.w);
#pragma unroll
          for (int r = 0; r < TR; ++r) {
            ap[r] = ffma2(st[r][2 * m], k01, ap[r]);
            ap[r] = ffma2(st[r][2 * m + 1], k23, ap[r]);
            ar[r] = ffma2(st[r][2 * m], q01, ar[r]);
            ar[r] = ffma2(st[r][2 * m + 1], q23, ar[r]);
          }
        }
        float vp[TR], vr[TR];
#pragma unroll
        for (int r = 0; r < TR; ++r) { vp[r] = ap[r].x + ap[r].y; vr[r] = ar[r].x + ar[r].y; }
        const float p0 = reduce_scatter<LPR>(vp, cg);
        const float r0 = reduce_scatter<LPR>(vr, cg);
        VS[t * D + g] = VS[t * D + g] - p0;   // same thread wrote nothing else here: row g
        R0s[t * D + g] = r0;
      }

      // ---- wait for group A's Z and T2' of this chunk
      wait(&ring_full[slot], (c / RING) & 1);
      VLA_MARK(2)
      const float* Zs = ringZ[slot];
      const float* T2p = ringT2[slot];
      group_bar(2, NG);  // KhS/QfS/VS/R0s/denp complete for every row
      VLA_MARK(3)

      // ---- H'[s][t] = z_s . q_t (C x C), same tiling as W; and the denominators
      {
        constexpr int P = NG / 16;
        const int tile = g / P, part = g % P;
        const int s0 = (tile >> 2) * 4, t0 = (tile & 3) * 4;
        float w[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) w[i] = 0.f;
#pragma unroll
        for (int step = 0; step < D / (4 * P); ++step) {
          const int f = step * P + part;
          float4 a[4], b[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            a[i] = reinterpret_cast<const float4*>(Zs + (s0 + i) * D)[f];
            b[i] = reinterpret_cast<const float4*>(QfS + (t0 + i) * D)[f];
          }
#pragma unroll
          for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              w[4 * i + j] = fmaf(a[i].x, b[j].x, w[4 * i + j]);
              w[4 * i + j] = fmaf(a[i].y, b[j].y, w[4 * i + j]);
              w[4 * i + j] = fmaf(a[i].z, b[j].z, w[4 * i + j]);
              w[4 * i + j] = fmaf(a[i].w, b[j].w, w[4 * i + j]);
            }
        }
#pragma unroll
        for (int off = P / 2; off >= 1; off >>= 1)
#pragma unroll
          for (int i = 0; i < 16; ++i) w[i] += __shfl_xor_sync(0xffffffffu, w[i], off);
        if (part == 0) {
#pragma unroll
          for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) Hs[(s0 + i) * CP + t0 + j] = w[4 * i + j];
        }
        if (!ident && g < C) {
          float dd = 0.f;
#pragma unroll
          for (int w2 = 0; w2 < NWG; ++w2) dd += denp[w2 * C + g];
          inv_den[g] = 1.0f / fmaxf(dd, eps);
        }
      }
      group_bar(2, NG);
      VLA_MARK(4)

      // ---- row g: e'_t = sum_{s<=t} b_s T2'[s][t];  o_t = (r0_t + sum_{s<=t} e'_s H'[s][t]) / den_t
      {
        float b[16], e[16], o[16];
#pragma unroll
        for (int t = 0; t < 16; ++t) { b[t] = VS[t * D + g]; e[t] = 0.f; o[t] = R0s[t * D + g]; }
#pragma unroll
        for (int s2 = 0; s2 < 16; ++s2) {
#pragma unroll
          for (int t4 = s2 / 4; t4 < 4; ++t4) {
            const float4 tt = reinterpret_cast<const float4*>(T2p + s2 * CP)[t4];
            if (4 * t4 + 0 >= s2) e[4 * t4 + 0] = fmaf(b[s2], tt.x, e[4 * t4 + 0]);
            if (4 * t4 + 1 >= s2) e[4 * t4 + 1] = fmaf(b[s2], tt.y, e[4 * t4 + 1]);
            if (4 * t4 + 2 >= s2) e[4 * t4 + 2] = fmaf(b[s2], tt.z, e[4 * t4 + 2]);
            if (4 * t4 + 3 >= s2) e[4 * t4 + 3] = fmaf(b[s2], tt.w, e[4 * t4 + 3]);
          }
        }
        // e[s2] is complete once every s <= s2 has been added: column t of T2' only has
        // rows s <= t, so after the loop above all of e is final.
#pragma unroll
        for (int s2 = 0; s2 < 16; ++s2) {
#pragma unroll
          for (int t4 = s2 / 4; t4 < 4; ++t4) {
            const float4 hh = reinterpret_cast<const float4*>(Hs + s2 * CP)[t4];
            if (4 * t4 + 0 >= s2) o[4 * t4 + 0] = fmaf(e[s2], hh.x, o[4 * t4 + 0]);
            if (4 * t4 + 1 >= s2) o[4 * t4 + 1] = fmaf(e[s2], hh.y, o[4 * t4 + 1]);
            if (4 * t4 + 2 >= s2) o[4 * t4 + 2] = fmaf(e[s2], hh.z, o[4 * t4 + 2]);
            if (4 * t4 + 3 >= s2) o[4 * t4 + 3] = fmaf(e[s2], hh.w, o[4 * t4 + 3]);
          }
        }
        float* ost = ostage + size_t(c & 1) * C * D;
#pragma unroll
        for (int t = 0; t < 16; ++t) {
          Eps[t * D + g] = e[t];
          ost[t * D + g] = o[t] * inv_den[t];
        }
      }
      fence_async_smem();
      group_bar(2, NG);
      VLA_MARK(5)
      if (g == 0) {
        bulk_store(gout + size_t(c) * C * D, ostage + size_t(c & 1) * C * D,
                   uint32_t(n) * D * sizeof(float));
        bulk_commit();
      }

      // ---- S <- S + E' Z^T
#pragma unroll 2
      for (int s2 = 0; s2 < C; ++s2) {
        float ev[TR];
#pragma unroll
        for (int r4 = 0; r4 < TR / 4; ++r4) {
          const float4 x = reinterpret_cast<const float4*>(Eps + s2 * D + rb * TR)[r4];
          ev[4 * r4 + 0] = x.x; ev[4 * r4 + 1] = x.y; ev[4 * r4 + 2] = x.z; ev[4 * r4 + 3] = x.w;
        }
#pragma unroll
        for (int m = 0; m < NV; ++m) {
          const float4 z4 = reinterpret_cast<const float4*>(Zs + s2 * D)[m * LPR + cg];
          const float2 z01 = make_float2(z4.x, z4.y), z23 = make_float2(z4.z, z4.w);
#pragma unroll
          for (int r = 0; r < TR; ++r) {
            const float2 ee = make_float2(ev[r], ev[r]);
            st[r][2 * m] = ffma2(ee, z01, st[r][2 * m]);
            st[r][2 * m + 1] = ffma2(ee, z23, st[r][2 * m + 1]);
          }
        }
      }
      group_bar(2, NG);
      VLA_MARK(6)
      if (g == 0) mbar_arrive(&ring_empty[slot]);
    }
    // final S and key sum
    if (p.S_T) {
#pragma unroll
      for (int r = 0; r < TR; ++r) {
        const int row = rb * TR + r;
#pragma unroll
        for (int m = 0; m < NV; ++m)
          reinterpret_cast<float4*>(p.S_T + (size_t(unit) * D + row) * D)[m * LPR + cg] =
              make_float4(st[r][2 * m].x, st[r][2 * m].y, st[r][2 * m + 1].x, st[r][2 * m + 1].y);
      }
    }
    if (p.zT) p.zT[size_t(unit) * D + g] = zk;
    if (g == 0) bulk_wait_all<0>();
  }
#ifdef VLA_SECTION_TIMERS
  if (p.dbg && unit == 0 && (g == 0 || g == 32)) {
    long long* d = p.dbg + ((is_A ? 0 : 2) + (g == 32 ? 1 : 0)) * 12;
    for (int i = 0; i < 12; ++i) d[i] = tsec[i];
  }
#endif
}

}  // namespace vla
