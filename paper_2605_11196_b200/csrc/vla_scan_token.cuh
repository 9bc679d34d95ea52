// VLA forward scan, "token" kernel: one CTA per (batch, head) unit, the whole fp32 state
// (S and A) in registers, one pass over the state per token (Section 3.3; Algorithm 1
// without projections and refresh).
//
// Thread (i, j), i = tid/4 in [0, D), j = tid%4: holds, of row i of A and of row i of S,
// the D/4 columns {(4m + j)*4 + e}.  A warp therefore covers 8 rows; the four lanes of a
// row read four consecutive float4 of a token vector (64 contiguous bytes, broadcast over
// the rows), and a row dot product finishes with two xor-shuffles.
//
// Per token (u = k_hat case): one read pass forms z_i = A_{t-1}[i,:].u, p_i = S_{t-1}[i,:].k_hat,
// r_i = S_{t-1}[i,:].q_f; the three scalars u.z, z.z, z.q_f are reduced per warp, exchanged
// through shared memory with ONE CTA barrier, and the update pass applies
// A -= z z^T/delta and S += e alpha^T with alpha = z / max(||z||, eps*delta)  (= A_t k_hat
// normalised, because A_t k_hat = z/delta when u = k_hat).  The readout uses
// S_t q_f = S_{t-1} q_f + e (alpha.q_f), so S is read once and written once per token.
// With an explicit u the write direction is a = A_{t-1}k_hat - z (k_hat.z)/delta and needs a
// second exchange.
//
// q/k/v[/u] arrive in chunks of 16 tokens through a ring of 1-D bulk-async (TMA) copies
// completed on mbarriers; a token-parallel "prep" pass per chunk widens them to fp32 and
// does everything that is off the dependency chain (phi, ||.||, the running key sum and the
// readout denominators).  Outputs are staged in shared memory and leave by bulk store.
#pragma once

#include "vla_common.cuh"

namespace vla {

template <int D, typename TIn, bool HAS_U>
struct TokenCfg {
  static constexpr int NT = 4 * D;        // threads per CTA
  static constexpr int CW = D / 4;        // state columns per thread (of A and of S)
  static constexpr int NV = CW / 4;       // float4 groups per thread
  static constexpr int C = 16;            // tokens per chunk (= NT / (D/4))
  static constexpr int NSTAGE = 3;        // chunks in flight
  static constexpr int NW = NT / 32;      // warps
  static constexpr int NIN = HAS_U ? 4 : 3;
  static constexpr int TOK_LANES = D / 4; // prep: threads per token

  static constexpr size_t raw_bytes = size_t(NSTAGE) * NIN * C * D * sizeof(TIn);
  static constexpr size_t work_floats = size_t(HAS_U ? 5 : 4) * C * D;  // khat, qf, v, kf[, u]
  static constexpr size_t ostage_floats = size_t(2) * C * D;
  static constexpr size_t vec_floats = size_t(4) * D;                   // zbuf[2], abuf[2]
  static constexpr size_t red_floats = size_t(4) * NW * 4;              // red[2][NW], red2[2][NW] (float4)
  static constexpr size_t smem_bytes = raw_bytes +
      (work_floats + ostage_floats + vec_floats + red_floats + C) * sizeof(float) +
      NSTAGE * sizeof(uint64_t) + 128;
};

template <int D, typename TIn, bool HAS_U>
__global__ void __launch_bounds__(4 * D) vla_scan_token_kernel(const ScanParams p) {
  using Cfg = TokenCfg<D, TIn, HAS_U>;
  constexpr int NT = Cfg::NT, NV = Cfg::NV, CW = Cfg::CW, C = Cfg::C, NSTAGE = Cfg::NSTAGE;
  constexpr int NW = Cfg::NW, NIN = Cfg::NIN, TOK_LANES = Cfg::TOK_LANES;
  static_assert(NT / TOK_LANES == C, "one prep item per thread per chunk");

  extern __shared__ __align__(128) unsigned char smem[];
  TIn* raw = reinterpret_cast<TIn*>(smem);
  float* w_khat = reinterpret_cast<float*>(smem + Cfg::raw_bytes);
  float* w_qf = w_khat + C * D;
  float* w_v = w_qf + C * D;
  float* w_kf = w_v + C * D;
  float* w_u = w_kf + C * D;                       // only when HAS_U
  float* ostage = w_khat + Cfg::work_floats;       // [2][C*D]
  float* zbuf = ostage + Cfg::ostage_floats;       // [2][D]
  float* abuf = zbuf + 2 * D;                      // [2][D]
  float4* red = reinterpret_cast<float4*>(abuf + 2 * D);  // [2][NW]
  float4* red2 = red + 2 * NW;                            // [2][NW]
  float* inv_den = reinterpret_cast<float*>(red2 + 2 * NW);  // [C]
  uint64_t* full = reinterpret_cast<uint64_t*>(
      (reinterpret_cast<uintptr_t>(inv_den + C) + 7) & ~uintptr_t(7));  // [NSTAGE]

  const int tid = threadIdx.x;
  const int lane = tid & 31, warp = tid >> 5;
  const int i = tid >> 2, j = tid & 3;
  const int unit = blockIdx.x;
  const int T = p.T;
  const bool ident = (p.flags & VLA_FLAG_IDENTITY_MAP) != 0;
  const bool lin = !HAS_U && (p.flags & VLA_FLAG_LINEAR_ATTENTION) != 0;
  const float eps = p.eps;
  const int nchunks = (T + C - 1) / C;

  const size_t tok_base = token_offset(p, unit, 0, D);   // element offset of this unit's token 0
  const size_t tok_step = token_stride(p, D);            // elements between its tokens
  const TIn* gq = static_cast<const TIn*>(p.q) + tok_base;
  const TIn* gk = static_cast<const TIn*>(p.k) + tok_base;
  const TIn* gv = static_cast<const TIn*>(p.v) + tok_base;
  const TIn* gu = HAS_U ? static_cast<const TIn*>(p.u) + tok_base : nullptr;
  float* gout = p.out + tok_base;

  // ---- ring set-up and the first loads (one elected thread)
  auto issue = [&](int c) {
    const int s = c % NSTAGE;
    const int n = min(C, T - c * C);
    const uint32_t bytes = uint32_t(n) * D * sizeof(TIn);
    TIn* dst = raw + size_t(s) * NIN * C * D;
    const size_t off = size_t(c) * C * tok_step;
    mbar_arrive_expect_tx(&full[s], NIN * bytes);
    bulk_load_rows(dst + 0 * C * D, gq + off, tok_step, n, D, &full[s]);
    bulk_load_rows(dst + 1 * C * D, gk + off, tok_step, n, D, &full[s]);
    bulk_load_rows(dst + 2 * C * D, gv + off, tok_step, n, D, &full[s]);
    if (HAS_U) bulk_load_rows(dst + 3 * C * D, gu + off, tok_step, n, D, &full[s]);
  };
  if (tid == 0) {
    for (int s = 0; s < NSTAGE; ++s) mbar_init(&full[s], 1);
    mbar_init_fence();
  }
  if (tid < C) inv_den[tid] = 1.0f;
  __syncthreads();
  if (tid == 0) {
    for (int c = 0; c < NSTAGE && c < nchunks; ++c) issue(c);
  }

  // ---- a0: state into registers
  float A[CW], S[CW];
  {
    const size_t row = (size_t(unit) * D + i) * D;
#pragma unroll
    for (int m = 0; m < NV; ++m) {
      const int c4 = m * 4 + j;
      float4 a, s;
      if (p.A0) {
        a = reinterpret_cast<const float4*>(p.A0 + row)[c4];
      } else {
        const float dg = 1.0f / p.lambda;
        a.x = (c4 * 4 + 0 == i) ? dg : 0.0f;
        a.y = (c4 * 4 + 1 == i) ? dg : 0.0f;
        a.z = (c4 * 4 + 2 == i) ? dg : 0.0f;
        a.w = (c4 * 4 + 3 == i) ? dg : 0.0f;
      }
      if (p.S0) s = reinterpret_cast<const float4*>(p.S0 + row)[c4];
      else s = make_float4(0.f, 0.f, 0.f, 0.f);
      A[4 * m + 0] = a.x; A[4 * m + 1] = a.y; A[4 * m + 2] = a.z; A[4 * m + 3] = a.w;
      S[4 * m + 0] = s.x; S[4 * m + 1] = s.y; S[4 * m + 2] = s.z; S[4 * m + 3] = s.w;
    }
  }
  float zk = 0.0f;  // running sum of phi(k), column tid (threads tid < D)
  if (tid < D && p.z0) zk = p.z0[size_t(unit) * D + tid];

  const int ptok = tid / TOK_LANES;   // prep: token within the chunk
  const int pc4 = tid % TOK_LANES;    // prep: float4 column group

  for (int c = 0; c < nchunks; ++c) {
    const int s = c % NSTAGE;
    const int n = min(C, T - c * C);
    const bool arrived = mbar_wait_bounded(&full[s], (c / NSTAGE) & 1);
    if (__syncthreads_or(!arrived)) {
      // A bounded wait ran out.  Report, give loads still in flight one more bounded
      // chance to land (they target this CTA's shared memory), drain the stores, leave.
      if (tid == 0) {
        if (p.status) atomicCAS(p.status, 0, int(VLA_ERR_DEVICE_TIMEOUT));
        for (int cc = c; cc < nchunks && cc < c + NSTAGE; ++cc)
          mbar_wait_bounded(&full[cc % NSTAGE], (cc / NSTAGE) & 1);
        bulk_wait_all<0>();
      }
      __syncthreads();
      return;
    }

    // ---- a2: prep, token-parallel (thread = (token ptok, float4 group pc4))
    {
      const TIn* rq = raw + (size_t(s) * NIN + 0) * C * D + ptok * D;
      const TIn* rk = raw + (size_t(s) * NIN + 1) * C * D + ptok * D;
      const TIn* rv = raw + (size_t(s) * NIN + 2) * C * D + ptok * D;
      const bool act = ptok < n;
      float4 kr = make_float4(1.f, 0.f, 0.f, 0.f), qr = kr, vr = kr;
      if (act) { kr = load4(rk, pc4); qr = load4(rq, pc4); vr = load4(rv, pc4); }
      float4 kf = kr, qf = qr;
      if (!ident) {
        kf.x = phi_elu1(kr.x); kf.y = phi_elu1(kr.y); kf.z = phi_elu1(kr.z); kf.w = phi_elu1(kr.w);
        qf.x = phi_elu1(qr.x); qf.y = phi_elu1(qr.y); qf.z = phi_elu1(qr.z); qf.w = phi_elu1(qr.w);
      }
      float ss = kf.x * kf.x + kf.y * kf.y + kf.z * kf.z + kf.w * kf.w;
#pragma unroll
      for (int off = TOK_LANES / 2; off >= 1; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
      // linear-attention mode writes along phi(k) itself: no normalisation
      const float inv = lin ? 1.0f : 1.0f / fmaxf(sqrtf(ss), eps);
      if (act) {
        reinterpret_cast<float4*>(w_khat + ptok * D)[pc4] =
            make_float4(kf.x * inv, kf.y * inv, kf.z * inv, kf.w * inv);
        reinterpret_cast<float4*>(w_qf + ptok * D)[pc4] = qf;
        reinterpret_cast<float4*>(w_v + ptok * D)[pc4] = vr;
        if (!ident) reinterpret_cast<float4*>(w_kf + ptok * D)[pc4] = kf;
        if (HAS_U) {
          const TIn* ru = raw + (size_t(s) * NIN + 3) * C * D + ptok * D;
          reinterpret_cast<float4*>(w_u + ptok * D)[pc4] =
              p.u_is_khat ? make_float4(kf.x * inv, kf.y * inv, kf.z * inv, kf.w * inv)
                          : load4(ru, pc4);
        }
      }
      if (!ident) {
        __syncthreads();
        // running key sum, column-parallel: w_kf[t][col] becomes zkey_t[col]
        if (tid < D) {
          for (int t = 0; t < n; ++t) {
            zk += w_kf[t * D + tid];
            w_kf[t * D + tid] = zk;
          }
        }
        __syncthreads();
        float4 zz = make_float4(0.f, 0.f, 0.f, 0.f);
        if (act) zz = reinterpret_cast<const float4*>(w_kf + ptok * D)[pc4];
        float dd = zz.x * qf.x + zz.y * qf.y + zz.z * qf.z + zz.w * qf.w;
#pragma unroll
        for (int off = TOK_LANES / 2; off >= 1; off >>= 1) dd += __shfl_xor_sync(0xffffffffu, dd, off);
        if (act && pc4 == 0) inv_den[ptok] = 1.0f / fmaxf(dd, eps);
      }
      if (tid == 0) bulk_wait_read<1>();  // the out stage of chunk c-2 has been read
    }
    __syncthreads();
    // raw[s] has been consumed by every thread: refill it
    if (tid == 0 && c + NSTAGE < nchunks) issue(c + NSTAGE);

    float* ost = ostage + size_t(c & 1) * C * D;

    // ---- a3..a8: the per-token chain
    for (int t = 0; t < n; ++t) {
      const int b = t & 1;
      const float* kh = w_khat + t * D;
      const float* qv = w_qf + t * D;
      const float* uv = HAS_U ? (w_u + t * D) : kh;

      float zi0 = 0.f, zi1 = 0.f, pi0 = 0.f, pi1 = 0.f, ri0 = 0.f, ri1 = 0.f, wi0 = 0.f, wi1 = 0.f;
#pragma unroll
      for (int m = 0; m < NV; ++m) {
        const int c4 = m * 4 + j;
        const float4 k4 = reinterpret_cast<const float4*>(kh)[c4];
        const float4 q4 = reinterpret_cast<const float4*>(qv)[c4];
        float4 u4 = k4;
        if (HAS_U) u4 = reinterpret_cast<const float4*>(uv)[c4];
        zi0 = fmaf(A[4 * m + 0], u4.x, zi0); zi1 = fmaf(A[4 * m + 1], u4.y, zi1);
        zi0 = fmaf(A[4 * m + 2], u4.z, zi0); zi1 = fmaf(A[4 * m + 3], u4.w, zi1);
        pi0 = fmaf(S[4 * m + 0], k4.x, pi0); pi1 = fmaf(S[4 * m + 1], k4.y, pi1);
        pi0 = fmaf(S[4 * m + 2], k4.z, pi0); pi1 = fmaf(S[4 * m + 3], k4.w, pi1);
        ri0 = fmaf(S[4 * m + 0], q4.x, ri0); ri1 = fmaf(S[4 * m + 1], q4.y, ri1);
        ri0 = fmaf(S[4 * m + 2], q4.z, ri0); ri1 = fmaf(S[4 * m + 3], q4.w, ri1);
        if (HAS_U) {
          wi0 = fmaf(A[4 * m + 0], k4.x, wi0); wi1 = fmaf(A[4 * m + 1], k4.y, wi1);
          wi0 = fmaf(A[4 * m + 2], k4.z, wi0); wi1 = fmaf(A[4 * m + 3], k4.w, wi1);
        }
      }
      float zi = zi0 + zi1, pi = pi0 + pi1, ri = ri0 + ri1, wi = wi0 + wi1;
      zi += __shfl_xor_sync(0xffffffffu, zi, 1); zi += __shfl_xor_sync(0xffffffffu, zi, 2);
      pi += __shfl_xor_sync(0xffffffffu, pi, 1); pi += __shfl_xor_sync(0xffffffffu, pi, 2);
      ri += __shfl_xor_sync(0xffffffffu, ri, 1); ri += __shfl_xor_sync(0xffffffffu, ri, 2);
      if (HAS_U) { wi += __shfl_xor_sync(0xffffffffu, wi, 1); wi += __shfl_xor_sync(0xffffffffu, wi, 2); }

      const float khi = kh[i], qi = qv[i], vi = w_v[t * D + i];
      const float ui = HAS_U ? uv[i] : khi;
      // Linear attention (Eq. "linear-attn"): the write direction is phi(k_t) itself, which takes
      // z's place in the exchange below (so that t2 = phi(k).phi(q) and the update adds v phi(k)^T)
      if (!HAS_U && lin) zi = khi;

      // warp partials over its 8 rows (each row's value sits on 4 lanes: offsets 4, 8, 16)
      float s0 = ui * zi;                     // u.z
      float s1 = HAS_U ? khi * zi : zi * zi;  // k_hat.z   |  z.z
      float s2 = HAS_U ? 0.0f : zi * qi;      //           |  z.q_f
#pragma unroll
      for (int off = 4; off <= 16; off <<= 1) {
        s0 += __shfl_xor_sync(0xffffffffu, s0, off);
        s1 += __shfl_xor_sync(0xffffffffu, s1, off);
        if (!HAS_U) s2 += __shfl_xor_sync(0xffffffffu, s2, off);
      }
      if (lane == 0) red[b * NW + warp] = make_float4(s0, s1, s2, 0.f);
      if (j == 0) zbuf[b * D + i] = zi;
      __syncthreads();

      float t0 = 0.f, t1 = 0.f, t2 = 0.f;
#pragma unroll
      for (int w = 0; w < NW; ++w) {
        const float4 r = red[b * NW + w];
        t0 += r.x; t1 += r.y; t2 += r.z;
      }
      const float delta = fmaxf(1.0f + t0, eps);  // Algorithm 1's clamp; delta >= 1 for A > 0
      const float inv_d = 1.0f / delta;
      const float ei = lin ? vi : vi - pi;        // e = v - S_{t-1} k_hat (linear attention: no residual)
      const float zs = lin ? 0.0f : zi * inv_d;   // (linear attention: A is not touched)
      float es, oi;
      const float* wvec;                          // direction alpha is proportional to
      if (!HAS_U) {
        // A_t k_hat = z/delta; alpha = (z/delta) / max(||z||/delta, eps)
        const float nz = sqrtf(t1);
        const float sc = lin ? 1.0f : inv_d / fmaxf(nz * inv_d, eps);
        es = ei * sc;
        oi = (ri + ei * (t2 * sc)) * inv_den[t];
        wvec = zbuf + b * D;
        // fmaxf drops a NaN operand, so the raw sums are tested, not delta or sc
        if ((p.flags & VLA_FLAG_CHECK_FINITE) && tid == 0 && p.status &&
            !isfinite(t0 + t1 + t2))
          atomicCAS(p.status, 0, int(VLA_ERR_NONFINITE));
      } else {
        // a = A_t k_hat = A_{t-1} k_hat - z (k_hat.z)/delta  (+ eta k_hat on a refresh step)
        float ai = fmaf(-zi, t1 * inv_d, wi);
        const bool refresh_now = p.refresh_period > 0 &&
            (p.step_offset + (long long)c * C + t + 1) % p.refresh_period == 0;
        if (refresh_now) ai = fmaf(p.refresh_eta, khi, ai);
        float a0 = ai * ai, a1 = ai * qi;
#pragma unroll
        for (int off = 4; off <= 16; off <<= 1) {
          a0 += __shfl_xor_sync(0xffffffffu, a0, off);
          a1 += __shfl_xor_sync(0xffffffffu, a1, off);
        }
        if (lane == 0) red2[b * NW + warp] = make_float4(a0, a1, 0.f, 0.f);
        if (j == 0) abuf[b * D + i] = ai;
        __syncthreads();
        float aa = 0.f, aq = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) {
          const float4 r = red2[b * NW + w];
          aa += r.x; aq += r.y;
        }
        const float sc = 1.0f / fmaxf(sqrtf(aa), eps);
        es = ei * sc;
        oi = (ri + ei * (aq * sc)) * inv_den[t];
        wvec = abuf + b * D;
        if ((p.flags & VLA_FLAG_CHECK_FINITE) && tid == 0 && p.status &&
            !isfinite(t0 + t1 + aa + aq))
          atomicCAS(p.status, 0, int(VLA_ERR_NONFINITE));
      }
      const float* zvec = zbuf + b * D;
      // Algorithm 1's periodic refresh: A += eta I right after the rank-1 downdate
      const float diag_add = (HAS_U && p.refresh_period > 0 &&
                              (p.step_offset + (long long)c * C + t + 1) % p.refresh_period == 0)
                                 ? p.refresh_eta : 0.0f;
#pragma unroll
      for (int m = 0; m < NV; ++m) {
        const int c4 = m * 4 + j;
        const float4 z4 = reinterpret_cast<const float4*>(zvec)[c4];
        float4 a4 = z4;
        if (HAS_U) a4 = reinterpret_cast<const float4*>(wvec)[c4];
        A[4 * m + 0] = fmaf(-zs, z4.x, A[4 * m + 0]); A[4 * m + 1] = fmaf(-zs, z4.y, A[4 * m + 1]);
        A[4 * m + 2] = fmaf(-zs, z4.z, A[4 * m + 2]); A[4 * m + 3] = fmaf(-zs, z4.w, A[4 * m + 3]);
        if (HAS_U) {
          A[4 * m + 0] += (c4 * 4 + 0 == i) ? diag_add : 0.0f;
          A[4 * m + 1] += (c4 * 4 + 1 == i) ? diag_add : 0.0f;
          A[4 * m + 2] += (c4 * 4 + 2 == i) ? diag_add : 0.0f;
          A[4 * m + 3] += (c4 * 4 + 3 == i) ? diag_add : 0.0f;
        }
        S[4 * m + 0] = fmaf(es, a4.x, S[4 * m + 0]); S[4 * m + 1] = fmaf(es, a4.y, S[4 * m + 1]);
        S[4 * m + 2] = fmaf(es, a4.z, S[4 * m + 2]); S[4 * m + 3] = fmaf(es, a4.w, S[4 * m + 3]);
      }
      if (j == 0) ost[t * D + i] = oi;
    }

    // ---- a9: this chunk's outputs leave by bulk store
    fence_async_smem();
    __syncthreads();
    if (tid == 0) {
      bulk_store_rows(gout + size_t(c) * C * tok_step, ost, tok_step, n, D);
      bulk_commit();
    }
  }

  // ---- final states
  {
    const size_t row = (size_t(unit) * D + i) * D;
#pragma unroll
    for (int m = 0; m < NV; ++m) {
      const int c4 = m * 4 + j;
      if (p.A_T)
        reinterpret_cast<float4*>(p.A_T + row)[c4] =
            make_float4(A[4 * m + 0], A[4 * m + 1], A[4 * m + 2], A[4 * m + 3]);
      if (p.S_T)
        reinterpret_cast<float4*>(p.S_T + row)[c4] =
            make_float4(S[4 * m + 0], S[4 * m + 1], S[4 * m + 2], S[4 * m + 3]);
    }
    if (tid < D && p.zT) p.zT[size_t(unit) * D + tid] = zk;
  }
  if (tid == 0) bulk_wait_all<0>();
}

}  // namespace vla
