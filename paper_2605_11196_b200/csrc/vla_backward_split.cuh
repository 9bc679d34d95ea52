// VLA backward pass as two reverse scans, run as one launch (u = k_hat; with the template flag UX
// the general path: explicit penalty directions u and / or the periodic refresh; d in {32, 64, 128}).
//
// The adjoint of the memory state, GS = dL/dS, obeys a recurrence of its own that never looks at
// the penalty side: GS_{t-1} = GS_t + dy qf^T - de k_hat^T.  So the reverse sweep splits into
//
//   S side (vla_backward_s_body): S and GS in registers.  Per token: dq, dv, and three
//     vectors for the other side: dalpha_t = dL/d alpha_t, the S-side part of dL/d k_hat_t, and
//     the running gradient of the key sum.
//   A side (vla_backward_a_body): A and GA = dL/dA in registers.  Per token it turns dalpha_t
//     into da, forms dz, ddelta and the remaining parts of dL/d k_hat_t, and writes dk.  It
//     carries the symmetric part of GA only; dA0 is formed afterwards (vla_backward_da0_kernel).
//
// each a CTA per unit holding TWO d x d matrices in registers, as R x RC blocks on a grid of
// 16 x TX threads (R = d / 16 rows, RC = d / TX columns; TX = 16, or 32 at d = 128, where the
// blocks of a 16-wide grid would leave no registers for the helper warps).  The blocks are kept
// as column pairs and every product with them is a packed fma.rn.f32x2.  The forward
// recurrence is not re-run here: the chunk kernel leaves z_t, e_t, delta_t (a_t on the general
// path), its readout o_t, the key sum after every 16 tokens and the final S, A, key sum in the
// workspace, and both sweeps walk the states back by undoing the rank-1 updates
// (S_{t-1} = S_t - e alpha^T, A_{t-1} = A_t + z z^T / delta).  Formulas per token: see
// vla_backward.cuh.  vla_backward_sa_kernel (end of this file) runs the S side and the A side
// of every unit as CTAs of one launch, the A side following the S side through a progress word.
//
// Both sides keep a ring of four per-token contexts in shared memory.  Opening a token
// (loading its rows, alpha, denominators: nothing that depends on the adjoints) and closing one
// (vector arithmetic on finished products, the stores) are done by helper warps off the path
// of the TX / 2 matrix warps; one CTA barrier per token.
#pragma once

#include "vla_backward.cuh"

namespace vla {

// Thread grid of the two reverse scans.
template <int D>
struct BwdSplitGeom {
  static constexpr int TX = D >= 128 ? 32 : 16;   // threads along a matrix row
  static constexpr int R = D / 16;                // rows of a thread's block
  static constexpr int RC = D / TX;               // columns of a thread's block
  static constexpr int NW = TX / 2;               // matrix warps
  static constexpr int NCLOSE = D >= 128 ? 2 : 1; // warps closing tokens on the S side (the sums over NW partials)
  static constexpr int NT_S = (NW + NCLOSE + 1) * 32;   // S side: matrix warps, closers, one opener
  static constexpr int NT_A = (NW + 2) * 32;            // A side: matrix warps, one closer, one opener
  static constexpr int MINB = D == 64 ? 3 : D == 32 ? 4 : 1;   // CTAs per SM the register budget is held to
};

// Dynamic shared memory of the two reverse scans (the kernels assert these against their layouts).
template <int D>
struct BackwardSplitSmem {
  static constexpr int NW = BwdSplitGeom<D>::NW;
  static constexpr size_t s_bytes = sizeof(float) * (4 * 8 * D + 4 * 4 + 3 * 1 * D + 2 * NW * 3 * D + D);
  static constexpr size_t a_bytes = sizeof(float) * (4 * 7 * D + 4 * 8 + 3 * 3 * D);
  // one launch for both sides: the larger layout plus the word the CTA's ticket travels through
  static constexpr size_t sa_bytes = (s_bytes > a_bytes ? s_bytes : a_bytes) + 16;
};

// The n threads that take part in this CTA's role, whichever loop they are in.
__device__ __forceinline__ void cta_sync(int n) { asm volatile("bar.sync 0, %0;" ::"r"(n) : "memory"); }

// progress of a unit's S side, read by its A side (another CTA of the same launch)
__device__ __forceinline__ void bwd_publish(int* p, int v) {
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ int bwd_observe(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

__device__ __forceinline__ float2 bwd_ffma2(float2 a, float2 b, float2 c) {
  uint64_t ra, rb, rc, rd;
  asm("mov.b64 %0, {%1, %2};" : "=l"(ra) : "f"(a.x), "f"(a.y));
  asm("mov.b64 %0, {%1, %2};" : "=l"(rb) : "f"(b.x), "f"(b.y));
  asm("mov.b64 %0, {%1, %2};" : "=l"(rc) : "f"(c.x), "f"(c.y));
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(rd) : "l"(ra), "l"(rb), "l"(rc));
  float2 d;
  asm("mov.b64 {%0, %1}, %2;" : "=f"(d.x), "=f"(d.y) : "l"(rd));
  return d;
}

// N consecutive fp32 values moved as one access (N = 1, 2, 4, 8; 8 as two of 4)
template <int N>
struct alignas(N >= 4 ? 16 : 4 * N) BwdVec { float v[N]; };
template <int N>
__device__ __forceinline__ void bwd_ld(const float* p, float (&out)[N]) {
  if constexpr (N > 4) {
#pragma unroll
    for (int i = 0; i < N / 4; ++i) {
      const BwdVec<4> x = reinterpret_cast<const BwdVec<4>*>(p)[i];
#pragma unroll
      for (int j = 0; j < 4; ++j) out[4 * i + j] = x.v[j];
    }
  } else {
    const BwdVec<N> x = *reinterpret_cast<const BwdVec<N>*>(p);
#pragma unroll
    for (int j = 0; j < N; ++j) out[j] = x.v[j];
  }
}
template <int N>
__device__ __forceinline__ void bwd_st(float* p, const float (&in)[N]) {
  static_assert(N <= 4, "one access");
  BwdVec<N> x;
#pragma unroll
  for (int j = 0; j < N; ++j) x.v[j] = in[j];
  *reinterpret_cast<BwdVec<N>*>(p) = x;
}
// N consecutive input values (fp32 or bf16 bits) widened to fp32
template <int N>
__device__ __forceinline__ void bwd_ld_in(const float* p, float (&out)[N]) { bwd_ld<N>(p, out); }
template <int N>
__device__ __forceinline__ void bwd_ld_in(const uint16_t* p, float (&out)[N]) {
  struct alignas(2 * N) H { uint16_t v[N]; };
  const H x = *reinterpret_cast<const H*>(p);
#pragma unroll
  for (int j = 0; j < N; ++j) out[j] = __uint_as_float(uint32_t(x.v[j]) << 16);
}

// Element offset of token t of a unit in the caller's sequence tensors (q, k, u, d_out and the
// gradients of q, k, v, u): [B, H, T, d], or [B, T, H, d] with VLA_FLAG_TOKEN_MAJOR.  The
// workspace vectors are always [units, T, d].
__device__ __forceinline__ size_t bwd_user_row(const BackwardSplitParams& p, int unit, int t, int D) {
  if (p.flags & VLA_FLAG_TOKEN_MAJOR) {
    const int b = unit / p.heads, h = unit - b * p.heads;
    return ((size_t(b) * size_t(p.T) + size_t(t)) * size_t(p.heads) + size_t(h)) * D;
  }
  return (size_t(unit) * size_t(p.T) + size_t(t)) * D;
}

// Sums of N per-thread values over the 2*OFF lanes of a row group, by halving: at each step a
// lane hands the half of its values that its partner keeps, so N values cost N - 1 shuffles
// (plus log2(lanes / N) for the last one) instead of N log2(lanes).  Afterwards v[0] of lane l
// of the group is the total of value number l / (lanes / N).
template <int N, int OFF>
__device__ __forceinline__ void rows_reduce(float* v, int lane) {
  if constexpr (N > 1) {
    constexpr int h = N / 2;
    const bool up = (lane & OFF) != 0;
#pragma unroll
    for (int i = 0; i < h; ++i) {
      const float send = up ? v[i] : v[i + h];
      const float keep = up ? v[i + h] : v[i];
      v[i] = keep + __shfl_xor_sync(0xffffffffu, send, OFF);
    }
    rows_reduce<h, OFF / 2>(v, lane);
  } else if constexpr (OFF >= 1) {
    v[0] += __shfl_xor_sync(0xffffffffu, v[0], OFF);
    rows_reduce<1, OFF / 2>(v, lane);
  }
}

// ------------------------------------------------------------------------------ S side
// UX: explicit penalty directions.  The S side only sees them through alpha_t, which then comes
// from the stashed a_t = A_t k_hat_t instead of z_t / delta_t.
template <int D, typename TIn, bool UX>
__device__ __forceinline__ void vla_backward_s_body(const BackwardSplitParams& p, const int unit,
                                                    unsigned char* smem_raw) {
  using G = BwdSplitGeom<D>;
  constexpr int R = G::R, RC = G::RC, TX = G::TX, NW = G::NW, NT = G::NT_S, NCLOSE = G::NCLOSE;
  constexpr int RP = RC / 2;          // column pairs of a block
  constexpr int EPL = D / 32;         // consecutive vector elements per lane of a helper warp
  constexpr int NCTX = 4;
  enum { cKf = 0, cKh, cQf, cGo, cDy, cEt, cAl, cZk, NV };
  enum { sDen = 0, sDenLive, sQal, sOdo };
  struct Smem {
    float ctx[NCTX][NV][D];
    float cscl[NCTX][4];
    float rowv[3][1][D];       // g1 = GS alpha, ring of three tokens
    float part[2][NW][3][D];   // column-sum partials by token parity and warp
    float gz[D];               // dL/d(key sum), carried by the closing warp
  };
  static_assert(sizeof(Smem) == BackwardSplitSmem<D>::s_bytes, "shared memory size of the S side");
  Smem& sm = *reinterpret_cast<Smem*>(smem_raw);
  auto& ctx = sm.ctx; auto& cscl = sm.cscl; auto& rowv = sm.rowv; auto& part = sm.part; auto& gz = sm.gz;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int ty = tid / TX, tx = tid % TX;
  const int row0 = ty * R, col0 = tx * RC;
  const int c0 = lane * EPL;          // first vector element of this lane in a helper warp
  const bool ident = (p.flags & VLA_FLAG_IDENTITY_MAP) != 0;
  const float eps = p.eps;
  const int T = p.T;
  const size_t ubase = size_t(unit) * size_t(T) * D;
  const TIn* gq = static_cast<const TIn*>(p.q);      // caller's tensors: rows through bwd_user_row
  const TIn* gk = static_cast<const TIn*>(p.k);
  const float* gdo = p.d_out;
  const float* zst = (UX ? p.ast : p.zst) + ubase;   // the vector alpha_t is parallel to
  const float* est = p.est + ubase;
  const float* dst = p.dst + size_t(unit) * T;

  for (int j = tid; j < D; j += NT) gz[j] = p.dz_T ? p.dz_T[size_t(unit) * D + j] : 0.0f;

  auto cvec = [&](int t, int which) { return ctx[t & (NCTX - 1)][which]; };
  // after rows_reduce<R, TX / 2> a lane holds the total of row myrow of its group's R rows
  const int myrow = tx / (TX / R);
  const bool row_writer = (tx % (TX / R)) == 0;
  constexpr int kCloser = NW, kOpener = NW + NCLOSE;   // warps kCloser .. kOpener - 1 close tokens

  // Segment t (one CTA barrier): the matrix warps take the column sums and the two rank-1
  // updates of token t, then the row dots of token t - 1; the closing warp finishes token
  // t + 1 and the opening warp prepares token t - 2.  The roles run loops of their own with
  // the same number of barriers, so that staging registers and matrix blocks never share a thread.
  if (warp == kOpener) {
    // rows come from global memory one segment before they are opened
    float pk[EPL], pq[EPL], pz[EPL], pe[EPL], pg[EPL], po[EPL];
    float pdelta = 1.0f;
    auto fetch_token = [&](int t) {
      if (t < 0) return;
      pdelta = dst[t];
      const size_t o = size_t(t) * D + c0;
      const size_t uo = bwd_user_row(p, unit, t, D) + c0;
      bwd_ld_in<EPL>(gk + uo, pk);
      bwd_ld_in<EPL>(gq + uo, pq);
      bwd_ld<EPL>(zst + o, pz);
      bwd_ld<EPL>(est + o, pe);
      bwd_ld<EPL>(gdo + uo, pg);
      bwd_ld<EPL>(p.ost + uo, po);   // the forward's readout o_t (laid out like the caller's tensors)
    };
    // the key sum seen by token t: from the forward's checkpoint at the last token of each group
    // of 16, else walked back one token from t + 1 (at most 15 subtractions from a checkpoint)
    const int nck = (T + 15) / 16;
    auto open_token = [&](int t) {
      const bool last = t == T - 1 || (t & 15) == 15;
      float kx[EPL], qx[EPL], khx[EPL], alx[EPL], zkx[EPL], dyx[EPL];
      float ss = 0.f, zz = 0.f, og = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        float kk = pk[e], qq = pq[e];
        if (!ident) { kk = bwd_phi(kk); qq = bwd_phi(qq); }
        kx[e] = kk; qx[e] = qq;
        ss = fmaf(kk, kk, ss);
        zz = fmaf(pz[e], pz[e], zz);
        og = fmaf(po[e], pg[e], og);
      }
      if (ident) {
#pragma unroll
        for (int e = 0; e < EPL; ++e) zkx[e] = 0.0f;   // not used: o = S q has no denominator
      } else if (last) {
        bwd_ld<EPL>(p.zkc + (size_t(unit) * nck + size_t(t >> 4)) * D + c0, zkx);
      } else {
        float nz[EPL], nk2[EPL];
        bwd_ld<EPL>(cvec(t + 1, cZk) + c0, nz);
        bwd_ld<EPL>(cvec(t + 1, cKf) + c0, nk2);
#pragma unroll
        for (int e = 0; e < EPL; ++e) zkx[e] = nz[e] - nk2[e];
      }
      // This warp sets the pace of the CTA (its token takes 2700 of the 2800 clk a token takes at
      // d = 128): all five sums go through the shuffles together, and the reciprocals and square
      // roots are the hardware estimates plus one Newton step, as in the forward kernels.
      float dn = 0.f, qz = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        dn = fmaf(zkx[e], qx[e], dn);
        qz = fmaf(qx[e], pz[e], qz);
      }
#pragma unroll
      for (int off = 16; off >= 1; off >>= 1) {
        ss += __shfl_xor_sync(0xffffffffu, ss, off);
        zz += __shfl_xor_sync(0xffffffffu, zz, off);
        og += __shfl_xor_sync(0xffffffffu, og, off);
        dn += __shfl_xor_sync(0xffffffffu, dn, off);
        qz += __shfl_xor_sync(0xffffffffu, qz, off);
      }
      const float ink = rcp_nr(fmaxf(sqrt_approx(ss), eps));
      const float idl = rcp_nr(pdelta);
      const float sc = UX ? rcp_nr(fmaxf(sqrt_approx(zz), eps)) : idl * rcp_nr(fmaxf(sqrt_approx(zz) * idl, eps));
      const float qa = sc * qz;      // qf . alpha
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        khx[e] = kx[e] * ink;
        alx[e] = sc * pz[e];
      }
      const float den = ident ? 1.0f : fmaxf(dn, eps);
      const float iden = rcp_nr(den);
#pragma unroll
      for (int e = 0; e < EPL; ++e) dyx[e] = pg[e] * iden;
      bwd_st<EPL>(cvec(t, cKf) + c0, kx);
      bwd_st<EPL>(cvec(t, cKh) + c0, khx);
      bwd_st<EPL>(cvec(t, cQf) + c0, qx);
      bwd_st<EPL>(cvec(t, cGo) + c0, pg);
      bwd_st<EPL>(cvec(t, cDy) + c0, dyx);
      bwd_st<EPL>(cvec(t, cEt) + c0, pe);
      bwd_st<EPL>(cvec(t, cAl) + c0, alx);
      bwd_st<EPL>(cvec(t, cZk) + c0, zkx);
      if (lane == 0) {
        float* os = cscl[t & (NCTX - 1)];
        os[sDen] = den;
        os[sDenLive] = (ident || dn < eps) ? 0.0f : 1.0f;
        os[sQal] = qa;
        os[sOdo] = og;   // o_t . dO_t: with S_t qf_t = den_t o_t it gives dden without the product S_t qf_t
      }
      __syncwarp();   // the next token opened reads this one's key sum and keys
    };
    if (T > 0) {
      fetch_token(T - 1);
      open_token(T - 1);
      fetch_token(T - 2);
      if (T >= 2) open_token(T - 2);
      fetch_token(T - 3);
    }
    cta_sync(NT);
    cta_sync(NT);
    for (int t = T - 1; t >= 0; --t) {
      if (t - 2 >= 0) {
        open_token(t - 2);
        fetch_token(t - 3);
      }
      cta_sync(NT);
    }
  } else if (warp >= kCloser) {
    // The vector results of token t from its finished products.  The query part (dq, the
    // gradient of the key sum) and the key part (dv, dalpha, dk_hat) share nothing but their
    // inputs: one warp does both, or one warp each.
    const bool do_q = NCLOSE == 1 || warp == kCloser;
    const bool do_k = NCLOSE == 1 || warp == kCloser + 1;
    auto close_token = [&](int t) {
      const int par = t & 1;
      const size_t tb = ubase + size_t(t) * D + c0;          // workspace vectors
      const size_t ub = bwd_user_row(p, unit, t, D) + c0;    // the caller's gradients
      if (do_q) {
        float qf[EPL], zkt[EPL], c1[EPL];
        const float den = cscl[t & (NCTX - 1)][sDen];
        const bool den_live = cscl[t & (NCTX - 1)][sDenLive] != 0.0f;
        const float og = cscl[t & (NCTX - 1)][sOdo];
#pragma unroll
        for (int e = 0; e < EPL; ++e) c1[e] = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) {
          float x1[EPL];
          bwd_ld<EPL>(part[par][w][0] + c0, x1);
#pragma unroll
          for (int e = 0; e < EPL; ++e) c1[e] += x1[e];
        }
        bwd_ld<EPL>(cvec(t, cQf) + c0, qf);
        bwd_ld<EPL>(cvec(t, cZk) + c0, zkt);
        const float dden = den_live ? -og * rcp_nr(den) : 0.0f;   // -(S_t qf . dO) / den^2 with S_t qf = den o_t
        float gzc[EPL], dq[EPL], gzo[EPL];
        bwd_ld<EPL>(gz + c0, gzc);
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
          dq[e] = fmaf(dden, zkt[e], c1[e]);
          if (!ident) {
            dq[e] *= qf[e] > 1.0f ? 1.0f : qf[e];     // phi'(q) from phi(q)
            gzc[e] = fmaf(dden, qf[e], gzc[e]);
          }
          gzo[e] = ident ? 0.0f : gzc[e];
        }
        if (!ident) bwd_st<EPL>(gz + c0, gzc);
        bwd_st<EPL>(p.dq + ub, dq);
        bwd_st<EPL>(p.gzt + tb, gzo);
      }
      if (do_k) {
        float dy[EPL], et[EPL], al[EPL], qf[EPL], g1[EPL], dex[EPL], c2[EPL], c3[EPL];
        bwd_ld<EPL>(cvec(t, cDy) + c0, dy);
        bwd_ld<EPL>(cvec(t, cEt) + c0, et);
        bwd_ld<EPL>(rowv[t % 3][0] + c0, g1);
        const float qal = cscl[t & (NCTX - 1)][sQal];
        float ede = 0.f, dye = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
          dex[e] = fmaf(dy[e], qal, g1[e]);
          ede = fmaf(et[e], dex[e], ede);
          dye = fmaf(dy[e], et[e], dye);
          c2[e] = 0.f; c3[e] = 0.f;
        }
#pragma unroll
        for (int w = 0; w < NW; ++w) {
          float x2[EPL], x3[EPL];
          bwd_ld<EPL>(part[par][w][1] + c0, x2);
          bwd_ld<EPL>(part[par][w][2] + c0, x3);
#pragma unroll
          for (int e = 0; e < EPL; ++e) { c2[e] += x2[e]; c3[e] += x3[e]; }
        }
        bwd_ld<EPL>(cvec(t, cAl) + c0, al);
        bwd_ld<EPL>(cvec(t, cQf) + c0, qf);
        ede = warp_sum(ede); dye = warp_sum(dye);
        float dalo[EPL], dko[EPL];
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
          dalo[e] = fmaf(qf[e], dye, c2[e]);          // (GS + dy qf^T)^T e
          dko[e] = -(c3[e] - al[e] * ede);            // -(S' - e alpha^T)^T de
        }
        bwd_st<EPL>(p.dv + ub, dex);
        bwd_st<EPL>(p.dal + tb, dalo);
        bwd_st<EPL>(p.dkS + tb, dko);
      }
    };
    cta_sync(NT);
    cta_sync(NT);
    for (int t = T - 1; t >= 0; --t) {
      // tokens >= t + 2 were closed (by both closing warps) before the last barrier: tell the
      // unit's A side every eighth token
      const int done = T - (t + 2);
      if (warp == kCloser && lane == 0 && done > 0 && (done & 7) == 0) bwd_publish(p.progress + unit, done);
      if (t + 1 <= T - 1) close_token(t + 1);
      cta_sync(NT);
    }
    if (T > 0) close_token(0);
  } else {
    float2 S[R][RP], GS[R][RP];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const size_t idx = (size_t(unit) * D + row0 + r) * D + col0;
      float sv[RC], gv[RC];
      bwd_ld<RC>(p.ST + idx, sv);
      if (p.dS_T) {
        bwd_ld<RC>(p.dS_T + idx, gv);
      } else {
#pragma unroll
        for (int c = 0; c < RC; ++c) gv[c] = 0.0f;
      }
#pragma unroll
      for (int m = 0; m < RP; ++m) {
        S[r][m] = make_float2(sv[2 * m], sv[2 * m + 1]);
        GS[r][m] = make_float2(gv[2 * m], gv[2 * m + 1]);
      }
    }
    auto row_dots = [&](int t) {   // g1 = GS alpha of token t
      float av[RC];
      bwd_ld<RC>(cvec(t, cAl) + col0, av);
      float a1[R];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        float2 x1 = make_float2(0.f, 0.f);
#pragma unroll
        for (int m = 0; m < RP; ++m) x1 = bwd_ffma2(GS[r][m], make_float2(av[2 * m], av[2 * m + 1]), x1);
        a1[r] = x1.x + x1.y;
      }
      rows_reduce<R, TX / 2>(a1, lane);
      if (row_writer) rowv[t % 3][0][row0 + myrow] = a1[0];
    };
    cta_sync(NT);
    if (T > 0) row_dots(T - 1);
    cta_sync(NT);
    for (int t = T - 1; t >= 0; --t) {
      const float qal = cscl[t & (NCTX - 1)][sQal];
      constexpr int RG = R >= 4 ? 4 : R;   // rows in hand at a time: their scalars are reloaded, not kept
      float2 cc[3][RP];
#pragma unroll
      for (int m = 0; m < RP; ++m) { cc[0][m] = make_float2(0.f, 0.f); cc[1][m] = cc[0][m]; cc[2][m] = cc[0][m]; }
#pragma unroll
      for (int rg = 0; rg < R / RG; ++rg) {
        float dyr[RG], der[RG], etr[RG];
        bwd_ld<RG>(cvec(t, cDy) + row0 + rg * RG, dyr);
        bwd_ld<RG>(rowv[t % 3][0] + row0 + rg * RG, der);
        bwd_ld<RG>(cvec(t, cEt) + row0 + rg * RG, etr);
#pragma unroll
        for (int i = 0; i < RG; ++i) {
          const int r = rg * RG + i;
          const float de = fmaf(dyr[i], qal, der[i]);      // (GS + dy qf^T) alpha
          const float2 d2 = make_float2(dyr[i], dyr[i]), e2 = make_float2(etr[i], etr[i]);
          const float2 r2 = make_float2(de, de);
#pragma unroll
          for (int m = 0; m < RP; ++m) {
            cc[0][m] = bwd_ffma2(S[r][m], d2, cc[0][m]);
            cc[1][m] = bwd_ffma2(GS[r][m], e2, cc[1][m]);
            cc[2][m] = bwd_ffma2(S[r][m], r2, cc[2][m]);
          }
        }
      }
      if constexpr (TX == 16) {
        // two thread rows per warp: each half keeps half of the columns of the pair's sum
        constexpr int HC = RC / 2;
        const bool up = (lane & 16) != 0;
#pragma unroll
        for (int k2 = 0; k2 < 3; ++k2) {
          float f[RC], o[HC];
#pragma unroll
          for (int m = 0; m < RP; ++m) { f[2 * m] = cc[k2][m].x; f[2 * m + 1] = cc[k2][m].y; }
#pragma unroll
          for (int c = 0; c < HC; ++c) {
            const float send = up ? f[c] : f[c + HC];
            const float keep = up ? f[c + HC] : f[c];
            o[c] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
          }
          bwd_st<HC>(part[t & 1][warp][k2] + col0 + (up ? HC : 0), o);
        }
      } else {
#pragma unroll
        for (int k2 = 0; k2 < 3; ++k2) {
          float f[RC];
#pragma unroll
          for (int m = 0; m < RP; ++m) { f[2 * m] = cc[k2][m].x; f[2 * m + 1] = cc[k2][m].y; }
          bwd_st<RC>(part[t & 1][warp][k2] + col0, f);
        }
      }
      float qv[RC], kv[RC], av[RC];
      bwd_ld<RC>(cvec(t, cQf) + col0, qv);
      bwd_ld<RC>(cvec(t, cKh) + col0, kv);
      bwd_ld<RC>(cvec(t, cAl) + col0, av);
#pragma unroll
      for (int rg = 0; rg < R / RG; ++rg) {
        float dyr[RG], der[RG], etr[RG];
        bwd_ld<RG>(cvec(t, cDy) + row0 + rg * RG, dyr);
        bwd_ld<RG>(rowv[t % 3][0] + row0 + rg * RG, der);
        bwd_ld<RG>(cvec(t, cEt) + row0 + rg * RG, etr);
#pragma unroll
        for (int i = 0; i < RG; ++i) {
          const int r = rg * RG + i;
          const float de = fmaf(dyr[i], qal, der[i]);
          const float2 d2 = make_float2(dyr[i], dyr[i]), e2 = make_float2(-etr[i], -etr[i]);
          const float2 r2 = make_float2(-de, -de);
#pragma unroll
          for (int m = 0; m < RP; ++m) {
            GS[r][m] = bwd_ffma2(d2, make_float2(qv[2 * m], qv[2 * m + 1]), GS[r][m]);
            GS[r][m] = bwd_ffma2(r2, make_float2(kv[2 * m], kv[2 * m + 1]), GS[r][m]);
            S[r][m] = bwd_ffma2(e2, make_float2(av[2 * m], av[2 * m + 1]), S[r][m]);
          }
        }
      }
      if (t >= 1) row_dots(t - 1);
      cta_sync(NT);
    }
    if (p.dS0) {
#pragma unroll
      for (int r = 0; r < R; ++r) {
        float gv[RC];
#pragma unroll
        for (int m = 0; m < RP; ++m) { gv[2 * m] = GS[r][m].x; gv[2 * m + 1] = GS[r][m].y; }
        bwd_st<RC>(p.dS0 + (size_t(unit) * D + row0 + r) * D + col0, gv);
      }
    }
  }
  cta_sync(NT);
  if (tid == 0) bwd_publish(p.progress + unit, T);   // every token's vectors are out
  if (p.dz0)
    for (int j = tid; j < D; j += NT) p.dz0[size_t(unit) * D + j] = gz[j];
}

// ------------------------------------------------------------------------------ A side
// GA enters the sweep only through (GA + GA^T) z and z^T GA z, so the kernel carries the
// symmetric part GAs = (GA + GA^T) / 2: both products become row dots of one matrix (no column
// sums, nothing to combine across warps), and the update GA += w k_hat^T, w = da + dz, becomes
// GAs += (w k_hat^T + k_hat w^T) / 2.  GA itself is needed for dA0 alone and is linear in the
// w_t: dA0 = dA_T + sum_t w_t k_hat_t^T, formed from the stored w_t by vla_backward_da0_kernel.
//
// UX (explicit u): z = A_{t-1} u, delta = 1 + u.z, a = A_t k_hat.  The adjoint of z then flows to
// u instead of k_hat: dz = ddelta u - (daz k_hat + 2 g + khz da) / delta, du = ddelta z + A_{t-1} dz,
// dk_hat = (S part) + A_t da, and the update is GAs += sym(da k_hat^T) + sym(dz u^T);
// dA0 = dA_T + sum_t (da_t k_hat_t^T + dz_t u_t^T).
template <int D, typename TIn, bool UX>
__device__ __forceinline__ void vla_backward_a_body(const BackwardSplitParams& p, const int unit,
                                                    unsigned char* smem_raw) {
  using G = BwdSplitGeom<D>;
  constexpr int R = G::R, RC = G::RC, TX = G::TX, NW = G::NW;
  constexpr int RP = RC / 2;
  constexpr int EPL = D / 32;
  constexpr int NCTX = 4;
  enum { cKf = 0, cKh, cZt, cDa, cDkS, cGz, cU, NV };
  enum { sDelta = 0, sKhz, sDaz, sNk, sUz };
  struct Smem {
    float ctx[NCTX][NV][D];
    float cscl[NCTX][8];
    float rowv[3][3][D];      // g = GAs z, r1 = A' da, r3 = A' dz, ring of three tokens
  };
  static_assert(sizeof(Smem) == BackwardSplitSmem<D>::a_bytes, "shared memory size of the A side");
  Smem& sm = *reinterpret_cast<Smem*>(smem_raw);
  auto& ctx = sm.ctx; auto& cscl = sm.cscl; auto& rowv = sm.rowv;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int NT = G::NT_A;
  if (tid >= NT) return;   // the launch is sized for the S side, which has one more warp at d = 128
  const int ty = tid / TX, tx = tid % TX;
  const int row0 = ty * R, col0 = tx * RC;
  const int c0 = lane * EPL;
  const bool ident = (p.flags & VLA_FLAG_IDENTITY_MAP) != 0;
  const float eps = p.eps;
  const int T = p.T;
  const size_t ubase = size_t(unit) * size_t(T) * D;
  const TIn* gk = static_cast<const TIn*>(p.k);      // caller's tensors: rows through bwd_user_row
  // general path without a u tensor (the periodic refresh alone): u = k_hat, formed here
  const TIn* gu = (UX && p.u) ? static_cast<const TIn*>(p.u) : nullptr;
  // Algorithm 1's refresh: A_t = (Sherman-Morrison step) + eta I at every refresh_period-th token
  auto refreshed = [&](int t) {
    return UX && p.refresh_period > 0 && (p.step_offset + t + 1) % p.refresh_period == 0;
  };
  const float* zst = p.zst + ubase;
  const float* dst = p.dst + size_t(unit) * T;

  auto cvec = [&](int t, int which) { return ctx[t & (NCTX - 1)][which]; };
  auto uvec = [&](int t) { return ctx[t & (NCTX - 1)][UX ? cU : cKh]; };   // the direction delta is taken along
  const int myrow = tx / (TX / R);
  const bool row_writer = (tx % (TX / R)) == 0;
  constexpr int kCloser = NW, kOpener = NW + 1;

  // the scalars of token t that hang on the adjoint: ddelta and the factors of dz
  //   dz = ddelta u + cK k_hat - idl (2 g + khz da),  cK = -idl daz,  ddelta = (z.g + daz khz) / delta^2
  //   (u = k_hat: one coefficient cK = ddelta - idl daz on k_hat, cU = 0)
  struct MidScalars { float idl, ddelta, cK, cU, khz, zg; };
  auto mid_scalars = [&](int t) {
    float zt[EPL], gv[EPL];
    bwd_ld<EPL>(cvec(t, cZt) + c0, zt);
    bwd_ld<EPL>(rowv[t % 3][0] + c0, gv);
    float zg = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) zg = fmaf(zt[e], gv[e], zg);
    zg = warp_sum(zg);
    const float* sc = cscl[t & (NCTX - 1)];
    MidScalars m;
    m.khz = sc[sKhz];
    m.idl = rcp_nr(sc[sDelta]);   // (on every matrix warp's path, once a token)
    m.zg = zg;
    const bool delta_live = (1.0f + sc[sUz]) >= eps;
    m.ddelta = delta_live ? fmaf(sc[sDaz], m.khz, zg) * m.idl * m.idl : 0.0f;
    m.cK = UX ? -m.idl * sc[sDaz] : fmaf(-m.idl, sc[sDaz], m.ddelta);
    m.cU = UX ? m.ddelta : 0.0f;
    return m;
  };

  // Segment t (one CTA barrier): the matrix warps form dz of token t, r3 = A' dz, the two
  // updates, then the row dots of token t - 1; the closing warp finishes token t + 1, the
  // opening warp prepares token t - 2.  Loops of their own, as on the S side.
  if (warp == kOpener) {
    float pk[EPL], pz[EPL], pa[EPL], ps[EPL], pgz[EPL], pu[EPL], pat[EPL];
    float pdelta = 1.0f;
    // The unit's S side (another CTA of this launch, dispatched earlier) publishes how many
    // tokens, counted from the end, have their vectors out.  Bounded wait; on a time-out the
    // status is set and the sweep goes on with whatever is there.
    int seen = 0;
    auto fetch_token = [&](int t) {
      if (t < 0) return;
      if (seen < T - t) {
        for (int it = 0; it < (1 << 22); ++it) {
          seen = bwd_observe(p.progress + unit);
          if (seen >= T - t) break;
          __nanosleep(256);
        }
        if (seen < T - t && lane == 0 && p.status) atomicCAS(p.status, 0, int(VLA_ERR_DEVICE_TIMEOUT));
      }
      pdelta = dst[t];
      const size_t o = size_t(t) * D + c0;
      const size_t uo = bwd_user_row(p, unit, t, D) + c0;
      bwd_ld_in<EPL>(gk + uo, pk);
      bwd_ld<EPL>(zst + o, pz);
      bwd_ld<EPL>(p.dal + ubase + o, pa);
      bwd_ld<EPL>(p.dkS + ubase + o, ps);
      bwd_ld<EPL>(p.gzt + ubase + o, pgz);
      if constexpr (UX) {
        if (gu) bwd_ld_in<EPL>(gu + uo, pu);
        bwd_ld<EPL>(p.ast + ubase + o, pat);
      }
    };
    // k_hat, alpha, da = (dalpha - alpha (alpha.dalpha)) / ||a|| and the scalars of token t
    auto open_token = [&](int t) {
      float kx[EPL], khx[EPL], dax[EPL];
      float ss = 0.f, zz = 0.f, zpa = 0.f, kz = 0.f, uz = 0.f, papz = 0.f, avpz = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        float kk = pk[e];
        if (!ident) kk = bwd_phi(kk);
        kx[e] = kk;
        const float av = UX ? pat[e] : pz[e];        // a_t up to the factor 1 / delta when u = k_hat
        ss = fmaf(kk, kk, ss);
        zz = fmaf(av, av, zz);
        zpa = fmaf(av, pa[e], zpa);
        kz = fmaf(kk, pz[e], kz);
        papz = fmaf(pa[e], pz[e], papz);             // for da . z below, so that no second round of sums is needed
        if (UX) avpz = fmaf(av, pz[e], avpz);
        if (UX && gu) uz = fmaf(pu[e], pz[e], uz);
      }
      // (this warp sets the pace of the CTA: every sum of the token in one pass through the
      // shuffles, reciprocals and square roots as in the forward kernels)
#pragma unroll
      for (int off = 16; off >= 1; off >>= 1) {
        ss += __shfl_xor_sync(0xffffffffu, ss, off);
        zz += __shfl_xor_sync(0xffffffffu, zz, off);
        zpa += __shfl_xor_sync(0xffffffffu, zpa, off);
        kz += __shfl_xor_sync(0xffffffffu, kz, off);
        papz += __shfl_xor_sync(0xffffffffu, papz, off);
        if (UX) avpz += __shfl_xor_sync(0xffffffffu, avpz, off);
        if (UX && gu) uz += __shfl_xor_sync(0xffffffffu, uz, off);
      }
      if (!UX) avpz = zz;
      const float ink = rcp_nr(fmaxf(sqrt_approx(ss), eps));
      if (UX && !gu) {
#pragma unroll
        for (int e = 0; e < EPL; ++e) pu[e] = kx[e] * ink;
        uz = kz * ink;
      }
      const float idl = rcp_nr(pdelta);
      const float na = UX ? sqrt_approx(zz) : sqrt_approx(zz) * idl;   // ||a||  (a = z / delta when u = k_hat)
      const float sc = (UX ? 1.0f : idl) * rcp_nr(fmaxf(na, eps));
      const float adal = sc * zpa;                   // alpha . dalpha
      const float khz = kz * ink;
      const float ina = rcp_nr(fmaxf(na, eps));
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        const float al = sc * (UX ? pat[e] : pz[e]);
        dax[e] = na > eps ? (pa[e] - al * adal) * ina : pa[e] * ina;
        khx[e] = kx[e] * ink;
      }
      // da . z from the sums above: (dalpha . z - (alpha . dalpha) (alpha . z)) / ||a||, alpha . z = sc (a . z)
      const float daz = na > eps ? (papz - adal * sc * avpz) * ina : papz * ina;
      bwd_st<EPL>(cvec(t, cKf) + c0, kx);
      bwd_st<EPL>(cvec(t, cKh) + c0, khx);
      bwd_st<EPL>(cvec(t, cZt) + c0, pz);
      bwd_st<EPL>(cvec(t, cDa) + c0, dax);
      bwd_st<EPL>(cvec(t, cDkS) + c0, ps);
      bwd_st<EPL>(cvec(t, cGz) + c0, pgz);
      if constexpr (UX) bwd_st<EPL>(cvec(t, cU) + c0, pu);
      if (lane == 0) {
        float* os = cscl[t & (NCTX - 1)];
        os[sDelta] = pdelta; os[sKhz] = khz; os[sDaz] = daz; os[sNk] = sqrt_approx(ss);
        os[sUz] = UX ? uz : khz;
      }
    };
    if (T > 0) {
      fetch_token(T - 1);
      open_token(T - 1);
      fetch_token(T - 2);
      if (T >= 2) open_token(T - 2);
      fetch_token(T - 3);
    }
    cta_sync(NT);
    cta_sync(NT);
    for (int t = T - 1; t >= 0; --t) {
      if (t - 2 >= 0) {
        open_token(t - 2);
        fetch_token(t - 3);
      }
      cta_sync(NT);
    }
  } else if (warp == kCloser) {
    // dk of token t; w_t = da + dz goes where dalpha_t was (read two segments ago) for dA0
    auto close_token = [&](int t) {
      const MidScalars ms = mid_scalars(t);
      float kf[EPL], kh[EPL], zt[EPL], da[EPL], dkS[EPL], gzv[EPL], gv[EPL], r1[EPL], r3[EPL], uv[EPL];
      bwd_ld<EPL>(uvec(t) + c0, uv);
      bwd_ld<EPL>(cvec(t, cKf) + c0, kf);
      bwd_ld<EPL>(cvec(t, cKh) + c0, kh);
      bwd_ld<EPL>(cvec(t, cZt) + c0, zt);
      bwd_ld<EPL>(cvec(t, cDa) + c0, da);
      bwd_ld<EPL>(cvec(t, cDkS) + c0, dkS);
      bwd_ld<EPL>(cvec(t, cGz) + c0, gzv);
      bwd_ld<EPL>(rowv[t % 3][0] + c0, gv);
      bwd_ld<EPL>(rowv[t % 3][1] + c0, r1);
      bwd_ld<EPL>(rowv[t % 3][2] + c0, r3);
      const float nkraw = cscl[t & (NCTX - 1)][sNk], daz = cscl[t & (NCTX - 1)][sDaz];
      const float uz = cscl[t & (NCTX - 1)][sUz];
      const float ink = rcp_nr(fmaxf(nkraw, eps));
      // z . dz = cU u.z + cK khz - idl (2 z.g + khz daz);  A dz = A' dz + z (z.dz) / delta
      const float zdz = fmaf(ms.cU, uz, fmaf(ms.cK, ms.khz, -ms.idl * fmaf(ms.khz, daz, 2.0f * ms.zg)));
      const float zs = fmaf(zdz, ms.idl, ms.ddelta);
      const bool rf = refreshed(t);
      float dkhx[EPL], out[EPL], wv[EPL], dzv[EPL], duv[EPL];
      float kd = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        const float dz = fmaf(ms.cU, uv[e], fmaf(ms.cK, kh[e], -ms.idl * fmaf(ms.khz, da[e], 2.0f * gv[e])));
        dzv[e] = dz;
        wv[e] = UX ? da[e] : da[e] + dz;
        // ddelta z + A_{t-1} dz: the gradient of u.  r3 is A_t dz; a refreshed A_t carries eta I
        // that A_{t-1} + (the step) does not
        duv[e] = fmaf(zt[e], zs, r3[e] - (rf ? p.refresh_eta * dz : 0.0f));
        dkhx[e] = dkS[e] + r1[e] + ((UX && gu) ? 0.0f : duv[e]);   // u = k_hat: it lands on k_hat
        kd = fmaf(kh[e], dkhx[e], kd);
      }
      kd = warp_sum(kd);
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        float dkf = nkraw > eps ? (dkhx[e] - kh[e] * kd) * ink : dkhx[e] * ink;
        if (!ident) {
          dkf += gzv[e];
          dkf *= kf[e] > 1.0f ? 1.0f : kf[e];     // phi'(k) from phi(k)
        }
        out[e] = dkf;
      }
      bwd_st<EPL>(p.dk + bwd_user_row(p, unit, t, D) + c0, out);
      if constexpr (UX) {
        if (gu) bwd_st<EPL>(p.du + bwd_user_row(p, unit, t, D) + c0, duv);
      }
      if (p.dA0) {   // for dA0: w_t (u = k_hat), or da_t and dz_t, over vectors this token no longer needs
        bwd_st<EPL>(p.dal + ubase + size_t(t) * D + c0, wv);
        if constexpr (UX) bwd_st<EPL>(p.dkS + ubase + size_t(t) * D + c0, dzv);
      }
    };
    cta_sync(NT);
    cta_sync(NT);
    for (int t = T - 1; t >= 0; --t) {
      if (t + 1 <= T - 1) close_token(t + 1);
      cta_sync(NT);
    }
    if (T > 0) close_token(0);
  } else {
    float2 A[R][RP], GA[R][RP];   // GA: the symmetric part
    // The adjoint sums one update per token; over tens of thousands of tokens the rounding of a
    // single fp32 accumulator (a random walk of one half-ulp of the SUM per token) reaches 1e-3 of
    // the early tokens' gradients, whose own scale is far below the sum's.  Two levels: updates go
    // to a small accumulator that is folded into the large one every kFold tokens, so the large one
    // is rounded T / kFold times instead of T (d <= 64; at d = 128 the registers are spoken for
    // and no workload is that long).
    constexpr bool TWO_LEVEL = D <= 64;
    constexpr int kFold = 1024;
    float2 GAs[TWO_LEVEL ? R : 1][TWO_LEVEL ? RP : 1];
#pragma unroll
    for (int r = 0; r < (TWO_LEVEL ? R : 1); ++r)
#pragma unroll
      for (int m = 0; m < (TWO_LEVEL ? RP : 1); ++m) GAs[r][m] = make_float2(0.f, 0.f);
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const size_t idx = (size_t(unit) * D + row0 + r) * D + col0;
      float sv[RC], gv[RC];
      bwd_ld<RC>(p.AT + idx, sv);
#pragma unroll
      for (int c = 0; c < RC; ++c)
        gv[c] = p.dA_T ? 0.5f * (p.dA_T[idx + c] + p.dA_T[(size_t(unit) * D + col0 + c) * D + row0 + r]) : 0.0f;
#pragma unroll
      for (int m = 0; m < RP; ++m) {
        A[r][m] = make_float2(sv[2 * m], sv[2 * m + 1]);
        GA[r][m] = make_float2(gv[2 * m], gv[2 * m + 1]);
      }
    }
    // g = GAs z and r1 = A' da for token t
    auto products = [&](int t) {
      float zc[RC], dc[RC];
      bwd_ld<RC>(cvec(t, cZt) + col0, zc);
      bwd_ld<RC>(cvec(t, cDa) + col0, dc);
      float a0[R], a1[R];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        float2 x0 = make_float2(0.f, 0.f), x1 = make_float2(0.f, 0.f);
#pragma unroll
        for (int m = 0; m < RP; ++m) {
          x0 = bwd_ffma2(GA[r][m], make_float2(zc[2 * m], zc[2 * m + 1]), x0);
          x1 = bwd_ffma2(A[r][m], make_float2(dc[2 * m], dc[2 * m + 1]), x1);
        }
        if constexpr (TWO_LEVEL) {
          float2 xs = make_float2(0.f, 0.f);
#pragma unroll
          for (int m = 0; m < RP; ++m) xs = bwd_ffma2(GAs[r][m], make_float2(zc[2 * m], zc[2 * m + 1]), xs);
          x0.x += xs.x; x0.y += xs.y;
        }
        a0[r] = x0.x + x0.y; a1[r] = x1.x + x1.y;
      }
      rows_reduce<R, TX / 2>(a0, lane);
      rows_reduce<R, TX / 2>(a1, lane);
      if (row_writer) { rowv[t % 3][0][row0 + myrow] = a0[0]; rowv[t % 3][1][row0 + myrow] = a1[0]; }
    };
    cta_sync(NT);
    if (T > 0) products(T - 1);
    cta_sync(NT);
    for (int t = T - 1; t >= 0; --t) {
      // dz of token t at this thread's columns; r3 = A' dz (before the update)
      const MidScalars ms = mid_scalars(t);
      float kc[RC], zc[RC], wc[RC], uc[RC], dzk[RC];   // UX: wc = da, dzk = dz at the columns
      bwd_ld<RC>(cvec(t, cKh) + col0, kc);
      if constexpr (UX) bwd_ld<RC>(cvec(t, cU) + col0, uc);
      {
        float dac[RC], gc[RC], dzc[RC];
        bwd_ld<RC>(cvec(t, cDa) + col0, dac);
        bwd_ld<RC>(rowv[t % 3][0] + col0, gc);
#pragma unroll
        for (int c = 0; c < RC; ++c) {
          dzc[c] = fmaf(ms.cK, kc[c], -ms.idl * fmaf(ms.khz, dac[c], 2.0f * gc[c]));
          if (UX) dzc[c] = fmaf(ms.cU, uc[c], dzc[c]);
          wc[c] = UX ? dac[c] : dac[c] + dzc[c];
          dzk[c] = dzc[c];
        }
        float b1[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
          float2 x1 = make_float2(0.f, 0.f);
#pragma unroll
          for (int m = 0; m < RP; ++m) x1 = bwd_ffma2(A[r][m], make_float2(dzc[2 * m], dzc[2 * m + 1]), x1);
          b1[r] = x1.x + x1.y;
        }
        rows_reduce<R, TX / 2>(b1, lane);
        if (row_writer) rowv[t % 3][2][row0 + myrow] = b1[0];
      }
      // GAs += (w k_hat^T + k_hat w^T) / 2,  A += z z^T / delta
      bwd_ld<RC>(cvec(t, cZt) + col0, zc);
      constexpr int RG = R >= 4 ? 4 : R;
#pragma unroll
      for (int rg = 0; rg < R / RG; ++rg) {
        float kr[RG], zr[RG], dar[RG], gr[RG], ur[RG];
        bwd_ld<RG>(cvec(t, cKh) + row0 + rg * RG, kr);
        bwd_ld<RG>(cvec(t, cZt) + row0 + rg * RG, zr);
        bwd_ld<RG>(cvec(t, cDa) + row0 + rg * RG, dar);
        bwd_ld<RG>(rowv[t % 3][0] + row0 + rg * RG, gr);
        if constexpr (UX) bwd_ld<RG>(cvec(t, cU) + row0 + rg * RG, ur);
#pragma unroll
        for (int i = 0; i < RG; ++i) {
          const int r = rg * RG + i;
          float dzr = fmaf(ms.cK, kr[i], -ms.idl * fmaf(ms.khz, dar[i], 2.0f * gr[i]));
          if (UX) dzr = fmaf(ms.cU, ur[i], dzr);
          const float hw = 0.5f * (UX ? dar[i] : dar[i] + dzr), hk = 0.5f * kr[i], zs = zr[i] * ms.idl;
          const float2 w2 = make_float2(hw, hw), k2 = make_float2(hk, hk), z2 = make_float2(zs, zs);
#pragma unroll
          for (int m = 0; m < RP; ++m) {
            float2& acc = TWO_LEVEL ? GAs[r][m] : GA[r][m];
            acc = bwd_ffma2(w2, make_float2(kc[2 * m], kc[2 * m + 1]), acc);
            acc = bwd_ffma2(k2, make_float2(wc[2 * m], wc[2 * m + 1]), acc);
            A[r][m] = bwd_ffma2(z2, make_float2(zc[2 * m], zc[2 * m + 1]), A[r][m]);
          }
          if constexpr (UX) {   // + sym(dz u^T)
            const float hz = 0.5f * dzr, hu = 0.5f * ur[i];
            const float2 dz2 = make_float2(hz, hz), u2 = make_float2(hu, hu);
#pragma unroll
            for (int m = 0; m < RP; ++m) {
              float2& acc = TWO_LEVEL ? GAs[r][m] : GA[r][m];
              acc = bwd_ffma2(dz2, make_float2(uc[2 * m], uc[2 * m + 1]), acc);
              acc = bwd_ffma2(u2, make_float2(dzk[2 * m], dzk[2 * m + 1]), acc);
            }
            if (refreshed(t)) {   // A_t = (the step) + eta I: take the refresh off the diagonal
#pragma unroll
              for (int m = 0; m < RP; ++m) {
                if (row0 + r == col0 + 2 * m) A[r][m].x -= p.refresh_eta;
                if (row0 + r == col0 + 2 * m + 1) A[r][m].y -= p.refresh_eta;
              }
            }
          }
        }
      }
      if constexpr (TWO_LEVEL) {
        if ((t % kFold) == 0) {
#pragma unroll
          for (int r = 0; r < R; ++r)
#pragma unroll
            for (int m = 0; m < RP; ++m) {
              GA[r][m].x += GAs[r][m].x; GA[r][m].y += GAs[r][m].y;
              GAs[r][m] = make_float2(0.f, 0.f);
            }
        }
      }
      if (t >= 1) products(t - 1);
      cta_sync(NT);
    }
  }
}

// Both reverse scans as ONE launch of 2 * units CTAs.  Each CTA draws a ticket when it starts:
// ticket x < units is the S side of unit x, ticket units + x its A side, so a unit's S side is
// running or finished whenever its A side starts, whatever order the CTAs are dispatched in;
// the A side follows it token by token through a progress word in global memory (released every
// eighth token).  With fewer units than SMs the two sides of a unit run side by side on two SMs;
// with many units the A-side CTAs fill the SMs the last wave of S-side CTAs leaves idle.
template <int D, typename TIn, bool UX>
__global__ void __launch_bounds__(BwdSplitGeom<D>::NT_S, BwdSplitGeom<D>::MINB)
vla_backward_sa_kernel(const BackwardSplitParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  // the ticket travels through the last word of the dynamic shared memory (behind both sides' layouts)
  int* ticket_s = reinterpret_cast<int*>(smem_raw + BackwardSplitSmem<D>::sa_bytes - sizeof(int));
  if (threadIdx.x == 0) *ticket_s = atomicAdd(p.progress + p.units, 1);   // the word after the units' own
  __syncthreads();
  const int ticket = *ticket_s;
  if (ticket < p.units) vla_backward_s_body<D, TIn, UX>(p, ticket, smem_raw);
  else vla_backward_a_body<D, TIn, UX>(p, ticket - p.units, smem_raw);
}

// dA0 = dA_T + sum_t w_t k_hat_t^T from the w_t the A side left in the workspace (only when
// the caller asks for dA0); with explicit u: + sum_t dz_t u_t^T, w_t = da_t.  One CTA of 256 threads per unit; thread (ty, tx) of a 16 x 16 grid
// accumulates an R x R block over tiles of 16 tokens staged in shared memory.
template <int D, typename TIn, bool UX>
__global__ void __launch_bounds__(256) vla_backward_da0_kernel(const BackwardSplitParams p) {
  constexpr int R = D / 16;
  constexpr int EPL = D / 32;
  constexpr int TT = 16;
  __shared__ float wt[TT][D];
  __shared__ float kt[TT][D];
  __shared__ float zt2[UX ? TT : 1][D];   // dz_t and u_t (explicit u)
  __shared__ float ut2[UX ? TT : 1][D];
  const int unit = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int ty = tid >> 4, tx = tid & 15;
  const int row0 = ty * R, col0 = tx * R;
  const bool ident = (p.flags & VLA_FLAG_IDENTITY_MAP) != 0;
  const size_t ubase = size_t(unit) * size_t(p.T) * D;
  const TIn* gk = static_cast<const TIn*>(p.k);
  float acc[R][R];
#pragma unroll
  for (int r = 0; r < R; ++r)
#pragma unroll
    for (int c = 0; c < R; ++c)
      acc[r][c] = p.dA_T ? p.dA_T[(size_t(unit) * D + row0 + r) * D + col0 + c] : 0.0f;
  for (int t0 = 0; t0 < p.T; t0 += TT) {
    __syncthreads();
    for (int i = warp; i < TT; i += 8) {
      const int t = t0 + i;
      float kx[EPL], wv[EPL];
      float ss = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        const int c = e * 32 + lane;
        float kk = t < p.T ? load1<TIn>(gk, bwd_user_row(p, unit, t, D) + c) : 0.0f;
        if (!ident && t < p.T) kk = bwd_phi(kk);
        kx[e] = kk;
        wv[e] = t < p.T ? p.dal[ubase + size_t(t) * D + c] : 0.0f;
        ss = fmaf(kk, kk, ss);
      }
      ss = warp_sum(ss);
      const float ink = 1.0f / fmaxf(sqrtf(ss), p.eps);
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        kt[i][e * 32 + lane] = kx[e] * ink;
        wt[i][e * 32 + lane] = wv[e];
        if constexpr (UX) {
          const int c = e * 32 + lane;
          zt2[i][c] = t < p.T ? p.dkS[ubase + size_t(t) * D + c] : 0.0f;
          ut2[i][c] = !p.u ? kx[e] * ink
                           : (t < p.T ? load1<TIn>(static_cast<const TIn*>(p.u), bwd_user_row(p, unit, t, D) + c) : 0.0f);
        }
      }
    }
    __syncthreads();
#pragma unroll 4
    for (int i = 0; i < TT; ++i)
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const float w = wt[i][row0 + r];
#pragma unroll
        for (int c = 0; c < R; ++c) acc[r][c] = fmaf(w, kt[i][col0 + c], acc[r][c]);
        if constexpr (UX) {
          const float z = zt2[i][row0 + r];
#pragma unroll
          for (int c = 0; c < R; ++c) acc[r][c] = fmaf(z, ut2[i][col0 + c], acc[r][c]);
        }
      }
  }
#pragma unroll
  for (int r = 0; r < R; ++r)
#pragma unroll
    for (int c = 0; c < R; ++c) p.dA0[(size_t(unit) * D + row0 + r) * D + col0 + c] = acc[r][c];
}

}  // namespace vla
