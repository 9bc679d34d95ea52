// VLA backward pass as two reverse scans (u = k_hat, d in {32, 64, 128}).
//
// The adjoint of the memory state, GS = dL/dS, obeys a recurrence of its own that never looks at
// the penalty side: GS_{t-1} = GS_t + dy qf^T - de k_hat^T.  So the reverse sweep splits into
//
//   S side (vla_backward_s_kernel): S and GS in registers.  Per token: dq, dv, and three
//     vectors for the other side: dalpha_t = dL/d alpha_t, the S-side part of dL/d k_hat_t, and
//     the running gradient of the key sum.
//   A side (vla_backward_a_kernel): A and GA = dL/dA in registers.  Per token it turns dalpha_t
//     into da, forms dz, ddelta and the remaining parts of dL/d k_hat_t, and writes dk.
//
// each a CTA per unit holding TWO d x d matrices in registers, as R x RC blocks on a grid of
// 16 x TX threads (R = d / 16 rows, RC = d / TX columns; TX = 16, or 32 at d = 128, where the
// blocks of a 16-wide grid would not leave registers for a ninth warp).  The forward recurrence is not re-run here: the chunk kernel
// leaves z_t, e_t, delta_t per token and the final S, A, key sum in the workspace, and both
// sweeps walk the states back by undoing the rank-1 updates (S_{t-1} = S_t - e alpha^T,
// A_{t-1} = A_t + z z^T / delta).  Formulas per token: see vla_backward.cuh.
//
// Both kernels keep a ring of four per-token contexts in shared memory so that opening a
// token (loading its rows, alpha, denominators: nothing that depends on the adjoints) and
// closing one (vector arithmetic on finished products) are done by a ninth warp off the path
// of the TX / 2 matrix warps; one CTA barrier per token.
#pragma once

#include "vla_backward.cuh"

namespace vla {

// Dynamic shared memory of the two reverse scans (the kernels assert these against their layouts).
template <int D>
struct BackwardSplitSmem {
  static constexpr int NW = (D >= 128 ? 32 : 16) / 2;
  static constexpr size_t s_bytes = sizeof(float) * (4 * 7 * D + 4 * 4 + 3 * 2 * D + 2 * NW * 3 * D + D);
  static constexpr size_t a_bytes = sizeof(float) * (4 * 6 * D + 4 * 4 + 3 * 3 * D + 2 * NW * D + NW * D + 4);
};

// Thread grid of the two reverse scans.
template <int D>
struct BwdSplitGeom {
  static constexpr int TX = D >= 128 ? 32 : 16;   // threads along a matrix row
  static constexpr int R = D / 16;                // rows of a thread's block
  static constexpr int RC = D / TX;               // columns of a thread's block
  static constexpr int NW = TX / 2;               // matrix warps; warp NW is the helper
  static constexpr int NT = NW * 32 + 32;
};

// All threads of the CTA, whichever loop they are in.
__device__ __forceinline__ void cta_sync() { asm volatile("bar.sync 0;" ::: "memory"); }

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
template <int D, typename TIn>
__global__ void __launch_bounds__(BwdSplitGeom<D>::NT) vla_backward_s_kernel(const BackwardSplitParams p) {
  using G = BwdSplitGeom<D>;
  constexpr int R = G::R, RC = G::RC, TX = G::TX, NW = G::NW, NT = G::NT;
  constexpr int EPL = D / 32;
  constexpr int NCTX = 4;
  enum { cKf = 0, cKh, cQf, cGo, cEt, cAl, cZk, NV };
  enum { sDen = 0, sDenLive, sQal };
  struct Smem {
    float ctx[NCTX][NV][D];
    float cscl[NCTX][4];
    float rowv[3][2][D];       // y = S' qf, g1 = GS alpha, ring of three tokens
    float part[2][NW][3][D];   // column-sum partials by token parity and warp
    float gz[D];               // dL/d(key sum), carried by the helper warp
  };
  static_assert(sizeof(Smem) == BackwardSplitSmem<D>::s_bytes, "shared memory size of the S side");
  extern __shared__ __align__(16) unsigned char smem_raw[];
  Smem& sm = *reinterpret_cast<Smem*>(smem_raw);
  auto& ctx = sm.ctx; auto& cscl = sm.cscl; auto& rowv = sm.rowv; auto& part = sm.part; auto& gz = sm.gz;

  const int unit = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int ty = tid / TX, tx = tid % TX;
  const int row0 = ty * R, col0 = tx * RC;
  const bool ident = (p.flags & VLA_FLAG_IDENTITY_MAP) != 0;
  const float eps = p.eps;
  const int T = p.T;
  const size_t ubase = size_t(unit) * size_t(T) * D;
  const TIn* gq = static_cast<const TIn*>(p.q) + ubase;
  const TIn* gk = static_cast<const TIn*>(p.k) + ubase;
  const float* gdo = p.d_out + ubase;
  const float* zst = p.zst + ubase;
  const float* est = p.est + ubase;
  const float* dst = p.dst + size_t(unit) * T;

  float S[R][RC], GS[R][RC];
#pragma unroll
  for (int r = 0; r < R; ++r)
#pragma unroll
    for (int c = 0; c < RC; ++c) {
      const size_t idx = (size_t(unit) * D + row0 + r) * D + col0 + c;
      const bool own = warp < NW;   // the helper warp holds no block
      S[r][c] = own ? p.ST[idx] : 0.0f;
      GS[r][c] = (own && p.dS_T) ? p.dS_T[idx] : 0.0f;
    }
  for (int j = tid; j < D; j += NT) gz[j] = p.dz_T ? p.dz_T[size_t(unit) * D + j] : 0.0f;

  auto cvec = [&](int t, int which) { return ctx[t & (NCTX - 1)][which]; };
  // after rows_reduce<R, TX / 2> a lane holds the total of row myrow of its group's R rows
  const int myrow = tx / (TX / R);
  const bool row_writer = (tx % (TX / R)) == 0;

  // the helper warp opens tokens two segments ahead; the rows come from global memory one more ahead
  float pk[EPL], pq[EPL], pz[EPL], pe[EPL], pg[EPL];
  float pdelta = 1.0f;
  auto fetch_token = [&](int t) {
    if (t < 0) return;
    pdelta = dst[t];
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      const int c = e * 32 + lane;
      pk[e] = load1<TIn>(gk, size_t(t) * D + c);
      pq[e] = load1<TIn>(gq, size_t(t) * D + c);
      pz[e] = zst[size_t(t) * D + c];
      pe[e] = est[size_t(t) * D + c];
      pg[e] = gdo[size_t(t) * D + c];
    }
  };
  auto open_token = [&](int t, bool last) {
    float* okf = cvec(t, cKf); float* okh = cvec(t, cKh); float* oqf = cvec(t, cQf);
    float* ogo = cvec(t, cGo); float* oet = cvec(t, cEt); float* oal = cvec(t, cAl);
    float* ozk = cvec(t, cZk);
    const float* nzk = cvec(t + 1, cZk);
    const float* nkf = cvec(t + 1, cKf);
    float zx[EPL], kx[EPL], qx[EPL];
    float ss = 0.f, zz = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      const int c = e * 32 + lane;
      float kk = pk[e], qq = pq[e];
      if (!ident) { kk = bwd_phi(kk); qq = bwd_phi(qq); }
      ogo[c] = pg[e];
      oet[c] = pe[e];
      okf[c] = kk;
      oqf[c] = qq;
      kx[e] = kk; qx[e] = qq; zx[e] = pz[e];
      ss = fmaf(kk, kk, ss);
      zz = fmaf(pz[e], pz[e], zz);
    }
    ss = warp_sum(ss);
    zz = warp_sum(zz);
    const float nk = fmaxf(sqrtf(ss), eps);
    const float idl = 1.0f / pdelta;
    const float sc = idl / fmaxf(sqrtf(zz) * idl, eps);
    float dn = 0.f, qa = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      const int c = e * 32 + lane;
      okh[c] = kx[e] / nk;
      oal[c] = sc * zx[e];
      const float zkc = last ? p.zT[size_t(unit) * D + c] : (ident ? nzk[c] : nzk[c] - nkf[c]);
      ozk[c] = zkc;
      dn = fmaf(zkc, qx[e], dn);
      qa = fmaf(qx[e], sc * zx[e], qa);
    }
    dn = warp_sum(dn);
    qa = warp_sum(qa);
    if (lane == 0) {
      float* os = cscl[t & (NCTX - 1)];
      os[sDen] = ident ? 1.0f : fmaxf(dn, eps);
      os[sDenLive] = (ident || dn < eps) ? 0.0f : 1.0f;
      os[sQal] = qa;
    }
  };
  // helper warp: the vector results of token t from its finished products
  auto close_token = [&](int t) {
    const int par = t & 1;
    const float* go = cvec(t, cGo); const float* et = cvec(t, cEt); const float* al = cvec(t, cAl);
    const float* qf = cvec(t, cQf); const float* zkt = cvec(t, cZk);
    const float* yv = rowv[t % 3][0]; const float* g1 = rowv[t % 3][1];
    const float den = cscl[t & (NCTX - 1)][sDen], qal = cscl[t & (NCTX - 1)][sQal];
    const bool den_live = cscl[t & (NCTX - 1)][sDenLive] != 0.0f;
    float odo = 0.f, ede = 0.f, dye = 0.f;
    float dex[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      const int c = e * 32 + lane;
      const float dy = go[c] / den;
      dex[e] = g1[c] + dy * qal;
      odo = fmaf(yv[c], go[c], odo);
      ede = fmaf(et[c], dex[e], ede);
      dye = fmaf(dy, et[c], dye);
    }
    odo = warp_sum(odo); ede = warp_sum(ede); dye = warp_sum(dye);
    const float dden = den_live ? -odo / (den * den) : 0.0f;
    const size_t tb = ubase + size_t(t) * D;
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      const int c = e * 32 + lane;
      float c1 = 0.f, c2 = 0.f, c3 = 0.f;
#pragma unroll
      for (int w = 0; w < NW; ++w) {
        c1 += part[par][w][0][c]; c2 += part[par][w][1][c]; c3 += part[par][w][2][c];
      }
      float dq = c1 + dden * zkt[c];
      float gzc = gz[c];
      if (!ident) {
        dq *= qf[c] > 1.0f ? 1.0f : qf[c];     // phi'(q) from phi(q)
        gzc += dden * qf[c];
        gz[c] = gzc;
      }
      p.dq[tb + c] = dq;
      p.dv[tb + c] = dex[e];
      p.dal[tb + c] = c2 + qf[c] * dye;               // (GS + dy qf^T)^T e
      p.dkS[tb + c] = -(c3 - al[c] * ede);            // -(S' - e alpha^T)^T de
      p.gzt[tb + c] = ident ? 0.0f : gzc;
    }
  };

  constexpr int kHelper = NW;   // the last warp opens and closes tokens; the others do the matrix work
  auto row_dots = [&](int t) {   // y = S' qf, g1 = GS alpha of token t
    const float* qf = cvec(t, cQf); const float* al = cvec(t, cAl);
    float a0[R], a1[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      float x0 = 0.f, x1 = 0.f;
#pragma unroll
      for (int c = 0; c < RC; ++c) {
        x0 = fmaf(S[r][c], qf[col0 + c], x0);
        x1 = fmaf(GS[r][c], al[col0 + c], x1);
      }
      a0[r] = x0; a1[r] = x1;
    }
    rows_reduce<R, TX / 2>(a0, lane);
    rows_reduce<R, TX / 2>(a1, lane);
    if (row_writer) { rowv[t % 3][0][row0 + myrow] = a0[0]; rowv[t % 3][1][row0 + myrow] = a1[0]; }
  };

  // Segment t (one CTA barrier): the matrix warps take the column sums and the two rank-1
  // updates of token t, then the row dots of token t - 1; the helper warp closes token t + 1
  // and opens token t - 2.  The two roles run loops of their own with the same number of
  // barriers, so that the helper's staging registers and the matrix blocks never share a thread.
  if (warp == kHelper) {
    if (T > 0) {
      fetch_token(T - 1);
      open_token(T - 1, true);
      fetch_token(T - 2);
      if (T >= 2) open_token(T - 2, false);
      fetch_token(T - 3);
    }
    cta_sync();
    cta_sync();
    for (int t = T - 1; t >= 0; --t) {
      if (t + 1 <= T - 1) close_token(t + 1);
      if (t - 2 >= 0) {
        open_token(t - 2, false);
        fetch_token(t - 3);
      }
      cta_sync();
    }
    if (T > 0) close_token(0);
  } else {
    cta_sync();
    if (T > 0) row_dots(T - 1);
    cta_sync();
    for (int t = T - 1; t >= 0; --t) {
      const float* go = cvec(t, cGo); const float* et = cvec(t, cEt);
      const float* kh = cvec(t, cKh); const float* qf = cvec(t, cQf); const float* al = cvec(t, cAl);
      const float* g1 = rowv[t % 3][1];
      const float den = cscl[t & (NCTX - 1)][sDen], qal = cscl[t & (NCTX - 1)][sQal];
      float dyr[R], der[R];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        dyr[r] = go[row0 + r] / den;
        der[r] = g1[row0 + r] + dyr[r] * qal;      // (GS + dy qf^T) alpha
      }
      float cc[3][RC];
#pragma unroll
      for (int c = 0; c < RC; ++c) {
        float s0 = 0.f, s1 = 0.f, s2 = 0.f;
#pragma unroll
        for (int r = 0; r < R; ++r) {
          s0 = fmaf(S[r][c], dyr[r], s0);
          s1 = fmaf(GS[r][c], et[row0 + r], s1);
          s2 = fmaf(S[r][c], der[r], s2);
        }
        cc[0][c] = s0; cc[1][c] = s1; cc[2][c] = s2;
      }
      if constexpr (TX == 16) {
        // two thread rows per warp: each half keeps half of the columns of the pair's sum
        constexpr int HC = RC / 2;
        const bool up = (lane & 16) != 0;
#pragma unroll
        for (int k2 = 0; k2 < 3; ++k2)
#pragma unroll
          for (int c = 0; c < HC; ++c) {
            const float send = up ? cc[k2][c] : cc[k2][c + HC];
            const float keep = up ? cc[k2][c + HC] : cc[k2][c];
            part[t & 1][warp][k2][col0 + (up ? HC : 0) + c] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
          }
      } else {
#pragma unroll
        for (int k2 = 0; k2 < 3; ++k2)
#pragma unroll
          for (int c = 0; c < RC; ++c) part[t & 1][warp][k2][col0 + c] = cc[k2][c];
      }
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const float er = et[row0 + r];
#pragma unroll
        for (int c = 0; c < RC; ++c) {
          GS[r][c] = fmaf(dyr[r], qf[col0 + c], GS[r][c]);
          GS[r][c] = fmaf(-der[r], kh[col0 + c], GS[r][c]);
          S[r][c] = fmaf(-er, al[col0 + c], S[r][c]);
        }
      }
      if (t >= 1) row_dots(t - 1);
      cta_sync();
    }
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
      for (int c = 0; c < RC; ++c)
        if (p.dS0) p.dS0[(size_t(unit) * D + row0 + r) * D + col0 + c] = GS[r][c];
  }
  cta_sync();
  if (p.dz0)
    for (int j = tid; j < D; j += NT) p.dz0[size_t(unit) * D + j] = gz[j];
}

// ------------------------------------------------------------------------------ A side
template <int D, typename TIn>
__global__ void __launch_bounds__(BwdSplitGeom<D>::NT) vla_backward_a_kernel(const BackwardSplitParams p) {
  using G = BwdSplitGeom<D>;
  constexpr int R = G::R, RC = G::RC, TX = G::TX, NW = G::NW, NT = G::NT;
  constexpr int EPL = D / 32;
  constexpr int NCTX = 4;
  enum { cKf = 0, cKh, cZt, cDa, cDkS, cGz, NV };
  enum { sDelta = 0, sKhz, sDaz, sNk };
  struct Smem {
    float ctx[NCTX][NV][D];
    float cscl[NCTX][4];
    float rowv[3][3][D];      // gaz = GA z, r1 = A' da, r3 = A' dz, ring of three tokens
    float part[2][NW][D];     // column-sum partials GA^T z by token parity and warp
    float dzw[NW][D];         // dz of the token in hand, one copy per matrix warp
    float rscl[2][2];         // ddelta, z.dz by token parity
  };
  static_assert(sizeof(Smem) == BackwardSplitSmem<D>::a_bytes, "shared memory size of the A side");
  extern __shared__ __align__(16) unsigned char smem_raw[];
  Smem& sm = *reinterpret_cast<Smem*>(smem_raw);
  auto& ctx = sm.ctx; auto& cscl = sm.cscl; auto& rowv = sm.rowv; auto& part = sm.part;
  auto& dzw = sm.dzw; auto& rscl = sm.rscl;

  const int unit = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int ty = tid / TX, tx = tid % TX;
  const int row0 = ty * R, col0 = tx * RC;
  const bool ident = (p.flags & VLA_FLAG_IDENTITY_MAP) != 0;
  const float eps = p.eps;
  const int T = p.T;
  const size_t ubase = size_t(unit) * size_t(T) * D;
  const TIn* gk = static_cast<const TIn*>(p.k) + ubase;
  const float* zst = p.zst + ubase;
  const float* dst = p.dst + size_t(unit) * T;

  float A[R][RC], GA[R][RC];
#pragma unroll
  for (int r = 0; r < R; ++r)
#pragma unroll
    for (int c = 0; c < RC; ++c) {
      const size_t idx = (size_t(unit) * D + row0 + r) * D + col0 + c;
      const bool own = warp < NW;   // the helper warp holds no block
      A[r][c] = own ? p.AT[idx] : 0.0f;
      GA[r][c] = (own && p.dA_T) ? p.dA_T[idx] : 0.0f;
    }

  auto cvec = [&](int t, int which) { return ctx[t & (NCTX - 1)][which]; };
  // after rows_reduce<R, TX / 2> a lane holds the total of row myrow of its group's R rows
  const int myrow = tx / (TX / R);
  const bool row_writer = (tx % (TX / R)) == 0;

  float pk[EPL], pz[EPL], pa[EPL], ps[EPL], pgz[EPL];
  float pdelta = 1.0f;
  auto fetch_token = [&](int t) {
    if (t < 0) return;
    pdelta = dst[t];
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      const int c = e * 32 + lane;
      pk[e] = load1<TIn>(gk, size_t(t) * D + c);
      pz[e] = zst[size_t(t) * D + c];
      pa[e] = p.dal[ubase + size_t(t) * D + c];
      ps[e] = p.dkS[ubase + size_t(t) * D + c];
      pgz[e] = p.gzt[ubase + size_t(t) * D + c];
    }
  };
  // one warp: k_hat, alpha, da = (dalpha - alpha (alpha.dalpha)) / ||a|| and the scalars of token t
  auto open_token = [&](int t) {
    float* okf = cvec(t, cKf); float* okh = cvec(t, cKh); float* ozt = cvec(t, cZt);
    float* oda = cvec(t, cDa); float* odk = cvec(t, cDkS); float* ogz = cvec(t, cGz);
    float kx[EPL];
    float ss = 0.f, zz = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      float kk = pk[e];
      if (!ident) kk = bwd_phi(kk);
      kx[e] = kk;
      ss = fmaf(kk, kk, ss);
      zz = fmaf(pz[e], pz[e], zz);
    }
    ss = warp_sum(ss);
    zz = warp_sum(zz);
    const float nk = fmaxf(sqrtf(ss), eps);
    const float idl = 1.0f / pdelta;
    const float na = sqrtf(zz) * idl;              // ||a||, a = z / delta
    const float sc = idl / fmaxf(na, eps);
    float adal = 0.f, khz = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      adal = fmaf(sc * pz[e], pa[e], adal);
      khz = fmaf(kx[e] / nk, pz[e], khz);
    }
    adal = warp_sum(adal);
    khz = warp_sum(khz);
    float daz = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      const int c = e * 32 + lane;
      const float al = sc * pz[e];
      const float da = na > eps ? (pa[e] - al * adal) / na : pa[e] / eps;
      okf[c] = kx[e];
      okh[c] = kx[e] / nk;
      ozt[c] = pz[e];
      oda[c] = da;
      odk[c] = ps[e];
      ogz[c] = pgz[e];
      daz = fmaf(da, pz[e], daz);
    }
    daz = warp_sum(daz);
    if (lane == 0) {
      float* os = cscl[t & (NCTX - 1)];
      os[sDelta] = pdelta; os[sKhz] = khz; os[sDaz] = daz; os[sNk] = sqrtf(ss);
    }
  };
  // every matrix warp: dz, ddelta of token t from gaz and the column sums, each warp for itself
  // (a copy of dz per warp: no CTA barrier between this and the updates that need it)
  auto mid_token = [&](int t) {
    const int par = t & 1;
    const float* kh = cvec(t, cKh); const float* zt = cvec(t, cZt); const float* da = cvec(t, cDa);
    const float* gaz = rowv[t % 3][0];
    const float delta = cscl[t & (NCTX - 1)][sDelta], khz = cscl[t & (NCTX - 1)][sKhz];
    const float daz = cscl[t & (NCTX - 1)][sDaz];
    float wx[EPL], c4[EPL];
    float zw = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      const int c = e * 32 + lane;
      float s = 0.f;
#pragma unroll
      for (int w = 0; w < NW; ++w) s += part[par][w][c];
      c4[e] = s;
      wx[e] = gaz[c] + da[c] * khz;                         // (GA + da k_hat^T) z
      zw = fmaf(zt[c], wx[e], zw);
    }
    zw = warp_sum(zw);
    const bool delta_live = (1.0f + khz) >= eps;
    const float ddelta = delta_live ? zw / (delta * delta) : 0.0f;
    float zdz = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      const int c = e * 32 + lane;
      const float dz = -(wx[e] + c4[e] + kh[c] * daz) / delta + ddelta * kh[c];
      dzw[warp][c] = dz;
      zdz = fmaf(zt[c], dz, zdz);
    }
    zdz = warp_sum(zdz);
    if (warp == 0 && lane == 0) { rscl[par][0] = ddelta; rscl[par][1] = zdz; }
    __syncwarp();
  };
  // helper warp: dk of token t
  auto close_token = [&](int t) {
    const int par = t & 1;
    const float* kf = cvec(t, cKf); const float* kh = cvec(t, cKh); const float* zt = cvec(t, cZt);
    const float* dkS = cvec(t, cDkS); const float* gzv = cvec(t, cGz);
    const float* r1 = rowv[t % 3][1]; const float* r3 = rowv[t % 3][2];
    const float ddelta = rscl[par][0], zdz = rscl[par][1];
    const float delta = cscl[t & (NCTX - 1)][sDelta], nkraw = cscl[t & (NCTX - 1)][sNk];
    const float nk = fmaxf(nkraw, eps);
    float dkhx[EPL];
    float kd = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      const int c = e * 32 + lane;
      const float du = ddelta * zt[c] + r3[c] + zt[c] * (zdz / delta);   // ddelta z + A dz
      dkhx[e] = dkS[c] + r1[c] + du;
      kd = fmaf(kh[c], dkhx[e], kd);
    }
    kd = warp_sum(kd);
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      const int c = e * 32 + lane;
      float dkf = nkraw > eps ? (dkhx[e] - kh[c] * kd) / nk : dkhx[e] / eps;
      if (!ident) {
        dkf += gzv[c];
        dkf *= kf[c] > 1.0f ? 1.0f : kf[c];     // phi'(k) from phi(k)
      }
      p.dk[ubase + size_t(t) * D + c] = dkf;
    }
  };
  // gaz = GA z, r1 = A' da and the column partials of GA^T z for token t
  auto products = [&](int t) {
    const float* zt = cvec(t, cZt); const float* da = cvec(t, cDa);
    float a0[R], a1[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      float x0 = 0.f, x1 = 0.f;
#pragma unroll
      for (int c = 0; c < RC; ++c) {
        x0 = fmaf(GA[r][c], zt[col0 + c], x0);
        x1 = fmaf(A[r][c], da[col0 + c], x1);
      }
      a0[r] = x0; a1[r] = x1;
    }
    rows_reduce<R, TX / 2>(a0, lane);
    rows_reduce<R, TX / 2>(a1, lane);
    if (row_writer) { rowv[t % 3][0][row0 + myrow] = a0[0]; rowv[t % 3][1][row0 + myrow] = a1[0]; }
    float cc[RC];
#pragma unroll
    for (int c = 0; c < RC; ++c) {
      float s2 = 0.f;
#pragma unroll
      for (int r = 0; r < R; ++r) s2 = fmaf(GA[r][c], zt[row0 + r], s2);
      cc[c] = s2;
    }
    if constexpr (TX == 16) {
      constexpr int HC = RC / 2;
      const bool up = (lane & 16) != 0;
#pragma unroll
      for (int c = 0; c < HC; ++c) {
        const float send = up ? cc[c] : cc[c + HC];
        const float keep = up ? cc[c + HC] : cc[c];
        part[t & 1][warp][col0 + (up ? HC : 0) + c] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
      }
    } else {
#pragma unroll
      for (int c = 0; c < RC; ++c) part[t & 1][warp][col0 + c] = cc[c];
    }
  };

  constexpr int kHelper = NW;
  // Segment t (one CTA barrier): the matrix warps form dz of token t, r3 = A' dz, the two
  // rank-1 updates, then the products of token t - 1; the helper warp closes token t + 1 and
  // opens token t - 2.  Two loops with the same number of barriers, as on the S side.
  if (warp == kHelper) {
    if (T > 0) {
      fetch_token(T - 1);
      open_token(T - 1);
      fetch_token(T - 2);
      if (T >= 2) open_token(T - 2);
      fetch_token(T - 3);
    }
    cta_sync();
    cta_sync();
    for (int t = T - 1; t >= 0; --t) {
      if (t + 1 <= T - 1) close_token(t + 1);
      if (t - 2 >= 0) {
        open_token(t - 2);
        fetch_token(t - 3);
      }
      cta_sync();
    }
    if (T > 0) close_token(0);
  } else {
    cta_sync();
    if (T > 0) products(T - 1);
    cta_sync();
    for (int t = T - 1; t >= 0; --t) {
      mid_token(t);
      const float* kh = cvec(t, cKh); const float* zt = cvec(t, cZt); const float* da = cvec(t, cDa);
      const float* dz = dzw[warp];
      const float delta = cscl[t & (NCTX - 1)][sDelta];
      float b1[R];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        float x1 = 0.f;
#pragma unroll
        for (int c = 0; c < RC; ++c) x1 = fmaf(A[r][c], dz[col0 + c], x1);
        b1[r] = x1;
      }
      rows_reduce<R, TX / 2>(b1, lane);
      if (row_writer) rowv[t % 3][2][row0 + myrow] = b1[0];
      const float idl = 1.0f / delta;
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const float zr = zt[row0 + r], dadz = da[row0 + r] + dz[row0 + r];
#pragma unroll
        for (int c = 0; c < RC; ++c) {
          GA[r][c] = fmaf(dadz, kh[col0 + c], GA[r][c]);
          A[r][c] = fmaf(zr * idl, zt[col0 + c], A[r][c]);
        }
      }
      __syncwarp();   // this warp's dz copy is rewritten in the next segment
      if (t >= 1) products(t - 1);
      cta_sync();
    }
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
      for (int c = 0; c < RC; ++c)
        if (p.dA0) p.dA0[(size_t(unit) * D + row0 + r) * D + col0 + c] = GA[r][c];
  }
}

}  // namespace vla
