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
// each a CTA of 256 threads per unit holding TWO d x d matrices as R x R blocks (R = d / 16),
// which is what fits d = 128.  The forward recurrence is not re-run here: the chunk kernel
// leaves z_t, e_t, delta_t per token and the final S, A, key sum in the workspace, and both
// sweeps walk the states back by undoing the rank-1 updates (S_{t-1} = S_t - e alpha^T,
// A_{t-1} = A_t + z z^T / delta).  Formulas per token: see vla_backward.cuh.
//
// Both kernels keep a ring of four per-token contexts in shared memory so that opening a
// token (loading its rows, alpha, denominators: nothing that depends on the adjoints) and
// closing one (vector arithmetic on finished products) are done by single warps off the
// path of the matrix work; two CTA barriers per token.
#pragma once

#include "vla_backward.cuh"

namespace vla {


// ------------------------------------------------------------------------------ S side
template <int D, typename TIn>
__global__ void __launch_bounds__(256) vla_backward_s_kernel(const BackwardSplitParams p) {
  constexpr int R = D / 16;
  constexpr int EPL = D / 32;
  constexpr int NCTX = 4;
  enum { cKf = 0, cKh, cQf, cGo, cEt, cAl, cZk, NV };
  enum { sDen = 0, sDenLive, sQal };
  __shared__ float ctx[NCTX][NV][D];
  __shared__ float cscl[NCTX][4];
  __shared__ float rowv[2][2][D];      // y = S' qf, g1 = GS alpha by token parity
  __shared__ float part[2][8][3][D];   // column-sum partials by token parity and warp
  __shared__ float gz[D];              // dL/d(key sum), carried by warp 0

  const int unit = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int ty = tid >> 4, tx = tid & 15;
  const int row0 = ty * R, col0 = tx * R;
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

  float S[R][R], GS[R][R];
#pragma unroll
  for (int r = 0; r < R; ++r)
#pragma unroll
    for (int c = 0; c < R; ++c) {
      const size_t idx = (size_t(unit) * D + row0 + r) * D + col0 + c;
      S[r][c] = p.ST[idx];
      GS[r][c] = p.dS_T ? p.dS_T[idx] : 0.0f;
    }
  for (int j = tid; j < D; j += 256) gz[j] = p.dz_T ? p.dz_T[size_t(unit) * D + j] : 0.0f;

  auto cvec = [&](int t, int which) { return ctx[t & (NCTX - 1)][which]; };
  auto reduce16 = [&](float x) {
#pragma unroll
    for (int off = 8; off >= 1; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
    return x;
  };

  // warp 1 opens tokens two iterations ahead; the rows come from global memory one more ahead
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
  // warp 0: the vector results of token t from its finished products
  auto close_token = [&](int t) {
    const int par = t & 1;
    const float* go = cvec(t, cGo); const float* et = cvec(t, cEt); const float* al = cvec(t, cAl);
    const float* qf = cvec(t, cQf); const float* zkt = cvec(t, cZk);
    const float* yv = rowv[par][0]; const float* g1 = rowv[par][1];
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
      for (int w = 0; w < 8; ++w) {
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

  if (T > 0 && warp == 1) {
    fetch_token(T - 1);
    open_token(T - 1, true);
    fetch_token(T - 2);
    if (T >= 2) open_token(T - 2, false);
    fetch_token(T - 3);
  }
  __syncthreads();

  float dyr[R], der[R];
  for (int t = T - 1; t >= -1; --t) {
    // off the matrix path: warp 0 closes token t + 1, warp 1 opens token t - 2
    if (warp == 0 && t + 1 <= T - 1) close_token(t + 1);
    if (warp == 1 && t - 2 >= 0) {
      open_token(t - 2, false);
      fetch_token(t - 3);
    }
    // ---- phase A: the two rank-1 updates of token t + 1, then the row dots of token t
    if (t + 1 <= T - 1) {
      const float* kh = cvec(t + 1, cKh); const float* qf = cvec(t + 1, cQf);
      const float* et = cvec(t + 1, cEt); const float* al = cvec(t + 1, cAl);
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const float er = et[row0 + r];
#pragma unroll
        for (int c = 0; c < R; ++c) {
          GS[r][c] = fmaf(dyr[r], qf[col0 + c], GS[r][c]);
          GS[r][c] = fmaf(-der[r], kh[col0 + c], GS[r][c]);
          S[r][c] = fmaf(-er, al[col0 + c], S[r][c]);
        }
      }
    }
    if (t < 0) break;
    {
      const float* qf = cvec(t, cQf); const float* al = cvec(t, cAl);
      float a0[R], a1[R];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        float x0 = 0.f, x1 = 0.f;
#pragma unroll
        for (int c = 0; c < R; ++c) {
          x0 = fmaf(S[r][c], qf[col0 + c], x0);
          x1 = fmaf(GS[r][c], al[col0 + c], x1);
        }
        a0[r] = reduce16(x0); a1[r] = reduce16(x1);
      }
      if (tx == 0) {
#pragma unroll
        for (int r = 0; r < R; ++r) { rowv[t & 1][0][row0 + r] = a0[r]; rowv[t & 1][1][row0 + r] = a1[r]; }
      }
    }
    __syncthreads();
    // ---- phase B: column sums S'^T dy, GS^T e, S'^T de (partials per warp)
    {
      const float* go = cvec(t, cGo); const float* et = cvec(t, cEt);
      const float* g1 = rowv[t & 1][1];
      const float den = cscl[t & (NCTX - 1)][sDen], qal = cscl[t & (NCTX - 1)][sQal];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        dyr[r] = go[row0 + r] / den;
        der[r] = g1[row0 + r] + dyr[r] * qal;
      }
      float cc[3][R];
#pragma unroll
      for (int c = 0; c < R; ++c) {
        float s0 = 0.f, s1 = 0.f, s2 = 0.f;
#pragma unroll
        for (int r = 0; r < R; ++r) {
          s0 = fmaf(S[r][c], dyr[r], s0);
          s1 = fmaf(GS[r][c], et[row0 + r], s1);
          s2 = fmaf(S[r][c], der[r], s2);
        }
        cc[0][c] = s0 + __shfl_xor_sync(0xffffffffu, s0, 16);
        cc[1][c] = s1 + __shfl_xor_sync(0xffffffffu, s1, 16);
        cc[2][c] = s2 + __shfl_xor_sync(0xffffffffu, s2, 16);
      }
      if (lane < 16) {
#pragma unroll
        for (int k2 = 0; k2 < 3; ++k2)
#pragma unroll
          for (int c = 0; c < R; ++c) part[t & 1][warp][k2][col0 + c] = cc[k2][c];
      }
    }
    __syncthreads();
  }
  __syncthreads();   // token 0 was closed at the top of the last iteration
#pragma unroll
  for (int r = 0; r < R; ++r)
#pragma unroll
    for (int c = 0; c < R; ++c)
      if (p.dS0) p.dS0[(size_t(unit) * D + row0 + r) * D + col0 + c] = GS[r][c];
  if (p.dz0)
    for (int j = tid; j < D; j += 256) p.dz0[size_t(unit) * D + j] = gz[j];
}

// ------------------------------------------------------------------------------ A side
template <int D, typename TIn>
__global__ void __launch_bounds__(256) vla_backward_a_kernel(const BackwardSplitParams p) {
  constexpr int R = D / 16;
  constexpr int EPL = D / 32;
  constexpr int NCTX = 4;
  enum { cKf = 0, cKh, cZt, cDa, cDkS, cGz, NV };
  enum { sDelta = 0, sKhz, sDaz, sNk };
  __shared__ float ctx[NCTX][NV][D];
  __shared__ float cscl[NCTX][4];
  __shared__ float rowv[2][3][D];      // gaz = GA z, r1 = A' da, r3 = A' dz by token parity
  __shared__ float part[8][D];         // column-sum partials GA^T z per warp
  __shared__ float dzv[2][D];          // dz by token parity
  __shared__ float rscl[2][2];         // ddelta, z.dz by token parity

  const int unit = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int ty = tid >> 4, tx = tid & 15;
  const int row0 = ty * R, col0 = tx * R;
  const bool ident = (p.flags & VLA_FLAG_IDENTITY_MAP) != 0;
  const float eps = p.eps;
  const int T = p.T;
  const size_t ubase = size_t(unit) * size_t(T) * D;
  const TIn* gk = static_cast<const TIn*>(p.k) + ubase;
  const float* zst = p.zst + ubase;
  const float* dst = p.dst + size_t(unit) * T;

  float A[R][R], GA[R][R];
#pragma unroll
  for (int r = 0; r < R; ++r)
#pragma unroll
    for (int c = 0; c < R; ++c) {
      const size_t idx = (size_t(unit) * D + row0 + r) * D + col0 + c;
      A[r][c] = p.AT[idx];
      GA[r][c] = p.dA_T ? p.dA_T[idx] : 0.0f;
    }

  auto cvec = [&](int t, int which) { return ctx[t & (NCTX - 1)][which]; };
  auto reduce16 = [&](float x) {
#pragma unroll
    for (int off = 8; off >= 1; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
    return x;
  };

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
  // warp 0: dz, ddelta of token t from gaz and the column sums (on the path of the updates)
  auto mid_token = [&](int t) {
    const int par = t & 1;
    const float* kh = cvec(t, cKh); const float* zt = cvec(t, cZt); const float* da = cvec(t, cDa);
    const float* gaz = rowv[par][0];
    const float delta = cscl[t & (NCTX - 1)][sDelta], khz = cscl[t & (NCTX - 1)][sKhz];
    const float daz = cscl[t & (NCTX - 1)][sDaz];
    float wx[EPL], c4[EPL];
    float zw = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      const int c = e * 32 + lane;
      float s = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) s += part[w][c];
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
      dzv[par][c] = dz;
      zdz = fmaf(zt[c], dz, zdz);
    }
    zdz = warp_sum(zdz);
    if (lane == 0) { rscl[par][0] = ddelta; rscl[par][1] = zdz; }
  };
  // warp 2: dk of token t
  auto close_token = [&](int t) {
    const int par = t & 1;
    const float* kf = cvec(t, cKf); const float* kh = cvec(t, cKh); const float* zt = cvec(t, cZt);
    const float* dkS = cvec(t, cDkS); const float* gzv = cvec(t, cGz);
    const float* r1 = rowv[par][1]; const float* r3 = rowv[par][2];
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

  if (T > 0 && warp == 1) {
    fetch_token(T - 1);
    open_token(T - 1);
    fetch_token(T - 2);
    if (T >= 2) open_token(T - 2);
    fetch_token(T - 3);
  }
  __syncthreads();

  // iteration t: phase A = [finish token t + 1: r3 = A' dz, the two rank-1 updates] + [row dots
  // and column partials of token t]; phase M = warp 0 forms dz of token t (others: open / close)
  for (int t = T - 1; t >= -1; --t) {
    if (t + 1 <= T - 1) {
      const int tp = t + 1, par = tp & 1;
      const float* kh = cvec(tp, cKh); const float* zt = cvec(tp, cZt); const float* da = cvec(tp, cDa);
      const float* dz = dzv[par];
      const float delta = cscl[tp & (NCTX - 1)][sDelta];
      float b1[R];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        float x1 = 0.f;
#pragma unroll
        for (int c = 0; c < R; ++c) x1 = fmaf(A[r][c], dz[col0 + c], x1);
        b1[r] = reduce16(x1);
      }
      if (tx == 0) {
#pragma unroll
        for (int r = 0; r < R; ++r) rowv[par][2][row0 + r] = b1[r];
      }
      const float idl = 1.0f / delta;
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const float zr = zt[row0 + r], dadz = da[row0 + r] + dz[row0 + r];
#pragma unroll
        for (int c = 0; c < R; ++c) {
          GA[r][c] = fmaf(dadz, kh[col0 + c], GA[r][c]);
          A[r][c] = fmaf(zr * idl, zt[col0 + c], A[r][c]);
        }
      }
    }
    if (t >= 0) {
      const float* zt = cvec(t, cZt); const float* da = cvec(t, cDa);
      float a0[R], a1[R];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        float x0 = 0.f, x1 = 0.f;
#pragma unroll
        for (int c = 0; c < R; ++c) {
          x0 = fmaf(GA[r][c], zt[col0 + c], x0);
          x1 = fmaf(A[r][c], da[col0 + c], x1);
        }
        a0[r] = reduce16(x0); a1[r] = reduce16(x1);
      }
      if (tx == 0) {
#pragma unroll
        for (int r = 0; r < R; ++r) { rowv[t & 1][0][row0 + r] = a0[r]; rowv[t & 1][1][row0 + r] = a1[r]; }
      }
#pragma unroll
      for (int c = 0; c < R; ++c) {
        float s = 0.f;
#pragma unroll
        for (int r = 0; r < R; ++r) s = fmaf(GA[r][c], zt[row0 + r], s);
        s += __shfl_xor_sync(0xffffffffu, s, 16);
        if (lane < 16) part[warp][col0 + c] = s;
      }
    }
    __syncthreads();
    // ---- phase M
    if (warp == 0) {
      if (t >= 0) mid_token(t);
    } else if (warp == 1) {
      if (t - 2 >= 0) {
        open_token(t - 2);
        fetch_token(t - 3);
      }
    } else if (warp == 2) {
      if (t + 1 <= T - 1) close_token(t + 1);
    }
    __syncthreads();
  }
#pragma unroll
  for (int r = 0; r < R; ++r)
#pragma unroll
    for (int c = 0; c < R; ++c)
      if (p.dA0) p.dA0[(size_t(unit) * D + row0 + r) * D + col0 + c] = GA[r][c];
}

}  // namespace vla
