// VLA backward pass, token kernel (first correct path): reverse-mode differentiation of the
// forward recurrence (Algorithm 1 without projections; Eqs. "sm", "s-update", "output") for
// u = k_hat.  Written for d in {16, 32, 64}; instantiated for d = 16, which has no chunk kernel
// to leave the stash the two reverse scans of vla_backward_split.cuh start from (they serve
// d >= 32).  The paper gives no backward algorithm; its Corollary on gradient flow (Section 4)
// is about these gradients.
//
// One CTA of 256 threads per (batch, head) unit.  Thread (ty, tx) of a 16 x 16 grid keeps the
// R x R blocks (R = d / 16) of FOUR matrices in registers: S, A and the adjoints GS = dL/dS,
// GA = dL/dA.  The kernel first runs the forward recurrence token by token, leaving z_t, e_t
// and delta_t of every token in the caller's workspace, and then walks the tokens backwards.
// No state is ever stored: the reverse sweep undoes the rank-1 updates
// (S_{t-1} = S_t - e alpha^T, A_{t-1} = A_t + z z^T / delta).
//
// Per token of the reverse sweep, with S' = S_t, A' = A_t (u = k_hat, so a = A' k_hat = z/delta):
//   dy = do/den;  dden = -(S' qf . do)/den^2;  dqf = S'^T dy + dden zk'
//   GS += dy qf^T;  de = GS alpha;  dalpha = GS^T e;  dv = de
//   S = S' - e alpha^T;  dk_hat = -S^T de;  GS -= de k_hat^T
//   da = (dalpha - alpha (alpha.dalpha))/||a||;  GA += da k_hat^T;  dk_hat += A' da
//   dz = -(GA + GA^T) z/delta;  ddelta = z^T GA z/delta^2;  dz += ddelta k_hat
//   A = A' + z z^T/delta;  GA += dz k_hat^T;  dk_hat += ddelta z + A dz
//   dkf = gz + (dk_hat - k_hat (k_hat.dk_hat))/||kf||;  dk = dkf phi'(k);  dq = dqf phi'(q)
// Products with a matrix are row dots (reduced over the 16 threads of a row block with
// shuffles) or column sums (reduced over the 16 row blocks through shared memory); the
// corrections for updates not yet applied (GS += dy qf^T and so on) are scalar multiples of
// known vectors, so all four column sums of a token share one reduction.  Three tokens are in
// flight: while warp 0 does the vector arithmetic of token t, warp 1 prepares the inputs of
// token t - 1 and warp 2 writes dk, dq of token t + 1; four CTA barriers per token.
#pragma once

#include "vla_backward_params.h"
#include "vla_common.cuh"

namespace vla {


__device__ __forceinline__ float bwd_dphi(float x) { return x > 0.0f ? 1.0f : __expf(x); }
__device__ __forceinline__ float bwd_phi(float x) { return x > 0.0f ? x + 1.0f : __expf(x); }

// sum over the lanes of a warp, result in every lane
__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
  return x;
}

template <int D, typename TIn>
__global__ void __launch_bounds__(256) vla_backward_token_kernel(const BackwardParams p) {
  constexpr int R = D / 16;                      // block edge per thread
  constexpr int EPL = D >= 32 ? D / 32 : 1;      // vector elements per lane of warp 0
  __shared__ __align__(16) float vec[14][D];     // named rows below
  __shared__ float ctx[3][8][D];                 // per-token vectors, ring of three tokens
  __shared__ float cscl[3][8];                   // per-token scalars
  __shared__ float res[2][4][D];                 // dk_hat (S part), dqf, A' da, A' dz by token parity
  __shared__ float rscl[2][4];                   // ddelta, z.dz, dden by token parity
  __shared__ float part[8][4][D];                // column-sum partials per warp
  float* kh = vec[0];   float* vv = vec[1];   float* zt = vec[2];   float* pv = vec[3];   // forward sweep
  float* yv = vec[4];   float* g1 = vec[5];   float* gaz = vec[6];
  float* cs = vec[7];   // rows 7..10: the four column sums
  float* dav = vec[11]; float* dzv = vec[12];
  float* zk = vec[13];  // key sum after the forward sweep
  __shared__ float gzbuf[D];
  float* gz = gzbuf;    // dL/d(key sum), carried by the closing warp

  const int unit = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int ty = tid >> 4, tx = tid & 15;
  const int row0 = ty * R, col0 = tx * R;
  const bool ident = (p.flags & VLA_FLAG_IDENTITY_MAP) != 0;
  const float eps = p.eps;
  const int T = p.T;
  const TIn* gq = static_cast<const TIn*>(p.q) + size_t(unit) * T * D;
  const TIn* gk = static_cast<const TIn*>(p.k) + size_t(unit) * T * D;
  const TIn* gv = static_cast<const TIn*>(p.v) + size_t(unit) * T * D;
  const float* gdo = p.d_out + size_t(unit) * T * D;
  float* zst = p.zst + size_t(unit) * T * D;
  float* est = p.est + size_t(unit) * T * D;
  float* dst = p.dst + size_t(unit) * T;

  float S[R][R], A[R][R], GS[R][R], GA[R][R];
#pragma unroll
  for (int r = 0; r < R; ++r)
#pragma unroll
    for (int c = 0; c < R; ++c) {
      const size_t idx = (size_t(unit) * D + row0 + r) * D + col0 + c;
      S[r][c] = p.S0 ? p.S0[idx] : 0.0f;
      A[r][c] = p.A0 ? p.A0[idx] : ((row0 + r == col0 + c) ? 1.0f / p.lambda : 0.0f);
      GS[r][c] = p.dS_T ? p.dS_T[idx] : 0.0f;
      GA[r][c] = p.dA_T ? p.dA_T[idx] : 0.0f;
    }
  for (int j = tid; j < D; j += 256) {
    zk[j] = p.z0 ? p.z0[size_t(unit) * D + j] : 0.0f;
    gz[j] = p.dz_T ? p.dz_T[size_t(unit) * D + j] : 0.0f;
  }
  __syncthreads();

  // row dots of up to three (matrix, vector) pairs at once: result of row row0 + r in lane
  // tx == 0 of the row block
  auto reduce16 = [&](float x) {
#pragma unroll
    for (int off = 8; off >= 1; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
    return x;
  };

  // ================================================================ forward sweep
  // warp 0 reads the rows of token t + 1 from global memory while token t is processed
  float nxk[EPL], nxv[EPL];
  auto fetch_kv = [&](int t) {
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      const int c = e * 32 + lane;
      nxk[e] = 0.f; nxv[e] = 0.f;
      if (c < D && t < T) {
        nxk[e] = load1<TIn>(gk, size_t(t) * D + c);
        nxv[e] = load1<TIn>(gv, size_t(t) * D + c);
      }
    }
  };
  if (warp == 0) fetch_kv(0);
  for (int t = 0; t < T; ++t) {
    if (warp == 0) {
      float kx[EPL];
      float ss = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        const int c = e * 32 + lane;
        float x = 0.f;
        if (c < D) {
          x = nxk[e];
          if (!ident) x = bwd_phi(x);
          vv[c] = nxv[e];
        }
        kx[e] = x;
        ss = fmaf(x, x, ss);
      }
      fetch_kv(t + 1);
      ss = warp_sum(ss);
      const float inv = 1.0f / fmaxf(sqrtf(ss), eps);
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        const int c = e * 32 + lane;
        if (c < D) {
          kh[c] = kx[e] * inv;
          if (!ident) {
            zk[c] += kx[e];
            // the reverse sweep restarts its walk back of the key sum from these (a walk from
            // the final sum alone would cancel catastrophically at the early tokens)
            if ((t & 15) == 15) p.zkc[(size_t(unit) * ((T + 15) / 16) + size_t(t >> 4)) * D + c] = zk[c];
          }
        }
      }
    }
    __syncthreads();
    {   // z = A k_hat, p = S k_hat
      float pz[R], ps[R];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        float a = 0.f, s = 0.f;
#pragma unroll
        for (int c = 0; c < R; ++c) {
          const float kc = kh[col0 + c];
          a = fmaf(A[r][c], kc, a);
          s = fmaf(S[r][c], kc, s);
        }
        pz[r] = reduce16(a);
        ps[r] = reduce16(s);
      }
      if (tx == 0) {
#pragma unroll
        for (int r = 0; r < R; ++r) { zt[row0 + r] = pz[r]; pv[row0 + r] = ps[r]; }
      }
    }
    __syncthreads();
    {
      float kz = 0.f, zz = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        const int c = e * 32 + lane;
        if (c < D) { kz = fmaf(kh[c], zt[c], kz); zz = fmaf(zt[c], zt[c], zz); }
      }
      kz = warp_sum(kz);
      zz = warp_sum(zz);
      const float delta = fmaxf(1.0f + kz, eps);
      const float idl = 1.0f / delta;
      const float sc = idl / fmaxf(sqrtf(zz) * idl, eps);
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const float zr = zt[row0 + r], er = vv[row0 + r] - pv[row0 + r];
#pragma unroll
        for (int c = 0; c < R; ++c) {
          const float zc = zt[col0 + c];
          A[r][c] = fmaf(-zr * idl, zc, A[r][c]);
          S[r][c] = fmaf(er, sc * zc, S[r][c]);
        }
      }
      if (tid < D) {
        zst[size_t(t) * D + tid] = zt[tid];
        est[size_t(t) * D + tid] = vv[tid] - pv[tid];
      }
      if (tid == 0) dst[t] = delta;
    }
    __syncthreads();   // kh, vv, zt, pv are rewritten for the next token
  }

  // ================================================================ reverse sweep
  // Three tokens are alive at a time, each in its own context (ring of three):
  //   token t     : the matrix work of this iteration (row dots, column sums, warp 0's vectors)
  //   token t - 1 : being opened by warp 1 (its inputs, alpha, denominator: nothing of this
  //                 depends on the adjoints)
  //   token t + 1 : being closed by warp 2 (dk, dq from the finished row dots)
  // so that only warp 0's vector arithmetic of token t sits between the CTA barriers.
  auto cvec = [&](int t, int which) { return ctx[((t % 3) + 3) % 3][which]; };
  auto cscal = [&](int t) { return cscl[((t % 3) + 3) % 3]; };
  enum { cKf = 0, cKh, cQf, cGo, cZt, cEt, cAl, cZk };
  enum { sDen = 0, sDenLive, sQal, sDelta, sNa, sNk };
  enum { rDdelta = 0, rZdz, rDden };

  // rows of the token that warp 1 opens next, read from global memory one iteration ahead
  float pk[EPL], pq[EPL], pz[EPL], pe[EPL], pg[EPL];
  float pdelta = 1.0f;
  auto fetch_token = [&](int t) {
    if (t < 0) return;
    pdelta = dst[t];
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      const int c = e * 32 + lane;
      pk[e] = pq[e] = pz[e] = pe[e] = pg[e] = 0.f;
      if (c < D) {
        pk[e] = load1<TIn>(gk, size_t(t) * D + c);
        pq[e] = load1<TIn>(gq, size_t(t) * D + c);
        pz[e] = zst[size_t(t) * D + c];
        pe[e] = est[size_t(t) * D + c];
        pg[e] = gdo[size_t(t) * D + c];
      }
    }
  };
  // one warp: context of token t from the fetched rows; zk_src = key sum INCLUDING token t
  // (for t = T - 1 the forward sweep's result, else the context of t + 1 minus its phi(k))
  auto open_token = [&](int t, bool last) {
    float* okf = cvec(t, cKf); float* okh = cvec(t, cKh); float* oqf = cvec(t, cQf);
    float* ogo = cvec(t, cGo); float* ozt = cvec(t, cZt); float* oet = cvec(t, cEt);
    float* oal = cvec(t, cAl); float* ozk = cvec(t, cZk);
    const float* nzk = last ? zk : cvec(t + 1, cZk);
    const float* nkf = cvec(t + 1, cKf);
    const float delta = pdelta;
    float zx[EPL], kx[EPL], qx[EPL];
    float ss = 0.f, zz = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      const int c = e * 32 + lane;
      float kk = 0.f, qq = 0.f, z = 0.f;
      if (c < D) {
        kk = pk[e]; qq = pq[e];
        if (!ident) { kk = bwd_phi(kk); qq = bwd_phi(qq); }
        z = pz[e];
        ogo[c] = pg[e];
        oet[c] = pe[e];
        ozt[c] = z;
        okf[c] = kk;
        oqf[c] = qq;
      }
      kx[e] = kk; qx[e] = qq; zx[e] = z;
      ss = fmaf(kk, kk, ss);
      zz = fmaf(z, z, zz);
    }
    ss = warp_sum(ss);
    zz = warp_sum(zz);
    const float nk = fmaxf(sqrtf(ss), eps);
    const float idl = 1.0f / delta;
    const float na_raw = sqrtf(zz) * idl;          // ||a||, a = z / delta
    const float sc = idl / fmaxf(na_raw, eps);
    float dn = 0.f, qa = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      const int c = e * 32 + lane;
      if (c < D) {
        okh[c] = kx[e] / nk;
        oal[c] = sc * zx[e];
        float zkc = last ? nzk[c] : (ident ? nzk[c] : nzk[c] - nkf[c]);
        if (!ident && !last && (t & 15) == 15)
          zkc = __ldcg(p.zkc + (size_t(unit) * ((T + 15) / 16) + size_t(t >> 4)) * D + c);
        ozk[c] = zkc;
        dn = fmaf(zkc, qx[e], dn);
        qa = fmaf(qx[e], sc * zx[e], qa);
      }
    }
    dn = warp_sum(dn);
    qa = warp_sum(qa);
    if (lane == 0) {
      float* os = cscal(t);
      os[sDen] = ident ? 1.0f : fmaxf(dn, eps);
      os[sDenLive] = (ident || dn < eps) ? 0.0f : 1.0f;
      os[sQal] = qa;
      os[sDelta] = delta;
      os[sNa] = na_raw;
      os[sNk] = sqrtf(ss);
    }
  };
  // one warp: dk, dq of token t from its finished products
  auto close_token = [&](int t) {
    const int par = t & 1;
    const float* ckf = cvec(t, cKf); const float* ckh = cvec(t, cKh); const float* cqf = cvec(t, cQf);
    const float* czt = cvec(t, cZt);
    const float* cdkS = res[par][0]; const float* cdqf = res[par][1];
    const float* cr1 = res[par][2]; const float* cr3 = res[par][3];
    const float ddelta = rscl[par][rDdelta], zdz = rscl[par][rZdz], dden = rscl[par][rDden];
    const float delta = cscal(t)[sDelta], nkraw = cscal(t)[sNk];
    const float nk = fmaxf(nkraw, eps);
    float dkhx[EPL];
    float kd = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      const int c = e * 32 + lane;
      dkhx[e] = 0.f;
      if (c < D) {
        const float du = ddelta * czt[c] + cr3[c] + czt[c] * (zdz / delta);   // ddelta z + A dz
        dkhx[e] = cdkS[c] + cr1[c] + du;
        kd = fmaf(ckh[c], dkhx[e], kd);
      }
    }
    kd = warp_sum(kd);
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      const int c = e * 32 + lane;
      if (c < D) {
        float dkf = nkraw > eps ? (dkhx[e] - ckh[c] * kd) / nk : dkhx[e] / eps;
        float dq = cdqf[c];
        if (!ident) {
          gz[c] += dden * cqf[c];
          dkf += gz[c];
          // phi'(x) from phi(x): 1 where phi > 1 (x > 0), phi itself otherwise (exp(x))
          dkf *= ckf[c] > 1.0f ? 1.0f : ckf[c];
          dq *= cqf[c] > 1.0f ? 1.0f : cqf[c];
        }
        p.dk[(size_t(unit) * T + t) * D + c] = dkf;
        p.dq[(size_t(unit) * T + t) * D + c] = dq;
      }
    }
  };

  if (T > 0) {
    if (warp == 1) {
      fetch_token(T - 1);
      open_token(T - 1, true);
      fetch_token(T - 2);
    }
    __syncthreads();
  }

  float dyr[R], der[R];     // dy and de of the token in flight, rows of this thread
  for (int t = T - 1; t >= -1; --t) {
    // ---- phase A: finish token t + 1 (row dots A' da, A' dz; the four rank-1 updates), then
    //      the three row dots of token t
    if (t + 1 <= T - 1) {
      const int tp = t + 1, par = tp & 1;
      const float* kh = cvec(tp, cKh); const float* qf = cvec(tp, cQf); const float* zt = cvec(tp, cZt);
      const float* et = cvec(tp, cEt); const float* al = cvec(tp, cAl);
      const float delta = cscal(tp)[sDelta];
      float b0[R], b1[R];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        float x0 = 0.f, x1 = 0.f;
#pragma unroll
        for (int c = 0; c < R; ++c) {
          x0 = fmaf(A[r][c], dav[col0 + c], x0);
          x1 = fmaf(A[r][c], dzv[col0 + c], x1);
        }
        b0[r] = reduce16(x0); b1[r] = reduce16(x1);
      }
      if (tx == 0) {
#pragma unroll
        for (int r = 0; r < R; ++r) { res[par][2][row0 + r] = b0[r]; res[par][3][row0 + r] = b1[r]; }
      }
      const float idl = 1.0f / delta;
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const float er = et[row0 + r], zr = zt[row0 + r], dadz = dav[row0 + r] + dzv[row0 + r];
#pragma unroll
        for (int c = 0; c < R; ++c) {
          const float khc = kh[col0 + c];
          GS[r][c] = fmaf(dyr[r], qf[col0 + c], GS[r][c]);
          GS[r][c] = fmaf(-der[r], khc, GS[r][c]);
          S[r][c] = fmaf(-er, al[col0 + c], S[r][c]);
          GA[r][c] = fmaf(dadz, khc, GA[r][c]);
          A[r][c] = fmaf(zr * idl, zt[col0 + c], A[r][c]);
        }
      }
    }
    if (t >= 0) {
      const float* qf = cvec(t, cQf); const float* zt = cvec(t, cZt); const float* al = cvec(t, cAl);
      float a0[R], a1[R], a2[R];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        float x0 = 0.f, x1 = 0.f, x2 = 0.f;
#pragma unroll
        for (int c = 0; c < R; ++c) {
          x0 = fmaf(S[r][c], qf[col0 + c], x0);
          x1 = fmaf(GS[r][c], al[col0 + c], x1);
          x2 = fmaf(GA[r][c], zt[col0 + c], x2);
        }
        a0[r] = reduce16(x0); a1[r] = reduce16(x1); a2[r] = reduce16(x2);
      }
      if (tx == 0) {
#pragma unroll
        for (int r = 0; r < R; ++r) { yv[row0 + r] = a0[r]; g1[row0 + r] = a1[r]; gaz[row0 + r] = a2[r]; }
      }
    }
    __syncthreads();
    if (t < 0) {   // epilogue: only token 0 is left to close
      if (warp == 2 && T > 0) close_token(0);
      break;
    }
    const float* kh = cvec(t, cKh); const float* qf = cvec(t, cQf); const float* go = cvec(t, cGo);
    const float* zt = cvec(t, cZt); const float* et = cvec(t, cEt); const float* al = cvec(t, cAl);
    const float* zkt = cvec(t, cZk);
    const float den = cscal(t)[sDen], qal = cscal(t)[sQal], delta = cscal(t)[sDelta];
    // ---- phase B: column sums S'^T dy, GS^T e, S'^T de, GA^T z (partials per warp)
    {
#pragma unroll
      for (int r = 0; r < R; ++r) {
        dyr[r] = go[row0 + r] / den;
        der[r] = g1[row0 + r] + dyr[r] * qal;      // (GS + dy qf^T) alpha
      }
      float cc[4][R];
#pragma unroll
      for (int c = 0; c < R; ++c) {
        float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
        for (int r = 0; r < R; ++r) {
          s0 = fmaf(S[r][c], dyr[r], s0);
          s1 = fmaf(GS[r][c], et[row0 + r], s1);
          s2 = fmaf(S[r][c], der[r], s2);
          s3 = fmaf(GA[r][c], zt[row0 + r], s3);
        }
        cc[0][c] = s0 + __shfl_xor_sync(0xffffffffu, s0, 16);
        cc[1][c] = s1 + __shfl_xor_sync(0xffffffffu, s1, 16);
        cc[2][c] = s2 + __shfl_xor_sync(0xffffffffu, s2, 16);
        cc[3][c] = s3 + __shfl_xor_sync(0xffffffffu, s3, 16);
      }
      if (lane < 16) {
#pragma unroll
        for (int k2 = 0; k2 < 4; ++k2)
#pragma unroll
          for (int c = 0; c < R; ++c) part[warp][k2][col0 + c] = cc[k2][c];
      }
    }
    __syncthreads();
    // ---- phase C: add the eight partials
    for (int j = tid; j < 4 * D; j += 256) {
      const int k2 = j / D, c = j % D;
      float s = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) s += part[w][k2][c];
      cs[k2 * D + c] = s;
    }
    __syncthreads();
    // ---- phase D: warp 0 forms da, dz, dqf, dk_hat (S part) of token t; warp 1 opens token
    //      t - 1; warp 2 closes token t + 1
    if (warp == 0) {
      const int par = t & 1;
      float* dkS = res[par][0]; float* dqf = res[par][1];
      const bool den_live = cscal(t)[sDenLive] != 0.0f;
      const float na = cscal(t)[sNa];
      float odo = 0.f, ede = 0.f, dye = 0.f;
      float dex[EPL];
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        const int c = e * 32 + lane;
        dex[e] = 0.f;
        if (c < D) {
          const float dy = go[c] / den;
          dex[e] = g1[c] + dy * qal;
          odo = fmaf(yv[c], go[c], odo);
          ede = fmaf(et[c], dex[e], ede);
          dye = fmaf(dy, et[c], dye);
        }
      }
      odo = warp_sum(odo); ede = warp_sum(ede); dye = warp_sum(dye);
      const float dden = den_live ? -odo / (den * den) : 0.0f;
      float dalx[EPL];
      float adal = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        const int c = e * 32 + lane;
        dalx[e] = 0.f;
        if (c < D) {
          dqf[c] = cs[0 * D + c] + dden * zkt[c];
          dalx[e] = cs[1 * D + c] + qf[c] * dye;               // (GS + dy qf^T)^T e
          dkS[c] = -(cs[2 * D + c] - al[c] * ede);             // -(S' - e alpha^T)^T de
          adal = fmaf(al[c], dalx[e], adal);
        }
      }
      adal = warp_sum(adal);
      float dax[EPL];
      float daz = 0.f, khz = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        const int c = e * 32 + lane;
        dax[e] = 0.f;
        if (c < D) {
          dax[e] = na > eps ? (dalx[e] - al[c] * adal) / na : dalx[e] / eps;
          daz = fmaf(dax[e], zt[c], daz);
          khz = fmaf(kh[c], zt[c], khz);
        }
      }
      daz = warp_sum(daz); khz = warp_sum(khz);
      float wx[EPL];
      float zw = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        const int c = e * 32 + lane;
        wx[e] = 0.f;
        if (c < D) {
          wx[e] = gaz[c] + dax[e] * khz;                       // (GA + da k_hat^T) z
          zw = fmaf(zt[c], wx[e], zw);
        }
      }
      zw = warp_sum(zw);
      const bool delta_live = (1.0f + khz) >= eps;
      const float ddelta = delta_live ? zw / (delta * delta) : 0.0f;
      float zdz = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        const int c = e * 32 + lane;
        if (c < D) {
          const float dz = -(wx[e] + cs[3 * D + c] + kh[c] * daz) / delta + ddelta * kh[c];
          dzv[c] = dz;
          dav[c] = dax[e];
          zdz = fmaf(zt[c], dz, zdz);
          p.dv[(size_t(unit) * T + t) * D + c] = dex[e];
        }
      }
      zdz = warp_sum(zdz);
      if (lane == 0) { rscl[par][rDdelta] = ddelta; rscl[par][rZdz] = zdz; rscl[par][rDden] = dden; }
    } else if (warp == 1) {
      if (t >= 1) {
        open_token(t - 1, false);
        fetch_token(t - 2);
      }
    } else if (warp == 2) {
      if (t + 1 <= T - 1) close_token(t + 1);
    }
    __syncthreads();
  }
  __syncthreads();

  // ---- gradients of the initial states
#pragma unroll
  for (int r = 0; r < R; ++r)
#pragma unroll
    for (int c = 0; c < R; ++c) {
      const size_t idx = (size_t(unit) * D + row0 + r) * D + col0 + c;
      if (p.dS0) p.dS0[idx] = GS[r][c];
      if (p.dA0) p.dA0[idx] = GA[r][c];
    }
  if (p.dz0)
    for (int j = tid; j < D; j += 256) p.dz0[size_t(unit) * D + j] = gz[j];
  if ((p.flags & VLA_FLAG_CHECK_FINITE) && p.status && tid == 0) {
    float s = 0.f;
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
      for (int c = 0; c < R; ++c) s += GS[r][c] + GA[r][c];
    if (!isfinite(s)) atomicCAS(p.status, 0, int(VLA_ERR_NONFINITE));
  }
}

}  // namespace vla
