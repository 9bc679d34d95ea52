// VLA forward scan, single-step ("decode") kernel: T = 1 with carried states, thousands of
// (batch, head) units.  One step reads and writes S and A once (2 * 2 * d^2 * 4 bytes per unit)
// for 5 d^2 FMAs: the path is bound by HBM, so the kernel is a copy pipeline with the
// arithmetic of Eqs. "sm", "s-update", "output" done in shared memory on the way through.
//
// A persistent CTA walks its units.  Each unit is two "jobs" -- its A matrix, then its S
// matrix -- that rotate through three d x d shared-memory buffers:
//
//   bulk load (TMA, mbarrier)  ->  compute in place  ->  bulk store (bulk group)
//
// While job m is computed, job m+1 is landing and job m-1 is leaving, so loads and stores
// of different units overlap with each other and with the arithmetic.  The copies are driven
// by one thread of an extra warp, so that the sixteen computing warps never wait for a store to
// drain: it stores a buffer as soon as the job in it is computed, waits until the store has
// read the buffer, and refills it with the job three ahead.  The unit's q, k, v rows and key
// sum travel with its A job.  Every mbarrier wait is bounded.
//
//   A job:  z = A k_hat;  delta = max(1 + k_hat.z, eps);  A <- A - z z^T / delta;
//           alpha = (z/delta) / max(||z||/delta, eps)          (u = k_hat: A_t k_hat = z/delta)
//   S job:  p = S k_hat, r = S q_f;  e = v - p;  S <- S + e alpha^T;
//           o = (r + e (alpha.q_f)) / den                      (= S_t q_f / den)
#pragma once

#include "vla_common.cuh"

namespace vla {

template <int D, typename TIn>
struct DecodeCfg {
  static constexpr int NC = D >= 64 ? 512 : 256;   // computing threads
  static constexpr int NT = NC + 32;         // + the copy warp
  static constexpr int NBUF = 3;
  static constexpr size_t mat_bytes = size_t(D) * D * sizeof(float);
  static constexpr size_t vec_in_bytes = 3 * size_t(D) * sizeof(TIn) + size_t(D) * sizeof(float);  // q,k,v,z0
  static constexpr size_t vec_stage_bytes = (vec_in_bytes + 127) / 128 * 128;
  static constexpr size_t work_floats = 8 * size_t(D) + 16;   // khat qf vf zsum | z alpha e r | scalars
  static constexpr size_t smem_bytes = NBUF * mat_bytes + 2 * vec_stage_bytes +
                                       work_floats * sizeof(float) + (2 * NBUF + 1) * sizeof(uint64_t) + 128;
};

template <int D, typename TIn>
__global__ void __launch_bounds__(DecodeCfg<D, TIn>::NT, 1) vla_decode_kernel(const ScanParams p) {
  using Cfg = DecodeCfg<D, TIn>;
  constexpr int NT = Cfg::NC, NBUF = Cfg::NBUF;   // NT: computing threads
  constexpr int LPR = D / 4;            // lanes that cover one row as float4
  constexpr int RPP = NT / LPR;         // rows per pass of the whole CTA
  constexpr int NPASS = D / RPP;        // passes over a matrix
  static_assert(D % 32 == 0 && LPR <= 32 && D % RPP == 0, "row mapping");

  extern __shared__ __align__(128) unsigned char smem[];
  float* mat = reinterpret_cast<float*>(smem);                                   // [NBUF][D*D]
  unsigned char* vst = smem + NBUF * Cfg::mat_bytes;                             // [2] vector stages
  float* work = reinterpret_cast<float*>(vst + 2 * Cfg::vec_stage_bytes);
  float* khat = work;            // [D]
  float* qf = khat + D;          // [D]
  float* vf = qf + D;            // [D]
  float* zv = vf + D;            // [D]  z = A k_hat
  float* alpha = zv + D;         // [D]
  float* ev = alpha + D;         // [D]  e = v - S k_hat
  float* rv = ev + D;            // [D]  r = S q_f
  float* scal = rv + D;          // [0] 1/den
  uint64_t* mfull = reinterpret_cast<uint64_t*>(
      (reinterpret_cast<uintptr_t>(scal + D + 16) + 7) & ~uintptr_t(7));        // [NBUF]
  uint64_t* mdone = mfull + NBUF;                                                // [NBUF] job computed
  volatile int* abort_flag = reinterpret_cast<volatile int*>(mdone + NBUF);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int rl = tid / LPR;             // row within a pass
  const int c4 = tid % LPR;             // float4 column group
  const bool ident = (p.flags & VLA_FLAG_IDENTITY_MAP) != 0;
  const float eps = p.eps;
  const int nunits = (p.units - int(blockIdx.x) + int(gridDim.x) - 1) / int(gridDim.x);
  const int njobs = 2 * nunits;

  auto wait = [&](uint64_t* bar, uint32_t parity) {
    if (*abort_flag) return;
    if (!mbar_wait_bounded(bar, parity)) {
      *abort_flag = 1;
      if (p.status) atomicCAS(p.status, 0, int(VLA_ERR_DEVICE_TIMEOUT));
    }
  };
  // job m: matrix of unit blockIdx.x + (m/2) * gridDim.x (A for even m, S for odd m)
  auto issue = [&](int m) {
    const int unit = int(blockIdx.x) + (m >> 1) * int(gridDim.x);
    const int b = m % NBUF;
    const bool is_A = (m & 1) == 0;
    uint32_t bytes = uint32_t(Cfg::mat_bytes);
    if (is_A) bytes += 3 * D * sizeof(TIn) + (p.z0 ? D * sizeof(float) : 0);
    mbar_arrive_expect_tx(&mfull[b], bytes);
    bulk_load(mat + size_t(b) * D * D, (is_A ? p.A0 : p.S0) + size_t(unit) * D * D,
              uint32_t(Cfg::mat_bytes), &mfull[b]);
    if (is_A) {
      unsigned char* vs = vst + size_t((m >> 1) & 1) * Cfg::vec_stage_bytes;
      const size_t row = size_t(unit) * D;   // T = 1: one row per unit
      bulk_load(vs + 0 * D * sizeof(TIn), static_cast<const TIn*>(p.q) + row, D * sizeof(TIn), &mfull[b]);
      bulk_load(vs + 1 * D * sizeof(TIn), static_cast<const TIn*>(p.k) + row, D * sizeof(TIn), &mfull[b]);
      bulk_load(vs + 2 * D * sizeof(TIn), static_cast<const TIn*>(p.v) + row, D * sizeof(TIn), &mfull[b]);
      if (p.z0) bulk_load(vs + 3 * D * sizeof(TIn), p.z0 + row, D * sizeof(float), &mfull[b]);
    }
  };

  if (tid == 0) {
    *abort_flag = 0;
    for (int b = 0; b < NBUF; ++b) {
      mbar_init(&mfull[b], 1);
      mbar_init(&mdone[b], 1);
    }
    mbar_init_fence();
  }
  __syncthreads();
  if (warp == NT / 32) {
    // ---- copy warp: one thread owns every bulk load and store of this CTA
    if (lane != 0) return;
    for (int m = 0; m < NBUF && m < njobs; ++m) issue(m);
    for (int m = 0; m < njobs; ++m) {
      const int unit = int(blockIdx.x) + (m >> 1) * int(gridDim.x);
      const int b = m % NBUF;
      wait(&mdone[b], uint32_t(m / NBUF) & 1u);
      if (*abort_flag) break;
      bulk_store(((m & 1) == 0 ? p.A_T : p.S_T) + size_t(unit) * D * D, mat + size_t(b) * D * D,
                 uint32_t(Cfg::mat_bytes));
      bulk_commit();
      if (m + NBUF < njobs) {
        bulk_wait_read<0>();     // the store has read the buffer: refill it
        issue(m + NBUF);
      }
    }
    bulk_wait_all<0>();
    return;
  }
  auto cta_bar = [&]() { asm volatile("bar.sync 1, %0;" ::"n"(Cfg::NC) : "memory"); };

  float delta_inv = 1.0f;   // 1/delta of the current unit
#pragma unroll 1
  for (int m = 0; m < njobs; ++m) {
    const int unit = int(blockIdx.x) + (m >> 1) * int(gridDim.x);
    const int b = m % NBUF;
    const bool is_A = (m & 1) == 0;
    float* M = mat + size_t(b) * D * D;
    wait(&mfull[b], uint32_t(m / NBUF) & 1u);

    if (is_A) {
      // ---- the unit's vectors (warp 0): k_hat, q_f, v, key sum, readout denominator
      if (warp == 0) {
        const unsigned char* vs = vst + size_t((m >> 1) & 1) * Cfg::vec_stage_bytes;
        const TIn* rq = reinterpret_cast<const TIn*>(vs);
        const TIn* rk = rq + D;
        const TIn* rv2 = rk + D;
        const float* rz0 = reinterpret_cast<const float*>(vs + 3 * D * sizeof(TIn));
        float kf[D / 32], qq[D / 32];
        float ss = 0.f, dn = 0.f;
#pragma unroll
        for (int e = 0; e < D / 32; ++e) {
          const int c = e * 32 + lane;
          float kx = load1<TIn>(rk, c), qx = load1<TIn>(rq, c);
          if (!ident) { kx = phi_elu1(kx); qx = phi_elu1(qx); }
          kf[e] = kx; qq[e] = qx;
          ss = fmaf(kx, kx, ss);
          const float zk = (p.z0 ? rz0[c] : 0.0f) + (ident ? 0.0f : kx);
          dn = fmaf(zk, qx, dn);
          if (p.zT) p.zT[size_t(unit) * D + c] = zk;
          qf[c] = qx;
          vf[c] = load1<TIn>(rv2, c);
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
          ss += __shfl_xor_sync(0xffffffffu, ss, off);
          dn += __shfl_xor_sync(0xffffffffu, dn, off);
        }
        const float inv = 1.0f / fmaxf(sqrtf(ss), eps);
#pragma unroll
        for (int e = 0; e < D / 32; ++e) khat[e * 32 + lane] = kf[e] * inv;
        if (lane == 0) scal[0] = ident ? 1.0f : 1.0f / fmaxf(dn, eps);
      }
      cta_bar();
      // ---- z = A k_hat (row dots: LPR lanes per row)
      const float4 k4 = reinterpret_cast<const float4*>(khat)[c4];
#pragma unroll
      for (int ps = 0; ps < NPASS; ++ps) {
        const int row = ps * RPP + rl;
        const float4 a = reinterpret_cast<const float4*>(M + size_t(row) * D)[c4];
        float s = a.x * k4.x + a.y * k4.y + a.z * k4.z + a.w * k4.w;
#pragma unroll
        for (int off = LPR / 2; off >= 1; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
        if (c4 == 0) zv[row] = s;
      }
      cta_bar();
      // ---- delta, ||z||, alpha (every warp forms the two sums itself)
      float kz = 0.f, zz = 0.f;
#pragma unroll
      for (int e = 0; e < D / 32; ++e) {
        const float z = zv[e * 32 + lane];
        kz = fmaf(khat[e * 32 + lane], z, kz);
        zz = fmaf(z, z, zz);
      }
#pragma unroll
      for (int off = 16; off >= 1; off >>= 1) {
        kz += __shfl_xor_sync(0xffffffffu, kz, off);
        zz += __shfl_xor_sync(0xffffffffu, zz, off);
      }
      const float delta = fmaxf(1.0f + kz, eps);
      delta_inv = 1.0f / delta;
      const float sc = delta_inv / fmaxf(sqrtf(zz) * delta_inv, eps);
      if ((p.flags & VLA_FLAG_CHECK_FINITE) && p.status && tid == 0 && !isfinite(kz + zz))
        atomicCAS(p.status, 0, int(VLA_ERR_NONFINITE));
      if (tid < D) alpha[tid] = sc * zv[tid];
      // ---- A <- A - z z^T / delta, in place
      const float4 z4 = reinterpret_cast<const float4*>(zv)[c4];
#pragma unroll
      for (int ps = 0; ps < NPASS; ++ps) {
        const int row = ps * RPP + rl;
        const float f = -zv[row] * delta_inv;
        float4* ap = reinterpret_cast<float4*>(M + size_t(row) * D) + c4;
        float4 a = *ap;
        a.x = fmaf(f, z4.x, a.x); a.y = fmaf(f, z4.y, a.y);
        a.z = fmaf(f, z4.z, a.z); a.w = fmaf(f, z4.w, a.w);
        *ap = a;
      }
    } else {
      // ---- p = S k_hat, r = S q_f; e = v - p
      const float4 k4 = reinterpret_cast<const float4*>(khat)[c4];
      const float4 q4 = reinterpret_cast<const float4*>(qf)[c4];
#pragma unroll
      for (int ps = 0; ps < NPASS; ++ps) {
        const int row = ps * RPP + rl;
        const float4 a = reinterpret_cast<const float4*>(M + size_t(row) * D)[c4];
        float s = a.x * k4.x + a.y * k4.y + a.z * k4.z + a.w * k4.w;
        float r = a.x * q4.x + a.y * q4.y + a.z * q4.z + a.w * q4.w;
#pragma unroll
        for (int off = LPR / 2; off >= 1; off >>= 1) {
          s += __shfl_xor_sync(0xffffffffu, s, off);
          r += __shfl_xor_sync(0xffffffffu, r, off);
        }
        if (c4 == 0) { ev[row] = vf[row] - s; rv[row] = r; }
      }
      cta_bar();
      // ---- o = (r + e (alpha.q_f)) / den
      float aq = 0.f;
#pragma unroll
      for (int e = 0; e < D / 32; ++e) aq = fmaf(alpha[e * 32 + lane], qf[e * 32 + lane], aq);
#pragma unroll
      for (int off = 16; off >= 1; off >>= 1) aq += __shfl_xor_sync(0xffffffffu, aq, off);
      if (tid < D) p.out[size_t(unit) * D + tid] = (rv[tid] + ev[tid] * aq) * scal[0];
      // ---- S <- S + e alpha^T, in place
      const float4 al4 = reinterpret_cast<const float4*>(alpha)[c4];
#pragma unroll
      for (int ps = 0; ps < NPASS; ++ps) {
        const int row = ps * RPP + rl;
        const float f = ev[row];
        float4* sp = reinterpret_cast<float4*>(M + size_t(row) * D) + c4;
        float4 a = *sp;
        a.x = fmaf(f, al4.x, a.x); a.y = fmaf(f, al4.y, a.y);
        a.z = fmaf(f, al4.z, a.z); a.w = fmaf(f, al4.w, a.w);
        *sp = a;
      }
    }
    // ---- the updated matrix is ready to leave: hand the buffer to the copy thread
    fence_async_smem();
    cta_bar();
    if (tid == 0) {
      asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&mdone[b])) : "memory");
    }
  }
}

}  // namespace vla
