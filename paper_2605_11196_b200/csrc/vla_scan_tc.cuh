// VLA forward scan, tensor-core form of the chunk kernel (d = 128, u = k_hat, no refresh).
//
// The 16-token chunk algebra of vla_scan_chunk.cuh (Section 3.3's recurrence in its exact
// Woodbury / LDL^T form; Section 3.4's observation that the chunked recurrence is a chain of
// dense products) with the d x d work on the 5th-generation tensor cores:
//
//   * both states live in tensor memory as fp32 accumulators (A: columns 0..127, S: 128..255,
//     lane = row), so a rank-16 update  A -= Z diag(1/delta) Z^T,  S += E' Z^T  is a handful
//     of tcgen05.mma instructions that accumulate straight into the state;
//   * the chunk products  Z0 = A K^T,  P = S K^T,  R0 = S Q^T  take the state as the
//     tensor-memory operand of the MMA;
//   * fp32 accuracy out of TF32 products: every operand x is used as hi(x) + lo(x), hi = the
//     upper 19 bits (what the tensor core reads of a 32-bit word), lo = x - hi (exact), and a
//     product is hi*hi + hi*lo + lo*hi (the dropped lo*lo term is ~2^-22 relative).  For the
//     state the lo part is recomputed once per chunk from tensor memory into a scratch region
//     of 128 columns that the two states take turns in;
//   * the 16 x 16 factorisation, the two row substitutions, the Gram matrices and the input
//     prep stay on the fp32 pipe, as in the FMA kernel.
//
// One CTA per unit, 12 warps: group A (warps 0-3) owns the A chain, group S (warps 4-7) the
// S chain and the readout, group P (warps 8-9) the TMA ring and the input prep; lane 0 of
// warps 10 and 11 issues the MMAs of group A and of group S.  Thread g of
// groups A and S owns row g of its state (tensor-memory lane g).  Every mbarrier wait is
// bounded; on expiry the CTA records VLA_ERR_DEVICE_TIMEOUT, stops waiting, frees its tensor
// memory and runs to its end.
//
// Operand layouts in shared memory (K-major, no swizzle, 8 x 16-byte core matrices): an
// operand with R rows and K columns is the float4 array [K/4][R], i.e. element (r, k) at
// float4 index (k/4) * R + r, component k%4.  Descriptor: stride (8-row groups) 128 B,
// leading (next 4 k) 16*R B; one MMA (K = 8) advances the start address by 32*R B.
#pragma once

#include "vla_common.cuh"
#include "vla_launch.h"
#include "vla_umma.cuh"

namespace vla {

// Unrolling, as measured: the chunk loop of the four roles is straight-line code that is fetched
// anew every chunk, so code size counts.  The Gram loops stay fully unrolled (rolled: 5 KB less,
// 25 % slower), the prep group's passes take two steps at a time (it has time to spare), the chunk
// loops themselves are not unrolled (twice: same work, 40 % slower).
constexpr int kTcGramUnroll = 4;
constexpr int kTcPrepUnroll = 2;
constexpr int kTcLoopUnroll = 1;
// ---------------------------------------------------------------- configuration
template <typename TIn>
struct TcCfg {
  static constexpr int D = 128;
  static constexpr int C = 16;                  // tokens per chunk
  static constexpr int NG = 128;                // threads of group A and of group S
  static constexpr int NP = 64;                 // threads of the prep group
  static constexpr int NI = 64;                 // two warps whose lane 0 issues the MMAs of group A / group S
  static constexpr int NT = 2 * NG + NP + NI;
  static constexpr int NSTAGE = sizeof(TIn) == 2 ? 2 : 1;   // raw q/k/v chunks in flight
  static constexpr int KRING = 2;               // widened chunks (prep -> A, S)
  static constexpr int RING = 1;                // Z / Gu / HT / sc slots (A -> S)
  static constexpr int CP = C + 4;              // padded row of the small C x C matrices
  static constexpr int VP = D + 4;              // padded row of the widened k_hat, q_f, v chunks
  // tensor-memory columns
  static constexpr uint32_t COL_A = 0, COL_S = 128, COL_LO = 256, COL_Z0 = 384, COL_PR = 432;   // 48, 64
  static constexpr uint32_t TMEM_COLS = 512;
  // shared memory (bytes)
  static constexpr size_t raw_bytes = size_t(NSTAGE) * 3 * C * D * sizeof(TIn);
  static constexpr int KQR = 64;                // operand rows of a chunk: hi(k_hat) | hi(q_f) | lo(k_hat) | lo(q_f)
  static constexpr size_t kq_bytes = size_t(KQR) * D * 4;           // [32][64] float4
  static constexpr size_t kp_bytes = size_t(2) * C * VP * 4;        // k_hat, q_f as plain fp32 rows [C][VP]
  static constexpr size_t kslot_bytes = kq_bytes + kp_bytes + size_t(C) * VP * 4 + 4 * C * 4;   // + v, nrm, 1/den, means of k_hat and q_f
  static constexpr size_t op16_bytes = size_t(D) * C * 4;           // [4][128] float4: a 128 x 16 operand
  static constexpr size_t zslot_bytes = 2 * op16_bytes + (2 * C * CP + 2 * C) * 4;  // Z, lo(Z), GuT, HT, sc, sums of z_t
  static constexpr size_t a_bytes = 2 * op16_bytes + size_t(C) * D * 4 + (2 * C * CP + 8 * C + 3 * C) * 4 + 64;   // (+ 64: keeps what follows 128-byte aligned)
  //   -Z/delta, lo | Z0 / Z rows [C][D] | W, L | N2p[4][C], ZSp[4][C] | delta, 1/delta, -1/delta
  static constexpr size_t s_bytes = 2 * op16_bytes + 2 * size_t(C) * D * 4;         // E', lo(E') | out stage [2]
  static constexpr size_t p_bytes = 2 * C * 4;                                      // denp[2][C]
  static constexpr int NBAR = NSTAGE + 2 * KRING + 2 * RING + 9;
  static constexpr size_t smem_bytes = raw_bytes + KRING * kslot_bytes + RING * zslot_bytes + a_bytes + s_bytes +
                                       p_bytes + NBAR * 8 + 16 + 128;
};

// G[i][j] = X[i] . Y[j] for two sets of 16 plain rows of length 128 (row stride XS and 128); result
// rows have stride CP.  4x4 output tiles, 8 threads per tile splitting the 128 index.
template <int CP, int XS>
__device__ __forceinline__ void gram16_tc(const float* X, const float* Y, float* G, int g) {
  constexpr int P = 8;
  constexpr int kGramUnroll = kTcGramUnroll;
  const int tile = g / P, part = g % P;
  const int i0 = (tile >> 2) * 4, j0 = (tile & 3) * 4;
  float2 w2[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) w2[i] = make_float2(0.f, 0.f);
#pragma unroll kGramUnroll   // rolled: the chunk loop of all roles together has to stay in the instruction cache
  for (int step = 0; step < 4; ++step) {
    const int f = step * P + part;
    float4 a[4], b[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      a[i] = reinterpret_cast<const float4*>(X + (i0 + i) * XS)[f];
      b[i] = reinterpret_cast<const float4*>(Y + (j0 + i) * 128)[f];
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        w2[4 * i + j] = ffma2(make_float2(a[i].x, a[i].y), make_float2(b[j].x, b[j].y), w2[4 * i + j]);
        w2[4 * i + j] = ffma2(make_float2(a[i].z, a[i].w), make_float2(b[j].z, b[j].w), w2[4 * i + j]);
      }
  }
  float w[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) w[i] = w2[i].x + w2[i].y;
  const int base = tile16_reduce_scatter<P>(w, part);
  tile16_store<P, CP>(G, i0, j0, w, base);
}

// Hand-over flags of the balanced schedule (see SchedParams): one word per unit and slot.
static __device__ unsigned int g_tc_sched_flags[kSchedSlots * kSchedMaxUnits];

// BALANCED: a persistent grid of one CTA per SM; the units' chunk sequences, laid end to end, are
// cut into equal pieces, and a unit that straddles a cut is started by one CTA (first thing it
// does) and finished by the next (last thing it does), with S, A, the key sum handed over through
// the caller's S_T / A_T / zT and a release/acquire flag per unit.
// TM: q, k, v, out are [B, T, H, d]: the 16 rows of a chunk are H * d apart and move as one tiled
// TMA request per array (rows past T arrive as zeros; the store clips them).
// STASH: the launch also leaves z_t, e_t, delta_t of every token and the key sum after every
// chunk in global memory (the forward of a backward pass); an instantiation of its own, so that
// the plain forward carries none of it.
template <typename TIn, bool BALANCED, bool TM = false, bool STASH = false>
__global__ void __launch_bounds__(TcCfg<TIn>::NT, 1) vla_scan_tc_kernel(
    const ScanParams p, const SchedParams sp, const __grid_constant__ typename ChunkMapsArg<TM>::type maps) {
  using Cfg = TcCfg<TIn>;
  constexpr int D = Cfg::D, C = Cfg::C, NG = Cfg::NG, NP = Cfg::NP, CP = Cfg::CP, VP = Cfg::VP;
  constexpr int NSTAGE = Cfg::NSTAGE, KRING = Cfg::KRING, RING = Cfg::RING;
  constexpr int kLoopUnroll = kTcLoopUnroll;
  constexpr int kPrepUnroll = kTcPrepUnroll;

  extern __shared__ __align__(128) unsigned char smem[];
  TIn* raw = reinterpret_cast<TIn*>(smem);
  unsigned char* kslots = smem + Cfg::raw_bytes;
  unsigned char* zslots = kslots + KRING * Cfg::kslot_bytes;
  unsigned char* abase = zslots + RING * Cfg::zslot_bytes;
  unsigned char* sbase = abase + Cfg::a_bytes;
  unsigned char* pbase = sbase + Cfg::s_bytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>((reinterpret_cast<uintptr_t>(pbase + Cfg::p_bytes) + 15) & ~uintptr_t(15));
  uint64_t* raw_full = bars;                      // [NSTAGE] TMA filled a raw stage
  uint64_t* k_full = raw_full + NSTAGE;           // [KRING] prep published a widened chunk
  uint64_t* k_empty = k_full + KRING;             // [KRING] groups A and S are done with it
  uint64_t* z_full = k_empty + KRING;             // [RING] group A published Z, Gu, HT, sc
  uint64_t* z_empty = z_full + RING;              // [RING] both rank-16 updates have read Z
  uint64_t* b_z0 = z_empty + RING;                // Z0 products complete
  uint64_t* b_aupd = b_z0 + 1;                    // update of A complete
  uint64_t* b_pr = b_aupd + 1;                    // P / R0 products complete
  uint64_t* b_supd = b_pr + 1;                    // update of S complete
  uint64_t* b_lo_s = b_supd + 1;                  // group A's products have read the lo scratch: S may fill it
  uint64_t* b_lo_a = b_lo_s + 1;                  // group S's products have read the lo scratch: A may fill it
  uint64_t* b_lo_rdy_a = b_lo_a + 1;              // group A has written the lo scratch
  uint64_t* b_lo_rdy_s = b_lo_rdy_a + 1;          // group S has written the lo scratch
  uint64_t* b_ep_rdy = b_lo_rdy_s + 1;            // group S has written E' and its lo part
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(b_ep_rdy + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x;
  // The warp index is read from lane 0 so that the compiler sees it as uniform over the warp:
  // the role branches below are then uniform branches, and the warp shuffles inside them are
  // compiled as plain shuffles (as code the compiler takes for divergent they are several
  // times longer, and the chunk loop then no longer fits the instruction cache).
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
  constexpr int WA = NG / 32, WP = NP / 32;
  const int grp = warp < WA ? 0 : (warp < 2 * WA ? 1 : (warp < 2 * WA + WP ? 2 : 3));   // A, S, prep, MMA issue
  const int gw = warp - (grp == 3 ? 2 * WA + WP : grp * WA);   // warp within its group
  const int lane = tid & 31;
  const int g = gw * 32 + lane;                                // thread within its group
  const bool ident = (p.flags & VLA_FLAG_IDENTITY_MAP) != 0;
  const float eps = p.eps;
  const int nch_unit = (p.T + C - 1) / C;   // chunks per unit
  // the piece of work in hand (set at the top of the piece loop): tokens [t_begin, t_begin + T)
  // of `unit`, nchunks chunks
  int unit = 0, T = 0, nchunks = 0, t_begin = 0;
  bool from_handoff = false;
  unsigned int* sched_flags = g_tc_sched_flags + size_t(sp.epoch % kSchedSlots) * kSchedMaxUnits;

  const uint32_t wait_limit = p.wait_limit ? p.wait_limit : kWaitProbeLimit;
  auto wait = [&](uint64_t* bar, uint32_t parity) {
    // one probe costs some 170 clk even when the phase is complete, a look at the abort flag
    // 90 more: the common case (complete) pays for the probe only
    if (mbar_try_wait(bar, parity)) return;
    if (*abort_flag) return;
    if (!mbar_wait_bounded(bar, parity, wait_limit)) {
      *abort_flag = 1;
      if (p.status) atomicCAS(p.status, 0, int(VLA_ERR_DEVICE_TIMEOUT));
    }
  };

#ifdef VLA_SECTION_TIMERS
  long long tsec[20];
  for (int i = 0; i < 20; ++i) tsec[i] = 0;
  long long tlast = clock64();
  const long long tk0_ = tlast;
  unsigned long long tg0_;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(tg0_));
#define VLA_MARK(i) { long long now_ = clock64(); tsec[i] += now_ - tlast; tlast = now_; }
#else
#define VLA_MARK(i)
#endif

  if (tid == 0) {
    *abort_flag = 0;
    for (int s = 0; s < NSTAGE; ++s) mbar_init(&raw_full[s], 1);
    for (int s = 0; s < KRING; ++s) { mbar_init(&k_full[s], 1); mbar_init(&k_empty[s], 2); }
    for (int s = 0; s < RING; ++s) { mbar_init(&z_full[s], 1); mbar_init(&z_empty[s], 2); }
    mbar_init(b_z0, 1); mbar_init(b_aupd, 1); mbar_init(b_pr, 1); mbar_init(b_supd, 1);
    mbar_init(b_lo_s, 1); mbar_init(b_lo_a, 1);
    mbar_init(b_lo_rdy_a, 1); mbar_init(b_lo_rdy_s, 1); mbar_init(b_ep_rdy, 1);
    mbar_init_fence();
  }
  if (tid < 32) {   // warp 0 allocates the CTA's tensor memory (all 512 columns: one CTA per SM)
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(Cfg::TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tbase = *tmem_slot;
  const uint32_t trow = tbase + (uint32_t((tid >> 5) & 3) << 21);   // this warp's 32 lanes: lane field = bits 16..

  // one state row: global (or the initial value) -> tensor memory; returns the row's sum
  auto state_in = [&](const float* src, float diag, uint32_t col, bool handed_over) -> float {
    // the row sum seeds (state . 1), which is then carried along exactly as the recurrence moves
    // it: an error made here stays for the rest of the unit, and for A the sum cancels to a
    // thousandth of its terms once many keys have been seen, so it is taken in fp64
    double rowsum = 0.0;
#pragma unroll 1
    for (int c0 = 0; c0 < D; c0 += 32) {
      uint32_t r[32];
      if (src) {
        const float4* s4 = reinterpret_cast<const float4*>(src + (size_t(unit) * D + g) * D + c0);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float4 x = handed_over ? __ldcg(s4 + i) : __ldg(s4 + i);   // written by another SM: past L1
          r[4 * i + 0] = __float_as_uint(x.x); r[4 * i + 1] = __float_as_uint(x.y);
          r[4 * i + 2] = __float_as_uint(x.z); r[4 * i + 3] = __float_as_uint(x.w);
        }
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) r[i] = __float_as_uint((c0 + i == g) ? diag : 0.0f);
      }
#pragma unroll
      for (int i = 0; i < 32; ++i) rowsum += double(__uint_as_float(r[i]));
      tmem_st32(trow + col + c0, r);
    }
    tmem_wait_st();
    return float(rowsum);
  };
  // One state row: tensor memory -> global.  During the scan the products see the state only
  // through centred operands plus the carried (state . 1), so what the stored state itself
  // holds along the all-ones direction is never used and drifts (the rank-16 updates accumulate
  // with truncation).  Before it leaves, the row is therefore corrected so that the state that
  // is written has the carried `tracked` as its row sum: X += dlt 1^T / D for S, and the
  // symmetric X += (dlt 1^T + 1 dlt^T) / D - (1^T dlt) 1 1^T / D^2 for A, dlt = tracked - X 1.
  // A later call (or the CTA that continues a cut unit) re-forms (state . 1) from these rows.
  // `dvec`: D floats of the group's shared memory; `bar_id`: the group's named barrier.
  auto state_out = [&](float* dst, uint32_t col, float tracked, bool symmetric, float* dvec, int bar_id) {
    double rowsum = 0.0;
#pragma unroll 1
    for (int c0 = 0; c0 < D; c0 += 32) {
      uint32_t r[32];
      tmem_ld32(trow + col + c0, r);
      tmem_wait_ld();
#pragma unroll
      for (int i = 0; i < 32; ++i) rowsum += double(__uint_as_float(r[i]));
    }
    const float dg = float(double(tracked) - rowsum);
    float total = 0.0f;
    if (symmetric) {
      dvec[g] = dg;
      group_bar(bar_id, NG);
      for (int j = 0; j < D; ++j) total += dvec[j];
    }
    const float own = dg * (1.0f / D) - (symmetric ? total * (1.0f / (D * D)) : 0.0f);
#pragma unroll 1
    for (int c0 = 0; c0 < D; c0 += 32) {
      uint32_t r[32];
      tmem_ld32(trow + col + c0, r);
      tmem_wait_ld();
      float4* d4 = reinterpret_cast<float4*>(dst + (size_t(unit) * D + g) * D + c0);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        float4 x = make_float4(__uint_as_float(r[4 * i + 0]), __uint_as_float(r[4 * i + 1]),
                               __uint_as_float(r[4 * i + 2]), __uint_as_float(r[4 * i + 3]));
        float4 cj = make_float4(own, own, own, own);
        if (symmetric) {
          const float4 dj = *reinterpret_cast<const float4*>(dvec + c0 + 4 * i);
          cj = make_float4(fmaf(dj.x, 1.0f / D, own), fmaf(dj.y, 1.0f / D, own), fmaf(dj.z, 1.0f / D, own),
                           fmaf(dj.w, 1.0f / D, own));
        }
        d4[i] = make_float4(x.x + cj.x, x.y + cj.y, x.z + cj.z, x.w + cj.w);
      }
    }
    if (symmetric) group_bar(bar_id, NG);   // dvec is free again
  };
  // lo scratch <- state - hi(state), this thread's row
  auto split_state = [&](uint32_t col) {
#pragma unroll 1
    for (int c0 = 0; c0 < D; c0 += 32) {
      uint32_t r[32];
      tmem_ld32(trow + col + c0, r);
      tmem_wait_ld();
#pragma unroll
      for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(tf32_state_lo(__uint_as_float(r[i])));
      tmem_st32(trow + Cfg::COL_LO + c0, r);
    }
    tmem_wait_st();
  };

  Piece pc;
#pragma unroll 1
  for (int pi = 0; get_piece<BALANCED>(sp, p.units, nch_unit, blockIdx.x, pi, pc); ++pi) {
  unit = pc.unit;
  t_begin = pc.cb * C;
  T = min(p.T, pc.ce * C) - t_begin;
  nchunks = pc.ce - pc.cb;
  from_handoff = t_begin > 0;                      // continues a unit another CTA started
  const bool to_handoff = t_begin + T < p.T;       // hands the unit over to the CTA that finishes it
  if (pi > 0) {
    // every role has finished the previous piece (CTA barrier at its end): all barrier phases
    // start over, so the per-piece chunk counters keep giving the parities
    if (tid == 0) {
      for (int i = 0; i < Cfg::NBAR; ++i)
        asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(smem_u32(&bars[i])) : "memory");
      for (int s2 = 0; s2 < NSTAGE; ++s2) mbar_init(&raw_full[s2], 1);
      for (int s2 = 0; s2 < KRING; ++s2) { mbar_init(&k_full[s2], 1); mbar_init(&k_empty[s2], 2); }
      for (int s2 = 0; s2 < RING; ++s2) { mbar_init(&z_full[s2], 1); mbar_init(&z_empty[s2], 2); }
      mbar_init(b_z0, 1); mbar_init(b_aupd, 1); mbar_init(b_pr, 1); mbar_init(b_supd, 1);
      mbar_init(b_lo_s, 1); mbar_init(b_lo_a, 1);
      mbar_init(b_lo_rdy_a, 1); mbar_init(b_lo_rdy_s, 1); mbar_init(b_ep_rdy, 1);
      mbar_init_fence();
    }
  }
  if (tid == 0 && from_handoff && !*abort_flag) {
    // the head of this unit is done once its flag shows this launch's id (bounded wait)
    bool seen = false;
    const uint64_t probes = 4ull * wait_limit;
    for (uint64_t it = 0; it < probes && !seen; ++it) {
      seen = ld_acquire_gpu(&sched_flags[unit]) == sp.epoch;
      if (!seen) __nanosleep(64);
    }
    if (!seen) {
      *abort_flag = 1;
      if (p.status) atomicCAS(p.status, 0, int(VLA_ERR_DEVICE_TIMEOUT));
    }
  }
  __syncthreads();

  if (grp == 0) {
    // =====================================================================  group A
    float* Zsf = reinterpret_cast<float*>(abase);            // [4][128] float4: -z_t / delta_t
    float* Zsl = Zsf + D * C;                                // its lo part
    float* Zp = Zsl + D * C;                                 // [C][D] rows: Z0, then Z
    float* Ws = Zp + C * D;                                  // [C][CP] K A K^T, then its factors
    float* Ls = Ws + C * CP;                                 // [C][CP] unit lower factor
    float* N2p = Ls + C * CP;                                // [4][C]
    float* ZSp = N2p + 4 * C;                                // [4][C] per-warp sums of the entries of z_t
    float* dlt = ZSp + 4 * C;                                // [C]
    float* idl = dlt + C;                                    // [C]  1/delta
    float* nidl = idl + C;                                   // [C] -1/delta
    // w1 = (A 1)[g], the row sum of A, carried along in fp32 (see "centred operands" below)
    float w1 = state_in(from_handoff ? p.A_T : p.A0, 1.0f / p.lambda, Cfg::COL_A, from_handoff);

#pragma unroll kLoopUnroll
    for (int c = 0; c < nchunks; ++c) {
      const int ks = c % KRING, zs = c % RING;
      unsigned char* kslot = kslots + size_t(ks) * Cfg::kslot_bytes;
      const float* Kp = reinterpret_cast<const float*>(kslot + Cfg::kq_bytes);   // [C][VP] k_hat
      const float* Qp = Kp + C * VP;                                             // [C][VP] q_f
      unsigned char* zslot = zslots + size_t(zs) * Cfg::zslot_bytes;
      float* Zf = reinterpret_cast<float*>(zslot);           // [4][128] float4: z_t
      float* Zl = Zf + D * C;
      float* GuT = Zl + D * C;                               // [C][CP]
      float* HT = GuT + C * CP;                              // [C][CP]
      float* scs = HT + C * CP;                              // [C]
      float* ssm = scs + C;                                  // [C] sum of the entries of z_t
      const float* ckm = reinterpret_cast<const float*>(kslot + Cfg::kq_bytes + Cfg::kp_bytes) + C * VP + 2 * C;   // [C] mean of k_hat_t

      VLA_MARK(8)
      // A is final once the update of the previous chunk has completed
      if (c > 0) wait(b_aupd, (c - 1) & 1);
      VLA_MARK(0)
      // the lo scratch is free once group S's products of the previous chunk have read it
      if (c > 0) wait(b_lo_a, (c - 1) & 1);
      tc_fence_after();
      VLA_MARK(9)
      split_state(Cfg::COL_A);
      tc_fence_before();
      group_bar(1, NG);
      if (g == 0) mbar_arrive(b_lo_rdy_a);
      VLA_MARK(1)
      wait(&k_full[ks], (c / KRING) & 1);   // (here it costs nothing: the products are still running)
      wait(b_z0, c & 1);
      tc_fence_after();
      VLA_MARK(2)
      float z[16];
      {
        uint32_t r0[16], r1[16];
        tmem_ld16(trow + Cfg::COL_Z0, r0);
        tmem_ld16(trow + Cfg::COL_Z0 + 32, r1);
        tmem_wait_ld();
        VLA_MARK(10)
        // (all shared-memory loads before the first store: the compiler cannot tell the arrays
        // apart and would otherwise wait for each load behind the store before it)
        float cm[16];
#pragma unroll
        for (int t = 0; t < 16; ++t) cm[t] = ckm[t];
#pragma unroll
        for (int t = 0; t < 16; ++t) {
          // row g of Z0 = A K^T = A (K - mean)^T + (A 1) mean^T
          z[t] = fmaf(w1, cm[t], __uint_as_float(r0[t]) + __uint_as_float(r1[t]));
        }
#pragma unroll
        for (int t = 0; t < 16; ++t) Zp[t * D + g] = z[t];
      }
      VLA_MARK(11)
      tc_fence_before();
      group_bar(1, NG);
      VLA_MARK(3)

      // ---- W = K Z0 (C x C, symmetric)
      gram16_tc<CP, VP>(Kp, Zp, Ws, g);
      group_bar(1, NG);
      VLA_MARK(4)

      // ---- warp 0: I + W = L diag(delta) L^T by elimination, in place: once column s is
      // eliminated its slots below the diagonal are free, and the row operations applied to the
      // identity fill them with L^-1.  At the end the row holds L^-1 (left of the diagonal),
      // delta (on it) and delta_s L[t][s] (right of it).
      if (gw == 0) {
        const int r = lane & 15, h = lane >> 4;
        float m[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) m[j] = Ws[r * CP + h * 8 + j] + ((h * 8 + j == r) ? 1.0f : 0.0f);
#pragma unroll
        for (int s2 = 0; s2 < 16; ++s2) {
          const int hs = s2 >> 3, js = s2 & 7;
          const float piv = fmaxf(__shfl_sync(0xffffffffu, m[js], s2 + 16 * hs), eps);
          const float mrs = __shfl_sync(0xffffffffu, m[js], r + 16 * hs);
          const float ipiv = rcp_nr(piv);
          const float l = (r > s2) ? mrs * ipiv : 0.0f;  // L[r][s2]
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float msj = __shfl_sync(0xffffffffu, m[j], s2 + 16 * h);
            m[j] = fmaf(-l, msj, m[j]);
          }
          if (h == hs && r > s2) m[js] = -l;             // (row r of the identity) -= l (row s2 of it)
          if (lane == 0) { dlt[s2] = piv; idl[s2] = ipiv; nidl[s2] = -ipiv; }
        }
        __syncwarp();
        *reinterpret_cast<float4*>(Ws + r * CP + h * 8) = make_float4(m[0], m[1], m[2], m[3]);
        *reinterpret_cast<float4*>(Ws + r * CP + h * 8 + 4) = make_float4(m[4], m[5], m[6], m[7]);
      }
      group_bar(1, NG);
      VLA_MARK(5)

      // ---- row g of Z = Z0 L^-T: z_t = z0_t + sum_{s<t} (L^-1)[t][s] z0_s, sixteen independent sums
      {
        float zn[16];
#pragma unroll
        for (int t = 0; t < 16; ++t) {
          float a0 = z[t], a1 = 0.f;
#pragma unroll
          for (int s4 = 0; s4 * 4 < t; ++s4) {
            const float4 x4 = reinterpret_cast<const float4*>(Ws + t * CP)[s4];
            if (4 * s4 + 0 < t) a0 = fmaf(x4.x, z[4 * s4 + 0], a0);
            if (4 * s4 + 1 < t) a1 = fmaf(x4.y, z[4 * s4 + 1], a1);
            if (4 * s4 + 2 < t) a0 = fmaf(x4.z, z[4 * s4 + 2], a0);
            if (4 * s4 + 3 < t) a1 = fmaf(x4.w, z[4 * s4 + 3], a1);
          }
          zn[t] = a0 + a1;
        }
#pragma unroll
        for (int t = 0; t < 16; ++t) z[t] = zn[t];
      }
      VLA_MARK(12)
      // both rank-16 updates of chunk c - RING have read the Z slot
      if (c >= RING) wait(&z_empty[zs], ((c / RING) + 1) & 1);
      VLA_MARK(13)
      {
        float sq[16];
        float4 nid[4];
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4) nid[k4] = *reinterpret_cast<const float4*>(nidl + 4 * k4);
#pragma unroll
        for (int t = 0; t < 16; ++t) {
          Zp[t * D + g] = z[t];
          sq[t] = z[t] * z[t];
        }
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4) {
          const float4 zz = make_float4(z[4 * k4], z[4 * k4 + 1], z[4 * k4 + 2], z[4 * k4 + 3]);
          const float4 ni = nid[k4];
          const float4 zsc = make_float4(zz.x * ni.x, zz.y * ni.y, zz.z * ni.z, zz.w * ni.w);
          float4 hi, lo;
          tf32_split4(zz, hi, lo);
          reinterpret_cast<float4*>(Zf)[k4 * 128 + g] = hi;
          reinterpret_cast<float4*>(Zl)[k4 * 128 + g] = lo;
          tf32_split4(zsc, hi, lo);
          reinterpret_cast<float4*>(Zsf)[k4 * 128 + g] = hi;
          reinterpret_cast<float4*>(Zsl)[k4 * 128 + g] = lo;
        }
        const float tot = warp_reduce_scatter16(sq, lane);
        if ((lane & 1) == 0) N2p[gw * C + (lane >> 1)] = tot;
#pragma unroll
        for (int t = 0; t < 16; ++t) sq[t] = z[t];
        const float tot1 = warp_reduce_scatter16(sq, lane);
        if ((lane & 1) == 0) ZSp[gw * C + (lane >> 1)] = tot1;
        if constexpr (STASH) {   // the backward pass walks the tokens back with these
          const int nv = min(C, T - c * C);
          if (p.stash_z) {
            float* zs = p.stash_z + (size_t(unit) * size_t(p.T) + size_t(t_begin) + size_t(c) * C) * D + g;
#pragma unroll
            for (int t = 0; t < 16; ++t)
              if (t < nv) zs[size_t(t) * D] = z[t];
          }
          if (p.stash_delta && g < nv) p.stash_delta[size_t(unit) * size_t(p.T) + size_t(t_begin) + size_t(c) * C + g] = dlt[g];
        }
      }
      group_bar(1, NG);
      VLA_MARK(6)

      // ---- A 1 after this chunk: w1 -= sum_t z_t[g] (z_t . 1) / delta_t
#pragma unroll
      for (int t = 0; t < 16; ++t) {
        const float st = (ZSp[t] + ZSp[C + t]) + (ZSp[2 * C + t] + ZSp[3 * C + t]);
        w1 = fmaf(-z[t], st * idl[t], w1);
      }
      // ---- warp 0: sc_t and GuT[t][s] = Gu[s][t] = sc_s delta_s L[t][s]
      if (gw == 0) {
        const int r = lane & 15, h = lane >> 4;
        const float n2 = N2p[r] + N2p[C + r] + N2p[2 * C + r] + N2p[3 * C + r];
        if (h == 1) ssm[r] = (ZSp[r] + ZSp[C + r]) + (ZSp[2 * C + r] + ZSp[3 * C + r]);
        const float id_r = idl[r], d_r = dlt[r];
        // alpha_r = sc_r z_r, sc_r = (1/delta) / max(||z||/delta, eps)      (A_t k_hat_t = z_t / delta_t)
        const float sc_r = id_r * rcp_nr(fmaxf(sqrt_approx(n2) * id_r, eps));
        if ((p.flags & VLA_FLAG_CHECK_FINITE) && p.status && !isfinite(n2 + d_r))
          atomicCAS(p.status, 0, int(VLA_ERR_NONFINITE));
        if (h == 0) scs[r] = sc_r;
        float us[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) us[j] = Ws[(h * 8 + j) * CP + r];    // Ws[s][t] = delta_s L[t][s]
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int s2 = h * 8 + j;
          const float sc_s = __shfl_sync(0xffffffffu, sc_r, s2);
          GuT[r * CP + s2] = (s2 < r) ? sc_s * us[j] : 0.0f;
        }
      }
      VLA_MARK(14)
      // ---- HT[t][s] = q_t . z_s
      gram16_tc<CP, VP>(Qp, Zp, HT, g);
      fence_async_smem();     // Z, lo(Z), -Z/delta: written here, read by the tensor core
      group_bar(1, NG);
      if (g == 0) {
        mbar_arrive(&z_full[zs]);    // group S and the issuing warp of the update of A
        mbar_arrive(&k_empty[ks]);
      }
      VLA_MARK(7)
    }
    if (nchunks > 0) wait(b_aupd, (nchunks - 1) & 1);
    tc_fence_after();
    if (p.A_T) state_out(p.A_T, Cfg::COL_A, w1, true, Zp, 1);
  } else if (grp == 1) {
    // =====================================================================  group S
    float* Epf = reinterpret_cast<float*>(sbase);            // [4][128] float4: e'_t
    float* Epl = Epf + D * C;
    float* ostage = Epl + D * C;                             // [2][C][D]
    float s1 = state_in(from_handoff ? p.S_T : p.S0, 0.0f, Cfg::COL_S, from_handoff);   // (S 1)[g], carried along in fp32

#pragma unroll kLoopUnroll
    for (int c = 0; c < nchunks; ++c) {
      const int n = min(C, T - c * C);
      const int ks = c % KRING, zs = c % RING;
      unsigned char* kslot = kslots + size_t(ks) * Cfg::kslot_bytes;
      const float* Vf = reinterpret_cast<const float*>(kslot + Cfg::kq_bytes + Cfg::kp_bytes);   // [C][VP]
      const float* inv_den = Vf + C * VP + C;
      const float* ckm = inv_den + C;                       // [C] mean of k_hat_t
      const float* cqm = ckm + C;                           // [C] mean of q_f,t
      unsigned char* zslot = zslots + size_t(zs) * Cfg::zslot_bytes;
      const float* GuT = reinterpret_cast<const float*>(zslot) + 2 * D * C;
      const float* HT = GuT + C * CP;
      const float* scs = HT + C * CP;
      const float* ssm = scs + C;

      VLA_MARK(8)
      if (c > 0) wait(b_supd, (c - 1) & 1);
      wait(&k_full[ks], (c / KRING) & 1);
      VLA_MARK(0)
      // the lo scratch is free once group A's products of this chunk have read it
      wait(b_lo_s, c & 1);
      tc_fence_after();
      VLA_MARK(9)
      split_state(Cfg::COL_S);
      tc_fence_before();
      group_bar(2, NG);
      if (g == 0) mbar_arrive(b_lo_rdy_s);
      VLA_MARK(1)
      wait(b_pr, c & 1);
      tc_fence_after();
      VLA_MARK(2)
      float e[16], r0v[16];
      {
        uint32_t x0[32], x1[32];
        tmem_ld32(trow + Cfg::COL_PR, x0);
        tmem_ld32(trow + Cfg::COL_PR + 32, x1);
        tmem_wait_ld();
#pragma unroll
        for (int t = 0; t < 16; ++t) {
          // (S k_hat_t)[g] and (S q_t)[g], each as S (x - mean)^T + (S 1) mean
          const float pt = fmaf(s1, ckm[t], __uint_as_float(x0[t]) + __uint_as_float(x1[t]));
          r0v[t] = fmaf(s1, cqm[t], __uint_as_float(x0[16 + t]) + __uint_as_float(x1[16 + t]));
          e[t] = Vf[t * VP + g] - pt;                                                 // b_t
        }
      }
      tc_fence_before();
      if (g == 0) bulk_wait_read<1>();   // the out stage of chunk c-2 has left shared memory
      VLA_MARK(3)
      wait(&z_full[zs], (c / RING) & 1);
      VLA_MARK(4)

      // ---- row g: e_t = b_t - sum_{s<t} Gu[s][t] e_s; e'_t = sc_t e_t;
      //             o_t = (r0_t + sum_{s<=t} e'_s HT[t][s]) / den_t
      float ep[16];
#pragma unroll
      for (int t = 0; t < 16; ++t) {
        float a0 = e[t], a1 = 0.f;
#pragma unroll
        for (int s4 = 0; s4 * 4 < t; ++s4) {
          const float4 g4 = reinterpret_cast<const float4*>(GuT + t * CP)[s4];
          if (4 * s4 + 0 < t) a0 = fmaf(-g4.x, e[4 * s4 + 0], a0);
          if (4 * s4 + 1 < t) a1 = fmaf(-g4.y, e[4 * s4 + 1], a1);
          if (4 * s4 + 2 < t) a0 = fmaf(-g4.z, e[4 * s4 + 2], a0);
          if (4 * s4 + 3 < t) a1 = fmaf(-g4.w, e[4 * s4 + 3], a1);
        }
        e[t] = a0 + a1;
        ep[t] = e[t] * scs[t];
        s1 = fmaf(ep[t], ssm[t], s1);          // S 1 after this chunk: += e'_t (z_t . 1)
        if constexpr (STASH) {
          if (p.stash_e && t < n) p.stash_e[(size_t(unit) * size_t(p.T) + size_t(t_begin) + size_t(c) * C + t) * D + g] = e[t];
        }
      }
#pragma unroll
      for (int t = 0; t < 16; ++t) {
        float a0 = r0v[t], a1 = 0.f;
#pragma unroll
        for (int s4 = 0; s4 * 4 <= t; ++s4) {
          const float4 h4 = reinterpret_cast<const float4*>(HT + t * CP)[s4];
          if (4 * s4 + 0 <= t) a0 = fmaf(h4.x, ep[4 * s4 + 0], a0);
          if (4 * s4 + 1 <= t) a1 = fmaf(h4.y, ep[4 * s4 + 1], a1);
          if (4 * s4 + 2 <= t) a0 = fmaf(h4.z, ep[4 * s4 + 2], a0);
          if (4 * s4 + 3 <= t) a1 = fmaf(h4.w, ep[4 * s4 + 3], a1);
        }
        r0v[t] = (a0 + a1) * inv_den[t];
      }
      VLA_MARK(5)
      group_bar(2, NG);  // bulk_wait_read above is ordered before the stage is rewritten
      {
        float* ost = ostage + size_t(c & 1) * C * D;
#pragma unroll
        for (int t = 0; t < 16; ++t) ost[t * D + g] = r0v[t];
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4) {
          const float4 ee = make_float4(ep[4 * k4], ep[4 * k4 + 1], ep[4 * k4 + 2], ep[4 * k4 + 3]);
          float4 hi, lo;
          tf32_split4(ee, hi, lo);
          reinterpret_cast<float4*>(Epf)[k4 * 128 + g] = hi;
          reinterpret_cast<float4*>(Epl)[k4 * 128 + g] = lo;
        }
      }
      fence_async_smem();
      group_bar(2, NG);
      if (g == 0) {
        mbar_arrive(&k_empty[ks]);
        if constexpr (!TM) {
          bulk_store(p.out + (size_t(unit) * size_t(p.T) + size_t(t_begin) + size_t(c) * C) * D,
                     ostage + size_t(c & 1) * C * D, uint32_t(n) * D * sizeof(float));
        } else {   // rows past T are clipped by the tensor map
          const int b = unit / p.heads, h = unit - b * p.heads;
          tma_store_4d(&maps.out, 0, h, t_begin + c * C, b, ostage + size_t(c & 1) * C * D);
        }
        bulk_commit();
        mbar_arrive(b_ep_rdy);
      }
      VLA_MARK(6)
    }
    if (nchunks > 0) wait(b_supd, (nchunks - 1) & 1);
    tc_fence_after();
    if (p.S_T) state_out(p.S_T, Cfg::COL_S, s1, false, nullptr, 2);
    if (g == 0) bulk_wait_all<0>();
  } else if (grp == 2) {
    // =====================================================================  group P: TMA ring + input prep
    float* denp = reinterpret_cast<float*>(pbase);           // [2][C]
    const int pw = g >> 5;                                   // prep warp: tokens 8 pw .. 8 pw + 7
    const int tl = lane & 7, fl = lane >> 3;                 // token within the warp's 8, float4 lane 0..3
    auto issue = [&](int c) {
      const int s = c % NSTAGE;
      const int n = min(C, T - c * C);
      const uint32_t bytes = uint32_t(n) * D * sizeof(TIn);
      TIn* dst = raw + size_t(s) * 3 * C * D;
      if constexpr (!TM) {
        mbar_arrive_expect_tx(&raw_full[s], 3 * bytes);
        const size_t tok = size_t(unit) * size_t(p.T) + size_t(t_begin) + size_t(c) * C;
        bulk_load(dst + 0 * C * D, static_cast<const TIn*>(p.q) + tok * D, bytes, &raw_full[s]);
        bulk_load(dst + 1 * C * D, static_cast<const TIn*>(p.k) + tok * D, bytes, &raw_full[s]);
        bulk_load(dst + 2 * C * D, static_cast<const TIn*>(p.v) + tok * D, bytes, &raw_full[s]);
      } else {
        // rows past T arrive as zeros and count towards the bytes like any other
        const int b = unit / p.heads, h = unit - b * p.heads, t0 = t_begin + c * C;
        mbar_arrive_expect_tx(&raw_full[s], 3 * uint32_t(C * D * sizeof(TIn)));
        tma_load_4d(dst + 0 * C * D, &maps.q, 0, h, t0, b, &raw_full[s]);
        tma_load_4d(dst + 1 * C * D, &maps.k, 0, h, t0, b, &raw_full[s]);
        tma_load_4d(dst + 2 * C * D, &maps.v, 0, h, t0, b, &raw_full[s]);
        (void)bytes;
      }
    };
    if (g == 0)
      for (int c = 0; c < NSTAGE && c < nchunks; ++c) issue(c);
    // running sum of phi(k), columns 2g and 2g + 1
    float2 zk = make_float2(0.f, 0.f);
    if (from_handoff) {
      if (p.zT) zk = __ldcg(reinterpret_cast<const float2*>(p.zT + size_t(unit) * D + 2 * g));
    } else if (p.z0) {
      zk = *reinterpret_cast<const float2*>(p.z0 + size_t(unit) * D + 2 * g);
    }

#pragma unroll kLoopUnroll
    for (int c = 0; c < nchunks; ++c) {
      const int s = c % NSTAGE, ks = c % KRING;
      const int n = min(C, T - c * C);
      unsigned char* kslot = kslots + size_t(ks) * Cfg::kslot_bytes;
      float4* KQ4 = reinterpret_cast<float4*>(kslot);
      float* Kp = reinterpret_cast<float*>(kslot + Cfg::kq_bytes);
      float* Qp = Kp + C * VP;
      float* Vf = Qp + C * VP;
      float* nrm = Vf + C * VP;
      float* inv_den = nrm + C;
      VLA_MARK(8)
      wait(&raw_full[s], (c / NSTAGE) & 1);
      VLA_MARK(0)
      if (c >= KRING) wait(&k_empty[ks], ((c / KRING) + 1) & 1);
      VLA_MARK(1)
      const TIn* rq = raw + (size_t(s) * 3 + 0) * C * D;
      const TIn* rk = raw + (size_t(s) * 3 + 1) * C * D;
      const TIn* rv = raw + (size_t(s) * 3 + 2) * C * D;
      {
        const int tt = 8 * pw + tl;
        const bool act = tt < n;
        // pass 1 (rolled; this group has time to spare and the chunk loop of all roles together
        // has to stay in the instruction cache): widen, feature map, plain rows; phi(k) is
        // parked in the row of k_hat until its norm is known
        float ss = 0.f, sk = 0.f, sqm = 0.f;
#pragma unroll kPrepUnroll
        for (int i = 0; i < 8; ++i) {
          const int f = fl + 4 * i;
          float4 vv = make_float4(0.f, 0.f, 0.f, 0.f);
          float4 kf = vv, qv = vv;
          if (act) {
            kf = load4(rk + tt * D, f);
            qv = load4(rq + tt * D, f);
            vv = load4(rv + tt * D, f);
            if (!ident) {
              kf.x = phi_fast(kf.x); kf.y = phi_fast(kf.y); kf.z = phi_fast(kf.z); kf.w = phi_fast(kf.w);
              qv.x = phi_fast(qv.x); qv.y = phi_fast(qv.y); qv.z = phi_fast(qv.z); qv.w = phi_fast(qv.w);
            }
          }
          reinterpret_cast<float4*>(Kp + tt * VP)[f] = kf;
          reinterpret_cast<float4*>(Qp + tt * VP)[f] = qv;
          reinterpret_cast<float4*>(Vf + tt * VP)[f] = vv;
          ss = fmaf(kf.x, kf.x, ss); ss = fmaf(kf.y, kf.y, ss);
          ss = fmaf(kf.z, kf.z, ss); ss = fmaf(kf.w, kf.w, ss);
          sk += (kf.x + kf.y) + (kf.z + kf.w);
          sqm += (qv.x + qv.y) + (qv.z + qv.w);
        }
        ss += __shfl_xor_sync(0xffffffffu, ss, 8);  ss += __shfl_xor_sync(0xffffffffu, ss, 16);
        sk += __shfl_xor_sync(0xffffffffu, sk, 8);  sk += __shfl_xor_sync(0xffffffffu, sk, 16);
        sqm += __shfl_xor_sync(0xffffffffu, sqm, 8); sqm += __shfl_xor_sync(0xffffffffu, sqm, 16);
        const float nr = fmaxf(sqrt_approx(ss), eps);   // max(||phi(k)||, eps)
        const float inv = rcp_nr(nr);
        // Centred operands: the tensor core truncates its addends towards zero, so a sum of
        // like-signed products (feature-mapped keys and queries are all positive) comes out
        // low by an amount that is the same in every row and piles up along the common
        // direction of the keys.  The products are therefore taken with x - mean(x), whose
        // entries have both signs, and the mean's share, (state . 1) mean(x), is added back in
        // fp32 by the groups, which carry state . 1 along with the state.
        const float mk = sk * inv * (1.0f / D), mq = sqm * (1.0f / D);
        // pass 2: k_hat, and the centred operand rows in hi/lo pairs (each thread re-reads what it wrote)
#pragma unroll kPrepUnroll
        for (int i = 0; i < 8; ++i) {
          const int f = fl + 4 * i;
          const float4 kf = reinterpret_cast<const float4*>(Kp + tt * VP)[f];
          const float4 qv = reinterpret_cast<const float4*>(Qp + tt * VP)[f];
          const float4 kh = make_float4(kf.x * inv, kf.y * inv, kf.z * inv, kf.w * inv);
          reinterpret_cast<float4*>(Kp + tt * VP)[f] = kh;
          float4 hi, lo;
          tf32_split4(make_float4(kh.x - mk, kh.y - mk, kh.z - mk, kh.w - mk), hi, lo);
          KQ4[f * Cfg::KQR + tt] = hi;
          KQ4[f * Cfg::KQR + 32 + tt] = lo;
          tf32_split4(make_float4(qv.x - mq, qv.y - mq, qv.z - mq, qv.w - mq), hi, lo);
          KQ4[f * Cfg::KQR + 16 + tt] = hi;
          KQ4[f * Cfg::KQR + 48 + tt] = lo;
        }
        // phi(k) = k_hat * nrm exactly as the recurrence sees it; 0 for padding rows
        if (fl == 0) {
          nrm[tt] = act ? nr : 0.0f;
          inv_den[C + tt] = act ? mk : 0.0f;          // mean of k_hat_t
          inv_den[2 * C + tt] = act ? mq : 0.0f;      // mean of q_f,t
        }
      }
      group_bar(3, NP);
      VLA_MARK(2)
      if (g == 0 && c + NSTAGE < nchunks) issue(c + NSTAGE);   // the raw stage has been consumed
      // ---- running key sum and readout denominators (columns 2g, 2g+1)
      if (!ident) {
        float pr[16];
#pragma unroll
        for (int t = 0; t < 16; ++t) {
          const float2 kh = *reinterpret_cast<const float2*>(Kp + t * VP + 2 * g);
          const float2 qf = *reinterpret_cast<const float2*>(Qp + t * VP + 2 * g);
          const float nt = nrm[t];
          zk.x = fmaf(kh.x, nt, zk.x);
          zk.y = fmaf(kh.y, nt, zk.y);
          pr[t] = fmaf(zk.x, qf.x, zk.y * qf.y);
        }
        const float tot = warp_reduce_scatter16(pr, lane);
        if ((lane & 1) == 0) denp[pw * C + (lane >> 1)] = tot;
        if constexpr (STASH) {
          // the backward pass restarts its walk back of the key sum from these (a walk from the
          // final sum alone would cancel catastrophically at the early tokens)
          if (p.stash_zk)
            *reinterpret_cast<float2*>(p.stash_zk + (size_t(unit) * size_t(nch_unit) + size_t(t_begin / C + c)) * D + 2 * g) = zk;
        }
        group_bar(3, NP);
        if (g < C) inv_den[g] = rcp_nr(fmaxf(denp[g] + denp[C + g], eps));
      } else {
        if (g < C) inv_den[g] = 1.0f;
      }
      fence_async_smem();   // the operand arrays are read by the tensor core
      group_bar(3, NP);
      if (g == 0) mbar_arrive(&k_full[ks]);
      VLA_MARK(3)
    }
    if (p.zT) *reinterpret_cast<float2*>(p.zT + size_t(unit) * D + 2 * g) = zk;
  } else {
    // =====================================================================  MMA issue (two warps)
    // Warp 0 of the group issues for group A, warp 1 for group S; the whole warp follows the
    // barriers and one elected lane issues.  Per chunk: the state (hi part, read in place)
    // times the chunk's operand rows; the lo scratch times the same; then the rank-16 update,
    // each a hi*hi + hi*lo + lo*hi triple.
    const bool forA = gw == 0;
    const bool leader = elect_one();
    const uint32_t col_state = forA ? Cfg::COL_A : Cfg::COL_S;
    const uint32_t col_acc = forA ? Cfg::COL_Z0 : Cfg::COL_PR;
    // operand rows of a chunk, 16 each: hi(K_hat) | hi(Q_f) | lo(K_hat) | lo(Q_f).
    // hi pass (the state, read in place): A takes rows 0..47 (the middle 16 columns are not used),
    // S all 64; lo pass (the lo scratch): A takes hi(K_hat), S takes hi(K_hat) | hi(Q_f).
    const uint32_t idesc_hi = forA ? umma_idesc_tf32(128, 48) : umma_idesc_tf32(128, 64);
    const uint32_t idesc_lo = forA ? umma_idesc_tf32(128, 16) : umma_idesc_tf32(128, 32);
    const uint32_t idesc_up = umma_idesc_tf32(128, 128);
    uint64_t* b_upd = forA ? b_aupd : b_supd;
    uint64_t* b_lo_rdy = forA ? b_lo_rdy_a : b_lo_rdy_s;
    uint64_t* b_prod = forA ? b_z0 : b_pr;
    uint64_t* b_lo_next = forA ? b_lo_s : b_lo_a;
    // left factor of the update: -Z/delta (A) or E' (S), and its lo part
    const float* Lf = reinterpret_cast<const float*>(forA ? abase : sbase);
    const uint64_t dLf = umma_desc(smem_u32(Lf), 16 * 128, 128);
    const uint64_t dLl = umma_desc(smem_u32(Lf + D * C), 16 * 128, 128);
#pragma unroll kLoopUnroll
    for (int c = 0; c < nchunks; ++c) {
      const int ks = c % KRING, zs = c % RING;
      const uint64_t dKQ = umma_desc(smem_u32(kslots + size_t(ks) * Cfg::kslot_bytes), 16 * Cfg::KQR, 128);
      const float* Zf = reinterpret_cast<const float*>(zslots + size_t(zs) * Cfg::zslot_bytes);
      const uint64_t dZf = umma_desc(smem_u32(Zf), 16 * 128, 128);
      const uint64_t dZl = umma_desc(smem_u32(Zf + D * C), 16 * 128, 128);
      // the state is final: the previous update has completed (first chunk: the group has stored
      // the initial state, which precedes its first arrival on b_lo_rdy)
      VLA_MARK(8)
      if (c > 0) wait(b_upd, (c - 1) & 1);
      else wait(b_lo_rdy, 0);
      wait(&k_full[ks], (c / KRING) & 1);
      tc_fence_after();
      VLA_MARK(0)
      if (leader) {
#pragma unroll 2
        for (int j = 0; j < 16; ++j)
          umma_ts(tbase + col_acc, tbase + col_state + 8 * j, dKQ + uint64_t(j * (2 * Cfg::KQR)), idesc_hi, j > 0);
      }
      VLA_MARK(1)
      wait(b_lo_rdy, c & 1);
      tc_fence_after();
      VLA_MARK(2)
      if (leader) {
#pragma unroll 2
        for (int j = 0; j < 16; ++j)
          umma_ts(tbase + col_acc, tbase + Cfg::COL_LO + 8 * j, dKQ + uint64_t(j * (2 * Cfg::KQR)), idesc_lo, 1);
        umma_commit(b_prod);
        umma_commit(b_lo_next);
      }
      VLA_MARK(3)
      if (forA) wait(&z_full[zs], (c / RING) & 1);   // Z, lo(Z), -Z/delta are in shared memory
      else wait(b_ep_rdy, c & 1);                    // so are E' and lo(E') (and Z: group S waited for it)
      tc_fence_after();
      VLA_MARK(4)
      if (leader) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          umma_ss(tbase + col_state, dLf + uint64_t(j * 256), dZf + uint64_t(j * 256), idesc_up, 1);
          umma_ss(tbase + col_state, dLf + uint64_t(j * 256), dZl + uint64_t(j * 256), idesc_up, 1);
          umma_ss(tbase + col_state, dLl + uint64_t(j * 256), dZf + uint64_t(j * 256), idesc_up, 1);
        }
        umma_commit(b_upd);
        umma_commit(&z_empty[zs]);
      }
      __syncwarp();
      VLA_MARK(5)
    }
    // the last arrivals this thread asked for have landed (the barriers are re-armed between pieces)
    if (nchunks > 0) {
      wait(b_lo_next, (nchunks - 1) & 1);
      wait(&z_empty[(nchunks - 1) % RING], ((nchunks - 1) / RING) & 1);
    }
  }

  // end of the piece: every role is done with it (states and key sum stored, MMAs and copies
  // that touch shared memory complete), so the barriers may be re-armed and, for a unit that is
  // handed over, the flag may be raised
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (to_handoff && tid == 0) {
    __threadfence();
    st_release_gpu(&sched_flags[unit], sp.epoch);
  }
  }  // pieces

#ifdef VLA_SECTION_TIMERS
  if (p.dbg && tid == 0) {
    unsigned smid_;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(smid_));
    p.dbg[120 + 2 * blockIdx.x] = clock64() - tk0_;
    p.dbg[120 + 2 * blockIdx.x + 1] = smid_;
  }
  if (p.dbg && blockIdx.x == 0) {
    const int role = tid == 0 ? 0 : tid == 32 ? 1 : tid == NG ? 2 : tid == 2 * NG ? 3 : tid == 2 * NG + NP ? 4
                   : tid == 2 * NG + NP + 32 ? 5 : -1;
    unsigned long long tg1_;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(tg1_));
    tsec[18] = clock64() - tk0_;
    tsec[19] = (long long)(tg1_ - tg0_);
    if (role >= 0) for (int i = 0; i < 20; ++i) p.dbg[role * 20 + i] = tsec[i];
  }
#endif
  tc_fence_before();
  __syncthreads();
  if (tid < 32) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tbase), "r"(Cfg::TMEM_COLS) : "memory");
  }
}

int encode_token_major_maps(const ScanParams& p, int d, int dtype, bool has_u, TokenMajorMaps* maps);

template <typename TIn, bool TM, bool STASH = false>
int launch_chunk_tc_t(const ScanParams& p, cudaStream_t st) {
  using Cfg = TcCfg<TIn>;
  static_assert(Cfg::smem_bytes <= 227 * 1024, "tensor-core chunk kernel exceeds the shared memory of one CTA");
  auto kern = vla_scan_tc_kernel<TIn, false, TM, STASH>;       // one CTA per unit
  auto kern_bal = vla_scan_tc_kernel<TIn, true, TM, STASH>;    // persistent grid, units cut at chunks
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(Cfg::smem_bytes)) != cudaSuccess ||
      cudaFuncSetAttribute(kern_bal, cudaFuncAttributeMaxDynamicSharedMemorySize, int(Cfg::smem_bytes)) != cudaSuccess) {
    cudaGetLastError();
    return VLA_ERR_CUDA;
  }
  typename ChunkMapsArg<TM>::type maps;
  if constexpr (TM) {
    const int rc = encode_token_major_maps(p, Cfg::D, sizeof(TIn) == 2 ? VLA_BF16 : VLA_F32, false, &maps);
    if (rc != VLA_OK) return rc;
  } else {
    maps.unused = 0;
  }
  SchedParams sp;
  sp.balanced = 0;
  sp.grid = p.units;
  sp.epoch = 0;
  // Balanced schedule, under the conditions of the FMA chunk kernel's: a last partial wave to
  // fill, all CTAs resident at once (one per SM: a CTA takes the SM's whole tensor memory),
  // S_T / A_T / zT there to carry the state across a cut, no stream capture (the launch id is
  // drawn on the host), a free flag slot.
  cudaStreamCaptureStatus capture = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(st, &capture) != cudaSuccess) {
    cudaGetLastError();
    capture = cudaStreamCaptureStatusActive;
  }
  int dev = 0, sms = 0;
  if (capture == cudaStreamCaptureStatusNone && cudaGetDevice(&dev) == cudaSuccess &&
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess) {
    const bool state_out = p.S_T && p.A_T && (p.zT || (p.flags & VLA_FLAG_IDENTITY_MAP));
    if (sms > 0 && p.units > sms && p.units % sms != 0 && p.T > 0 && state_out && p.units <= kSchedMaxUnits) {
      const unsigned int epoch = next_launch_epoch();
      if (sched_slot_free(epoch)) {
        sp.balanced = 1;
        sp.grid = sms;
        sp.epoch = epoch;
      }
    }
  } else {
    cudaGetLastError();
  }
  if (sp.balanced) {
    kern_bal<<<sp.grid, Cfg::NT, Cfg::smem_bytes, st>>>(p, sp, maps);
    sched_slot_mark(sp.epoch, st);
  } else {
    kern<<<sp.grid, Cfg::NT, Cfg::smem_bytes, st>>>(p, sp, maps);
  }
  note_launch(STASH ? "vla_scan_tc_kernel(stash)" : "vla_scan_tc_kernel", Cfg::D, sizeof(TIn) == 2 ? VLA_BF16 : VLA_F32, sp.grid,
              sp.balanced);
  return cudaGetLastError() == cudaSuccess ? VLA_OK : VLA_ERR_CUDA;
}

}  // namespace vla
