// VLA forward scan, "chunk" kernel: the recurrence of Section 3.3 evaluated
// C = 16 tokens at a time in exact algebra, so that the fp32 FMA pipe works on rank-16
// updates instead of a chain of rank-1 steps.  One CTA works on one (batch, head) unit at a
// time (see "work distribution" below), two warp groups of D threads each:
//
//   group A holds A (the inverse penalty matrix) in registers, thread tile TR x TW;
//   group S holds S (the memory state) in registers, same tiling.
//
// For a chunk with keys K (rows k_hat_t), queries Q (rows q_f,t), values V, and the states
// A, S at the chunk start (Eqs. "sm", "s-update", "output"):
//
//   Z0 = A K^T                          W = K Z0 = K A K^T
//   I + W = L diag(delta) L^T           delta_t is Eq. "sm"'s 1 + u.z;  L[t,s] = (z_s.k_t)/delta_s
//   Z L^T = Z0                          column t is z_t = A_{t-1} k_hat_t (forward substitution)
//   alpha_t = sc_t z_t,  sc_t = (1/delta_t) / max(||z_t||/delta_t, eps)      (A_t k_hat_t = z_t/delta_t)
//   A <- A - Z diag(1/delta) Z^T        (Woodbury form of 16 Sherman-Morrison steps)
//   B  = V^T - S K^T                    e_t = b_t - sum_{s<t} Gu[s,t] e_s,  Gu[s,t] = alpha_s.k_hat_t
//   e'_t = sc_t e_t                     o_t = (S q_t + sum_{s<=t} e'_s (z_s.q_t)) / den_t
//   S <- S + E' Z^T
//
// The lines above are the u = k_hat case.  General path (explicit u, or refresh): Z0 = A U^T and
// W = U Z0 give delta, L and Z as above; W0 = A K^T and X = U W0 give, by the same
// elimination, N[s,t] = z_s.k_hat_t and a_t = A_t k_hat_t = W0_t - sum_{s<=t} z_s N[s,t]/delta_s;
// alpha_t = a_t / max(||a_t||, eps), Gu[s,t] = alpha_s.k_hat_t, and a takes Z's place in the
// S update and in the readout.  Algorithm 1's periodic refresh (A += eta I after every
// period-th token) runs on the general path: with rho(t) refreshes after tokens < t of the
// chunk, Z0_t += eta rho(t) u_t, W[s,t] += eta rho(min(s,t)) u_s.u_t, X[s,t] += eta rho(s) u_s.k_t,
// a_t += eta rho(t+1) k_hat_t, and the chunk ends with A += eta rho(n) I.
//
// Group A runs ahead of group S.  It owns the input stream: q/k/v arrive through a ring of
// 1-D bulk-async (TMA) copies, and group A widens them (phi, k_hat, ||phi(k)||) into a
// three-slot fp32 ring one chunk ahead, overlapped with the LDL^T factorisation.  Z, Gu, sc
// and the small matrix z_s.q_t travel to group S through a two-slot ring.  Both rings are
// guarded by mbarriers, and every mbarrier wait is bounded: if one runs out the CTA records
// VLA_ERR_DEVICE_TIMEOUT, stops waiting and runs to its end.
#pragma once

#include "vla_common.cuh"

namespace vla {

template <int D>
struct ChunkTile {
  static constexpr int TW = (D >= 64) ? 16 : 8;  // state columns per thread
  static constexpr int TR = D / TW;              // state rows per thread (= lanes per row block)
};

// How the penalty direction u_t is obtained and which algebra the chunk uses:
//   kUKhat    u = k_hat, no refresh: A_t k_hat_t = z_t / delta_t, one product with A per chunk
//   kUTensor  u read from the caller's tensor: general path (a_t = A_t k_hat_t by a second
//             elimination), three products with A per chunk
//   kUKhatGen u = k_hat on the general path: used for Algorithm 1's periodic refresh, after
//             which A_t k_hat_t is no longer parallel to z_t; one product with A per chunk
enum : int { kUKhat = 0, kUTensor = 1, kUKhatGen = 2 };

template <int D, typename TIn, int UM = kUKhat, bool TRI = false>
struct ChunkCfg {
  static constexpr bool GEN = UM != kUKhat;      // general path
  static constexpr bool UT = UM == kUTensor;     // a fourth input tensor
  static constexpr int C = 16;                   // tokens per chunk
  static constexpr int TW = ChunkTile<D>::TW;
  static constexpr int TR = ChunkTile<D>::TR;
  static constexpr int LPR = D / TW;             // lanes that share a row block (== TR)
  static constexpr int NV = TW / 4;              // float4 operand groups per thread
  static constexpr int NG = D;                   // threads per warp group
  static constexpr int NGROUPS = TRI ? 3 : 2;    // A, S [, transfer scan]
  // d <= 64: group A is one or two warps, and widening the next chunk's inputs around the
  // factorisation was an eighth to a fifth of its chain; there a warp of its own does it (not in
  // the three-group kernel at d = 64, whose two CTAs per SM leave it no registers)
  static constexpr bool PREPW = D == 32 || (D == 64 && !TRI);
  static constexpr int NT = NGROUPS * D + (PREPW ? 32 : 0);   // threads per CTA
  static constexpr int NWG = D / 32;             // warps per group
  static constexpr int NIN = UT ? 4 : 3;         // q, k, v[, u]
  // raw q/k/v[/u] chunks in flight (fewer on the general path: shared memory is the limit)
  // (the three-group kernel with 16-bit inputs keeps one stage: two of its CTAs then share an SM)
  static constexpr int NSTAGE = TRI ? (sizeof(TIn) == 2 ? 1 : 2)
                                    : UT ? (sizeof(TIn) == 2 ? 2 : 1) : (sizeof(TIn) == 2 ? 4 : 2);
  static constexpr int RING = 2;                 // Z / Gu / HT / sc slots (group A -> group S)
  static constexpr int KRING = 3;                // widened k_hat / q_f / v / ||phi(k)|| slots
  static constexpr int CP = C + 4;               // padded row of the small C x C matrices

  // shared memory layout (floats unless noted)
  static constexpr size_t raw_bytes = size_t(NSTAGE) * NIN * C * D * sizeof(TIn);
  static constexpr size_t kslot_floats = size_t(3) * C * D + C;             // Kh, Qf, Vf, nrm
  static constexpr size_t slot_floats = size_t(C) * D + 2 * C * CP + 2 * C; // Zs, GuT, HT, sc, inv_den
  static constexpr int a_big = UT ? 4 : 1;       // Z0s [, W0s, Uf[2]]
  static constexpr int a_small = UT ? 6 : (GEN ? 4 : 2);
  //   Ws, Ls [, PTs, Guu] [, Xs, Guk]
  static constexpr size_t a_floats = size_t(a_big) * C * D + size_t(a_small) * C * CP +
                                     2 * NWG * C + 3 * C + 32;
  //   ... | N2p, denp | delta, 1/delta, -1/delta | eta * refresh counts [C + 1] (padded)
  // group S forms q_t . z_s itself where it is the group with time to spare (d <= 64)
  static constexpr bool S_HT = !GEN && D <= 64;
  static constexpr size_t s_floats = size_t(3) * C * D + 2 * C * D + ((GEN || S_HT) ? 2 * C * CP : 0);
  //   VS(B), R0s, Eps | ostage[2] [| GuL, HTL]
  static constexpr size_t smem_bytes = raw_bytes +
      (KRING * kslot_floats + RING * slot_floats + a_floats + (NGROUPS - 1) * s_floats) * sizeof(float) +
      (NSTAGE + 2 * RING + (PREPW ? KRING + 1 : 0)) * sizeof(uint64_t) + 16 + 128;
};

// Reduce-scatter of NTOK x LPR values over LPR consecutive lanes: on return v[k][0] is the
// sum, over those lanes, of v[k][position of this lane in the group].
template <int LPR, int NTOK>
__device__ __forceinline__ void reduce_scatter(float (&v)[NTOK][LPR], int cg) {
#pragma unroll
  for (int off = LPR / 2; off >= 1; off >>= 1) {
    const bool up = (cg & off) != 0;
#pragma unroll
    for (int k = 0; k < NTOK; ++k)
#pragma unroll
      for (int i = 0; i < off; ++i) {
        const float send = up ? v[k][i] : v[k][i + off];
        const float keep = up ? v[k][i + off] : v[k][i];
        v[k][i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
      }
  }
}

// For every token t of the chunk: sink(t, row g of (state tile) . op[t]).  Two tokens per
// pass so that the shuffle rounds of the reduce-scatter are paid once per pair, and the
// reduce-scatter of one pair is issued alongside the FMAs of the next (software pipeline).
template <int TR, int TW, int LPR, int D, int C, bool UNR = false, typename Sink>
__device__ __forceinline__ void tile_matvec_chunk(const float2 (&st)[TR][TW / 2], const float* op,
                                                  int cg, Sink sink) {
  constexpr int NV = TW / 4;
  // partial row sums of tokens t, t+1 over this thread's columns, folded to one float per row
  auto pair_partial = [&](int t, float (&v)[2][LPR]) {
    float2 acc[2][TR];
#pragma unroll
    for (int k = 0; k < 2; ++k)
#pragma unroll
      for (int r = 0; r < TR; ++r) acc[k][r] = make_float2(0.f, 0.f);
#pragma unroll
    for (int m = 0; m < NV; ++m) {
      const float4 a4 = reinterpret_cast<const float4*>(op + t * D)[m * LPR + cg];
      const float4 b4 = reinterpret_cast<const float4*>(op + (t + 1) * D)[m * LPR + cg];
      const float2 a01 = make_float2(a4.x, a4.y), a23 = make_float2(a4.z, a4.w);
      const float2 b01 = make_float2(b4.x, b4.y), b23 = make_float2(b4.z, b4.w);
#pragma unroll
      for (int r = 0; r < TR; ++r) {
        acc[0][r] = ffma2(st[r][2 * m], a01, acc[0][r]);
        acc[1][r] = ffma2(st[r][2 * m], b01, acc[1][r]);
        acc[0][r] = ffma2(st[r][2 * m + 1], a23, acc[0][r]);
        acc[1][r] = ffma2(st[r][2 * m + 1], b23, acc[1][r]);
      }
    }
#pragma unroll
    for (int k = 0; k < 2; ++k)
#pragma unroll
      for (int r = 0; r < TR; ++r) v[k][r] = acc[k][r].x + acc[k][r].y;
  };
  float v[2][LPR];
  pair_partial(0, v);
  // rolled, except (UNR) in the two-group kernel at d = 64: there a group is two warps, one per
  // scheduler, and what the rolled loop cannot overlap (operand loads behind the previous pair's
  // stores, the reduce-scatter) was a quarter of group S's chain; at d = 32 and d = 128, and in the
  // three-group kernel (two CTAs per SM, 146 registers a thread), the longer code costs more than it saves
#pragma unroll(UNR ? C / 2 : 1)
  for (int t = 2; t < C; t += 2) {
    float vn[2][LPR];
    pair_partial(t, vn);          // independent of the shuffles below: issued together
    reduce_scatter<LPR, 2>(v, cg);
    sink(t - 2, v[0][0]);
    sink(t - 1, v[1][0]);
#pragma unroll
    for (int k = 0; k < 2; ++k)
#pragma unroll
      for (int r = 0; r < LPR; ++r) v[k][r] = vn[k][r];
  }
  reduce_scatter<LPR, 2>(v, cg);
  sink(C - 2, v[0][0]);
  sink(C - 1, v[1][0]);
}

// tile += sum_s scale[s] * coef[s][rows of the tile] (x) vec[s][cols of the tile]   (rank-16
// update; scale == nullptr means 1)
template <int TR, int TW, int LPR, int D, int C, bool UNR = false>
__device__ __forceinline__ void tile_rank_update(float2 (&st)[TR][TW / 2], const float* coef,
                                                 const float* vec, const float* scale, int rb,
                                                 int cg) {
  constexpr int NV = TW / 4;
  // (UNR: the two-group kernel at d = 64, as for the mat-vec: eight tokens' operand loads in
  // flight instead of two; at d = 32 and d = 128 deeper unrolling was slower)
  constexpr int kRuUnroll = UNR ? 8 : 2;
#pragma unroll(kRuUnroll)
  for (int s2 = 0; s2 < C; ++s2) {
    const float sc = scale ? scale[s2] : 1.0f;
    float cf[TR];
#pragma unroll
    for (int r4 = 0; r4 < TR / 4; ++r4) {
      const float4 x = reinterpret_cast<const float4*>(coef + s2 * D + rb * TR)[r4];
      cf[4 * r4 + 0] = x.x * sc; cf[4 * r4 + 1] = x.y * sc;
      cf[4 * r4 + 2] = x.z * sc; cf[4 * r4 + 3] = x.w * sc;
    }
#pragma unroll
    for (int m = 0; m < NV; ++m) {
      const float4 z4 = reinterpret_cast<const float4*>(vec + s2 * D)[m * LPR + cg];
      const float2 z01 = make_float2(z4.x, z4.y), z23 = make_float2(z4.z, z4.w);
#pragma unroll
      for (int r = 0; r < TR; ++r) {
        const float2 cc = make_float2(cf[r], cf[r]);
        st[r][2 * m] = ffma2(cc, z01, st[r][2 * m]);
        st[r][2 * m + 1] = ffma2(cc, z23, st[r][2 * m + 1]);
      }
    }
  }
}

// G[i][j] = X[i] . Y[j] for two sets of C = 16 row vectors of length D (row stride D): 4x4
// output tiles, NG/16 threads per tile splitting the D index; result rows have stride CP.
template <int D, int NG, int CP>
__device__ __forceinline__ void gram16(const float* X, const float* Y, float* G, int g) {
  constexpr int P = NG / 16;
  const int tile = g / P, part = g % P;
  const int i0 = (tile >> 2) * 4, j0 = (tile & 3) * 4;
  float2 w2[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) w2[i] = make_float2(0.f, 0.f);
#pragma unroll
  for (int step = 0; step < D / (4 * P); ++step) {
    const int f = step * P + part;
    float4 a[4], b[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      a[i] = reinterpret_cast<const float4*>(X + (i0 + i) * D)[f];
      b[i] = reinterpret_cast<const float4*>(Y + (j0 + i) * D)[f];
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

// ---------------------------------------------------------------- work distribution
// Plain: one CTA per unit.  Balanced: a persistent grid of G co-resident CTAs; the units'
// chunk sequences are laid end to end and cut into G equal segments, so a unit may be
// started by one CTA (its "head", executed FIRST by that CTA) and finished by the next
// (its "tail", executed LAST), with the state handed over through the caller's S_T / A_T /
// zT buffers and a per-unit flag.  This removes the idle SMs of a last partial wave
// (512 units on 148 SMs: 3.46 segments of work per SM instead of 4).
static __device__ unsigned int g_sched_flags[kSchedSlots * kSchedMaxUnits];

// TRI: a third warp group runs the segment's transfer scan (S from I, v = 0; sequence-parallel
// launches at d <= 64) next to group S, on the same products of group A.  Its readout goes to
// out2 and its final state to S_T[n_main + unit].
// STASH: the launch also leaves z_t, e_t, delta_t of every token in global memory (and may
// drop the readout) for the backward pass; a separate instantiation so that the plain forward
// kernel carries none of it.
// TM: q, k, v, u, out are [B, T, H, d]: the 16 rows of a chunk are H * d apart, so they move as
// one tiled TMA request per array (box d x 1 x 16 x 1 of the 4-d tensor) through the tensor maps
// in `maps`; the head-major instantiations take an empty struct there.
template <int D, typename TIn, bool BALANCED, int UM, bool TRI = false, bool STASH = false, bool TM = false>
__global__ void __launch_bounds__((ChunkCfg<D, TIn, UM, TRI>::NT), (TRI && sizeof(TIn) == 2) ? 2 : 1)
vla_scan_chunk_kernel(const ScanParams p, const SchedParams sp,
                      const __grid_constant__ typename ChunkMapsArg<TM>::type maps) {
  using Cfg = ChunkCfg<D, TIn, UM, TRI>;
  static_assert(!TM || !TRI, "token-major tensors: not with the three-group kernel");
  static_assert(!TM || (Cfg::raw_bytes + sizeof(float) * (Cfg::KRING * Cfg::kslot_floats + Cfg::RING * Cfg::slot_floats +
                                                          Cfg::a_floats + 3 * Cfg::C * D)) % 128 == 0,
                "the out stage must be 128-byte aligned for a tiled TMA store");
  static_assert(!TRI || (D <= 64 && !BALANCED), "three groups: d <= 64, one CTA per unit");
  static_assert(!STASH || !TRI, "the stash: not with the three-group kernel");
  constexpr bool HAS_U = Cfg::GEN;   // general path: a_t = A_t k_hat_t formed explicitly
  constexpr bool kUnrollMatvec = D == 64 && !TRI;
  constexpr bool UT = Cfg::UT;       // u comes from the caller's tensor
  constexpr int NIN = Cfg::NIN;
  constexpr int C = Cfg::C, TW = Cfg::TW, TR = Cfg::TR, LPR = Cfg::LPR, NV = Cfg::NV;
  constexpr int NG = Cfg::NG, NWG = Cfg::NWG, NSTAGE = Cfg::NSTAGE, RING = Cfg::RING;
  constexpr int KRING = Cfg::KRING, CP = Cfg::CP;
  static_assert(TR == LPR, "row ownership after the reduce-scatter needs TR == D/TW");
  static_assert(C == 16, "the small-matrix code is written for 16-token chunks");

  extern __shared__ __align__(128) unsigned char smem[];
  TIn* raw = reinterpret_cast<TIn*>(smem);
  float* fbase = reinterpret_cast<float*>(smem + Cfg::raw_bytes);
  float* kring = fbase;                               // [KRING] { Kh, Qf, Vf : [C][D], nrm[C] }
  float* zring = kring + KRING * Cfg::kslot_floats;   // [RING] { Zs[C][D], GuT, HT : [C][CP], sc, inv_den : [C] }
  float* abase = zring + RING * Cfg::slot_floats;
  float* Z0s = abase;                              // [C][D]  A U^T, then Z in place (general path)
  float* W0s = UT ? Z0s + C * D : Z0s;             // [C][D]  A K^T (== A U^T unless u is a tensor)
  float* Ufs = Z0s + 2 * C * D;                    // [2][C][D] widened u      (u tensor only)
  float* Ws = abase + Cfg::a_big * C * D;          // [C][CP] U A U^T (K A K^T when u = k_hat)
  float* Ls = Ws + C * CP;                         // [C][CP] unit lower factor
  float* PTs = Ls + C * CP;                        // [C][CP] PT[t][s] = (z_s.k_t)/delta_s (general path)
  float* Guu = PTs + C * CP;                       // [C][CP] U U^T, refresh only (general path)
  float* Xs = UT ? Guu + C * CP : Ws;              // [C][CP] U A K^T (== W unless u is a tensor)
  float* Guk = UT ? Xs + C * CP : Guu;             // [C][CP] U K^T, refresh only
  float* N2p = Ws + Cfg::a_small * C * CP;         // [NWG][C]
  float* denp = N2p + NWG * C;                     // [NWG][C]
  float* dlt = denp + NWG * C;                     // [C]
  float* idl = dlt + C;                            // [C]  1/delta
  float* nidl = idl + C;                           // [C] -1/delta
  float* nrs = nidl + C;                           // [C+1] eta * (refreshes before token t of the chunk)
  // The warp index is read from lane 0 so that the compiler sees it (and the group derived from
  // it) as uniform over the warp: the role branches are then uniform branches and the warp
  // shuffles inside them compile to plain shuffles.  Taken as divergent code they are several
  // times longer, and the chunk loop then overflows the instruction cache.
  const int warp_u = __shfl_sync(0xffffffffu, int(threadIdx.x >> 5), 0);
  const int grp = warp_u / (Cfg::NG / 32);   // 0: A, 1: S, 2: transfer scan (TRI)
  float* sbase = abase + Cfg::a_floats + (grp == 2 ? Cfg::s_floats : 0);
  float* VS = sbase;                // [C][D]  B = V^T - S K^T
  float* R0s = VS + C * D;          // [C][D]
  float* Eps = R0s + C * D;         // [C][D]
  float* ostage = Eps + C * D;      // [2][C][D]
  float* GuL = ostage + 2 * C * D;  // [C][CP] GuL[t][s] = k_hat_t . a_s   (general path)
  float* HTL = GuL + C * CP;        // [C][CP] HTL[t][s] = q_t . a_s       (general path)
  uint64_t* bars = reinterpret_cast<uint64_t*>(
      (reinterpret_cast<uintptr_t>(abase + Cfg::a_floats + (Cfg::NGROUPS - 1) * Cfg::s_floats) + 15) &
      ~uintptr_t(15));
  uint64_t* full = bars;                    // [NSTAGE] raw stage filled by TMA
  uint64_t* ring_full = full + NSTAGE;      // [RING] group A published chunk c
  uint64_t* ring_empty = ring_full + RING;  // [RING] group S is done with chunk c
  uint64_t* kfull = ring_empty + RING;      // [KRING] the prep warp has widened chunk c      (PREPW)
  uint64_t* kgo = kfull + KRING;            // group A: the slot of chunk c + 1 may be written (PREPW)
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ring_empty + RING + (Cfg::PREPW ? KRING + 1 : 0));

  const int tid = threadIdx.x;
  const bool is_A = grp == 0;
  const bool is_P = Cfg::PREPW && grp == Cfg::NGROUPS;   // the prep warp
  const int gw = warp_u - grp * (NG / 32);   // warp within its group
  const int lane = tid & 31;
  const int g = gw * 32 + lane;          // thread within its group; also the row it owns
  const int sbar = 1 + grp;              // named barrier of this S-like group
  const int cg = g % LPR;                // column group
  const int rb = g / LPR;                // row block: rows rb*TR .. rb*TR+TR-1
  const bool ident = (p.flags & VLA_FLAG_IDENTITY_MAP) != 0;
  const float eps = p.eps;
  const int nch_unit = (p.T + C - 1) / C;   // chunks per unit
  unsigned int* sched_flags = g_sched_flags + size_t(sp.epoch % kSchedSlots) * kSchedMaxUnits;

  // Bounded wait shared by every mbarrier in this kernel.
  // (the caller's limit is read from the parameters where it is needed: no register is spent on
  // it in the FMA loops)
  auto wait = [&](uint64_t* bar, uint32_t parity) {
    // (a probe costs some 170 clk even when the phase is complete, a look at the abort flag 90
    // more: the common case pays for the probe only)
    if (mbar_try_wait(bar, parity)) return;
    if (*abort_flag) return;
    const bool done = p.wait_limit == 0 ? mbar_wait_bounded(bar, parity)
                                        : mbar_wait_bounded(bar, parity, p.wait_limit);
    if (!done) {
      *abort_flag = 1;
      if (p.status) atomicCAS(p.status, 0, int(VLA_ERR_DEVICE_TIMEOUT));
    }
  };
  if (tid == 0) *abort_flag = 0;

#ifdef VLA_SECTION_TIMERS
  long long tsec[12];
  for (int i = 0; i < 12; ++i) tsec[i] = 0;
  long long tlast = clock64();
#define VLA_MARK(i) { long long now_ = clock64(); tsec[i] += now_ - tlast; tlast = now_; }
#else
#define VLA_MARK(i)
#endif

  float2 st[TR][TW / 2];   // this thread's TR x TW tile of A (group A) or S (group S), as column pairs
  Piece pc;
#pragma unroll 1
  for (int pi = 0; get_piece<BALANCED>(sp, p.units, nch_unit, blockIdx.x, pi, pc); ++pi) {
  const int unit = pc.unit;
  // transfer scan of a sequence-parallel launch: inputs of unit `uin`, v = 0, S0 = I
  // TRI: the third group is the transfer scan of this very unit; otherwise transfer scans are
  // the CTAs of units >= n_main
  const bool pscan_cta = !TRI && p.n_main > 0 && unit >= p.n_main;
  const bool pscan = TRI ? (grp == 2) : pscan_cta;
  const int uin = pscan_cta ? unit - p.n_main : unit;
  const int t_begin = pc.cb * C;
  const int T = min(p.T, pc.ce * C) - t_begin;   // tokens of this piece
  const int nchunks = pc.ce - pc.cb;
  // A piece either starts its unit (from S0 / A0 / z0) or continues it (from the hand-off),
  // and either finishes it or hands it over; both kinds of end write S_T / A_T / zT.
  const bool from_handoff = t_begin > 0;
  const bool to_handoff = t_begin + T < p.T;

  // global addresses are formed where they are used (two threads of the CTA), so that they
  // do not occupy registers in the FMA loops
  auto issue = [&](int c) {
    const int s = c % NSTAGE;
    const int n = min(C, T - c * C);
    const uint32_t bytes = uint32_t(n) * D * sizeof(TIn);
    TIn* dst = raw + size_t(s) * NIN * C * D;
    if constexpr (!TM) {
      mbar_arrive_expect_tx(&full[s], (pscan_cta ? NIN - 1 : NIN) * bytes);
      const size_t tok = size_t(uin) * size_t(p.T) + size_t(t_begin) + size_t(c) * C;
      bulk_load(dst + 0 * C * D, static_cast<const TIn*>(p.q) + tok * D, bytes, &full[s]);
      bulk_load(dst + 1 * C * D, static_cast<const TIn*>(p.k) + tok * D, bytes, &full[s]);
      if (!pscan_cta) bulk_load(dst + 2 * C * D, static_cast<const TIn*>(p.v) + tok * D, bytes, &full[s]);
      if (UT) bulk_load(dst + 3 * C * D, static_cast<const TIn*>(p.u) + tok * D, bytes, &full[s]);
    } else {
      // [B, T, H, d] tensors: one tiled request per array; rows past T arrive as zeros and
      // count towards the bytes like any other
      const int b = uin / p.heads, h = uin - b * p.heads, t0 = t_begin + c * C;
      mbar_arrive_expect_tx(&full[s], NIN * uint32_t(C * D * sizeof(TIn)));
      tma_load_4d(dst + 0 * C * D, &maps.q, 0, h, t0, b, &full[s]);
      tma_load_4d(dst + 1 * C * D, &maps.k, 0, h, t0, b, &full[s]);
      tma_load_4d(dst + 2 * C * D, &maps.v, 0, h, t0, b, &full[s]);
      if (UT) tma_load_4d(dst + 3 * C * D, &maps.u, 0, h, t0, b, &full[s]);
      (void)bytes;
    }
  };

  // (re)arm the barriers of this piece; a tail piece also waits for its unit's head
  __syncthreads();
  if (tid == 0) {
    for (int s = 0; s < NSTAGE; ++s) {
      if (pi > 0) asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(smem_u32(&full[s])) : "memory");
      mbar_init(&full[s], 1);
    }
    for (int r = 0; r < RING; ++r) {
      if (pi > 0) {
        asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(smem_u32(&ring_full[r])) : "memory");
        asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(smem_u32(&ring_empty[r])) : "memory");
      }
      mbar_init(&ring_full[r], 1);
      mbar_init(&ring_empty[r], Cfg::NGROUPS - 1);
    }
    if constexpr (Cfg::PREPW) {
      for (int r = 0; r <= KRING; ++r) {   // kfull[KRING], kgo
        if (pi > 0) asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(smem_u32(&kfull[r])) : "memory");
        mbar_init(&kfull[r], 1);
      }
    }
    mbar_init_fence();
    if (from_handoff && !*abort_flag) {
      bool seen = false;
      // four times the probes of a barrier wait: a probe here is one acquire load and a short sleep
      const uint64_t probes = 4ull * (p.wait_limit ? p.wait_limit : kWaitProbeLimit);
      for (uint64_t it = 0; it < probes && !seen; ++it) {
        seen = ld_acquire_gpu(&sched_flags[unit]) == sp.epoch;
        if (!seen) __nanosleep(64);
      }
      if (!seen) {
        *abort_flag = 1;
        if (p.status) atomicCAS(p.status, 0, int(VLA_ERR_DEVICE_TIMEOUT));
      }
    }
  }
  __syncthreads();
  if (tid == 0) {  // thread 0 of group A is the TMA producer
    for (int c = 0; c < NSTAGE && c < nchunks; ++c) issue(c);
  }

  // ---- a0: load the state tile
  if (!is_P) {
    // a tail piece continues from the state its head left in the caller's output buffers
    // (written by another SM: read past L1)
    const float* src = from_handoff ? (is_A ? p.A_T : p.S_T) : (is_A ? p.A0 : (pscan ? nullptr : p.S0));
    const int usrc = from_handoff ? unit : uin;   // a transfer-scan CTA reads the A0 of its partner
#pragma unroll
    for (int r = 0; r < TR; ++r) {
      const int row = rb * TR + r;
#pragma unroll
      for (int m = 0; m < NV; ++m) {
        const int c4 = m * LPR + cg;
        float4 x;
        if (src) {
          x = __ldcg(reinterpret_cast<const float4*>(src + (size_t(usrc) * D + row) * D) + c4);
        } else {
          const float dg = is_A ? 1.0f / p.lambda : (pscan ? 1.0f : 0.0f);
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

  // Input prep of tokens [tok_lo, tok_hi) of chunk c by the warps [w0, w0 + nw): k_hat,
  // ||phi(k)||, q_f and v as fp32 rows in ring slot c % KRING (zero rows past the end of
  // the sequence).  tok_lo and tok_hi are multiples of the tokens a warp takes per pass.
  auto prep_inputs = [&](int c, int w0, int nw, int tok_lo = 0, int tok_hi = Cfg::C) {
    constexpr int LPT = (D >= 128) ? 16 : 8;   // lanes per token
    constexpr int NF = D / (4 * LPT);          // float4 groups per lane and tensor
    constexpr int TPW = 32 / LPT;              // tokens per warp pass
    const int s = c % NSTAGE;
    const int n = min(C, T - c * C);
    wait(&full[s], (c / NSTAGE) & 1);
    const TIn* rq = raw + (size_t(s) * NIN + 0) * C * D;
    const TIn* rk = raw + (size_t(s) * NIN + 1) * C * D;
    const TIn* rv = raw + (size_t(s) * NIN + 2) * C * D;
    const TIn* ru = raw + (size_t(s) * NIN + (UT ? 3 : 0)) * C * D;
    float* Uf = Ufs + size_t(c & 1) * C * D;   // penalty directions, verbatim
    float* Kh = kring + size_t(c % KRING) * Cfg::kslot_floats;
    float* Qf = Kh + C * D;
    float* Vf = Qf + C * D;
    float* nrm = Vf + C * D;
    const int sub = lane / LPT, pl = lane % LPT;
    // one token per 8 lanes; `token` does the elementwise work and returns the partial
    // sum of squares, `finish` normalises once the 8 lanes have been summed
    auto token = [&](int tt, float4 (&kf)[NF]) -> float {
      const bool act = tt < n;
      float ss = 0.f;
#pragma unroll
      for (int i = 0; i < NF; ++i) {
        const int f = i * LPT + pl;
        float4 qf = make_float4(0.f, 0.f, 0.f, 0.f), vv = qf;
        kf[i] = qf;
        if (act) {
          kf[i] = load4(rk + tt * D, f);
          qf = load4(rq + tt * D, f);
          if (!pscan_cta) vv = load4(rv + tt * D, f);
          if (!ident) {
            kf[i].x = phi_fast(kf[i].x); kf[i].y = phi_fast(kf[i].y);
            kf[i].z = phi_fast(kf[i].z); kf[i].w = phi_fast(kf[i].w);
            qf.x = phi_fast(qf.x); qf.y = phi_fast(qf.y);
            qf.z = phi_fast(qf.z); qf.w = phi_fast(qf.w);
          }
        }
        reinterpret_cast<float4*>(Qf + tt * D)[f] = qf;
        reinterpret_cast<float4*>(Vf + tt * D)[f] = vv;
        if (UT)
          reinterpret_cast<float4*>(Uf + tt * D)[f] =
              act ? load4(ru + tt * D, f) : make_float4(0.f, 0.f, 0.f, 0.f);
        ss = fmaf(kf[i].x, kf[i].x, ss); ss = fmaf(kf[i].y, kf[i].y, ss);
        ss = fmaf(kf[i].z, kf[i].z, ss); ss = fmaf(kf[i].w, kf[i].w, ss);
      }
      return ss;
    };
    auto finish = [&](int tt, float ss, const float4 (&kf)[NF]) {
      const float nr = fmaxf(sqrt_approx(ss), eps);   // max(||phi(k)||, eps)
      const float inv = rcp_nr(nr);
#pragma unroll
      for (int i = 0; i < NF; ++i)
        reinterpret_cast<float4*>(Kh + tt * D)[i * LPT + pl] =
            make_float4(kf[i].x * inv, kf[i].y * inv, kf[i].z * inv, kf[i].w * inv);
      // phi(k) = k_hat * nrm exactly as the recurrence sees it; 0 for padding rows
      if (pl == 0) nrm[tt] = (tt < n) ? nr : 0.0f;
    };
    // two tokens per lane group and iteration, so that their dependency chains interleave
    for (int tok0 = tok_lo + (gw - w0) * TPW; tok0 < tok_hi; tok0 += 2 * nw * TPW) {
      const int ta = tok0 + sub, tb = tok0 + nw * TPW + sub;
      const bool two = tok0 + nw * TPW < tok_hi;   // warp-uniform
      float4 ka[NF], kb[NF];
      float sa = token(ta, ka), sb = 0.f;
      if (two) sb = token(tb, kb);
#pragma unroll
      for (int off = LPT / 2; off >= 1; off >>= 1) {
        sa += __shfl_xor_sync(0xffffffffu, sa, off);
        sb += __shfl_xor_sync(0xffffffffu, sb, off);
      }
      finish(ta, sa, ka);
      if (two) finish(tb, sb, kb);
    }
  };

  // tokens [0, kPrepSplit) of the next chunk are widened by warps 1.., the rest by warp 0
  // after the factorisation
  constexpr int kPrepSplit = (NWG == 1) ? 0 : (NWG == 2) ? 12 : C;

  if (is_A) {
    // =====================================================================  group A
    float zk = 0.0f;  // running sum of phi(k), column g
    if (from_handoff) {
      if (p.zT) zk = __ldcg(p.zT + size_t(unit) * D + g);
    } else if (p.z0) {
      zk = p.z0[size_t(uin) * D + g];
    }

    // Periodic refresh (general path): ph = tokens since the last refresh boundary
    const bool rf_on = HAS_U && p.refresh_period > 0;
    const int rfP = rf_on ? p.refresh_period : 1;
    int ph = rf_on ? int((p.step_offset + t_begin) % rfP) : 0;

    if constexpr (!Cfg::PREPW) {
      if (nchunks > 0) prep_inputs(0, 0, NWG);
      group_bar(1, NG);
      if (g == 0 && NSTAGE < nchunks) issue(NSTAGE);   // raw stage 0 is free again
    }

    for (int c = 0; c < nchunks; ++c) {
      const int slot = c % RING;
      if constexpr (Cfg::PREPW) wait(&kfull[c % KRING], (c / KRING) & 1);   // the prep warp has widened chunk c
      const float* Kh = kring + size_t(c % KRING) * Cfg::kslot_floats;
      const float* Qf = Kh + C * D;
      float* Zs = zring + size_t(slot) * Cfg::slot_floats;
      float* GuT = Zs + C * D;
      float* HT = GuT + C * CP;
      float* scs = HT + C * CP;
      float* inv_den = scs + C;
      VLA_MARK(0)

      // ---- refresh counts: nrs[t] = eta * (refreshes after tokens < t of this chunk), so that
      //      token t sees A + nrs[t] I in its Sherman-Morrison step and A + nrs[t+1] I in a_t
      const int nv = min(C, T - c * C);                 // valid tokens of the chunk
      const bool rf_chunk = rf_on && (ph + nv) >= rfP;  // at least one refresh inside
      if (rf_on) {
        if (g <= C) nrs[g] = p.refresh_eta * float((ph + min(g, nv)) / rfP);
        ph = (ph + nv) % rfP;
      }

      // ---- running key sum and readout denominators (thread = column g): partial sums
      //      over this warp's columns of q_f,t . zkey_t
      if (!ident) {
        const float* nrm = Kh + 3 * C * D;
        float pr[16];
#pragma unroll
        for (int t = 0; t < 16; ++t) {
          zk = fmaf(Kh[t * D + g], nrm[t], zk);
          pr[t] = zk * Qf[t * D + g];
        }
        const float tot = warp_reduce_scatter16(pr, lane);
        if ((lane & 1) == 0) denp[gw * C + (lane >> 1)] = tot;
        // the backward pass restarts its walk back of the key sum from these (a walk from the
        // final sum alone would cancel catastrophically at the early tokens)
        if (STASH && p.stash_zk) p.stash_zk[(size_t(unit) * size_t(nch_unit) + size_t(pc.cb + c)) * D + g] = zk;
      }

      // ---- Z0 = A U^T (U = K when no u is given); with an explicit u also W0 = A K^T
      const float* Uf = UT ? (Ufs + size_t(c & 1) * C * D) : Kh;
      tile_matvec_chunk<TR, TW, LPR, D, C, kUnrollMatvec>(st, Uf, cg, [&](int t, float x) { Z0s[t * D + g] = x; });
      if (UT)
        tile_matvec_chunk<TR, TW, LPR, D, C, kUnrollMatvec>(st, Kh, cg, [&](int t, float x) { W0s[t * D + g] = x; });
      group_bar(1, NG);
      VLA_MARK(1)

      // ---- W = U Z0 (C x C, symmetric); with an explicit u also X[s][t] = u_s . (A k_hat_t)
      gram16<D, NG, CP>(Uf, Z0s, Ws, g);
      if (UT) gram16<D, NG, CP>(Uf, W0s, Xs, g);
      if (rf_chunk) {   // U U^T and U K^T for the refresh terms
        gram16<D, NG, CP>(Uf, Uf, Guu, g);
        if (UT) gram16<D, NG, CP>(Uf, Kh, Guk, g);
      }
      group_bar(1, NG);
      VLA_MARK(2)

      // Group S must be done with chunk c - RING: that frees Z slot `slot` and, because
      // KRING = RING + 1, the input slot that chunk c + 1 is about to overwrite.
      if (c >= RING) wait(&ring_empty[slot], ((c / RING) + 1) & 1);
      if constexpr (Cfg::PREPW) {
        if (g == 0) mbar_arrive(kgo);    // the prep warp may widen chunk c + 1 into that input slot
      }
      if (gw == NWG - 1 && lane < C) {   // denominators of this chunk into the (now free) slot
        float dd = 0.f;
#pragma unroll
        for (int w2 = 0; w2 < NWG; ++w2) dd += denp[w2 * C + lane];
        inv_den[lane] = ident ? 1.0f : rcp_nr(fmaxf(dd, eps));
      }
      VLA_MARK(3)

      // ---- warp 0: I + W = L diag(delta) L^T.  The other warps widen the next chunk's inputs.
      if (gw == 0) {
        // lane l holds row r = l & 15, columns h*8 .. h*8+7 (h = l >> 4) of M = I + W
        const int r = lane & 15, h = lane >> 4;
        float m[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) m[j] = Ws[r * CP + h * 8 + j] + ((h * 8 + j == r) ? 1.0f : 0.0f);
        if (rf_chunk) {
          // tokens s <= t: u_s . (A + nrs[s] I) u_t, i.e. the count of the earlier token
#pragma unroll
          for (int j = 0; j < 8; ++j)
            m[j] = fmaf(nrs[min(r, h * 8 + j)], Guu[r * CP + h * 8 + j], m[j]);
        }
#pragma unroll
        for (int s2 = 0; s2 < 16; ++s2) {
          const int hs = s2 >> 3, js = s2 & 7;
          // Algorithm 1 clamps delta at eps; delta >= 1 whenever A is positive definite
          const float piv = fmaxf(__shfl_sync(0xffffffffu, m[js], s2 + 16 * hs), eps);
          const float mrs = __shfl_sync(0xffffffffu, m[js], r + 16 * hs);
          const float ipiv = rcp_nr(piv);
          const float l = (r > s2) ? mrs * ipiv : 0.0f;  // L[r][s2]
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float msj = __shfl_sync(0xffffffffu, m[j], s2 + 16 * h);
            m[j] = fmaf(-l, msj, m[j]);
          }
          if (h == hs) Ls[r * CP + s2] = l;
          if (lane == 0) {
            dlt[s2] = piv; idl[s2] = ipiv; nidl[s2] = -ipiv;
            if (STASH && p.stash_delta && s2 < nv)
              p.stash_delta[size_t(unit) * size_t(p.T) + size_t(t_begin) + size_t(c) * C + s2] = piv;
          }
        }
        if (HAS_U) {
          // N[s][t] = z_s . k_hat_t (s <= t) from X by the same elimination:
          //   N[s][t] = X[s][t] - sum_{r<s} L[s][r] N[r][t];  PT[t][s] = N[s][t] / delta_s.
          // Lane t < 16 owns column t (both halves of the warp compute the same thing).
          __syncwarp();
          const int t = lane & 15;
          float nn[16];
#pragma unroll
          for (int s2 = 0; s2 < 16; ++s2) {
            float a0 = Xs[s2 * CP + t], a1 = 0.f;
            if (rf_chunk) a0 = fmaf(nrs[s2], Guk[s2 * CP + t], a0);
#pragma unroll
            for (int r4 = 0; r4 * 4 < s2; ++r4) {
              const float4 l4 = reinterpret_cast<const float4*>(Ls + s2 * CP)[r4];
              if (4 * r4 + 0 < s2) a0 = fmaf(-l4.x, nn[4 * r4 + 0], a0);
              if (4 * r4 + 1 < s2) a1 = fmaf(-l4.y, nn[4 * r4 + 1], a1);
              if (4 * r4 + 2 < s2) a0 = fmaf(-l4.z, nn[4 * r4 + 2], a0);
              if (4 * r4 + 3 < s2) a1 = fmaf(-l4.w, nn[4 * r4 + 3], a1);
            }
            nn[s2] = a0 + a1;
            if (h == 0) PTs[t * CP + s2] = (s2 <= t) ? nn[s2] * idl[s2] : 0.0f;
          }
        }
        VLA_MARK(8)
        // the factorising warp takes the tail of the prep where the other warps would
        // otherwise finish after it (one other warp at d = 64, none at d = 32)
        if constexpr (!Cfg::PREPW) {
          if (c + 1 < nchunks && kPrepSplit < C) prep_inputs(c + 1, 0, 1, kPrepSplit, C);
        }
      } else {
        if constexpr (!Cfg::PREPW) {
          if (c + 1 < nchunks) prep_inputs(c + 1, 1, NWG - 1, 0, kPrepSplit);
        }
        VLA_MARK(8)
      }
      group_bar(1, NG);
      // the raw stage of chunk c + 1 has been consumed: refill it
      if constexpr (!Cfg::PREPW) {
        if (g == 0 && c + 1 + NSTAGE < nchunks) issue(c + 1 + NSTAGE);
      }
      VLA_MARK(4)

      // ---- row g of Z by forward substitution: z_t = z0_t - sum_{s<t} L[t][s] z_s
      const float rf_tot = rf_chunk ? nrs[nv] : 0.0f;   // eta * refreshes in this chunk
      {
        float z[16];
#pragma unroll
        for (int t = 0; t < 16; ++t) {
          float a0 = Z0s[t * D + g], a1 = 0.f;
          if (rf_chunk) a0 = fmaf(nrs[t], Uf[t * D + g], a0);
#pragma unroll
          for (int s4 = 0; s4 * 4 < t; ++s4) {
            const float4 l4 = reinterpret_cast<const float4*>(Ls + t * CP)[s4];
            if (4 * s4 + 0 < t) a0 = fmaf(-l4.x, z[4 * s4 + 0], a0);
            if (4 * s4 + 1 < t) a1 = fmaf(-l4.y, z[4 * s4 + 1], a1);
            if (4 * s4 + 2 < t) a0 = fmaf(-l4.z, z[4 * s4 + 2], a0);
            if (4 * s4 + 3 < t) a1 = fmaf(-l4.w, z[4 * s4 + 3], a1);
          }
          z[t] = a0 + a1;
        }
        float sq[16];
        if (!HAS_U) {
          // A_t k_hat_t = z_t / delta_t: group S gets Z itself (and sc carries the 1/delta)
#pragma unroll
          for (int t = 0; t < 16; ++t) {
            Zs[t * D + g] = z[t];
            sq[t] = z[t] * z[t];
          }
          if (STASH && p.stash_z) {   // the backward pass walks the tokens back with these
            float* zs = p.stash_z + (size_t(unit) * size_t(p.T) + size_t(t_begin) + size_t(c) * C) * D + g;
#pragma unroll
            for (int t = 0; t < 16; ++t)
              if (t < nv) zs[size_t(t) * D] = z[t];
          }
        } else {
          // a_t = A_t k_hat_t = A k_hat_t - sum_{s<=t} z_s (z_s.k_hat_t)/delta_s: group S gets a;
          // Z stays with group A (in place over Z0) for the update of A
#pragma unroll
          for (int t = 0; t < 16; ++t) {
            float a0 = W0s[t * D + g], a1 = 0.f;
            if (rf_chunk) a0 = fmaf(nrs[t + 1], Kh[t * D + g], a0);
#pragma unroll
            for (int s4 = 0; s4 * 4 <= t; ++s4) {
              const float4 p4 = reinterpret_cast<const float4*>(PTs + t * CP)[s4];
              if (4 * s4 + 0 <= t) a0 = fmaf(-p4.x, z[4 * s4 + 0], a0);
              if (4 * s4 + 1 <= t) a1 = fmaf(-p4.y, z[4 * s4 + 1], a1);
              if (4 * s4 + 2 <= t) a0 = fmaf(-p4.z, z[4 * s4 + 2], a0);
              if (4 * s4 + 3 <= t) a1 = fmaf(-p4.w, z[4 * s4 + 3], a1);
            }
            const float at = a0 + a1;
            Zs[t * D + g] = at;
            Z0s[t * D + g] = z[t];
            sq[t] = at * at;
            if (STASH && p.stash_z && t < nv) {   // backward pass with explicit u: z_t and a_t = A_t k_hat_t
              const size_t o = (size_t(unit) * size_t(p.T) + size_t(t_begin) + size_t(c) * C + t) * D + g;
              p.stash_z[o] = z[t];
              p.stash_a[o] = at;
            }
          }
        }
        const float tot = warp_reduce_scatter16(sq, lane);
        if ((lane & 1) == 0) N2p[gw * C + (lane >> 1)] = tot;
      }
      group_bar(1, NG);
      VLA_MARK(5)

      // ---- warp 0: sc_t and GuT[t][s] = Gu[s][t] = sc_s delta_s L[t][s]
      if (gw == 0) {
        const int r = lane & 15, h = lane >> 4;
        float n2 = 0.f;
#pragma unroll
        for (int w2 = 0; w2 < NWG; ++w2) n2 += N2p[w2 * C + r];
        const float id_r = idl[r], d_r = dlt[r];
        // u = k_hat:   alpha_r = sc_r z_r, sc_r = (1/delta) / max(||z||/delta, eps)
        // explicit u:  alpha_r = sc_r a_r, sc_r = 1 / max(||a||, eps)
        const float sc_r = HAS_U ? rcp_nr(fmaxf(sqrt_approx(n2), eps))
                                 : id_r * rcp_nr(fmaxf(sqrt_approx(n2) * id_r, eps));
        if ((p.flags & VLA_FLAG_CHECK_FINITE) && p.status && !isfinite(n2 + d_r))
          atomicCAS(p.status, 0, int(VLA_ERR_NONFINITE));
        if (h == 0) scs[r] = sc_r;
        if (!HAS_U) {
          const float scd = sc_r * d_r;   // multiplies column r of L
          // lane (r, h) writes GuT[r][h*8 .. h*8+7]: GuT[r][s] = scd_s L[r][s]
          float lr[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) lr[j] = Ls[r * CP + h * 8 + j];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int s2 = h * 8 + j;
            const float scd_s = __shfl_sync(0xffffffffu, scd, s2);
            GuT[r * CP + s2] = (s2 < r) ? scd_s * lr[j] : 0.0f;
          }
        }
      }
      // ---- HT[t][s] = q_t . z_s (C x C), then publish the chunk to group S.  On the general
      //      path group S forms its two small matrices from a itself, and at d <= 64 it forms
      //      HT as well (there group A is the longer chain).
      if (!HAS_U && !Cfg::S_HT) gram16<D, NG, CP>(Qf, Zs, HT, g);
      group_bar(1, NG);
      if (g == 0) mbar_arrive(&ring_full[slot]);
      VLA_MARK(6)

      // ---- A <- A - Z diag(1/delta) Z^T
      {
        const float* Zown = HAS_U ? Z0s : Zs;
        tile_rank_update<TR, TW, LPR, D, C, kUnrollMatvec>(st, Zown, Zown, nidl, rb, cg);
        if (rf_chunk) {   // + eta I per refresh: the diagonal entries that fall in this tile
#pragma unroll
          for (int r = 0; r < TR; ++r)
#pragma unroll
            for (int m = 0; m < NV; ++m) {
              const int dcol = rb * TR + r - (m * LPR + cg) * 4;   // row - first column of the quad
              if (dcol == 0) st[r][2 * m].x += rf_tot;
              if (dcol == 1) st[r][2 * m].y += rf_tot;
              if (dcol == 2) st[r][2 * m + 1].x += rf_tot;
              if (dcol == 3) st[r][2 * m + 1].y += rf_tot;
            }
        }
      }
      VLA_MARK(7)
    }
    if (p.zT) p.zT[size_t(unit) * D + g] = zk;
    // final (or handed-over) A
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
  } else if (is_P) {
    // =====================================================================  prep warp (d <= 64)
    // Chunk c + 1 is widened once group A, in chunk c, has seen group S finish the chunk whose
    // input slot it takes; the raw stage it consumed is refilled straight away.
    for (int c = 0; c < nchunks; ++c) {
      if (c > 0) wait(kgo, (c - 1) & 1);
      prep_inputs(c, 0, 1);
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(&kfull[c % KRING]);
        if (c + NSTAGE < nchunks) issue(c + NSTAGE);
      }
    }
  } else {
    // =====================================================================  group S
    for (int c = 0; c < nchunks; ++c) {
      const int n = min(C, T - c * C);
      const int slot = c % RING;
      VLA_MARK(0)
      // ---- group A's products of this chunk: k_hat, q_f, v, ||phi(k)||, Z, Gu, HT, sc
      wait(&ring_full[slot], (c / RING) & 1);
      const float* Kh = kring + size_t(c % KRING) * Cfg::kslot_floats;
      const float* Qf = Kh + C * D;
      const float* Vf = Qf + C * D;
      const float* Zs = zring + size_t(slot) * Cfg::slot_floats;
      const float* GuT = Zs + C * D;
      const float* HT = GuT + C * CP;
      const float* scs = HT + C * CP;
      const float* inv_den = scs + C;
      VLA_MARK(1)

      // ---- B = V^T - S K^T and R0 = S Q^T, row g of each
      tile_matvec_chunk<TR, TW, LPR, D, C, kUnrollMatvec>(st, Kh, cg, [&](int t, float x) {
        VS[t * D + g] = (TRI && pscan ? 0.0f : Vf[t * D + g]) - x;
      });
      tile_matvec_chunk<TR, TW, LPR, D, C, kUnrollMatvec>(st, Qf, cg, [&](int t, float x) { R0s[t * D + g] = x; });
      if (g == 0) bulk_wait_read<1>();  // the out stage of chunk c-2 has left shared memory
      // explicit u: the ring's Z slot carries a_t = A_t k_hat_t; the two small matrices
      // k_hat_t . a_s and q_t . a_s are formed here (for u = k_hat they come from group A)
      const float* Gm = GuT;
      const float* Hm = HT;
      if (HAS_U) {
        gram16<D, NG, CP>(Kh, Zs, GuL, g);
        gram16<D, NG, CP>(Qf, Zs, HTL, g);
        group_bar(sbar, NG);
        Gm = GuL;
        Hm = HTL;
      } else if (Cfg::S_HT) {
        gram16<D, NG, CP>(Qf, Zs, HTL, g);
        group_bar(sbar, NG);
        Hm = HTL;
      }
      VLA_MARK(2)

      // ---- row g: e_t = b_t - sum_{s<t} Gu[s][t] e_s; e'_t = sc_t e_t;
      //             o_t = (r0_t + sum_{s<=t} e'_s HT[t][s]) / den_t
      //      (u = k_hat: Gm holds Gu with sc folded in; explicit u: Gm holds k_hat_t . a_s and
      //       Gu[s][t] e_s = Gm[t][s] e'_s)
      float o[16];
      {
        // (every shared-memory load of a loop ahead of its stores: the compiler cannot tell the
        // arrays apart, and a load that follows a store in program order waits for it)
        float e[16], ep[16], scv[16];
#pragma unroll
        for (int t = 0; t < 16; ++t) {
          e[t] = VS[t * D + g];
          scv[t] = scs[t];
        }
#pragma unroll
        for (int t = 0; t < 16; ++t) {
          float a0 = e[t], a1 = 0.f;
#pragma unroll
          for (int s4 = 0; s4 * 4 < t; ++s4) {
            const float4 g4 = reinterpret_cast<const float4*>(Gm + t * CP)[s4];
            if (4 * s4 + 0 < t) a0 = fmaf(-g4.x, HAS_U ? ep[4 * s4 + 0] : e[4 * s4 + 0], a0);
            if (4 * s4 + 1 < t) a1 = fmaf(-g4.y, HAS_U ? ep[4 * s4 + 1] : e[4 * s4 + 1], a1);
            if (4 * s4 + 2 < t) a0 = fmaf(-g4.z, HAS_U ? ep[4 * s4 + 2] : e[4 * s4 + 2], a0);
            if (4 * s4 + 3 < t) a1 = fmaf(-g4.w, HAS_U ? ep[4 * s4 + 3] : e[4 * s4 + 3], a1);
          }
          e[t] = a0 + a1;
          ep[t] = e[t] * scv[t];
        }
        if (STASH && p.stash_e) {
          float* es = p.stash_e + (size_t(unit) * size_t(p.T) + size_t(t_begin) + size_t(c) * C) * D + g;
#pragma unroll
          for (int t = 0; t < 16; ++t)
            if (t < n) es[size_t(t) * D] = e[t];
        }
#pragma unroll
        for (int t = 0; t < 16; ++t) {
          float a0 = R0s[t * D + g], a1 = 0.f;
#pragma unroll
          for (int s4 = 0; s4 * 4 <= t; ++s4) {
            const float4 h4 = reinterpret_cast<const float4*>(Hm + t * CP)[s4];
            if (4 * s4 + 0 <= t) a0 = fmaf(h4.x, ep[4 * s4 + 0], a0);
            if (4 * s4 + 1 <= t) a1 = fmaf(h4.y, ep[4 * s4 + 1], a1);
            if (4 * s4 + 2 <= t) a0 = fmaf(h4.z, ep[4 * s4 + 2], a0);
            if (4 * s4 + 3 <= t) a1 = fmaf(h4.w, ep[4 * s4 + 3], a1);
          }
          o[t] = a0 + a1;
        }
#pragma unroll
        for (int t = 0; t < 16; ++t) o[t] *= inv_den[t];
#pragma unroll
        for (int t = 0; t < 16; ++t) Eps[t * D + g] = ep[t];
      }
      group_bar(sbar, NG);  // bulk_wait_read above is ordered before the stage is rewritten
      {
        float* ost = ostage + size_t(c & 1) * C * D;
#pragma unroll
        for (int t = 0; t < 16; ++t) ost[t * D + g] = o[t];
      }
      fence_async_smem();
      group_bar(sbar, NG);  // Eps and the out stage complete
      if (g == 0) {
        const size_t tq = size_t(t_begin) + size_t(c) * C;
        float* odst = pscan ? p.out2 : p.out;
        if (!STASH || odst) {   // a backward pass that only wants the stash passes no readout buffer
          if constexpr (!TM) {
            bulk_store(odst + (size_t(uin) * size_t(p.T) + tq) * D, ostage + size_t(c & 1) * C * D,
                       uint32_t(n) * D * sizeof(float));
          } else {   // rows past T are clipped by the tensor map
            const int b = uin / p.heads, h = uin - b * p.heads;
            tma_store_4d(&maps.out, 0, h, int(tq), b, ostage + size_t(c & 1) * C * D);
          }
          bulk_commit();
        }
      }
      VLA_MARK(3)

      // ---- S <- S + E' Z^T
      tile_rank_update<TR, TW, LPR, D, C, kUnrollMatvec>(st, Eps, Zs, nullptr, rb, cg);
      group_bar(sbar, NG);
      if (g == 0) mbar_arrive(&ring_empty[slot]);
      VLA_MARK(4)
    }
    // final (or handed-over) S
    if (p.S_T) {
#pragma unroll
      for (int r = 0; r < TR; ++r) {
        const int row = rb * TR + r;
#pragma unroll
        for (int m = 0; m < NV; ++m)
          reinterpret_cast<float4*>(p.S_T + (size_t(TRI && pscan ? unit + p.n_main : unit) * D + row) * D)[m * LPR + cg] =
              make_float4(st[r][2 * m].x, st[r][2 * m].y, st[r][2 * m + 1].x, st[r][2 * m + 1].y);
      }
    }
    if (g == 0) bulk_wait_all<0>();
  }
  if (to_handoff) {   // every thread's state stores precede the flag
    __syncthreads();
    if (tid == 0) {
      __threadfence();
      st_release_gpu(&sched_flags[unit], sp.epoch);
    }
  }
  }  // pieces
#ifdef VLA_SECTION_TIMERS
  if (p.dbg && blockIdx.x == 0 && (g == 0 || g == 32)) {
    long long* d = p.dbg + ((is_A ? 0 : 2) + (g == 32 ? 1 : 0)) * 12;
    for (int i = 0; i < 12; ++i) d[i] = tsec[i];
  }
#endif
}

}  // namespace vla
