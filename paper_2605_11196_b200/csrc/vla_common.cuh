// Shared device-side pieces of the VLA scan kernels (sm_100a): launch parameters,
// bounded mbarrier waits, 1-D bulk-async (TMA) copies, small math helpers.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "vla.h"

namespace vla {

struct ScanParams {
  const void* q;       // [units, T, D]
  const void* k;       // [units, T, D]
  const void* v;       // [units, T, D]
  const void* u;       // [units, T, D] or nullptr
  const float* S0;     // [units, D, D] or nullptr
  const float* A0;     // [units, D, D] or nullptr
  const float* z0;     // [units, D] or nullptr
  float* out;          // [units, T, D]
  float* S_T;          // may be nullptr
  float* A_T;          // may be nullptr
  float* zT;           // may be nullptr
  int* status;         // may be nullptr
  float lambda;
  float eps;
  int T;
  int units;
  uint32_t flags;
  int refresh_period;        // <= 0: no periodic refresh of A
  float refresh_eta;
  long long step_offset;     // tokens processed before this call
  int u_is_khat;             // token kernel, two-exchange path: use u = k_hat although no u was given
  // Sequence-parallel scans (chunk kernel only).  With n_main > 0, units [n_main, units) are
  // "transfer" scans: unit x reads q, k, u, A0, z0 of unit x - n_main, takes v = 0 and
  // S0 = I, and writes its readout to out2 instead of out; its S_T is then the product of
  // the segment's right-acting maps I - k_hat alpha^T.  n_main <= 0: no such units.
  int n_main;
  float* out2;               // [units - n_main, T, D]
  // Backward pass (chunk kernel, u = k_hat path): per-token z_t, e_t [units, T, D] and delta_t
  // [units, T] of the forward recurrence are left here; nullptr: not wanted.  With a stash the
  // readout may be dropped (out == nullptr).
  float* stash_z;
  float* stash_e;
  float* stash_delta;
  float* stash_zk;           // [units, ceil(T / 16), D]: the key sum after each chunk of 16 tokens
  float* stash_a;            // [units, T, D]: a_t = A_t k_hat_t (explicit u only; with u = k_hat it is z_t / delta_t)
  // Token-major tensors (VLA_FLAG_TOKEN_MAJOR): q, k, v, u, out are [B, T, heads, D] instead of
  // [B, heads, T, D]; unit = b * heads + h.  The states keep their [units, D, D] layout.
  int heads;
  // Failed probes after which a device-side wait gives up and reports VLA_ERR_DEVICE_TIMEOUT
  // (0: the library's default, kWaitProbeLimit).
  uint32_t wait_limit = 0;
#ifdef VLA_SECTION_TIMERS
  long long* dbg;      // debug builds only: per-section clock64 totals of unit 0
#endif
};

// ---------------------------------------------------------------- PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t arrivals) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(arrivals));
}

// Makes freshly initialised barriers visible to the async proxy (TMA).
__device__ __forceinline__ void mbar_init_fence() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
               "r"(bytes)
               : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n"
      "  .reg .pred p;\n"
      "  mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "  selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(done)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return done != 0;
}

// Every wait in these kernels is bounded: try_wait itself blocks for a
// hardware-defined slice, so this many failed probes is on the order of a second.
constexpr uint32_t kWaitProbeLimit = 1u << 22;

// Returns false when the limit ran out (the caller reports VLA_ERR_DEVICE_TIMEOUT and
// leaves through the common exit so that no thread is left at a CTA barrier).
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity,
                                                  uint32_t limit = kWaitProbeLimit) {
  for (uint32_t it = 0; it < limit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
  }
  return false;
}

// global -> shared bulk copy, completion counted in bytes on `bar`.
// dst, src 16-byte aligned; bytes a multiple of 16.  No multicast.
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gmem_src, uint32_t bytes,
                                          uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::
          "r"(smem_u32(smem_dst)),
      "l"(gmem_src), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}

// shared -> global bulk copy in the calling thread's bulk group.
__device__ __forceinline__ void bulk_store(void* gmem_dst, const void* smem_src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gmem_dst),
               "r"(smem_u32(smem_src)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() {
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// Where the tokens of a unit lie in q, k, v, u, out: element offset of token t and the distance
// between consecutive tokens, for both tensor layouts.
__device__ __forceinline__ size_t token_offset(const ScanParams& p, int unit, size_t t, int D) {
  if (p.flags & VLA_FLAG_TOKEN_MAJOR) {
    const int b = unit / p.heads, h = unit - b * p.heads;
    return ((size_t(b) * size_t(p.T) + t) * size_t(p.heads) + size_t(h)) * D;
  }
  return (size_t(unit) * size_t(p.T) + t) * D;
}
__device__ __forceinline__ size_t token_stride(const ScanParams& p, int D) {
  return (p.flags & VLA_FLAG_TOKEN_MAJOR) ? size_t(p.heads) * D : size_t(D);
}
// n rows of row_bytes each, `stride` elements apart in global memory, to (from) dense rows in
// shared memory: one bulk copy when the rows are adjacent, else one per row
template <typename TEl>
__device__ __forceinline__ void bulk_load_rows(TEl* smem_dst, const TEl* gmem_src, size_t stride, int n,
                                               int D, uint64_t* bar) {
  if (stride == size_t(D)) {
    bulk_load(smem_dst, gmem_src, uint32_t(n) * D * sizeof(TEl), bar);
  } else {
    for (int i = 0; i < n; ++i)
      bulk_load(smem_dst + size_t(i) * D, gmem_src + size_t(i) * stride, uint32_t(D * sizeof(TEl)), bar);
  }
}
template <typename TEl>
__device__ __forceinline__ void bulk_store_rows(TEl* gmem_dst, const TEl* smem_src, size_t stride, int n, int D) {
  if (stride == size_t(D)) {
    bulk_store(gmem_dst, smem_src, uint32_t(n) * D * sizeof(TEl));
  } else {
    for (int i = 0; i < n; ++i)
      bulk_store(gmem_dst + size_t(i) * stride, smem_src + size_t(i) * D, uint32_t(D * sizeof(TEl)));
  }
}

// ---- tiled TMA through a tensor map (token-major tensors).  The innermost coordinate is always
// 0 here (16-byte rule), loads may run past the tensor's end (zero fill), stores are clipped.
struct EmptyMaps { char unused; };
struct alignas(64) TokenMajorMaps { CUtensorMap q, k, v, u, out; };
template <bool TM> struct ChunkMapsArg { using type = EmptyMaps; };
template <> struct ChunkMapsArg<true> { using type = TokenMajorMaps; };

__device__ __forceinline__ void tma_load_4d(void* smem_dst, const CUtensorMap* map, int c0, int c1, int c2,
                                            int c3, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];" ::
          "r"(smem_u32(smem_dst)),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void tma_store_4d(const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                             const void* smem_src) {
  asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group [%0, {%1, %2, %3, %4}], [%5];" ::"l"(
                   reinterpret_cast<uint64_t>(map)),
               "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(smem_u32(smem_src))
               : "memory");
}

template <int N>
__device__ __forceinline__ void bulk_wait_read() {  // <= N groups still reading shared memory
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
template <int N>
__device__ __forceinline__ void bulk_wait_all() {  // <= N groups not yet complete
  asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory");
}
// Orders generic-proxy writes to shared memory before a later bulk store reads them.
__device__ __forceinline__ void fence_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// ---------------------------------------------------------------- math helpers
// phi(x) = ELU(x) + 1 (Section 3.3): x + 1 for x > 0, exp(x) otherwise.
__device__ __forceinline__ float phi_elu1(float x) { return x > 0.0f ? x + 1.0f : expf(x); }

__device__ __forceinline__ float bf16_bits_to_f32(uint32_t bits16) {
  return __uint_as_float(bits16 << 16);
}

// one element of a row of inputs, widened to fp32
template <typename TIn>
__device__ __forceinline__ float load1(const TIn* p, size_t i);
template <>
__device__ __forceinline__ float load1<float>(const float* p, size_t i) { return p[i]; }
template <>
__device__ __forceinline__ float load1<uint16_t>(const uint16_t* p, size_t i) {
  return __uint_as_float(uint32_t(p[i]) << 16);
}

// four consecutive elements of a shared-memory row, widened to fp32
__device__ __forceinline__ float4 load4(const float* row, int c4) {
  return reinterpret_cast<const float4*>(row)[c4];
}
__device__ __forceinline__ float4 load4(const uint16_t* row, int c4) {
  uint2 r = reinterpret_cast<const uint2*>(row)[c4];
  float4 f;
  f.x = bf16_bits_to_f32(r.x & 0xffffu);
  f.y = bf16_bits_to_f32(r.x >> 16);
  f.z = bf16_bits_to_f32(r.y & 0xffffu);
  f.w = bf16_bits_to_f32(r.y >> 16);
  return f;
}

// ---------------------------------------------------------------- helpers of the chunk kernels
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

// Fast elementwise helpers of the prep pass (relative error ~1e-6, far inside the parity bound).
// Branch-free: both sides are evaluated and selected, so a warp never diverges here.
__device__ __forceinline__ float phi_fast(float x) {
  const float xm = x > 0.0f ? 0.0f : x;   // keeps a NaN (fminf would drop it)
  float e;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(xm * 1.4426950408889634f));
  return x > 0.0f ? x + 1.0f : e;
}
__device__ __forceinline__ float sqrt_approx(float x) {
  float r;
  asm("sqrt.approx.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}
__device__ __forceinline__ float rcp_approx(float x) {
  float r;
  asm("rcp.approx.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}
// 1/x to within an ulp or so: hardware estimate plus one Newton step
__device__ __forceinline__ float rcp_nr(float x) {
  const float r = rcp_approx(x);
  return fmaf(r, fmaf(-x, r, 1.0f), r);
}

// The 16 entries of a 4 x 4 output tile, each a partial sum held by the P consecutive lanes that
// split the contraction (P = 2, 4 or 8): sum over the P lanes by halving, so that lane `part` ends
// with entries base .. base + 16/P - 1 (row-major in the tile) in w[0 .. 16/P - 1].  15 - 16/P + ...
// shuffles instead of the 16 log2(P) of an all-reduce (14 against 48 at P = 8).  Returns base.
template <int P>
__device__ __forceinline__ int tile16_reduce_scatter(float (&w)[16], int part) {
  int base = 0, n = 16;
#pragma unroll
  for (int off = P / 2; off >= 1; off >>= 1) {
    n >>= 1;
    const bool up = (part & off) != 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if (i < n) {
        const float send = up ? w[i] : w[i + n];
        const float keep = up ? w[i + n] : w[i];
        w[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
      }
    }
    if (up) base += n;
  }
  return base;
}
// ... and their store into G (row stride CP floats, tile origin (i0, j0))
template <int P, int CP>
__device__ __forceinline__ void tile16_store(float* G, int i0, int j0, const float (&w)[16], int base) {
  constexpr int CNT = 16 / P;   // 2, 4 or 8 consecutive entries
  float* dst = G + (i0 + base / 4) * CP + j0 + base % 4;
  if constexpr (CNT == 2) {
    *reinterpret_cast<float2*>(dst) = make_float2(w[0], w[1]);
  } else if constexpr (CNT == 4) {
    *reinterpret_cast<float4*>(dst) = make_float4(w[0], w[1], w[2], w[3]);
  } else {
    *reinterpret_cast<float4*>(dst) = make_float4(w[0], w[1], w[2], w[3]);
    *reinterpret_cast<float4*>(dst + CP) = make_float4(w[4], w[5], w[6], w[7]);
  }
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
  return v[0];  // token index = lane >> 1
}

// ---------------------------------------------------------------- work distribution (chunk kernels)
constexpr int kSchedSlots = 16;        // launches whose flags may be live at the same time
constexpr int kSchedMaxUnits = 4096;   // units per launch in balanced mode

struct SchedParams {
  int balanced;        // 0: plain, 1: balanced
  int grid;            // number of CTAs (balanced)
  unsigned int epoch;  // launch id; flag value that means "head of this unit is done"
};

struct Piece {
  int unit, cb, ce;      // chunks [cb, ce) of the unit
  bool from_handoff;     // state comes from S_T / A_T / zT once the unit's flag shows the epoch
  bool to_handoff;       // state goes to S_T / A_T / zT and the flag is raised
};

template <bool BALANCED>
__device__ __forceinline__ bool get_piece(const SchedParams& sp, int units, int nch, int cta,
                                          int pi, Piece& out) {
  if (!BALANCED) {
    if (pi > 0) return false;
    out.unit = cta; out.cb = 0; out.ce = nch; out.from_handoff = false; out.to_handoff = false;
    return true;
  }
  const long long N = 1LL * units * nch;
  const long long lo = cta * N / sp.grid, hi = (cta + 1) * N / sp.grid;
  if (hi <= lo) return false;
  const int xf = int(lo / nch), xl = int((hi - 1) / nch);
  const bool tail = lo > 1LL * xf * nch;                                    // first unit began earlier
  const bool head = hi < 1LL * (xl + 1) * nch && 1LL * xl * nch >= lo;      // last unit ends later
  const int wf = xf + (tail ? 1 : 0), wl = xl - (head ? 1 : 0);
  const int nwhole = wl >= wf ? wl - wf + 1 : 0;
  if (head) {
    if (pi == 0) {
      out.unit = xl; out.cb = 0; out.ce = int(hi - 1LL * xl * nch);
      out.from_handoff = false; out.to_handoff = true;
      return true;
    }
    --pi;
  }
  if (pi < nwhole) {
    out.unit = wf + pi; out.cb = 0; out.ce = nch; out.from_handoff = false; out.to_handoff = false;
    return true;
  }
  pi -= nwhole;
  if (tail && pi == 0) {
    out.unit = xf; out.cb = int(lo - 1LL * xf * nch); out.ce = nch;
    out.from_handoff = true; out.to_handoff = false;
    return true;
  }
  return false;
}

__device__ __forceinline__ unsigned int ld_acquire_gpu(const unsigned int* p) {
  unsigned int v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_gpu(unsigned int* p, unsigned int v) {
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

}  // namespace vla
