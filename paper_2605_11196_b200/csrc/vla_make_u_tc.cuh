// Penalty directions from a projection at d = 128 on the tensor cores (Algorithm 1, the step
// u_t = L2norm(W_u k_t) / sqrt(d_h)):
//   y_t = W_u[h] k_t,   u_t = scale * y_t / max(||y_t||, eps).
// Per head this is a dense [tokens, 128] x [128, 128] product, so it runs as tcgen05.mma
// kind::tf32 with the accumulator in tensor memory: a CTA stages W_u[h] once as an operand in
// hi/lo pairs (split around the nearest TF32 value) and then takes tiles of 128 tokens:
// Y = K Wh^T + K Wl^T (+ Kl Wh^T for fp32 keys; bf16 keys are exact in TF32), fp32 accumulation.
// Thread t of the CTA owns token t of the tile: it widens the token's row into the operand
// array, and after the products reads row t of the accumulator (tensor-memory lane t), takes its
// norm and writes the scaled row.
//
// u feeds the recurrence, whose 1e-4 bound leaves no room for a single reduced-precision pass;
// the hi/lo passes keep the product at fp32 accuracy (the dropped lo*lo term is 2^-22 of a term).
// One mbarrier, every wait on it bounded: when a wait runs out the CTA stops, frees its tensor
// memory and returns (the rows it has not reached stay unwritten).
#pragma once

#include "vla_common.cuh"
#include "vla_make_u.cuh"
#include "vla_umma.cuh"

namespace vla {

struct MakeUTcCfg {
  static constexpr int D = 128;
  static constexpr int TILE = 128;                              // tokens per tile = accumulator rows
  static constexpr size_t op_bytes = size_t(D) * TILE * 4;      // one [D/4][128] float4 operand array
  static constexpr size_t smem_bytes = 3 * op_bytes + 64;       // W hi, W lo, the keys | barrier, tensor-memory slot
};

template <typename TIn>
__device__ __forceinline__ void make_u_load8(const TIn* row, int j8, float (&x)[8]);
template <>
__device__ __forceinline__ void make_u_load8<float>(const float* row, int j8, float (&x)[8]) {
  const float4 a = __ldg(reinterpret_cast<const float4*>(row) + 2 * j8);
  const float4 b = __ldg(reinterpret_cast<const float4*>(row) + 2 * j8 + 1);
  x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
}
template <>
__device__ __forceinline__ void make_u_load8<uint16_t>(const uint16_t* row, int j8, float (&x)[8]) {
  const uint4 r = __ldg(reinterpret_cast<const uint4*>(row) + j8);
  x[0] = bf16_bits_to_f32(r.x & 0xffffu); x[1] = bf16_bits_to_f32(r.x >> 16);
  x[2] = bf16_bits_to_f32(r.y & 0xffffu); x[3] = bf16_bits_to_f32(r.y >> 16);
  x[4] = bf16_bits_to_f32(r.z & 0xffffu); x[5] = bf16_bits_to_f32(r.z >> 16);
  x[6] = bf16_bits_to_f32(r.w & 0xffffu); x[7] = bf16_bits_to_f32(r.w >> 16);
}

__device__ __forceinline__ void make_u_store8(float* row, int j8, const float (&x)[8]) {
  reinterpret_cast<float4*>(row)[2 * j8] = make_float4(x[0], x[1], x[2], x[3]);
  reinterpret_cast<float4*>(row)[2 * j8 + 1] = make_float4(x[4], x[5], x[6], x[7]);
}
__device__ __forceinline__ void make_u_store8(uint16_t* row, int j8, const float (&x)[8]) {
  auto rne = [](float v) {   // bf16, round to nearest even
    uint32_t b = __float_as_uint(v);
    b += 0x7fffu + ((b >> 16) & 1u);
    return b >> 16;
  };
  uint4 r;
  r.x = rne(x[0]) | (rne(x[1]) << 16); r.y = rne(x[2]) | (rne(x[3]) << 16);
  r.z = rne(x[4]) | (rne(x[5]) << 16); r.w = rne(x[6]) | (rne(x[7]) << 16);
  reinterpret_cast<uint4*>(row)[j8] = r;
}

template <typename TIn, typename TOut>
__global__ void __launch_bounds__(MakeUTcCfg::TILE, 1) vla_make_u_tc_kernel(const MakeUParams p) {
  using Cfg = MakeUTcCfg;
  constexpr int D = Cfg::D, TILE = Cfg::TILE;
  constexpr bool kSplitKeys = sizeof(TIn) == 4;   // fp32 keys need their lo part; bf16 keys are exact in TF32
  extern __shared__ __align__(128) unsigned char smem[];
  float4* Wh = reinterpret_cast<float4*>(smem);                      // [D/4][128 c]   hi(W[c][4 j4 ..])
  float4* Wl = reinterpret_cast<float4*>(smem + Cfg::op_bytes);      // its lo part
  float4* Kop = reinterpret_cast<float4*>(smem + 2 * Cfg::op_bytes); // [D/4][128 tokens]
  uint64_t* bar = reinterpret_cast<uint64_t*>(smem + 3 * Cfg::op_bytes);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar + 1);

  const int tid = threadIdx.x;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
  const int tiles_per_unit = (p.T + kMakeUTokensPerCta - 1) / kMakeUTokensPerCta;
  const int unit = blockIdx.x / tiles_per_unit;
  const int t_first = (blockIdx.x % tiles_per_unit) * kMakeUTokensPerCta;
  const int t_last = min(p.T, t_first + kMakeUTokensPerCta);
  const int head = unit % p.heads;
  const float* W = p.W + size_t(head) * D * D;
  const TIn* gk = static_cast<const TIn*>(p.k) + size_t(unit) * size_t(p.T) * D;
  TOut* gu = static_cast<TOut*>(p.u) + size_t(unit) * size_t(p.T) * D;

  if (tid == 0) {
    mbar_init(bar, 1);
    mbar_init_fence();
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(uint32_t(D))
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // W_u[h] as the operand whose rows are the output columns: thread c takes row c
  {
    const float4* wrow = reinterpret_cast<const float4*>(W + size_t(tid) * D);
#pragma unroll 4
    for (int j4 = 0; j4 < D / 4; ++j4) {
      float4 hi, lo;
      tf32_split4(__ldg(wrow + j4), hi, lo);
      Wh[j4 * TILE + tid] = hi;
      Wl[j4 * TILE + tid] = lo;
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tbase = *tmem_slot;
  const uint32_t trow = tbase + (uint32_t(warp & 3) << 21);   // this warp's 32 lanes of tensor memory

  const uint64_t dK = umma_desc(smem_u32(Kop), 16 * TILE, 128);
  const uint64_t dWh = umma_desc(smem_u32(Wh), 16 * TILE, 128);
  const uint64_t dWl = umma_desc(smem_u32(Wl), 16 * TILE, 128);
  const uint32_t idesc = umma_idesc_tf32(TILE, D);
  uint32_t commits = 0;
  bool ok = true;

  // this thread's token row into the operand array: the keys themselves (part 0; rounded to the
  // nearest TF32 value when they are fp32) or what that rounding left (part 1)
  auto stage_keys = [&](int t0, int n, int part) {
    const TIn* row = gk + size_t(t0 + tid) * D;
#pragma unroll 4
    for (int j8 = 0; j8 < D / 8; ++j8) {
      float x[8];
      if (tid < n) {
        make_u_load8<TIn>(row, j8, x);
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) x[i] = 0.0f;
      }
      if constexpr (kSplitKeys) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float hi = tf32_rn(x[i]);
          x[i] = part == 0 ? hi : tf32_rn(x[i] - hi);
        }
      }
      Kop[(2 * j8) * TILE + tid] = make_float4(x[0], x[1], x[2], x[3]);
      Kop[(2 * j8 + 1) * TILE + tid] = make_float4(x[4], x[5], x[6], x[7]);
    }
    fence_async_smem();   // written by threads, read by the tensor core
  };
  auto wait_products = [&]() {   // (the verdict is taken by the CTA as a whole: every thread leaves the loop together)
    const bool mine = ok && mbar_wait_bounded(bar, (commits - 1) & 1);
    ok = __syncthreads_and(mine) != 0;
    tc_fence_after();
  };

  // 16-bit keys: the next tile's row is fetched into registers while this tile's products and
  // read-out run (a CTA has the SM to itself, so nothing else hides the load)
  constexpr bool kPrefetch = sizeof(TIn) == 2;
  uint4 pre[kPrefetch ? D / 8 : 1];
  auto fetch_next = [&](int t0) {
    if constexpr (kPrefetch) {
      const bool live = t0 < t_last && t0 + tid < t_last;
      const uint4* row = reinterpret_cast<const uint4*>(gk + size_t(live ? t0 + tid : 0) * D);
#pragma unroll
      for (int j8 = 0; j8 < D / 8; ++j8) pre[j8] = live ? __ldg(row + j8) : make_uint4(0u, 0u, 0u, 0u);
    }
  };
  auto put_prefetched = [&]() {
    if constexpr (kPrefetch) {
#pragma unroll
      for (int j8 = 0; j8 < D / 8; ++j8) {
        const uint4 r = pre[j8];
        Kop[(2 * j8) * TILE + tid] = make_float4(bf16_bits_to_f32(r.x & 0xffffu), bf16_bits_to_f32(r.x >> 16),
                                                 bf16_bits_to_f32(r.y & 0xffffu), bf16_bits_to_f32(r.y >> 16));
        Kop[(2 * j8 + 1) * TILE + tid] = make_float4(bf16_bits_to_f32(r.z & 0xffffu), bf16_bits_to_f32(r.z >> 16),
                                                     bf16_bits_to_f32(r.w & 0xffffu), bf16_bits_to_f32(r.w >> 16));
      }
      fence_async_smem();
    }
  };
  fetch_next(t_first);

  for (int t0 = t_first; t0 < t_last && ok; t0 += TILE) {
    const int n = min(TILE, t_last - t0);
    if constexpr (kPrefetch) {
      put_prefetched();
      fetch_next(t0 + TILE);
    } else {
      stage_keys(t0, n, 0);
    }
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
#pragma unroll 4
      for (int j = 0; j < D / 8; ++j)
        umma_ss(tbase, dK + uint64_t(j * 2 * TILE), dWh + uint64_t(j * 2 * TILE), idesc, j > 0);
#pragma unroll 4
      for (int j = 0; j < D / 8; ++j)
        umma_ss(tbase, dK + uint64_t(j * 2 * TILE), dWl + uint64_t(j * 2 * TILE), idesc, 1);
      umma_commit(bar);
    }
    ++commits;
    if constexpr (kSplitKeys) {
      wait_products();             // the key operand has been read: its place takes the lo part
      stage_keys(t0, n, 1);
      tc_fence_before();
      __syncthreads();
      if (tid == 0) {
        tc_fence_after();
#pragma unroll 4
        for (int j = 0; j < D / 8; ++j)
          umma_ss(tbase, dK + uint64_t(j * 2 * TILE), dWh + uint64_t(j * 2 * TILE), idesc, 1);
        umma_commit(bar);
      }
      ++commits;
    }
    wait_products();
    if (ok) {
      // row tid of Y: its norm, then the scaled row
      float ss = 0.0f;
#pragma unroll 1
      for (int c0 = 0; c0 < D; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(trow + c0, r);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) ss = fmaf(__uint_as_float(r[i]), __uint_as_float(r[i]), ss);
      }
      const float f = p.scale / fmaxf(sqrtf(ss), p.eps);
#pragma unroll 1
      for (int c0 = 0; c0 < D; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(trow + c0, r);
        tmem_wait_ld();
        if (tid < n) {
          TOut* orow = gu + size_t(t0 + tid) * D;
#pragma unroll
          for (int i8 = 0; i8 < 4; ++i8) {
            float x[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) x[i] = __uint_as_float(r[8 * i8 + i]) * f;
            make_u_store8(orow, c0 / 8 + i8, x);
          }
        }
      }
    }
    tc_fence_before();
    __syncthreads();   // the accumulator and the key operand are free again
    tc_fence_after();
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tbase), "r"(uint32_t(D)) : "memory");
  }
}

}  // namespace vla
