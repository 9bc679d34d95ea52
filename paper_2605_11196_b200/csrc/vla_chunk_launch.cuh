// Launchers of the chunk kernel for one (d, input type).  Each vla_chunk_d*_*.cu instantiates
// them once through VLA_DEFINE_CHUNK_TU.
#pragma once

#include "vla.h"
#include "vla_launch.h"
#include "vla_scan_chunk.cuh"

namespace vla {

// Tensor maps of q, k, v[, u], out as 4-d tensors (d, H, T, B) with a box of one chunk
// (d x 1 x 16 x 1).  Defined in vla_launch.cu.
int encode_token_major_maps(const ScanParams& p, int d, int dtype, bool has_u, TokenMajorMaps* maps);

// TM: q, k, v, u, out are [B, T, H, d] (an instantiation of its own: one bulk copy per token row).
// STASH: the forward of a backward pass (per-token z, e, delta, ... left in p.stash_*); its
// token-major instantiation exists on the plain grid only.
template <int D, typename TIn, int UM, bool TM, bool STASH = false>
int launch_chunk_um_tm(const ScanParams& p, cudaStream_t st) {
  using Cfg = ChunkCfg<D, TIn, UM>;
  static_assert(Cfg::smem_bytes <= 227 * 1024, "chunk kernel exceeds the shared memory of one CTA");
  constexpr bool BAL = !(STASH && TM);
  auto kern = vla_scan_chunk_kernel<D, TIn, false, UM, false, STASH, TM>;     // one CTA per unit
  auto kern_bal = vla_scan_chunk_kernel<D, TIn, BAL, UM, false, STASH, TM>;   // persistent grid, units cut at chunks
  if (TM && p.n_main > 0) return VLA_ERR_UNSUPPORTED;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           int(Cfg::smem_bytes)) != cudaSuccess ||
      cudaFuncSetAttribute(kern_bal, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           int(Cfg::smem_bytes)) != cudaSuccess) {
    cudaGetLastError();
    return VLA_ERR_CUDA;
  }
  SchedParams sp;
  sp.balanced = 0;
  sp.grid = p.units;
  sp.epoch = 0;
  // Balanced schedule: only when a plain launch would leave SMs idle in its last wave, every
  // CTA of the persistent grid is resident at once, and the caller's S_T / A_T / zT can carry
  // a unit's state from the CTA that starts it to the CTA that finishes it.
  // Not while the stream is being captured into a CUDA graph: the hand-over flags are keyed by a
  // launch number drawn here, on the host, and every replay of the graph would carry the same one.
  cudaStreamCaptureStatus capture = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(st, &capture) != cudaSuccess) {
    cudaGetLastError();
    capture = cudaStreamCaptureStatusActive;
  }
  int dev = 0, sms = 0, per_sm = 0;
  if (capture == cudaStreamCaptureStatusNone && cudaGetDevice(&dev) == cudaSuccess &&
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess &&
      cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern_bal, Cfg::NT, Cfg::smem_bytes) ==
          cudaSuccess) {
    const int resident = sms * per_sm;
    const bool state_out = p.S_T && p.A_T && (p.zT || (p.flags & VLA_FLAG_IDENTITY_MAP));
    if (BAL && resident > 0 && p.units > resident && p.units % resident != 0 && p.T > 0 && state_out &&
        p.units <= kSchedMaxUnits && p.n_main <= 0) {
      // the flag slot of this launch id must not still be in use by an earlier launch that may
      // overlap this one on the device (another stream): then the plain grid runs instead
      const unsigned int epoch = next_launch_epoch();
      if (sched_slot_free(epoch)) {
        sp.balanced = 1;
        sp.grid = resident;
        sp.epoch = epoch;
      }
    }
  } else {
    cudaGetLastError();
  }
  typename ChunkMapsArg<TM>::type maps;
  if constexpr (TM) {
    const int rc = encode_token_major_maps(p, D, sizeof(TIn) == 2 ? VLA_BF16 : VLA_F32, UM == kUTensor, &maps);
    if (rc != VLA_OK) return rc;
  } else {
    maps.unused = 0;
  }
  if (sp.balanced) {
    kern_bal<<<sp.grid, Cfg::NT, Cfg::smem_bytes, st>>>(p, sp, maps);
    sched_slot_mark(sp.epoch, st);
  } else {
    kern<<<sp.grid, Cfg::NT, Cfg::smem_bytes, st>>>(p, sp, maps);
  }
  note_launch(STASH ? "vla_scan_chunk_kernel(stash)" : "vla_scan_chunk_kernel", D, sizeof(TIn) == 2 ? VLA_BF16 : VLA_F32,
              sp.grid, sp.balanced);
  return cudaGetLastError() == cudaSuccess ? VLA_OK : VLA_ERR_CUDA;
}

template <int D, typename TIn, int UM>
int launch_chunk_um(const ScanParams& p, cudaStream_t st) {
  // no tokens: nothing is read or written in either layout
  if ((p.flags & VLA_FLAG_TOKEN_MAJOR) && p.T > 0) return launch_chunk_um_tm<D, TIn, UM, true>(p, st);
  return launch_chunk_um_tm<D, TIn, UM, false>(p, st);
}

template <int D, typename TIn, int UM>
int launch_chunk_stash_um(const ScanParams& p, cudaStream_t st) {
  if ((p.flags & VLA_FLAG_TOKEN_MAJOR) && p.T > 0) return launch_chunk_um_tm<D, TIn, UM, true, true>(p, st);
  return launch_chunk_um_tm<D, TIn, UM, false, true>(p, st);
}

template <int D, typename TIn>
int launch_chunk_stash_t(const ScanParams& p, cudaStream_t st) {
  if (p.u) return launch_chunk_stash_um<D, TIn, kUTensor>(p, st);
  if (p.refresh_period > 0) return launch_chunk_stash_um<D, TIn, kUKhatGen>(p, st);
  return launch_chunk_stash_um<D, TIn, kUKhat>(p, st);
}

template <int D, typename TIn>
int launch_chunk_t(const ScanParams& p, cudaStream_t st) {
  if (p.u) return launch_chunk_um<D, TIn, kUTensor>(p, st);
  // The periodic refresh makes A_t k_hat_t leave the direction of z_t: general path, u = k_hat.
  if (p.refresh_period > 0) return launch_chunk_um<D, TIn, kUKhatGen>(p, st);
  return launch_chunk_um<D, TIn, kUKhat>(p, st);
}

// Three warp groups per CTA (sequence-parallel launches at d <= 64): one CTA per segment runs
// the segment and its transfer scan on one pass of group A.  p.units CTAs, p.n_main == p.units.
template <int D, typename TIn, int UM>
int launch_chunk_tri_um(const ScanParams& p, cudaStream_t st) {
  using Cfg = ChunkCfg<D, TIn, UM, true>;
  static_assert(Cfg::smem_bytes <= 227 * 1024, "chunk kernel exceeds the shared memory of one CTA");
  auto kern = vla_scan_chunk_kernel<D, TIn, false, UM, true>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           int(Cfg::smem_bytes)) != cudaSuccess) {
    cudaGetLastError();
    return VLA_ERR_CUDA;
  }
  SchedParams sp;
  sp.balanced = 0;
  sp.grid = p.units;
  sp.epoch = 0;
  kern<<<p.units, Cfg::NT, Cfg::smem_bytes, st>>>(p, sp, EmptyMaps{0});
  note_launch("vla_scan_chunk_kernel(three groups)", D, sizeof(TIn) == 2 ? VLA_BF16 : VLA_F32, p.units, 0);
  return cudaGetLastError() == cudaSuccess ? VLA_OK : VLA_ERR_CUDA;
}

template <int D, typename TIn>
int launch_chunk_tri_t(const ScanParams& p, cudaStream_t st) {
  if constexpr (D <= 64) {
    if (p.refresh_period > 0) return VLA_ERR_UNSUPPORTED;
    if (p.u) return launch_chunk_tri_um<D, TIn, kUTensor>(p, st);
    return launch_chunk_tri_um<D, TIn, kUKhat>(p, st);
  } else {
    return VLA_ERR_UNSUPPORTED;
  }
}

template <int D, typename TIn, bool TRI>
int chunk_resident_ctas_t() {
  using Cfg = ChunkCfg<D, TIn, kUKhat, TRI>;
  auto kern = vla_scan_chunk_kernel<D, TIn, false, kUKhat, TRI>;
  int dev = 0, sms = 0, per_sm = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(Cfg::smem_bytes));
  if (e == cudaSuccess)
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, Cfg::NT, Cfg::smem_bytes);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  return sms * per_sm;
}

template <int D, typename TIn>
int chunk_resident_t(bool tri) {
  if constexpr (D <= 64) {
    if (tri) return chunk_resident_ctas_t<D, TIn, true>();
  }
  return chunk_resident_ctas_t<D, TIn, false>();
}

}  // namespace vla

// The entry points of one (d, input type): the forward kernels in one translation unit, the
// forward-with-stash kernels of the backward pass in another (they compile in parallel).
#define VLA_DEFINE_CHUNK_TU(D, TIN, TAG)                                                        \
  namespace vla {                                                                               \
  int launch_chunk_##TAG(const ScanParams& p, cudaStream_t st) { return launch_chunk_t<D, TIN>(p, st); } \
  int launch_chunk_tri_##TAG(const ScanParams& p, cudaStream_t st) {                            \
    return launch_chunk_tri_t<D, TIN>(p, st);                                                   \
  }                                                                                             \
  int chunk_resident_##TAG(bool tri) { return chunk_resident_t<D, TIN>(tri); }                  \
  }
#define VLA_DEFINE_CHUNK_STASH_TU(D, TIN, TAG)                                                  \
  namespace vla {                                                                               \
  int launch_chunk_stash_##TAG(const ScanParams& p, cudaStream_t st) {                          \
    return launch_chunk_stash_t<D, TIN>(p, st);                                                 \
  }                                                                                             \
  }
