// Dispatch from (d, input type) to the translation unit that holds the kernels, the token
// kernel's launchers, and the helper launches of the sequence-parallel path.
#include "vla.h"
#include "vla_launch.h"
#include "vla_backward.cuh"
#include "vla_backward_split.cuh"
#include "vla_make_u.cuh"
#include "vla_make_u_tc.cuh"
#include "vla_decode.cuh"
#include "vla_scan_token.cuh"
#include "vla_seqpar.cuh"

namespace vla {

#define VLA_DECLARE_CHUNK_TU(TAG)                                   \
  int launch_chunk_##TAG(const ScanParams& p, cudaStream_t st);     \
  int launch_chunk_tri_##TAG(const ScanParams& p, cudaStream_t st); \
  int chunk_resident_##TAG(bool tri);                               \
  int launch_chunk_stash_##TAG(const ScanParams& p, cudaStream_t st);
VLA_DECLARE_CHUNK_TU(d32_f32)
VLA_DECLARE_CHUNK_TU(d32_bf16)
VLA_DECLARE_CHUNK_TU(d64_f32)
VLA_DECLARE_CHUNK_TU(d64_bf16)
VLA_DECLARE_CHUNK_TU(d128_f32)
VLA_DECLARE_CHUNK_TU(d128_bf16)
#undef VLA_DECLARE_CHUNK_TU

#define VLA_CHUNK_DISPATCH(FN, ...)                                                         \
  do {                                                                                      \
    const bool f32 = dtype == VLA_F32;                                                      \
    switch (d) {                                                                            \
      case 32: return f32 ? FN##_d32_f32(__VA_ARGS__) : FN##_d32_bf16(__VA_ARGS__);         \
      case 64: return f32 ? FN##_d64_f32(__VA_ARGS__) : FN##_d64_bf16(__VA_ARGS__);         \
      case 128: return f32 ? FN##_d128_f32(__VA_ARGS__) : FN##_d128_bf16(__VA_ARGS__);      \
      default: break;                                                                       \
    }                                                                                       \
  } while (0)

int launch_chunk(int d, int dtype, const ScanParams& p, cudaStream_t st) {
  VLA_CHUNK_DISPATCH(launch_chunk, p, st);
  return VLA_ERR_UNSUPPORTED;
}

int launch_chunk_tri(int d, int dtype, const ScanParams& p, cudaStream_t st) {
  VLA_CHUNK_DISPATCH(launch_chunk_tri, p, st);
  return VLA_ERR_UNSUPPORTED;
}

int launch_chunk_stash(int d, int dtype, const ScanParams& p, cudaStream_t st) {
  VLA_CHUNK_DISPATCH(launch_chunk_stash, p, st);
  return VLA_ERR_UNSUPPORTED;
}

int chunk_resident_ctas(int d, int dtype, bool tri) {
  VLA_CHUNK_DISPATCH(chunk_resident, tri);
  return 0;
}

// ---------------------------------------------------------------- token kernel
namespace {

template <int D, typename TIn, bool HAS_U>
int launch_token_t(const ScanParams& p, cudaStream_t st) {
  using Cfg = TokenCfg<D, TIn, HAS_U>;
  auto kern = vla_scan_token_kernel<D, TIn, HAS_U>;
  // Idempotent; needed once per device and cheap enough to repeat (no global state kept).
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           int(Cfg::smem_bytes)) != cudaSuccess) {
    cudaGetLastError();
    return VLA_ERR_CUDA;
  }
  kern<<<p.units, Cfg::NT, Cfg::smem_bytes, st>>>(p);
  note_launch("vla_scan_token_kernel", D, sizeof(TIn) == 2 ? VLA_BF16 : VLA_F32, p.units, 0);
  return cudaGetLastError() == cudaSuccess ? VLA_OK : VLA_ERR_CUDA;
}

template <int D>
int launch_token_d(const ScanParams& p_in, int dtype, cudaStream_t st) {
  // The periodic refresh lives in the two-exchange variant (the write direction is no longer
  // parallel to z on a refresh step); without an explicit u that variant is told to use k_hat.
  ScanParams p = p_in;
  if (p.refresh_period > 0 && p.u == nullptr) {
    p.u = p.k;   // a valid address for the ring's fourth tensor; its contents are not used
    p.u_is_khat = 1;
  }
  const bool has_u = p.u != nullptr;
  if (dtype == VLA_F32)
    return has_u ? launch_token_t<D, float, true>(p, st) : launch_token_t<D, float, false>(p, st);
  return has_u ? launch_token_t<D, uint16_t, true>(p, st) : launch_token_t<D, uint16_t, false>(p, st);
}

}  // namespace

int launch_token(int d, int dtype, const ScanParams& p, cudaStream_t st) {
  switch (d) {
    case 16: return launch_token_d<16>(p, dtype, st);
    case 32: return launch_token_d<32>(p, dtype, st);
    case 64: return launch_token_d<64>(p, dtype, st);
    case 128: return launch_token_d<128>(p, dtype, st);
    default: return VLA_ERR_UNSUPPORTED;
  }
}

// ---------------------------------------------------------------- fp32 FMA rate probe
namespace {

// Register-only chains of fma.rn.f32: 16 independent accumulators per thread, 2048 threads
// per SM.  The result is stored only if it equals a value it cannot take, so that the loop
// is kept but no memory traffic is timed.
__global__ void __launch_bounds__(1024) fp32_fma_probe_kernel(float* sink, int iters) {
  float acc[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) acc[i] = 1.0f + 1e-3f * float(i) + 1e-6f * float(threadIdx.x);
  const float m = 0.999f, c = 1e-3f;
#pragma unroll 1
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int r = 0; r < 8; ++r)
#pragma unroll
      for (int i = 0; i < 16; ++i) acc[i] = fmaf(acc[i], m, c);
  }
  float s = 0.0f;
#pragma unroll
  for (int i = 0; i < 16; ++i) s += acc[i];
  if (s == 123456.789f) sink[0] = s;
}

}  // namespace

int launch_fp32_probe(int iters, float* sink, double* flops, cudaStream_t st) {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    cudaGetLastError();
    return VLA_ERR_CUDA;
  }
  const int grid = 2 * sms, block = 1024;
  fp32_fma_probe_kernel<<<grid, block, 0, st>>>(sink, iters);
  if (flops) *flops = 2.0 * 16.0 * 8.0 * double(iters) * double(grid) * double(block);
  return cudaGetLastError() == cudaSuccess ? VLA_OK : VLA_ERR_CUDA;
}

// ---------------------------------------------------------------- backward (token kernel)
int launch_backward(int d, int dtype, const BackwardParams& p, cudaStream_t st) {
  const bool f32 = dtype == VLA_F32;
  switch (d) {
    case 16:
      if (f32) vla_backward_token_kernel<16, float><<<p.units, 256, 0, st>>>(p);
      else vla_backward_token_kernel<16, uint16_t><<<p.units, 256, 0, st>>>(p);
      break;
    default: return VLA_ERR_UNSUPPORTED;   // d >= 32: the two reverse scans (launch_backward_split)
  }
  return cudaGetLastError() == cudaSuccess ? VLA_OK : VLA_ERR_CUDA;
}

// The two reverse scans (after the chunk kernel has left the stash), d in {32, 64, 128}.
namespace {
template <int D, typename TIn, bool UX>
int launch_backward_split_ux(const BackwardSplitParams& p, cudaStream_t st) {
  using G = BwdSplitGeom<D>;
  using M = BackwardSplitSmem<D>;
  auto ksa = vla_backward_sa_kernel<D, TIn, UX>;
  constexpr size_t smem = M::sa_bytes;
  if (cudaFuncSetAttribute(ksa, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)) != cudaSuccess ||
      cudaMemsetAsync(p.progress, 0, (size_t(p.units) + 1) * sizeof(int), st) != cudaSuccess) {
    cudaGetLastError();
    return VLA_ERR_CUDA;
  }
  if (p.units > 0x3fffffff) return VLA_ERR_INVALID_ARG;
  // one launch: the first `units` CTAs to start are the S sides, the others the A sides that follow them
  ksa<<<2 * p.units, G::NT_S, smem, st>>>(p);
  if (p.dA0) vla_backward_da0_kernel<D, TIn, UX><<<p.units, 256, 0, st>>>(p);
  return cudaGetLastError() == cudaSuccess ? VLA_OK : VLA_ERR_CUDA;
}
template <int D, typename TIn>
int launch_backward_split_t(const BackwardSplitParams& p, cudaStream_t st) {
  if (p.general) return launch_backward_split_ux<D, TIn, true>(p, st);
  return launch_backward_split_ux<D, TIn, false>(p, st);
}
}  // namespace

int launch_backward_split(int d, int dtype, const BackwardSplitParams& p, cudaStream_t st) {
  const bool f32 = dtype == VLA_F32;
  switch (d) {
    case 32: return f32 ? launch_backward_split_t<32, float>(p, st) : launch_backward_split_t<32, uint16_t>(p, st);
    case 64: return f32 ? launch_backward_split_t<64, float>(p, st) : launch_backward_split_t<64, uint16_t>(p, st);
    case 128: return f32 ? launch_backward_split_t<128, float>(p, st) : launch_backward_split_t<128, uint16_t>(p, st);
    default: return VLA_ERR_UNSUPPORTED;
  }
}

// ---------------------------------------------------------------- tensor maps (token-major tensors)
namespace {
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn() {
  // resolved through the runtime, so the library needs no link against the driver
  static EncodeTiledFn fn = [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess) {
      cudaGetLastError();
      f = nullptr;
    }
    return reinterpret_cast<EncodeTiledFn>(f);
  }();
  return fn;
}
int encode_one(CUtensorMap* m, const void* base, int d, int heads, int T, int B, bool f32) {
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) return VLA_ERR_CUDA;
  const cuuint64_t es = f32 ? 4 : 2;
  const cuuint64_t dims[4] = {cuuint64_t(d), cuuint64_t(heads), cuuint64_t(T), cuuint64_t(B)};
  const cuuint64_t strides[3] = {cuuint64_t(d) * es, cuuint64_t(heads) * d * es, cuuint64_t(T) * heads * d * es};
  const cuuint32_t box[4] = {cuuint32_t(d), 1u, 16u, 1u};
  const cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
  const CUresult r = enc(m, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4,
                         const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? VLA_OK : VLA_ERR_CUDA;
}
}  // namespace

int encode_token_major_maps(const ScanParams& p, int d, int dtype, bool has_u, TokenMajorMaps* maps) {
  if (p.heads <= 0 || p.units % p.heads != 0 || p.T <= 0) return VLA_ERR_INVALID_ARG;
  const int B = p.units / p.heads;
  const bool f32 = dtype == VLA_F32;
  int rc = encode_one(&maps->q, p.q, d, p.heads, p.T, B, f32);
  if (rc == VLA_OK) rc = encode_one(&maps->k, p.k, d, p.heads, p.T, B, f32);
  if (rc == VLA_OK) rc = encode_one(&maps->v, p.v, d, p.heads, p.T, B, f32);
  if (rc == VLA_OK) rc = encode_one(&maps->u, has_u ? p.u : p.k, d, p.heads, p.T, B, f32);
  // a forward that only leaves the backward pass's stash has no readout buffer
  if (rc == VLA_OK && p.out) rc = encode_one(&maps->out, p.out, d, p.heads, p.T, B, true);
  else if (rc == VLA_OK) maps->out = maps->q;
  return rc;
}

// ---------------------------------------------------------------- penalty directions from W_u
namespace {
template <int D, typename TIn, typename TOut>
int launch_make_u_t(const MakeUParams& p, cudaStream_t st) {
  using Cfg = MakeUCfg<D>;
  auto kern = vla_make_u_kernel<D, TIn, TOut>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(Cfg::smem_bytes)) !=
      cudaSuccess) {
    cudaGetLastError();
    return VLA_ERR_CUDA;
  }
  const long long ctas = (long long)p.units * ((p.T + kMakeUTokensPerCta - 1) / kMakeUTokensPerCta);
  if (ctas <= 0) return VLA_OK;
  if (ctas > 0x7fffffffLL) return VLA_ERR_INVALID_ARG;
  kern<<<unsigned(ctas), 256, Cfg::smem_bytes, st>>>(p);
  return cudaGetLastError() == cudaSuccess ? VLA_OK : VLA_ERR_CUDA;
}
// d = 128: the product runs on the tensor cores
template <typename TIn, typename TOut>
int launch_make_u_tc_t(const MakeUParams& p, cudaStream_t st) {
  using Cfg = MakeUTcCfg;
  auto kern = vla_make_u_tc_kernel<TIn, TOut>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(Cfg::smem_bytes)) !=
      cudaSuccess) {
    cudaGetLastError();
    return VLA_ERR_CUDA;
  }
  const long long ctas = (long long)p.units * ((p.T + kMakeUTokensPerCta - 1) / kMakeUTokensPerCta);
  if (ctas <= 0) return VLA_OK;
  if (ctas > 0x7fffffffLL) return VLA_ERR_INVALID_ARG;
  kern<<<unsigned(ctas), Cfg::TILE, Cfg::smem_bytes, st>>>(p);
  return cudaGetLastError() == cudaSuccess ? VLA_OK : VLA_ERR_CUDA;
}
int launch_make_u_tc(int in_dtype, int out_dtype, const MakeUParams& p, cudaStream_t st) {
  const bool fi = in_dtype == VLA_F32, fo = out_dtype == VLA_F32;
  if (fi) return fo ? launch_make_u_tc_t<float, float>(p, st) : launch_make_u_tc_t<float, uint16_t>(p, st);
  return fo ? launch_make_u_tc_t<uint16_t, float>(p, st) : launch_make_u_tc_t<uint16_t, uint16_t>(p, st);
}

template <int D>
int launch_make_u_d(int in_dtype, int out_dtype, const MakeUParams& p, cudaStream_t st) {
  const bool fi = in_dtype == VLA_F32, fo = out_dtype == VLA_F32;
  if (fi) return fo ? launch_make_u_t<D, float, float>(p, st) : launch_make_u_t<D, float, uint16_t>(p, st);
  return fo ? launch_make_u_t<D, uint16_t, float>(p, st) : launch_make_u_t<D, uint16_t, uint16_t>(p, st);
}
}  // namespace

int launch_make_u(int d, int in_dtype, int out_dtype, const MakeUParams& p, cudaStream_t st) {
  switch (d) {
    case 16: return launch_make_u_d<16>(in_dtype, out_dtype, p, st);
    case 32: return launch_make_u_d<32>(in_dtype, out_dtype, p, st);
    case 64: return launch_make_u_d<64>(in_dtype, out_dtype, p, st);
    case 128: return launch_make_u_tc(in_dtype, out_dtype, p, st);
    default: return VLA_ERR_UNSUPPORTED;
  }
}

// ---------------------------------------------------------------- decode kernel
namespace {

template <int D, typename TIn>
int launch_decode_t(const ScanParams& p, cudaStream_t st) {
  using Cfg = DecodeCfg<D, TIn>;
  static_assert(Cfg::smem_bytes <= 227 * 1024, "decode kernel exceeds the shared memory of one CTA");
  auto kern = vla_decode_kernel<D, TIn>;
  int dev = 0, sms = 0, per_sm = 0;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           int(Cfg::smem_bytes)) != cudaSuccess ||
      cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
      cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, Cfg::NT, Cfg::smem_bytes) !=
          cudaSuccess ||
      per_sm < 1) {
    cudaGetLastError();
    return VLA_ERR_CUDA;
  }
  const int grid = p.units < sms * per_sm ? p.units : sms * per_sm;   // persistent CTAs
  kern<<<grid, Cfg::NT, Cfg::smem_bytes, st>>>(p);
  note_launch("vla_decode_kernel", D, sizeof(TIn) == 2 ? VLA_BF16 : VLA_F32, grid, 0);
  return cudaGetLastError() == cudaSuccess ? VLA_OK : VLA_ERR_CUDA;
}

}  // namespace

int launch_decode(int d, int dtype, const ScanParams& p, cudaStream_t st) {
  const bool f32 = dtype == VLA_F32;
  switch (d) {
    case 32: return f32 ? launch_decode_t<32, float>(p, st) : launch_decode_t<32, uint16_t>(p, st);
    case 64: return f32 ? launch_decode_t<64, float>(p, st) : launch_decode_t<64, uint16_t>(p, st);
    case 128: return f32 ? launch_decode_t<128, float>(p, st) : launch_decode_t<128, uint16_t>(p, st);
    default: return VLA_ERR_UNSUPPORTED;
  }
}

// ---------------------------------------------------------------- sequence-parallel helpers
namespace {

template <int D>
int seqpar_before_d(int dtype, const SeqParParams& sp, cudaStream_t st) {
  const int N = sp.units * sp.P;
  // the Gram kernel's CTAs add into these
  if (cudaMemsetAsync(sp.Gd, 0, size_t(N) * D * D * sizeof(double), st) != cudaSuccess ||
      cudaMemsetAsync(sp.zsum, 0, size_t(N) * D * sizeof(float), st) != cudaSuccess)
    return VLA_ERR_CUDA;
  if (dtype == VLA_F32) seqpar_gram_kernel<D, float><<<dim3(N, kGramSplit), 256, 0, st>>>(sp);
  else seqpar_gram_kernel<D, uint16_t><<<dim3(N, kGramSplit), 256, 0, st>>>(sp);
  if (sp.A0) seqpar_m0_kernel<D><<<sp.units, 256, 0, st>>>(sp);
  seqpar_invert_kernel<D><<<N, 256, 0, st>>>(sp);
  return cudaGetLastError() == cudaSuccess ? VLA_OK : VLA_ERR_CUDA;
}

template <int D>
int seqpar_after_d(const SeqParParams& sp, float* A_T, float* zT, const float* AT2, const float* zT2,
                   cudaStream_t st) {
  const int N = sp.units * sp.P;
  const int Ls = sp.T / sp.P;
  const size_t comb_smem = (16 + size_t(D)) * (D + 1) * sizeof(float);
  const size_t corr_smem = (size_t(D) + 64) * (D + 4) * sizeof(float);
  if (cudaFuncSetAttribute(seqpar_combine_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           int(comb_smem)) != cudaSuccess ||
      cudaFuncSetAttribute(seqpar_correct_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           int(corr_smem)) != cudaSuccess) {
    cudaGetLastError();
    return VLA_ERR_CUDA;
  }
  seqpar_combine_kernel<D><<<dim3(sp.units, D / 16), 256, comb_smem, st>>>(sp);
  const int per_cta = kCorrectTile * kCorrectTiles;
  seqpar_correct_kernel<D><<<dim3(N, (Ls + per_cta - 1) / per_cta), 256, corr_smem, st>>>(sp);
  if (cudaGetLastError() != cudaSuccess) return VLA_ERR_CUDA;
  // final A and key sum: those of each unit's last segment
  const size_t P = size_t(sp.P);
  if (A_T &&
      cudaMemcpy2DAsync(A_T, size_t(D) * D * 4, AT2 + (P - 1) * D * D, P * D * D * 4, size_t(D) * D * 4,
                        size_t(sp.units), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return VLA_ERR_CUDA;
  if (zT && cudaMemcpy2DAsync(zT, size_t(D) * 4, zT2 + (P - 1) * D, P * D * 4, size_t(D) * 4,
                              size_t(sp.units), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return VLA_ERR_CUDA;
  return VLA_OK;
}

}  // namespace

int seqpar_before_scan(int d, int dtype, const SeqParParams& sp, cudaStream_t st) {
  switch (d) {
    case 32: return seqpar_before_d<32>(dtype, sp, st);
    case 64: return seqpar_before_d<64>(dtype, sp, st);
    case 128: return seqpar_before_d<128>(dtype, sp, st);
    default: return VLA_ERR_UNSUPPORTED;
  }
}

int seqpar_after_scan(int d, const SeqParParams& sp, float* A_T, float* zT, const float* AT2,
                      const float* zT2, cudaStream_t st) {
  switch (d) {
    case 32: return seqpar_after_d<32>(sp, A_T, zT, AT2, zT2, st);
    case 64: return seqpar_after_d<64>(sp, A_T, zT, AT2, zT2, st);
    case 128: return seqpar_after_d<128>(sp, A_T, zT, AT2, zT2, st);
    default: return VLA_ERR_UNSUPPORTED;
  }
}

// ---------------------------------------------------------------- the bounded wait, tested
// One warp waits, with the kernels' own mbar_wait_bounded, on a barrier that expects two
// arrivals and gets one: the wait can only end by running out of probes.  The kernel then does
// what the scan kernels do: it records VLA_ERR_DEVICE_TIMEOUT in the caller's status word and
// returns normally (no trap, the context stays usable).
namespace {
__global__ void wait_selftest_kernel(unsigned int probe_limit, int* status) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 2);
    mbar_init_fence();
  }
  __syncthreads();
  if (threadIdx.x == 0) mbar_arrive(&bar);      // one of the two arrivals; the other never comes
  __syncthreads();
  if (!mbar_wait_bounded(&bar, 0, probe_limit) && threadIdx.x == 0)
    atomicCAS(status, 0, int(VLA_ERR_DEVICE_TIMEOUT));
}
}  // namespace

int launch_wait_selftest(unsigned int probe_limit, int* status, cudaStream_t st) {
  wait_selftest_kernel<<<1, 32, 0, st>>>(probe_limit, status);
  note_launch("wait_selftest_kernel", 0, VLA_F32, 1, 0);
  return cudaGetLastError() == cudaSuccess ? VLA_OK : VLA_ERR_CUDA;
}

}  // namespace vla
