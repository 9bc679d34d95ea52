// C ABI of the VLA forward scan (declared in include/vla.h): host-side validation,
// kernel selection and launch.  No allocation and no synchronisation on the device-pointer
// calls.  Process-wide state kept here: the launch counter and the per-slot events of the
// balanced schedule's hand-off flags, the device address of the built-in staging buffer of
// vla_forward_host_static, and a per-thread note of the last launch (vla_last_launch).
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>

#include <cstdio>

#include <atomic>
#include <cstdint>
#include <cstring>
#include <mutex>

#include "vla.h"
#include "vla_launch.h"
#include "vla_backward_params.h"
#include "vla_make_u_params.h"

namespace {

using vla::ScanParams;

// NVTX range around the host side of an entry point (a profiler shows the launches inside it).
struct NvtxRange {
  explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
  ~NvtxRange() { nvtxRangePop(); }
};

constexpr int kMaxDevices = 64;

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int resolve_opts(const vla_opts_t* opts, vla_opts_t* r) {
  std::memset(r, 0, sizeof(*r));
  r->struct_size = sizeof(vla_opts_t);
  r->qkv_dtype = VLA_F32;
  if (opts) {
    if (opts->struct_size < offsetof(vla_opts_t, kernel) || opts->struct_size > sizeof(vla_opts_t))
      return VLA_ERR_INVALID_ARG;
    std::memcpy(r, opts, opts->struct_size);  // fields past the caller's struct stay 0
    r->struct_size = sizeof(vla_opts_t);
  }
  if (!(r->eps > 0.0f)) r->eps = 1e-4f;
  if (r->qkv_dtype != VLA_F32 && r->qkv_dtype != VLA_BF16) return VLA_ERR_INVALID_ARG;
  if (r->flags & ~uint32_t(VLA_FLAG_IDENTITY_MAP | VLA_FLAG_CHECK_FINITE | VLA_FLAG_TOKEN_MAJOR |
                           VLA_FLAG_LINEAR_ATTENTION))
    return VLA_ERR_INVALID_ARG;
  if (r->kernel != VLA_KERNEL_AUTO && r->kernel != VLA_KERNEL_TOKEN && r->kernel != VLA_KERNEL_CHUNK &&
      r->kernel != VLA_KERNEL_DECODE && r->kernel != VLA_KERNEL_CHUNK_TC)
    return VLA_ERR_INVALID_ARG;
  if (r->refresh_period > 0 && (r->step_offset < 0 || !(r->refresh_eta == r->refresh_eta)))
    return VLA_ERR_INVALID_ARG;
  return VLA_OK;
}

bool shape_supported(int d_k, int d_v) {
  return d_k == d_v && (d_k == 16 || d_k == 32 || d_k == 64 || d_k == 128);
}

// Launch ids for the balanced schedule's hand-off flags (a flag equal to the launch's id
// means "done"; ids never repeat within 2^32 launches, so the flags never need clearing).
std::atomic<unsigned int> g_launch_epoch{0};

// The chunk kernel covers d in {32, 64, 128}; d = 16 runs on the token kernel.  Both are CUDA
// paths; there is no host fallback.
bool chunk_covers(const ScanParams&, int d) { return d >= 32; }

// Very short sequences (single-step decode and the like) are bound by reading and writing
// the states once; there the token kernel is faster than a 16-token chunk that is mostly
// padding (measured crossover: T ~ 12 at d = 128, T ~ 20 at d = 64).
bool chunk_pays_off(const ScanParams& p, int d) { return p.T > (d >= 128 ? 8 : 16); }

// The single-step kernel streams the states through shared memory once: T = 1, states carried
// in and out, u = k_hat, no refresh.
bool decode_covers(const ScanParams& p, int d) {
  return p.T == 1 && d >= 32 && p.S0 && p.A0 && p.S_T && p.A_T && !p.u && p.refresh_period <= 0;
}

// The tensor-core form of the chunk kernel: d = 128, u = k_hat, no refresh; [B,H,T,d] or [B,T,H,d].
bool chunk_tc_covers(const ScanParams& p, int d) {
  return d == 128 && !p.u && p.refresh_period <= 0 && p.T > 0;
}

int launch(const ScanParams& p, int d, int dtype, int kernel, cudaStream_t st) {
  // the linear-attention comparison mode lives in the token kernel (u = k_hat instantiation)
  if (p.flags & VLA_FLAG_LINEAR_ATTENTION) {
    if (p.u || p.refresh_period > 0 || (kernel != VLA_KERNEL_AUTO && kernel != VLA_KERNEL_TOKEN))
      return VLA_ERR_UNSUPPORTED;
    return vla::launch_token(d, dtype, p, st);
  }
  if (kernel == VLA_KERNEL_CHUNK_TC)
    return chunk_tc_covers(p, d) ? vla::launch_chunk_tc(d, dtype, p, st) : VLA_ERR_UNSUPPORTED;
  if (kernel == VLA_KERNEL_DECODE && !decode_covers(p, d)) return VLA_ERR_UNSUPPORTED;
  if ((kernel == VLA_KERNEL_DECODE || kernel == VLA_KERNEL_AUTO) && decode_covers(p, d))
    return vla::launch_decode(d, dtype, p, st);
  bool chunk = chunk_covers(p, d);
  if (kernel == VLA_KERNEL_CHUNK && !chunk) return VLA_ERR_UNSUPPORTED;
  if (kernel == VLA_KERNEL_AUTO && !chunk_pays_off(p, d)) chunk = false;
  if (kernel == VLA_KERNEL_TOKEN) chunk = false;
  // d = 128: the same chunk algebra runs faster with the d x d products on the tensor cores
  if (chunk && kernel == VLA_KERNEL_AUTO && chunk_tc_covers(p, d)) return vla::launch_chunk_tc(d, dtype, p, st);
  if (chunk) return vla::launch_chunk(d, dtype, p, st);
  return vla::launch_token(d, dtype, p, st);
}

// Argument checks shared by the device- and host-pointer entry points.
int check_common(const void* q, const void* k, const void* v, float lambda_, int B, int H, int T,
                 int d_k, int d_v, const float* A0, const float* out) {
  if (B < 0 || H < 0 || T < 0 || d_k <= 0 || d_v <= 0) return VLA_ERR_INVALID_ARG;
  if (!shape_supported(d_k, d_v)) return VLA_ERR_UNSUPPORTED;
  if (!A0 && !(lambda_ > 0.0f)) return VLA_ERR_INVALID_ARG;
  const long long units = 1LL * B * H;
  if (units > 0x7fffffffLL) return VLA_ERR_INVALID_ARG;
  if (units > 0 && T > 0 && (!q || !k || !v || !out)) return VLA_ERR_INVALID_ARG;
  return VLA_OK;
}

inline size_t round256(size_t x) { return (x + 255) & ~size_t(255); }

// ---- built-in staging buffer of vla_forward_host_static
// Lives in every device's memory for as long as the library is loaded.  In host code the
// array's NAME is only a handle: the device address has to be asked for with
// cudaGetSymbolAddress, once per device, with that device current.
static __device__ __align__(256) unsigned char g_static_scratch[VLA_STATIC_SCRATCH_BYTES];

std::mutex g_scratch_mutex;
void* g_scratch_addr[kMaxDevices] = {};   // per device, filled on the first call there

// Device address of the built-in buffer on the current device.  VLA_OK and *out set, or
// VLA_ERR_INVALID_ARG when the address is not known yet and `st` is being captured into a graph
// (the one-time look-up must not happen inside a capture), or VLA_ERR_CUDA.
int static_scratch_for_current_device(cudaStream_t st, void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    cudaGetLastError();
    return VLA_ERR_CUDA;
  }
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_addr[dev]) {
    cudaStreamCaptureStatus capture = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &capture) != cudaSuccess) {
      cudaGetLastError();
      return VLA_ERR_CUDA;
    }
    if (capture != cudaStreamCaptureStatusNone) return VLA_ERR_INVALID_ARG;
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess) {
      cudaGetLastError();
      return VLA_ERR_CUDA;
    }
    g_scratch_addr[dev] = ptr;
  }
  *out = g_scratch_addr[dev];
  return VLA_OK;
}

// ---- sequence-parallel entry point: workspace layout and segment choice
struct SeqParLayout {
  size_t Gd, zsum, Astart, zstart, ST2, AT2, zT2, wn, Sstart, M0, total;
};

SeqParLayout seqpar_layout(size_t units, size_t T, size_t D, size_t P) {
  const size_t N = units * P;
  SeqParLayout L;
  size_t off = 0;
  auto take = [&](size_t bytes) { const size_t at = off; off += round256(bytes); return at; };
  L.Gd = take(N * D * D * sizeof(double));
  L.zsum = take(N * D * sizeof(float));
  L.Astart = take(N * D * D * sizeof(float));
  L.zstart = take(N * D * sizeof(float));
  L.ST2 = take(2 * N * D * D * sizeof(float));
  L.AT2 = take(2 * N * D * D * sizeof(float));
  L.zT2 = take(2 * N * D * sizeof(float));
  L.wn = take(units * T * D * sizeof(float));
  L.Sstart = take(N * D * D * sizeof(float));
  L.M0 = take(units * D * D * sizeof(double));
  L.total = off + 256;
  return L;
}

// The sequence-parallel path runs a segment and its transfer scan in one three-group CTA at
// d <= 64, and as two CTAs at d = 128 (where two states fill the register file).
constexpr bool seqpar_tri(int d) { return d <= 64; }

// Segments per unit: as many as fill the device with 2 * units * P scans, P a divisor of the
// number of 16-token chunks, at least kSeqparMinTokens tokens per segment.  1 = not worth cutting.
constexpr int kSeqparMinTokens = 64;   // shortest segment worth its Gram matrix, inversion and correction
int seqpar_choose_segments(int units, int T, int d, int dtype) {
  if (units <= 0 || T <= 0 || T % 16 != 0 || d < 32) return 1;
  const int resident = vla::chunk_resident_ctas(d, dtype, seqpar_tri(d));
  const int target = resident / ((seqpar_tri(d) ? 1 : 2) * units);
  const int nch = T / 16;
  int best = 1;
  for (int P = 2; P <= target && P <= nch; ++P)
    if (nch % P == 0 && T / P >= kSeqparMinTokens) best = P;
  return best;
}

// One event per (device, flag slot) of the balanced schedule, recorded behind the launch that
// used the slot last.  Created on first use; they live until the process exits.
constexpr int kSlotCount = 16;   // == kSchedSlots of the chunk kernel
std::mutex g_slot_mutex;
cudaEvent_t g_slot_event[kMaxDevices][kSlotCount] = {};

struct LaunchNote { char kernel[48]; int d, dtype, grid, balanced; };
thread_local LaunchNote g_last_launch = {"", 0, 0, 0, 0};

}  // namespace

namespace vla {
unsigned int next_launch_epoch() {
  unsigned int e = ++g_launch_epoch;
  if (e == 0) e = ++g_launch_epoch;   // 0 is the flags' initial value
  return e;
}

bool sched_slot_free(unsigned int epoch) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    cudaGetLastError();
    return false;
  }
  std::lock_guard<std::mutex> lock(g_slot_mutex);
  cudaEvent_t& ev = g_slot_event[dev][epoch % kSlotCount];
  if (!ev) {
    if (cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) != cudaSuccess) {
      cudaGetLastError();
      ev = nullptr;
      return false;
    }
    return true;   // never used
  }
  const cudaError_t q = cudaEventQuery(ev);
  if (q == cudaSuccess) return true;
  cudaGetLastError();   // cudaErrorNotReady (or a failure): treat the slot as busy
  return false;
}

void sched_slot_mark(unsigned int epoch, cudaStream_t st) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    cudaGetLastError();
    return;
  }
  std::lock_guard<std::mutex> lock(g_slot_mutex);
  cudaEvent_t ev = g_slot_event[dev][epoch % kSlotCount];
  if (ev && cudaEventRecord(ev, st) != cudaSuccess) cudaGetLastError();
}

void note_launch(const char* kernel, int d, int dtype, int grid, int balanced) {
  std::snprintf(g_last_launch.kernel, sizeof(g_last_launch.kernel), "%s", kernel);
  g_last_launch.d = d; g_last_launch.dtype = dtype; g_last_launch.grid = grid; g_last_launch.balanced = balanced;
}
}  // namespace vla

extern "C" {

int vla_forward(const void* q, const void* k, const void* v, float lambda_, int B, int H, int T,
                int d_k, int d_v, const float* S0, const float* A0, float* out, float* S_T,
                float* A_T, const vla_opts_t* opts, void* stream) {
  NvtxRange nvtx_range("vla_forward");
  vla_opts_t o;
  int rc = resolve_opts(opts, &o);
  if (rc != VLA_OK) return rc;
  rc = check_common(q, k, v, lambda_, B, H, T, d_k, d_v, A0, out);
  if (rc != VLA_OK) return rc;
  const void* ptrs[] = {q, k, v, o.u, S0, A0, out, S_T, A_T, o.z0, o.zT};
  for (const void* ptr : ptrs)
    if (!aligned16(ptr)) return VLA_ERR_ALIGNMENT;
  if (o.status && (reinterpret_cast<uintptr_t>(o.status) & 3u)) return VLA_ERR_ALIGNMENT;
  const int units = B * H;
  if (units == 0) return VLA_OK;

  // Few units and scratch memory at hand: cut the sequences into concurrently scanned segments
  if (o.kernel == VLA_KERNEL_AUTO && o.workspace && d_k >= 32 && o.refresh_period <= 0 &&
      !(o.flags & (VLA_FLAG_TOKEN_MAJOR | VLA_FLAG_LINEAR_ATTENTION)) && T > 0 && T % 16 == 0) {
    const int P = seqpar_choose_segments(units, T, d_k, o.qkv_dtype);
    if (P > 1 && o.workspace_bytes >= seqpar_layout(size_t(units), size_t(T), size_t(d_k), size_t(P)).total)
      return vla_forward_seqpar(q, k, v, lambda_, B, H, T, d_k, d_v, S0, A0, out, S_T, A_T, &o, P, o.workspace,
                                o.workspace_bytes, stream);
  }

  ScanParams p;
  p.q = q; p.k = k; p.v = v; p.u = o.u;
  p.S0 = S0; p.A0 = A0; p.z0 = o.z0;
  p.out = out; p.S_T = S_T; p.A_T = A_T; p.zT = o.zT;
  p.status = o.status;
  p.lambda = lambda_; p.eps = o.eps;
  p.T = T; p.units = units; p.flags = o.flags;
  p.refresh_period = o.refresh_period; p.refresh_eta = o.refresh_eta;
  p.step_offset = o.step_offset; p.u_is_khat = 0;
  p.n_main = 0; p.out2 = nullptr;
  p.stash_z = nullptr; p.stash_e = nullptr; p.stash_delta = nullptr; p.stash_zk = nullptr; p.stash_a = nullptr;
  p.heads = H;
  p.wait_limit = o.wait_probe_limit;
  return launch(p, d_k, o.qkv_dtype, o.kernel, static_cast<cudaStream_t>(stream));
}

size_t vla_host_workspace_bytes(int B, int H, int T, int d_k, int d_v, int qkv_dtype, int has_u) {
  if (B < 0 || H < 0 || T < 0 || d_k <= 0 || d_v <= 0) return 0;
  if (qkv_dtype != VLA_F32 && qkv_dtype != VLA_BF16) return 0;
  const size_t es = qkv_dtype == VLA_F32 ? 4 : 2;
  const size_t units = size_t(B) * size_t(H);
  const size_t qk = round256(units * T * d_k * es), vv = round256(units * T * d_v * es);
  const size_t ob = round256(units * T * d_v * 4);
  const size_t Sb = round256(units * d_v * d_k * 4), Ab = round256(units * d_k * d_k * 4);
  const size_t zb = round256(units * d_k * 4);
  return qk * (has_u ? 3 : 2) + vv + ob + 2 * Sb + 2 * Ab + 2 * zb + 256;
}

int vla_forward_host(const void* q, const void* k, const void* v, float lambda_, int B, int H,
                     int T, int d_k, int d_v, const float* S0, const float* A0, float* out,
                     float* S_T, float* A_T, const vla_opts_t* opts, void* workspace,
                     size_t workspace_bytes, void* stream) {
  NvtxRange nvtx_range("vla_forward_host");
  vla_opts_t o;
  int rc = resolve_opts(opts, &o);
  if (rc != VLA_OK) return rc;
  rc = check_common(q, k, v, lambda_, B, H, T, d_k, d_v, A0, out);
  if (rc != VLA_OK) return rc;
  const size_t need = vla_host_workspace_bytes(B, H, T, d_k, d_v, o.qkv_dtype, o.u != nullptr);
  if (!workspace || workspace_bytes < need) return VLA_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return VLA_ERR_ALIGNMENT;
  const size_t units = size_t(B) * size_t(H);
  if (units == 0) return VLA_OK;
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  const size_t es = o.qkv_dtype == VLA_F32 ? 4 : 2;
  const size_t qk_b = units * T * d_k * es, v_b = units * T * d_v * es;
  const size_t o_b = units * T * d_v * 4;
  const size_t S_b = units * d_v * d_k * 4, A_b = units * d_k * d_k * 4, z_b = units * d_k * 4;
  unsigned char* w = static_cast<unsigned char*>(workspace);
  auto take = [&](size_t bytes) { void* r = w; w += round256(bytes); return r; };
  void* dq = take(qk_b); void* dk = take(qk_b); void* dv = take(v_b);
  void* du = o.u ? take(qk_b) : nullptr;
  float* dout = static_cast<float*>(take(o_b));
  float* dS0 = static_cast<float*>(take(S_b)); float* dST = static_cast<float*>(take(S_b));
  float* dA0 = static_cast<float*>(take(A_b)); float* dAT = static_cast<float*>(take(A_b));
  float* dz0 = static_cast<float*>(take(z_b)); float* dzT = static_cast<float*>(take(z_b));

  // Large batches are cut into slices of whole units and pipelined over short-lived internal
  // streams by role: one stream carries every copy-in back to back (the host->device engine never
  // waits for anything: each slice has its own part of the workspace), a few streams carry the
  // scans (a slice has few units, so consecutive slices share the GPU), one stream carries every
  // copy-out.  Events order a slice's scan after its copy-in and its copy-out after its scan.
  // What stays exposed is the first copy-in and the last scan and copy-out.  Smaller problems
  // run on the caller's stream alone.
  constexpr int kMaxSlices = 32, kScanLanes = 4;
  const bool token_major = (o.flags & VLA_FLAG_TOKEN_MAJOR) != 0;
  int nslices = 1;
  {
    const size_t moved = 2 * qk_b + v_b + o_b;
    if (moved >= (size_t(64) << 20)) nslices = int(units / 8 < size_t(kMaxSlices) ? units / 8 : size_t(kMaxSlices));
    if (nslices < 1) nslices = 1;
    // [B,T,H,d] tensors: a slice is a range of batch indices (contiguous in that layout, and its
    // units b*H .. are contiguous in the [B,H,...] states), scanned as a batch of its own
    if (token_major && nslices > B) nslices = B;
  }
  cudaStream_t s_in = st, s_out = st, s_scan[kScanLanes] = {st, st, st, st};
  cudaEvent_t ev_begin = nullptr, ev_in[kMaxSlices] = {}, ev_scan[kMaxSlices] = {}, ev_done[kScanLanes + 2] = {};
  bool own_streams = false;
  auto destroy_all = [&]() {
    if (s_in != st && s_in) cudaStreamDestroy(s_in);
    if (s_out != st && s_out) cudaStreamDestroy(s_out);
    for (int i = 0; i < kScanLanes; ++i)
      if (s_scan[i] != st && s_scan[i]) cudaStreamDestroy(s_scan[i]);
    if (ev_begin) cudaEventDestroy(ev_begin);
    for (int i = 0; i < kMaxSlices; ++i) {
      if (ev_in[i]) cudaEventDestroy(ev_in[i]);
      if (ev_scan[i]) cudaEventDestroy(ev_scan[i]);
    }
    for (int i = 0; i < kScanLanes + 2; ++i)
      if (ev_done[i]) cudaEventDestroy(ev_done[i]);
  };
  if (nslices > 1) {
    auto mk_stream = [&](cudaStream_t* out) {
      *out = nullptr;
      return cudaStreamCreateWithFlags(out, cudaStreamNonBlocking) == cudaSuccess &&
             cudaStreamWaitEvent(*out, ev_begin, 0) == cudaSuccess;
    };
    auto mk_event = [&](cudaEvent_t* e) { return cudaEventCreateWithFlags(e, cudaEventDisableTiming) == cudaSuccess; };
    own_streams = mk_event(&ev_begin) && cudaEventRecord(ev_begin, st) == cudaSuccess && mk_stream(&s_in) &&
                  mk_stream(&s_out);
    for (int i = 0; i < kScanLanes && own_streams; ++i) own_streams = mk_stream(&s_scan[i]);
    for (int i = 0; i < nslices && own_streams; ++i) own_streams = mk_event(&ev_in[i]) && mk_event(&ev_scan[i]);
    for (int i = 0; i < kScanLanes + 2 && own_streams; ++i) own_streams = mk_event(&ev_done[i]);
    if (!own_streams) {   // could not set the pipeline up: run everything on the caller's stream
      cudaGetLastError();
      destroy_all();
      s_in = s_out = st;
      for (int i = 0; i < kScanLanes; ++i) s_scan[i] = st;
      ev_begin = nullptr;
      for (int i = 0; i < kMaxSlices; ++i) ev_in[i] = ev_scan[i] = nullptr;
      for (int i = 0; i < kScanLanes + 2; ++i) ev_done[i] = nullptr;
      nslices = 1;
    }
  }

  bool bad = false;
  int rc_scan = VLA_OK;
  for (int sl = 0; sl < nslices; ++sl) {
    const size_t u0 = token_major ? size_t(size_t(B) * sl / nslices) * H : units * sl / nslices;
    const size_t u1 = token_major ? size_t(size_t(B) * (sl + 1) / nslices) * H : units * (sl + 1) / nslices;
    const size_t nu = u1 - u0;
    cudaStream_t ls = s_scan[sl % kScanLanes];
    auto h2d = [&](void* d, const void* h, size_t per_unit) {
      const size_t off = u0 * per_unit, bytes = nu * per_unit;
      if (bytes && cudaMemcpyAsync(static_cast<unsigned char*>(d) + off,
                                   static_cast<const unsigned char*>(h) + off, bytes,
                                   cudaMemcpyHostToDevice, s_in) != cudaSuccess) bad = true;
    };
    auto d2h = [&](void* h, const void* d, size_t per_unit) {
      const size_t off = u0 * per_unit, bytes = nu * per_unit;
      if (bytes && cudaMemcpyAsync(static_cast<unsigned char*>(h) + off,
                                   static_cast<const unsigned char*>(d) + off, bytes,
                                   cudaMemcpyDeviceToHost, s_out) != cudaSuccess) bad = true;
    };
    auto at = [&](void* base, size_t per_unit) {
      return base ? static_cast<void*>(static_cast<unsigned char*>(base) + u0 * per_unit) : nullptr;
    };
    const size_t qk_u = size_t(T) * d_k * es, v_u = size_t(T) * d_v * es, o_u = size_t(T) * d_v * 4;
    const size_t S_u = size_t(d_v) * d_k * 4, A_u = size_t(d_k) * d_k * 4, z_u = size_t(d_k) * 4;
    h2d(dq, q, qk_u); h2d(dk, k, qk_u); h2d(dv, v, v_u);
    if (o.u) h2d(du, o.u, qk_u);
    if (S0) h2d(dS0, S0, S_u);
    if (A0) h2d(dA0, A0, A_u);
    if (o.z0) h2d(dz0, o.z0, z_u);
    if (bad) break;
    if (own_streams && (cudaEventRecord(ev_in[sl], s_in) != cudaSuccess ||
                        cudaStreamWaitEvent(ls, ev_in[sl], 0) != cudaSuccess)) { bad = true; break; }

    vla_opts_t od = o;
    od.workspace = nullptr;        // the slices run concurrently: they must not share scratch
    od.workspace_bytes = 0;
    od.u = at(du, qk_u);
    od.z0 = o.z0 ? static_cast<const float*>(at(dz0, z_u)) : nullptr;
    od.zT = static_cast<float*>(at(dzT, z_u));   // device copies of the final states are always
                                                 // kept: they let the scan cut units across CTAs
    rc_scan = vla_forward(at(dq, qk_u), at(dk, qk_u), at(dv, v_u), lambda_,
                          token_major ? int(nu / size_t(H)) : 1, token_major ? H : int(nu), T, d_k, d_v,
                          S0 ? static_cast<const float*>(at(dS0, S_u)) : nullptr,
                          A0 ? static_cast<const float*>(at(dA0, A_u)) : nullptr,
                          static_cast<float*>(at(dout, o_u)), static_cast<float*>(at(dST, S_u)),
                          static_cast<float*>(at(dAT, A_u)), &od, ls);
    if (rc_scan != VLA_OK) break;
    if (own_streams && (cudaEventRecord(ev_scan[sl], ls) != cudaSuccess ||
                        cudaStreamWaitEvent(s_out, ev_scan[sl], 0) != cudaSuccess)) { bad = true; break; }
    d2h(out, dout, o_u);
    if (S_T) d2h(S_T, dST, S_u);
    if (A_T) d2h(A_T, dAT, A_u);
    if (o.zT) d2h(o.zT, dzT, z_u);
    if (bad) break;
  }
  if (own_streams) {
    // the caller's stream continues only after every internal stream has drained; destroying a
    // stream or event with work pending is deferred by the runtime until that work is done
    cudaStream_t all[kScanLanes + 2] = {s_in, s_out, s_scan[0], s_scan[1], s_scan[2], s_scan[3]};
    for (int i = 0; i < kScanLanes + 2; ++i)
      if (cudaEventRecord(ev_done[i], all[i]) != cudaSuccess || cudaStreamWaitEvent(st, ev_done[i], 0) != cudaSuccess)
        bad = true;
    destroy_all();
  }
  if (rc_scan != VLA_OK) return rc_scan;
  if (bad) { cudaGetLastError(); return VLA_ERR_CUDA; }
  return VLA_OK;
}

int vla_forward_host_static(const void* q, const void* k, const void* v, float lambda_, int B,
                            int H, int T, int d_k, int d_v, const float* S0, const float* A0,
                            float* out, float* S_T, float* A_T, const vla_opts_t* opts,
                            void* stream) {
  NvtxRange nvtx_range("vla_forward_host_static");
  // Size check first: it needs no CUDA call and gives the clearest answer.
  vla_opts_t o;
  int rc = resolve_opts(opts, &o);
  if (rc != VLA_OK) return rc;
  rc = check_common(q, k, v, lambda_, B, H, T, d_k, d_v, A0, out);
  if (rc != VLA_OK) return rc;
  const size_t need = vla_host_workspace_bytes(B, H, T, d_k, d_v, o.qkv_dtype, o.u != nullptr);
  if (need > size_t(VLA_STATIC_SCRATCH_BYTES)) return VLA_ERR_TOO_LARGE;
  void* scratch = nullptr;
  rc = static_scratch_for_current_device(static_cast<cudaStream_t>(stream), &scratch);
  if (rc != VLA_OK) return rc;
  // Every staging region is written (by a copy or by the scan) before it is read, so
  // nothing left behind by the previous call needs clearing.
  return vla_forward_host(q, k, v, lambda_, B, H, T, d_k, d_v, S0, A0, out, S_T, A_T, opts, scratch,
                          size_t(VLA_STATIC_SCRATCH_BYTES), stream);
}

int vla_seqpar_segments(int B, int H, int T, int d_k, int qkv_dtype) {
  if (B <= 0 || H <= 0) return 1;
  if (qkv_dtype != VLA_F32 && qkv_dtype != VLA_BF16) return 1;
  const long long units = 1LL * B * H;
  if (units > 0x7fffffffLL) return 1;
  return seqpar_choose_segments(int(units), T, d_k, qkv_dtype);
}

size_t vla_seqpar_workspace_bytes(int B, int H, int T, int d_k, int segments) {
  if (B < 0 || H < 0 || T < 0 || d_k <= 0 || segments < 1) return 0;
  return seqpar_layout(size_t(B) * size_t(H), size_t(T), size_t(d_k), size_t(segments)).total;
}

int vla_forward_seqpar(const void* q, const void* k, const void* v, float lambda_, int B, int H,
                       int T, int d_k, int d_v, const float* S0, const float* A0, float* out,
                       float* S_T, float* A_T,
                       const vla_opts_t* opts, int segments, void* workspace,
                       size_t workspace_bytes, void* stream) {
  NvtxRange nvtx_range("vla_forward_seqpar");
  vla_opts_t o;
  int rc = resolve_opts(opts, &o);
  if (rc != VLA_OK) return rc;
  rc = check_common(q, k, v, lambda_, B, H, T, d_k, d_v, A0, out);
  if (rc != VLA_OK) return rc;
  if (d_k < 32 || o.refresh_period > 0 || o.kernel == VLA_KERNEL_TOKEN ||
      (o.flags & (VLA_FLAG_TOKEN_MAJOR | VLA_FLAG_LINEAR_ATTENTION)))
    return VLA_ERR_UNSUPPORTED;
  const void* ptrs[] = {q, k, v, o.u, S0, A0, out, S_T, A_T, o.z0, o.zT};
  for (const void* ptr : ptrs)
    if (!aligned16(ptr)) return VLA_ERR_ALIGNMENT;
  if (o.status && (reinterpret_cast<uintptr_t>(o.status) & 3u)) return VLA_ERR_ALIGNMENT;
  const int units = B * H;
  if (units == 0) return VLA_OK;
  int P = segments;
  if (P <= 0) P = seqpar_choose_segments(units, T, d_k, o.qkv_dtype);
  if (P == 1)   // nothing to cut: the plain scan
    return vla_forward(q, k, v, lambda_, B, H, T, d_k, d_v, S0, A0, out, S_T, A_T, opts, stream);
  if (T % 16 != 0 || (T / 16) % P != 0) return VLA_ERR_INVALID_ARG;
  if (2LL * units * P > 0x7fffffffLL) return VLA_ERR_INVALID_ARG;
  const SeqParLayout L = seqpar_layout(size_t(units), size_t(T), size_t(d_k), size_t(P));
  if (!workspace || workspace_bytes < L.total) return VLA_ERR_INVALID_ARG;
  unsigned char* w = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(workspace) + 255) & ~uintptr_t(255));
  const int N = units * P;

  vla::SeqParParams sp;
  sp.k = k; sp.u = o.u; sp.S0 = S0; sp.A0 = A0; sp.z0 = o.z0; sp.out = out; sp.S_T = S_T;
  sp.M0 = reinterpret_cast<double*>(w + L.M0);
  sp.Gd = reinterpret_cast<double*>(w + L.Gd);
  sp.zsum = reinterpret_cast<float*>(w + L.zsum);
  sp.Astart = reinterpret_cast<float*>(w + L.Astart);
  sp.zstart = reinterpret_cast<float*>(w + L.zstart);
  sp.ST2 = reinterpret_cast<float*>(w + L.ST2);
  sp.wn = reinterpret_cast<float*>(w + L.wn);
  sp.Sstart = reinterpret_cast<float*>(w + L.Sstart);
  sp.lambda = lambda_; sp.eps = o.eps; sp.T = T; sp.P = P; sp.units = units; sp.flags = o.flags;
  float* AT2 = reinterpret_cast<float*>(w + L.AT2);
  float* zT2 = reinterpret_cast<float*>(w + L.zT2);

  // every segment and its transfer scan as one launch of 2N units of T / P tokens: a unit's
  // segments are consecutive blocks of its [T, d] arrays, so the inputs need no copy
  ScanParams p;
  p.q = q; p.k = k; p.v = v; p.u = o.u;
  p.S0 = nullptr; p.A0 = sp.Astart; p.z0 = sp.zstart;
  p.out = out; p.out2 = reinterpret_cast<float*>(w + L.wn);
  p.S_T = reinterpret_cast<float*>(w + L.ST2); p.A_T = AT2; p.zT = zT2;
  p.status = o.status;
  p.lambda = lambda_; p.eps = o.eps;
  // d <= 64: N CTAs of three warp groups; d = 128: 2N CTAs, the transfer scans second
  p.T = T / P; p.units = seqpar_tri(d_k) ? N : 2 * N; p.n_main = N; p.flags = o.flags;
  p.refresh_period = 0; p.refresh_eta = 0.0f; p.step_offset = 0; p.u_is_khat = 0;
  p.stash_z = nullptr; p.stash_e = nullptr; p.stash_delta = nullptr; p.stash_zk = nullptr; p.stash_a = nullptr;
  p.heads = H;
  p.wait_limit = o.wait_probe_limit;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  rc = vla::seqpar_before_scan(d_k, o.qkv_dtype, sp, st);
  if (rc != VLA_OK) return rc;
  rc = seqpar_tri(d_k) ? vla::launch_chunk_tri(d_k, o.qkv_dtype, p, st)
                       : vla::launch_chunk(d_k, o.qkv_dtype, p, st);
  if (rc != VLA_OK) return rc;
  return vla::seqpar_after_scan(d_k, sp, A_T, o.zT, AT2, zT2, st);
}

size_t vla_backward_workspace_bytes(int B, int H, int T, int d_k) {
  if (B < 0 || H < 0 || T < 0 || d_k <= 0) return 0;
  const size_t units = size_t(B) * size_t(H);
  const size_t vec = round256(units * T * d_k * sizeof(float));
  const size_t mat = round256(units * d_k * d_k * sizeof(float));
  // z, e, dalpha, dk_hat (S part), key-sum gradient per token; delta per token; S_T, A_T, key sum;
  // the key sum after every 16 tokens; a_t per token (explicit u); the forward's readout; progress words
  const size_t ck = round256(units * ((size_t(T) + 15) / 16) * d_k * sizeof(float));
  return 7 * vec + round256(units * T * sizeof(float)) + 2 * mat + round256(units * d_k * sizeof(float)) + ck +
         round256((units + 1) * sizeof(int)) + 256;
}

int vla_backward(const void* q, const void* k, const void* v, float lambda_, int B, int H, int T,
                 int d_k, int d_v, const float* S0, const float* A0, const float* d_out,
                 const float* dS_T, const float* dA_T, const float* dz_T, float* dq, float* dk,
                 float* dv, float* dS0, float* dA0, float* dz0, const vla_opts_t* opts,
                 void* workspace, size_t workspace_bytes, void* stream) {
  NvtxRange nvtx_range("vla_backward");
  vla_opts_t o;
  int rc = resolve_opts(opts, &o);
  if (rc != VLA_OK) return rc;
  rc = check_common(q, k, v, lambda_, B, H, T, d_k, d_v, A0, d_out);
  if (rc != VLA_OK) return rc;
  // explicit u, the refresh, token-major tensors: the two reverse scans only
  const bool general = o.u || o.refresh_period > 0;
  if ((general || (o.flags & VLA_FLAG_TOKEN_MAJOR)) && d_k < 32) return VLA_ERR_UNSUPPORTED;
  if (o.flags & VLA_FLAG_LINEAR_ATTENTION) return VLA_ERR_UNSUPPORTED;   // a forward-only comparison mode
  const int units = B * H;
  if (units > 0 && T > 0 && (!dq || !dk || !dv || (o.u && !o.du))) return VLA_ERR_INVALID_ARG;
  const void* ptrs[] = {q, k, v, S0, A0, d_out, dS_T, dA_T, dz_T, dq, dk, dv, dS0, dA0, dz0, o.z0, o.u, o.du};
  for (const void* ptr : ptrs)
    if (!aligned16(ptr)) return VLA_ERR_ALIGNMENT;
  if (o.status && (reinterpret_cast<uintptr_t>(o.status) & 3u)) return VLA_ERR_ALIGNMENT;
  if (units == 0) return VLA_OK;
  if (!workspace || workspace_bytes < vla_backward_workspace_bytes(B, H, T, d_k)) return VLA_ERR_INVALID_ARG;
  unsigned char* w = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(workspace) + 255) & ~uintptr_t(255));
  const size_t vec = round256(size_t(units) * T * d_k * sizeof(float));
  const size_t mat = round256(size_t(units) * d_k * d_k * sizeof(float));
  const size_t sca = round256(size_t(units) * T * sizeof(float));
  float* zst = reinterpret_cast<float*>(w);
  float* est = reinterpret_cast<float*>(w + vec);
  float* dst = reinterpret_cast<float*>(w + 2 * vec);
  const size_t ckb = round256(size_t(units) * ((size_t(T) + 15) / 16) * d_k * sizeof(float));
  float* zkcw = reinterpret_cast<float*>(w + 5 * vec + sca + 2 * mat + round256(size_t(units) * d_k * sizeof(float)));
  float* astw = reinterpret_cast<float*>(w + 5 * vec + sca + 2 * mat + round256(size_t(units) * d_k * sizeof(float)) + ckb);
  int* progw = reinterpret_cast<int*>(w + 6 * vec + sca + 2 * mat + round256(size_t(units) * d_k * sizeof(float)) + ckb);
  float* outw = reinterpret_cast<float*>(w + 6 * vec + sca + 2 * mat + round256(size_t(units) * d_k * sizeof(float)) + ckb +
                                         round256((size_t(units) + 1) * sizeof(int)));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (d_k == 16) {
    // d = 16 has no chunk kernel: the single kernel runs its own token-level forward sweep
    vla::BackwardParams p;
    p.q = q; p.k = k; p.v = v; p.S0 = S0; p.A0 = A0; p.z0 = o.z0;
    p.d_out = d_out; p.dS_T = dS_T; p.dA_T = dA_T; p.dz_T = dz_T;
    p.dq = dq; p.dk = dk; p.dv = dv; p.dS0 = dS0; p.dA0 = dA0; p.dz0 = dz0;
    p.zst = zst; p.est = est; p.dst = dst; p.zkc = zkcw;
    p.status = o.status; p.lambda = lambda_; p.eps = o.eps; p.T = T; p.units = units; p.flags = o.flags;
    return vla::launch_backward(d_k, o.qkv_dtype, p, st);
  }
  // 1. the forward recurrence on the chunk kernel, leaving z_t, e_t, delta_t and the final states
  float* dalw = reinterpret_cast<float*>(w + 2 * vec + sca);
  float* dkSw = reinterpret_cast<float*>(w + 3 * vec + sca);
  float* gztw = reinterpret_cast<float*>(w + 4 * vec + sca);
  float* STw = reinterpret_cast<float*>(w + 5 * vec + sca);
  float* ATw = reinterpret_cast<float*>(w + 5 * vec + sca + mat);
  float* zTw = reinterpret_cast<float*>(w + 5 * vec + sca + 2 * mat);
  ScanParams f;
  f.q = q; f.k = k; f.v = v; f.u = o.u;
  f.S0 = S0; f.A0 = A0; f.z0 = o.z0;
  f.out = outw; f.S_T = STw; f.A_T = ATw; f.zT = zTw;
  f.status = o.status; f.lambda = lambda_; f.eps = o.eps;
  f.T = T; f.units = units; f.flags = o.flags;
  f.refresh_period = o.refresh_period; f.refresh_eta = o.refresh_eta; f.step_offset = o.step_offset;
  f.u_is_khat = 0;
  f.n_main = 0; f.out2 = nullptr;
  f.stash_z = zst; f.stash_e = est; f.stash_delta = dst; f.stash_zk = zkcw; f.stash_a = general ? astw : nullptr;
  f.heads = H;
  f.wait_limit = o.wait_probe_limit;
  // d = 128, u = k_hat, no refresh: the tensor-core form of the chunk kernel leaves the same stash
  if (chunk_tc_covers(f, d_k)) rc = vla::launch_chunk_tc_stash(d_k, o.qkv_dtype, f, st);
  else rc = vla::launch_chunk_stash(d_k, o.qkv_dtype, f, st);
  if (rc != VLA_OK) return rc;
  // 2. the S-side and A-side reverse scans
  vla::BackwardSplitParams p;
  p.q = q; p.k = k; p.u = o.u; p.ast = astw; p.du = o.du; p.z0 = o.z0; p.d_out = d_out; p.dS_T = dS_T; p.dA_T = dA_T; p.dz_T = dz_T;
  p.ST = STw; p.AT = ATw; p.zT = zTw; p.zst = zst; p.est = est; p.dst = dst; p.zkc = zkcw; p.ost = outw;
  p.dal = dalw; p.dkS = dkSw; p.gzt = gztw;
  p.dq = dq; p.dk = dk; p.dv = dv; p.dS0 = dS0; p.dA0 = dA0; p.dz0 = dz0;
  p.status = o.status; p.eps = o.eps; p.T = T; p.units = units; p.flags = o.flags;
  p.general = general ? 1 : 0;
  p.heads = H;
  p.progress = progw;
  p.refresh_period = o.refresh_period; p.refresh_eta = o.refresh_eta; p.step_offset = o.step_offset;
  return vla::launch_backward_split(d_k, o.qkv_dtype, p, st);
}

int vla_make_u(const void* k, const float* W_u, int B, int H, int T, int d_k, int k_dtype, int u_dtype,
               float scale, float eps, void* u, void* stream) {
  NvtxRange nvtx_range("vla_make_u");
  if (B < 0 || H < 0 || T < 0) return VLA_ERR_INVALID_ARG;
  if ((k_dtype != VLA_F32 && k_dtype != VLA_BF16) || (u_dtype != VLA_F32 && u_dtype != VLA_BF16))
    return VLA_ERR_INVALID_ARG;
  if (!(scale == scale)) return VLA_ERR_INVALID_ARG;
  if (d_k != 16 && d_k != 32 && d_k != 64 && d_k != 128) return VLA_ERR_UNSUPPORTED;
  const long long units = (long long)B * H;
  if (units > 0x7fffffffLL) return VLA_ERR_INVALID_ARG;
  if (units == 0 || T == 0) return VLA_OK;
  if (!k || !W_u || !u) return VLA_ERR_INVALID_ARG;
  if (!aligned16(k) || !aligned16(W_u) || !aligned16(u)) return VLA_ERR_ALIGNMENT;
  vla::MakeUParams p;
  p.k = k; p.W = W_u; p.u = u; p.scale = scale; p.eps = eps > 0.0f ? eps : 1e-4f;
  p.T = T; p.units = int(units); p.heads = H;
  return vla::launch_make_u(d_k, k_dtype, u_dtype, p, static_cast<cudaStream_t>(stream));
}

int vla_probe_fp32_fma(int iters, float* sink, double* flops, void* stream) {
  if (iters <= 0 || !sink) return VLA_ERR_INVALID_ARG;
  return vla::launch_fp32_probe(iters, sink, flops, static_cast<cudaStream_t>(stream));
}

int vla_query_support(int d_k, int d_v, int qkv_dtype, uint32_t flags) {
  if (qkv_dtype != VLA_F32 && qkv_dtype != VLA_BF16) return VLA_ERR_UNSUPPORTED;
  if (flags & ~uint32_t(VLA_FLAG_IDENTITY_MAP | VLA_FLAG_CHECK_FINITE | VLA_FLAG_TOKEN_MAJOR |
                        VLA_FLAG_LINEAR_ATTENTION))
    return VLA_ERR_UNSUPPORTED;
  return shape_supported(d_k, d_v) ? VLA_OK : VLA_ERR_UNSUPPORTED;
}

const char* vla_status_string(int status) {
  switch (status) {
    case VLA_OK: return "ok";
    case VLA_ERR_INVALID_ARG: return "invalid argument";
    case VLA_ERR_UNSUPPORTED: return "unsupported shape, dtype or flag (no kernel; there is no CPU fallback)";
    case VLA_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
    case VLA_ERR_CUDA: return "CUDA runtime or launch error";
    case VLA_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait ran out";
    case VLA_ERR_NONFINITE: return "non-finite delta or write-direction norm";
    case VLA_ERR_TOO_LARGE:
      return "problem needs more staging memory than the built-in buffer of "
             "vla_forward_host_static (VLA_STATIC_SCRATCH_BYTES); use vla_forward_host";
    default: return "unknown status";
  }
}

int vla_selftest_wait_timeout(uint32_t probe_limit, int32_t* status, void* stream) {
  if (!status || probe_limit == 0) return VLA_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(status) & 3u) return VLA_ERR_ALIGNMENT;
  return vla::launch_wait_selftest(probe_limit, status, static_cast<cudaStream_t>(stream));
}

int vla_last_launch(char* buf, size_t len) {
  if (!buf || len == 0) return VLA_ERR_INVALID_ARG;
  const LaunchNote& n = g_last_launch;
  if (!n.kernel[0]) {
    buf[0] = 0;
    return VLA_OK;
  }
  std::snprintf(buf, len, "%s<%d,%s> grid=%d%s", n.kernel, n.d, n.dtype == VLA_BF16 ? "bf16" : "f32", n.grid,
                n.balanced ? " balanced" : "");
  return VLA_OK;
}

int vla_version(void) { return 200; }

}  // extern "C"
