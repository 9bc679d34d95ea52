// Host-side interface between the C ABI (vla_api.cu) and the translation units that hold the
// kernels.  The kernels are spread over several .cu files only so that they compile in
// parallel; none of this is visible outside the library.
#pragma once

#include <cuda_runtime.h>

#include "vla_common.cuh"
#include "vla_seqpar_params.h"

namespace vla {
struct BackwardParams;
struct BackwardSplitParams;
struct MakeUParams;
}

namespace vla {

// Token kernel, d in {16, 32, 64, 128}.  Returns a vla_status_t.
int launch_token(int d, int dtype, const ScanParams& p, cudaStream_t st);

// Single-step kernel (T = 1, carried states in and out, u = k_hat, no refresh), d in {32, 64, 128}.
int launch_decode(int d, int dtype, const ScanParams& p, cudaStream_t st);

// Chunk kernel, d in {32, 64, 128}: plain or balanced grid, chosen from the shape.
int launch_chunk(int d, int dtype, const ScanParams& p, cudaStream_t st);

// Tensor-core form of the chunk kernel: d = 128, u = k_hat, no refresh, [B,H,T,d] tensors.
int launch_chunk_tc(int d, int dtype, const ScanParams& p, cudaStream_t st);

// Chunk kernel as the forward of a backward pass: leaves z_t, e_t, delta_t per token (p.stash_*).
int launch_chunk_stash(int d, int dtype, const ScanParams& p, cudaStream_t st);
// The tensor-core form of the same (d = 128, u = k_hat, no refresh).
int launch_chunk_tc_stash(int d, int dtype, const ScanParams& p, cudaStream_t st);

// Chunk kernel with three warp groups per CTA (d in {32, 64}; sequence-parallel launches).
int launch_chunk_tri(int d, int dtype, const ScanParams& p, cudaStream_t st);

// CTAs of the chunk kernel (u = k_hat variant) that the current device holds at a time.
int chunk_resident_ctas(int d, int dtype, bool tri);

// Sequence-parallel helpers: Gram matrices + inversion before the scan, combination +
// correction + final-state copies after it.
int seqpar_before_scan(int d, int dtype, const SeqParParams& sp, cudaStream_t st);
int seqpar_after_scan(int d, const SeqParParams& sp, float* A_T, float* zT, const float* AT2,
                      const float* zT2, cudaStream_t st);

// Backward pass, token kernel, d in {16, 32, 64}, u = k_hat.
int launch_backward(int d, int dtype, const BackwardParams& p, cudaStream_t st);

// Backward pass as two reverse scans over the chunk kernel's stash, d in {32, 64, 128}, u = k_hat.
int launch_backward_split(int d, int dtype, const BackwardSplitParams& p, cudaStream_t st);
// u = scale * L2norm(W_u k): in_dtype of k, out_dtype of u
int launch_make_u(int d, int in_dtype, int out_dtype, const MakeUParams& p, cudaStream_t st);

// Register-only fp32 FMA loop over the whole device (measurement helper); *flops = work launched.
int launch_fp32_probe(int iters, float* sink, double* flops, cudaStream_t st);

// Launch ids for the balanced schedule's hand-off flags (never 0, never repeated within
// 2^32 launches).
unsigned int next_launch_epoch();

// The hand-off flags of a balanced launch live in one of kSchedSlots slots (launch id modulo the
// slot count).  A slot may be taken again only once the launch that used it last has finished:
// sched_slot_free() asks the event recorded behind that launch, sched_slot_mark() records it.
// A launch that finds its slot busy runs on the plain grid instead (no flags needed).
bool sched_slot_free(unsigned int epoch);
void sched_slot_mark(unsigned int epoch, cudaStream_t st);

// What the calling thread launched last (read back by vla_last_launch).
void note_launch(const char* kernel, int d, int dtype, int grid, int balanced);

// Test kernel of the bounded wait: a barrier that never completes.
int launch_wait_selftest(unsigned int probe_limit, int* status, cudaStream_t st);

}  // namespace vla
