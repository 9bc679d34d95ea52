// Chunk kernel with the backward pass's stash, d = 128, fp32 inputs.
#include "vla_chunk_launch.cuh"

VLA_DEFINE_CHUNK_STASH_TU(128, float, d128_f32)
