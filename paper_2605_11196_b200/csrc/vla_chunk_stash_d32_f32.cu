// Chunk kernel with the backward pass's stash, d = 32, fp32 inputs.
#include "vla_chunk_launch.cuh"

VLA_DEFINE_CHUNK_STASH_TU(32, float, d32_f32)
