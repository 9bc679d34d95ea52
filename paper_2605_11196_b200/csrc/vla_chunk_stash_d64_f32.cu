// Chunk kernel with the backward pass's stash, d = 64, fp32 inputs.
#include "vla_chunk_launch.cuh"

VLA_DEFINE_CHUNK_STASH_TU(64, float, d64_f32)
