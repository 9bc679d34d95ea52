// Chunk kernel with the backward pass's stash, d = 32, bf16 inputs.
#include "vla_chunk_launch.cuh"

VLA_DEFINE_CHUNK_STASH_TU(32, uint16_t, d32_bf16)
