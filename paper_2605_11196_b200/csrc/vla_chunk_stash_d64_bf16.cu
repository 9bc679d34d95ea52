// Chunk kernel with the backward pass's stash, d = 64, bf16 inputs.
#include "vla_chunk_launch.cuh"

VLA_DEFINE_CHUNK_STASH_TU(64, uint16_t, d64_bf16)
