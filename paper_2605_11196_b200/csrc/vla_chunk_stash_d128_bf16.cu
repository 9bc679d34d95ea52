// Chunk kernel with the backward pass's stash, d = 128, bf16 inputs.
#include "vla_chunk_launch.cuh"

VLA_DEFINE_CHUNK_STASH_TU(128, uint16_t, d128_bf16)
