// Chunk kernel, d = 32, bf16 inputs.
#include "vla_chunk_launch.cuh"

VLA_DEFINE_CHUNK_TU(32, uint16_t, d32_bf16)
