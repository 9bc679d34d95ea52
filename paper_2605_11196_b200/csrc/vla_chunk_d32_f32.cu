// Chunk kernel, d = 32, fp32 inputs.
#include "vla_chunk_launch.cuh"

VLA_DEFINE_CHUNK_TU(32, float, d32_f32)
