// Chunk kernel, d = 64, fp32 inputs.
#include "vla_chunk_launch.cuh"

VLA_DEFINE_CHUNK_TU(64, float, d64_f32)
