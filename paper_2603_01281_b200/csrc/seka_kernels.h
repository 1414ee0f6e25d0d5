// Internal host-side launchers shared by the translation units of the library.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "seka_common.cuh"

namespace seka {

void launch_prep_fragments(const float* U, uint4* frags, int Hkv, int D, int r, int M, int r_pad, cudaStream_t st);
void launch_compact_mask(const uint8_t* mask, int T, int* list, int* count, cudaStream_t st);
void launch_convert_bf16(const float* in, void* out, size_t n, cudaStream_t st);

seka_status validate_shape(const seka_shape* s);

}  // namespace seka
