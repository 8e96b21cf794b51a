// tcgen05 / TMA (sm_100a) prefill path: interface towards the API layer.
#pragma once

#include "gta_common.cuh"

namespace gta {

// True when the tensor-core kernels cover this shape (bf16, d_h = 128, d_l % 256 == 0, ...).
bool sm100_prefill_supported(const Dims& d, int dtype);

// Enqueues the tensor-core prefill (attention kernel + decoder kernel) on `stream`.
gta_status_t launch_sm100_prefill(const Dims& d, const void* q, const void* k, const void* c, const void* x,
                                  const void* w_p, const void* w_g, void* out, void* workspace,
                                  int32_t* status_word, cudaStream_t stream, int stages, int* launches);

// Decoder + gate kernel alone: out = (L W_P) (.) sigmoid(X W_G) with L[B, n_q, N, d_l] in bf16.
gta_status_t launch_sm100_decoder(const Dims& d, const void* l_bf16, const void* x, const void* w_p, const void* w_g,
                                  void* out, int32_t* status_word, cudaStream_t stream);

}  // namespace gta
