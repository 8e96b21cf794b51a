// tcgen05 / TMA (sm_100a) prefill path: interface towards the API layer.
#pragma once

#include "gta_common.cuh"

namespace gta {

// True when the tensor-core kernels cover this shape (bf16, d_h = 128, d_l % 256 == 0, ...).
bool sm100_prefill_supported(const Dims& d, int dtype);

// Enqueues the tensor-core prefill (attention kernel + decoder kernel) on `stream`.
gta_status_t launch_sm100_prefill(const Dims& d, const void* q, const void* k, const void* c, const void* x,
                                  const void* w_p, const void* w_g, void* out, void* workspace,
                                  int32_t* status_word, cudaStream_t stream, int stages, int* launches,
                                  const PageMap& pm = PageMap());

// Attention kernel alone: L[B, n_q, N, d_l] (bf16) = Softmax(scale Q K^T) C per attention map; bf16, d_h = 64 or
// 128, d_l a multiple of 128 or exactly 64.  With a page map, k and c are paged pools (page_size a multiple of 64)
// and token t of sequence b is looked up through the block table.
gta_status_t launch_sm100_attention(const Dims& d, const void* q, const void* k, const void* c, void* l_out,
                                    int32_t* status_word, cudaStream_t stream, const PageMap& pm = PageMap());

// Test hooks of the attention kernel's bounded waits (see gta_debug_attention_wait in gta.h).
gta_status_t sm100_attention_debug_wait(unsigned long long limit_ns, int withhold_first_arrive);

// Decoder + gate kernel alone: out = (L W_P) (.) sigmoid(X W_G) with L[B, n_q, N, d_l] in bf16.
// step_lens (optional; the fused append + decode step): lengths that the kernel advances by one, where there is room
// below step_cap, once the kernel before it in the stream is complete.
gta_status_t launch_sm100_decoder(const Dims& d, const void* l_bf16, const void* x, const void* w_p, const void* w_g,
                                  void* out, int32_t* status_word, cudaStream_t stream, int32_t* step_lens = nullptr,
                                  int step_batch = 0, int step_cap = 0);

// Linear maps of the attention layer around the operator (App. B.1.1), bf16 with fp32 accumulation.
// True when the tcgen05 kernel covers the layer's projections for this shape.
bool sm100_linear_supported(const Dims& d, int dtype);

// [Q | K | C] = X W_qkc for the B x N tokens of a chunk that starts at position pos0: RoPE on q and k,
// q to q_out [B, n_q, N, d_h], k and c to rows pos0 + t of the caches [B, groups, S_cap, width] (with a page map:
// of the paged pools, S_cap then being page_size * max_pages).
// rope_table: sm100_rope_table_bytes(d) bytes of scratch (cos / sin of the chunk's positions).
size_t sm100_rope_table_bytes(const Dims& d);
gta_status_t launch_sm100_project(const Dims& d, int pos0, int S_cap, double rope_base, const void* x,
                                  const void* w_qkc, void* q_out, void* k_cache, void* c_cache, void* rope_table,
                                  int32_t* status_word, cudaStream_t stream, const PageMap& pm = PageMap());

// One decode step of the same projection: one new token per sequence at position seq_lens[b] (RoPE there,
// k and c to that cache row, q to q_out [B, n_q, d_h]), then seq_lens[b] += 1; a sequence whose cache is full
// is skipped and raises GTA_ERR_CACHE_FULL.  With a page map, k_cache / c_cache are the paged pools.  prep: sm100_decode_prep_bytes(d) bytes of scratch.
size_t sm100_decode_prep_bytes(const Dims& d);
gta_status_t launch_sm100_project_step(const Dims& d, int S_cap, double rope_base, const void* x_t, const void* w_qkc,
                                       void* q_out, void* k_cache, void* c_cache, int32_t* seq_lens, void* prep,
                                       int32_t* status_word, cudaStream_t stream, const PageMap& pm = PageMap());

// C[M, n_cols] = A[M, K] W[K, n_cols], row-major.
gta_status_t launch_sm100_matmul(long long M, int K, int n_cols, const void* a, const void* w, void* c_out,
                                 int32_t* status_word, cudaStream_t stream);

// The stream kernel of a decode step over 8-bit caches on the tcgen05 tensor pipe (gta_decode_fp8_tc.cu): same
// schedule (G CTAs, sub-tiles of T tokens) and partial results as decode_stream_fp8_kernel.
bool decode_fp8_tc_supported(const Dims& d, int T);
cudaError_t launch_decode_fp8_tc_stream(const Dims& d, int G, int T, int S_cap, const void* q, const void* k_codes,
                                        const void* c_codes, const float* k_scale, const float* c_scale,
                                        const int32_t* seq_lens, float* part_o, float* part_ml, int32_t* status_word,
                                        cudaStream_t stream);

// The stream kernel of a decode step over bf16 caches on the tcgen05 tensor pipe (gta_decode_tc.cu): same schedule
// (G CTAs, sub-tiles of T tokens), step lengths and partial results as decode_stream_kernel; k_new / c_new != nullptr:
// the fused append + decode step.
bool decode_tc_supported(const Dims& d, int T, int occ, int page_size);
cudaError_t launch_decode_tc_stream(const Dims& d, int G, int T, int S_cap, const void* q, const void* k_cache,
                                    const void* c_cache, const int32_t* seq_lens, float* part_o, float* part_ml,
                                    int32_t* status_word, cudaStream_t stream, const void* k_new, const void* c_new,
                                    const PageMap& pm);

// Test hooks of the bounded waits of the two tensor-memory decode stream kernels (see gta_debug_decode_wait in gta.h).
gta_status_t decode_tc_debug_wait(unsigned long long limit_ns, int withhold_first_arrive);
gta_status_t decode_fp8_tc_debug_wait(unsigned long long limit_ns, int withhold_first_arrive);

}  // namespace gta
