// Internal helpers shared by the kernels of the GTA library (not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gta.h"

namespace gta {

// Head -> group maps (contiguous blocks), Sec. 3.2 "Input projections and grouping".
struct Dims {
    int B, N, H, n_h, n_q, n_k, n_c, d_h, d_l, causal;
    float scale;  // softmax scale, already resolved (1/sqrt(d_h) when the caller passed 0)
    // Prefill of a chunk against longer K / C (a cache): the N queries are the LAST N of Nk attended
    // positions (query t sees keys 0 .. t + Nk - N), and K / C rows are S apart per group.  A plain
    // prefill has Nk = S = N.
    int Nk, S;
    __host__ __device__ int head_to_q(int i) const { return (int)(((long long)i * n_q) / n_h); }
    __host__ __device__ int q_to_k(int g) const { return (int)(((long long)g * n_k) / n_q); }
    __host__ __device__ int q_to_c(int g) const { return (int)(((long long)g * n_c) / n_q); }
};

// Element access that widens the storage type to fp32 / narrows with round-to-nearest-even.
template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ void raise_status(int32_t* status_word, int code) {
    if (status_word) atomicMax(status_word, code);
}

// Where the cached rows of a sequence live (decode and append).  table == nullptr: caches
// [B][groups][S_cap][width], the rows of one (sequence, group) contiguous.  Otherwise a paged pool
// [n_pages][groups][page_size][width]: token t of sequence b is row t % page_size of page
// table[b * max_pages + t / page_size], and S_cap = max_pages * page_size.
struct PageMap {
    const int32_t* table = nullptr;
    int page_size = 0, max_pages = 0, n_pages = 0;
};

// Page that holds token t of sequence b; an entry outside the pool raises GTA_ERR_BAD_PAGE and
// yields -1 (the caller skips the access).
__device__ __forceinline__ int page_of(const PageMap& pm, int b, int t, int32_t* status_word) {
    const int page = pm.table[(size_t)b * pm.max_pages + t / pm.page_size];
    if (page < 0 || page >= pm.n_pages) {
        raise_status(status_word, GTA_ERR_BAD_PAGE);
        return -1;
    }
    return page;
}

// Row index (in rows of the cache tensor) of token t of group g of sequence b, or -1 (bad page).
__device__ __forceinline__ long long cache_row(const PageMap& pm, int b, int groups, int g, int S_cap, int t,
                                               int32_t* status_word) {
    if (pm.table == nullptr) return ((long long)b * groups + g) * S_cap + t;
    const int page = page_of(pm, b, t, status_word);
    if (page < 0) return -1;
    return ((long long)page * groups + g) * pm.page_size + t % pm.page_size;
}

// Launchers implemented in the .cu files; each returns cudaGetLastError() of its launches and
// adds the number of launches it made to *launches.
cudaError_t launch_generic_prefill(const Dims& d, int dtype, const void* q, const void* k, const void* c,
                                   const void* x, const void* w_p, const void* w_g, void* out,
                                   float* o_lat_ws, cudaStream_t stream, int stages, int* launches,
                                   const PageMap& pm = PageMap(), int32_t* status_word = nullptr);

cudaError_t launch_generic_attention_bf16(const Dims& d, const void* q, const void* k, const void* c,
                                          void* o_lat_bf16, cudaStream_t stream, int* launches);

cudaError_t launch_decode(const Dims& d, int dtype, const void* q, const void* k_cache, const void* c_cache,
                          const int32_t* seq_lens, int S_cap, const void* x_t, const void* w_p,
                          const void* w_g, void* out, void* workspace, int32_t* status_word,
                          cudaStream_t stream, int stages, int* launches, const PageMap& pm = PageMap());
size_t decode_workspace_bytes(const Dims& d, int dtype, int S_cap, int page_size = 0);
// The plain-ALU decode kernels regardless of shape (caches reachable by ordinary loads: device memory or mapped,
// page-locked host memory).
size_t decode_plain_workspace_bytes(const Dims& d, int S_cap);
cudaError_t launch_decode_plain(const Dims& d, int dtype, const void* q, const void* k_cache, const void* c_cache,
                                const int32_t* seq_lens, int S_cap, const void* x_t, const void* w_p,
                                const void* w_g, void* out, void* workspace, int32_t* status_word,
                                cudaStream_t stream, int* launches);

// bf16 bandwidth-oriented decode (persistent streaming kernel + cluster finish kernel).
bool decode_fast_supported(const Dims& d, int dtype, int page_size = 0);
size_t decode_fast_workspace_bytes(const Dims& d);
cudaError_t launch_decode_fast(const Dims& d, const void* q, const void* k_cache, const void* c_cache,
                               const int32_t* seq_lens, int S_cap, const void* x_t, const void* w_p,
                               const void* w_g, void* out, void* workspace, int32_t* status_word,
                               cudaStream_t stream, int stages, int* launches, const PageMap& pm = PageMap(),
                               const void* k_new = nullptr, const void* c_new = nullptr);

// Host-side argument checks of a decode call (everything but the workspace and the device), shared by
// gta_decode and gta_decode_static so that both report the same errors; *empty: the batch is empty.
gta_status_t decode_check_args(const gta_shape_t* shape, const void* q, const void* k_cache, const void* c_cache,
                               const int32_t* seq_lens, int32_t S_cap, const void* x_t, const void* w_p,
                               const void* w_g, const void* out, const int32_t* status_word, Dims* d, bool* empty);
// GTA_OK when the current device is one the kernels are built for, GTA_ERR_UNSUPPORTED otherwise.
gta_status_t check_current_device();

// Decode and append over 8-bit caches (e4m3 codes [B, groups, S_cap, width] + one fp32 scale per row
// [B, groups, S_cap]); plain-ALU kernels.
size_t decode_fp8_workspace_bytes(const Dims& d, int S_cap);
// 8-bit caches on the bandwidth-oriented kernels (bf16 operator tensors, d_h = 128, one latent group, ...)
bool decode_fp8_fast_supported(const Dims& d, int dtype, int S_cap);
size_t decode_fp8_fast_workspace_bytes(const Dims& d);
cudaError_t launch_decode_fp8_fast(const Dims& d, const void* q, const void* k_codes, const void* c_codes,
                                   const float* k_scale, const float* c_scale, const int32_t* seq_lens, int S_cap,
                                   const void* x_t, const void* w_p, const void* w_g, void* out, void* workspace,
                                   int32_t* status_word, cudaStream_t stream, int* launches);
cudaError_t launch_decode_fp8(const Dims& d, int dtype, const void* q, const void* k_codes, const void* c_codes,
                              const float* k_scale, const float* c_scale, const int32_t* seq_lens, int S_cap,
                              const void* x_t, const void* w_p, const void* w_g, void* out, void* workspace,
                              int32_t* status_word, cudaStream_t stream, int* launches);
cudaError_t launch_cache_append_fp8(const Dims& d, int dtype, void* k_codes, void* c_codes, float* k_scale,
                                    float* c_scale, int S_cap, const void* k_new, const void* c_new, int n_new,
                                    int32_t* seq_lens, int32_t* status_word, cudaStream_t stream, int* launches);

// Comparison operator (App. B.3, GQA / Sec. 3.1, MHA): one decode step on the stream and merge kernels.
bool gqa_decode_supported(int B, int n_h, int n_kv, int d_h, int dtype);
size_t gqa_decode_workspace_bytes(int B, int n_h, int n_kv, int d_h);
cudaError_t launch_gqa_decode(int B, int n_h, int n_kv, int d_h, float scale, const void* q, const void* k_cache,
                              const void* v_cache, const int32_t* seq_lens, int S_cap, void* out, void* workspace,
                              int32_t* status_word, cudaStream_t stream, int* launches);

cudaError_t launch_cache_append(const Dims& d, int elem_size, void* k_cache, void* c_cache, int S_cap,
                                const void* k_new, const void* c_new, int n_new, int32_t* seq_lens,
                                int32_t* status_word, cudaStream_t stream, int* launches,
                                const PageMap& pm = PageMap());

}  // namespace gta
