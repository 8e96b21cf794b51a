// Cache append: bit-exact 16-byte copies of the new key / latent rows behind the live part of
// each sequence's caches, then the length update (Sec. 3.3 last paragraph; App. B.1.3).
#include "gta_common.cuh"
#include "sm100_ptx.cuh"

namespace gta {

constexpr int kAppendThreads = 256;

struct AppendArgs {
    uint4* k_cache; uint4* c_cache;
    const uint4* k_new; const uint4* c_new;
    int B, n_k, n_c, S_cap, n_new;
    int k_row_vecs, c_row_vecs;   // 16-byte vectors per row
    PageMap pm;                   // table == nullptr: contiguous caches
    int32_t* status_word;
};

// Copies slice `part` of `n_parts` of sequence b's new rows.  Does not touch seq_lens.
__device__ __forceinline__ void append_copy(const AppendArgs& a, int b, int len, int part, int n_parts) {
    const long long k_vecs = (long long)a.n_k * a.n_new * a.k_row_vecs;
    const long long c_vecs = (long long)a.n_c * a.n_new * a.c_row_vecs;
    const long long total = k_vecs + c_vecs;
    for (long long idx = (long long)part * kAppendThreads + threadIdx.x; idx < total;
         idx += (long long)n_parts * kAppendThreads) {
        if (idx < k_vecs) {
            const int v = (int)(idx % a.k_row_vecs);
            const long long row = idx / a.k_row_vecs;          // g * n_new + n
            const int n = (int)(row % a.n_new), g = (int)(row / a.n_new);
            const long long dst = cache_row(a.pm, b, a.n_k, g, a.S_cap, len + n, a.status_word);
            if (dst >= 0)
                a.k_cache[(size_t)dst * a.k_row_vecs + v] =
                    a.k_new[(((size_t)b * a.n_k + g) * a.n_new + n) * a.k_row_vecs + v];
        } else {
            const long long cidx = idx - k_vecs;
            const int v = (int)(cidx % a.c_row_vecs);
            const long long row = cidx / a.c_row_vecs;
            const int n = (int)(row % a.n_new), g = (int)(row / a.n_new);
            const long long dst = cache_row(a.pm, b, a.n_c, g, a.S_cap, len + n, a.status_word);
            if (dst >= 0)
                a.c_cache[(size_t)dst * a.c_row_vecs + v] =
                    a.c_new[(((size_t)b * a.n_c + g) * a.n_new + n) * a.c_row_vecs + v];
        }
    }
}

// One CTA per sequence: copy, then advance the length (few new rows, e.g. one decode step).
__global__ void __launch_bounds__(kAppendThreads)
append_small_kernel(AppendArgs a, int32_t* __restrict__ seq_lens, int32_t* status_word) {
    // Launched with programmatic stream serialisation (the launch latency of a decode step's first
    // kernel hides behind the step before): nothing is read or written before the kernel ahead in
    // the stream is complete, and only then may the kernel behind this one be scheduled.
    ptx::grid_dependency_wait();
    ptx::grid_launch_dependents();
    const int b = blockIdx.x;
    const int len = seq_lens[b];
    __syncthreads();   // every thread has read the old length before thread 0 rewrites it
    if (len < 0 || (long long)len + a.n_new > a.S_cap) {
        if (threadIdx.x == 0) raise_status(status_word, GTA_ERR_CACHE_FULL);
        return;
    }
    append_copy(a, b, len, 0, 1);
    if (threadIdx.x == 0) seq_lens[b] = len + a.n_new;
}

// Bulk load (many new rows): grid (parts, B) copies; lengths advance in a second launch.
__global__ void __launch_bounds__(kAppendThreads)
append_bulk_copy_kernel(AppendArgs a, const int32_t* __restrict__ seq_lens) {
    const int b = blockIdx.y;
    const int len = seq_lens[b];
    if (len < 0 || (long long)len + a.n_new > a.S_cap) return;
    append_copy(a, b, len, blockIdx.x, gridDim.x);
}

__global__ void append_advance_kernel(int B, int S_cap, int n_new, int32_t* __restrict__ seq_lens,
                                      int32_t* status_word) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const int len = seq_lens[b];
    if (len < 0 || (long long)len + n_new > S_cap) raise_status(status_word, GTA_ERR_CACHE_FULL);
    else seq_lens[b] = len + n_new;
}

cudaError_t launch_cache_append(const Dims& d, int elem_size, void* k_cache, void* c_cache, int S_cap,
                                const void* k_new, const void* c_new, int n_new, int32_t* seq_lens,
                                int32_t* status_word, cudaStream_t stream, int* launches, const PageMap& pm) {
    AppendArgs a;
    a.pm = pm;
    a.status_word = status_word;
    a.k_cache = (uint4*)k_cache; a.c_cache = (uint4*)c_cache;
    a.k_new = (const uint4*)k_new; a.c_new = (const uint4*)c_new;
    a.B = d.B; a.n_k = d.n_k; a.n_c = d.n_c; a.S_cap = S_cap; a.n_new = n_new;
    a.k_row_vecs = d.d_h * elem_size / 16;
    a.c_row_vecs = d.d_l * elem_size / 16;
    const long long vecs_per_seq = (long long)n_new * ((long long)d.n_k * a.k_row_vecs + (long long)d.n_c * a.c_row_vecs);
    if (vecs_per_seq <= 8 * kAppendThreads) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(d.B);
        cfg.blockDim = dim3(kAppendThreads);
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cudaError_t e = cudaLaunchKernelEx(&cfg, append_small_kernel, a, seq_lens, status_word);
        if (e != cudaSuccess) return e;
        *launches += 1;
        return cudaGetLastError();
    }
    long long parts = (vecs_per_seq + 8 * kAppendThreads - 1) / (8 * kAppendThreads);
    if (parts > 1024) parts = 1024;
    append_bulk_copy_kernel<<<dim3((unsigned)parts, d.B), kAppendThreads, 0, stream>>>(a, seq_lens);
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return err;
    append_advance_kernel<<<(d.B + 127) / 128, 128, 0, stream>>>(d.B, S_cap, n_new, seq_lens, status_word);
    *launches += 2;
    return cudaGetLastError();
}

}  // namespace gta
