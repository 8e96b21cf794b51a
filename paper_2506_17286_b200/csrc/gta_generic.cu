// Plain-ALU (fp32 FMA) prefill kernels: any supported shape, fp32 or bf16 storage.
// They carry the fp32 workload (tensor-core tf32 would not meet its 1e-4 bound) and every
// shape the tcgen05 kernels do not cover.  Two kernels:
//   generic_attention_kernel : shared attention map per query group, online softmax, latent
//                              P·C  ->  normalised L[B, n_q, N, d_l] (fp32, workspace)
//   generic_decoder_kernel   : out_i = (L_{q(i)} W_P,i) (.) sigmoid(X W_G,i)
// (Sec. 3.3 reformulated equation; causal sum of App. B.1.1.)
#include "gta_common.cuh"

namespace gta {

constexpr int kAttnWarps = 16;   // query rows per CTA, one warp each
constexpr int kMaxAccPerLane = 32;  // d_l <= 32 * 32

template <typename T, typename TO>
__global__ void __launch_bounds__(kAttnWarps * 32)
generic_attention_kernel(Dims d, const T* __restrict__ q, const T* __restrict__ k,
                         const T* __restrict__ c, TO* __restrict__ o_lat, const PageMap pm, int32_t* status_word) {
    extern __shared__ float q_smem[];  // [kAttnWarps][d_h]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int t = blockIdx.x * kAttnWarps + warp;
    const int g = blockIdx.y, b = blockIdx.z;
    if (t >= d.N) return;  // no block-wide barrier below
    const int kg = d.q_to_k(g), cg = d.q_to_c(g);
    const T* q_row = q + (((size_t)b * d.n_q + g) * d.N + t) * d.d_h;
    // rows of the attended keys and latents: planes of S rows, or (with a page map) pages of a pool; a key whose
    // block-table entry lies outside the pool takes no part (its score stays -inf)
    float* qs = q_smem + warp * d.d_h;
    for (int e = lane; e < d.d_h; e += 32) qs[e] = to_f32(q_row[e]);
    __syncwarp();

    const int n_keys = d.causal ? t + 1 + (d.Nk - d.N) : d.Nk;
    const int n_acc = (d.d_l + 31) / 32;
    float acc[kMaxAccPerLane];
#pragma unroll
    for (int a = 0; a < kMaxAccPerLane; ++a) acc[a] = 0.f;
    float m = -INFINITY, l = 0.f;

    for (int j0 = 0; j0 < n_keys; j0 += 32) {
        const int j = j0 + lane;
        float s = -INFINITY;
        long long c_idx = -1;
        if (j < n_keys) {
            const long long k_idx = cache_row(pm, b, d.n_k, kg, d.S, j, status_word);
            c_idx = cache_row(pm, b, d.n_c, cg, d.S, j, status_word);
            if (k_idx >= 0 && c_idx >= 0) {
                const T* k_row = k + (size_t)k_idx * d.d_h;
                float dot = 0.f;
                for (int e = 0; e < d.d_h; ++e) dot = fmaf(qs[e], to_f32(k_row[e]), dot);
                s = dot * d.scale;
            } else {
                c_idx = -1;
            }
        }
        const float m_new = fmaxf(m, warp_max(s));
        if (m_new == -INFINITY) continue;            // only keys on bad pages so far
        const float p = (c_idx >= 0) ? expf(s - m_new) : 0.f;
        const float corr = expf(m - m_new);          // exp(-inf) = 0 on the first tile
        l = l * corr + warp_sum(p);
        m = m_new;
#pragma unroll
        for (int a = 0; a < kMaxAccPerLane; ++a) acc[a] *= corr;
        const int live = min(32, n_keys - j0);
        for (int jj = 0; jj < live; ++jj) {
            const float pj = __shfl_sync(0xffffffffu, p, jj);
            const long long cj = __shfl_sync(0xffffffffu, c_idx, jj);
            if (cj < 0) continue;
            const T* c_row = c + (size_t)cj * d.d_l;
#pragma unroll
            for (int a = 0; a < kMaxAccPerLane; ++a) {
                const int col = lane + 32 * a;
                if (a < n_acc && col < d.d_l) acc[a] = fmaf(pj, to_f32(c_row[col]), acc[a]);
            }
        }
    }
    const float inv_l = l > 0.f ? 1.f / l : 0.f;
    TO* o_row = o_lat + (((size_t)b * d.n_q + g) * d.N + t) * d.d_l;
#pragma unroll
    for (int a = 0; a < kMaxAccPerLane; ++a) {
        const int col = lane + 32 * a;
        if (a < n_acc && col < d.d_l) o_row[col] = from_f32<TO>(acc[a] * inv_l);
    }
}

// ---- decoder + gate: 32 x 64 output tile per CTA, 256 threads, 2 x 4 outputs per thread ----
constexpr int kDecBM = 32, kDecBN = 64, kDecBK = 32;

template <typename TA, typename TW>
__device__ __forceinline__ void tile_gemm_accumulate(const TW* __restrict__ w, size_t ldw, int col0,
                                                     int n_cols_valid, int K, float (*As)[kDecBK + 1],
                                                     float (*Ws)[kDecBN], const TA* __restrict__ a_tile_base,
                                                     size_t a_row_stride, int rows_valid,
                                                     float acc[2][4]) {
    const int tid = threadIdx.x;
    const int ty = tid >> 4, tx = tid & 15;
    for (int k0 = 0; k0 < K; k0 += kDecBK) {
        // A tile: kDecBM x kDecBK
        for (int idx = tid; idx < kDecBM * kDecBK; idx += 256) {
            const int r = idx / kDecBK, kk = idx % kDecBK;
            float v = 0.f;
            if (r < rows_valid && k0 + kk < K) v = to_f32(a_tile_base[(size_t)r * a_row_stride + k0 + kk]);
            As[r][kk] = v;
        }
        // W tile: kDecBK x kDecBN
        for (int idx = tid; idx < kDecBK * kDecBN; idx += 256) {
            const int kk = idx / kDecBN, cc = idx % kDecBN;
            float v = 0.f;
            if (k0 + kk < K && cc < n_cols_valid) v = to_f32(w[(size_t)(k0 + kk) * ldw + col0 + cc]);
            Ws[kk][cc] = v;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < kDecBK; ++kk) {
            const float a0 = As[ty * 2][kk], a1 = As[ty * 2 + 1][kk];
#pragma unroll
            for (int cidx = 0; cidx < 4; ++cidx) {
                const float wv = Ws[kk][tx * 4 + cidx];
                acc[0][cidx] = fmaf(a0, wv, acc[0][cidx]);
                acc[1][cidx] = fmaf(a1, wv, acc[1][cidx]);
            }
        }
        __syncthreads();
    }
}

template <typename T>
__global__ void __launch_bounds__(256)
generic_decoder_kernel(Dims d, const float* __restrict__ o_lat, const T* __restrict__ x,
                       const T* __restrict__ w_p, const T* __restrict__ w_g, T* __restrict__ out) {
    __shared__ float As[kDecBM][kDecBK + 1];
    __shared__ float Ws[kDecBK][kDecBN];
    // rows of this tile all belong to one batch entry: grid.x = B * ceil(N / kDecBM)
    const int tiles_per_seq = (d.N + kDecBM - 1) / kDecBM;
    const int b = blockIdx.x / tiles_per_seq;
    const int t0 = (blockIdx.x % tiles_per_seq) * kDecBM;
    const int i = blockIdx.y;                 // head
    const int col0 = blockIdx.z * kDecBN;     // first column of this tile inside the head
    const int n_cols_valid = min(kDecBN, d.d_h - col0);
    const int rows_valid = min(kDecBM, d.N - t0);
    const int g = d.head_to_q(i);

    float acc_p[2][4] = {}, acc_g[2][4] = {};
    const float* l_base = o_lat + (((size_t)b * d.n_q + g) * d.N + t0) * d.d_l;
    tile_gemm_accumulate<float, T>(w_p + (size_t)i * d.d_l * d.d_h, (size_t)d.d_h, col0,
                                   n_cols_valid, d.d_l, As, Ws, l_base, (size_t)d.d_l, rows_valid, acc_p);
    const T* x_base = x + ((size_t)b * d.N + t0) * d.H;
    tile_gemm_accumulate<T, T>(w_g, (size_t)d.n_h * d.d_h, i * d.d_h + col0, n_cols_valid,
                               d.H, As, Ws, x_base, (size_t)d.H, rows_valid, acc_g);

    const int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
        const int r = ty * 2 + rr;
        if (r >= rows_valid) continue;
        T* o_row = out + (((size_t)b * d.N + t0 + r) * d.n_h + i) * d.d_h + col0;
#pragma unroll
        for (int cidx = 0; cidx < 4; ++cidx) {
            const int cc = tx * 4 + cidx;
            if (cc < n_cols_valid) {
                const float gate = 1.f / (1.f + expf(-acc_g[rr][cidx]));
                o_row[cc] = from_f32<T>(acc_p[rr][cidx] * gate);
            }
        }
    }
}

template <typename T>
static cudaError_t launch_typed(const Dims& d, const void* q, const void* k, const void* c, const void* x,
                                const void* w_p, const void* w_g, void* out, float* o_lat_ws,
                                cudaStream_t stream, int stages, int* launches, const PageMap& pm,
                                int32_t* status_word) {
    if (stages & 1) {
        dim3 grid_a((d.N + kAttnWarps - 1) / kAttnWarps, d.n_q, d.B);
        const size_t smem = (size_t)kAttnWarps * d.d_h * sizeof(float);
        generic_attention_kernel<T, float><<<grid_a, kAttnWarps * 32, smem, stream>>>(
            d, (const T*)q, (const T*)k, (const T*)c, o_lat_ws, pm, status_word);
        cudaError_t err = cudaGetLastError();
        if (err != cudaSuccess) return err;
        *launches += 1;
    }
    if (stages & 2) {
        const int tiles_per_seq = (d.N + kDecBM - 1) / kDecBM;
        dim3 grid_d(d.B * tiles_per_seq, d.n_h, (d.d_h + kDecBN - 1) / kDecBN);
        generic_decoder_kernel<T><<<grid_d, 256, 0, stream>>>(d, o_lat_ws, (const T*)x, (const T*)w_p,
                                                             (const T*)w_g, (T*)out);
        *launches += 1;
    }
    return cudaGetLastError();
}

cudaError_t launch_generic_prefill(const Dims& d, int dtype, const void* q, const void* k, const void* c,
                                   const void* x, const void* w_p, const void* w_g, void* out,
                                   float* o_lat_ws, cudaStream_t stream, int stages, int* launches,
                                   const PageMap& pm, int32_t* status_word) {
    if (dtype == GTA_F32)
        return launch_typed<float>(d, q, k, c, x, w_p, w_g, out, o_lat_ws, stream, stages, launches, pm, status_word);
    return launch_typed<__nv_bfloat16>(d, q, k, c, x, w_p, w_g, out, o_lat_ws, stream, stages, launches, pm,
                                       status_word);
}

// Attention stage only, bf16 storage in and out (L written as bf16): feeds the tensor-core
// decoder when the tensor-core attention kernel does not cover a shape.
cudaError_t launch_generic_attention_bf16(const Dims& d, const void* q, const void* k, const void* c,
                                          void* o_lat_bf16, cudaStream_t stream, int* launches) {
    dim3 grid_a((d.N + kAttnWarps - 1) / kAttnWarps, d.n_q, d.B);
    const size_t smem = (size_t)kAttnWarps * d.d_h * sizeof(float);
    generic_attention_kernel<__nv_bfloat16, __nv_bfloat16><<<grid_a, kAttnWarps * 32, smem, stream>>>(
        d, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)c, (__nv_bfloat16*)o_lat_bf16,
        PageMap(), nullptr);
    *launches += 1;
    return cudaGetLastError();
}

}  // namespace gta
