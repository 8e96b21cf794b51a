// Single-token decode over the grouped key cache and the latent value cache (App. B.1.3).
// HBM-bound: every live cache byte is read exactly once with 16-byte vector loads.
//
//   decode_partial_kernel : grid (chunk, sequence).  One CTA streams one chunk of one
//       sequence: the K rows of every key group (scores of all n_q maps), a local softmax,
//       then the latent rows C, read ONCE and applied to all the maps that share them.
//       Writes per-(chunk, map) partials (max, sum, unnormalised latent sum) to workspace.
//   decode_gate_kernel    : Z = x_t W_G for all sequences at once (weights read once),
//       split over H; partial sums to workspace.
//   decode_finish_kernel  : log-sum-exp merge of the chunk partials, decoder GEMV with
//       W_P,i for 8 sequences per CTA (weights reused), gate sigmoid, store.
#include <type_traits>

#include "gta_common.cuh"

namespace gta {

constexpr int kDecodeThreads = 256;
constexpr int kFinishSeqs = 8;      // sequences per finish CTA
constexpr int kGateBatch = 32;      // sequences per accumulator block in the gate kernel
constexpr int kGateMaxSlice = 256;  // rows of W_G per gate CTA (upper bound)

struct DecodePlan {
    int chunk;       // tokens per partial CTA
    int n_chunks;    // ceil(S_cap / chunk)
    int gate_slice;  // rows of W_G per gate CTA
    int gate_splits; // ceil(H / gate_slice)
    size_t off_ml, off_z, total;  // byte offsets inside the workspace (part_o at 0)
};

static size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

static DecodePlan make_plan(const Dims& d, int S_cap) {
    DecodePlan p;
    // Aim at >= 8 chunk CTAs per SM over the whole batch, chunks of 64..256 tokens.
    long long want = ((long long)d.B * (S_cap > 0 ? S_cap : 1)) / (148 * 8);
    int chunk = (int)((want + 63) / 64) * 64;
    if (chunk < 64) chunk = 64;
    if (chunk > 256) chunk = 256;
    p.chunk = chunk;
    p.n_chunks = S_cap > 0 ? (S_cap + chunk - 1) / chunk : 1;
    p.gate_slice = d.H <= 2048 ? 128 : kGateMaxSlice;
    p.gate_splits = (d.H + p.gate_slice - 1) / p.gate_slice;
    const size_t part_o = (size_t)d.B * p.n_chunks * d.n_q * d.d_l * sizeof(float);
    const size_t part_ml = (size_t)d.B * p.n_chunks * d.n_q * 2 * sizeof(float);
    const size_t z = (size_t)p.gate_splits * d.B * d.n_h * d.d_h * sizeof(float);
    p.off_ml = align256(part_o);
    p.off_z = p.off_ml + align256(part_ml);
    p.total = p.off_z + align256(z);
    return p;
}

size_t decode_workspace_bytes(const Dims& d, int dtype, int S_cap, int page_size) {
    // the kernel family is a function of shape, dtype and page size only, so the size is that family's
    if (decode_fast_supported(d, dtype, page_size) && S_cap > 0) return decode_fast_workspace_bytes(d);
    return make_plan(d, S_cap).total;
}

// ---- 16-byte vector of storage elements, widened to fp32 ----
template <typename T> struct Vec16;
template <> struct Vec16<float> {
    static constexpr int N = 4;
    static __device__ __forceinline__ void widen(const uint4& r, float (&v)[4]) {
        v[0] = __uint_as_float(r.x); v[1] = __uint_as_float(r.y); v[2] = __uint_as_float(r.z); v[3] = __uint_as_float(r.w);
    }
    static __device__ __forceinline__ void load(const float* p, float (&v)[4]) {
        widen(__ldg(reinterpret_cast<const uint4*>(p)), v);
    }
};
template <> struct Vec16<__nv_bfloat16> {
    static constexpr int N = 8;
    static __device__ __forceinline__ void widen(const uint4& r, float (&v)[8]) {
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {  // bf16 is the upper half of an fp32
            v[2 * i] = __uint_as_float(w[i] << 16);
            v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    static __device__ __forceinline__ void load(const __nv_bfloat16* p, float (&v)[8]) {
        widen(__ldg(reinterpret_cast<const uint4*>(p)), v);
    }
};

// e4m3 codes (1 sign, 4 exponent, 3 mantissa bits, bias 7): the seven low bits, put where fp32 keeps the low four
// exponent bits and the top three mantissa bits, are the value times 2^-120 -- for the subnormal codes too --,
// so one exact multiplication by 2^120 finishes the conversion.
struct Fp8 { uint8_t bits; };
__device__ __forceinline__ float e4m3_to_f32(uint32_t b) {
    return __uint_as_float(((b & 0x80u) << 24) | ((b & 0x7fu) << 20)) * 1.329227995784916e36f;   // 2^120
}
template <> struct Vec16<Fp8> {
    static constexpr int N = 16;
    static __device__ __forceinline__ void widen(const uint4& r, float (&v)[16]) {
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) v[4 * i + j] = e4m3_to_f32(w[i] >> (8 * j));
    }
    static __device__ __forceinline__ void load(const Fp8* p, float (&v)[16]) {
        widen(__ldg(reinterpret_cast<const uint4*>(p)), v);
    }
};

template <typename T> __device__ __forceinline__ float exp_fn(float x);
template <> __device__ __forceinline__ float exp_fn<float>(float x) { return expf(x); }
template <> __device__ __forceinline__ float exp_fn<__nv_bfloat16>(float x) { return __expf(x); }

// Dynamic shared memory of decode_partial_kernel (floats):
//   q_s [n_q][d_h] | p_s [chunk][n_q] | ml_s [n_q][2] | red [R][d_l]
// CT: storage type of the caches (T, or Fp8 with one fp32 scale per cached row in k_scale / c_scale).
// kReadOnce: every cached row is loaded exactly once, for caches that sit behind the host link, where a row
// that is loaded again crosses the link again: a key row's vector is kept in registers for all the maps of its
// key group, and the maps of a latent group need not be a multiple of NGB (the last accumulators of the last
// pass idle).  On device memory the repeated loads hit L1 / L2 and the leaner loops are faster.
template <typename T, int NGB, typename CT = T, bool kReadOnce = false>
__global__ void __launch_bounds__(kDecodeThreads)
decode_partial_kernel(Dims d, int chunk, int n_chunks, int S_cap, const T* __restrict__ q,
                      const CT* __restrict__ k_cache, const CT* __restrict__ c_cache,
                      const int32_t* __restrict__ seq_lens, float* __restrict__ part_o,
                      float* __restrict__ part_ml, PageMap pm, int32_t* status_word,
                      const float* __restrict__ k_scale, const float* __restrict__ c_scale) {
    constexpr int VEC = Vec16<CT>::N;
    constexpr bool kScaled = !std::is_same<CT, T>::value;
    const int b = blockIdx.y, ck = blockIdx.x;
    int len = seq_lens[b];
    len = len < 0 ? 0 : (len > S_cap ? S_cap : len);
    const int j_begin = ck * chunk;
    if (j_begin >= len) return;
    const int n_tok = min(chunk, len - j_begin);

    extern __shared__ __align__(16) float smem[];
    float* q_s = smem;
    float* p_s = q_s + d.n_q * d.d_h;
    float* ml_s = p_s + chunk * d.n_q;
    float* red = ml_s + 2 * d.n_q;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    for (int e = tid; e < d.n_q * d.d_h; e += kDecodeThreads)
        q_s[e] = to_f32(q[(size_t)b * d.n_q * d.d_h + e]);
    __syncthreads();

    // ---- scores: LPR lanes share one K row, one 16-byte vector per lane and step ----
    if constexpr (kReadOnce) {
        constexpr int kScoreRows = 4;                       // rows per lane group whose loads are issued together
        constexpr int kMapsAtOnce = 8;                      // maps of a key group per pass over a row's registers
        constexpr int kSlots = (256 / VEC + 31) / 32;       // vectors per lane and row (d_h <= 256): 2 for fp32, else 1
        const int vecs_per_row = d.d_h / VEC;
        int lpr = 1;
        while (lpr < vecs_per_row && lpr < 32) lpr <<= 1;
        const int rows_per_warp = 32 / lpr;
        const int sub = lane / lpr, sl = lane % lpr;
        const int q_per_k = d.n_q / d.n_k;
        const int n_row_iters = (n_tok + rows_per_warp - 1) / rows_per_warp;
        const int total_iters = d.n_k * n_row_iters;
        constexpr int kWarps = kDecodeThreads / 32;
        for (int it0 = warp; it0 < total_iters; it0 += kWarps * kScoreRows) {
            uint4 raw[kScoreRows][kSlots];
            float row_scale[kScoreRows];
#pragma unroll
            for (int u = 0; u < kScoreRows; ++u) {
                const int it = it0 + u * kWarps;
                const bool in = it < total_iters;
                const int kg = in ? it / n_row_iters : 0;
                const int j = in ? (it % n_row_iters) * rows_per_warp + sub : 0;
                const long long k_idx = cache_row(pm, b, d.n_k, kg, S_cap, j_begin + (j < n_tok ? j : 0), status_word);
                const CT* k_row = k_cache + (size_t)(k_idx < 0 ? 0 : k_idx) * d.d_h;
                row_scale[u] = kScaled ? d.scale * k_scale[k_idx < 0 ? 0 : k_idx] : d.scale;
#pragma unroll
                for (int s = 0; s < kSlots; ++s) {
                    raw[u][s] = make_uint4(0u, 0u, 0u, 0u);
                    if (in && j < n_tok && sl + s * lpr < vecs_per_row)
                        raw[u][s] = __ldg(reinterpret_cast<const uint4*>(k_row + (sl + s * lpr) * VEC));
                }
            }
#pragma unroll
            for (int u = 0; u < kScoreRows; ++u) {
                const int it = it0 + u * kWarps;
                if (it >= total_iters) break;       // uniform over the warp
                const int kg = it / n_row_iters;
                const int j = (it % n_row_iters) * rows_per_warp + sub;
                float kv[kSlots][VEC];
#pragma unroll
                for (int s = 0; s < kSlots; ++s) Vec16<CT>::widen(raw[u][s], kv[s]);
                for (int g0 = 0; g0 < q_per_k; g0 += kMapsAtOnce) {
                    float dot[kMapsAtOnce];
#pragma unroll
                    for (int gi = 0; gi < kMapsAtOnce; ++gi) {
                        dot[gi] = 0.f;
                        if (g0 + gi < q_per_k) {
                            const float* qv = q_s + (kg * q_per_k + g0 + gi) * d.d_h + sl * VEC;
#pragma unroll
                            for (int s = 0; s < kSlots; ++s) {
                                if (sl + s * lpr < vecs_per_row) {
#pragma unroll
                                    for (int e = 0; e < VEC; ++e) dot[gi] = fmaf(qv[s * lpr * VEC + e], kv[s][e], dot[gi]);
                                }
                            }
                        }
                    }
                    for (int o = lpr >> 1; o > 0; o >>= 1) {
#pragma unroll
                        for (int gi = 0; gi < kMapsAtOnce; ++gi) dot[gi] += __shfl_xor_sync(0xffffffffu, dot[gi], o);
                    }
                    if (j < n_tok && sl == 0) {
#pragma unroll
                        for (int gi = 0; gi < kMapsAtOnce; ++gi)
                            if (g0 + gi < q_per_k) p_s[j * d.n_q + kg * q_per_k + g0 + gi] = dot[gi] * row_scale[u];
                    }
                }
            }
        }
    } else {
        const int vecs_per_row = d.d_h / VEC;
        int lpr = 1;
        while (lpr < vecs_per_row && lpr < 32) lpr <<= 1;
        const int rows_per_warp = 32 / lpr;
        const int sub = lane / lpr, sl = lane % lpr;
        const int q_per_k = d.n_q / d.n_k;
        const int n_row_iters = (n_tok + rows_per_warp - 1) / rows_per_warp;
        for (int it = warp; it < d.n_k * n_row_iters; it += kDecodeThreads / 32) {
            const int kg = it / n_row_iters;
            const int j = (it % n_row_iters) * rows_per_warp + sub;
            const bool live = j < n_tok;
            // (a block-table entry outside the pool raises the status word; row 0 of the pool stands in)
            const long long k_idx = cache_row(pm, b, d.n_k, kg, S_cap, j_begin + (live ? j : 0), status_word);
            const CT* k_row = k_cache + (size_t)(k_idx < 0 ? 0 : k_idx) * d.d_h;
            const float row_scale = kScaled ? d.scale * k_scale[k_idx < 0 ? 0 : k_idx] : d.scale;
            for (int gi = 0; gi < q_per_k; ++gi) {
                const int g = kg * q_per_k + gi;
                float dot = 0.f;
                for (int v = sl; v < vecs_per_row; v += lpr) {
                    float kv[VEC];
                    Vec16<CT>::load(k_row + v * VEC, kv);
                    const float* qv = q_s + g * d.d_h + v * VEC;
#pragma unroll
                    for (int e = 0; e < VEC; ++e) dot = fmaf(qv[e], kv[e], dot);
                }
                for (int o = lpr >> 1; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
                if (live && sl == 0) p_s[j * d.n_q + g] = dot * row_scale;
            }
        }
    }
    __syncthreads();

    // ---- chunk-local softmax per map: m = max, p = exp(s - m), l = sum p ----
    for (int g = warp; g < d.n_q; g += kDecodeThreads / 32) {
        float m = -INFINITY;
        for (int j = lane; j < n_tok; j += 32) m = fmaxf(m, p_s[j * d.n_q + g]);
        m = warp_max(m);
        float l = 0.f;
        for (int j = lane; j < n_tok; j += 32) {
            const float p = exp_fn<T>(p_s[j * d.n_q + g] - m);
            p_s[j * d.n_q + g] = p;
            l += p;
        }
        l = warp_sum(l);
        if (lane == 0) {
            ml_s[2 * g] = m;
            ml_s[2 * g + 1] = l;
            float* ml = part_ml + (((size_t)b * n_chunks + ck) * d.n_q + g) * 2;
            ml[0] = m;
            ml[1] = l;
        }
    }
    __syncthreads();

    // ---- latent sum: each C row is read once and applied to NGB maps at a time ----
    const int tpr = d.d_l / VEC;                 // threads per latent row
    const int R = kDecodeThreads / tpr;          // rows in flight
    const bool active = tid < R * tpr;
    const int r = tid / tpr, v = tid % tpr;
    const int maps_per_c = d.n_q / d.n_c;
    for (int cg = 0; cg < d.n_c; ++cg) {
        auto c_idx = [&](int j) -> size_t {   // row of token j_begin + j in the latent cache
            const long long idx = cache_row(pm, b, d.n_c, cg, S_cap, j_begin + j, status_word);
            return (size_t)(idx < 0 ? 0 : idx);
        };
        const int g_end = (cg + 1) * maps_per_c;
        for (int g0 = cg * maps_per_c; g0 < g_end; g0 += NGB) {
            float acc[NGB][VEC];
#pragma unroll
            for (int gi = 0; gi < NGB; ++gi)
#pragma unroll
                for (int e = 0; e < VEC; ++e) acc[gi][e] = 0.f;
            if (active) {
                constexpr int U = kScaled ? 2 : 4;         // independent 16-byte loads in flight
                int j = r;
                for (; j + (U - 1) * R < n_tok; j += U * R) {
                    float cv[U][VEC];
                    float cs[U];
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        const size_t idx = c_idx(j + u * R);
                        Vec16<CT>::load(c_cache + idx * d.d_l + v * VEC, cv[u]);
                        cs[u] = kScaled ? c_scale[idx] : 1.f;
                    }
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        const float* pj = p_s + (j + u * R) * d.n_q + g0;
#pragma unroll
                        for (int gi = 0; gi < NGB; ++gi) {
                            if (kReadOnce && g0 + gi >= g_end) break;
                            const float p = pj[gi] * cs[u];      // the row's scale folded into its probability
#pragma unroll
                            for (int e = 0; e < VEC; ++e) acc[gi][e] = fmaf(p, cv[u][e], acc[gi][e]);
                        }
                    }
                }
                for (; j < n_tok; j += R) {
                    float cv[VEC];
                    const size_t idx = c_idx(j);
                    Vec16<CT>::load(c_cache + idx * d.d_l + v * VEC, cv);
                    const float cs = kScaled ? c_scale[idx] : 1.f;
                    const float* pj = p_s + j * d.n_q + g0;
#pragma unroll
                    for (int gi = 0; gi < NGB; ++gi) {
                        if (kReadOnce && g0 + gi >= g_end) break;
                        const float p = pj[gi] * cs;
#pragma unroll
                        for (int e = 0; e < VEC; ++e) acc[gi][e] = fmaf(p, cv[e], acc[gi][e]);
                    }
                }
            }
            // reduce the R row slots through shared memory, one map at a time
#pragma unroll
            for (int gi = 0; gi < NGB; ++gi) {
                if (kReadOnce && g0 + gi >= g_end) break;      // uniform over the CTA
                __syncthreads();
                if (active) {
#pragma unroll
                    for (int e = 0; e < VEC; ++e) red[r * d.d_l + v * VEC + e] = acc[gi][e];
                }
                __syncthreads();
                float* dst = part_o + (((size_t)b * n_chunks + ck) * d.n_q + g0 + gi) * d.d_l;
                for (int col = tid; col < d.d_l; col += kDecodeThreads) {
                    float s = 0.f;
                    for (int rr = 0; rr < R; ++rr) s += red[rr * d.d_l + col];
                    dst[col] = s;
                }
            }
        }
    }
}

// Z partial sums: z_part[split][b][col] = sum_{h in slice} x_t[b][h] * W_G[h][col]
template <typename T>
__global__ void __launch_bounds__(128)
decode_gate_kernel(Dims d, int slice, const T* __restrict__ x_t, const T* __restrict__ w_g,
                   float* __restrict__ z_part) {
    __shared__ float x_s[kGateBatch][kGateMaxSlice];
    const int n_cols = d.n_h * d.d_h;
    const int col = blockIdx.x * 128 + threadIdx.x;
    const int h0 = blockIdx.y * slice;
    const int n_h_rows = min(slice, d.H - h0);
    for (int b0 = 0; b0 < d.B; b0 += kGateBatch) {
        const int nb = min(kGateBatch, d.B - b0);
        __syncthreads();
        for (int idx = threadIdx.x; idx < kGateBatch * slice; idx += 128) {
            const int bb = idx / slice, hh = idx % slice;
            x_s[bb][hh] = (bb < nb && hh < n_h_rows) ? to_f32(x_t[(size_t)(b0 + bb) * d.H + h0 + hh]) : 0.f;
        }
        __syncthreads();
        if (col < n_cols) {
            float acc[kGateBatch];
#pragma unroll
            for (int bb = 0; bb < kGateBatch; ++bb) acc[bb] = 0.f;
            for (int hh = 0; hh < n_h_rows; ++hh) {
                const float w = to_f32(w_g[(size_t)(h0 + hh) * n_cols + col]);
#pragma unroll
                for (int bb = 0; bb < kGateBatch; ++bb) acc[bb] = fmaf(x_s[bb][hh], w, acc[bb]);
            }
#pragma unroll
            for (int bb = 0; bb < kGateBatch; ++bb)
                if (bb < nb) z_part[((size_t)blockIdx.y * d.B + b0 + bb) * n_cols + col] = acc[bb];
        }
    }
}

// Merge + decoder + gate for one head and kFinishSeqs sequences.
// Dynamic shared memory (floats): o_s [kFinishSeqs][d_l] | red [KH][kFinishSeqs][d_h] | w_s [n_chunks]
template <typename T>
__global__ void __launch_bounds__(kDecodeThreads)
decode_finish_kernel(Dims d, int chunk, int n_chunks, int S_cap, int gate_splits,
                     const int32_t* __restrict__ seq_lens, const float* __restrict__ part_o,
                     const float* __restrict__ part_ml, const float* __restrict__ z_part,
                     const T* __restrict__ w_p, T* __restrict__ out) {
    extern __shared__ __align__(16) float smem[];
    float* o_s = smem;
    float* red = o_s + kFinishSeqs * d.d_l;
    float* w_s = red + max(1, kDecodeThreads / d.d_h) * kFinishSeqs * d.d_h;
    const int i = blockIdx.x, b0 = blockIdx.y * kFinishSeqs;
    const int g = d.head_to_q(i);
    const int tid = threadIdx.x;
    const int nb = min(kFinishSeqs, d.B - b0);

    // log-sum-exp merge of the chunk partials of map g
    for (int bb = 0; bb < kFinishSeqs; ++bb) {
        int len = bb < nb ? seq_lens[b0 + bb] : 0;
        len = len < 0 ? 0 : (len > S_cap ? S_cap : len);
        const int live = (len + chunk - 1) / chunk;
        const float* ml = part_ml + (((size_t)(b0 + bb) * n_chunks) * d.n_q + g) * 2;
        const size_t ml_stride = (size_t)d.n_q * 2;
        float m = -INFINITY;
        for (int ck = 0; ck < live; ++ck) m = fmaxf(m, ml[ck * ml_stride]);
        __syncthreads();   // previous round's readers of w_s are done
        for (int ck = tid; ck < live; ck += kDecodeThreads) w_s[ck] = expf(ml[ck * ml_stride] - m);
        __syncthreads();
        float l = 0.f;
        for (int ck = 0; ck < live; ++ck) l = fmaf(ml[ck * ml_stride + 1], w_s[ck], l);
        const float inv_l = live > 0 ? 1.f / l : 0.f;
        const float* po = part_o + (((size_t)(b0 + bb) * n_chunks) * d.n_q + g) * d.d_l;
        const size_t po_stride = (size_t)d.n_q * d.d_l;
        for (int col = tid; col < d.d_l; col += kDecodeThreads) {
            float s = 0.f;
            for (int ck = 0; ck < live; ++ck) s = fmaf(po[ck * po_stride + col], w_s[ck], s);
            o_s[bb * d.d_l + col] = s * inv_l;
        }
    }
    __syncthreads();

    // decoder GEMV: KH slices of d_l, one output column per thread
    const int KH = max(1, kDecodeThreads / d.d_h);
    const int e = tid % d.d_h, kh = tid / d.d_h;
    const bool active = kh < KH;
    float acc[kFinishSeqs];
#pragma unroll
    for (int bb = 0; bb < kFinishSeqs; ++bb) acc[bb] = 0.f;
    if (active) {
        const int l_per = (d.d_l + KH - 1) / KH;
        const int l_end = min(d.d_l, (kh + 1) * l_per);
        const T* wp = w_p + (size_t)i * d.d_l * d.d_h + e;
        for (int l = kh * l_per; l < l_end; ++l) {
            const float w = to_f32(wp[(size_t)l * d.d_h]);
#pragma unroll
            for (int bb = 0; bb < kFinishSeqs; ++bb) acc[bb] = fmaf(o_s[bb * d.d_l + l], w, acc[bb]);
        }
#pragma unroll
        for (int bb = 0; bb < kFinishSeqs; ++bb) red[(kh * kFinishSeqs + bb) * d.d_h + e] = acc[bb];
    }
    __syncthreads();
    const int n_cols = d.n_h * d.d_h;
    for (int idx = tid; idx < nb * d.d_h; idx += kDecodeThreads) {
        const int bb = idx / d.d_h, ee = idx % d.d_h;
        float y = 0.f;
        for (int s = 0; s < KH; ++s) y += red[(s * kFinishSeqs + bb) * d.d_h + ee];
        float z = 0.f;
        for (int s = 0; s < gate_splits; ++s)
            z += z_part[((size_t)s * d.B + b0 + bb) * n_cols + i * d.d_h + ee];
        const float gate = 1.f / (1.f + expf(-z));
        out[((size_t)(b0 + bb) * d.n_h + i) * d.d_h + ee] = from_f32<T>(y * gate);
    }
}

// kReadOnce: the caches are read over the host link (see decode_partial_kernel)
template <typename T, bool kReadOnce = false>
static cudaError_t launch_decode_typed(const Dims& d, const void* q, const void* k_cache, const void* c_cache,
                                       const int32_t* seq_lens, int S_cap, const void* x_t, const void* w_p,
                                       const void* w_g, void* out, void* workspace, int32_t* status_word,
                                       cudaStream_t stream, int stages, int* launches, const PageMap& pm) {
    constexpr int VEC = Vec16<T>::N;
    const DecodePlan p = make_plan(d, S_cap);
    float* part_o = reinterpret_cast<float*>(workspace);
    float* part_ml = reinterpret_cast<float*>(static_cast<char*>(workspace) + p.off_ml);
    float* z_part = reinterpret_cast<float*>(static_cast<char*>(workspace) + p.off_z);
    cudaError_t err;

    if (stages & 1) {   // gate partial sums (independent of the caches)
        dim3 grid((d.n_h * d.d_h + 127) / 128, p.gate_splits);
        decode_gate_kernel<T><<<grid, 128, 0, stream>>>(d, p.gate_slice, (const T*)x_t, (const T*)w_g, z_part);
        if ((err = cudaGetLastError()) != cudaSuccess) return err;
        *launches += 1;
    }
    if ((stages & 2) && S_cap > 0) {
        const int tpr = d.d_l / VEC;
        const int R = kDecodeThreads / tpr;
        const size_t smem = ((size_t)d.n_q * d.d_h + (size_t)p.chunk * d.n_q + 2 * d.n_q + (size_t)R * d.d_l) * sizeof(float);
        const int maps_per_c = d.n_q / d.n_c;
        dim3 grid(p.n_chunks, d.B);
#define GTA_LAUNCH_PARTIAL(NGB)                                                                        \
        do {                                                                                           \
            auto kern = decode_partial_kernel<T, NGB, T, kReadOnce>;                                   \
            if (smem > 48 * 1024) {                                                                    \
                err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
                if (err != cudaSuccess) return err;                                                    \
            }                                                                                          \
            kern<<<grid, kDecodeThreads, smem, stream>>>(d, p.chunk, p.n_chunks, S_cap, (const T*)q,   \
                                                         (const T*)k_cache, (const T*)c_cache, seq_lens, \
                                                         part_o, part_ml, pm, status_word, nullptr, nullptr); \
        } while (0)
        if (kReadOnce) {    // as few passes over the latent rows as the accumulators allow
            if (maps_per_c >= 5) GTA_LAUNCH_PARTIAL(8);
            else if (maps_per_c >= 3) GTA_LAUNCH_PARTIAL(4);
            else if (maps_per_c == 2) GTA_LAUNCH_PARTIAL(2);
            else GTA_LAUNCH_PARTIAL(1);
        } else if (maps_per_c % 8 == 0) GTA_LAUNCH_PARTIAL(8);
        else if (maps_per_c % 4 == 0) GTA_LAUNCH_PARTIAL(4);
        else if (maps_per_c % 2 == 0) GTA_LAUNCH_PARTIAL(2);
        else GTA_LAUNCH_PARTIAL(1);
#undef GTA_LAUNCH_PARTIAL
        if ((err = cudaGetLastError()) != cudaSuccess) return err;
        *launches += 1;
    }
    if (stages & 4) {
        const int KH = kDecodeThreads / d.d_h > 0 ? kDecodeThreads / d.d_h : 1;
        const size_t smem = ((size_t)kFinishSeqs * d.d_l + (size_t)KH * kFinishSeqs * d.d_h + p.n_chunks) * sizeof(float);
        auto kern = decode_finish_kernel<T>;
        if (smem > 48 * 1024) {
            err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (err != cudaSuccess) return err;
        }
        dim3 grid(d.n_h, (d.B + kFinishSeqs - 1) / kFinishSeqs);
        kern<<<grid, kDecodeThreads, smem, stream>>>(d, p.chunk, p.n_chunks, S_cap, p.gate_splits, seq_lens,
                                                    part_o, part_ml, z_part, (const T*)w_p, (T*)out);
        if ((err = cudaGetLastError()) != cudaSuccess) return err;
        *launches += 1;
    }
    return cudaSuccess;
}

// ---- 8-bit caches: e4m3 codes with one fp32 scale per cached row (token and group).  Reading (the paper
//      fixes none; its Sec. 5.3 / App. C.2 only observe that decode is bound by the bytes of the cache):
//      scale = max|row| / 448 (1 for an all-zero row), code = round-to-nearest-even(x / scale), both
//      divisions in fp32; the operator runs on code * scale.
size_t decode_fp8_workspace_bytes(const Dims& d, int S_cap) { return make_plan(d, S_cap).total; }

template <typename T>
static cudaError_t launch_decode_fp8_typed(const Dims& d, const void* q, const void* k_codes, const void* c_codes,
                                           const float* k_scale, const float* c_scale, const int32_t* seq_lens,
                                           int S_cap, const void* x_t, const void* w_p, const void* w_g, void* out,
                                           void* workspace, int32_t* status_word, cudaStream_t stream, int* launches) {
    const DecodePlan p = make_plan(d, S_cap);
    float* part_o = reinterpret_cast<float*>(workspace);
    float* part_ml = reinterpret_cast<float*>(static_cast<char*>(workspace) + p.off_ml);
    float* z_part = reinterpret_cast<float*>(static_cast<char*>(workspace) + p.off_z);
    cudaError_t err;
    dim3 ggrid((d.n_h * d.d_h + 127) / 128, p.gate_splits);
    decode_gate_kernel<T><<<ggrid, 128, 0, stream>>>(d, p.gate_slice, (const T*)x_t, (const T*)w_g, z_part);
    if ((err = cudaGetLastError()) != cudaSuccess) return err;
    {
        constexpr int VEC = 16;
        const int tpr = d.d_l / VEC;
        const int R = kDecodeThreads / tpr;
        const size_t smem = ((size_t)d.n_q * d.d_h + (size_t)p.chunk * d.n_q + 2 * d.n_q + (size_t)R * d.d_l) * sizeof(float);
        const int maps_per_c = d.n_q / d.n_c;
        dim3 grid(p.n_chunks, d.B);
#define GTA_LAUNCH_PARTIAL8(NGB)                                                                       \
        do {                                                                                           \
            auto kern = decode_partial_kernel<T, NGB, Fp8>;                                            \
            if (smem > 48 * 1024) {                                                                    \
                err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
                if (err != cudaSuccess) return err;                                                    \
            }                                                                                          \
            kern<<<grid, kDecodeThreads, smem, stream>>>(d, p.chunk, p.n_chunks, S_cap, (const T*)q,   \
                                                         (const Fp8*)k_codes, (const Fp8*)c_codes, seq_lens, \
                                                         part_o, part_ml, PageMap(), status_word, k_scale, c_scale); \
        } while (0)
        if (maps_per_c % 4 == 0) GTA_LAUNCH_PARTIAL8(4);
        else if (maps_per_c % 2 == 0) GTA_LAUNCH_PARTIAL8(2);
        else GTA_LAUNCH_PARTIAL8(1);
#undef GTA_LAUNCH_PARTIAL8
        if ((err = cudaGetLastError()) != cudaSuccess) return err;
    }
    {
        const int KH = kDecodeThreads / d.d_h > 0 ? kDecodeThreads / d.d_h : 1;
        const size_t smem = ((size_t)kFinishSeqs * d.d_l + (size_t)KH * kFinishSeqs * d.d_h + p.n_chunks) * sizeof(float);
        auto kern = decode_finish_kernel<T>;
        if (smem > 48 * 1024) {
            err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (err != cudaSuccess) return err;
        }
        dim3 grid(d.n_h, (d.B + kFinishSeqs - 1) / kFinishSeqs);
        kern<<<grid, kDecodeThreads, smem, stream>>>(d, p.chunk, p.n_chunks, S_cap, p.gate_splits, seq_lens, part_o,
                                                    part_ml, z_part, (const T*)w_p, (T*)out);
        if ((err = cudaGetLastError()) != cudaSuccess) return err;
    }
    *launches += 3;
    return cudaSuccess;
}

cudaError_t launch_decode_fp8(const Dims& d, int dtype, const void* q, const void* k_codes, const void* c_codes,
                              const float* k_scale, const float* c_scale, const int32_t* seq_lens, int S_cap,
                              const void* x_t, const void* w_p, const void* w_g, void* out, void* workspace,
                              int32_t* status_word, cudaStream_t stream, int* launches) {
    if (dtype == GTA_F32)
        return launch_decode_fp8_typed<float>(d, q, k_codes, c_codes, k_scale, c_scale, seq_lens, S_cap, x_t, w_p, w_g,
                                              out, workspace, status_word, stream, launches);
    return launch_decode_fp8_typed<__nv_bfloat16>(d, q, k_codes, c_codes, k_scale, c_scale, seq_lens, S_cap, x_t, w_p,
                                                  w_g, out, workspace, status_word, stream, launches);
}

// Quantising append: one warp per new row (token and group): the row's largest magnitude, its scale, its codes.
// One CTA per sequence; the length advances when all its rows are written.  src rows [B][groups][n_new][width].
__device__ __forceinline__ uint32_t f32_to_e4m3(float y) {
    uint16_t r;   // the low byte of the pair is the second source operand
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(0.f), "f"(y));
    return r & 0xffu;
}
template <typename T>
__device__ __forceinline__ void quantise_row(const T* __restrict__ src, uint8_t* __restrict__ dst,
                                             float* __restrict__ scale_out, int width, int lane) {
    float amax = 0.f;
    for (int e = lane; e < width; e += 32) amax = fmaxf(amax, fabsf(to_f32(src[e])));
    amax = warp_max(amax);
    const float scale = amax > 0.f ? __fdiv_rn(amax, 448.f) : 1.f;
    for (int e = lane * 4; e < width; e += 128) {        // widths are multiples of 8: four codes per store
        uint32_t w = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) w |= f32_to_e4m3(__fdiv_rn(to_f32(src[e + i]), scale)) << (8 * i);
        *reinterpret_cast<uint32_t*>(dst + e) = w;
    }
    if (lane == 0) *scale_out = scale;
}
template <typename T>
__global__ void __launch_bounds__(256)
append_fp8_kernel(Dims d, int S_cap, int n_new, uint8_t* __restrict__ k_codes, uint8_t* __restrict__ c_codes,
                  float* __restrict__ k_scale, float* __restrict__ c_scale, const T* __restrict__ k_new,
                  const T* __restrict__ c_new, int32_t* __restrict__ seq_lens, int32_t* status_word) {
    const int b = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int len = seq_lens[b];
    __syncthreads();   // every thread has read the old length before thread 0 rewrites it
    if (len < 0 || (long long)len + n_new > S_cap) {
        if (threadIdx.x == 0) raise_status(status_word, GTA_ERR_CACHE_FULL);
        return;
    }
    const int k_rows = d.n_k * n_new, rows = k_rows + d.n_c * n_new;
    for (int r = warp; r < rows; r += 8) {
        if (r < k_rows) {
            const int g = r / n_new, n = r % n_new;
            const size_t row = ((size_t)b * d.n_k + g) * S_cap + len + n;
            quantise_row(k_new + (((size_t)b * d.n_k + g) * n_new + n) * d.d_h, k_codes + row * d.d_h, k_scale + row,
                         d.d_h, lane);
        } else {
            const int g = (r - k_rows) / n_new, n = (r - k_rows) % n_new;
            const size_t row = ((size_t)b * d.n_c + g) * S_cap + len + n;
            quantise_row(c_new + (((size_t)b * d.n_c + g) * n_new + n) * d.d_l, c_codes + row * d.d_l, c_scale + row,
                         d.d_l, lane);
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) seq_lens[b] = len + n_new;
}

cudaError_t launch_cache_append_fp8(const Dims& d, int dtype, void* k_codes, void* c_codes, float* k_scale,
                                    float* c_scale, int S_cap, const void* k_new, const void* c_new, int n_new,
                                    int32_t* seq_lens, int32_t* status_word, cudaStream_t stream, int* launches) {
    if (dtype == GTA_F32)
        append_fp8_kernel<float><<<d.B, 256, 0, stream>>>(d, S_cap, n_new, (uint8_t*)k_codes, (uint8_t*)c_codes, k_scale,
                                                           c_scale, (const float*)k_new, (const float*)c_new, seq_lens,
                                                           status_word);
    else
        append_fp8_kernel<__nv_bfloat16><<<d.B, 256, 0, stream>>>(d, S_cap, n_new, (uint8_t*)k_codes, (uint8_t*)c_codes,
                                                                   k_scale, c_scale, (const __nv_bfloat16*)k_new,
                                                                   (const __nv_bfloat16*)c_new, seq_lens, status_word);
    *launches += 1;
    return cudaGetLastError();
}

size_t decode_plain_workspace_bytes(const Dims& d, int S_cap) { return make_plan(d, S_cap).total; }

// The plain-ALU kernels whatever the shape: they read the caches with ordinary 16-byte loads, which is what a cache
// in page-locked host memory (reached over the host link) needs; the TMA path is kept to device memory.
cudaError_t launch_decode_plain(const Dims& d, int dtype, const void* q, const void* k_cache, const void* c_cache,
                                const int32_t* seq_lens, int S_cap, const void* x_t, const void* w_p,
                                const void* w_g, void* out, void* workspace, int32_t* status_word,
                                cudaStream_t stream, int* launches) {
    if (dtype == GTA_F32)
        return launch_decode_typed<float, true>(d, q, k_cache, c_cache, seq_lens, S_cap, x_t, w_p, w_g, out,
                                                workspace, status_word, stream, 7, launches, PageMap());
    return launch_decode_typed<__nv_bfloat16, true>(d, q, k_cache, c_cache, seq_lens, S_cap, x_t, w_p, w_g, out,
                                                    workspace, status_word, stream, 7, launches, PageMap());
}

cudaError_t launch_decode(const Dims& d, int dtype, const void* q, const void* k_cache, const void* c_cache,
                          const int32_t* seq_lens, int S_cap, const void* x_t, const void* w_p,
                          const void* w_g, void* out, void* workspace, int32_t* status_word,
                          cudaStream_t stream, int stages, int* launches, const PageMap& pm) {
    if (decode_fast_supported(d, dtype, pm.table ? pm.page_size : 0) && S_cap > 0)
        return launch_decode_fast(d, q, k_cache, c_cache, seq_lens, S_cap, x_t, w_p, w_g, out, workspace,
                                  status_word, stream, stages, launches, pm);
    if (dtype == GTA_F32)
        return launch_decode_typed<float>(d, q, k_cache, c_cache, seq_lens, S_cap, x_t, w_p, w_g, out,
                                          workspace, status_word, stream, stages, launches, pm);
    return launch_decode_typed<__nv_bfloat16>(d, q, k_cache, c_cache, seq_lens, S_cap, x_t, w_p, w_g, out,
                                              workspace, status_word, stream, stages, launches, pm);
}

}  // namespace gta
