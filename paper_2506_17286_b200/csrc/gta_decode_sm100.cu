// Bandwidth-oriented decode for bf16 caches (App. B.1.3), d_h = 128, one latent group.
//
//   decode_stream_kernel : persistent, two CTAs per SM.  The live tokens of all sequences are
//       cut into sub-tiles of TS tokens; CTA c owns the contiguous sub-tile range
//       [c n / G, (c+1) n / G), so every CTA streams the same number of cache bytes whatever
//       the length mix.  A producer warp copies each sub-tile (the K rows of every key group and
//       the latent rows) into a 3-stage shared-memory ring with bulk async copies; 256 consumer
//       threads compute the scores of all maps, a running softmax (the maximum is only raised
//       when it grows by more than 2^8) and the latent sums, each latent row being read once and
//       applied to all maps with packed fp32x2 FMAs.  When the range crosses into the next
//       sequence, and at its end, the partial (max, sum, latent sum) goes to slot c + b.
//   decode_finish_kernel : clusters of 8 CTAs per head split the reduction dimensions of the
//       decoder (d_l) and of the gate (H); every CTA merges the slots of its d_l slice
//       (log-sum-exp), multiplies by its slices of W_P,i and W_G,i for 32 sequences at a time,
//       and the cluster adds the eight partial results through distributed shared memory before
//       the sigmoid gate is applied.
#include <cooperative_groups.h>

#include "gta_common.cuh"
#include "sm100_ptx.cuh"

namespace cg = cooperative_groups;

namespace gta {

constexpr int kStreamConsumers = 256;
constexpr int kStreamThreads = kStreamConsumers + 32;
constexpr int kStreamStages = 3;
constexpr int kStreamStageBytes = 32768;
constexpr int kStreamMaxBatch = 512;
constexpr int kStreamMaxTS = 32;
constexpr int kFinSplit = 8;
constexpr int kFinBlockB = 32;
constexpr int kFinThreads = 256;

struct FastPlan {
    int TS;        // tokens per sub-tile
    int G;         // stream CTAs
    int slots;     // G + B partial slots
    size_t off_ml, off_prefix, total;
};

static size_t align256f(size_t v) { return (v + 255) & ~(size_t)255; }

bool decode_fast_supported(const Dims& d, int dtype) {
    if (dtype != GTA_BF16 || d.d_h != 128 || d.n_c != 1) return false;
    if (d.d_l != 256 && d.d_l != 512 && d.d_l != 1024) return false;
    if (d.n_q != 1 && d.n_q != 2 && d.n_q != 4 && d.n_q != 8) return false;
    if (d.B > kStreamMaxBatch || d.H % 64 != 0) return false;
    const int tok_bytes = (d.n_k * d.d_h + d.d_l) * 2;
    return tok_bytes * 4 <= kStreamStageBytes;
}

static int sm_count() {
    static int n = [] {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0)
            v = 148;
        return v;
    }();
    return n;
}

static FastPlan make_fast_plan(const Dims& d) {
    FastPlan p;
    const int tok_bytes = (d.n_k * d.d_h + d.d_l) * 2;
    int ts = 1;
    while (ts * 2 * tok_bytes <= kStreamStageBytes && ts * 2 <= kStreamMaxTS) ts *= 2;
    p.TS = ts;
    p.G = 2 * sm_count();
    p.slots = p.G + d.B;
    const size_t part_o = (size_t)p.slots * d.n_q * d.d_l * sizeof(float);
    const size_t part_ml = (size_t)p.slots * d.n_q * 2 * sizeof(float);
    p.off_ml = align256f(part_o);
    p.off_prefix = p.off_ml + align256f(part_ml);
    p.total = p.off_prefix + align256f((size_t)(d.B + 1) * sizeof(int32_t));
    return p;
}

size_t decode_fast_workspace_bytes(const Dims& d) { return make_fast_plan(d).total; }

// ---------------------------------------------------------------------------------------------
// Bulk async copy global -> shared, completion counted on `bar`; the cache bytes are read once, so
// they are marked evict-first in L2 (the weights of the finish kernel stay resident).
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void bulk_copy_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar,
                                              uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(ptx::smem_addr(dst)), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(ptx::smem_addr(bar)),
          "l"(policy)
        : "memory");
}
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
    return (uint64_t)__float_as_uint(lo) | ((uint64_t)__float_as_uint(hi) << 32);
}
__device__ __forceinline__ void ffma2(uint64_t& acc, uint64_t a, uint64_t b) {
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(acc) : "l"(a), "l"(b));
}
__device__ __forceinline__ uint64_t fmul2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ int clamp_len(int len, int S_cap) { return len < 0 ? 0 : (len > S_cap ? S_cap : len); }

// Which stream CTA owns sub-tile `st` when n sub-tiles are dealt to G CTAs in contiguous ranges
// [c n / G, (c + 1) n / G).
__device__ __forceinline__ int owner_of(long long st, long long n, int G) {
    int c = (int)((st * G) / n);
    while (c + 1 < G && ((long long)(c + 1) * n) / G <= st) ++c;
    while (c > 0 && ((long long)c * n) / G > st) --c;
    return c;
}

// With fewer sub-tiles than CTAs some CTAs own nothing and never write their slot.
__device__ __forceinline__ bool owns_any(int c, long long n, int G) {
    return ((long long)c * n) / G < ((long long)(c + 1) * n) / G;
}

template <int NQ>
__global__ void __launch_bounds__(kStreamThreads, 2)
decode_stream_kernel(Dims d, int TS, int S_cap, const __nv_bfloat16* __restrict__ q,
                     const __nv_bfloat16* __restrict__ k_cache, const __nv_bfloat16* __restrict__ c_cache,
                     const int32_t* __restrict__ seq_lens, float* __restrict__ part_o, float* __restrict__ part_ml,
                     int32_t* __restrict__ prefix_g, int32_t* status_word) {
    extern __shared__ __align__(128) uint8_t smem[];
    uint8_t* ring = smem;                                                    // 3 x 32 KB
    float* q_s = reinterpret_cast<float*>(smem + kStreamStages * kStreamStageBytes);   // [NQ][128]
    float2* p2_s = reinterpret_cast<float2*>(q_s + NQ * 128);                // [2][TS][NQ] pairs (p, p)
    float* a_s = reinterpret_cast<float*>(p2_s + 2 * kStreamMaxTS * NQ);     // [2][NQ] rescale factors
    float* red = a_s + 2 * NQ;                                               // [R][d_l / 2]; scan scratch at start
    int32_t* prefix = reinterpret_cast<int32_t*>(red + 1024);                // [B + 1]
    int32_t* scan_tmp = reinterpret_cast<int32_t*>(red);                     // [kStreamThreads] (start-up only)
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(prefix + kStreamMaxBatch + 2);
    full_bar = reinterpret_cast<uint64_t*>((reinterpret_cast<uintptr_t>(full_bar) + 7) & ~(uintptr_t)7);
    uint64_t* empty_bar = full_bar + kStreamStages;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(empty_bar + kStreamStages);
    volatile int* drain_flag = abort_flag + 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int G = gridDim.x, cta = blockIdx.x;

    // ---- exclusive prefix sum of the sub-tile counts: prefix[b] = sum_{b' < b} ceil(len / TS)
    {
        const int per = (d.B + kStreamThreads - 1) / kStreamThreads;
        const int lo = min(tid * per, d.B), hi = min(lo + per, d.B);
        int sum = 0;
        for (int b = lo; b < hi; ++b) sum += (clamp_len(seq_lens[b], S_cap) + TS - 1) / TS;
        scan_tmp[tid] = sum;
        if (tid == 0) {
            for (int s = 0; s < kStreamStages; ++s) { ptx::mbar_init(&full_bar[s], 1); ptx::mbar_init(&empty_bar[s], 8); }
            *abort_flag = 0;
            *drain_flag = 0;
            ptx::fence_mbar_init();
        }
        __syncthreads();
        int base = 0;
        for (int t = 0; t < tid; ++t) base += scan_tmp[t];
        for (int b = lo; b < hi; ++b) {
            prefix[b] = base;
            base += (clamp_len(seq_lens[b], S_cap) + TS - 1) / TS;
        }
        if (hi == d.B && lo < d.B) prefix[d.B] = base;
        if (d.B == 0 && tid == 0) prefix[0] = 0;
        __syncthreads();
        if (cta == 0)
            for (int b = tid; b <= d.B; b += kStreamThreads) prefix_g[b] = prefix[b];
    }
    const long long n_st = prefix[d.B];
    const long long st_begin = ((long long)cta * n_st) / G, st_end = ((long long)(cta + 1) * n_st) / G;
    if (st_begin >= st_end) return;      // uniform: nothing armed, nothing allocated
    int b0;
    {   // largest b with prefix[b] <= st_begin and a non-empty sequence
        int lo = 0, hi = d.B - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (prefix[mid] <= st_begin) lo = mid; else hi = mid - 1;
        }
        b0 = lo;
    }
    const int tok_bytes_k = d.n_k * 256;
    const int row_bytes_c = d.d_l * 2;
    const uint32_t c_off = (uint32_t)d.n_k * TS * 256;   // latent rows start here inside a stage

    if (warp == kStreamConsumers / 32) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            const uint64_t policy = l2_evict_first_policy();
            int b = b0;
            long long k = st_begin - prefix[b0];
            int it = 0;
            for (long long st = st_begin; st < st_end; ++st, ++it, ++k) {
                while (k >= prefix[b + 1] - prefix[b]) { ++b; k = 0; }
                const int s = it % kStreamStages;
                const uint32_t ph = (it / kStreamStages) & 1;
                if (!ptx::mbar_wait(&empty_bar[s], ph ^ 1, abort_flag)) break;
                const int len = clamp_len(seq_lens[b], S_cap);
                const int tok0 = (int)k * TS;
                const int n_valid = min(TS, len - tok0);
                uint8_t* stage = ring + s * kStreamStageBytes;
                ptx::mbar_arrive_expect_tx(&full_bar[s], (uint32_t)n_valid * (tok_bytes_k + row_bytes_c));
                for (int kg = 0; kg < d.n_k; ++kg)
                    bulk_copy_g2s(stage + kg * TS * 256,
                                  k_cache + (((size_t)b * d.n_k + kg) * S_cap + tok0) * 128, n_valid * 256, &full_bar[s], policy);
                bulk_copy_g2s(stage + c_off, c_cache + ((size_t)b * S_cap + tok0) * d.d_l, n_valid * row_bytes_c,
                              &full_bar[s], policy);
            }
            if (*abort_flag) {
                for (int back = 1; back <= kStreamStages && it - back >= 0; ++back) {
                    const int iq = it - back;
                    ptx::mbar_wait(&full_bar[iq % kStreamStages], (iq / kStreamStages) & 1, drain_flag);
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ consumers
        const int tpr = d.d_l / 8;                 // threads per latent row (32, 64 or 128)
        const int R = kStreamConsumers / tpr;      // latent rows in flight
        const int r = tid / tpr, v = tid % tpr;
        const int qpk = NQ / d.n_k;
        const int n_it = (TS + 7) / 8;             // score iterations: 8 key rows per warp and iteration
        const float c_scale = d.scale * 1.4426950408889634f;
        const int quad = lane >> 2, ql = lane & 3;
        float m_run = -INFINITY, l_run = 0.f;      // softmax state of map `warp` (warps < NQ)
        uint64_t acc[NQ][4];
#pragma unroll
        for (int g = 0; g < NQ; ++g)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[g][e] = 0ull;

        auto load_q = [&](int b) {
            for (int e = tid; e < NQ * 128; e += kStreamConsumers)
                q_s[e] = __bfloat162float(q[(size_t)b * NQ * 128 + e]);
            m_run = -INFINITY;
            l_run = 0.f;
            consumer_sync();
        };
        auto flush = [&](int b) {
            const int slot = cta + b;
            const int half_cols = d.d_l / 2;
#pragma unroll
            for (int g = 0; g < NQ; ++g) {
                for (int h = 0; h < 2; ++h) {
                    consumer_sync();
                    if ((v * 8) / half_cols == h) {
                        float* dst = red + r * half_cols + (v * 8 - h * half_cols);
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            dst[2 * e] = __uint_as_float((uint32_t)acc[g][e]);
                            dst[2 * e + 1] = __uint_as_float((uint32_t)(acc[g][e] >> 32));
                        }
                    }
                    consumer_sync();
                    float* out_row = part_o + ((size_t)slot * NQ + g) * d.d_l + h * half_cols;
                    for (int col = tid; col < half_cols; col += kStreamConsumers) {
                        float s = 0.f;
                        for (int rr = 0; rr < R; ++rr) s += red[rr * half_cols + col];
                        out_row[col] = s;
                    }
                }
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[g][e] = 0ull;
            }
            if (warp < NQ && lane == 0) {
                part_ml[((size_t)slot * NQ + warp) * 2] = m_run;
                part_ml[((size_t)slot * NQ + warp) * 2 + 1] = l_run;
            }
            consumer_sync();
        };

        int b = b0;
        long long k = st_begin - prefix[b0];
        load_q(b);
        int it = 0;
        bool ok = true;
        for (long long st = st_begin; st < st_end; ++st, ++it, ++k) {
            if (k >= prefix[b + 1] - prefix[b]) {
                flush(b);
                do { ++b; } while (prefix[b + 1] == prefix[b]);
                k = 0;
                load_q(b);
            }
            const int s = it % kStreamStages;
            const uint32_t ph = (it / kStreamStages) & 1;
            ok = __all_sync(0xffffffffu, ptx::mbar_wait(&full_bar[s], ph, abort_flag));
            if (!ok) break;
            const int len = clamp_len(seq_lens[b], S_cap);
            const int n_valid = min(TS, len - (int)k * TS);
            const uint8_t* stage = ring + s * kStreamStageBytes;
            float2* p2 = p2_s + (it & 1) * kStreamMaxTS * NQ;     // [TS][NQ] pairs (p, p)
            float* alpha_s = a_s + (it & 1) * NQ;

            // ---- scores + running softmax of map `warp`: a quad of lanes per key row
            if (warp < NQ) {
                const int g = warp, kg = g / qpk;
                const float* qv = q_s + g * 128;
                float sc[4];
                float m_loc = -INFINITY;
#pragma unroll
                for (int i8 = 0; i8 < 4; ++i8) {
                    sc[i8] = -INFINITY;
                    if (i8 < n_it) {
                        const int tok = i8 * 8 + quad;
                        const uint8_t* row = stage + (size_t)(kg * TS + min(tok, TS - 1)) * 256;
                        float dot = 0.f;
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int vec = ql + 4 * u;
                            const uint4 kv = *reinterpret_cast<const uint4*>(row + vec * 16);
                            const float4 qa = *reinterpret_cast<const float4*>(qv + vec * 8);
                            const float4 qb = *reinterpret_cast<const float4*>(qv + vec * 8 + 4);
                            dot = fmaf(qa.x, __uint_as_float(kv.x << 16), dot);
                            dot = fmaf(qa.y, __uint_as_float(kv.x & 0xffff0000u), dot);
                            dot = fmaf(qa.z, __uint_as_float(kv.y << 16), dot);
                            dot = fmaf(qa.w, __uint_as_float(kv.y & 0xffff0000u), dot);
                            dot = fmaf(qb.x, __uint_as_float(kv.z << 16), dot);
                            dot = fmaf(qb.y, __uint_as_float(kv.z & 0xffff0000u), dot);
                            dot = fmaf(qb.z, __uint_as_float(kv.w << 16), dot);
                            dot = fmaf(qb.w, __uint_as_float(kv.w & 0xffff0000u), dot);
                        }
                        dot += __shfl_xor_sync(0xffffffffu, dot, 1);
                        dot += __shfl_xor_sync(0xffffffffu, dot, 2);
                        if (tok < n_valid) sc[i8] = dot * c_scale;
                        m_loc = fmaxf(m_loc, sc[i8]);
                    }
                }
                m_loc = fmaxf(m_loc, __shfl_xor_sync(0xffffffffu, m_loc, 4));
                m_loc = fmaxf(m_loc, __shfl_xor_sync(0xffffffffu, m_loc, 8));
                m_loc = fmaxf(m_loc, __shfl_xor_sync(0xffffffffu, m_loc, 16));
                float alpha = 1.f;
                if (m_loc > m_run + 8.f) { alpha = ex2f(m_run - m_loc); m_run = m_loc; }
                float sum = 0.f;
#pragma unroll
                for (int i8 = 0; i8 < 4; ++i8) {
                    if (i8 < n_it) {
                        const int tok = i8 * 8 + quad;
                        const float p = ex2f(sc[i8] - m_run);
                        sum += p;
                        if (ql == 0 && tok < TS) p2[tok * NQ + g] = make_float2(p, p);
                    }
                }
                sum += __shfl_xor_sync(0xffffffffu, sum, 4);
                sum += __shfl_xor_sync(0xffffffffu, sum, 8);
                sum += __shfl_xor_sync(0xffffffffu, sum, 16);
                l_run = l_run * alpha + sum;     // every lane of a quad holds the same p: sum counts each token once
                if (lane == 0) alpha_s[g] = alpha;
            }
            consumer_sync();
            // ---- latent sums: each row read once, applied to all maps
            {
                bool rescale = false;
#pragma unroll
                for (int g = 0; g < NQ; ++g) rescale |= (alpha_s[g] != 1.f);
                if (rescale) {
#pragma unroll
                    for (int g = 0; g < NQ; ++g) {
                        const uint64_t a2 = pack2(alpha_s[g], alpha_s[g]);
#pragma unroll
                        for (int e = 0; e < 4; ++e) acc[g][e] = fmul2(acc[g][e], a2);
                    }
                }
                const uint8_t* c_rows = stage + c_off + v * 16;
#pragma unroll 2
                for (int j = r; j < n_valid; j += R) {
                    const uint4 cv = *reinterpret_cast<const uint4*>(c_rows + (size_t)j * row_bytes_c);
                    const uint32_t w[4] = {cv.x, cv.y, cv.z, cv.w};
                    uint64_t c2[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        c2[e] = (uint64_t)(w[e] << 16) | ((uint64_t)(w[e] & 0xffff0000u) << 32);
                    const uint64_t* pj = reinterpret_cast<const uint64_t*>(p2 + j * NQ);
#pragma unroll
                    for (int g = 0; g < NQ; ++g) {
                        const uint64_t pp = pj[g];
#pragma unroll
                        for (int e = 0; e < 4; ++e) ffma2(acc[g][e], pp, c2[e]);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&empty_bar[s]);
        }
        if (ok) flush(b);
    }
    __syncthreads();
    if (tid == 0 && *abort_flag) raise_status(status_word, GTA_ERR_TIMEOUT);
}

// ---------------------------------------------------------------------------------------------
// Dynamic shared memory (floats): o_s [d_l/8][32] | x_s [H/8][32] | part_s [2][32][128] |
//                                  mrg [32][4] (max, 1/sum, first slot, last slot)
__global__ void __cluster_dims__(kFinSplit, 1, 1) __launch_bounds__(kFinThreads)
decode_finish_cluster_kernel(Dims d, int G, int TS, int S_cap, const int32_t* __restrict__ seq_lens,
                             const int32_t* __restrict__ prefix_g, const float* __restrict__ part_o,
                             const float* __restrict__ part_ml, const __nv_bfloat16* __restrict__ x_t,
                             const __nv_bfloat16* __restrict__ w_p, const __nv_bfloat16* __restrict__ w_g,
                             __nv_bfloat16* __restrict__ out) {
    cg::cluster_group cluster = cg::this_cluster();
    extern __shared__ __align__(16) float fsm[];
    const int dl8 = d.d_l / kFinSplit, h8 = d.H / kFinSplit;
    float* o_s = fsm;
    float* x_s = o_s + dl8 * kFinBlockB;
    float* part_s = x_s + h8 * kFinBlockB;
    float* mrg = part_s + 2 * kFinBlockB * 128;
    const int split = blockIdx.x;            // = rank inside the cluster
    const int i = blockIdx.y;                // head
    const int g = d.head_to_q(i);
    const int tid = threadIdx.x;
    const long long n_st = prefix_g[d.B];
    const int n_cols = d.n_h * 128;

    for (int b0 = 0; b0 < d.B; b0 += kFinBlockB) {
        const int nb = min(kFinBlockB, d.B - b0);
        // ---- per sequence: slot range, merged maximum and 1 / merged sum
        if (tid < kFinBlockB) {
            float M = -INFINITY, inv_l = 0.f;
            int c_lo = 0, c_hi = -1;
            if (tid < nb) {
                const int b = b0 + tid;
                const long long s_lo = prefix_g[b], s_hi = prefix_g[b + 1];
                if (s_hi > s_lo) {
                    c_lo = owner_of(s_lo, n_st, G);
                    c_hi = owner_of(s_hi - 1, n_st, G);
                    for (int c = c_lo; c <= c_hi; ++c)
                        if (owns_any(c, n_st, G)) M = fmaxf(M, part_ml[((size_t)(c + b) * d.n_q + g) * 2]);
                    float l = 0.f;
                    for (int c = c_lo; c <= c_hi; ++c) {
                        if (!owns_any(c, n_st, G)) continue;
                        const float* ml = part_ml + ((size_t)(c + b) * d.n_q + g) * 2;
                        l = fmaf(ml[1], ex2f(ml[0] - M), l);
                    }
                    inv_l = 1.f / l;
                }
            }
            mrg[tid * 4] = M; mrg[tid * 4 + 1] = inv_l;
            mrg[tid * 4 + 2] = __int_as_float(c_lo); mrg[tid * 4 + 3] = __int_as_float(c_hi);
        }
        __syncthreads();
        // ---- merged latent slice o_s[l][bb] and hidden-state slice x_s[h][bb]
        {
            const int bb = tid >> 3, l8 = tid & 7;
            const float M = mrg[bb * 4], inv_l = mrg[bb * 4 + 1];
            const int c_lo = __float_as_int(mrg[bb * 4 + 2]), c_hi = __float_as_int(mrg[bb * 4 + 3]);
            const int b = b0 + bb;
            for (int l0 = 0; l0 < dl8; l0 += 8 * 4) {
                float sum[4] = {0.f, 0.f, 0.f, 0.f};
                for (int c = c_lo; c <= c_hi; ++c) {
                    if (!owns_any(c, n_st, G)) continue;
                    const size_t pi = (size_t)(c + b) * d.n_q + g;
                    const float w = ex2f(part_ml[pi * 2] - M);
                    const float* po = part_o + pi * d.d_l + split * dl8 + l0 + l8;
#pragma unroll
                    for (int u = 0; u < 4; ++u) sum[u] = fmaf(po[u * 8], w, sum[u]);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) o_s[(l0 + l8 + u * 8) * kFinBlockB + bb] = sum[u] * inv_l;
            }
            for (int h = l8; h < h8; h += 8)
                x_s[h * kFinBlockB + bb] = bb < nb ? __bfloat162float(x_t[(size_t)b * d.H + split * h8 + h]) : 0.f;
        }
        __syncthreads();
        // ---- partial decoder and gate sums: one output column per thread, two K halves
        {
            const int e = tid & 127, kh = tid >> 7;
            float acc_y[kFinBlockB], acc_z[kFinBlockB];
#pragma unroll
            for (int bb = 0; bb < kFinBlockB; ++bb) { acc_y[bb] = 0.f; acc_z[bb] = 0.f; }
            {
                const int l_lo = kh * (dl8 / 2), l_hi = l_lo + dl8 / 2;
                const __nv_bfloat16* wp = w_p + ((size_t)i * d.d_l + split * dl8) * 128 + e;
#pragma unroll 4
                for (int l = l_lo; l < l_hi; ++l) {
                    const float w = __bfloat162float(wp[(size_t)l * 128]);
                    const float4* ov = reinterpret_cast<const float4*>(o_s + l * kFinBlockB);
#pragma unroll
                    for (int b4 = 0; b4 < kFinBlockB / 4; ++b4) {
                        const float4 o4 = ov[b4];
                        acc_y[4 * b4] = fmaf(o4.x, w, acc_y[4 * b4]);
                        acc_y[4 * b4 + 1] = fmaf(o4.y, w, acc_y[4 * b4 + 1]);
                        acc_y[4 * b4 + 2] = fmaf(o4.z, w, acc_y[4 * b4 + 2]);
                        acc_y[4 * b4 + 3] = fmaf(o4.w, w, acc_y[4 * b4 + 3]);
                    }
                }
            }
            {
                const int h_lo = kh * (h8 / 2), h_hi = (kh == 0) ? h8 / 2 : h8;
                const __nv_bfloat16* wg = w_g + (size_t)(split * h8) * n_cols + i * 128 + e;
#pragma unroll 4
                for (int h = h_lo; h < h_hi; ++h) {
                    const float w = __bfloat162float(wg[(size_t)h * n_cols]);
                    const float4* xv = reinterpret_cast<const float4*>(x_s + h * kFinBlockB);
#pragma unroll
                    for (int b4 = 0; b4 < kFinBlockB / 4; ++b4) {
                        const float4 x4 = xv[b4];
                        acc_z[4 * b4] = fmaf(x4.x, w, acc_z[4 * b4]);
                        acc_z[4 * b4 + 1] = fmaf(x4.y, w, acc_z[4 * b4 + 1]);
                        acc_z[4 * b4 + 2] = fmaf(x4.z, w, acc_z[4 * b4 + 2]);
                        acc_z[4 * b4 + 3] = fmaf(x4.w, w, acc_z[4 * b4 + 3]);
                    }
                }
            }
            if (kh == 1) {
#pragma unroll
                for (int bb = 0; bb < kFinBlockB; ++bb) {
                    part_s[bb * 128 + e] = acc_y[bb];
                    part_s[(kFinBlockB + bb) * 128 + e] = acc_z[bb];
                }
            }
            __syncthreads();
            if (kh == 0) {
#pragma unroll
                for (int bb = 0; bb < kFinBlockB; ++bb) {
                    part_s[bb * 128 + e] += acc_y[bb];
                    part_s[(kFinBlockB + bb) * 128 + e] += acc_z[bb];
                }
            }
        }
        cluster.sync();
        // ---- cluster reduction: rank r finishes sequences [4 r, 4 r + 4) of this block
        for (int idx = tid; idx < (kFinBlockB / kFinSplit) * 128; idx += kFinThreads) {
            const int bb = split * (kFinBlockB / kFinSplit) + idx / 128, e = idx % 128;
            float y = 0.f, z = 0.f;
#pragma unroll
            for (int rk = 0; rk < kFinSplit; ++rk) {
                const float* remote = cluster.map_shared_rank(part_s, rk);
                y += remote[bb * 128 + e];
                z += remote[(kFinBlockB + bb) * 128 + e];
            }
            if (bb < nb) {
                const float gate = __fdividef(1.f, 1.f + __expf(-z));
                out[((size_t)(b0 + bb) * d.n_h + i) * 128 + e] = __float2bfloat16_rn(y * gate);
            }
        }
        cluster.sync();   // the partial sums may be overwritten (next block) or the CTA may exit
    }
}

// ---------------------------------------------------------------------------------------------
cudaError_t launch_decode_fast(const Dims& d, const void* q, const void* k_cache, const void* c_cache,
                               const int32_t* seq_lens, int S_cap, const void* x_t, const void* w_p,
                               const void* w_g, void* out, void* workspace, int32_t* status_word,
                               cudaStream_t stream, int stages, int* launches) {
    const FastPlan p = make_fast_plan(d);
    float* part_o = reinterpret_cast<float*>(workspace);
    float* part_ml = reinterpret_cast<float*>(static_cast<char*>(workspace) + p.off_ml);
    int32_t* prefix_g = reinterpret_cast<int32_t*>(static_cast<char*>(workspace) + p.off_prefix);
    cudaError_t err;
    if (stages & 2) {
        const size_t smem = (size_t)kStreamStages * kStreamStageBytes +
                            (size_t)(d.n_q * 128 + 4 * kStreamMaxTS * d.n_q + 2 * d.n_q + 1024) * sizeof(float) +
                            (size_t)(kStreamMaxBatch + 2) * sizeof(int32_t) + 8 +
                            2 * kStreamStages * sizeof(uint64_t) + 16;
#define GTA_LAUNCH_STREAM(NQ)                                                                              \
        do {                                                                                               \
            auto kern = decode_stream_kernel<NQ>;                                                          \
            err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);      \
            if (err != cudaSuccess) return err;                                                            \
            kern<<<p.G, kStreamThreads, smem, stream>>>(d, p.TS, S_cap, (const __nv_bfloat16*)q,           \
                                                        (const __nv_bfloat16*)k_cache,                     \
                                                        (const __nv_bfloat16*)c_cache, seq_lens, part_o,   \
                                                        part_ml, prefix_g, status_word);                   \
        } while (0)
        switch (d.n_q) {
            case 1: GTA_LAUNCH_STREAM(1); break;
            case 2: GTA_LAUNCH_STREAM(2); break;
            case 4: GTA_LAUNCH_STREAM(4); break;
            default: GTA_LAUNCH_STREAM(8); break;
        }
#undef GTA_LAUNCH_STREAM
        if ((err = cudaGetLastError()) != cudaSuccess) return err;
        *launches += 1;
    }
    if (stages & 4) {
        const size_t smem = ((size_t)(d.d_l / kFinSplit + d.H / kFinSplit) * kFinBlockB + 2 * kFinBlockB * 128 +
                             kFinBlockB * 4) * sizeof(float);
        err = cudaFuncSetAttribute(decode_finish_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return err;
        dim3 grid(kFinSplit, d.n_h);
        decode_finish_cluster_kernel<<<grid, kFinThreads, smem, stream>>>(
            d, p.G, p.TS, S_cap, seq_lens, prefix_g, part_o, part_ml, (const __nv_bfloat16*)x_t,
            (const __nv_bfloat16*)w_p, (const __nv_bfloat16*)w_g, (__nv_bfloat16*)out);
        if ((err = cudaGetLastError()) != cudaSuccess) return err;
        *launches += 1;
    }
    return cudaSuccess;
}

}  // namespace gta
