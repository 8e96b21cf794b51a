// Bandwidth-oriented decode for bf16 caches (App. B.1.3), d_h = 128, one latent group.
//
//   decode_stream_kernel : persistent, one CTA per SM.  The live tokens of all sequences are cut
//       into sub-tiles of T tokens; CTA c owns the contiguous sub-tile range [c n / G, (c+1) n / G),
//       so every CTA streams the same number of cache bytes whatever the length mix.  A producer
//       warp brings each sub-tile (the K rows of every key group and the latent rows) into a
//       3-stage shared-memory ring with TMA tensor loads (128-byte swizzle, evict-first in L2).
//       Eight consumer warps compute, per sub-tile, the scores of all maps and the latent sums
//       with warp-level m16n8k16 MMAs whose M rows are the attention maps (1 .. 8 valid rows of
//       16): the cache data never passes through the ALUs element by element, which keeps the
//       kernel on the HBM roofline instead of the issue-slot limit.  Scores go through a small
//       shared buffer so that every warp can build the probability fragments for its own
//       d_l / 8 slice of the latent sum; one CTA barrier per sub-tile.  When the range crosses
//       into the next sequence, and at its end, the partial (max, sum, latent sum) goes to
//       slot c + b of the workspace.
//   decode_merge_kernel (batches of more than 16): log-sum-exp merge of the slots into L (bf16);
//       the tcgen05 decoder + gate kernel of the prefill path then runs with the batch as its token axis.
//   decode_finish_kernel (small batches): clusters of 4 or 8 CTAs per (head, 64-column half) split the reduction
//       dimensions of the decoder (d_l) and of the gate (H).  Launched with programmatic stream
//       serialisation: while the stream kernel drains, each CTA requests its weight slice (TMA)
//       and its hidden-state slice and works out which stream CTAs own which sequence; after the
//       dependency wait it merges, for 32 sequences at a time, the slots of its d_l slice
//       (log-sum-exp), multiplies by W_P,i and W_G,i with warp-level MMAs, and the cluster adds the
//       partial results through distributed shared memory before the sigmoid gate is applied.
#include <cooperative_groups.h>

#include "gta_common.cuh"
#include "gta_sm100.cuh"
#include "sm100_ptx.cuh"
#include "tma_host.cuh"

namespace cg = cooperative_groups;

namespace gta {

constexpr int kStreamConsumers = 256;
constexpr int kStreamThreads = kStreamConsumers + 32;
constexpr int kStreamStages = 3;
constexpr int kStreamStageBytes = 65536;
constexpr int kStreamMaxBatch = 512;
constexpr int kStreamMaxT = 128;     // tokens per sub-tile: at most 64, or 128 for the narrowest caches (d_l = 128)
constexpr int kFinBlockB = 32;
constexpr int kFinThreads = 256;
constexpr int kFinCols = 64;
constexpr int kFinMaxSlots = 1024;  // >= stream CTAs + batch

struct FastPlan {
    int T;         // tokens per sub-tile (16, 32 or 64)
    int G;         // stream CTAs
    int slots;     // G + B partial slots
    size_t off_ml, off_l, total;   // byte offsets in the workspace (part_o at 0)
};
constexpr int kFinMaxBatchClusters = 16;   // larger batches finish through the merge kernel + the tcgen05 decoder kernel
                                           // (measured: faster from 32 sequences on; the weights then feed 128-row MMAs)

static size_t align256f(size_t v) { return (v + 255) & ~(size_t)255; }
static int finish_split(const Dims& d);

bool decode_fast_supported(const Dims& d, int dtype) {
    if (dtype != GTA_BF16 || (d.d_h != 128 && d.d_h != 64)) return false;
    if (d.d_l != 128 && d.d_l != 256 && d.d_l != 512 && d.d_l != 1024) return false;
    if (d.n_q < 1 || d.n_q > 8) return false;                    // the maps are the rows of the warp-level MMAs
    if (d.n_k != 1 && d.n_k != 2 && d.n_k != 4 && d.n_k != 8) return false;   // key groups are dealt to the 8 warps
    if (d.H % 64 != 0 || d.B > kStreamMaxBatch) return false;
    // the finish: clusters (small batches; written for d_h = 128, power-of-two map counts, d_l >= 256), else the
    // merge kernel + the tcgen05 decoder kernel, which cuts the output columns in blocks inside one attention map
    const bool clusters = d.B <= kFinMaxBatchClusters && d.d_h == 128 && d.d_l >= 256 && (d.n_q & (d.n_q - 1)) == 0 &&
                          d.n_c == 1;
    if (clusters && finish_split(d) == 0) return false;
    if (!clusters && ((d.n_h / d.n_q) * d.d_h) % (d.B > 128 ? 128 : 64) != 0) return false;
    const int tok_bytes = (d.n_k * d.d_h + d.n_c * d.d_l) * 2;
    return tok_bytes * 16 <= kStreamStageBytes;
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
    const int tok_bytes = (d.n_k * d.d_h + d.n_c * d.d_l) * 2;
    int t = 16;
    const int t_max = d.d_l == 128 ? 128 : 64;       // matches the KTM of the stream kernel's instantiation
    while (t * 2 * tok_bytes <= kStreamStageBytes && t * 2 <= t_max) t *= 2;
    p.T = t;
    p.G = sm_count() < kFinMaxSlots - kStreamMaxBatch ? sm_count() : kFinMaxSlots - kStreamMaxBatch;
    p.slots = p.G + d.B;
    const size_t part_o = (size_t)p.slots * d.n_q * d.d_l * sizeof(float);
    const size_t part_ml = (size_t)p.slots * d.n_q * 2 * sizeof(float);
    p.off_ml = align256f(part_o);
    p.off_l = p.off_ml + align256f(part_ml);
    p.total = p.off_l + align256f((size_t)d.n_q * d.B * d.d_l * sizeof(__nv_bfloat16));
    return p;
}

size_t decode_fast_workspace_bytes(const Dims& d) { return make_fast_plan(d).total; }

// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ int clamp_len(int len, int S_cap) { return len < 0 ? 0 : (len > S_cap ? S_cap : len); }

// Shared-memory layout of one ring stage (all tiles are [T rows][64 bf16] = T x 128 bytes with
// the 128-byte TMA swizzle: the 16-byte chunk c of row r sits at chunk c ^ (r & 7)):
//   K tiles : key group kg, half h (columns 64 h .. 64 h + 63)  at (KH kg + h) T 128
//   C tiles : latent group cg, columns 64 j .. 64 j + 63         at c_off + (NT cg + j) T 128
// NT = d_l / 64 = MMA n-tiles (8 latent columns each) per consumer warp; KH = d_h / 64 = 64-column
// tiles per key row; KTM = most 16-token MMA k-steps per sub-tile (sub-tiles of up to 16 KTM tokens:
// the narrower a cached token, the more tokens a sub-tile needs to be worth its fixed cost)
// ONE_C: a single latent group (the latent-sum loop then has no group pass and no masking)
template <int NT, int KH, int KTM, bool ONE_C>
__global__ void __launch_bounds__(kStreamThreads, 1)
decode_stream_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_c, Dims d,
                     int T, int S_cap, const __nv_bfloat16* __restrict__ q, const int32_t* __restrict__ seq_lens,
                     float* __restrict__ part_o, float* __restrict__ part_ml, int32_t* status_word) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* ring = smem;                                                              // 3 x 64 KB
    float* s_buf = reinterpret_cast<float*>(smem + kStreamStages * kStreamStageBytes);   // [2][n_q][T]
    int32_t* prefix = reinterpret_cast<int32_t*>(s_buf + 2 * 8 * kStreamMaxT);           // [B + 1]
    int32_t* scan_tmp = prefix + kStreamMaxBatch + 2;                                    // [kStreamThreads]
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(scan_tmp + kStreamThreads);
    uint64_t* empty_bar = full_bar + kStreamStages;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(empty_bar + kStreamStages);
    volatile int* drain_flag = abort_flag + 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int G = gridDim.x, cta = blockIdx.x;
    const int NQ = d.n_q;
    if (tid == kStreamConsumers) {   // the descriptors are on their way while the prefix sum runs
        ptx::prefetch_tensormap(&tm_k);
        ptx::prefetch_tensormap(&tm_c);
    }

    // This kernel is itself launched with programmatic stream serialisation: it may have been
    // scheduled while the kernel before it in the stream (a cache append, the previous decode
    // step) was still draining, and must not read that kernel's results (lengths, caches) earlier.
    ptx::grid_dependency_wait();
    // Only now may the kernels after this one be scheduled: they read inputs (sequence lengths,
    // hidden states, weights) before their own dependency wait, which orders them against this
    // kernel alone -- whatever ran before this kernel is complete and visible from here on.
    ptx::grid_launch_dependents();

    // ---- exclusive prefix sum of the sub-tile counts: prefix[b] = sum_{b' < b} ceil(len / T)
    //      (thread t owns sequences [t per, (t + 1) per); warp scan, then a scan of the warp totals)
    {
        const int per = (d.B + kStreamThreads - 1) / kStreamThreads;
        const int lo = min(tid * per, d.B), hi = min(lo + per, d.B);
        int sum = 0;
        for (int b = lo; b < hi; ++b) sum += (clamp_len(seq_lens[b], S_cap) + T - 1) / T;
        int incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) scan_tmp[warp] = incl;
        if (tid == 0) {
            for (int s = 0; s < kStreamStages; ++s) { ptx::mbar_init(&full_bar[s], 1); ptx::mbar_init(&empty_bar[s], 8); }
            *abort_flag = 0;
            *drain_flag = 0;
            ptx::fence_mbar_init();
        }
        __syncthreads();
        int base = incl - sum;
        for (int w = 0; w < warp; ++w) base += scan_tmp[w];
        for (int b = lo; b < hi; ++b) {
            prefix[b] = base;
            base += (clamp_len(seq_lens[b], S_cap) + T - 1) / T;
        }
        if (tid == kStreamThreads - 1) prefix[d.B] = base;
        __syncthreads();
    }
    const long long n_st = prefix[d.B];
    const long long st_begin = ((long long)cta * n_st) / G, st_end = ((long long)(cta + 1) * n_st) / G;
    if (st_begin >= st_end) return;      // uniform: nothing armed
    int b0;
    {   // largest b with prefix[b] <= st_begin: a non-empty sequence, since st_begin < n_st
        int lo = 0, hi = d.B - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (prefix[mid] <= st_begin) lo = mid; else hi = mid - 1;
        }
        b0 = lo;
    }
    const uint32_t tile_bytes = (uint32_t)T * 128;
    const uint32_t c_off = (uint32_t)d.n_k * KH * tile_bytes;
    const int n_c_tiles = ONE_C ? NT : d.n_c * NT;
    const uint32_t stage_tx = c_off + (uint32_t)n_c_tiles * tile_bytes;

    if (warp == kStreamConsumers / 32) {
        // ------------------------------------------------------------------ producer
        // Lane 0 waits for the stage and arms its barrier; then every lane issues one of the (up
        // to 32) tensor loads of the sub-tile, so that issuing them does not pace the stream.
        {
            const uint64_t policy = ptx::l2_evict_first_policy();
            const int n_k_ops = KH * d.n_k;
            int b = b0;
            long long k = st_begin - prefix[b0];
            int it = 0;
            bool ok = true;
            for (long long st = st_begin; st < st_end; ++st, ++it, ++k) {
                while (k >= prefix[b + 1] - prefix[b]) { ++b; k = 0; }
                const int s = it % kStreamStages;
                const uint32_t ph = (it / kStreamStages) & 1;
                if (lane == 0) {
                    ok = ptx::mbar_wait(&empty_bar[s], ph ^ 1, abort_flag);
                    if (ok) ptx::mbar_arrive_expect_tx(&full_bar[s], stage_tx);
                }
                ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                if (!ok) break;
                const int tok0 = (int)k * T;
                uint8_t* stage = ring + s * kStreamStageBytes;
                for (int op = lane; op < n_k_ops + n_c_tiles; op += 32) {
                    if (op < n_k_ops)
                        ptx::tma_load_3d_hint(stage + op * tile_bytes, &tm_k, &full_bar[s], (op % KH) * 64, tok0,
                                              b * d.n_k + op / KH, policy);
                    else
                        ptx::tma_load_3d_hint(stage + c_off + (op - n_k_ops) * tile_bytes, &tm_c, &full_bar[s],
                                              ((op - n_k_ops) % NT) * 64, tok0, b * d.n_c + (op - n_k_ops) / NT, policy);
                }
            }
            if (lane == 0 && *abort_flag) {
                for (int back = 1; back <= kStreamStages && it - back >= 0; ++back) {
                    const int iq = it - back;
                    ptx::mbar_wait(&full_bar[iq % kStreamStages], (iq / kStreamStages) & 1, drain_flag);
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ consumers
        const int quad = lane >> 2, sub = lane & 3;       // MMA fragment coordinates
        const int mat = lane >> 3, mrow = lane & 7;       // ldmatrix: which 8x8 matrix, which row of it
        const int qpk = NQ / d.n_k;                       // maps per key group
        const int kg_w = warp % d.n_k;                    // this warp scores key group kg_w (n_k divides 8)
        const int KT = T >> 4;                            // 16-token MMA k-steps per sub-tile
        const int n_units = (T >> 3) * d.n_k;             // (8-token n-tile, key group) scoring units
        const float c_scale = d.scale * 1.4426950408889634f;
        const uint32_t ring_addr = ptx::smem_addr(ring);
        const bool map_lane = quad < NQ;                  // this lane carries softmax state of map `quad`
        float m_run = -INFINITY, l_run = 0.f;
        float acc[NT][4];
#pragma unroll
        for (int n = 0; n < NT; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
        uint32_t qa[4 * KH][2];                           // A fragments of Q for key group kg_w

        auto load_q = [&](int b) {
            const uint32_t* qrow =
                reinterpret_cast<const uint32_t*>(q + ((size_t)b * NQ + kg_w * qpk + (quad < qpk ? quad : 0)) * (64 * KH));
#pragma unroll
            for (int ks = 0; ks < 4 * KH; ++ks) {
                qa[ks][0] = quad < qpk ? __ldg(qrow + 8 * ks + sub) : 0u;
                qa[ks][1] = quad < qpk ? __ldg(qrow + 8 * ks + 4 + sub) : 0u;
            }
        };
        auto flush = [&](int b) {
            const int slot = cta + b;
            if (map_lane) {
                float* o = part_o + ((size_t)slot * NQ + quad) * d.d_l + warp * (NT * 8) + 2 * sub;
#pragma unroll
                for (int n = 0; n < NT; ++n) *reinterpret_cast<float2*>(o + 8 * n) = make_float2(acc[n][0], acc[n][1]);
                if (warp == 0 && sub == 0) {
                    part_ml[((size_t)slot * NQ + quad) * 2] = m_run;
                    part_ml[((size_t)slot * NQ + quad) * 2 + 1] = l_run;
                }
            }
#pragma unroll
            for (int n = 0; n < NT; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
            m_run = -INFINITY;
            l_run = 0.f;
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
            const int n_valid = min(T, len - (int)k * T);
            const uint32_t stage = ring_addr + s * kStreamStageBytes;
            float* sb = s_buf + (it & 1) * (NQ * T);

            // ---- scores of the maps of key group kg_w, 8 tokens per unit: S = Q K^T
            for (int u = warp; u < n_units; u += 8) {
                const int nt = u / d.n_k;
                const int token = nt * 8 + mrow;
                const uint32_t krow = stage + (uint32_t)(KH * kg_w) * tile_bytes + token * 128;
                float sc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int kp = 0; kp < 2 * KH; ++kp) {
                    const int chunk = 4 * kp + mat;     // 16-byte chunk of the K row (128 KH bytes)
                    uint32_t k0, k1, k2, k3;
                    ptx::ldsm_x4(krow + (chunk >> 3) * tile_bytes + (((chunk & 7) ^ (token & 7)) << 4), k0, k1, k2, k3);
                    ptx::mma_bf16_16816(sc, qa[2 * kp][0], 0u, qa[2 * kp][1], 0u, k0, k1);
                    ptx::mma_bf16_16816(sc, qa[2 * kp + 1][0], 0u, qa[2 * kp + 1][1], 0u, k2, k3);
                }
                if (quad < qpk) {
                    const int t0 = nt * 8 + 2 * sub;
                    float2 v;
                    v.x = t0 < n_valid ? sc[0] * c_scale : -INFINITY;
                    v.y = t0 + 1 < n_valid ? sc[1] * c_scale : -INFINITY;
                    *reinterpret_cast<float2*>(sb + (kg_w * qpk + quad) * T + t0) = v;
                }
            }
            // ---- rows past the live length hold whatever the cache holds there: their
            //      probabilities are zero, so the latent rows are cleared (0 x garbage could be NaN)
            if (n_valid < T) {
                const int vec_per_row = n_c_tiles * 8;   // 16-byte vectors per token over all latent groups
                const int n_vec = (T - n_valid) * vec_per_row;
                for (int idx = tid; idx < n_vec; idx += kStreamConsumers) {
                    const int row = n_valid + idx / vec_per_row, v = idx % vec_per_row;   // v >> 3 = tile (group, 64 columns)
                    uint8_t* p = ring + s * kStreamStageBytes + c_off + (v >> 3) * tile_bytes + row * 128 + (v & 7) * 16;
                    *reinterpret_cast<uint4*>(p) = make_uint4(0u, 0u, 0u, 0u);
                }
                ptx::fence_proxy_async_smem();   // the next TMA write of this stage follows generic writes
            }
            consumer_sync();

            // ---- softmax state of map `quad` (every warp keeps its own copy) and the probability
            //      fragments: lane (quad, sub) holds tokens 16 kt + 2 sub + {0, 1, 8, 9}
            uint32_t pa[KTM][2];
            float alpha = 1.f;
            {
                float sv[KTM][4];
                float m_t = -INFINITY;
#pragma unroll
                for (int kt = 0; kt < KTM; ++kt) {
                    if (kt < KT && map_lane) {
                        const float2 x = *reinterpret_cast<const float2*>(sb + quad * T + 16 * kt + 2 * sub);
                        const float2 y = *reinterpret_cast<const float2*>(sb + quad * T + 16 * kt + 8 + 2 * sub);
                        sv[kt][0] = x.x; sv[kt][1] = x.y; sv[kt][2] = y.x; sv[kt][3] = y.y;
                    } else {
                        sv[kt][0] = sv[kt][1] = sv[kt][2] = sv[kt][3] = -INFINITY;
                    }
                    m_t = fmaxf(fmaxf(m_t, fmaxf(sv[kt][0], sv[kt][1])), fmaxf(sv[kt][2], sv[kt][3]));
                }
                m_t = fmaxf(m_t, __shfl_xor_sync(0xffffffffu, m_t, 1));
                m_t = fmaxf(m_t, __shfl_xor_sync(0xffffffffu, m_t, 2));
                const float m_new = fmaxf(m_run, m_t);     // finite on map lanes: token 0 of a tile is live
                const float m_sub = map_lane ? m_new : 0.f;
                alpha = map_lane ? ex2f(m_run - m_new) : 1.f;
                float sum = 0.f;
#pragma unroll
                for (int kt = 0; kt < KTM; ++kt) {
                    const float p0 = ex2f(sv[kt][0] - m_sub), p1 = ex2f(sv[kt][1] - m_sub);
                    const float p2 = ex2f(sv[kt][2] - m_sub), p3 = ex2f(sv[kt][3] - m_sub);
                    sum += (p0 + p1) + (p2 + p3);
                    pa[kt][0] = pack_bf16(p0, p1);
                    pa[kt][1] = pack_bf16(p2, p3);
                }
                sum += __shfl_xor_sync(0xffffffffu, sum, 1);
                sum += __shfl_xor_sync(0xffffffffu, sum, 2);
                l_run = l_run * alpha + sum;
                m_run = m_new;
            }
#pragma unroll
            for (int n = 0; n < NT; ++n) { acc[n][0] *= alpha; acc[n][1] *= alpha; }

            // ---- latent sums of this warp's d_l / 8 columns, all maps at once: O += P C.  With several
            //      latent groups, one pass per group with the probabilities of the other groups' maps
            //      zeroed (a lane's fragment registers belong to its own map's row).
            const int n_c_loop = ONE_C ? 1 : d.n_c;
            for (int cg = 0; cg < n_c_loop; ++cg) {
                const uint32_t cbase = stage + c_off + (uint32_t)(cg * NT) * tile_bytes;
                const bool mine = ONE_C || d.q_to_c(quad < NQ ? quad : 0) == cg;
#pragma unroll
                for (int kt = 0; kt < KTM; ++kt) {
                    if (kt < KT) {
                        const uint32_t a0 = mine ? pa[kt][0] : 0u, a2 = mine ? pa[kt][1] : 0u;
                        const int token = 16 * kt + (mat & 1) * 8 + mrow;
                        const uint32_t crow = cbase + token * 128;
#pragma unroll
                        for (int np = 0; np < NT / 2; ++np) {
                            const int chunk = warp * NT + 2 * np + (mat >> 1);   // 16-byte chunk of the latent row
                            uint32_t c0, c1, c2, c3;
                            ptx::ldsm_x4_trans(crow + (chunk >> 3) * tile_bytes + (((chunk & 7) ^ (token & 7)) << 4),
                                               c0, c1, c2, c3);
                            ptx::mma_bf16_16816(acc[2 * np], a0, 0u, a2, 0u, c0, c1);
                            ptx::mma_bf16_16816(acc[2 * np + 1], a0, 0u, a2, 0u, c2, c3);
                        }
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
// One CTA = one head, 64 of its 128 output columns, 1 / S of the reduction dimensions (S = cluster
// size, 4 or 8).  Dynamic shared memory:
//   w_s [(d_l + H) / S rows][64 bf16] (swizzled weight slice: W_P rows first) |
//   a_s [32][KA + 8 bf16] (merged latent slice, then hidden-state slice, per sequence) |
//   part_s [2][32][64] fp32 (partial decoder / gate sums) | ml_s, w_all [slots] | prefix_s, rng_s [B] |
//   bound_s [G + 1] | scan scratch | barrier
struct FinSmem {
    uint32_t a_off, part_off, ml_off, w_all_off, prefix_off, rng_off, bound_off, scan_off, bar_off, total;
};
__host__ __device__ inline FinSmem fin_smem_layout(int KA) {
    FinSmem L;
    L.a_off = (uint32_t)KA * 128u;
    L.part_off = L.a_off + (uint32_t)kFinBlockB * (KA + 8) * 2;
    L.ml_off = L.part_off + 2u * kFinBlockB * kFinCols * 4;
    L.w_all_off = L.ml_off + kFinMaxSlots * 8;
    L.prefix_off = L.w_all_off + kFinMaxSlots * 4;
    L.rng_off = L.prefix_off + (kStreamMaxBatch + 2) * 4;
    L.bound_off = L.rng_off + 2 * kStreamMaxBatch * 4;
    L.scan_off = L.bound_off + (kFinMaxSlots - kStreamMaxBatch + 2) * 4;
    L.bar_off = L.scan_off + 8 * 4;
    L.total = L.bar_off + 16 + 1024;   // + slack to align the base to 1024 bytes
    return L;
}

__device__ __forceinline__ void cp_async_16(void* dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ptx::smem_addr(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// Merge of the split-KV partial latent sums of one block of 32 sequences into a_s (bf16).  A
// thread owns one 4-column chunk of its CTA's d_l slice for SQ sequences (SQ x dls / 4 = 256
// threads x ... : dls = 64, 128, 256 -> SQ = 2, 4, 8).  Loads go out in rounds of up to kFinRound
// slots per sequence, all of a round in flight at once.
struct FinMergeArgs {
    const float* part_o; const float* w_all;
    const int32_t* rng_s;    // [B][2] first / last stream CTA that owns sub-tiles of the sequence
    __nv_bfloat16* a_s;
    int n_q, d_l, g, col_base, dls, a_stride, b0, nb, tid;
};
constexpr int kFinMaxSQ = 8;
struct FinMergeRegs { float4 v[32]; };

template <int SQ>
__device__ __forceinline__ void fin_merge_load(const FinMergeArgs& a, FinMergeRegs& r, int j0) {
    constexpr int kRound = 32 / SQ;              // slots per sequence and round
    const int tps = a.dls / 4;                   // threads per sequence
    const int chunk = a.tid % tps, bgrp = a.tid / tps, nbg = kFinThreads / tps;
#pragma unroll
    for (int sq = 0; sq < SQ; ++sq) {
        const int bb = bgrp + sq * nbg, b = a.b0 + bb;
        const int c_lo = bb < a.nb ? a.rng_s[2 * b] : 0, c_hi = bb < a.nb ? a.rng_s[2 * b + 1] : -1;
#pragma unroll
        for (int j = 0; j < kRound; ++j) {
            const int c = c_lo + j0 + j;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (c <= c_hi)
                v = *reinterpret_cast<const float4*>(a.part_o + ((size_t)(c + b) * a.n_q + a.g) * a.d_l + a.col_base + 4 * chunk);
            r.v[sq * kRound + j] = v;
        }
    }
}

template <int SQ>
__device__ __forceinline__ void fin_merge_finish(const FinMergeArgs& a, FinMergeRegs& r) {
    constexpr int kRound = 32 / SQ;
    const int tps = a.dls / 4;
    const int chunk = a.tid % tps, bgrp = a.tid / tps, nbg = kFinThreads / tps;
    float4 sum[SQ];
#pragma unroll
    for (int sq = 0; sq < SQ; ++sq) sum[sq] = make_float4(0.f, 0.f, 0.f, 0.f);
    int n_max = 0;
#pragma unroll
    for (int sq = 0; sq < SQ; ++sq) {
        const int bb = bgrp + sq * nbg, b = a.b0 + bb;
        if (bb < a.nb) n_max = max(n_max, a.rng_s[2 * b + 1] - a.rng_s[2 * b] + 1);
    }
    for (int j0 = 0;; j0 += kRound) {
#pragma unroll
        for (int sq = 0; sq < SQ; ++sq) {
            const int bb = bgrp + sq * nbg, b = a.b0 + bb;
            const int c_lo = bb < a.nb ? a.rng_s[2 * b] : 0, c_hi = bb < a.nb ? a.rng_s[2 * b + 1] : -1;
#pragma unroll
            for (int j = 0; j < kRound; ++j) {
                const int c = c_lo + j0 + j;
                if (c <= c_hi) {
                    const float w = a.w_all[c + b];   // 0 for a CTA that owns nothing: its slot holds stale bits
                    if (w != 0.f) {
                        const float4 v = r.v[sq * kRound + j];
                        sum[sq].x = fmaf(v.x, w, sum[sq].x); sum[sq].y = fmaf(v.y, w, sum[sq].y);
                        sum[sq].z = fmaf(v.z, w, sum[sq].z); sum[sq].w = fmaf(v.w, w, sum[sq].w);
                    }
                }
            }
        }
        if (j0 + kRound >= n_max) break;
        fin_merge_load<SQ>(a, r, j0 + kRound);   // sequences that span more CTAs than one round covers
    }
#pragma unroll
    for (int sq = 0; sq < SQ; ++sq) {
        const int bb = bgrp + sq * nbg;
        uint2 packed;
        packed.x = pack_bf16(sum[sq].x, sum[sq].y);
        packed.y = pack_bf16(sum[sq].z, sum[sq].w);
        *reinterpret_cast<uint2*>(a.a_s + bb * a.a_stride + 4 * chunk) = packed;
    }
}

__global__ void __launch_bounds__(kFinThreads)
decode_finish_kernel(const __grid_constant__ CUtensorMap tm_wp, const __grid_constant__ CUtensorMap tm_wg, Dims d,
                     int G, int T, int S_cap, const int32_t* __restrict__ seq_lens,
                     const float* __restrict__ part_o, const float* __restrict__ part_ml,
                     const __nv_bfloat16* __restrict__ x_t, __nv_bfloat16* __restrict__ out, int32_t* status_word) {
    cg::cluster_group cluster = cg::this_cluster();
    const int S = (int)cluster.num_blocks();     // = gridDim.x
    extern __shared__ uint8_t fin_raw[];
    uint8_t* fsm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(fin_raw) + 1023) & ~(uintptr_t)1023);
    const int dls = d.d_l / S, hs = d.H / S;     // this CTA's slice of the latent and of the hidden dimension
    const int KA = dls + hs, a_stride = KA + 8;  // bf16 elements per a_s row (row = 16-byte multiple)
    const FinSmem L = fin_smem_layout(KA);
    uint8_t* w_s = fsm;
    __nv_bfloat16* a_s = reinterpret_cast<__nv_bfloat16*>(fsm + L.a_off);
    float* part_s = reinterpret_cast<float*>(fsm + L.part_off);
    float2* ml_s = reinterpret_cast<float2*>(fsm + L.ml_off);             // (max, sum) of map g per slot
    float* w_all = reinterpret_cast<float*>(fsm + L.w_all_off);           // merge weight per slot
    int32_t* prefix_s = reinterpret_cast<int32_t*>(fsm + L.prefix_off);   // [B + 1]
    int32_t* rng_s = reinterpret_cast<int32_t*>(fsm + L.rng_off);         // [B][2] first / last owning CTA
    int32_t* bound_s = reinterpret_cast<int32_t*>(fsm + L.bound_off);     // [G + 1] first sub-tile of CTA c
    int32_t* scan_s = reinterpret_cast<int32_t*>(fsm + L.scan_off);
    uint64_t* w_bar = reinterpret_cast<uint64_t*>(fsm + L.bar_off);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(w_bar + 1);

    const int split = blockIdx.x;                // = rank inside the cluster
    const int i = blockIdx.y >> 1;               // head
    const int col0 = (blockIdx.y & 1) * kFinCols;   // first of this CTA's output columns inside the head
    const int g = d.head_to_q(i);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int quad = lane >> 2, sub = lane & 3, mat = lane >> 3, mrow = lane & 7;

    // ---- weight slice: independent of the stream kernel's results, so it is requested first
    if (tid == 0) {
        ptx::mbar_init(w_bar, 1);
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::mbar_arrive_expect_tx(w_bar, (uint32_t)KA * 128);
        ptx::tma_load_3d(w_s, &tm_wp, w_bar, col0, split * dls, i);
        for (int r0 = 0; r0 < hs; r0 += 256)
            ptx::tma_load_2d(w_s + (size_t)(dls + r0) * 128, &tm_wg, w_bar, i * 128 + col0, split * hs + r0);
    }
    // ---- also independent of it: the hidden-state slice of a block of sequences (asynchronous copies)
    auto load_x = [&](int b0, int nb) {
        const int xv = hs / 8;                      // 16-byte vectors per sequence
        for (int idx = tid; idx < kFinBlockB * xv; idx += kFinThreads) {
            const int xb = idx / xv, v = idx % xv;
            __nv_bfloat16* dst = a_s + xb * a_stride + dls + v * 8;
            if (xb < nb) cp_async_16(dst, x_t + (size_t)(b0 + xb) * d.H + split * hs + v * 8);
            else *reinterpret_cast<uint4*>(dst) = make_uint4(0u, 0u, 0u, 0u);
        }
    };
    load_x(0, min(kFinBlockB, d.B));
    // ---- and which stream CTAs own sub-tiles of which sequence.  Same
    //      arithmetic as in the stream kernel: prefix sums of ceil(len / T), ranges c n / G.  This
    //      runs while the stream kernel drains (the launch is programmatically serialised).
    {
        const int per = (d.B + kFinThreads - 1) / kFinThreads;
        const int lo = min(tid * per, d.B), hi = min(lo + per, d.B);
        int sum = 0;
        for (int b = lo; b < hi; ++b) sum += (clamp_len(seq_lens[b], S_cap) + T - 1) / T;
        int incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) scan_s[warp] = incl;
        __syncthreads();
        int base = incl - sum;
        for (int w = 0; w < warp; ++w) base += scan_s[w];
        for (int b = lo; b < hi; ++b) {
            prefix_s[b] = base;
            base += (clamp_len(seq_lens[b], S_cap) + T - 1) / T;
        }
        if (tid == kFinThreads - 1) prefix_s[d.B] = base;
        __syncthreads();
        const long long n_st = prefix_s[d.B];
        for (int c = tid; c <= G; c += kFinThreads) bound_s[c] = (int32_t)(((long long)c * n_st) / G);
        // the owner of sub-tile st is the largest c with floor(c n / G) <= st = floor(((st + 1) G - 1) / n)
        for (int b = tid; b < d.B; b += kFinThreads) {
            const long long s_lo = prefix_s[b], s_hi = prefix_s[b + 1];
            int c_lo = 0, c_hi = -1;
            if (s_hi > s_lo) {
                c_lo = (int)(((s_lo + 1) * G - 1) / n_st);
                c_hi = (int)((s_hi * G - 1) / n_st);
            }
            rng_s[2 * b] = c_lo;
            rng_s[2 * b + 1] = c_hi;
        }
    }
    __syncthreads();
    ptx::grid_dependency_wait();   // everything below reads what the stream kernel wrote
    const uint32_t w_addr = ptx::smem_addr(w_s), a_addr = ptx::smem_addr(a_s);

    // ---- for this head's map, the (max, sum) pair of every slot (slots nobody wrote hold stale
    //      bits that are never used)
    const int n_slots = G + d.B;
    for (int j = tid; j < n_slots; j += kFinThreads)
        ml_s[j] = *reinterpret_cast<const float2*>(part_ml + ((size_t)j * d.n_q + g) * 2);

    for (int b0 = 0; b0 < d.B; b0 += kFinBlockB) {
        const int nb = min(kFinBlockB, d.B - b0);
        if (b0 > 0) load_x(b0, nb);   // (block 0: already requested before the dependency wait)
        // ---- merged latent slice (bf16): a thread owns one 4-column chunk of SQ sequences.  The
        //      first round of partial-result loads is issued before the merge weights exist (block 0
        //      computes them meanwhile), so their latency overlaps that work.
        const FinMergeArgs ma = {part_o, w_all, rng_s, a_s, d.n_q, d.d_l, g, split * dls, dls, a_stride, b0, nb, tid};
        FinMergeRegs mr;
        if (dls == 64) fin_merge_load<2>(ma, mr, 0);
        else if (dls == 128) fin_merge_load<4>(ma, mr, 0);
        else fin_merge_load<8>(ma, mr, 0);
        if (b0 == 0) {
            __syncthreads();   // the (max, sum) pairs are in shared memory
            // per sequence (eight lanes each): the normalised merge weight of each of its slots c + b:
            //      w = 2^(m_slot - M) / sum_slots l_slot 2^(m_slot - M)
            for (int b8 = 0; b8 < d.B; b8 += kFinThreads / 8) {
                const int b = b8 + (tid >> 3), l8 = tid & 7;
                const bool live = b < d.B;
                const int c_lo = live ? rng_s[2 * b] : 0, c_hi = live ? rng_s[2 * b + 1] : -1;
                float M = -INFINITY, l = 0.f;
                for (int c = c_lo + l8; c <= c_hi; c += 8)
                    if (bound_s[c] < bound_s[c + 1]) M = fmaxf(M, ml_s[c + b].x);
                M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, 1));
                M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, 2));
                M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, 4));
                for (int c = c_lo + l8; c <= c_hi; c += 8) {
                    float w = 0.f;
                    if (bound_s[c] < bound_s[c + 1]) {   // a CTA with an empty range wrote nothing
                        w = ex2f(ml_s[c + b].x - M);
                        l = fmaf(ml_s[c + b].y, w, l);
                    }
                    w_all[c + b] = w;
                }
                l += __shfl_xor_sync(0xffffffffu, l, 1);
                l += __shfl_xor_sync(0xffffffffu, l, 2);
                l += __shfl_xor_sync(0xffffffffu, l, 4);
                const float inv_l = 1.f / l;
                for (int c = c_lo + l8; c <= c_hi; c += 8) w_all[c + b] *= inv_l;
            }
            __syncthreads();
        }
        if (dls == 64) fin_merge_finish<2>(ma, mr);
        else if (dls == 128) fin_merge_finish<4>(ma, mr);
        else fin_merge_finish<8>(ma, mr);
        cp_async_wait_all();
        __syncthreads();
        if (b0 == 0) ptx::mbar_wait(w_bar, 0, abort_flag);   // on give-up the results are wrong and the status word says so
        // ---- partial sums: warp w owns output columns 8 w .. 8 w + 7; rows = the 32 sequences
        {
            // four accumulator sets per m-tile, used round-robin over the k-steps: the dependent
            // chain of MMAs is a quarter as long (the loop is latency-bound, not throughput-bound)
            float acc[2][4][4] = {};     // [y / z][set][fragment], m-tile 0
            float bcc[2][4][4] = {};     // same, m-tile 1
            const int a_row = (mat & 1) * 8 + mrow, a_col = (mat >> 1) * 8;
            const int n_ks = KA / 16, ks_y = dls / 16;
            for (int ks0 = 0; ks0 < n_ks; ks0 += 4) {
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int ks = ks0 + u;
                    if (ks >= n_ks) break;
                    const int yz = ks < ks_y ? 0 : 1;
                    const int krow = 16 * ks + (lane & 15);
                    uint32_t w0, w1;
                    ptx::ldsm_x2_trans(w_addr + krow * 128 + ((warp ^ (krow & 7)) << 4), w0, w1);
                    uint32_t a0, a1, a2, a3;
                    ptx::ldsm_x4(a_addr + (uint32_t)(a_row * a_stride + 16 * ks + a_col) * 2, a0, a1, a2, a3);
                    uint32_t e0, e1, e2, e3;
                    ptx::ldsm_x4(a_addr + (uint32_t)((16 + a_row) * a_stride + 16 * ks + a_col) * 2, e0, e1, e2, e3);
                    if (yz == 0) {
                        ptx::mma_bf16_16816(acc[0][u], a0, a1, a2, a3, w0, w1);
                        ptx::mma_bf16_16816(bcc[0][u], e0, e1, e2, e3, w0, w1);
                    } else {
                        ptx::mma_bf16_16816(acc[1][u], a0, a1, a2, a3, w0, w1);
                        ptx::mma_bf16_16816(bcc[1][u], e0, e1, e2, e3, w0, w1);
                    }
                }
            }
            float acc_y[2][4], acc_z[2][4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                acc_y[0][e] = (acc[0][0][e] + acc[0][1][e]) + (acc[0][2][e] + acc[0][3][e]);
                acc_y[1][e] = (bcc[0][0][e] + bcc[0][1][e]) + (bcc[0][2][e] + bcc[0][3][e]);
                acc_z[0][e] = (acc[1][0][e] + acc[1][1][e]) + (acc[1][2][e] + acc[1][3][e]);
                acc_z[1][e] = (bcc[1][0][e] + bcc[1][1][e]) + (bcc[1][2][e] + bcc[1][3][e]);
            }
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
                float* py = part_s + (mt * 16 + quad) * kFinCols + warp * 8 + 2 * sub;
                float* pz = py + kFinBlockB * kFinCols;
                *reinterpret_cast<float2*>(py) = make_float2(acc_y[mt][0], acc_y[mt][1]);
                *reinterpret_cast<float2*>(py + 8 * kFinCols) = make_float2(acc_y[mt][2], acc_y[mt][3]);
                *reinterpret_cast<float2*>(pz) = make_float2(acc_z[mt][0], acc_z[mt][1]);
                *reinterpret_cast<float2*>(pz + 8 * kFinCols) = make_float2(acc_z[mt][2], acc_z[mt][3]);
            }
        }
        cluster.sync();
        // ---- cluster reduction: rank r finishes sequences [r 32 / S, (r + 1) 32 / S) of this block
        const int rows_per_rank = kFinBlockB / S;
        for (int idx = tid; idx < rows_per_rank * kFinCols; idx += kFinThreads) {
            const int bb = split * rows_per_rank + idx / kFinCols, e = idx % kFinCols;
            float yv[8], zv[8];
#pragma unroll
            for (int rk = 0; rk < 8; ++rk) {      // all remote loads in flight together
                yv[rk] = zv[rk] = 0.f;
                if (rk < S) {
                    const float* remote = cluster.map_shared_rank(part_s, rk);
                    yv[rk] = remote[bb * kFinCols + e];
                    zv[rk] = remote[(kFinBlockB + bb) * kFinCols + e];
                }
            }
            const float y = ((yv[0] + yv[1]) + (yv[2] + yv[3])) + ((yv[4] + yv[5]) + (yv[6] + yv[7]));
            const float z = ((zv[0] + zv[1]) + (zv[2] + zv[3])) + ((zv[4] + zv[5]) + (zv[6] + zv[7]));
            if (bb < nb) {
                const float gate = __fdividef(1.f, 1.f + __expf(-z));
                out[((size_t)(b0 + bb) * d.n_h + i) * 128 + col0 + e] = __float2bfloat16_rn(y * gate);
            }
        }
        cluster.sync();   // the partial sums may be overwritten (next block) or the CTA may exit
    }
    if (tid == 0 && *abort_flag) raise_status(status_word, GTA_ERR_TIMEOUT);
}

// Cluster size (= split of the reduction dimensions) of the finish kernel: 4 when the larger
// weight slice still fits in shared memory (fewer CTAs per cluster pack onto the GPCs in one wave),
// else 8; 0 if neither split gives whole MMA steps and whole TMA boxes.
static int finish_split(const Dims& d) {
    for (int S = 4; S <= 8; S *= 2) {
        const int hs = d.H / S, dls = d.d_l / S;
        if (d.H % (16 * S) != 0 || (hs > 256 && hs % 256 != 0) || dls > 256) continue;
        if (fin_smem_layout(dls + hs).total <= 200u * 1024u) return S;
    }
    return 0;
}

// ---------------------------------------------------------------------------------------------
// Large batches: log-sum-exp merge of the split-KV slots of one (attention map, sequence) pair per
// CTA into the normalised latent L[n_q][B][d_l] (bf16), which the tcgen05 decoder + gate kernel of
// the prefill path then consumes with the batch in the role of the token axis.
// Launched with programmatic stream serialisation: while the stream kernel still runs, the CTA
// works out from the sequence lengths (inputs, not results of that kernel) which stream CTAs own
// sub-tiles of its sequence -- the same arithmetic as in the stream kernel: prefix sums of
// ceil(len / T), ranges c n / G -- so that after the dependency wait a single round of loads
// (every slot's (max, sum) pair and its partial sums together) is all that is left.
__global__ void __launch_bounds__(256)
decode_merge_kernel(Dims d, int G, int T, int S_cap, const int32_t* __restrict__ seq_lens,
                    const float* __restrict__ part_o, const float* __restrict__ part_ml,
                    __nv_bfloat16* __restrict__ l_out) {
    __shared__ long long red_s[2][8];
    __shared__ int live_s[kFinMaxSlots];        // slot j of the range holds something
    ptx::grid_launch_dependents();
    const int g = blockIdx.x, b = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    long long before = 0, total = 0;            // sub-tiles of the sequences before b, of all sequences
    for (int i = tid; i < d.B; i += 256) {
        const int n = (clamp_len(seq_lens[i], S_cap) + T - 1) / T;
        total += n;
        if (i < b) before += n;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        before += __shfl_xor_sync(0xffffffffu, before, o);
        total += __shfl_xor_sync(0xffffffffu, total, o);
    }
    if (lane == 0) { red_s[0][warp] = before; red_s[1][warp] = total; }
    __syncthreads();
    long long s_lo = 0, n_st = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) { s_lo += red_s[0][w]; n_st += red_s[1][w]; }
    const long long s_hi = s_lo + (clamp_len(seq_lens[b], S_cap) + T - 1) / T;
    // the owner of sub-tile st is the largest c with floor(c n / G) <= st = floor(((st + 1) G - 1) / n)
    int c_lo = 0, c_hi = -1;
    if (s_hi > s_lo) {
        c_lo = (int)(((s_lo + 1) * G - 1) / n_st);
        c_hi = (int)((s_hi * G - 1) / n_st);
    }
    for (int j = tid; c_lo + j <= c_hi; j += 256) {   // a CTA with an empty range wrote nothing
        const int c = c_lo + j;
        live_s[j] = ((long long)c * n_st) / G < ((long long)(c + 1) * n_st) / G;
    }
    __syncthreads();
    ptx::grid_dependency_wait();

    const int col = tid * 4;
    if (col >= d.d_l) return;
    float M = -INFINITY, l = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int c0 = c_lo; c0 <= c_hi; c0 += 8) {       // eight slots per round of loads
        float2 ml[8];
        float4 v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int c = c0 + j;
            ml[j] = make_float2(-INFINITY, 0.f);
            v[j] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (c <= c_hi && live_s[c - c_lo]) {
                const size_t pi = (size_t)(c + b) * d.n_q + g;
                ml[j] = *reinterpret_cast<const float2*>(part_ml + pi * 2);
                v[j] = *reinterpret_cast<const float4*>(part_o + pi * d.d_l + col);
            }
        }
        float Mn = M;
#pragma unroll
        for (int j = 0; j < 8; ++j) Mn = fmaxf(Mn, ml[j].x);
        if (Mn == -INFINITY) continue;               // nothing live so far
        const float scale = ex2f(M - Mn);            // 0 on the first live round (M = -inf)
        l *= scale;
        acc.x *= scale; acc.y *= scale; acc.z *= scale; acc.w *= scale;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float w = ex2f(ml[j].x - Mn);      // 0 for a slot that is not there
            l = fmaf(ml[j].y, w, l);
            acc.x = fmaf(v[j].x, w, acc.x); acc.y = fmaf(v[j].y, w, acc.y);
            acc.z = fmaf(v[j].z, w, acc.z); acc.w = fmaf(v[j].w, w, acc.w);
        }
        M = Mn;
    }
    const float inv_l = l > 0.f ? 1.f / l : 0.f;     // an empty sequence gives zeros
    uint2 packed;
    packed.x = pack_bf16(acc.x * inv_l, acc.y * inv_l);
    packed.y = pack_bf16(acc.z * inv_l, acc.w * inv_l);
    *reinterpret_cast<uint2*>(l_out + ((size_t)g * d.B + b) * d.d_l + col) = packed;
}

// ---------------------------------------------------------------------------------------------
cudaError_t launch_decode_fast(const Dims& d, const void* q, const void* k_cache, const void* c_cache,
                               const int32_t* seq_lens, int S_cap, const void* x_t, const void* w_p,
                               const void* w_g, void* out, void* workspace, int32_t* status_word,
                               cudaStream_t stream, int stages, int* launches) {
    const FastPlan p = make_fast_plan(d);
    float* part_o = reinterpret_cast<float*>(workspace);
    float* part_ml = reinterpret_cast<float*>(static_cast<char*>(workspace) + p.off_ml);
    __nv_bfloat16* l_g = reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(workspace) + p.off_l);
    const bool big_batch = !(d.B <= kFinMaxBatchClusters && d.d_h == 128 && d.d_l >= 256 &&
                             (d.n_q & (d.n_q - 1)) == 0 && d.n_c == 1);
    cudaError_t err;
    if (stages & 2) {
        CUtensorMap tm_k, tm_c;
        const uint32_t box[3] = {64, (uint32_t)p.T, 1};
        const uint64_t dk[3] = {(uint64_t)d.d_h, (uint64_t)S_cap, (uint64_t)d.B * d.n_k};
        const uint64_t dc[3] = {(uint64_t)d.d_l, (uint64_t)S_cap, (uint64_t)d.B * d.n_c};
        if (!make_bf16_map(&tm_k, k_cache, 3, dk, box) || !make_bf16_map(&tm_c, c_cache, 3, dc, box))
            return cudaErrorInvalidValue;
        const size_t smem = (size_t)kStreamStages * kStreamStageBytes + 2 * 8 * kStreamMaxT * sizeof(float) +
                            (size_t)(kStreamMaxBatch + 2 + kStreamThreads) * sizeof(int32_t) +
                            2 * kStreamStages * sizeof(uint64_t) + 16 + 1024;
#define GTA_LAUNCH_STREAM_(NT, KH, ONE)                                                                    \
        do {                                                                                               \
            auto kern = decode_stream_kernel<NT, KH, (NT == 2 ? 8 : 4), ONE>;                              \
            err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);      \
            if (err != cudaSuccess) return err;                                                            \
            cudaLaunchConfig_t cfg = {};                                                                   \
            cfg.gridDim = dim3(p.G);                                                                       \
            cfg.blockDim = dim3(kStreamThreads);                                                           \
            cfg.dynamicSmemBytes = smem;                                                                   \
            cfg.stream = stream;                                                                           \
            cudaLaunchAttribute attr[1];                                                                   \
            attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;                               \
            attr[0].val.programmaticStreamSerializationAllowed = 1;                                        \
            cfg.attrs = attr;                                                                              \
            cfg.numAttrs = 1;                                                                              \
            err = cudaLaunchKernelEx(&cfg, kern, tm_k, tm_c, d, p.T, S_cap, (const __nv_bfloat16*)q,       \
                                     seq_lens, part_o, part_ml, status_word);                              \
            if (err != cudaSuccess) return err;                                                            \
        } while (0)
#define GTA_LAUNCH_STREAM(NT)                                                                              \
        do {                                                                                               \
            if (d.d_h == 128 && d.n_c == 1) GTA_LAUNCH_STREAM_(NT, 2, true);                               \
            else if (d.d_h == 128) GTA_LAUNCH_STREAM_(NT, 2, false);                                       \
            else if (d.n_c == 1) GTA_LAUNCH_STREAM_(NT, 1, true);                                          \
            else GTA_LAUNCH_STREAM_(NT, 1, false);                                                         \
        } while (0)
        switch (d.d_l) {
            case 128: GTA_LAUNCH_STREAM(2); break;
            case 256: GTA_LAUNCH_STREAM(4); break;
            case 512: GTA_LAUNCH_STREAM(8); break;
            default: GTA_LAUNCH_STREAM(16); break;
        }
#undef GTA_LAUNCH_STREAM
#undef GTA_LAUNCH_STREAM_
        if ((err = cudaGetLastError()) != cudaSuccess) return err;
        *launches += 1;
    }
    if ((stages & 4) && big_batch) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(d.n_q, d.B);
        cfg.blockDim = dim3(256);
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        err = cudaLaunchKernelEx(&cfg, decode_merge_kernel, d, p.G, p.T, S_cap, seq_lens, (const float*)part_o,
                                 (const float*)part_ml, l_g);
        if (err != cudaSuccess) return err;
        // the batch takes the role of the token axis: L [n_q][B][d_l], x_t [B][H], out [B][n_h][d_h]
        Dims dd = d;
        dd.B = 1;
        dd.N = d.B;
        if (launch_sm100_decoder(dd, l_g, x_t, w_p, w_g, out, status_word, stream) != GTA_OK) return cudaErrorUnknown;
        *launches += 2;
    } else if (stages & 4) {
        const int S = finish_split(d);
        const int dls = d.d_l / S, hs = d.H / S, KA = dls + hs;
        CUtensorMap tm_wp, tm_wg;
        {
            const uint64_t dims[3] = {128, (uint64_t)d.d_l, (uint64_t)d.n_h};
            const uint32_t box[3] = {64, (uint32_t)dls, 1};
            if (!make_bf16_map(&tm_wp, w_p, 3, dims, box)) return cudaErrorInvalidValue;
        }
        {
            const uint64_t dims[2] = {(uint64_t)d.n_h * 128, (uint64_t)d.H};
            const uint32_t box[2] = {64, (uint32_t)(hs < 256 ? hs : 256)};
            if (!make_bf16_map(&tm_wg, w_g, 2, dims, box)) return cudaErrorInvalidValue;
        }
        const size_t smem = fin_smem_layout(KA).total;
        err = cudaFuncSetAttribute(decode_finish_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return err;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(S, d.n_h * 2);
        cfg.blockDim = dim3(kFinThreads);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = stream;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = S;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        // the kernel may be scheduled while the stream kernel drains; it waits for it on the device
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 2;
        err = cudaLaunchKernelEx(&cfg, decode_finish_kernel, tm_wp, tm_wg, d, p.G, p.T, S_cap, seq_lens,
                                 (const float*)part_o, (const float*)part_ml, (const __nv_bfloat16*)x_t,
                                 (__nv_bfloat16*)out, status_word);
        if (err != cudaSuccess) return err;
        if ((err = cudaGetLastError()) != cudaSuccess) return err;
        *launches += 1;
    }
    return cudaSuccess;
}

}  // namespace gta
