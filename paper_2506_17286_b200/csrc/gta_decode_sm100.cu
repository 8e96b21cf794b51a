// Bandwidth-oriented decode for bf16 caches (App. B.1.3): d_h = 64 or 128, up to 8 attention maps.
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
//   decode_merge_kernel : log-sum-exp merge of the slots into the normalised latent L (bf16); the
//       tcgen05 decoder + gate kernel of the prefill path then runs with the batch as its token
//       axis.  Both are launched with programmatic stream serialisation behind the stream kernel.
#include "gta_common.cuh"
#include "gta_sm100.cuh"
#include "sm100_ptx.cuh"
#include "tma_host.cuh"

namespace gta {

constexpr int kStreamConsumers = 256;
constexpr int kStreamThreads = kStreamConsumers + 32;
constexpr int kStreamStages = 3;
constexpr int kStreamStageBytes = 65536;
constexpr int kStreamMaxBatch = 512;
constexpr int kStreamMaxT = 64;      // tokens per sub-tile
constexpr int kFinMaxSlots = 1024;  // >= stream CTAs + batch

struct FastPlan {
    int T;         // tokens per sub-tile (16, 32 or 64)
    int G;         // stream CTAs
    int slots;     // G + B partial slots
    int occ;       // stream CTAs per SM (1, or 2 for narrow caches)
    size_t off_ml, off_l, total;   // byte offsets in the workspace (part_o at 0)
};

static size_t align256f(size_t v) { return (v + 255) & ~(size_t)255; }

bool decode_fast_supported(const Dims& d, int dtype, int page_size) {
    if (dtype != GTA_BF16 || (d.d_h != 128 && d.d_h != 64)) return false;
    if (page_size % kStreamMaxT != 0) return false;              // a sub-tile never straddles two pages
    if (d.d_l != 64 && d.d_l != 128 && d.d_l != 256 && d.d_l != 512 && d.d_l != 1024) return false;
    if (d.n_q < 1 || d.n_q > 8) return false;                    // the maps are the rows of the warp-level MMAs
    if (d.n_k != 1 && d.n_k != 2 && d.n_k != 4 && d.n_k != 8) return false;   // key groups are dealt to the 8 warps
    if (d.H % 64 != 0 || d.B > kStreamMaxBatch) return false;
    // the finish (merge kernel + tcgen05 decoder kernel) cuts the output columns in blocks inside one attention map
    if (((d.n_h / d.n_q) * d.d_h) % (d.B > 128 ? 128 : 64) != 0) return false;
    const int tok_bytes = (d.n_k * d.d_h + d.n_c * d.d_l) * 2;
    return tok_bytes * 16 <= kStreamStageBytes;
}

// SM count of the CURRENT device (the grid, the slot count and hence the workspace size follow it),
// looked up once per device ordinal and thread; 148 when there is no device to ask (a host without GPUs).
static int sm_count() {
    static thread_local int cached_dev = -1, cached_n = 148;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        return 148;
    }
    if (dev != cached_dev) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) {
            cudaGetLastError();
            v = 148;
        }
        cached_dev = dev;
        cached_n = v;
    }
    return cached_n;
}

static FastPlan make_fast_plan(const Dims& d) {
    FastPlan p;
    const int tok_bytes = (d.n_k * d.d_h + d.n_c * d.d_l) * 2;
    int t = 16;
    // Narrow caches (a 64-token sub-tile within 32 KB): two CTAs per SM with half-size ring stages.  The
    // work per byte is the same, but a sub-tile is small against its fixed latency chain (barrier,
    // score -> softmax -> latent sum), which two independent CTAs on an SM hide behind one another.
    p.occ = (d.d_l <= 128 && kStreamMaxT * tok_bytes <= kStreamStageBytes / 2) ? 2 : 1;
    while (t * 2 * tok_bytes <= kStreamStageBytes / p.occ && t * 2 <= kStreamMaxT) t *= 2;
    p.T = t;
    const int ctas = p.occ * sm_count();
    p.G = ctas < kFinMaxSlots - kStreamMaxBatch ? ctas : kFinMaxSlots - kStreamMaxBatch;
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
// Length a decode step attends over.  With `append` (the fused append + decode step) the stored length does not
// count the new token yet: a sequence with room for it (0 <= len < S_cap) attends over len + 1 tokens, the last
// of which comes from the new rows; a full or invalid one is left as it is (and reported by the kernel).
struct StepLens {
    const int32_t* seq_lens;
    int S_cap, append;
    __device__ __forceinline__ bool appends(int b) const {
        const int len = seq_lens[b];
        return append && len >= 0 && len < S_cap;
    }
    __device__ __forceinline__ int len(int b) const { return clamp_len(seq_lens[b], S_cap) + (appends(b) ? 1 : 0); }
};

// Shared-memory layout of one ring stage (all tiles are [T rows][64 bf16] = T x 128 bytes with
// the 128-byte TMA swizzle: the 16-byte chunk c of row r sits at chunk c ^ (r & 7)):
//   K tiles : key group kg, half h (columns 64 h .. 64 h + 63)  at (KH kg + h) T 128
//   C tiles : latent group cg, columns 64 j .. 64 j + 63         at c_off + (NT cg + j) T 128
// NT = d_l / 64 = MMA n-tiles (8 latent columns each) per consumer warp; KH = d_h / 64 = 64-column
// tiles per key row; ONE_C: a single latent group (the latent-sum loop then has no group pass and no
// masking); OCC: CTAs per SM (ring stages of 64 KB / OCC)
template <int NT, int KH, bool ONE_C, int OCC>
__global__ void __launch_bounds__(kStreamThreads, OCC)
decode_stream_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_c, Dims d,
                     int T, int S_cap, const __nv_bfloat16* __restrict__ q, const int32_t* __restrict__ seq_lens,
                     float* __restrict__ part_o, float* __restrict__ part_ml, int32_t* status_word, PageMap pm,
                     const uint4* __restrict__ k_new, const uint4* __restrict__ c_new, uint4* __restrict__ k_rows,
                     uint4* __restrict__ c_rows) {
    // k_new != nullptr: the fused append + decode step (contiguous caches).  k_new [B][n_k][d_h] / c_new
    // [B][n_c][d_l] are the new token's rows, k_rows / c_rows the caches as writable 16-byte vectors.
    const StepLens L{seq_lens, S_cap, k_new != nullptr};
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* ring = smem;                                                              // 3 x 64 KB
    constexpr int KTM = kStreamMaxT / 16;                     // most 16-token MMA k-steps per sub-tile
    constexpr int kStageBytes = kStreamStageBytes / OCC;
    float* s_buf = reinterpret_cast<float*>(smem + kStreamStages * kStageBytes);   // [2][n_q][T]
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
        for (int b = lo; b < hi; ++b) sum += (L.len(b) + T - 1) / T;
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
            base += (L.len(b) + T - 1) / T;
        }
        if (tid == kStreamThreads - 1) prefix[d.B] = base;
        __syncthreads();
    }
    if (L.append && cta == 0) {      // a sequence without room for the new token is left as it is and reported
        for (int b = tid; b < d.B; b += kStreamThreads)
            if (!L.appends(b)) raise_status(status_word, GTA_ERR_CACHE_FULL);
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
                // Contiguous caches: rows tok0 .. of plane b groups + g.  Paged pool: the sub-tile lies inside
                // one page (T divides the page size), at rows tok0 % page_size .. of plane page groups + g; the
                // block-table entry is fetched before the wait for the stage.  An entry outside the pool raises
                // the status word, and the load (of page 0 then) still completes the stage.
                int tok0 = (int)k * T, plane = b;
                if (pm.table != nullptr) {
                    const int page = page_of(pm, b, tok0, lane == 0 ? status_word : nullptr);
                    plane = page < 0 ? 0 : page;
                    tok0 %= pm.page_size;
                }
                if (lane == 0) {
                    ok = ptx::mbar_wait(&empty_bar[s], ph ^ 1, abort_flag);
                    if (ok) ptx::mbar_arrive_expect_tx(&full_bar[s], stage_tx);
                }
                ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                if (!ok) break;
                uint8_t* stage = ring + s * kStageBytes;
                for (int op = lane; op < n_k_ops + n_c_tiles; op += 32) {
                    if (op < n_k_ops)
                        ptx::tma_load_3d_hint(stage + op * tile_bytes, &tm_k, &full_bar[s], (op % KH) * 64, tok0,
                                              plane * d.n_k + op / KH, policy);
                    else
                        ptx::tma_load_3d_hint(stage + c_off + (op - n_k_ops) * tile_bytes, &tm_c, &full_bar[s],
                                              ((op - n_k_ops) % NT) * 64, tok0, plane * d.n_c + (op - n_k_ops) / NT, policy);
                }
            }
            if (lane == 0 && *abort_flag) {
                for (int back = 1; back <= kStreamStages && it - back >= 0; ++back) {
                    const int iq = it - back;
                    ptx::mbar_wait_drain(&full_bar[iq % kStreamStages], (iq / kStreamStages) & 1, drain_flag);
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

        // Fused append: the new token's rows of the current sequence, two 16-byte vectors per thread at most
        // (vector v < k_vecs belongs to K, the others to C), fetched when the sequence is taken up so that the
        // latency has passed when its last sub-tile -- the one that holds the new token -- comes round.
        const int k_vecs = d.n_k * KH * 8, new_vecs = k_vecs + n_c_tiles * 8;      // 8 vectors per 64-column tile row
        uint4 nv[2];
        auto load_new = [&](int b) {
            if (!L.appends(b)) return;
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const int v = tid + i * kStreamConsumers;
                if (v < k_vecs) nv[i] = __ldg(k_new + (size_t)b * k_vecs + v);
                else if (v < new_vecs) nv[i] = __ldg(c_new + (size_t)b * (new_vecs - k_vecs) + (v - k_vecs));
            }
        };
        int b = b0;
        long long k = st_begin - prefix[b0];
        load_q(b);
        load_new(b);
        int it = 0;
        bool ok = true;
        for (long long st = st_begin; st < st_end; ++st, ++it, ++k) {
            if (k >= prefix[b + 1] - prefix[b]) {
                flush(b);
                do { ++b; } while (prefix[b + 1] == prefix[b]);
                k = 0;
                load_q(b);
                load_new(b);
            }
            const int s = it % kStreamStages;
            const uint32_t ph = (it / kStreamStages) & 1;
            // A wait that gives up raises the CTA's abort flag, after which every wait returns at once.  The warp does
            // NOT leave the loop then: other consumer warps may already stand at a CTA barrier of this or a later
            // sub-tile, which needs all eight.  It skips the work and keeps the appointments (as many barriers as the
            // sub-tile has) to the end of its range; nothing is flushed.
            ok = __all_sync(0xffffffffu, ptx::mbar_wait(&full_bar[s], ph, abort_flag));   // (once false, false for good: the flag)
            if (!ok) {
                if (L.appends(b) && ((int)k + 1) * T >= L.len(b)) consumer_sync();
                consumer_sync();
                continue;
            }
            const int len = L.len(b);
            const int n_valid = min(T, len - (int)k * T);
            // the sub-tile that ends the sequence holds the new token (row n_valid - 1): what TMA brought for that
            // row is whatever the cache held; the new rows are put over it here, and written to the caches
            const bool patch = L.appends(b) && ((int)k + 1) * T >= len;
            if (patch) {
                const int row = n_valid - 1;
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const int v = tid + i * kStreamConsumers;
                    if (v < new_vecs) {
                        // vector v: tile v >> 3 of the stage (K tiles first, then the C tiles), 16-byte chunk v & 7
                        uint8_t* p = ring + s * kStageBytes + (v >> 3) * tile_bytes + row * 128 + (((v & 7) ^ (row & 7)) << 4);
                        *reinterpret_cast<uint4*>(p) = nv[i];
                        if (v < k_vecs) {       // K row of group v / (8 KH): vector v % (8 KH) of its d_h columns
                            const int g = v / (8 * KH);
                            k_rows[(((size_t)b * d.n_k + g) * S_cap + (len - 1)) * (8 * KH) + v % (8 * KH)] = nv[i];
                        } else {
                            const int cv = v - k_vecs, g = cv / (8 * NT);
                            c_rows[(((size_t)b * d.n_c + g) * S_cap + (len - 1)) * (8 * NT) + cv % (8 * NT)] = nv[i];
                        }
                    }
                }
                ptx::fence_proxy_async_smem();   // the next TMA write of this stage follows generic writes
                consumer_sync();                 // the scores below read the row
            }
            const uint32_t stage = ring_addr + s * kStageBytes;
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
                    uint8_t* p = ring + s * kStageBytes + c_off + (v >> 3) * tile_bytes + row * 128 + (v & 7) * 16;
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
                        if constexpr (NT == 1) {     // 64 latent columns: one 8-column n-tile per warp
                            const int chunk = warp;   // 16-byte chunk of the latent row
                            uint32_t c0, c1;
                            ptx::ldsm_x2_trans(crow + (((chunk & 7) ^ (token & 7)) << 4), c0, c1);
                            ptx::mma_bf16_16816(acc[0], a0, 0u, a2, 0u, c0, c1);
                        } else {
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
// Log-sum-exp merge of the split-KV slots of one (attention map, sequence) pair per
// CTA into the normalised latent (bf16), row (g, b) at l_out + g stride_g + b stride_b: L[n_q][B][d_l] for the
// tcgen05 decoder + gate kernel of the prefill path, which then consumes it with the batch in the role of the
// token axis (the comparison operators take it head by head as their output).
// Launched with programmatic stream serialisation: while the stream kernel still runs, the CTA
// works out from the sequence lengths (inputs, not results of that kernel) which stream CTAs own
// sub-tiles of its sequence -- the same arithmetic as in the stream kernel: prefix sums of
// ceil(len / T), ranges c n / G -- so that after the dependency wait a single round of loads
// (every slot's (max, sum) pair and its partial sums together) is all that is left.
__global__ void __launch_bounds__(256)
decode_merge_kernel(Dims d, int G, int T, int S_cap, const int32_t* __restrict__ seq_lens,
                    const float* __restrict__ part_o, const float* __restrict__ part_ml,
                    __nv_bfloat16* __restrict__ l_out, long long stride_g, long long stride_b, int append) {
    const StepLens L{seq_lens, S_cap, append};
    __shared__ long long red_s[2][8];
    __shared__ int live_s[kFinMaxSlots];        // slot j of the range holds something
    ptx::grid_launch_dependents();
    const int g = blockIdx.x, b = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    long long before = 0, total = 0;            // sub-tiles of the sequences before b, of all sequences
    for (int i = tid; i < d.B; i += 256) {
        const int n = (L.len(i) + T - 1) / T;
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
    const long long s_hi = s_lo + (L.len(b) + T - 1) / T;
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
    *reinterpret_cast<uint2*>(l_out + g * stride_g + b * stride_b + col) = packed;
}

// ---------------------------------------------------------------------------------------------
// Stream kernel (stages & 2) and merge kernel (stages & 4) of one decode step: the normalised latent rows go to
// l_out (row (g, b) at g stride_g + b stride_b elements).
static cudaError_t launch_stream_and_merge(const Dims& d, const FastPlan& p, const void* q, const void* k_cache,
                                           const void* c_cache, const int32_t* seq_lens, int S_cap, float* part_o,
                                           float* part_ml, __nv_bfloat16* l_out, long long stride_g,
                                           long long stride_b, int32_t* status_word, cudaStream_t stream, int stages,
                                           int* launches, const PageMap& pm, const void* k_new = nullptr,
                                           const void* c_new = nullptr) {
    cudaError_t err;
    if ((stages & 2) && decode_tc_supported(d, p.T, p.occ, pm.table ? pm.page_size : 0)) {
        // the cached tokens as the rows of tcgen05 MMAs (gta_decode_tc.cu)
        err = launch_decode_tc_stream(d, p.G, p.T, S_cap, q, k_cache, c_cache, seq_lens, part_o, part_ml, status_word,
                                      stream, k_new, c_new, pm);
        if (err != cudaSuccess) return err;
        *launches += 1;
    } else if (stages & 2) {
        CUtensorMap tm_k, tm_c;
        const uint32_t box[3] = {64, (uint32_t)p.T, 1};
        // planes of rows: one per (sequence, group), S_cap rows each -- or one per (page, group), page_size rows
        const uint64_t rows = pm.table ? (uint64_t)pm.page_size : (uint64_t)S_cap;
        const uint64_t outer = pm.table ? (uint64_t)pm.n_pages : (uint64_t)d.B;
        const uint64_t dk[3] = {(uint64_t)d.d_h, rows, outer * d.n_k};
        const uint64_t dc[3] = {(uint64_t)d.d_l, rows, outer * d.n_c};
        if (!make_bf16_map(&tm_k, k_cache, 3, dk, box) || !make_bf16_map(&tm_c, c_cache, 3, dc, box))
            return cudaErrorInvalidValue;
        const size_t smem = (size_t)kStreamStages * (kStreamStageBytes / p.occ) + 2 * 8 * kStreamMaxT * sizeof(float) +
                            (size_t)(kStreamMaxBatch + 2 + kStreamThreads) * sizeof(int32_t) +
                            2 * kStreamStages * sizeof(uint64_t) + 16 + 1024;
#define GTA_LAUNCH_STREAM_(NT, KH, ONE, OCC)                                                               \
        do {                                                                                               \
            auto kern = decode_stream_kernel<NT, KH, ONE, OCC>;                                            \
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
                                     seq_lens, part_o, part_ml, status_word, pm, (const uint4*)k_new,      \
                                     (const uint4*)c_new, (uint4*)const_cast<void*>(k_cache),              \
                                     (uint4*)const_cast<void*>(c_cache));                                  \
            if (err != cudaSuccess) return err;                                                            \
        } while (0)
#define GTA_LAUNCH_STREAM(NT)                                                                              \
        do {                                                                                               \
            if (d.d_h == 128 && d.n_c == 1) GTA_LAUNCH_STREAM_(NT, 2, true, 1);                            \
            else if (d.d_h == 128) GTA_LAUNCH_STREAM_(NT, 2, false, 1);                                    \
            else if (d.n_c == 1) GTA_LAUNCH_STREAM_(NT, 1, true, 1);                                       \
            else GTA_LAUNCH_STREAM_(NT, 1, false, 1);                                                      \
        } while (0)
#define GTA_LAUNCH_STREAM_NARROW(NT)   /* d_l <= 128, two CTAs per SM */                                   \
        do {                                                                                               \
            if (d.d_h == 128 && d.n_c == 1) GTA_LAUNCH_STREAM_(NT, 2, true, 2);                            \
            else if (d.d_h == 128) GTA_LAUNCH_STREAM_(NT, 2, false, 2);                                    \
            else if (d.n_c == 1) GTA_LAUNCH_STREAM_(NT, 1, true, 2);                                       \
            else GTA_LAUNCH_STREAM_(NT, 1, false, 2);                                                      \
        } while (0)
        switch (d.d_l) {
            case 64:
                if (p.occ == 2) GTA_LAUNCH_STREAM_NARROW(1);
                else GTA_LAUNCH_STREAM(1);
                break;
            case 128:
                if (p.occ == 2) GTA_LAUNCH_STREAM_NARROW(2);
                else GTA_LAUNCH_STREAM(2);
                break;
            case 256: GTA_LAUNCH_STREAM(4); break;
            case 512: GTA_LAUNCH_STREAM(8); break;
            default: GTA_LAUNCH_STREAM(16); break;
        }
#undef GTA_LAUNCH_STREAM
#undef GTA_LAUNCH_STREAM_NARROW
#undef GTA_LAUNCH_STREAM_
        if ((err = cudaGetLastError()) != cudaSuccess) return err;
        *launches += 1;
    }
    if (stages & 4) {
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
                                 (const float*)part_ml, l_out, stride_g, stride_b, k_new != nullptr ? 1 : 0);
        if (err != cudaSuccess) return err;
        *launches += 1;
    }
    return cudaSuccess;
}

// ---------------------------------------------------------------------------------------------
// The stream kernel for 8-bit caches: K and C rows as e4m3 codes with one fp32 scale per cached row.
// Same schedule, ring, barriers and partial results as decode_stream_kernel; what differs is the arithmetic:
//   * the warp-level MMAs are m16n8k32 on e4m3 operands, so the codes go from shared memory into the tensor
//     pipe as they are.  The other operand has to be e4m3 too, and one e4m3 number (4 significant bits) cannot
//     hold a bf16 query element or a probability (8 significant bits): each is written as the SUM OF TWO e4m3
//     numbers -- x scaled by a power of two, p1 = x rounded to e4m3, p2 = x - p1 (exact: what is left has at
//     most 4 significant bits) -- and the two pieces take rows g and g + 8 of the 16-row operand, so one MMA
//     multiplies both; the two halves of the accumulator are added afterwards.  The sum is exact for every
//     element above 2^-10 of its row's largest; below that the error is 2^-18 of the largest.
//   * a key row's scale multiplies its score after the MMA.  A latent row's scale s_j would have to multiply
//     its probability before the MMA; instead log2(s_j) is added to the score that the WEIGHTS are taken from,
//     w_j = 2^(score_j + log2 s_j - m), with m the running maximum of those shifted scores, so that the
//     weights again fill [0, 1] and sum_j w_j code_j = sum_j 2^(score_j - m) c_j; the row sum l is taken from
//     the unshifted scores against the same m.  (m, l, sums) is a valid partial for the merge kernel: any
//     reference m works as long as nothing overflows, and 2^(score - m) <= 1 / min s_j.
//   * the latent operand B[token][column] is read with transposing 16-bit ldmatrix loads, which deliver two
//     tokens x two columns per register; a byte permute of two such registers gives four tokens of one
//     column.  Which tokens share a register is a permutation of the 32 tokens of a k-step that the weight
//     fragments follow, and the even / odd column split is undone when the sums are written.
//   * the exponentials and the e4m3 conversions of the weights are done once per CTA (each warp takes T / 8
//     tokens) and handed to the other warps through shared memory in fragment order, not once per warp.
// What bounds it: on this architecture the warp-level e4m3 MMA is carried out as f16 MMAs behind conversions of its
// operands on the conversion unit (16 lanes per clock and SM: measured 3.4 conversion instructions per MMA, that
// unit 58 % busy), so the kernel runs at about the token rate of the bf16 kernel -- half its byte rate.  Converting
// the codes to f16 here and issuing f16 MMAs (for the scores only, or for both contractions) was measured slower.
// d_h = 128 (a key row is one 128-byte swizzle row), one latent group, d_l = 128 CH; T = 32 or 64 tokens.
template <int CH>
__global__ void __launch_bounds__(kStreamThreads, 1)
decode_stream_fp8_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_c, Dims d,
                         int T, int S_cap, const __nv_bfloat16* __restrict__ q, const float* __restrict__ k_scale,
                         const float* __restrict__ c_scale, const int32_t* __restrict__ seq_lens,
                         float* __restrict__ part_o, float* __restrict__ part_ml, int32_t* status_word) {
    const StepLens L{seq_lens, S_cap, 0};
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    constexpr int KTM = kStreamMaxT / 32;                      // most 32-token MMA k-steps per sub-tile
    const uint32_t tile_bytes = (uint32_t)T * 128;
    const uint32_t c_off = (uint32_t)d.n_k * tile_bytes;       // the CH latent tiles follow the n_k key tiles
    const uint32_t scale_off = c_off + CH * tile_bytes;        // then [n_k][T] key scales and [T] latent scales
    const uint32_t stage_stride = scale_off + (((uint32_t)(d.n_k + 1) * T * 4 + 1023) & ~1023u);
    uint8_t* ring = smem;
    float* s_buf = reinterpret_cast<float*>(smem + kStreamStages * stage_stride);        // [2][2][n_q][T]: scores, shifted scores
    uint4* w_buf = reinterpret_cast<uint4*>(s_buf + 4 * 8 * kStreamMaxT);                // [KTM][8 maps][4]: weight fragments
    float* den_buf = reinterpret_cast<float*>(w_buf + KTM * 32);                         // [8 warps][32 lanes]: row-sum shares
    int32_t* prefix = reinterpret_cast<int32_t*>(den_buf + 256);                         // [B + 1]
    int32_t* scan_tmp = prefix + kStreamMaxBatch + 2;                                    // [kStreamThreads]
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(scan_tmp + kStreamThreads);
    uint64_t* empty_bar = full_bar + kStreamStages;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(empty_bar + kStreamStages);
    volatile int* drain_flag = abort_flag + 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int G = gridDim.x, cta = blockIdx.x;
    const int NQ = d.n_q;
    if (tid == kStreamConsumers) {
        ptx::prefetch_tensormap(&tm_k);
        ptx::prefetch_tensormap(&tm_c);
    }
    // launched with programmatic stream serialisation: nothing of global memory is read before the kernel ahead
    // (a quantising append) is complete, and only then may the kernels behind this one be scheduled
    ptx::grid_dependency_wait();
    ptx::grid_launch_dependents();

    {   // exclusive prefix sum of the sub-tile counts (as in decode_stream_kernel)
        const int per = (d.B + kStreamThreads - 1) / kStreamThreads;
        const int lo = min(tid * per, d.B), hi = min(lo + per, d.B);
        int sum = 0;
        for (int b = lo; b < hi; ++b) sum += (L.len(b) + T - 1) / T;
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
            base += (L.len(b) + T - 1) / T;
        }
        if (tid == kStreamThreads - 1) prefix[d.B] = base;
        __syncthreads();
    }
    const long long n_st = prefix[d.B];
    const long long st_begin = ((long long)cta * n_st) / G, st_end = ((long long)(cta + 1) * n_st) / G;
    if (st_begin >= st_end) return;      // uniform: nothing armed
    int b0;
    {
        int lo = 0, hi = d.B - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (prefix[mid] <= st_begin) lo = mid; else hi = mid - 1;
        }
        b0 = lo;
    }

    if (warp == kStreamConsumers / 32) {
        // ------------------------------------------------------------------ producer: one load per lane
        const uint64_t policy = ptx::l2_evict_first_policy();
        const int n_tiles = d.n_k + CH, n_ops = n_tiles + d.n_k + 1;      // tensor tiles, then the scale rows
        int b = b0;
        long long k = st_begin - prefix[b0];
        int it = 0;
        bool ok = true;
        for (long long st = st_begin; st < st_end; ++st, ++it, ++k) {
            while (k >= prefix[b + 1] - prefix[b]) { ++b; k = 0; }
            const int s = it % kStreamStages;
            const uint32_t ph = (it / kStreamStages) & 1;
            const int tok0 = (int)k * T;
            const uint32_t n_sc = (uint32_t)min(T, S_cap - tok0) * 4;     // bytes of a scale row (S_cap is a multiple of 4)
            if (lane == 0) {
                ok = ptx::mbar_wait(&empty_bar[s], ph ^ 1, abort_flag);
                if (ok) ptx::mbar_arrive_expect_tx(&full_bar[s], scale_off + (uint32_t)(d.n_k + 1) * n_sc);
            }
            ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
            if (!ok) break;
            uint8_t* stage = ring + s * stage_stride;
            for (int op = lane; op < n_ops; op += 32) {
                if (op < d.n_k)
                    ptx::tma_load_3d_hint(stage + op * tile_bytes, &tm_k, &full_bar[s], 0, tok0, b * d.n_k + op, policy);
                else if (op < n_tiles)
                    ptx::tma_load_3d_hint(stage + op * tile_bytes, &tm_c, &full_bar[s], (op - d.n_k) * 128, tok0, b, policy);
                else if (op < n_tiles + d.n_k)
                    ptx::bulk_load_1d(stage + scale_off + (op - n_tiles) * T * 4,
                                      k_scale + ((size_t)b * d.n_k + (op - n_tiles)) * S_cap + tok0, n_sc, &full_bar[s]);
                else
                    ptx::bulk_load_1d(stage + scale_off + d.n_k * T * 4, c_scale + (size_t)b * S_cap + tok0, n_sc,
                                      &full_bar[s]);
            }
        }
        if (lane == 0 && *abort_flag) {
            for (int back = 1; back <= kStreamStages && it - back >= 0; ++back) {
                const int iq = it - back;
                ptx::mbar_wait_drain(&full_bar[iq % kStreamStages], (iq / kStreamStages) & 1, drain_flag);
            }
        }
    } else {
        // ------------------------------------------------------------------ consumers
        const int quad = lane >> 2, sub = lane & 3;       // MMA fragment coordinates
        const int mat = lane >> 3, mrow = lane & 7;       // ldmatrix: which 8x8 matrix, which row of it
        const int qpk = NQ / d.n_k;                       // maps per key group
        const int kg_w = warp % d.n_k;                    // this warp scores key group kg_w
        const int KT = T >> 5;                            // 32-token MMA k-steps per sub-tile
        const int n_units = (T >> 3) * d.n_k;             // (8-token n-tile, key group) scoring units
        const uint32_t ring_addr = ptx::smem_addr(ring);
        const bool map_lane = quad < NQ;
        float m_run = -INFINITY, l_run = 0.f;
        float acc[2 * CH][4];
#pragma unroll
        for (int n = 0; n < 2 * CH; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
        uint32_t qa[4][4];                                // A fragments of the query pieces, d_h = 4 k-steps of 32
        float q_mul = 0.f;                                // power-of-two scale of the query row x softmax scale x log2(e)

        // x0 .. x3 -> the four codes of each piece, packed lowest element first
        auto split4 = [](float x0, float x1, float x2, float x3, uint32_t& hi, uint32_t& lo) {
            const uint32_t h01 = ptx::cvt_e4m3x2(x0, x1), h23 = ptx::cvt_e4m3x2(x2, x3);
            const float2 b01 = ptx::e4m3x2_to_f32(h01), b23 = ptx::e4m3x2_to_f32(h23);
            hi = h01 | (h23 << 16);
            lo = ptx::cvt_e4m3x2(x0 - b01.x, x1 - b01.y) | (ptx::cvt_e4m3x2(x2 - b23.x, x3 - b23.y) << 16);
        };
        auto load_q = [&](int b) {
            const bool live = quad < qpk;
            const __nv_bfloat16* qrow = q + ((size_t)b * NQ + kg_w * qpk + (live ? quad : 0)) * 128;
            float v[4][8];
            float amax = 0.f;
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {             // elements 32 ks + 16 h + 4 sub .. + 3
                    const uint2 raw = __ldg(reinterpret_cast<const uint2*>(qrow + 32 * ks + 16 * h + 4 * sub));
                    const float2 lo = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.x));
                    const float2 hi = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.y));
                    v[ks][4 * h] = live ? lo.x : 0.f; v[ks][4 * h + 1] = live ? lo.y : 0.f;
                    v[ks][4 * h + 2] = live ? hi.x : 0.f; v[ks][4 * h + 3] = live ? hi.y : 0.f;
#pragma unroll
                    for (int e = 0; e < 4; ++e) amax = fmaxf(amax, fabsf(v[ks][4 * h + e]));
                }
            }
            amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
            amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
            // power of two that brings the row's largest element into [128, 256) (e4m3 reaches 448)
            uint32_t e = (__float_as_uint(amax) >> 23) & 0xffu;
            e = e < 8u ? 8u : e;
            const float scale = __uint_as_float((e - 7u) << 23), inv = __uint_as_float((261u - e) << 23);
            q_mul = scale * d.scale * 1.4426950408889634f;
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                split4(v[ks][0] * inv, v[ks][1] * inv, v[ks][2] * inv, v[ks][3] * inv, qa[ks][0], qa[ks][1]);
                split4(v[ks][4] * inv, v[ks][5] * inv, v[ks][6] * inv, v[ks][7] * inv, qa[ks][2], qa[ks][3]);
            }
        };
        auto flush = [&](int b) {
            const int slot = cta + b;
            if (map_lane) {
                float* o = part_o + ((size_t)slot * NQ + quad) * d.d_l + warp * (CH * 16) + 4 * sub;
#pragma unroll
                for (int c = 0; c < CH; ++c) {
                    // even / odd columns of the chunk, pieces added, the weights' factor 2^8 taken out
                    const float4 v = make_float4((acc[2 * c][0] + acc[2 * c][2]) * 0.00390625f,
                                                 (acc[2 * c + 1][0] + acc[2 * c + 1][2]) * 0.00390625f,
                                                 (acc[2 * c][1] + acc[2 * c][3]) * 0.00390625f,
                                                 (acc[2 * c + 1][1] + acc[2 * c + 1][3]) * 0.00390625f);
                    *reinterpret_cast<float4*>(o + 16 * c) = v;
                }
                if (warp == 0 && sub == 0) {
                    part_ml[((size_t)slot * NQ + quad) * 2] = m_run;
                    part_ml[((size_t)slot * NQ + quad) * 2 + 1] = l_run;
                }
            }
#pragma unroll
            for (int n = 0; n < 2 * CH; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
            m_run = -INFINITY;
            l_run = 0.f;
        };

        int b = b0;
        long long k = st_begin - prefix[b0];
        load_q(b);
        int it = 0;
        bool ok = true;
        long long st = st_begin;
        for (; st < st_end; ++st, ++it, ++k) {
            if (k >= prefix[b + 1] - prefix[b]) {
                flush(b);
                do { ++b; } while (prefix[b + 1] == prefix[b]);
                k = 0;
                load_q(b);
            }
            const int s = it % kStreamStages;
            const uint32_t ph = (it / kStreamStages) & 1;
            ok = __all_sync(0xffffffffu, ptx::mbar_wait(&full_bar[s], ph, abort_flag));
            if (!ok) break;      // (the appointments of the remaining sub-tiles are kept below)
            const int n_valid = min(T, L.len(b) - (int)k * T);
            const uint32_t stage = ring_addr + s * stage_stride;
            const float* ksc = reinterpret_cast<const float*>(ring + s * stage_stride + scale_off);
            const float* csc = ksc + d.n_k * T;
            float* sb = s_buf + (it & 1) * (2 * NQ * T);      // scores [n_q][T]
            float* sbw = sb + NQ * T;                          // scores shifted by log2 of the latent row's scale

            // ---- scores of the maps of key group kg_w, 8 tokens per unit
            for (int u = warp; u < n_units; u += 8) {
                const int nt = u / d.n_k;
                const int token = nt * 8 + mrow;
                const uint32_t krow = stage + (uint32_t)kg_w * tile_bytes + token * 128;
                float sc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int kp = 0; kp < 2; ++kp) {
                    const int chunk = 4 * kp + mat;     // 16-byte chunk (16 codes) of the key row
                    uint32_t k0, k1, k2, k3;
                    ptx::ldsm_x4(krow + (((chunk & 7) ^ (token & 7)) << 4), k0, k1, k2, k3);
                    ptx::mma_e4m3_16832(sc, qa[2 * kp][0], qa[2 * kp][1], qa[2 * kp][2], qa[2 * kp][3], k0, k1);
                    ptx::mma_e4m3_16832(sc, qa[2 * kp + 1][0], qa[2 * kp + 1][1], qa[2 * kp + 1][2], qa[2 * kp + 1][3], k2, k3);
                }
                if (quad < qpk) {
                    const int t0 = nt * 8 + 2 * sub;
                    const float2 ks2 = *reinterpret_cast<const float2*>(ksc + kg_w * T + t0);
                    const float2 cs2 = *reinterpret_cast<const float2*>(csc + t0);
                    float2 v, y;
                    v.x = t0 < n_valid ? (sc[0] + sc[2]) * q_mul * ks2.x : -INFINITY;
                    v.y = t0 + 1 < n_valid ? (sc[1] + sc[3]) * q_mul * ks2.y : -INFINITY;
                    y.x = t0 < n_valid ? v.x + __log2f(cs2.x) : -INFINITY;
                    y.y = t0 + 1 < n_valid ? v.y + __log2f(cs2.y) : -INFINITY;
                    *reinterpret_cast<float2*>(sb + (kg_w * qpk + quad) * T + t0) = v;
                    *reinterpret_cast<float2*>(sbw + (kg_w * qpk + quad) * T + t0) = y;
                }
            }
            // ---- rows past the live length hold whatever the cache holds there (NaN codes included): their
            //      weights are zero, so the latent rows are cleared
            if (n_valid < T) {
                const int vec_per_row = CH * 8;
                const int n_vec = (T - n_valid) * vec_per_row;
                for (int idx = tid; idx < n_vec; idx += kStreamConsumers) {
                    const int row = n_valid + idx / vec_per_row, v = idx % vec_per_row;
                    uint8_t* p = ring + s * stage_stride + c_off + (v >> 3) * tile_bytes + row * 128 + (v & 7) * 16;
                    *reinterpret_cast<uint4*>(p) = make_uint4(0u, 0u, 0u, 0u);
                }
                ptx::fence_proxy_async_smem();   // the next TMA write of this stage follows generic writes
            }
            consumer_sync();

            // ---- (A) every warp: the running maximum of map `quad` over the shifted scores of all T tokens
            float alpha = 1.f, m_sub = 0.f;
            bool any = false;
            {
                float m_t = -INFINITY;
#pragma unroll
                for (int kt = 0; kt < KTM; ++kt) {
                    if (kt < KT && map_lane) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const float2 y = *reinterpret_cast<const float2*>(sbw + quad * T + 32 * kt + 8 * j + 2 * sub);
                            m_t = fmaxf(m_t, fmaxf(y.x, y.y));
                        }
                    }
                }
                m_t = fmaxf(m_t, __shfl_xor_sync(0xffffffffu, m_t, 1));
                m_t = fmaxf(m_t, __shfl_xor_sync(0xffffffffu, m_t, 2));
                const float m_new = fmaxf(m_run, m_t);
                any = map_lane && m_new > -INFINITY;       // false: nothing but rows with a zero scale so far
                m_sub = any ? m_new : 0.f;
                alpha = any ? ex2f(m_run - m_new) : 1.f;
                m_run = any ? m_new : m_run;
            }
            // ---- (B) the weights of T / 8 tokens per warp (the exponentials and the conversions are the costly part
            //      of a sub-tile: each is done once per CTA, not once per warp) go to shared memory as the 16-bit halves
            //      of the fragment registers of the lanes that need them: lane (quad, s') holds, of k-step kt, the token
            //      pairs 32 kt + 8 j + 2 s' + {0, 1}, j = 0 .. 3, in {a0, a1, a2, a3} = {piece 1 of j = 0 | 1, piece 2 of
            //      j = 0 | 1, piece 1 of j = 2 | 3, piece 2 of j = 2 | 3}
            {
                const int ppw = T >> 4;                    // token pairs per warp
                float den = 0.f;
                if (sub < ppw) {
                    const int gp = warp * ppw + sub;       // token pair 2 gp, 2 gp + 1 of the sub-tile
                    float2 x = make_float2(-INFINITY, -INFINITY), y = x;
                    if (map_lane) {
                        x = *reinterpret_cast<const float2*>(sb + quad * T + 2 * gp);
                        y = *reinterpret_cast<const float2*>(sbw + quad * T + 2 * gp);
                    }
                    const float w0 = ex2f(y.x - m_sub) * 256.f, w1 = ex2f(y.y - m_sub) * 256.f;
                    den = any ? ex2f(x.x - m_sub) + ex2f(x.y - m_sub) : 0.f;
                    const uint32_t hi = ptx::cvt_e4m3x2(w0, w1);
                    const float2 back = ptx::e4m3x2_to_f32(hi);
                    const uint32_t lo = ptx::cvt_e4m3x2(w0 - back.x, w1 - back.y);
                    const int r = gp & 15, j = r >> 2;
                    uint16_t* wp = reinterpret_cast<uint16_t*>(w_buf + ((gp >> 4) * 8 + quad) * 4 + (r & 3));
                    wp[(j >> 1) * 4 + (j & 1)] = (uint16_t)hi;
                    wp[(j >> 1) * 4 + 2 + (j & 1)] = (uint16_t)lo;
                }
                den_buf[warp * 32 + lane] = den;
            }
            consumer_sync();
            uint32_t pa[KTM][4];
#pragma unroll
            for (int kt = 0; kt < KTM; ++kt) {
                const uint4 f = kt < KT ? w_buf[(kt * 8 + quad) * 4 + sub] : make_uint4(0u, 0u, 0u, 0u);
                pa[kt][0] = f.x; pa[kt][1] = f.y; pa[kt][2] = f.z; pa[kt][3] = f.w;
            }
            if (warp == 0) {                               // the row sum is kept (and written out) by warp 0 alone
                float sum = 0.f;
#pragma unroll
                for (int w8 = 0; w8 < 8; ++w8) sum += den_buf[w8 * 32 + lane];
                sum += __shfl_xor_sync(0xffffffffu, sum, 1);
                sum += __shfl_xor_sync(0xffffffffu, sum, 2);
                l_run = l_run * alpha + sum;
            }
#pragma unroll
            for (int n = 0; n < 2 * CH; ++n) { acc[n][0] *= alpha; acc[n][1] *= alpha; acc[n][2] *= alpha; acc[n][3] *= alpha; }

            // ---- latent sums of this warp's 16 CH columns, all maps and both pieces at once
#pragma unroll
            for (int kt = 0; kt < KTM; ++kt) {
                if (kt < KT) {
                    const int token = 32 * kt + 8 * mat + mrow;
#pragma unroll
                    for (int c = 0; c < CH; ++c) {
                        const int chunk = warp * CH + c;      // 16-byte chunk (16 columns) of the latent row
                        uint32_t r0, r1, r2, r3;
                        ptx::ldsm_x4_trans(stage + c_off + (chunk >> 3) * tile_bytes + token * 128 +
                                               (((chunk & 7) ^ (token & 7)) << 4), r0, r1, r2, r3);
                        // r_i: tokens 8 i + 2 sub + {0, 1} x columns 2 quad + {0, 1}
                        const uint32_t be0 = ptx::byte_perm(r0, r1, 0x6420u), be1 = ptx::byte_perm(r2, r3, 0x6420u);
                        const uint32_t bo0 = ptx::byte_perm(r0, r1, 0x7531u), bo1 = ptx::byte_perm(r2, r3, 0x7531u);
                        ptx::mma_e4m3_16832(acc[2 * c], pa[kt][0], pa[kt][1], pa[kt][2], pa[kt][3], be0, be1);
                        ptx::mma_e4m3_16832(acc[2 * c + 1], pa[kt][0], pa[kt][1], pa[kt][2], pa[kt][3], bo0, bo1);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&empty_bar[s]);
        }
        if (ok) flush(b);
        // A wait that gave up (it raises the CTA's abort flag, after which every wait returns at once): other consumer
        // warps may already stand at a CTA barrier of this or a later sub-tile, which needs all eight, so the warp
        // keeps its appointments -- two barriers per sub-tile -- to the end of the range before it leaves.
        for (; st < st_end; ++st) {
            consumer_sync();
            consumer_sync();
        }
    }
    __syncthreads();
    if (tid == 0 && *abort_flag) raise_status(status_word, GTA_ERR_TIMEOUT);
}

// k_new / c_new != nullptr: the fused append + decode step -- seq_lens does not count the new token yet, the stream
// kernel puts its rows into the caches and attends over them, the decoder kernel advances the lengths at the end.
cudaError_t launch_decode_fast(const Dims& d, const void* q, const void* k_cache, const void* c_cache,
                               const int32_t* seq_lens, int S_cap, const void* x_t, const void* w_p,
                               const void* w_g, void* out, void* workspace, int32_t* status_word,
                               cudaStream_t stream, int stages, int* launches, const PageMap& pm, const void* k_new,
                               const void* c_new) {
    const FastPlan p = make_fast_plan(d);
    float* part_o = reinterpret_cast<float*>(workspace);
    float* part_ml = reinterpret_cast<float*>(static_cast<char*>(workspace) + p.off_ml);
    __nv_bfloat16* l_g = reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(workspace) + p.off_l);
    cudaError_t err = launch_stream_and_merge(d, p, q, k_cache, c_cache, seq_lens, S_cap, part_o, part_ml, l_g,
                                              (long long)d.B * d.d_l, d.d_l, status_word, stream, stages, launches, pm,
                                              k_new, c_new);
    if (err != cudaSuccess) return err;
    if (stages & 4) {
        // the batch takes the role of the token axis: L [n_q][B][d_l], x_t [B][H], out [B][n_h][d_h]
        Dims dd = d;
        dd.B = 1;
        dd.N = d.B;
        if (launch_sm100_decoder(dd, l_g, x_t, w_p, w_g, out, status_word, stream,
                                 k_new ? const_cast<int32_t*>(seq_lens) : nullptr, d.B, S_cap) != GTA_OK)
            return cudaErrorUnknown;
        *launches += 1;
    }
    return cudaSuccess;
}

// ---------------------------------------------------------------------------------------------
// One decode step over 8-bit caches on the stream kernel above, the merge kernel and the tcgen05 decoder kernel.
bool decode_fp8_fast_supported(const Dims& d, int dtype, int S_cap) {
    if (dtype != GTA_BF16 || d.d_h != 128 || d.n_c != 1) return false;
    if (d.d_l != 128 && d.d_l != 256 && d.d_l != 512 && d.d_l != 1024) return false;
    if (d.n_q < 1 || d.n_q > 8) return false;
    if (d.n_k != 1 && d.n_k != 2 && d.n_k != 4 && d.n_k != 8) return false;
    if (d.H % 64 != 0 || d.B > kStreamMaxBatch) return false;
    if (S_cap % 4 != 0) return false;                           // scale rows are copied in 16-byte pieces
    if (((d.n_h / d.n_q) * d.d_h) % (d.B > 128 ? 128 : 64) != 0) return false;
    return (d.n_k * 128 + d.d_l) * 32 <= kStreamStageBytes;     // a 32-token sub-tile fits a ring stage
}

static FastPlan make_fp8_plan(const Dims& d) {
    FastPlan p;
    const int tok_bytes = d.n_k * 128 + d.d_l;
    p.occ = 1;
    p.T = tok_bytes * 64 <= kStreamStageBytes ? 64 : 32;
    const int ctas = sm_count();
    p.G = ctas < kFinMaxSlots - kStreamMaxBatch ? ctas : kFinMaxSlots - kStreamMaxBatch;
    p.slots = p.G + d.B;
    p.off_ml = align256f((size_t)p.slots * d.n_q * d.d_l * sizeof(float));
    p.off_l = p.off_ml + align256f((size_t)p.slots * d.n_q * 2 * sizeof(float));
    p.total = p.off_l + align256f((size_t)d.n_q * d.B * d.d_l * sizeof(__nv_bfloat16));
    return p;
}

size_t decode_fp8_fast_workspace_bytes(const Dims& d) { return make_fp8_plan(d).total; }

cudaError_t launch_decode_fp8_fast(const Dims& d, const void* q, const void* k_codes, const void* c_codes,
                                   const float* k_scale, const float* c_scale, const int32_t* seq_lens, int S_cap,
                                   const void* x_t, const void* w_p, const void* w_g, void* out, void* workspace,
                                   int32_t* status_word, cudaStream_t stream, int* launches) {
    const FastPlan p = make_fp8_plan(d);
    float* part_o = reinterpret_cast<float*>(workspace);
    float* part_ml = reinterpret_cast<float*>(static_cast<char*>(workspace) + p.off_ml);
    __nv_bfloat16* l_g = reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(workspace) + p.off_l);
    cudaError_t err;
    if (decode_fp8_tc_supported(d, p.T)) {     // the tokens as the rows of tcgen05 MMAs
        err = launch_decode_fp8_tc_stream(d, p.G, p.T, S_cap, q, k_codes, c_codes, k_scale, c_scale, seq_lens, part_o, part_ml,
                                          status_word, stream);
        if (err != cudaSuccess) return err;
        *launches += 1;
    } else {
        CUtensorMap tm_k, tm_c;
        const uint32_t box[3] = {128, (uint32_t)p.T, 1};
        const uint64_t dk[3] = {128, (uint64_t)S_cap, (uint64_t)d.B * d.n_k};
        const uint64_t dc[3] = {(uint64_t)d.d_l, (uint64_t)S_cap, (uint64_t)d.B};
        if (!make_u8_map(&tm_k, k_codes, 3, dk, box) || !make_u8_map(&tm_c, c_codes, 3, dc, box))
            return cudaErrorInvalidValue;
        const int CH = d.d_l / 128;
        const size_t stage = (size_t)(d.n_k + CH) * p.T * 128 + ((((size_t)d.n_k + 1) * p.T * 4 + 1023) & ~(size_t)1023);
        const size_t smem = kStreamStages * stage + 4 * 8 * kStreamMaxT * sizeof(float) +      // scores, shifted scores
                            (kStreamMaxT / 32) * 32 * 16 + 256 * sizeof(float) +               // weight fragments, row-sum shares
                            (size_t)(kStreamMaxBatch + 2 + kStreamThreads) * sizeof(int32_t) +
                            2 * kStreamStages * sizeof(uint64_t) + 16 + 1024;
#define GTA_LAUNCH_FP8(CHV)                                                                                \
        do {                                                                                               \
            auto kern = decode_stream_fp8_kernel<CHV>;                                                     \
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
            err = cudaLaunchKernelEx(&cfg, kern, tm_k, tm_c, d, p.T, S_cap, (const __nv_bfloat16*)q, k_scale, \
                                     c_scale, seq_lens, part_o, part_ml, status_word);                     \
            if (err != cudaSuccess) return err;                                                            \
        } while (0)
        switch (CH) {
            case 1: GTA_LAUNCH_FP8(1); break;
            case 2: GTA_LAUNCH_FP8(2); break;
            case 4: GTA_LAUNCH_FP8(4); break;
            default: GTA_LAUNCH_FP8(8); break;
        }
#undef GTA_LAUNCH_FP8
        if ((err = cudaGetLastError()) != cudaSuccess) return err;
        *launches += 1;
    }
    {
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
                                 (const float*)part_ml, l_g, (long long)d.B * d.d_l, (long long)d.d_l, 0);
        if (err != cudaSuccess) return err;
        *launches += 1;
    }
    Dims dd = d;      // the batch takes the role of the token axis
    dd.B = 1;
    dd.N = d.B;
    if (launch_sm100_decoder(dd, l_g, x_t, w_p, w_g, out, status_word, stream) != GTA_OK) return cudaErrorUnknown;
    *launches += 1;
    return cudaSuccess;
}

// ---------------------------------------------------------------------------------------------
// Comparison operator (App. B.3, GQA; one key / value head per query head gives the multi-head attention of
// Sec. 3.1): one decode step on the same stream and merge kernels.  Every (sequence, key / value head) pair
// is streamed as a sequence of its own whose maps are the n_h / n_kv query heads that share the head, whose
// key group is the head's K rows and whose "latent" is the head's V rows (d_h wide); no decoder, no gate:
// the merged, normalised rows ARE the output [B, n_h, d_h].
__global__ void gqa_expand_lens_kernel(const int32_t* __restrict__ seq_lens, int32_t* __restrict__ out, int B, int n_kv) {
    ptx::grid_dependency_wait();          // the lengths may come from the kernel before (an append)
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < B * n_kv) out[i] = seq_lens[i / n_kv];
}

static Dims gqa_stream_dims(int B, int n_h, int n_kv, int d_h, float scale) {
    Dims d = {};
    d.B = B * n_kv; d.N = 0; d.H = 64; d.n_h = n_h / n_kv; d.n_q = n_h / n_kv; d.n_k = 1; d.n_c = 1;
    d.d_h = d_h; d.d_l = d_h; d.causal = 1; d.scale = scale; d.Nk = 0; d.S = 0;
    return d;
}

bool gqa_decode_supported(int B, int n_h, int n_kv, int d_h, int dtype) {
    if (dtype != GTA_BF16 || n_kv < 1 || n_h % n_kv != 0 || (d_h != 64 && d_h != 128)) return false;
    const int r = n_h / n_kv;
    return r >= 1 && r <= 8 && (long long)B * n_kv <= kStreamMaxBatch;
}

size_t gqa_decode_workspace_bytes(int B, int n_h, int n_kv, int d_h) {
    const Dims d = gqa_stream_dims(B, n_h, n_kv, d_h, 1.f);
    return make_fast_plan(d).off_l + align256f((size_t)d.B * sizeof(int32_t));
}

cudaError_t launch_gqa_decode(int B, int n_h, int n_kv, int d_h, float scale, const void* q, const void* k_cache,
                              const void* v_cache, const int32_t* seq_lens, int S_cap, void* out, void* workspace,
                              int32_t* status_word, cudaStream_t stream, int* launches) {
    const Dims d = gqa_stream_dims(B, n_h, n_kv, d_h, scale);
    const FastPlan p = make_fast_plan(d);
    float* part_o = reinterpret_cast<float*>(workspace);
    float* part_ml = reinterpret_cast<float*>(static_cast<char*>(workspace) + p.off_ml);
    int32_t* lens = reinterpret_cast<int32_t*>(static_cast<char*>(workspace) + p.off_l);
    {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((d.B + 255) / 256);
        cfg.blockDim = dim3(256);
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cudaError_t err = cudaLaunchKernelEx(&cfg, gqa_expand_lens_kernel, seq_lens, lens, B, n_kv);
        if (err != cudaSuccess) return err;
        *launches += 1;
    }
    // row (g, b') of the merge = query head j r + g of sequence b, b' = b n_kv + j: out + (b' r + g) d_h
    return launch_stream_and_merge(d, p, q, k_cache, v_cache, lens, S_cap, part_o, part_ml,
                                   static_cast<__nv_bfloat16*>(out), d.d_l, (long long)d.n_q * d.d_l, status_word, stream,
                                   6, launches, PageMap());
}

}  // namespace gta
