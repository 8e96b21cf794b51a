// The decode stream kernel for bf16 caches on the tcgen05 tensor pipe (App. B.1.3: one query row per map against
// the K cache and the latent C cache; a decode step is bound by the bytes of those caches).
//
// Both contractions are TRANSPOSED so that the cached tokens, not the handful of attention maps, fill the 128 rows
// of a tcgen05.mma (kind::f16, bf16 operands, K = 16), and the cache rows go from HBM through TMA into shared memory
// and from there into the tensor pipe without passing a register:
//
//   scores   S^T [key group, token][map] = K tiles [key group, token][d_h]  x  Q^T [map][d_h]
//            The K tiles of a sub-tile of T tokens lie back to back per 64-column half, key group after key group,
//            so the 128 rows of A are the T tokens of 128 / T consecutive key groups.  A thread (= a TMEM lane)
//            reads the scores of its (key group, token) for the maps of that key group as a few columns.
//   sums     O^T [latent column][map] += C tile^T [column][token]  x  P^T [map][token]
//            A = two 64-column halves of the latent tile as they lie in shared memory, read MN-major; B = the
//            weights written by the token threads; the accumulators (d_l / 128 blocks of 16 columns) stay in
//            tensor memory over all sub-tiles of a sequence.
//
// Warps 0-3 (group A, one per TMEM lane quarter): read a sub-tile's scores, keep the reference maxima (raised only
// when a sub-tile exceeds them by more than 2^8), leave the exponents in shared memory.  Warps 4-7 (group B):
// exponentials, the weights into the B operand, rescaling of the sums when a maximum was raised, clearing of latent
// rows past the length, the partial result at the end of a sequence.  A works on sub-tile i + 1 while B works on i.
// Warp 8: TMA producer.  Warp 9: MMA issue; in the fused append + decode step its lanes also put the new token's
// rows over the last row of the sequence's last sub-tile (in shared memory and in the caches) before the scores of
// that sub-tile are issued.  The token threads run one warp per scheduler, at the latency of every instruction:
// sub-tile size, key groups, maps per group and latent blocks are template parameters so that their loops unroll.
//
// Schedule (equal sub-tile ranges per CTA over the live tokens of all sequences), partial results (slot c + b:
// reference maximum, row sum, unnormalised latent sums) and the step's lengths are those of decode_stream_kernel,
// so decode_merge_kernel and the decoder kernel follow unchanged.
#include "gta_common.cuh"
#include "gta_sm100.cuh"
#include "sm100_ptx.cuh"
#include "tma_host.cuh"

namespace gta {
namespace {

// Test hooks of the bounded waits (gta_debug_decode_wait): the time limit of every wait of this kernel, and a switch
// that makes one warp of group B keep its very first arrival to itself, so that the MMA warp runs into that limit and
// the whole unwinding path can be exercised on a healthy GPU.  Read once per thread at kernel start.
__device__ unsigned long long g_bt_wait_limit_ns = ptx::kWaitLimitNs;
__device__ int g_bt_withhold_first_arrive = 0;

constexpr int kBtStages = 3;
constexpr int kBtThreads = 320;
constexpr int kBtMaxBatch = 512;
constexpr uint32_t kBtOperand = 16 * 128;       // bytes of a [16 rows][128 bytes] B operand panel
constexpr uint32_t kBtTmemCols = 256;           // 2 x 32 score columns at 0, up to 128 sum columns at 128
constexpr float kBtLag = 8.f;                   // a reference maximum may lag the true one by 2^8

__device__ __forceinline__ float bt_ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// byte offset of (row, byte column) in a [rows][128 bytes] operand with the 128-byte swizzle
__device__ __forceinline__ uint32_t bt_swz(int row, int col) {
    return (uint32_t)row * 128u + ((((uint32_t)col >> 4) ^ ((uint32_t)row & 7u)) << 4) + ((uint32_t)col & 15u);
}
// Length a decode step attends over (as in decode_stream_kernel): with `append` the stored length does not count the
// new token yet; a sequence with room for it attends over len + 1 tokens, a full or invalid one is left as it is.
struct BtLens {
    const int32_t* seq_lens;
    int S_cap, append;
    __device__ __forceinline__ bool appends(int b) const {
        const int len = seq_lens[b];
        return append && len >= 0 && len < S_cap;
    }
    __device__ __forceinline__ int len(int b) const {
        const int len = seq_lens[b];
        return (len < 0 ? 0 : (len > S_cap ? S_cap : len)) + (appends(b) ? 1 : 0);
    }
};

struct BtSmem {
    uint32_t stage_stride, c_off, q_off, p_off, e_off, misc_off, total;
};
__host__ __device__ inline BtSmem bt_smem_layout(int T, int n_k, int ch) {
    BtSmem s;
    const uint32_t tb = (uint32_t)T * 128;
    s.c_off = 2u * n_k * tb;                          // K: [2 halves][n_k][T][128 B]; C: [2 ch halves][T][128 B]
    s.stage_stride = (s.c_off + 2u * ch * tb + 1023u) & ~1023u;
    s.q_off = kBtStages * s.stage_stride;             // [2 sequence parities][2 halves][16][128 B]
    s.p_off = s.q_off + 4 * kBtOperand;               // [2 sub-tile parities][16][128 B]
    s.e_off = s.p_off + 2 * kBtOperand;               // exponents [2 parities][8 maps][64 tokens] floats
    s.misc_off = s.e_off + 2 * 8 * 64 * 4;
    // prefix [B + 2] | scan [threads] | mx [2][16][8] | l_red [16][8] | hdr [2][24] | 24 barriers | 4 words
    s.total = s.misc_off + (kBtMaxBatch + 2 + kBtThreads) * 4 + (256 + 128 + 48) * 4 + 24 * 8 + 16 + 1024;
    return s;
}

template <int T, int NK, int QPK, int CH>
__global__ void __launch_bounds__(kBtThreads, 1)
decode_stream_tc_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_c, Dims d,
                        int S_cap, const __nv_bfloat16* __restrict__ q, const int32_t* __restrict__ seq_lens,
                        float* __restrict__ part_o, float* __restrict__ part_ml, int32_t* status_word,
                        const uint4* __restrict__ k_new, const uint4* __restrict__ c_new, uint4* __restrict__ k_rows,
                        uint4* __restrict__ c_rows, const PageMap pm) {
    constexpr int NQ = NK * QPK;
    constexpr int R = 128 / T;                        // key groups on the rows of one score MMA
    constexpr int SETS = (NK + R - 1) / R;
    constexpr int kSeg = T < 32 ? T : 32;             // lanes that share a (key group, 32-token stretch)
    constexpr uint32_t tb = T * 128;
    static_assert(NQ <= 8 && SETS <= 2 && CH <= 8, "instantiation outside the kernel's limits");
    const BtLens L{seq_lens, S_cap, k_new != nullptr};
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const BtSmem lay = bt_smem_layout(T, NK, CH);
    uint8_t* ring = smem;
    uint8_t* q_buf = smem + lay.q_off;
    uint8_t* p_buf = smem + lay.p_off;
    float* e_buf = reinterpret_cast<float*>(smem + lay.e_off);               // [2 parities][8 maps][64 tokens]
    int32_t* prefix = reinterpret_cast<int32_t*>(smem + lay.misc_off);       // [B + 1]
    int32_t* scan_tmp = prefix + kBtMaxBatch + 2;                             // [kBtThreads]
    float* mx_buf = reinterpret_cast<float*>(scan_tmp + kBtThreads);          // [2 parities][16 key groups][8 maps per group]
    float* l_red = mx_buf + 256;                                              // [16 (set, segment)][8 maps per group]
    float* hdr = l_red + 128;                                                 // [2 parities][8 alpha | 8 maxima | grow | -]
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(hdr + 48);               // [3] TMA bytes of a stage have landed
    uint64_t* empty_bar = full_bar + kBtStages;                               // [3] the sums of its sub-tile are complete
    uint64_t* s_ready = empty_bar + kBtStages;                                // [2] scores of sub-tile i are in buffer i & 1
    uint64_t* p_ready = s_ready + 2;                                          // [2] 4 warps of B: weights written, O rescaled
    uint64_t* pv_done = p_ready + 2;                                          // [2] the sums of sub-tile i are complete
    uint64_t* q_ready = pv_done + 2;                                          // [2] 4 warps of A: queries of sequence n in buffer n & 1
    uint64_t* s_free = q_ready + 2;                                           // [2] 4 warps of A: the scores have been read
    uint64_t* xy_ready = s_free + 2;                                          // [2] 4 warps of A: exponents and header of sub-tile i
    uint64_t* xy_free = xy_ready + 2;                                         // [2] 4 warps of B: ... have been read
    uint64_t* drain_bar = xy_free + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain_bar + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile int* drain_flag = abort_flag + 1;
    const uint64_t wait_limit = g_bt_wait_limit_ns;
    const bool withhold_first_arrive = g_bt_withhold_first_arrive != 0;
    // every wait of this kernel: bounded by wait_limit, ended early by the CTA's abort flag
    auto wait = [&](uint64_t* bar, uint32_t parity) { return ptx::mbar_wait_sleep(bar, parity, abort_flag, 0, wait_limit); };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int G = gridDim.x, cta = blockIdx.x;

    if (tid == 0) {
        for (int s = 0; s < kBtStages; ++s) { ptx::mbar_init(&full_bar[s], 1); ptx::mbar_init(&empty_bar[s], 1); }
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(&s_ready[s], 1); ptx::mbar_init(&p_ready[s], 4);
            ptx::mbar_init(&pv_done[s], 1); ptx::mbar_init(&q_ready[s], 4);
            ptx::mbar_init(&s_free[s], 4); ptx::mbar_init(&xy_ready[s], 4); ptx::mbar_init(&xy_free[s], 4);
        }
        ptx::mbar_init(drain_bar, 1);
        *abort_flag = 0;
        *drain_flag = 0;
        ptx::fence_mbar_init();
    }
    if (warp == 8 && lane == 0) {
        ptx::prefetch_tensormap(&tm_k);
        ptx::prefetch_tensormap(&tm_c);
    }
    if (warp == 9) ptx::tmem_alloc(tmem_slot, kBtTmemCols);
    // rows of the B operands that belong to no map stay zero for the whole kernel
    for (uint32_t i = tid; i < 6 * kBtOperand / 16; i += kBtThreads)
        reinterpret_cast<uint4*>(q_buf)[i] = make_uint4(0u, 0u, 0u, 0u);
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // launched with programmatic stream serialisation: nothing of global memory is read before the kernel ahead is
    // complete, and only then may the kernels behind this one be scheduled
    ptx::grid_dependency_wait();
    ptx::grid_launch_dependents();

    {   // exclusive prefix sum of the sub-tile counts (as in the other stream kernels)
        const int per = (d.B + kBtThreads - 1) / kBtThreads;
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
        __syncthreads();
        int base = incl - sum;
        for (int w = 0; w < warp; ++w) base += scan_tmp[w];
        for (int b = lo; b < hi; ++b) {
            prefix[b] = base;
            base += (L.len(b) + T - 1) / T;
        }
        if (tid == kBtThreads - 1) prefix[d.B] = base;
        __syncthreads();
    }
    if (L.append && cta == 0) {      // a sequence without room for the new token is left as it is and reported
        for (int b = tid; b < d.B; b += kBtThreads)
            if (!L.appends(b)) raise_status(status_word, GTA_ERR_CACHE_FULL);
    }
    const long long n_st = prefix[d.B];
    const long long st_begin = ((long long)cta * n_st) / G, st_end = ((long long)(cta + 1) * n_st) / G;
    const int n_sub = (int)(st_end - st_begin);      // sub-tiles of this CTA
    int b0 = 0;
    if (n_sub > 0) {
        int lo = 0, hi = d.B - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (prefix[mid] <= st_begin) lo = mid; else hi = mid - 1;
        }
        b0 = lo;
    }
    const int k0 = n_sub > 0 ? (int)(st_begin - prefix[b0]) : 0;     // first sub-tile of sequence b0 in this range
    const uint32_t ring_addr = ptx::smem_addr(ring);

    if (n_sub > 0 && warp == 8) {
        // ------------------------------------------------------------------ producer: one load per lane
        const uint64_t policy = ptx::l2_evict_first_policy();
        constexpr int n_ops = 2 * NK + 2 * CH;
        int b = b0, k = k0, it = 0;
        bool ok = true;
        for (; it < n_sub; ++it, ++k) {
            while (k >= prefix[b + 1] - prefix[b]) { ++b; k = 0; }
            const int s = it % kBtStages;
            const uint32_t ph = (it / kBtStages) & 1;
            // Contiguous caches: rows tok0 .. of plane b groups + g.  Paged pool: the sub-tile lies inside one page
            // (T divides the page size), at rows tok0 % page_size .. of plane page groups + g; the block-table entry
            // is fetched before the wait for the stage.  An entry outside the pool raises the status word, and the
            // load (of page 0 then) still completes the stage.
            int tok0 = k * T, plane = b;
            if (pm.table != nullptr) {
                const int page = page_of(pm, b, tok0, lane == 0 ? status_word : nullptr);
                plane = page < 0 ? 0 : page;
                tok0 %= pm.page_size;
            }
            if (lane == 0) {
                ok = wait(&empty_bar[s], ph ^ 1);
                if (ok) ptx::mbar_arrive_expect_tx(&full_bar[s], (uint32_t)n_ops * tb);
            }
            ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
            if (!ok) break;
            uint8_t* stage = ring + s * lay.stage_stride;
            for (int op = lane; op < n_ops; op += 32) {
                if (op < 2 * NK)        // half op / NK of key group op % NK
                    ptx::tma_load_3d_hint(stage + op * tb, &tm_k, &full_bar[s], (op / NK) * 64, tok0, plane * NK + op % NK, policy);
                else
                    ptx::tma_load_3d_hint(stage + op * tb, &tm_c, &full_bar[s], (op - 2 * NK) * 64, tok0, plane, policy);
            }
        }
        if (lane == 0 && *abort_flag) {
            for (int back = 1; back <= kBtStages && it - back >= 0; ++back) {
                const int iq = it - back;
                ptx::mbar_wait_drain(&full_bar[iq % kBtStages], (iq / kBtStages) & 1, drain_flag);
            }
        }
    } else if (n_sub > 0 && warp == 9) {
        // ------------------------------------------------------------------ MMA issue (lane 0) and the append
        constexpr uint32_t idesc_s = ptx::make_idesc_bf16(128, 16, 0, 0);    // key tiles and queries, both K-major
        constexpr uint32_t idesc_o = ptx::make_idesc_bf16(128, 16, 1, 0);    // latent tile MN-major, weights K-major
        const uint64_t desc_kmajor = ptx::make_smem_desc(0, 16, 1024);
        const uint64_t desc_latent = ptx::make_smem_desc(0, tb, 1024);       // the next 64 columns one tile further on
        const uint32_t q_addr = ptx::smem_addr(q_buf), p_addr = ptx::smem_addr(p_buf);
        const uint32_t tmem_o = tmem_base + 128;
        bool ok = true;
        int sb = b0, sk = k0, sn = 0;        // for the scores (one sub-tile ahead of the sums)
        int pb = b0, pk = k0;                // for the sums
        auto issue_scores = [&](int j) -> bool {
            bool first = (j == 0);
            while (sk >= prefix[sb + 1] - prefix[sb]) { ++sb; sk = 0; first = true; }
            if (first && j > 0) ++sn;
            const int s = j % kBtStages;
            // (every lane of the warp waits: its lanes share the append below; the outcome is made uniform)
            bool w = !first || wait(&q_ready[sn & 1], (sn >> 1) & 1);
            w = w && wait(&full_bar[s], (j / kBtStages) & 1);
            // the buffer held the scores of sub-tile j - 2
            w = w && (j < 2 || wait(&s_free[j & 1], ((j >> 1) - 1) & 1));
            if (!__all_sync(0xffffffffu, w)) return false;
            const uint32_t stage = ring_addr + s * lay.stage_stride;
            // the sub-tile that ends a sequence of the fused step holds the new token (its last live row): what TMA
            // brought for that row is whatever the cache held; the new rows are put over it and written to the caches
            if (L.append) {
                const int len = L.len(sb);
                if (L.appends(sb) && (sk + 1) * T >= len) {
                    const int row = len - 1 - sk * T;
                    uint8_t* st = ring + s * lay.stage_stride;
                    for (int v = lane; v < 16 * NK + 16 * CH; v += 32) {
                        const int chunk = v & 7;
                        if (v < 16 * NK) {       // key group kg, half h: 8 vectors
                            const int kg = v >> 4, h = (v >> 3) & 1;
                            const uint4 nv = __ldg(k_new + ((size_t)sb * NK + kg) * 16 + h * 8 + chunk);
                            *reinterpret_cast<uint4*>(st + (h * NK + kg) * tb + row * 128 + ((chunk ^ (row & 7)) << 4)) = nv;
                            k_rows[(((size_t)sb * NK + kg) * S_cap + (len - 1)) * 16 + h * 8 + chunk] = nv;
                        } else {                 // 64-column half c of the latent row
                            const int c = (v - 16 * NK) >> 3;
                            const uint4 nv = __ldg(c_new + (size_t)sb * (16 * CH) + c * 8 + chunk);
                            *reinterpret_cast<uint4*>(st + lay.c_off + c * tb + row * 128 + ((chunk ^ (row & 7)) << 4)) = nv;
                            c_rows[((size_t)sb * S_cap + (len - 1)) * (16 * CH) + c * 8 + chunk] = nv;
                        }
                    }
                    ptx::fence_proxy_async_smem();
                }
            }
            __syncwarp();
            ptx::tc_fence_after_sync();
            if (lane == 0) {
#pragma unroll
                for (int set = 0; set < SETS; ++set) {
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        // 128 rows: the T tokens of key groups set R .. set R + R - 1 (behind the last key tile come
                        // other rows of the stage, whose "scores" nobody reads)
                        const uint64_t dk = desc_kmajor + ((stage + (h * NK + set * R) * tb) >> 4);
                        const uint64_t dq = desc_kmajor + ((q_addr + ((sn & 1) * 2 + h) * kBtOperand) >> 4);
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)      // 16 elements = 32 bytes of the 128-byte rows per step
                            ptx::mma_ss(tmem_base + (j & 1) * 32 + set * 16, dk + 2 * ks, dq + 2 * ks, idesc_s,
                                        (h > 0 || ks > 0) ? 1u : 0u);
                    }
                }
                ptx::tc_commit(&s_ready[j & 1]);
            }
            ++sk;
            return true;
        };
        ok = issue_scores(0);
        for (int i = 0; i < n_sub && ok; ++i) {
            // the scores of the next sub-tile go into the other buffer, once group A has read it
            if (i + 1 < n_sub) ok = issue_scores(i + 1);
            if (!ok) break;
            bool first = (i == 0);
            while (pk >= prefix[pb + 1] - prefix[pb]) { ++pb; pk = 0; first = true; }
            ++pk;
            ok = __all_sync(0xffffffffu, wait(&p_ready[i & 1], (i >> 1) & 1));
            if (!ok) break;
            ptx::tc_fence_after_sync();
            if (lane == 0) {
                const int s = i % kBtStages;
                const uint32_t stage = ring_addr + s * lay.stage_stride;
                const uint64_t dp = desc_kmajor + ((p_addr + (i & 1) * kBtOperand) >> 4);
#pragma unroll
                for (int c = 0; c < CH; ++c) {
                    const uint64_t dc = desc_latent + ((stage + lay.c_off + 2 * c * tb) >> 4);
#pragma unroll
                    for (int kk = 0; kk < T / 16; ++kk)      // 16 tokens = 2048 bytes of a tile, 32 bytes of the weights' rows
                        ptx::mma_ss(tmem_o + c * 16, dc + kk * (2048 >> 4), dp + 2 * kk, idesc_o, (first && kk == 0) ? 0u : 1u);
                }
                ptx::tc_commit(&pv_done[i & 1]);
                ptx::tc_commit(&empty_bar[s]);
            }
            __syncwarp();
        }
        if (lane == 0 && *abort_flag) {      // unwinding: the MMAs issued so far must be complete before tensor memory is freed
            ptx::tc_commit(drain_bar);
            ptx::mbar_wait_drain(drain_bar, 0, drain_flag);
        }
    } else if (n_sub > 0 && warp < 8) {
        // ------------------------------------------------------------------ groups A and B
        // TMEM lane l = 32 quarter + lane: scores of key group (set R + l / T), token l % T; sums: latent column l of
        // each 128-column block.  A thread of B takes over the (key group, token) of the thread of A in the same place.
        const bool group_b = warp >= 4;
        const int quarter = warp & 3;
        const int gtid = tid & 127;
        const uint32_t lane_base = ((uint32_t)(quarter * 32) << 16);
        const uint32_t tmem_o = tmem_base + 128 + lane_base;
        const int gsel = gtid / T, token = gtid % T;
        const int seg = gtid / kSeg;                     // 32-token stretch of a key group (or the whole of it)
        const float q_mul = d.scale * 1.4426950408889634f;
        int b = b0, k = k0, n = 0;          // sequence, its sub-tile, its ordinal in this range
        int len_b = L.len(b), n_sub_b = prefix[b + 1] - prefix[b];
        bool ok = true, first = true;

        if (!group_b) {
            // the queries of sequence b into buffer par: warp w takes the maps 2 w and 2 w + 1, a lane four elements
            auto write_q = [&](int bq, int par) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int g = 2 * quarter + h;
                    if (g < NQ) {
                        const uint2 raw = __ldg(reinterpret_cast<const uint2*>(q + ((size_t)bq * NQ + g) * 128 + 4 * lane));
                        // element 4 lane: half (lane >> 4), byte column 8 (lane & 15) of row g
                        *reinterpret_cast<uint2*>(q_buf + (par * 2 + (lane >> 4)) * kBtOperand + bt_swz(g, 8 * (lane & 15))) = raw;
                    }
                }
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&q_ready[par]);
            };
            // the next sequence after bq that has sub-tiles in this range (-1: none)
            auto next_seq = [&](int bq) {
                int nb = bq + 1;
                while (nb < d.B && prefix[nb + 1] == prefix[nb]) ++nb;
                return (nb < d.B && prefix[nb] < st_end) ? nb : -1;
            };
            float m_run[8];
#pragma unroll
            for (int g = 0; g < 8; ++g) m_run[g] = -INFINITY;
            write_q(b, 0);
            for (int i = 0; i < n_sub; ++i, ++k) {
                if (k >= n_sub_b) {
                    do { ++b; } while (prefix[b + 1] == prefix[b]);
                    k = 0;
                    ++n;
                    first = true;
                    len_b = L.len(b);
                    n_sub_b = prefix[b + 1] - prefix[b];
#pragma unroll
                    for (int g = 0; g < 8; ++g) m_run[g] = -INFINITY;
                }
                if (first) {    // the buffer of the sequence before this one is free: every score of it has been read
                    const int nb = next_seq(b);
                    if (nb >= 0) write_q(nb, (n + 1) & 1);
                }
                const int n_valid = min(T, len_b - k * T);
                ok = wait(&s_ready[i & 1], (i >> 1) & 1) && ok;
                ptx::tc_fence_after_sync();

                // ---- this (key group, token)'s scores of the key group's maps, in log2 units
                uint32_t r[SETS][16];
#pragma unroll
                for (int set = 0; set < SETS; ++set) ptx::tmem_ld16(tmem_base + lane_base + (i & 1) * 32 + set * 16, r[set]);
                ptx::tmem_wait_ld();
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&s_free[i & 1]);
                const bool live = token < n_valid;
                float x[SETS][QPK];
#pragma unroll
                for (int set = 0; set < SETS; ++set) {
#pragma unroll
                    for (int j = 0; j < QPK; ++j) {
                        float v = -INFINITY;
#pragma unroll
                        for (int gs = 0; gs < R; ++gs)
                            if (set * R + gs < NK && gs == gsel) v = __uint_as_float(r[set][(set * R + gs) * QPK + j]) * q_mul;
                        x[set][j] = live ? v : -INFINITY;
                        float m = x[set][j];
#pragma unroll
                        for (int o = kSeg / 2; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
                        // (set, segment) -> key group set R + seg kSeg / T, stretch seg % (T / kSeg)
                        if ((gtid & (kSeg - 1)) == 0) mx_buf[(((i & 1) * 2 + set) * (128 / kSeg) + seg) * 8 + j] = m;
                    }
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");

                // ---- the reference maxima: raised only when the sub-tile exceeds them by more than kBtLag
                float alpha[8], m_sub[8];
                bool grow = false;
#pragma unroll
                for (int g = 0; g < 8; ++g) {
                    alpha[g] = 1.f;
                    m_sub[g] = 0.f;
                    if (g < NQ) {
                        constexpr int spg = T / kSeg;                        // segments per key group
                        const int kg = g / QPK, set = kg / R, s0 = (kg % R) * spg;
                        float m_tile = mx_buf[(((i & 1) * 2 + set) * (128 / kSeg) + s0) * 8 + g % QPK];
                        if (spg == 2) m_tile = fmaxf(m_tile, mx_buf[(((i & 1) * 2 + set) * (128 / kSeg) + s0 + 1) * 8 + g % QPK]);
                        const bool up = m_tile > m_run[g] + kBtLag;
                        grow = grow || up;
                        alpha[g] = up ? bt_ex2(m_run[g] - m_tile) : 1.f;
                        m_run[g] = up ? m_tile : m_run[g];
                        m_sub[g] = m_run[g] > -INFINITY ? m_run[g] : 0.f;
                    }
                }
                // ---- hand-over to group B (the buffers of sub-tile i - 2 have been read)
                if (i >= 2) ok = wait(&xy_free[i & 1], ((i >> 1) - 1) & 1) && ok;
#pragma unroll
                for (int set = 0; set < SETS; ++set) {
                    const int kg = set * R + gsel;
                    if (kg < NK) {
#pragma unroll
                        for (int j = 0; j < QPK; ++j) {
                            float ms = 0.f;
#pragma unroll
                            for (int g = 0; g < 8; ++g) if (g < NQ && g == kg * QPK + j) ms = m_sub[g];
                            e_buf[((i & 1) * 8 + kg * QPK + j) * 64 + token] = x[set][j] - ms;
                        }
                    }
                }
                if (gtid < 8) {
                    float a = 1.f, m = -INFINITY;
#pragma unroll
                    for (int g = 0; g < 8; ++g) if (g == gtid) { a = alpha[g]; m = m_run[g]; }
                    hdr[(i & 1) * 24 + gtid] = a;
                    hdr[(i & 1) * 24 + 8 + gtid] = m;
                    if (gtid == 0) hdr[(i & 1) * 24 + 16] = grow ? 1.f : 0.f;
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&xy_ready[i & 1]);
                first = false;
            }
        } else {
            float l_own[SETS][QPK], m_cur[8];
#pragma unroll
            for (int set = 0; set < SETS; ++set)
#pragma unroll
                for (int j = 0; j < QPK; ++j) l_own[set][j] = 0.f;
#pragma unroll
            for (int g = 0; g < 8; ++g) m_cur[g] = -INFINITY;
            for (int i = 0; i < n_sub; ++i, ++k) {
                if (k >= n_sub_b) {
                    do { ++b; } while (prefix[b + 1] == prefix[b]);
                    k = 0;
                    first = true;
                    len_b = L.len(b);
                    n_sub_b = prefix[b + 1] - prefix[b];
                }
                const int s = i % kBtStages;
                const int n_valid = min(T, len_b - k * T);
                uint8_t* stage = ring + s * lay.stage_stride;
                ok = wait(&xy_ready[i & 1], (i >> 1) & 1) && ok;
                float alpha[8];
#pragma unroll
                for (int g = 0; g < 8; ++g) {
                    alpha[g] = g < NQ ? hdr[(i & 1) * 24 + g] : 1.f;
                    m_cur[g] = g < NQ ? hdr[(i & 1) * 24 + 8 + g] : -INFINITY;
                }
                const bool grow = hdr[(i & 1) * 24 + 16] != 0.f;
                float e[SETS][QPK];
#pragma unroll
                for (int set = 0; set < SETS; ++set) {
                    const int kg = set * R + gsel;
#pragma unroll
                    for (int j = 0; j < QPK; ++j) {
                        e[set][j] = -INFINITY;
                        if (kg < NK) {
                            e[set][j] = e_buf[((i & 1) * 8 + kg * QPK + j) * 64 + token];
                            float a = 1.f;
#pragma unroll
                            for (int g = 0; g < 8; ++g) if (g < NQ && g == kg * QPK + j) a = alpha[g];
                            l_own[set][j] *= a;
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&xy_free[i & 1]);

                // ---- rows past the live length hold whatever the cache holds there (NaN patterns included): their
                //      weights are zero, so the latent rows are cleared
                if (n_valid < T) {
                    ok = wait(&full_bar[s], (i / kBtStages) & 1) && ok;
                    const int n_vec = (T - n_valid) * CH * 16;
                    for (int idx = gtid; idx < n_vec; idx += 128) {
                        const int row = n_valid + idx / (CH * 16), v = idx % (CH * 16);
                        *reinterpret_cast<uint4*>(stage + lay.c_off + (v >> 3) * tb + row * 128 + (v & 7) * 16) =
                            make_uint4(0u, 0u, 0u, 0u);
                    }
                }
                // ---- the sums so far are rescaled when a maximum was raised (the first sub-tile of a sequence
                //      overwrites them)
                if (grow && !first) {       // uniform over the group
                    ok = wait(&pv_done[(i - 1) & 1], ((i - 1) >> 1) & 1) && ok;
                    ptx::tc_fence_after_sync();
#pragma unroll
                    for (int c = 0; c < CH; ++c) {
                        uint32_t r[16];
                        ptx::tmem_ld16(tmem_o + c * 16, r);
                        ptx::tmem_wait_ld();
#pragma unroll
                        for (int g = 0; g < 8; ++g) r[g] = __float_as_uint(__uint_as_float(r[g]) * alpha[g]);
                        ptx::tmem_st16(tmem_o + c * 16, r);
                    }
                    ptx::tmem_wait_st();
                }
                // ---- the weights of this (key group, token) into the B operand of the sums (free once the sums of
                //      sub-tile i - 2 are complete)
                if (i >= 2) ok = wait(&pv_done[i & 1], ((i >> 1) - 1) & 1) && ok;
#pragma unroll
                for (int set = 0; set < SETS; ++set) {
                    const int kg = set * R + gsel;
                    if (kg < NK) {
#pragma unroll
                        for (int j = 0; j < QPK; ++j) {
                            const float w = bt_ex2(e[set][j]);
                            l_own[set][j] += w;
                            *reinterpret_cast<__nv_bfloat16*>(p_buf + (i & 1) * kBtOperand + bt_swz(kg * QPK + j, 2 * token)) =
                                __float2bfloat16_rn(w);
                        }
                    }
                }
                ptx::fence_proxy_async_smem();      // the weights and the cleared rows, before the tensor pipe reads them
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0 && !(withhold_first_arrive && i == 0 && quarter == 0)) ptx::mbar_arrive(&p_ready[i & 1]);
                first = false;

                // ---- the last sub-tile of the sequence in this range: its partial result goes to slot cta + b
                const bool last = (i + 1 == n_sub) || (k + 1 >= n_sub_b);
                if (last) {
                    ok = wait(&pv_done[i & 1], (i >> 1) & 1) && ok;
                    ptx::tc_fence_after_sync();
                    const size_t slot = (size_t)cta + b;
#pragma unroll
                    for (int c = 0; c < CH; ++c) {
                        uint32_t r[16];
                        ptx::tmem_ld16(tmem_o + c * 16, r);
                        ptx::tmem_wait_ld();
#pragma unroll
                        for (int g = 0; g < 8; ++g)
                            if (g < NQ) part_o[(slot * NQ + g) * d.d_l + c * 128 + quarter * 32 + lane] = __uint_as_float(r[g]);
                    }
#pragma unroll
                    for (int set = 0; set < SETS; ++set) {
#pragma unroll
                        for (int j = 0; j < QPK; ++j) {
                            float v = l_own[set][j];
#pragma unroll
                            for (int o = kSeg / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                            if ((gtid & (kSeg - 1)) == 0) l_red[(set * (128 / kSeg) + seg) * 8 + j] = v;
                            l_own[set][j] = 0.f;
                        }
                    }
                    asm volatile("bar.sync 2, 128;" ::: "memory");
                    if (gtid < NQ) {
                        constexpr int spg = T / kSeg;
                        const int kg = gtid / QPK, set = kg / R, s0 = (kg % R) * spg, j = gtid % QPK;
                        float mg = -INFINITY;
#pragma unroll
                        for (int g = 0; g < 8; ++g) if (g == gtid) mg = m_cur[g];
                        float lsum = l_red[(set * (128 / kSeg) + s0) * 8 + j];
                        if (spg == 2) lsum += l_red[(set * (128 / kSeg) + s0 + 1) * 8 + j];
                        part_ml[(slot * NQ + gtid) * 2] = mg;
                        part_ml[(slot * NQ + gtid) * 2 + 1] = lsum;
                    }
                    ptx::tc_fence_before_sync();
                }
            }
        }
        (void)ok;
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 9) ptx::tmem_dealloc(tmem_base, kBtTmemCols);
    if (tid == 0 && *abort_flag) raise_status(status_word, GTA_ERR_TIMEOUT);
}

template <int T, int NK, int QPK, int CH>
cudaError_t launch_bt(const CUtensorMap& tm_k, const CUtensorMap& tm_c, const Dims& d, int G, int S_cap, const void* q,
                      const int32_t* seq_lens, float* part_o, float* part_ml, int32_t* status_word, cudaStream_t stream,
                      const void* k_new, const void* c_new, void* k_cache, void* c_cache, const PageMap& pm) {
    auto kern = decode_stream_tc_kernel<T, NK, QPK, CH>;
    const size_t smem = bt_smem_layout(T, NK, CH).total;
    cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(G);
    cfg.blockDim = dim3(kBtThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, tm_k, tm_c, d, S_cap, (const __nv_bfloat16*)q, seq_lens, part_o, part_ml,
                              status_word, (const uint4*)k_new, (const uint4*)c_new, (uint4*)k_cache, (uint4*)c_cache, pm);
}

// The instantiations: (sub-tile, key groups, maps per group, 128-column latent blocks); the sub-tile is the one the
// stream kernels' plan arrives at (the largest of 16, 32, 64 tokens whose rows fit a 64 KB ring stage).  They are the
// groupings on which this kernel was measured faster than decode_stream_kernel (32 sequences of 4096 tokens, every
// grouping of 1, 2, 4, 8 key groups x 1, 2, 4, 8 maps with at most 8 maps, d_l = 256, 512, 1024): those whose key
// groups fill, or nearly fill, the 128 rows of the score MMAs, i.e. whose sub-tiles are 48 - 64 KB.  With fewer key
// groups a sub-tile is small against the microsecond its chain through the two token-warp groups and the MMA warp
// takes, and the warp-level kernel is 3 - 15 % faster.
#define GTA_BT_SHAPES(X) \
    X(64, 1, 1, 2) X(64, 1, 2, 2) X(64, 2, 1, 2) X(64, 2, 2, 2) X(64, 2, 4, 2) X(32, 4, 1, 2) X(32, 4, 2, 2) X(16, 8, 1, 2) \
    X(32, 4, 1, 4) X(32, 4, 2, 4) X(16, 8, 1, 4) \
    X(16, 8, 1, 8)

}  // namespace

// d_h = 128, one latent group, one CTA per SM, one of the instantiated shapes; a paged pool's pages hold whole sub-tiles
bool decode_tc_supported(const Dims& d, int T, int occ, int page_size) {
    if (occ != 1 || d.d_h != 128 || d.n_c != 1 || d.B > kBtMaxBatch) return false;
    if (page_size % T != 0) return false;
    const int ch = d.d_l / 128, qpk = d.n_k > 0 ? d.n_q / d.n_k : 0;
    if (d.d_l % 128 != 0) return false;
#define GTA_BT_MATCH(TV, NKV, QPKV, CHV) if (T == TV && d.n_k == NKV && qpk == QPKV && ch == CHV) return true;
    GTA_BT_SHAPES(GTA_BT_MATCH)
#undef GTA_BT_MATCH
    return false;
}

cudaError_t launch_decode_tc_stream(const Dims& d, int G, int T, int S_cap, const void* q, const void* k_cache,
                                    const void* c_cache, const int32_t* seq_lens, float* part_o, float* part_ml,
                                    int32_t* status_word, cudaStream_t stream, const void* k_new, const void* c_new,
                                    const PageMap& pm) {
    CUtensorMap tm_k, tm_c;
    const uint32_t box[3] = {64, (uint32_t)T, 1};
    // planes of rows: one per (sequence, group), S_cap rows each -- or one per (page, group), page_size rows
    const uint64_t rows = pm.table ? (uint64_t)pm.page_size : (uint64_t)S_cap;
    const uint64_t outer = pm.table ? (uint64_t)pm.n_pages : (uint64_t)d.B;
    const uint64_t dk[3] = {(uint64_t)d.d_h, rows, outer * d.n_k};
    const uint64_t dc[3] = {(uint64_t)d.d_l, rows, outer};
    if (!make_bf16_map(&tm_k, k_cache, 3, dk, box) || !make_bf16_map(&tm_c, c_cache, 3, dc, box))
        return cudaErrorInvalidValue;
    const int ch = d.d_l / 128, qpk = d.n_q / d.n_k;
    cudaError_t err = cudaErrorInvalidValue;
#define GTA_BT_LAUNCH(TV, NKV, QPKV, CHV)                                                                          \
    if (T == TV && d.n_k == NKV && qpk == QPKV && ch == CHV)                                                       \
        err = launch_bt<TV, NKV, QPKV, CHV>(tm_k, tm_c, d, G, S_cap, q, seq_lens, part_o, part_ml, status_word,    \
                                            stream, k_new, c_new, const_cast<void*>(k_cache), const_cast<void*>(c_cache), pm);
    GTA_BT_SHAPES(GTA_BT_LAUNCH)
#undef GTA_BT_LAUNCH
    if (err != cudaSuccess) return err;
    return cudaGetLastError();
}

gta_status_t decode_tc_debug_wait(unsigned long long limit_ns, int withhold_first_arrive) {
    const unsigned long long lim = limit_ns ? limit_ns : ptx::kWaitLimitNs;
    const int sw = withhold_first_arrive ? 1 : 0;
    if (cudaMemcpyToSymbol(g_bt_wait_limit_ns, &lim, sizeof(lim)) != cudaSuccess ||
        cudaMemcpyToSymbol(g_bt_withhold_first_arrive, &sw, sizeof(sw)) != cudaSuccess) {
        cudaGetLastError();
        return GTA_ERR_CUDA;
    }
    return GTA_OK;
}

}  // namespace gta
