// The decode stream kernel for 8-bit caches on the tcgen05 tensor pipe.
//
// K and C rows are e4m3 codes with one fp32 scale per cached row (the reading of the paper's Sec. 5.3 /
// App. C.2 observation that a decode step is bound by the bytes of its cache).  The arithmetic is the one of
// decode_stream_fp8_kernel -- the other operand of an 8-bit MMA has to be 8-bit too, so a query row and a
// weight are each the SUM OF TWO e4m3 numbers; a key row's scale multiplies its score after the MMA, a latent
// row's scale s_j is folded into the softmax, w_j = 2^(score_j + log2 s_j - m), and the row sum is taken from
// the unshifted scores against the same m -- but both contractions are TRANSPOSED so that the cached tokens,
// not the handful of attention maps, fill the 128 rows of a tcgen05.mma (kind::f8f6f4, K = 32):
//
//   scores   S^T [token][2 map + piece] = K tile [token][d_h]  x  Q^T           A = the key tile as it lies in
//            shared memory (K-major), B = the query pieces [16 rows][128 codes]; one accumulator of 16 columns
//            per key group, so a thread (= a token, TMEM lane) reads its scores of all maps as a few columns.
//   sums     O^T [latent column][2 map + piece] += C tile^T [column][token]  x  P^T [2 map + piece][token]
//            A = the latent tile as it lies in shared memory, read MN-major (128 columns = one 128-byte row
//            of the tile per token), B = the weights' pieces written by the token threads; the accumulators
//            (d_l / 128 blocks of 16 columns) stay in tensor memory over all sub-tiles of a sequence.
//
// The codes go from HBM through TMA into shared memory and from there into the tensor pipe without passing a
// register; per sub-tile of 64 tokens a token thread does 8 exponential pairs and 16 byte stores.  The warp-level
// e4m3 MMA of decode_stream_fp8_kernel is carried out as f16 MMAs behind operand conversions and paces that
// kernel at the bf16 kernel's token rate; this one is paced by the loads.
//
// Schedule, ring, scale rows, partial results (slot c + b: running maximum, row sum, unnormalised latent sums) are
// those of the other stream kernels, so decode_merge_kernel and the decoder kernel follow unchanged.
// Warps 0-3 (group A, one per TMEM lane quarter): read a sub-tile's scores, keep the running maxima, leave the
// exponents of the weights and of the row-sum terms in shared memory.  Warps 4-7 (group B, again one per lane
// quarter): exponentials, the weights' pieces into the B operand, rescaling of the sums when a maximum has grown,
// the partial result at the end of a sequence.  A works on sub-tile i + 1 while B works on sub-tile i: a single
// warp per scheduler runs at the latency of its dependent instructions, not at its issue rate, so the chain of a
// sub-tile is cut in two.  Warp 8: TMA producer.  Warp 9: MMA issue.
#include "gta_common.cuh"
#include "gta_sm100.cuh"
#include "sm100_ptx.cuh"
#include "tma_host.cuh"

namespace gta {
namespace {

// Test hooks of the bounded waits (gta_debug_decode_wait): the time limit of every wait of this kernel, and a switch
// that makes one warp of group B keep its very first arrival to itself, so that the MMA warp runs into that limit and
// the whole unwinding path can be exercised on a healthy GPU.  Read once per thread at kernel start.
__device__ unsigned long long g_tc_wait_limit_ns = ptx::kWaitLimitNs;
__device__ int g_tc_withhold_first_arrive = 0;

constexpr int kTcMaxT = 64;                     // most tokens per sub-tile (64, or 32 for wide tokens)
constexpr int kTcStages = 3;
constexpr int kTcThreads = 320;
constexpr int kTcMaxBatch = 512;
constexpr uint32_t kTcOperand = 16 * 128;       // bytes of a [16 rows][128 codes] B operand (Q pieces, weights' pieces)
constexpr uint32_t kTcExpBytes = 2 * 2 * 8 * kTcMaxT * 4;   // exponents handed from group A to group B
constexpr uint32_t kTcTmemCols = 256;           // 2 x 64 score columns, 64 sum columns
constexpr float kTcWeightScale = 64.f;          // the weights are scaled into e4m3's range ...
constexpr float kTcLag = 2.f;                   // ... with room for a running maximum that lags by 2^2

__device__ __forceinline__ float tc_ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void tc_group_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
__device__ __forceinline__ int tc_len(const int32_t* seq_lens, int b, int S_cap) {
    const int len = seq_lens[b];
    return len < 0 ? 0 : (len > S_cap ? S_cap : len);
}
// byte offset of (row, byte column) in a [rows][128 bytes] operand with the 128-byte swizzle
__device__ __forceinline__ uint32_t tc_swz(int row, int col) {
    return (uint32_t)row * 128u + ((((uint32_t)col >> 4) ^ ((uint32_t)row & 7u)) << 4) + ((uint32_t)col & 15u);
}

struct TcSmem {
    uint32_t stage_stride, scale_off, q_off, p_off, misc_off, total;
};
__host__ __device__ inline TcSmem tc_smem_layout(int T, int n_k, int ch) {
    TcSmem s;
    s.scale_off = (uint32_t)(n_k + ch) * (uint32_t)T * 128u;
    s.stage_stride = s.scale_off + (((uint32_t)(n_k + 1) * T * 4 + 1023u) & ~1023u);
    s.q_off = kTcStages * s.stage_stride;            // [2 sequence parities][16][128]
    s.p_off = s.q_off + 2 * kTcOperand;              // [2 sub-tile parities][16][128]
    s.misc_off = s.p_off + 2 * kTcOperand;
    // exponents [2][2][8][64] | prefix [B + 2] | scan [kTcThreads] | mx [2][4][8] | l_red [4][8] | qmul [2][8] |
    // hdr [2][8 alpha, 8 maxima, grow, pad 7] | 24 barriers | 4 words
    s.total = s.misc_off + kTcExpBytes + (kTcMaxBatch + 2 + kTcThreads) * 4 + (64 + 32 + 16 + 48) * 4 + 24 * 8 + 16 + 1024;
    return s;
}

// CH: 128-column blocks of the latent; NK: key groups; QPK: maps per key group (compile-time, so that the per-map
// loops of the token threads unroll into straight code: those threads run one warp per scheduler, at the latency of
// every instruction they issue).
template <int T, int CH, int NK, int QPK>
__global__ void __launch_bounds__(kTcThreads, 1)
decode_stream_fp8_tc_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_c, Dims d,
                            int S_cap, const __nv_bfloat16* __restrict__ q, const float* __restrict__ k_scale,
                            const float* __restrict__ c_scale, const int32_t* __restrict__ seq_lens,
                            float* __restrict__ part_o, float* __restrict__ part_ml, int32_t* status_word) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    constexpr int kTcT = T;
    constexpr uint32_t kTcTile = T * 128;            // bytes of a [T tokens][128 codes] tile
    constexpr int R = 128 / T;                        // key groups on the 128 rows of a score MMA
    constexpr int SETS = (NK + R - 1) / R;
    constexpr int WPG = T / 32;                       // warps of a group per key group
    static_assert(SETS <= 2 && NK * QPK <= 8 && CH <= 8, "instantiation outside the kernel's limits");
    const TcSmem lay = tc_smem_layout(T, NK, CH);
    uint8_t* ring = smem;
    uint8_t* q_buf = smem + lay.q_off;
    uint8_t* p_buf = smem + lay.p_off;
    float* e_buf = reinterpret_cast<float*>(smem + lay.misc_off);             // [2 parities][weights, row sums][8 maps][64 tokens]
    int32_t* prefix = reinterpret_cast<int32_t*>(smem + lay.misc_off + kTcExpBytes);   // [B + 1]
    int32_t* scan_tmp = prefix + kTcMaxBatch + 2;                             // [kTcThreads]
    float* mx_buf = reinterpret_cast<float*>(scan_tmp + kTcThreads);          // [2 parities][4 warps][8 maps]
    float* l_red = mx_buf + 64;                                               // [4 warps][8 maps]
    float* qmul = l_red + 32;                                                 // [2 parities][8 maps]
    float* hdr = qmul + 16;                                                   // [2 parities][8 alpha | 8 maxima | grow | -]
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(hdr + 48);               // [3] TMA bytes of a stage have landed
    uint64_t* empty_bar = full_bar + kTcStages;                               // [3] the sums of its sub-tile are complete
    uint64_t* s_ready = empty_bar + kTcStages;                                // [2] scores of sub-tile i are in buffer i & 1
    uint64_t* p_ready = s_ready + 2;                                          // [2] 4 warps of B: weights written, O rescaled
    uint64_t* pv_done = p_ready + 2;                                          // [2] the sums of sub-tile i are complete
    uint64_t* q_ready = pv_done + 2;                                          // [2] 4 warps: query pieces of sequence n in buffer n & 1
    uint64_t* s_free = q_ready + 2;                                           // [2] 4 warps of A: the scores have been read
    uint64_t* xy_ready = s_free + 2;                                          // [2] 4 warps of A: exponents and header of sub-tile i
    uint64_t* xy_free = xy_ready + 2;                                         // [2] 4 warps of B: ... have been read
    uint64_t* drain_bar = xy_free + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain_bar + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile int* drain_flag = abort_flag + 1;
    const uint64_t wait_limit = g_tc_wait_limit_ns;
    const bool withhold_first_arrive = g_tc_withhold_first_arrive != 0;
    // every wait of this kernel: bounded by wait_limit, ended early by the CTA's abort flag
    auto wait = [&](uint64_t* bar, uint32_t parity) { return ptx::mbar_wait_sleep(bar, parity, abort_flag, 0, wait_limit); };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int G = gridDim.x, cta = blockIdx.x;
    constexpr int NQ = NK * QPK;
    constexpr int qpk = QPK;

    if (tid == 0) {
        for (int s = 0; s < kTcStages; ++s) { ptx::mbar_init(&full_bar[s], 1); ptx::mbar_init(&empty_bar[s], 1); }
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
    if (warp == 9) ptx::tmem_alloc(tmem_slot, kTcTmemCols);
    // rows of the B operands that belong to no map stay zero for the whole kernel
    for (uint32_t i = tid; i < 4 * kTcOperand / 16; i += kTcThreads)
        reinterpret_cast<uint4*>(q_buf)[i] = make_uint4(0u, 0u, 0u, 0u);
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // launched with programmatic stream serialisation: nothing of global memory is read before the kernel ahead
    // (a quantising append) is complete, and only then may the kernels behind this one be scheduled
    ptx::grid_dependency_wait();
    ptx::grid_launch_dependents();

    {   // exclusive prefix sum of the sub-tile counts (as in the other stream kernels)
        const int per = (d.B + kTcThreads - 1) / kTcThreads;
        const int lo = min(tid * per, d.B), hi = min(lo + per, d.B);
        int sum = 0;
        for (int b = lo; b < hi; ++b) sum += (tc_len(seq_lens, b, S_cap) + kTcT - 1) / kTcT;
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
            base += (tc_len(seq_lens, b, S_cap) + kTcT - 1) / kTcT;
        }
        if (tid == kTcThreads - 1) prefix[d.B] = base;
        __syncthreads();
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
        const int n_tiles = NK + CH, n_ops = n_tiles + NK + 1;      // tensor tiles, then the scale rows
        int b = b0, k = k0, it = 0;
        bool ok = true;
        for (; it < n_sub; ++it, ++k) {
            while (k >= prefix[b + 1] - prefix[b]) { ++b; k = 0; }
            const int s = it % kTcStages;
            const uint32_t ph = (it / kTcStages) & 1;
            const int tok0 = k * kTcT;
            const uint32_t n_sc = (uint32_t)min(kTcT, S_cap - tok0) * 4;   // bytes of a scale row (S_cap is a multiple of 4)
            if (lane == 0) {
                ok = wait(&empty_bar[s], ph ^ 1);
                if (ok) ptx::mbar_arrive_expect_tx(&full_bar[s], lay.scale_off + (uint32_t)(NK + 1) * n_sc);
            }
            ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
            if (!ok) break;
            uint8_t* stage = ring + s * lay.stage_stride;
            for (int op = lane; op < n_ops; op += 32) {
                if (op < NK)
                    ptx::tma_load_3d_hint(stage + op * kTcTile, &tm_k, &full_bar[s], 0, tok0, b * NK + op, policy);
                else if (op < n_tiles)
                    ptx::tma_load_3d_hint(stage + op * kTcTile, &tm_c, &full_bar[s], (op - NK) * 128, tok0, b, policy);
                else if (op < n_tiles + NK)
                    ptx::bulk_load_1d(stage + lay.scale_off + (op - n_tiles) * kTcT * 4,
                                      k_scale + ((size_t)b * NK + (op - n_tiles)) * S_cap + tok0, n_sc, &full_bar[s]);
                else
                    ptx::bulk_load_1d(stage + lay.scale_off + NK * kTcT * 4, c_scale + (size_t)b * S_cap + tok0, n_sc,
                                      &full_bar[s]);
            }
        }
        if (lane == 0 && *abort_flag) {
            for (int back = 1; back <= kTcStages && it - back >= 0; ++back) {
                const int iq = it - back;
                ptx::mbar_wait_drain(&full_bar[iq % kTcStages], (iq / kTcStages) & 1, drain_flag);
            }
        }
    } else if (n_sub > 0 && warp == 9) {
        // ------------------------------------------------------------------ MMA issue (one thread)
        if (ptx::elect_one()) {
            constexpr uint32_t idesc_s = ptx::make_idesc_e4m3(128, 16, 0, 0);    // key tile and query pieces, both K-major
            constexpr uint32_t idesc_o = ptx::make_idesc_e4m3(128, 16, 1, 0);    // latent tile MN-major, weights K-major
            const uint64_t desc_kmajor = ptx::make_smem_desc(0, 16, 1024);
            const uint64_t desc_latent = ptx::make_smem_desc(0, kTcTile, 1024);  // 8 tokens per 1024 bytes; one 128-column panel
            const uint32_t q_addr = ptx::smem_addr(q_buf), p_addr = ptx::smem_addr(p_buf);
            const uint32_t tmem_o = tmem_base + 128;
            bool ok = true;
            // sequence bookkeeping of sub-tile j: which sequence ordinal it belongs to, whether it is its first here
            int sb = b0, sk = k0, sn = 0;        // for the scores (one sub-tile ahead of the sums)
            int pb = b0, pk = k0;                // for the sums
            auto issue_scores = [&](int j) -> bool {
                bool first = (j == 0);
                while (sk >= prefix[sb + 1] - prefix[sb]) { ++sb; sk = 0; first = true; }
                if (first && j > 0) ++sn;
                const int s = j % kTcStages;
                if (first && !wait(&q_ready[sn & 1], (sn >> 1) & 1)) return false;
                if (!wait(&full_bar[s], (j / kTcStages) & 1)) return false;
                // the buffer held the scores of sub-tile j - 2
                if (j >= 2 && !wait(&s_free[j & 1], ((j >> 1) - 1) & 1)) return false;
                ptx::tc_fence_after_sync();
                const uint32_t stage = ring_addr + s * lay.stage_stride;
                const uint64_t dq = desc_kmajor + ((q_addr + (sn & 1) * kTcOperand) >> 4);
                // The 128 rows of A are the 64 tokens of key group 2 kp and, 8 KB further on, the same 64 tokens of key
                // group 2 kp + 1 (the tiles of a stage lie back to back; behind the last key tile come latent rows,
                // whose "scores" nobody reads): lanes 0-63 and 64-127 of the accumulator.
                for (int kp = 0; kp < SETS; ++kp) {
                    const uint64_t dk = desc_kmajor + ((stage + kp * R * kTcTile) >> 4);
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)      // 32 codes = 32 bytes of the 128-byte rows per step
                        ptx::mma_ss_f8(tmem_base + (j & 1) * 64 + kp * 16, dk + 2 * ks, dq + 2 * ks, idesc_s, ks > 0 ? 1u : 0u);
                }
                ptx::tc_commit(&s_ready[j & 1]);
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
                ok = wait(&p_ready[i & 1], (i >> 1) & 1);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const int s = i % kTcStages;
                const uint32_t stage = ring_addr + s * lay.stage_stride;
                const uint64_t dp = desc_kmajor + ((p_addr + (i & 1) * kTcOperand) >> 4);
#pragma unroll
                for (int c = 0; c < CH; ++c) {
                    const uint64_t dc = desc_latent + ((stage + (NK + c) * kTcTile) >> 4);
#pragma unroll
                    for (int kk = 0; kk < T / 32; ++kk)      // 32 tokens = 4096 bytes of the tile, 32 bytes of the weights' rows
                        ptx::mma_ss_f8(tmem_o + c * 16, dc + kk * (4096 >> 4), dp + 2 * kk, idesc_o,
                                       (first && kk == 0) ? 0u : 1u);
                }
                ptx::tc_commit(&pv_done[i & 1]);
                ptx::tc_commit(&empty_bar[s]);
            }
            if (*abort_flag) {      // unwinding: the MMAs issued so far must be complete before tensor memory is freed
                ptx::tc_commit(drain_bar);
                ptx::mbar_wait_drain(drain_bar, 0, drain_flag);
            }
        }
    } else if (n_sub > 0 && warp < 8) {
        // ------------------------------------------------------------------ groups A and B
        // Scores: quarters 0 / 1 hold tokens 0-31 / 32-63 for the even key groups, quarters 2 / 3 the same tokens for
        // the odd ones; a thread of B takes over the (token, maps) of the thread of A in the same place.  Sums: lane
        // 32 quarter + lane is a latent column of each 128-column block.
        const bool group_b = warp >= 4;
        const int quarter = warp & 3;
        const int gtid = tid & 127;                      // thread index inside the group
        const uint32_t lane_base = ((uint32_t)(quarter * 32) << 16);
        const uint32_t tmem_o = tmem_base + 128 + lane_base;
        const int half = gtid / T;                       // key group of this thread inside a set of R
        const int token = gtid % T;                      // of the sub-tile
        const uint32_t tok_swz = (uint32_t)token >> 4, tok_low = (uint32_t)token & 15u;
        int kg_of[8];                       // key group of map g
        bool mine[8];                       // this thread handles map g
#pragma unroll
        for (int g = 0; g < 8; ++g) {
            kg_of[g] = g / qpk;
            mine[g] = g < NQ && (kg_of[g] % R) == half;
        }
        int b = b0, k = k0, n = 0;          // sequence, its sub-tile, its ordinal in this range
        int len_b = tc_len(seq_lens, b, S_cap), n_sub_b = prefix[b + 1] - prefix[b];
        bool ok = true, first = true;

        if (!group_b) {
        // the query pieces of sequence b into buffer par: warp w takes the maps 2 w and 2 w + 1, a lane four elements
        auto write_q = [&](int b, int par) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int g = 2 * quarter + h;
                if (g < NQ) {     // uniform over the warp
                    const uint2 raw = __ldg(reinterpret_cast<const uint2*>(q + ((size_t)b * NQ + g) * 128 + 4 * lane));
                    const float2 v01 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.x));
                    const float2 v23 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.y));
                    float amax = fmaxf(fmaxf(fabsf(v01.x), fabsf(v01.y)), fmaxf(fabsf(v23.x), fabsf(v23.y)));
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
                    // power of two that brings the row's largest element into [128, 256) (e4m3 reaches 448)
                    uint32_t e = (__float_as_uint(amax) >> 23) & 0xffu;
                    e = e < 8u ? 8u : e;
                    const float scale = __uint_as_float((e - 7u) << 23), inv = __uint_as_float((261u - e) << 23);
                    const float x0 = v01.x * inv, x1 = v01.y * inv, x2 = v23.x * inv, x3 = v23.y * inv;
                    const uint32_t h01 = ptx::cvt_e4m3x2(x0, x1), h23 = ptx::cvt_e4m3x2(x2, x3);
                    const float2 b01 = ptx::e4m3x2_to_f32(h01), b23 = ptx::e4m3x2_to_f32(h23);
                    const uint32_t hi = h01 | (h23 << 16);
                    const uint32_t lo = ptx::cvt_e4m3x2(x0 - b01.x, x1 - b01.y) | (ptx::cvt_e4m3x2(x2 - b23.x, x3 - b23.y) << 16);
                    uint8_t* dst = q_buf + par * kTcOperand;
                    *reinterpret_cast<uint32_t*>(dst + tc_swz(2 * g, 4 * lane)) = hi;
                    *reinterpret_cast<uint32_t*>(dst + tc_swz(2 * g + 1, 4 * lane)) = lo;
                    if (lane == 0) qmul[par * 8 + g] = scale * d.scale * 1.4426950408889634f;
                }
            }
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&q_ready[par]);
        };
        // the next sequence after b that has sub-tiles in this range (-1: none)
        auto next_seq = [&](int b) {
            int nb = b + 1;
            while (nb < d.B && prefix[nb + 1] == prefix[nb]) ++nb;
            return (nb < d.B && prefix[nb] < st_end) ? nb : -1;
        };


            float m_run[8];
#pragma unroll
            for (int g = 0; g < 8; ++g) m_run[g] = -INFINITY;
            write_q(b, 0);
            asm volatile("bar.sync 1, 128;" ::: "memory");      // qmul of the first sequence is visible to all of A
            for (int i = 0; i < n_sub; ++i, ++k) {
                if (k >= n_sub_b) {
                    do { ++b; } while (prefix[b + 1] == prefix[b]);
                    k = 0;
                    ++n;
                    first = true;
                    len_b = tc_len(seq_lens, b, S_cap);
                    n_sub_b = prefix[b + 1] - prefix[b];
#pragma unroll
                    for (int g = 0; g < 8; ++g) m_run[g] = -INFINITY;
                }
                if (first) {    // the buffer of the sequence before this one is free: every score of it has been read
                    const int nb = next_seq(b);
                    if (nb >= 0) write_q(nb, (n + 1) & 1);
                }
                const int s = i % kTcStages;
                const int n_valid = min(kTcT, len_b - k * kTcT);
                const float* ksc = reinterpret_cast<const float*>(ring + s * lay.stage_stride + lay.scale_off);
                const float* csc = ksc + NK * kTcT;
                ok = wait(&full_bar[s], (i / kTcStages) & 1) && ok;
                ok = wait(&s_ready[i & 1], (i >> 1) & 1) && ok;
                ptx::tc_fence_after_sync();

                // ---- this token's scores of this thread's maps, plain (x) and shifted by log2 of the latent row's scale (y)
                float x[8], y[8];
#pragma unroll
                for (int g = 0; g < 8; ++g) x[g] = y[g] = -INFINITY;
                const bool live = token < n_valid;
                const float shift = live ? __log2f(csc[token]) : 0.f;
                uint32_t r[2][16];
#pragma unroll
                for (int kp = 0; kp < 2; ++kp)
                    if (kp < SETS) ptx::tmem_ld16(tmem_base + lane_base + (i & 1) * 64 + kp * 16, r[kp]);
                ptx::tmem_wait_ld();
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&s_free[i & 1]);
#pragma unroll
                for (int kp = 0; kp < 2; ++kp) {
                    if (kp < SETS && kp * R + half < NK) {
                        const float ks = live ? ksc[(kp * R + half) * kTcT + token] : 0.f;
#pragma unroll
                        for (int g = 0; g < 8; ++g) {
                            if (mine[g] && (kg_of[g] / R) == kp && live) {
                                x[g] = (__uint_as_float(r[kp][2 * g]) + __uint_as_float(r[kp][2 * g + 1])) * qmul[(n & 1) * 8 + g] * ks;
                                y[g] = x[g] + shift;
                            }
                        }
                    }
                }
#pragma unroll
                for (int g = 0; g < 8; ++g) {
                    if (mine[g]) {      // uniform over the warp
                        const float mw = ptx::warp_max_redux(y[g]);
                        if (lane == 0) mx_buf[((i & 1) * 4 + quarter) * 8 + g] = mw;
                    }
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");

                // ---- the running maxima: a reference is raised only when the sub-tile exceeds it by more than kTcLag
                //      (the weights, scaled by kTcWeightScale, then stay within e4m3's range: 64 x 2^2 = 256 <= 448)
                float alpha[8], m_sub[8];
                bool grow = false;
#pragma unroll
                for (int g = 0; g < 8; ++g) {
                    alpha[g] = 1.f;
                    m_sub[g] = 0.f;
                    if (g < NQ) {
                        const int w0 = (i & 1) * 4 + WPG * (kg_of[g] % R);    // the warps that score map g
                        float m_tile = mx_buf[w0 * 8 + g];
                        if (WPG == 2) m_tile = fmaxf(m_tile, mx_buf[(w0 + 1) * 8 + g]);
                        const bool up = m_tile > m_run[g] + kTcLag;
                        grow = grow || up;
                        alpha[g] = up ? tc_ex2(m_run[g] - m_tile) : 1.f;
                        m_run[g] = up ? m_tile : m_run[g];
                        m_sub[g] = m_run[g] > -INFINITY ? m_run[g] : 0.f;
                    }
                }
                // ---- hand-over to group B (the buffers of sub-tile i - 2 have been read)
                if (i >= 2) ok = wait(&xy_free[i & 1], ((i >> 1) - 1) & 1) && ok;
                float* eb = e_buf + (i & 1) * (2 * 8 * kTcT) + token;
#pragma unroll
                for (int g = 0; g < 8; ++g) {
                    if (mine[g]) {
                        eb[g * kTcT] = y[g] - m_sub[g];
                        eb[(8 + g) * kTcT] = x[g] - m_sub[g];
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
            float l_thr[8], m_cur[8];
#pragma unroll
            for (int g = 0; g < 8; ++g) { l_thr[g] = 0.f; m_cur[g] = -INFINITY; }
            for (int i = 0; i < n_sub; ++i, ++k) {
                if (k >= n_sub_b) {
                    do { ++b; } while (prefix[b + 1] == prefix[b]);
                    k = 0;
                    first = true;
                    len_b = tc_len(seq_lens, b, S_cap);
                    n_sub_b = prefix[b + 1] - prefix[b];
                }
                const int s = i % kTcStages;
                const int n_valid = min(kTcT, len_b - k * kTcT);
                uint8_t* stage = ring + s * lay.stage_stride;
                ok = wait(&xy_ready[i & 1], (i >> 1) & 1) && ok;
                float alpha[8];
#pragma unroll
                for (int g = 0; g < 8; ++g) {
                    alpha[g] = g < NQ ? hdr[(i & 1) * 24 + g] : 1.f;
                    m_cur[g] = g < NQ ? hdr[(i & 1) * 24 + 8 + g] : -INFINITY;
                    l_thr[g] *= alpha[g];
                }
                const bool grow = hdr[(i & 1) * 24 + 16] != 0.f;
                float ew[8], el[8];
                const float* eb = e_buf + (i & 1) * (2 * 8 * kTcT) + token;
#pragma unroll
                for (int g = 0; g < 8; ++g) {
                    ew[g] = el[g] = -INFINITY;
                    if (mine[g]) { ew[g] = eb[g * kTcT]; el[g] = eb[(8 + g) * kTcT]; }
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&xy_free[i & 1]);

                // ---- rows past the live length hold whatever the cache holds there (NaN codes included): their
                //      weights are zero, so the latent rows are cleared
                if (n_valid < kTcT) {
                    ok = wait(&full_bar[s], (i / kTcStages) & 1) && ok;
                    const int n_vec = (kTcT - n_valid) * CH * 8;
                    for (int idx = gtid; idx < n_vec; idx += 128) {
                        const int row = n_valid + idx / (CH * 8), v = idx % (CH * 8);
                        *reinterpret_cast<uint4*>(stage + (NK + (v >> 3)) * kTcTile + row * 128 + (v & 7) * 16) =
                            make_uint4(0u, 0u, 0u, 0u);
                    }
                }
                // ---- the sums so far are rescaled when a maximum has grown (the first sub-tile of a sequence
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
                        for (int e = 0; e < 16; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha[e >> 1]);
                        ptx::tmem_st16(tmem_o + c * 16, r);
                    }
                    ptx::tmem_wait_st();
                }
                // ---- the weights' pieces of this token into the B operand of the sums (free once the sums of
                //      sub-tile i - 2 are complete)
                if (i >= 2) ok = wait(&pv_done[i & 1], ((i >> 1) - 1) & 1) && ok;
                {
                    uint8_t* dst = p_buf + (i & 1) * kTcOperand + tok_low;
#pragma unroll
                    for (int g = 0; g < 8; ++g) {
                        if (mine[g]) {
                            const float w = tc_ex2(ew[g]) * kTcWeightScale;
                            l_thr[g] += tc_ex2(el[g]);
                            const uint32_t hi = ptx::cvt_e4m3x2(w, 0.f);
                            const uint32_t lo = ptx::cvt_e4m3x2(w - ptx::e4m3x2_to_f32(hi).x, 0.f);
                            // rows 2 g and 2 g + 1 of the operand, byte `token` (128-byte swizzle)
                            dst[(2 * g) * 128 + ((tok_swz ^ ((2 * g) & 7)) << 4)] = (uint8_t)hi;
                            dst[(2 * g + 1) * 128 + ((tok_swz ^ ((2 * g + 1) & 7)) << 4)] = (uint8_t)lo;
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
                            if (g < NQ)     // both pieces, the weights' factor taken out
                                part_o[(slot * NQ + g) * d.d_l + c * 128 + quarter * 32 + lane] =
                                    (__uint_as_float(r[2 * g]) + __uint_as_float(r[2 * g + 1])) * (1.f / kTcWeightScale);
                    }
#pragma unroll
                    for (int g = 0; g < 8; ++g) {
                        if (mine[g]) {
                            float v = l_thr[g];
#pragma unroll
                            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                            if (lane == 0) l_red[quarter * 8 + g] = v;
                        }
                    }
                    asm volatile("bar.sync 2, 128;" ::: "memory");
                    if (gtid < NQ) {
                        float mg = -INFINITY;
#pragma unroll
                        for (int g = 0; g < 8; ++g) if (g == gtid) mg = m_cur[g];
                        const int w0 = WPG * ((gtid / qpk) % R);    // the warps that hold map gtid's row-sum shares
                        part_ml[(slot * NQ + gtid) * 2] = mg;
                        part_ml[(slot * NQ + gtid) * 2 + 1] = l_red[w0 * 8 + gtid] + (WPG == 2 ? l_red[(w0 + 1) * 8 + gtid] : 0.f);
                    }
#pragma unroll
                    for (int g = 0; g < 8; ++g) l_thr[g] = 0.f;
                    ptx::tc_fence_before_sync();
                }
            }
        }
        (void)ok;
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 9) ptx::tmem_dealloc(tmem_base, kTcTmemCols);
    if (tid == 0 && *abort_flag) raise_status(status_word, GTA_ERR_TIMEOUT);
}

}  // namespace

// the instantiations: (sub-tile, 128-column latent blocks, key groups, maps per group).  64-token sub-tiles where a
// token is at most 1 KB of codes and scales (d_l <= 512, at most four key groups), 32-token ones above that.
#define GTA_TC_SHAPES(X)                                                                                   \
    X(64, 1, 1, 1) X(64, 1, 1, 2) X(64, 1, 1, 4) X(64, 1, 1, 8) X(64, 1, 2, 1) X(64, 1, 2, 2) X(64, 1, 2, 4)   \
    X(64, 1, 4, 1) X(64, 1, 4, 2)                                                                          \
    X(64, 2, 1, 1) X(64, 2, 1, 2) X(64, 2, 1, 4) X(64, 2, 1, 8) X(64, 2, 2, 1) X(64, 2, 2, 2) X(64, 2, 2, 4)   \
    X(64, 2, 4, 1) X(64, 2, 4, 2)                                                                          \
    X(64, 4, 1, 1) X(64, 4, 1, 2) X(64, 4, 1, 4) X(64, 4, 1, 8) X(64, 4, 2, 1) X(64, 4, 2, 2) X(64, 4, 2, 4)   \
    X(64, 4, 4, 1) X(64, 4, 4, 2)                                                                          \
    X(32, 8, 1, 1) X(32, 8, 1, 2) X(32, 8, 1, 4) X(32, 8, 1, 8) X(32, 8, 2, 1) X(32, 8, 2, 2) X(32, 8, 2, 4)   \
    X(32, 8, 4, 1) X(32, 8, 4, 2) X(32, 8, 8, 1) X(32, 4, 8, 1) X(32, 2, 8, 1) X(32, 1, 8, 1)

// d_h = 128, one latent group, one of the instantiated shapes with the sub-tile size the plan has chosen
bool decode_fp8_tc_supported(const Dims& d, int T) {
    if (d.d_h != 128 || d.n_c != 1 || d.n_k < 1 || d.n_q % d.n_k != 0 || d.d_l % 128 != 0 || d.B > kTcMaxBatch) return false;
    const int ch = d.d_l / 128, qpk = d.n_q / d.n_k;
#define GTA_TC_MATCH(TV, CHV, NKV, QPKV) \
    if (T == TV && ch == CHV && d.n_k == NKV && qpk == QPKV) return tc_smem_layout(TV, NKV, CHV).total <= 232448u;
    GTA_TC_SHAPES(GTA_TC_MATCH)
#undef GTA_TC_MATCH
    return false;
}

namespace {
template <int T, int CH, int NK, int QPK>
cudaError_t launch_tc(const CUtensorMap& tm_k, const CUtensorMap& tm_c, const Dims& d, int G, int S_cap, const void* q,
                      const float* k_scale, const float* c_scale, const int32_t* seq_lens, float* part_o, float* part_ml,
                      int32_t* status_word, cudaStream_t stream) {
    auto kern = decode_stream_fp8_tc_kernel<T, CH, NK, QPK>;
    const size_t smem = tc_smem_layout(T, NK, CH).total;
    cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(G);
    cfg.blockDim = dim3(kTcThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, tm_k, tm_c, d, S_cap, (const __nv_bfloat16*)q, k_scale, c_scale, seq_lens, part_o,
                              part_ml, status_word);
}
}  // namespace

cudaError_t launch_decode_fp8_tc_stream(const Dims& d, int G, int T, int S_cap, const void* q, const void* k_codes,
                                        const void* c_codes, const float* k_scale, const float* c_scale,
                                        const int32_t* seq_lens, float* part_o, float* part_ml, int32_t* status_word,
                                        cudaStream_t stream) {
    CUtensorMap tm_k, tm_c;
    const uint32_t box[3] = {128, (uint32_t)T, 1};
    const uint64_t dk[3] = {128, (uint64_t)S_cap, (uint64_t)d.B * d.n_k};
    const uint64_t dc[3] = {(uint64_t)d.d_l, (uint64_t)S_cap, (uint64_t)d.B};
    if (!make_u8_map(&tm_k, k_codes, 3, dk, box) || !make_u8_map(&tm_c, c_codes, 3, dc, box)) return cudaErrorInvalidValue;
    const int ch = d.d_l / 128, qpk = d.n_q / d.n_k;
    cudaError_t err = cudaErrorInvalidValue;
#define GTA_TC_LAUNCH(TV, CHV, NKV, QPKV)                                                                         \
    if (T == TV && ch == CHV && d.n_k == NKV && qpk == QPKV)                                                      \
        err = launch_tc<TV, CHV, NKV, QPKV>(tm_k, tm_c, d, G, S_cap, q, k_scale, c_scale, seq_lens, part_o, part_ml, \
                                            status_word, stream);
    GTA_TC_SHAPES(GTA_TC_LAUNCH)
#undef GTA_TC_LAUNCH
    if (err != cudaSuccess) return err;
    return cudaGetLastError();
}

gta_status_t decode_fp8_tc_debug_wait(unsigned long long limit_ns, int withhold_first_arrive) {
    const unsigned long long lim = limit_ns ? limit_ns : ptx::kWaitLimitNs;
    const int sw = withhold_first_arrive ? 1 : 0;
    if (cudaMemcpyToSymbol(g_tc_wait_limit_ns, &lim, sizeof(lim)) != cudaSuccess ||
        cudaMemcpyToSymbol(g_tc_withhold_first_arrive, &sw, sizeof(sw)) != cudaSuccess) {
        cudaGetLastError();
        return GTA_ERR_CUDA;
    }
    return GTA_OK;
}

}  // namespace gta
