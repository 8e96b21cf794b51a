// tcgen05 / TMA (sm_100a) prefill path for bf16, d_h = 128.
//
//   sm100_attention_kernel : shared attention map per query group, online softmax, latent P C
//       (Sec. 3.3, reformulated equation; causal sum of App. B.1.1) -> normalised L (bf16).
//   The decoder + gate kernel that consumes L is in gta_sm100_decoder.cu.
#include "gta_sm100.cuh"

#include <cuda.h>

#include "sm100_ptx.cuh"
#include "tma_host.cuh"

namespace gta {

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// --------------------------------------------------------------------------- attention kernel
// A work item = two adjacent 128-row query tiles of one attention map x one 256-column slice of
// the latent, run by a CTA pair (cluster of 2, tcgen05 cta_group::2): each CTA owns one query tile
// (its own S / P / O in its own TMEM) and stages HALF of every key tile (64 of the 128 keys for
// S = Q K^T, 128 of the 256 latent columns for O += P C), so K and C cross L2 -> shared memory once
// per 256 query rows and the ring is four key tiles deep.  (The 128 x d_l fp32 output does not fit
// the 512 TMEM columns next to the score tiles, so d_l is cut in slices of 256 and each slice item
// recomputes the scores.)  Persistent: a pair walks a static list of items, heaviest (latest)
// query tiles first, dealt to the pairs in snake order.  Per 128-key tile j:
//   S_j = Q K_j^T            tcgen05.mma M = 256, smem x smem -> TMEM (two S buffers, ping-pong)
//   P_j = exp2(S_j c - m)    256 softmax threads per CTA, two per row (64 keys each, row maximum
//                            exchanged through shared memory); P_j (bf16) overwrites S_j in TMEM
//   O  += P_j C_j            tcgen05.mma M = 256, TMEM x smem (C is the MN-major B operand) -> TMEM
// The running maximum is only raised when it grows by more than 2^8 (the accumulators stay in
// range and O needs rescaling on few tiles); O is divided by the row sum at the end and written
// as bf16 to L[B, n_q, N, d_l].  The ring and the score pipeline run on across items.  The lower
// query tile of a pair sees one fully masked key tile per item (its probabilities are zero).
constexpr int kAttnThreads = 320;
constexpr int kAttnStages = 4;
constexpr int kKeyTile = 128;
constexpr int kSlice = 256;
constexpr uint32_t kQBytes = 128 * 128 * 2;                 // 32 KB: this CTA's query tile
constexpr uint32_t kKHalfBytes = (kKeyTile / 2) * 128 * 2;  // 16 KB: this CTA's 64 keys
constexpr uint32_t kCHalfBytes = kKeyTile * (kSlice / 2) * 2;   // 32 KB: this CTA's 128 latent columns
constexpr uint32_t kAttnStageBytes = kKHalfBytes + kCHalfBytes;   // 48 KB
constexpr uint32_t kAttnRingOff = kQBytes;
constexpr uint32_t kAttnXchgOff = kAttnRingOff + kAttnStages * kAttnStageBytes;   // float [2][4][2][32]
constexpr uint32_t kAttnBarOff = kAttnXchgOff + 2 * 4 * 2 * 32 * 4;
constexpr uint32_t kAttnAlignSlack = 768;   // the 227 KB limit leaves no more; checked in the kernel
constexpr uint32_t kAttnSmemTotal = kAttnBarOff + 256 + kAttnAlignSlack;
static_assert(kAttnSmemTotal <= 232448, "attention kernel shared memory exceeds the per-CTA limit");

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// 2^x on the FMA pipe (x <= ~8; anything below -126 gives ~1e-38): round to the nearest integer with
// the 1.5 * 2^23 trick, cubic for the fraction in [-1/2, 1/2] (relative error < 8e-5, well inside the
// bf16 rounding of P), exponent patched in with integer arithmetic.  Used for one element in four so
// that the MUFU unit, which paces the exponential phase, carries three quarters of them.
__device__ __forceinline__ float poly_exp2(float x) {
    x = fmaxf(x, -126.f);
    const float t = x + 12582912.f;
    const float f = x - (t - 12582912.f);
    float p = fmaf(f, 0.05517165f, 0.24261113f);
    p = fmaf(f, p, 0.69326097f);
    p = fmaf(f, p, 0.99992806f);
    return __int_as_float(__float_as_int(p) + (__float_as_int(t) << 23));
}
__device__ __forceinline__ void pair_sync(int quarter) {   // the two softmax warps of a TMEM lane quarter
    asm volatile("bar.sync %0, 64;" ::"r"(quarter + 1) : "memory");
}

struct AttnItem {
    int b, g, slice, qp, n_tiles;   // qp: pair of query tiles (2 qp, 2 qp + 1)
};

// Item `n` of CTA pair `pr`: position p in the list sorted by descending query tile, rounds dealt
// alternately left-to-right and right-to-left.  Returns false past the end of the list.
__device__ __forceinline__ bool attn_item(const Dims& d, int n_qt, int n_qp, int n_slices, long long total, int G,
                                          int pr, int n, AttnItem* it) {
    const long long p = (long long)n * G + ((n & 1) ? (G - 1 - pr) : pr);
    if (p >= total) return false;
    long long r = p;
    it->slice = (int)(r % n_slices); r /= n_slices;
    it->g = (int)(r % d.n_q); r /= d.n_q;
    it->b = (int)(r % d.B); r /= d.B;
    it->qp = n_qp - 1 - (int)r;
    it->n_tiles = d.causal ? min(2 * it->qp + 2, n_qt) : n_qt;
    return true;
}

__global__ void __launch_bounds__(kAttnThreads, 1)
sm100_attention_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                       const __grid_constant__ CUtensorMap tm_c, Dims d, __nv_bfloat16* __restrict__ o_lat,
                       int32_t* status_word) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    float* xchg = reinterpret_cast<float*>(smem + kAttnXchgOff);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kAttnBarOff);
    uint64_t* q_full = bars;            // leader CTA; both producers arrive
    uint64_t* q_empty = bars + 1;       // both CTAs (multicast commit)
    uint64_t* full = bars + 2;          // [4] leader CTA; both producers arrive
    uint64_t* empty = bars + 6;         // [4] both CTAs (multicast commit)
    uint64_t* s_full = bars + 10;       // [2] both CTAs (multicast commit)
    uint64_t* p_full = bars + 12;       // [2] leader CTA; 16 softmax warps arrive
    uint64_t* o_done = bars + 14;       // both CTAs (multicast commit)
    uint64_t* o_free = bars + 15;       // leader CTA; 16 softmax warps arrive
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 16);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile int* drain_flag = abort_flag + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();          // 0 = leader
    const int G = gridDim.x >> 1, pr = blockIdx.x >> 1;    // CTA pairs, this pair
    // the decoder + gate kernel may be scheduled as SMs free up: its gate phase does not need L, and
    // it waits for this whole grid before it reads L
    ptx::grid_launch_dependents();
    const bool bad_align = (uint32_t)(smem - smem_raw) > kAttnAlignSlack;   // cannot happen with a 256-byte aligned window
    const int n_slices = d.d_l / kSlice;
    const int n_qt = (d.N + 127) / 128, n_qp = (n_qt + 1) / 2;
    const long long total = bad_align ? 0 : (long long)n_qp * n_slices * d.n_q * d.B;

    if (threadIdx.x == 0) {
        ptx::mbar_init(q_full, 2);
        ptx::mbar_init(q_empty, 1);
        for (int s = 0; s < kAttnStages; ++s) { ptx::mbar_init(&full[s], 2); ptx::mbar_init(&empty[s], 1); }
        for (int s = 0; s < 2; ++s) { ptx::mbar_init(&s_full[s], 1); ptx::mbar_init(&p_full[s], 16); }
        ptx::mbar_init(o_done, 1);
        ptx::mbar_init(o_free, 16);
        *abort_flag = 0;
        *drain_flag = 0;
        ptx::fence_mbar_init();
        if (bad_align) raise_status(status_word, GTA_ERR_CUDA);
    }
    if (warp == 1) ptx::tmem_alloc_pair(tmem_slot, 512);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_arrive();     // the peer's barriers exist before anything is signalled to them
    ptx::cluster_wait();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_o = tmem_base + 256;

    if (warp == 0) {
        if (ptx::elect_one()) {
            ptx::prefetch_tensormap(&tm_q); ptx::prefetch_tensormap(&tm_k); ptx::prefetch_tensormap(&tm_c);
            const uint32_t q_full_leader = ptx::map_to_cta(ptx::smem_addr(q_full), 0);
            int tj = 0;                 // key tiles issued so far (ring position), across items
            bool ok = true;
            AttnItem w;
            for (int n = 0; ok && attn_item(d, n_qt, n_qp, n_slices, total, G, pr, n, &w); ++n) {
                const int kg = d.q_to_k(w.g), cg = d.q_to_c(w.g);
                const int q0 = (2 * w.qp + (int)rank) * 128;       // this CTA's query rows
                ok = ptx::mbar_wait(q_empty, (n & 1) ^ 1, abort_flag);
                if (!ok) break;
                ptx::mbar_arrive_expect_tx_cluster(q_full_leader, kQBytes);
                ptx::tma_load_3d_pair(smem, &tm_q, q_full_leader, 0, q0, w.b * d.n_q + w.g);
                ptx::tma_load_3d_pair(smem + 16384, &tm_q, q_full_leader, 64, q0, w.b * d.n_q + w.g);
                for (int j = 0; j < w.n_tiles; ++j, ++tj) {
                    const int s = tj % kAttnStages;
                    const uint32_t ph = (tj / kAttnStages) & 1;
                    ok = ptx::mbar_wait(&empty[s], ph ^ 1, abort_flag);
                    if (!ok) break;
                    uint8_t* k_s = smem + kAttnRingOff + s * kAttnStageBytes;
                    uint8_t* c_s = k_s + kKHalfBytes;
                    const uint32_t bar = ptx::map_to_cta(ptx::smem_addr(&full[s]), 0);
                    ptx::mbar_arrive_expect_tx_cluster(bar, kAttnStageBytes);
                    const int key0 = j * kKeyTile + (int)rank * 64;         // this CTA's 64 keys of the tile
                    ptx::tma_load_3d_pair(k_s, &tm_k, bar, 0, key0, w.b * d.n_k + kg);
                    ptx::tma_load_3d_pair(k_s + 8192, &tm_k, bar, 64, key0, w.b * d.n_k + kg);
                    const int col0 = w.slice * kSlice + (int)rank * 128;     // this CTA's 128 latent columns
                    ptx::tma_load_3d_pair(c_s, &tm_c, bar, col0, j * kKeyTile, w.b * d.n_c + cg);
                    ptx::tma_load_3d_pair(c_s + 16384, &tm_c, bar, col0 + 64, j * kKeyTile, w.b * d.n_c + cg);
                }
            }
            if (*abort_flag && rank == 0) {   // drain what was armed (bounded), so no copy lands after exit
                ptx::mbar_wait(q_full, 0, drain_flag);
                ptx::mbar_wait(q_full, 1, drain_flag);
                for (int back = 1; back <= kAttnStages && tj - back >= 0; ++back) {
                    const int jq = tj - back;
                    ptx::mbar_wait(&full[jq % kAttnStages], (jq / kAttnStages) & 1, drain_flag);
                }
            }
        }
    } else if (warp == 1) {
        if (rank == 0 && ptx::elect_one()) {
            constexpr uint32_t idesc_qk = ptx::make_idesc_bf16(256, kKeyTile, 0, 0);   // both K-major
            constexpr uint32_t idesc_pv = ptx::make_idesc_bf16(256, kSlice, 0, 1);     // B = C, MN-major
            const uint32_t q_addr = ptx::smem_addr(smem);
            bool ok = true;
            // S = Q K^T of ring tile tj; `first` / `last`: first / last key tile of its item n
            auto issue_qk = [&](int tj, int n, bool first, bool last) {
                if (first) ok = ptx::mbar_wait(q_full, n & 1, abort_flag);
                if (ok) ok = ptx::mbar_wait(&full[tj % kAttnStages], (tj / kAttnStages) & 1, abort_flag);
                if (!ok) return;
                ptx::tc_fence_after_sync();
                const uint32_t k_addr = ptx::smem_addr(smem + kAttnRingOff + (tj % kAttnStages) * kAttnStageBytes);
                const uint32_t s_tmem = tmem_base + (tj & 1) * 128;
#pragma unroll
                for (int k8 = 0; k8 < 8; ++k8)
                    ptx::mma_ss_pair(s_tmem, ptx::make_smem_desc(q_addr + (k8 >> 2) * 16384 + (k8 & 3) * 32, 16, 1024),
                                     ptx::make_smem_desc(k_addr + (k8 >> 2) * 8192 + (k8 & 3) * 32, 16, 1024), idesc_qk,
                                     k8 ? 1u : 0u);
                ptx::tc_commit_pair(&s_full[tj & 1], 3);
                if (last) ptx::tc_commit_pair(q_empty, 3);
            };
            int tj = 0;
            AttnItem w, nxt;
            bool have = attn_item(d, n_qt, n_qp, n_slices, total, G, pr, 0, &w);
            if (have) issue_qk(0, 0, true, w.n_tiles == 1);
            for (int n = 0; have && ok; ++n) {
                const bool have_next = attn_item(d, n_qt, n_qp, n_slices, total, G, pr, n + 1, &nxt);
                for (int j = 0; j < w.n_tiles && ok; ++j, ++tj) {
                    // look ahead: the item's next score tile goes to the tensor pipe before this
                    // tile's P C, so the softmax warps never wait for scores
                    if (j + 1 < w.n_tiles) issue_qk(tj + 1, n, false, j + 2 == w.n_tiles);
                    if (!ok) break;
                    ok = ptx::mbar_wait(&p_full[tj & 1], (tj >> 1) & 1, abort_flag);
                    if (ok && j == 0 && n > 0) ok = ptx::mbar_wait(o_free, (n - 1) & 1, abort_flag);
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    const uint32_t c_addr =
                        ptx::smem_addr(smem + kAttnRingOff + (tj % kAttnStages) * kAttnStageBytes + kKHalfBytes);
                    const uint32_t p_tmem = tmem_base + (tj & 1) * 128;
#pragma unroll
                    for (int k8 = 0; k8 < 8; ++k8)
                        ptx::mma_ts_pair(tmem_o, p_tmem + k8 * 8, ptx::make_smem_desc(c_addr + k8 * 2048, 16384, 1024),
                                         idesc_pv, (j > 0 || k8 > 0) ? 1u : 0u);
                    ptx::tc_commit_pair(o_done, 3);
                    ptx::tc_commit_pair(&empty[tj % kAttnStages], 3);
                    // ... but the NEXT item's first score tile has to wait for that item's Q, which can
                    // only be requested once this item's last Q K^T is done: it goes after the last P C
                    if (j + 1 == w.n_tiles && have_next) issue_qk(tj + 1, n + 1, true, nxt.n_tiles == 1);
                }
                w = nxt;
                have = have_next;
            }
        }
    } else {
        const int quarter = warp & 3;
        const int half = (warp - 2) >> 2;            // which 64 keys of a tile / which 128 output columns
        const int row = quarter * 32 + lane;
        const uint32_t lane_base = ((uint32_t)(quarter * 32) << 16);
        const float c_scale = d.scale * 1.4426950408889634f;
        const uint32_t p_full_leader[2] = {ptx::map_to_cta(ptx::smem_addr(&p_full[0]), 0),
                                           ptx::map_to_cta(ptx::smem_addr(&p_full[1]), 0)};
        const uint32_t o_free_leader = ptx::map_to_cta(ptx::smem_addr(o_free), 0);
        bool ok = true;
        int tj = 0;
        AttnItem w;
        for (int n = 0; ok && attn_item(d, n_qt, n_qp, n_slices, total, G, pr, n, &w); ++n) {
            const int t = (2 * w.qp + (int)rank) * 128 + row;
            float m = -INFINITY, l = 0.f;            // m in scaled (log2) units; l = this thread's share of the row sum
            for (int j = 0; j < w.n_tiles && ok; ++j, ++tj) {
                ok = __all_sync(0xffffffffu, ptx::mbar_wait(&s_full[tj & 1], (tj >> 1) & 1, abort_flag));
                if (!ok) break;   // warp-uniform: the TMEM instructions below are warp-collective
                ptx::tc_fence_after_sync();
                const uint32_t s_tmem = tmem_base + lane_base + (tj & 1) * 128;
                float sv[64];
                {
                    uint32_t r0[32], r1[32];
                    ptx::tmem_ld32(s_tmem + half * 64, r0);
                    ptx::tmem_ld32(s_tmem + half * 64 + 32, r1);
                    ptx::tmem_wait_ld();
#pragma unroll
                    for (int e = 0; e < 32; ++e) { sv[e] = __uint_as_float(r0[e]); sv[32 + e] = __uint_as_float(r1[e]); }
                }
                // mask: keys past the sequence end, and (causal) keys after the query, on boundary tiles
                const int key0 = j * kKeyTile + half * 64;
                const int last_key = d.causal ? min(t, d.N - 1) : d.N - 1;
                if (key0 + 63 > last_key) {
#pragma unroll
                    for (int e = 0; e < 64; ++e)
                        if (key0 + e > last_key) sv[e] = -INFINITY;
                }
                float mx[4] = {sv[0], sv[1], sv[2], sv[3]};
#pragma unroll
                for (int e = 4; e < 64; e += 4) {
                    mx[0] = fmaxf(mx[0], sv[e]); mx[1] = fmaxf(mx[1], sv[e + 1]);
                    mx[2] = fmaxf(mx[2], sv[e + 2]); mx[3] = fmaxf(mx[3], sv[e + 3]);
                }
                const float m_half = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * c_scale;   // c_scale > 0
                float* xs = xchg + (tj & 1) * 256 + quarter * 64;
                xs[half * 32 + lane] = m_half;
                pair_sync(quarter);
                const float m_tile = fmaxf(m_half, xs[(half ^ 1) * 32 + lane]);
                float alpha = 1.f;
                const bool raise = m_tile > m + 8.f;     // also true on the first live tile (m = -inf); same in both halves
                if (raise) {
                    alpha = fast_exp2(m - m_tile);
                    m = m_tile;
                }
                const float neg_m = (m == -INFINITY) ? 0.f : -m;   // a fully masked row keeps p = 0
                float sum[4] = {0.f, 0.f, 0.f, 0.f};
                uint32_t packed[32];
#pragma unroll
                for (int e = 0; e < 32; ++e) {
                    const float x0 = fmaf(sv[2 * e], c_scale, neg_m), x1 = fmaf(sv[2 * e + 1], c_scale, neg_m);
                    const float p0 = fast_exp2(x0);
                    const float p1 = (e & 1) ? poly_exp2(x1) : fast_exp2(x1);
                    sum[e & 3] += p0 + p1;
                    packed[e] = pack_bf16x2(p0, p1);
                }
                l = l * alpha + ((sum[0] + sum[1]) + (sum[2] + sum[3]));
                // P_j (bf16 pairs): this thread's 64 keys = packed columns [32 half, 32 half + 32) of S_j
                ptx::tmem_st32(s_tmem + half * 32, packed);
                if (j > 0) {
                    // Every completion of o_done is waited for, in order, whether or not O has to be
                    // rescaled: a parity wait is only meaningful one phase at a time, and the
                    // epilogue's wait below must not find the barrier two phases behind.
                    ok = __all_sync(0xffffffffu, ptx::mbar_wait(o_done, (tj - 1) & 1, abort_flag));
                    if (!ok) break;
                    if (__any_sync(0xffffffffu, raise)) {
                        ptx::tc_fence_after_sync();
#pragma unroll 1
                        for (int ch = 0; ch < 4; ++ch) {     // this thread's 128 of the 256 output columns
                            uint32_t r[32];
                            ptx::tmem_ld32(tmem_o + lane_base + half * 128 + ch * 32, r);
                            ptx::tmem_wait_ld();
#pragma unroll
                            for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
                            ptx::tmem_st32(tmem_o + lane_base + half * 128 + ch * 32, r);
                        }
                    }
                }
                ptx::tmem_wait_st();
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive_cluster(p_full_leader[tj & 1]);
            }
            if (!ok) break;
            // ---- item epilogue: whole row sum, normalise, store this thread's 128 columns
            float* xs = xchg + (tj & 1) * 256 + quarter * 64;   // tj already points past the item: next parity
            xs[half * 32 + lane] = l;
            pair_sync(quarter);
            const float inv_l = 1.f / (l + xs[(half ^ 1) * 32 + lane]);
            ok = __all_sync(0xffffffffu, ptx::mbar_wait(o_done, (tj - 1) & 1, abort_flag));
            if (!ok) break;
            ptx::tc_fence_after_sync();
            __nv_bfloat16* o_row = o_lat + (((size_t)w.b * d.n_q + w.g) * d.N + (t < d.N ? t : 0)) * d.d_l +
                                   w.slice * kSlice + half * 128;
#pragma unroll 1
            for (int ch = 0; ch < 4; ++ch) {
                uint32_t r[32];
                ptx::tmem_ld32(tmem_o + lane_base + half * 128 + ch * 32, r);
                ptx::tmem_wait_ld();
                if (t < d.N) {
#pragma unroll
                    for (int v = 0; v < 2; ++v) {      // 2 x 32 bytes: whole sectors, half as many stores
                        uint32_t ww[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            ww[e] = pack_bf16x2(__uint_as_float(r[16 * v + 2 * e]) * inv_l,
                                                __uint_as_float(r[16 * v + 2 * e + 1]) * inv_l);
                        ptx::st_global_256(o_row + ch * 32 + v * 16, ww);
                    }
                }
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_cluster(o_free_leader);
            pair_sync(quarter);   // the exchange slot may be rewritten by the next tile of the same parity
        }
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_arrive();     // neither CTA leaves (or frees TMEM) while the other may still signal it
    ptx::cluster_wait();
    if (warp == 1) ptx::tmem_dealloc_pair(tmem_base, 512);
    if (threadIdx.x == 0 && *abort_flag) raise_status(status_word, GTA_ERR_TIMEOUT);
}

// --------------------------------------------------------------------------- host side
bool sm100_prefill_supported(const Dims& d, int dtype) {
    return dtype == GTA_BF16 && d.d_h == 128 && d.d_l % 256 == 0 && d.d_l <= 1024 && d.H % 64 == 0 && d.N >= 1;
}

gta_status_t launch_sm100_prefill(const Dims& d, const void* q, const void* k, const void* c, const void* x,
                                  const void* w_p, const void* w_g, void* out, void* workspace,
                                  int32_t* status_word, cudaStream_t stream, int stages, int* launches) {
    if (stages & 1) {
        CUtensorMap tm_q, tm_k, tm_c;
        const uint32_t box[3] = {64, 128, 1}, box_k[3] = {64, 64, 1};
        const uint64_t dq[3] = {(uint64_t)d.d_h, (uint64_t)d.N, (uint64_t)d.B * d.n_q};
        const uint64_t dk[3] = {(uint64_t)d.d_h, (uint64_t)d.N, (uint64_t)d.B * d.n_k};
        const uint64_t dc[3] = {(uint64_t)d.d_l, (uint64_t)d.N, (uint64_t)d.B * d.n_c};
        if (!make_bf16_map(&tm_q, q, 3, dq, box) || !make_bf16_map(&tm_k, k, 3, dk, box_k) ||
            !make_bf16_map(&tm_c, c, 3, dc, box))
            return GTA_ERR_CUDA;
        if (cudaFuncSetAttribute(sm100_attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kAttnSmemTotal) != cudaSuccess)
            return GTA_ERR_CUDA;
        const int n_qt = (d.N + 127) / 128, n_qp = (n_qt + 1) / 2;
        const long long n_items = (long long)n_qp * (d.d_l / kSlice) * d.n_q * d.B;
        if (n_items > 0x3fffffffLL) return GTA_ERR_UNSUPPORTED;
        cudaLaunchConfig_t cfg = {};
        cfg.blockDim = dim3(kAttnThreads);
        cfg.dynamicSmemBytes = kAttnSmemTotal;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        // a persistent grid must be resident at once: as many CTA pairs as the device can hold
        static thread_local int cached_dev = -1, cached_pairs = 0;
        int dev = 0, sms = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return GTA_ERR_CUDA;
        if (dev != cached_dev) {
            if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 2)
                return GTA_ERR_CUDA;
            cfg.gridDim = dim3(2 * (sms / 2));
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, sm100_attention_kernel, &cfg) != cudaSuccess || n < 1)
                return GTA_ERR_CUDA;
            cached_dev = dev;
            cached_pairs = n;
        }
        const int pairs = (int)(n_items < cached_pairs ? n_items : cached_pairs);
        cfg.gridDim = dim3(2 * pairs);
        if (cudaLaunchKernelEx(&cfg, sm100_attention_kernel, tm_q, tm_k, tm_c, d, (__nv_bfloat16*)workspace,
                               status_word) != cudaSuccess)
            return GTA_ERR_CUDA;
        if (cudaGetLastError() != cudaSuccess) return GTA_ERR_CUDA;
        *launches += 1;
    }
    if (stages & 2) {
        gta_status_t st = launch_sm100_decoder(d, workspace, x, w_p, w_g, out, status_word, stream);
        if (st != GTA_OK) return st;
        *launches += 1;
    }
    return GTA_OK;
}

}  // namespace gta
