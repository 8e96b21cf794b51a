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
// per 256 query rows and the ring is three key tiles deep.  (The 128 x d_l fp32 output does not fit
// the 512 TMEM columns next to the score tiles, so d_l is cut in slices of 256 and each slice item
// recomputes the scores.)  Persistent: a pair walks a static list of items, heaviest (latest)
// query tiles first, dealt to the pairs in snake order.  Per 128-key tile j:
//   S_j = Q K_j^T            tcgen05.mma M = 256, smem x smem -> TMEM (two S buffers, ping-pong)
//   P_j = exp2(S_j c - m)    512 softmax threads per CTA, four per row (32 keys each, row maximum
//                            exchanged through shared memory); P_j (bf16) overwrites S_j in TMEM
//   O  += P_j C_j            tcgen05.mma M = 256, TMEM x smem (C is the MN-major B operand) -> TMEM
// The running maximum is only raised when it grows by more than 2^8 (the accumulators stay in
// range and O needs rescaling on few tiles).  At the end of an item the softmax threads only hand
// their row sums over: four epilogue warps (one per TMEM lane quarter) divide O by the row sum,
// stage it in shared memory as bf16 and write it to L[B, n_q, N, d_l] with TMA tensor stores
// (whole 128-byte lines, clipped at the sequence end), while the softmax threads are already on
// the first score tile of the next item.  The ring and the score pipeline run on across items.  The lower
// query tile of a pair sees one fully masked key tile per item (its probabilities are zero).
constexpr int kAttnThreads = 64 + 512 + 128;   // TMA warp, MMA warp, 16 softmax warps, 4 epilogue warps
constexpr int kAttnStages = 3;
constexpr int kKeyTile = 128;
constexpr int kSlice = 256;      // widest latent slice of an item (template parameter SLICE: 256 or 128)
constexpr uint32_t kQBytes = 128 * 128 * 2;                 // 32 KB: this CTA's query tile
constexpr uint32_t kKHalfBytes = (kKeyTile / 2) * 128 * 2;  // 16 KB: this CTA's 64 keys
constexpr uint32_t kCHalfBytes = kKeyTile * (kSlice / 2) * 2;   // 32 KB: this CTA's 128 latent columns
constexpr uint32_t kAttnStageBytes = kKHalfBytes + kCHalfBytes;   // 48 KB
constexpr uint32_t kAttnRingOff = kQBytes;
// Two 32 KB buffers alternate between two roles: buffer n & 1 holds the query tile of item n, then
// (once the item's last Q K^T is done) the two 128 x 64 output boxes of its epilogue, then the query
// tile of item n + 2.  So the next item's Q is loaded long before the current item ends.
constexpr uint32_t kAttnOutOff = kAttnRingOff + kAttnStages * kAttnStageBytes;   // the second buffer (the first is at 0)
constexpr uint32_t kAttnOutBoxBytes = 128 * 64 * 2;
constexpr uint32_t kAttnXchgOff = kAttnOutOff + 2 * kAttnOutBoxBytes;   // 2 KB, per lane quarter: bf16 [2][4][32] or float [4][32]
constexpr uint32_t kAttnSumOff = kAttnXchgOff + 2 * 4 * 2 * 32 * 4;      // 4 KB: float [2 items][4 quarters][4 parts][32] row sums
constexpr uint32_t kAttnBarOff = kAttnSumOff + 2 * 4 * 4 * 32 * 4;
constexpr uint32_t kAttnAlignSlack = 1024;  // checked in the kernel
constexpr uint32_t kAttnSmemTotal = kAttnBarOff + 256 + kAttnAlignSlack;
static_assert(kAttnSmemTotal <= 232448, "attention kernel shared memory exceeds the per-CTA limit");

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// 2^x for a pair of values on the FMA pipe (x <= ~8; anything below -126 gives ~1e-38): round to the
// nearest integer with the 1.5 * 2^23 trick, cubic for the fraction in [-1/2, 1/2] (relative error
// < 8e-5, well inside the bf16 rounding of P), exponent patched in with integer arithmetic.  Used for
// some of the pairs so that the MUFU unit, which paces the exponential phase, carries fewer of them.
__device__ __forceinline__ void poly_exp2_pair(uint64_t x2, float& p0, float& p1) {
    float x0, x1;
    ptx::f32x2_split(x2, x0, x1);
    x2 = ptx::f32x2(fmaxf(x0, -126.f), fmaxf(x1, -126.f));
    const uint64_t t2 = ptx::add2(x2, ptx::f32x2(12582912.f, 12582912.f));
    const uint64_t u2 = ptx::add2(t2, ptx::f32x2(-12582912.f, -12582912.f));
    const uint64_t f2 = ptx::fma2(u2, ptx::f32x2(-1.f, -1.f), x2);
    uint64_t q2 = ptx::fma2(f2, ptx::f32x2(0.05517165f, 0.05517165f), ptx::f32x2(0.24261113f, 0.24261113f));
    q2 = ptx::fma2(f2, q2, ptx::f32x2(0.69326097f, 0.69326097f));
    q2 = ptx::fma2(f2, q2, ptx::f32x2(0.99992806f, 0.99992806f));
    float q0, q1, t0, t1;
    ptx::f32x2_split(q2, q0, q1);
    ptx::f32x2_split(t2, t0, t1);
    p0 = __int_as_float(__float_as_int(q0) + (__float_as_int(t0) << 23));
    p1 = __int_as_float(__float_as_int(q1) + (__float_as_int(t1) << 23));
}
// which of every eight pairs of exponentials run on the FMA pipe instead of the MUFU unit
__device__ constexpr bool kPolyPair[8] = {false, false, true, false, false, true, false, true};
__device__ __forceinline__ void epilogue_sync() {   // the four epilogue warps
    asm volatile("bar.sync 5, 128;" ::: "memory");
}
__device__ __forceinline__ void quarter_sync(int quarter) {   // the four softmax warps of a TMEM lane quarter
    asm volatile("bar.sync %0, 128;" ::"r"(quarter + 1) : "memory");
}
struct AttnItem {
    int b, g, slice, qp, n_tiles;   // qp: pair of query tiles (2 qp, 2 qp + 1)
};

// Item `n` of CTA pair `pr`: position p in the list sorted by descending query tile, rounds dealt
// alternately left-to-right and right-to-left.  Returns false past the end of the list.
__device__ __forceinline__ bool attn_item(const Dims& d, int n_kt, int n_qp, int n_slices, long long total, int G,
                                          int pr, int n, AttnItem* it) {
    // the host refuses more than 2^30 items, so 32-bit arithmetic is enough (64-bit divisions are
    // slow enough to show at every item boundary)
    const long long p64 = (long long)n * G + ((n & 1) ? (G - 1 - pr) : pr);
    if (p64 >= total) return false;
    unsigned r = (unsigned)p64;
    it->slice = (int)(r % (unsigned)n_slices); r /= (unsigned)n_slices;
    it->g = (int)(r % (unsigned)d.n_q); r /= (unsigned)d.n_q;
    it->b = (int)(r % (unsigned)d.B); r /= (unsigned)d.B;
    it->qp = n_qp - 1 - (int)r;
    // key tiles the pair's 256 query rows see: up to their last row's key (2 qp + 2) 128 - 1 + Nk - N
    it->n_tiles = d.causal ? min((((2 * it->qp + 2) * 128 - 1 + d.Nk - d.N) >> 7) + 1, n_kt) : n_kt;
    return true;
}

// DH: head dimension of Q and K (64 or 128); SLICE: latent columns per item (128 or 256).  The
// shared-memory layout is the one of the largest case; the smaller ones use the front of each area.
template <int DH, int SLICE>
__global__ void __launch_bounds__(kAttnThreads, 1)
sm100_attention_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                       const __grid_constant__ CUtensorMap tm_c, const __grid_constant__ CUtensorMap tm_o, Dims d,
                       int32_t* status_word) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    float* xchg = reinterpret_cast<float*>(smem + kAttnXchgOff);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kAttnBarOff);
    uint64_t* q_full = bars;            // leader CTA; both producers arrive
    uint64_t* stage_free = bars + 1;    // this CTA; its epilogue's stores have read the buffer (one thread arrives)
    uint64_t* full = bars + 2;          // [4] leader CTA; both producers arrive
    uint64_t* empty = bars + 6;         // [4] both CTAs (multicast commit)
    uint64_t* s_full = bars + 10;       // [2] both CTAs (multicast commit)
    uint64_t* p_full = bars + 12;       // [2] leader CTA; 32 softmax warps arrive
    uint64_t* o_done = bars + 14;       // both CTAs (multicast commit)
    uint64_t* o_free = bars + 15;       // leader CTA; 8 epilogue warps arrive
    uint64_t* epi_ready = bars + 16;    // this CTA; its 16 softmax warps arrive (row sums of an item are in place)
    uint64_t* o_item = bars + 17;       // both CTAs (multicast commit): the last sum of an item is complete
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 18);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile int* drain_flag = abort_flag + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();          // 0 = leader
    const int G = gridDim.x >> 1, pr = blockIdx.x >> 1;    // CTA pairs, this pair
    const bool bad_align = (uint32_t)(smem - smem_raw) > kAttnAlignSlack;   // cannot happen with a 256-byte aligned window
    constexpr uint32_t kQLoadBytes = 128 * DH * 2;                 // this CTA's query tile
    constexpr uint32_t kKLoadBytes = (kKeyTile / 2) * DH * 2;      // this CTA's 64 keys
    constexpr uint32_t kCLoadBytes = kKeyTile * (SLICE / 2) * 2;   // this CTA's SLICE / 2 latent columns
    const int n_slices = d.d_l / SLICE;
    const int n_qt = (d.N + 127) / 128, n_qp = (n_qt + 1) / 2;
    const int n_kt = (d.Nk + 127) / 128;          // key tiles
    const long long total = bad_align ? 0 : (long long)n_qp * n_slices * d.n_q * d.B;

    if (threadIdx.x == 0) {
        ptx::mbar_init(q_full, 2);
        ptx::mbar_init(stage_free, 1);
        for (int s = 0; s < kAttnStages; ++s) { ptx::mbar_init(&full[s], 2); ptx::mbar_init(&empty[s], 1); }
        for (int s = 0; s < 2; ++s) { ptx::mbar_init(&s_full[s], 1); ptx::mbar_init(&p_full[s], 32); }
        ptx::mbar_init(o_done, 1);
        ptx::mbar_init(o_free, 8);
        ptx::mbar_init(epi_ready, 16);
        ptx::mbar_init(o_item, 1);
        *abort_flag = 0;
        *drain_flag = 0;
        ptx::fence_mbar_init();
    }
    if (warp == 1) ptx::tmem_alloc_pair(tmem_slot, 512);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_arrive();     // the peer's barriers exist before anything is signalled to them
    ptx::cluster_wait();
    ptx::tc_fence_after_sync();
    // The kernel is launched with programmatic stream serialisation: everything above may have run
    // while the kernel before it in the stream was draining; nothing of global memory is touched
    // before this wait.  Only then may the decoder + gate kernel be scheduled (as SMs free up): its
    // gate phase reads X and W_G before its own wait, which orders it against this kernel alone.
    ptx::grid_dependency_wait();
    ptx::grid_launch_dependents();
    if (threadIdx.x == 0 && bad_align) raise_status(status_word, GTA_ERR_CUDA);
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_o = tmem_base + 256;

    if (warp == 0) {
        if (ptx::elect_one()) {
            ptx::prefetch_tensormap(&tm_q); ptx::prefetch_tensormap(&tm_k); ptx::prefetch_tensormap(&tm_c);
            const uint32_t q_full_leader = ptx::map_to_cta(ptx::smem_addr(q_full), 0);
            int tj = 0;                 // key tiles issued so far (ring position), across items
            bool ok = true;
            AttnItem w;
            for (int n = 0; ok && attn_item(d, n_kt, n_qp, n_slices, total, G, pr, n, &w); ++n) {
                const int kg = d.q_to_k(w.g), cg = d.q_to_c(w.g);
                const int q0 = (2 * w.qp + (int)rank) * 128;       // this CTA's query rows
                // buffer n & 1 is free once the epilogue of item n - 2 has stored out of it (which
                // also means every Q K^T of that item is done); every completion is waited for, in order
                if (n >= 2) ok = ptx::mbar_wait(stage_free, n & 1, abort_flag);
                if (!ok) break;
                uint8_t* q_s = smem + ((n & 1) ? kAttnOutOff : 0u);
                ptx::mbar_arrive_expect_tx_cluster(q_full_leader, kQLoadBytes);
                ptx::tma_load_3d_pair(q_s, &tm_q, q_full_leader, 0, q0, w.b * d.n_q + w.g);
                if (DH == 128) ptx::tma_load_3d_pair(q_s + 16384, &tm_q, q_full_leader, 64, q0, w.b * d.n_q + w.g);
                for (int j = 0; j < w.n_tiles; ++j, ++tj) {
                    const int s = tj % kAttnStages;
                    const uint32_t ph = (tj / kAttnStages) & 1;
                    ok = ptx::mbar_wait(&empty[s], ph ^ 1, abort_flag);
                    if (!ok) break;
                    uint8_t* k_s = smem + kAttnRingOff + s * kAttnStageBytes;
                    uint8_t* c_s = k_s + kKHalfBytes;
                    const uint32_t bar = ptx::map_to_cta(ptx::smem_addr(&full[s]), 0);
                    ptx::mbar_arrive_expect_tx_cluster(bar, kKLoadBytes + kCLoadBytes);
                    const int key0 = j * kKeyTile + (int)rank * 64;         // this CTA's 64 keys of the tile
                    ptx::tma_load_3d_pair(k_s, &tm_k, bar, 0, key0, w.b * d.n_k + kg);
                    if (DH == 128) ptx::tma_load_3d_pair(k_s + 8192, &tm_k, bar, 64, key0, w.b * d.n_k + kg);
                    const int col0 = w.slice * SLICE + (int)rank * (SLICE / 2);     // this CTA's latent columns
                    ptx::tma_load_3d_pair(c_s, &tm_c, bar, col0, j * kKeyTile, w.b * d.n_c + cg);
                    if (SLICE == 256)
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
            constexpr uint32_t idesc_pv = ptx::make_idesc_bf16(256, SLICE, 0, 1);      // B = C, MN-major
            bool ok = true;
            // S = Q K^T of ring tile tj; `first`: first key tile of its item n
            auto issue_qk = [&](int tj, int n, bool first) {
                if (first) ok = ptx::mbar_wait(q_full, n & 1, abort_flag);
                if (ok) ok = ptx::mbar_wait(&full[tj % kAttnStages], (tj / kAttnStages) & 1, abort_flag);
                if (!ok) return;
                ptx::tc_fence_after_sync();
                const uint32_t q_addr = ptx::smem_addr(smem + ((n & 1) ? kAttnOutOff : 0u));
                const uint32_t k_addr = ptx::smem_addr(smem + kAttnRingOff + (tj % kAttnStages) * kAttnStageBytes);
                const uint32_t s_tmem = tmem_base + (tj & 1) * 128;
#pragma unroll
                for (int k8 = 0; k8 < DH / 16; ++k8)
                    ptx::mma_ss_pair(s_tmem, ptx::make_smem_desc(q_addr + (k8 >> 2) * 16384 + (k8 & 3) * 32, 16, 1024),
                                     ptx::make_smem_desc(k_addr + (k8 >> 2) * 8192 + (k8 & 3) * 32, 16, 1024), idesc_qk,
                                     k8 ? 1u : 0u);
                ptx::tc_commit_pair(&s_full[tj & 1], 3);
            };
            int tj = 0;
            AttnItem w, nxt;
            bool have = attn_item(d, n_kt, n_qp, n_slices, total, G, pr, 0, &w);
            if (have) issue_qk(0, 0, true);
            for (int n = 0; have && ok; ++n) {
                const bool have_next = attn_item(d, n_kt, n_qp, n_slices, total, G, pr, n + 1, &nxt);
                for (int j = 0; j < w.n_tiles && ok; ++j, ++tj) {
                    // look ahead: the next score tile goes to the tensor pipe before this tile's P C, so
                    // the softmax warps never wait for scores.  Across items too, when the next
                    // item's Q has landed (it normally has: it is loaded into the other buffer well
                    // before this item ends); otherwise after this item's last P C, below.
                    bool next_item_early = false;
                    if (j + 1 < w.n_tiles) {
                        issue_qk(tj + 1, n, false);
                    } else if (have_next && ptx::mbar_test_wait(q_full, (n + 1) & 1)) {
                        issue_qk(tj + 1, n + 1, true);
                        next_item_early = true;
                    }
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
                    if (j + 1 == w.n_tiles) ptx::tc_commit_pair(o_item, 3);   // for the epilogue warps
                    ptx::tc_commit_pair(&empty[tj % kAttnStages], 3);
                    if (j + 1 == w.n_tiles && have_next && !next_item_early)
                        issue_qk(tj + 1, n + 1, true);
                }
                w = nxt;
                have = have_next;
            }
        }
    } else if (warp < 18) {
        // 16 softmax warps: four per TMEM lane quarter (warp % 4), each thread 32 of the 128 keys of its
        // row and 64 of the 256 output columns.  Four warps per scheduler hide the latencies of the
        // TMEM loads, the exchange and the exponentials behind one another.
        const int quarter = warp & 3;
        const int part = (warp - 2) >> 2;            // which 32 keys of a tile / which 64 output columns
        const int row = quarter * 32 + lane;
        const uint32_t lane_base = ((uint32_t)(quarter * 32) << 16);
        const float c_scale = d.scale * 1.4426950408889634f;
        const uint32_t p_full_leader[2] = {ptx::map_to_cta(ptx::smem_addr(&p_full[0]), 0),
                                           ptx::map_to_cta(ptx::smem_addr(&p_full[1]), 0)};
        __nv_bfloat16* xm = reinterpret_cast<__nv_bfloat16*>(xchg);   // [4 quarters][2][4][32] partial row maxima
        float* xsum = reinterpret_cast<float*>(smem + kAttnSumOff);
        // A wait that gives up raises the CTA's abort flag, after which every wait returns at once:
        // these warps then run their loops to the end all the same (on meaningless data), so that
        // the named barriers below are always reached by all of their threads.
        bool ok = true;
        int tj = 0;
        AttnItem w;
        for (int n = 0; attn_item(d, n_kt, n_qp, n_slices, total, G, pr, n, &w); ++n) {
            const int t = (2 * w.qp + (int)rank) * 128 + row;
            float m = -INFINITY, l = 0.f;            // m in scaled (log2) units; l = this thread's share of the row sum
            for (int j = 0; j < w.n_tiles; ++j, ++tj) {
                ok = __all_sync(0xffffffffu, ptx::mbar_wait(&s_full[tj & 1], (tj >> 1) & 1, abort_flag));
                ptx::tc_fence_after_sync();
                const uint32_t s_tmem = tmem_base + lane_base + (tj & 1) * 128;
                float sv[32];
                {
                    uint32_t r0[32];
                    ptx::tmem_ld32(s_tmem + part * 32, r0);
                    ptx::tmem_wait_ld();
#pragma unroll
                    for (int e = 0; e < 32; ++e) sv[e] = __uint_as_float(r0[e]);
                }
                // mask: keys past the sequence end, and (causal) keys after the query, on boundary tiles
                const int key0 = j * kKeyTile + part * 32;
                const int last_key = d.causal ? min(t + d.Nk - d.N, d.Nk - 1) : d.Nk - 1;
                if (key0 + 31 > last_key) {
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        if (key0 + e > last_key) sv[e] = -INFINITY;
                }
                float mx[2] = {ptx::max3(sv[0], sv[1], sv[2]), ptx::max3(sv[3], sv[4], sv[5])};
#pragma unroll
                for (int e = 6; e < 30; e += 4) {
                    mx[0] = ptx::max3(mx[0], sv[e], sv[e + 1]);
                    mx[1] = ptx::max3(mx[1], sv[e + 2], sv[e + 3]);
                }
                const float m_part = ptx::max3(mx[0], mx[1], fmaxf(sv[30], sv[31])) * c_scale;   // c_scale > 0
                __nv_bfloat16* xs = xm + (quarter * 2 + (tj & 1)) * 128;   // 512 bytes per quarter, shared with xl
                xs[part * 32 + lane] = __float2bfloat16_ru(m_part);
                quarter_sync(quarter);
                const float m_tile = fmaxf(fmaxf(__bfloat162float(xs[lane]), __bfloat162float(xs[32 + lane])),
                                           fmaxf(__bfloat162float(xs[64 + lane]), __bfloat162float(xs[96 + lane])));
                float alpha = 1.f;
                const bool raise = m_tile > m + 8.f;     // also true on the first live tile (m = -inf); same in all four threads
                if (raise) {
                    alpha = fast_exp2(m - m_tile);
                    m = m_tile;
                }
                const float neg_m = (m == -INFINITY) ? 0.f : -m;   // a fully masked row keeps p = 0
                const uint64_t cs2 = ptx::f32x2(c_scale, c_scale), nm2 = ptx::f32x2(neg_m, neg_m);
                uint64_t sum2[2] = {0ull, 0ull};         // two-wide fp32 arithmetic: half the issue slots
                uint32_t packed[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                    const uint64_t x2 = ptx::fma2(ptx::f32x2(sv[2 * e], sv[2 * e + 1]), cs2, nm2);
                    float p0, p1;
                    if (kPolyPair[e & 7]) {
                        poly_exp2_pair(x2, p0, p1);
                    } else {
                        float x0, x1;
                        ptx::f32x2_split(x2, x0, x1);
                        p0 = fast_exp2(x0);
                        p1 = fast_exp2(x1);
                    }
                    sum2[e & 1] = ptx::add2(sum2[e & 1], ptx::f32x2(p0, p1));
                    packed[e] = pack_bf16x2(p0, p1);
                }
                float s0, s1;
                ptx::f32x2_split(ptx::add2(sum2[0], sum2[1]), s0, s1);
                l = l * alpha + (s0 + s1);
                // P_j (bf16 pairs): this thread's 32 keys = packed columns [16 part, 16 part + 16) of S_j
                // (columns that other threads of the row read as scores: they did so before the exchange)
                ptx::tmem_st16(s_tmem + part * 16, packed);
                if (tj > 0) {
                    // Every completion of o_done is waited for, in order, whether or not O has to be
                    // rescaled (on the first tile of an item it never is): a parity wait is only
                    // meaningful one phase at a time.
                    ok = __all_sync(0xffffffffu, ptx::mbar_wait(o_done, (tj - 1) & 1, abort_flag));
                    if (j > 0 && __any_sync(0xffffffffu, raise)) {
                        ptx::tc_fence_after_sync();
#pragma unroll 1
                        for (int ch = 0; ch < SLICE / 128; ++ch) {     // this thread's quarter of the output columns
                            uint32_t r[32];
                            ptx::tmem_ld32(tmem_o + lane_base + part * (SLICE / 4) + ch * 32, r);
                            ptx::tmem_wait_ld();
                            const uint64_t a2 = ptx::f32x2(alpha, alpha);
#pragma unroll
                            for (int e = 0; e < 32; e += 2) {
                                float v0, v1;
                                ptx::f32x2_split(ptx::mul2(ptx::f32x2(__uint_as_float(r[e]), __uint_as_float(r[e + 1])), a2), v0, v1);
                                r[e] = __float_as_uint(v0);
                                r[e + 1] = __float_as_uint(v1);
                            }
                            ptx::tmem_st32(tmem_o + lane_base + part * (SLICE / 4) + ch * 32, r);
                        }
                    }
                }
                ptx::tmem_wait_st();
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive_cluster(p_full_leader[tj & 1]);
            }
            // ---- end of the item: the row sums go to the epilogue warps (double-buffered by item:
            //      the epilogue of item n reads them before it hands O back, which the sums of
            //      item n + 1 wait for, long before item n + 2 ends)
            xsum[(((n & 1) * 4 + quarter) * 4 + part) * 32 + lane] = l;
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(epi_ready);
        }
    } else {
        // 4 epilogue warps, one per TMEM lane quarter, a row per thread.  After the last sum of an item
        // (o_item: one completion per item, and the next cannot come before this item's O has been
        // handed back) they divide O by the row sum, round to bf16 into the staging boxes (box = 64 columns x
        // 128 rows, 128-byte swizzle: 16-byte chunk c of row r sits at chunk c ^ (r & 7)) and store
        // them with TMA: two passes of 128 columns.  O is handed back as soon as it has been read.
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const uint32_t lane_base = ((uint32_t)(quarter * 32) << 16);
        const uint32_t o_free_leader = ptx::map_to_cta(ptx::smem_addr(o_free), 0);
        const float* xsum = reinterpret_cast<const float*>(smem + kAttnSumOff);
        const bool store_issuer = warp == 18 && lane == 0;
        bool ok = true;      // as for the softmax warps: on a wait that gave up the loops run to their end
        AttnItem w;
        for (int n = 0; attn_item(d, n_kt, n_qp, n_slices, total, G, pr, n, &w); ++n) {
            ok = __all_sync(0xffffffffu, ptx::mbar_wait_backoff(o_item, n & 1, abort_flag, 100));
            ok = __all_sync(0xffffffffu, ptx::mbar_wait(epi_ready, n & 1, abort_flag));
            ptx::tc_fence_after_sync();
            const float* xs = xsum + ((n & 1) * 4 + quarter) * 128;
            const float inv_l = 1.f / ((xs[lane] + xs[32 + lane]) + (xs[64 + lane] + xs[96 + lane]));
            const int q0 = (2 * w.qp + (int)rank) * 128;
            const uint64_t inv2 = ptx::f32x2(inv_l, inv_l);
            uint8_t* stage = smem + ((n & 1) ? kAttnOutOff : 0u);    // the buffer that held this item's Q
            // Four passes of 64 columns = one box each, the two halves of the buffer used alternately:
            // a pass only waits for the store of the pass before last.  O is handed back as soon as
            // its last columns are in registers.
#pragma unroll 1
            for (int pass = 0; pass < SLICE / 64; ++pass) {
                uint8_t* box_row = stage + (pass & 1) * kAttnOutBoxBytes + row * 128;
                if (pass >= 2) {
                    if (store_issuer) ptx::bulk_wait_group_read_but_one();
                    epilogue_sync();
                }
#pragma unroll 1
                for (int ch = 0; ch < 2; ++ch) {     // 32 columns at a time: 16-byte chunks 4 ch .. 4 ch + 3 of the row
                    uint32_t r[32];
                    ptx::tmem_ld32(tmem_o + lane_base + pass * 64 + ch * 32, r);
                    ptx::tmem_wait_ld();
                    if (pass == SLICE / 64 - 1 && ch == 1) {      // O has been read completely: the next item's sums may start
                        ptx::tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive_cluster(o_free_leader);
                    }
                    // two-wide multiplies: these warps share their schedulers with the softmax warps,
                    // and every issue slot they need delays handing O back
                    uint32_t pk[16];
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        float v0, v1;
                        ptx::f32x2_split(ptx::mul2(ptx::f32x2(__uint_as_float(r[2 * e]), __uint_as_float(r[2 * e + 1])), inv2), v0, v1);
                        pk[e] = pack_bf16x2(v0, v1);
                    }
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const int chunk = (ch * 4 + c) ^ (row & 7);
                        *reinterpret_cast<uint4*>(box_row + chunk * 16) =
                            make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
                    }
                }
                ptx::fence_proxy_async_smem();
                epilogue_sync();
                if (store_issuer && q0 < d.N) {
                    ptx::tma_store_3d(&tm_o, stage + (pass & 1) * kAttnOutBoxBytes, w.slice * SLICE + pass * 64, q0,
                                      w.b * d.n_q + w.g);
                    ptx::bulk_commit_group();
                }
            }
            // the buffer may take the query tile of item n + 2 once the stores have read it
            if (store_issuer) {
                ptx::bulk_wait_group_read_all();
                ptx::mbar_arrive(stage_free);
            }
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
    // the decoder + gate kernel cuts the output columns in blocks of at least 128 inside one attention map
    const bool blocks_ok = d.n_q > 0 && ((d.n_h / d.n_q) * d.d_h) % 128 == 0;
    return dtype == GTA_BF16 && (d.d_h == 128 || d.d_h == 64) && d.d_l % 128 == 0 && d.d_l <= 1024 &&
           d.H % 64 == 0 && d.N >= 1 && blocks_ok;
}

// One instantiation of the attention kernel: its occupancy (asked once per device) and its launch.
template <int DH, int SLICE>
static gta_status_t launch_attention(const Dims& d, const CUtensorMap& tm_q, const CUtensorMap& tm_k,
                                     const CUtensorMap& tm_c, const CUtensorMap& tm_o, int32_t* status_word,
                                     cudaStream_t stream) {
    auto kern = sm100_attention_kernel<DH, SLICE>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAttnSmemTotal) != cudaSuccess)
        return GTA_ERR_CUDA;
    const int n_qt = (d.N + 127) / 128, n_qp = (n_qt + 1) / 2;
    const long long n_items = (long long)n_qp * (d.d_l / SLICE) * d.n_q * d.B;
    if (n_items > 0x3fffffffLL) return GTA_ERR_UNSUPPORTED;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kAttnThreads);
    cfg.dynamicSmemBytes = kAttnSmemTotal;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;   // the occupancy query below takes the cluster attribute only
    // a persistent grid must be resident at once: as many CTA pairs as the device can hold
    static thread_local int cached_dev = -1, cached_pairs = 0;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return GTA_ERR_CUDA;
    if (dev != cached_dev) {
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 2)
            return GTA_ERR_CUDA;
        cfg.gridDim = dim3(2 * (sms / 2));
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n < 1) return GTA_ERR_CUDA;
        cached_dev = dev;
        cached_pairs = n;
    }
    const int pairs = (int)(n_items < cached_pairs ? n_items : cached_pairs);
    cfg.gridDim = dim3(2 * pairs);
    cfg.numAttrs = 2;
    if (cudaLaunchKernelEx(&cfg, kern, tm_q, tm_k, tm_c, tm_o, d, status_word) != cudaSuccess) return GTA_ERR_CUDA;
    return cudaGetLastError() == cudaSuccess ? GTA_OK : GTA_ERR_CUDA;
}

gta_status_t launch_sm100_prefill(const Dims& d, const void* q, const void* k, const void* c, const void* x,
                                  const void* w_p, const void* w_g, void* out, void* workspace,
                                  int32_t* status_word, cudaStream_t stream, int stages, int* launches) {
    if (stages & 1) {
        CUtensorMap tm_q, tm_k, tm_c, tm_o;
        const uint32_t box[3] = {64, 128, 1}, box_k[3] = {64, 64, 1};
        const uint64_t dq[3] = {(uint64_t)d.d_h, (uint64_t)d.N, (uint64_t)d.B * d.n_q};
        // K / C: Nk of the S rows of a plane take part; the rest (the unused tail of a cache, which may hold
        // anything, NaN bit patterns included) lies outside the maps and reads as zeros
        const uint64_t dk[3] = {(uint64_t)d.d_h, (uint64_t)d.Nk, (uint64_t)d.B * d.n_k};
        const uint64_t dc[3] = {(uint64_t)d.d_l, (uint64_t)d.Nk, (uint64_t)d.B * d.n_c};
        const uint64_t ak[3] = {(uint64_t)d.d_h, (uint64_t)d.S, (uint64_t)d.B * d.n_k};
        const uint64_t ac[3] = {(uint64_t)d.d_l, (uint64_t)d.S, (uint64_t)d.B * d.n_c};
        if (!make_bf16_map(&tm_q, q, 3, dq, box) || !make_bf16_map(&tm_k, k, 3, dk, box_k, ak) ||
            !make_bf16_map(&tm_c, c, 3, dc, box, ac))
            return GTA_ERR_CUDA;
        {   // L [B n_q][N][d_l], stored in boxes of 128 rows x 64 columns
            const uint64_t dl[3] = {(uint64_t)d.d_l, (uint64_t)d.N, (uint64_t)d.B * d.n_q};
            const uint32_t box_o[3] = {64, 128, 1};
            if (!make_bf16_map(&tm_o, workspace, 3, dl, box_o)) return GTA_ERR_CUDA;
        }
        gta_status_t st;
        if (d.d_h == 128)
            st = d.d_l % 256 == 0 ? launch_attention<128, 256>(d, tm_q, tm_k, tm_c, tm_o, status_word, stream)
                                  : launch_attention<128, 128>(d, tm_q, tm_k, tm_c, tm_o, status_word, stream);
        else
            st = d.d_l % 256 == 0 ? launch_attention<64, 256>(d, tm_q, tm_k, tm_c, tm_o, status_word, stream)
                                  : launch_attention<64, 128>(d, tm_q, tm_k, tm_c, tm_o, status_word, stream);
        if (st != GTA_OK) return st;
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
