// tcgen05 / TMA (sm_100a) prefill path for bf16, d_h = 64 or 128.
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
// query tiles first, dealt to the pairs in snake order.
//
// The scores are produced and consumed in SUB-TILES of 64 keys (32 of each CTA's 64 keys of a ring
// tile), four of which are in flight, each in its own 64-column TMEM buffer with its own group of
// 128 softmax threads (a query row per thread).  Per sub-tile u (buffer and group u mod 4):
//   S_u = Q K_u^T            tcgen05.mma M = 256, N = 64, smem x smem -> TMEM
//   P_u = exp2(S_u c - m)    the group's threads; P_u (bf16) overwrites S_u in TMEM
//   O  += P_u C_u            tcgen05.mma M = 256, K = 64, TMEM x smem (C is the MN-major B operand)
// With four sub-tiles in flight the tensor pipe's own chain for a buffer (sum of sub-tile u, scores of
// sub-tile u + 4 into the buffer it frees, two barrier hand-offs) and the softmax of a sub-tile both
// hide behind the work on the other three; the four softmax warps of an SM sub-partition sit at
// different points of their sub-tiles, which keeps its issue slots and its exponential unit busy.
// The running maximum of a row is a chain over the sub-tiles: the thread of sub-tile u publishes it
// in shared memory as soon as it has the maximum of its own sub-tile (before its exponentials) and
// the thread of sub-tile u + 1 (the next group) picks it up there.  It is only raised when it grows
// by more than 2^8 (the accumulators stay in range and O needs rescaling on few sub-tiles).  At the
// end of an item the softmax threads only hand their (maximum, row sum) pairs over: four epilogue
// warps (one per TMEM lane quarter) combine the groups' sums, divide O by the row sum, round it to
// bf16 and write it to L[B, n_q, N, d_l] with 32-byte stores (a full sector of the thread's own row,
// nothing past the sequence end), while the softmax threads are already on the next item.  The
// ring and the score pipeline run on across items.  The lower query tile of a pair sees one fully
// masked key tile per item (its probabilities are zero).
constexpr int kAttnGroups = 4;                     // softmax groups = score buffers = sub-tiles in flight
constexpr int kSubKeys = 64;                       // keys per sub-tile (32 from each CTA of the pair)
constexpr int kAttnThreads = 128 * kAttnGroups + 128 + 96;   // warps 0-15 softmax, 16-19 epilogue, 20 TMA, 21 / 22 MMA issue (sums / scores)
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
constexpr uint32_t kAttnXchgOff = kAttnOutOff + 2 * kAttnOutBoxBytes;   // 2 KB: float [4 groups][128 rows] running maxima
constexpr uint32_t kAttnSumOff = kAttnXchgOff + kAttnGroups * 128 * 4;  // 8 KB: float2 [2 items][4 groups][128] (max, sum)
constexpr uint32_t kAttnBarOff = kAttnSumOff + 2 * kAttnGroups * 128 * 8;
constexpr uint32_t kAttnAlignSlack = 1024;  // checked in the kernel
constexpr uint32_t kAttnSmemTotal = kAttnBarOff + 512 + kAttnAlignSlack;
static_assert(kAttnSmemTotal <= 232448, "attention kernel shared memory exceeds the per-CTA limit");

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// The four warps of a softmax group (ids 1 .. 4) or the epilogue warps (id 6): one of them polls a
// barrier of the tensor pipe, the others sleep here at no cost in issue slots until it has seen it.
__device__ __forceinline__ void wait_group_sync(int id) {
    asm volatile("bar.sync %0, 128;" ::"r"(id) : "memory");
}
// Scores of keys past `last_key` (past the sequence end, or -- causal -- after the query) become -inf.
// Only called on boundary tiles (a warp-level branch around it costs the other tiles nothing).
__device__ __forceinline__ void mask_chunk(uint32_t (&r)[32], int key0, int last_key) {
#pragma unroll
    for (int e = 0; e < 32; ++e)
        if (key0 + e > last_key) r[e] = 0xff800000u;     // -inf
}
// exp2(s c - m) of 32 scores of one row (raw TMEM words), packed to bf16 pairs; their sum is added to sum2
__device__ __forceinline__ void softmax_chunk(const uint32_t (&r)[32], uint64_t cs2, uint64_t nm2, uint64_t (&sum2)[2],
                                              uint32_t (&packed)[16]) {
#pragma unroll
    for (int e = 0; e < 16; ++e) {
        const uint64_t x2 = ptx::fma2(ptx::f32x2(__uint_as_float(r[2 * e]), __uint_as_float(r[2 * e + 1])), cs2, nm2);
        // (a polynomial on the FMA pipe for part of the pairs, to spare the exponential unit, was measured
        // slower here: the unit is under half busy, the issue slots are what is short)
        float x0, x1;
        ptx::f32x2_split(x2, x0, x1);
        const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
        sum2[e & 1] = ptx::add2(sum2[e & 1], ptx::f32x2(p0, p1));
        packed[e] = pack_bf16x2(p0, p1);
    }
}
// maximum of 32 scores of one row (raw TMEM words) and mx
__device__ __forceinline__ float max_chunk(const uint32_t (&r)[32], float mx) {
    float a = mx, b = -INFINITY;
#pragma unroll
    for (int e = 0; e < 32; e += 4) {
        a = ptx::max3(a, __uint_as_float(r[e]), __uint_as_float(r[e + 1]));
        b = ptx::max3(b, __uint_as_float(r[e + 2]), __uint_as_float(r[e + 3]));
    }
    return fmaxf(a, b);
}
// Test hooks of the bounded waits (gta_debug_attention_wait): the time limit of every wait of the attention
// kernel, and a switch that makes one softmax warp keep its very first arrival to itself, so that the
// thread that issues the sums runs into that limit and the whole unwinding path can be exercised on a
// healthy GPU.  Both live in device memory of the library and are read once per thread at kernel start.
static __device__ unsigned long long g_attn_wait_limit_ns = ptx::kWaitLimitNs;
static __device__ int g_attn_withhold_first_arrive = 0;

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
                       const __grid_constant__ CUtensorMap tm_c, __nv_bfloat16* __restrict__ l_out, Dims d,
                       const PageMap pm, int32_t* status_word) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    float* xchg = reinterpret_cast<float*>(smem + kAttnXchgOff);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kAttnBarOff);
    uint64_t* q_full = bars;            // [2] (slots 0 and 41) leader CTA; both producers arrive; item n uses barrier n & 1
    uint64_t* stage_free = bars + 1;    // this CTA; its epilogue's stores have read the buffer (one thread arrives)
    uint64_t* full = bars + 2;          // [4] leader CTA; both producers arrive
    uint64_t* empty = bars + 6;         // [4] both CTAs (multicast commit)
    uint64_t* s_full = bars + 10;       // [4] both CTAs (multicast commit): scores of a sub-tile are in its buffer
    uint64_t* p_full = bars + 14;       // [4] leader CTA; the 4 warps of a softmax group of both CTAs arrive
    uint64_t* o_done = bars + 18;       // [4] both CTAs (multicast commit): the sum of a sub-tile is complete
    uint64_t* o_free = bars + 22;       // leader CTA; 8 epilogue warps arrive
    // this CTA; its 16 softmax warps arrive (maxima and row sums of an item are in place).  One barrier for the even
    // items (slot 23) and one for the odd ones (slot 47): a group that is done with item n early goes on to a short
    // item n + 1 and may arrive for it before the last group has arrived for item n; on a single barrier that arrival
    // would complete item n's phase with that group's pair still missing.
    uint64_t* epi_ready = bars + 23;
    uint64_t* o_item = bars + 24;       // both CTAs (multicast commit): the last sum of an item is complete
    uint64_t* chain = bars + 25;        // [4 groups][4 quarters] this CTA; one warp arrives: its rows' running maxima are published
    uint64_t* mma_drain = bars + 42;    // [2] leader CTA: used once by an MMA-issuing thread that unwinds (all its MMAs are done)
    uint64_t* tail_bar = bars + 46;     // this CTA, paged pools only: the latent block whose last rows the producer clears
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 44);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile int* drain_flag = abort_flag + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();          // 0 = leader
    const uint64_t wait_limit = g_attn_wait_limit_ns;
    const bool withhold_first_arrive = g_attn_withhold_first_arrive != 0;
    // every wait of this kernel: bounded by wait_limit, ended early by the CTA's abort flag
    auto wait = [&](uint64_t* bar, uint32_t parity, uint32_t sleep_ns = 0) {
        return ptx::mbar_wait_sleep(bar, parity, abort_flag, sleep_ns, wait_limit);
    };
    const int G = gridDim.x >> 1, pr = blockIdx.x >> 1;    // CTA pairs, this pair
    const bool bad_align = (uint32_t)(smem - smem_raw) > kAttnAlignSlack;   // cannot happen with a 256-byte aligned window
    constexpr uint32_t kQLoadBytes = 128 * DH * 2;                 // this CTA's query tile
    constexpr uint32_t kKLoadBytes = (kKeyTile / 2) * DH * 2;      // this CTA's 64 keys
    constexpr uint32_t kCLoadBytes = kKeyTile * (SLICE / 2) * 2;   // this CTA's SLICE / 2 latent columns
    // A latent of only SLICE / 2 columns (the comparison operators with d_h = 64 values): both CTAs of the
    // pair stage the same columns, so the second half of O repeats the first and is not stored.
    const bool narrow = d.d_l * 2 == SLICE;
    const bool paged = pm.table != nullptr;
    const int n_slices = narrow ? 1 : d.d_l / SLICE;
    const int n_qt = (d.N + 127) / 128, n_qp = (n_qt + 1) / 2;
    const int n_kt = (d.Nk + 127) / 128;          // key tiles
    const long long total = bad_align ? 0 : (long long)n_qp * n_slices * d.n_q * d.B;

    if (threadIdx.x == 0) {
        ptx::mbar_init(&q_full[0], 2);
        ptx::mbar_init(&q_full[41], 2);
        ptx::mbar_init(&mma_drain[0], 1);
        ptx::mbar_init(&mma_drain[1], 1);
        ptx::mbar_init(stage_free, 1);
        ptx::mbar_init(tail_bar, 1);
        for (int s = 0; s < kAttnStages; ++s) { ptx::mbar_init(&full[s], 2); ptx::mbar_init(&empty[s], 1); }
        for (int s = 0; s < kAttnGroups; ++s) {
            ptx::mbar_init(&s_full[s], 1); ptx::mbar_init(&p_full[s], 8); ptx::mbar_init(&o_done[s], 1);
        }
        ptx::mbar_init(o_free, 8);
        ptx::mbar_init(&epi_ready[0], 4 * kAttnGroups);
        ptx::mbar_init(&epi_ready[24], 4 * kAttnGroups);
        ptx::mbar_init(o_item, 1);
        for (int s = 0; s < 4 * kAttnGroups; ++s) ptx::mbar_init(&chain[s], 1);
        *abort_flag = 0;
        *drain_flag = 0;
        ptx::fence_mbar_init();
    }
    if (warp == 21) ptx::tmem_alloc_pair(tmem_slot, 512);
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

    if (warp == 20) {
        if (ptx::elect_one()) {
            ptx::prefetch_tensormap(&tm_q); ptx::prefetch_tensormap(&tm_k); ptx::prefetch_tensormap(&tm_c);
            int tj = 0;                 // key tiles issued so far (ring position), across items
            int n_armed = 0;            // query tiles whose load has been issued
            int tail_armed = 0;         // loads through tail_bar
            const uint32_t tail_bar_addr = ptx::map_to_cta(ptx::smem_addr(tail_bar), rank);
            // Block-table entries of the two 64-token halves of key tile j of sequence b (kPastKeys for a half past the
            // attended keys, whose entry may not exist).  They are fetched one tile ahead, before the wait for the ring
            // stage: a table look-up behind that wait would add its latency to every tile.
            constexpr int kPastKeys = -0x40000000;
            auto page_entries = [&](int b, int j, int& e0, int& e1) {
                const int t0 = j * kKeyTile;
                const int32_t* row = pm.table + (size_t)b * pm.max_pages;
                e0 = t0 < d.Nk ? row[t0 / pm.page_size] : kPastKeys;
                e1 = t0 + 64 < d.Nk ? row[(t0 + 64) / pm.page_size] : kPastKeys;
            };
            // (row, plane) coordinates of the 64 cached tokens from `token` on, given their block-table entry
            auto page_block = [&](int entry, int token, int groups, int grp, int& row, int& plane) {
                row = pm.page_size;     // past the page: the box reads as zeros
                plane = 0;
                if (entry == kPastKeys) return;
                if (entry < 0 || entry >= pm.n_pages) { raise_status(status_word, GTA_ERR_BAD_PAGE); return; }
                row = token % pm.page_size;
                plane = entry * groups + grp;
            };
            bool ok = true;
            AttnItem w;
            for (int n = 0; ok && attn_item(d, n_kt, n_qp, n_slices, total, G, pr, n, &w); ++n) {
                const uint32_t q_full_leader = ptx::map_to_cta(ptx::smem_addr(&q_full[(n & 1) * 41]), 0);
                const int kg = d.q_to_k(w.g), cg = d.q_to_c(w.g);
                const int q0 = (2 * w.qp + (int)rank) * 128;       // this CTA's query rows
                // buffer n & 1 is free once the epilogue of item n - 2 has stored out of it (which
                // also means every Q K^T of that item is done); every completion is waited for, in order
                if (n >= 2) ok = wait(stage_free, n & 1);
                if (!ok) break;
                uint8_t* q_s = smem + ((n & 1) ? kAttnOutOff : 0u);
                ptx::mbar_arrive_expect_tx_cluster(q_full_leader, kQLoadBytes);
                ++n_armed;
                ptx::tma_load_3d_pair(q_s, &tm_q, q_full_leader, 0, q0, w.b * d.n_q + w.g);
                if (DH == 128) ptx::tma_load_3d_pair(q_s + 16384, &tm_q, q_full_leader, 64, q0, w.b * d.n_q + w.g);
                int e_cur[2] = {kPastKeys, kPastKeys}, e_next[2] = {kPastKeys, kPastKeys};
                if (paged) page_entries(w.b, 0, e_next[0], e_next[1]);
                for (int j = 0; j < w.n_tiles; ++j, ++tj) {
                    const int s = tj % kAttnStages;
                    const uint32_t ph = (tj / kAttnStages) & 1;
                    e_cur[0] = e_next[0]; e_cur[1] = e_next[1];
                    if (paged && j + 1 < w.n_tiles) page_entries(w.b, j + 1, e_next[0], e_next[1]);
                    ok = wait(&empty[s], ph ^ 1, 64);   // the ring is three tiles ahead
                    if (!ok) break;
                    uint8_t* k_s = smem + kAttnRingOff + s * kAttnStageBytes;
                    uint8_t* c_s = k_s + kKHalfBytes;
                    const uint32_t bar = ptx::map_to_cta(ptx::smem_addr(&full[s]), 0);
                    const int key0 = j * kKeyTile + (int)rank * 64;         // this CTA's 64 keys of the tile
                    const int col0 = narrow ? 0 : w.slice * SLICE + (int)rank * (SLICE / 2);     // this CTA's latent columns
                    if (!paged) {
                        ptx::mbar_arrive_expect_tx_cluster(bar, kKLoadBytes + kCLoadBytes);
                        ptx::tma_load_3d_pair(k_s, &tm_k, bar, 0, key0, w.b * d.n_k + kg);
                        if (DH == 128) ptx::tma_load_3d_pair(k_s + 8192, &tm_k, bar, 64, key0, w.b * d.n_k + kg);
                        ptx::tma_load_3d_pair(c_s, &tm_c, bar, col0, j * kKeyTile, w.b * d.n_c + cg);
                        if (SLICE == 256)
                            ptx::tma_load_3d_pair(c_s + 16384, &tm_c, bar, col0 + 64, j * kKeyTile, w.b * d.n_c + cg);
                        continue;
                    }
                    // Paged pools: the maps are [pages x groups][page_size][width] and every load is a block of 64
                    // tokens, which lies inside one page (page_size is a multiple of 64).  A block past the attended
                    // keys, or one whose page number is outside the pool, is loaded from a row coordinate past the
                    // page, i.e. as zeros.
                    int k_row, k_plane, c_row[2], c_plane[2];
                    page_block(rank ? e_cur[1] : e_cur[0], key0, d.n_k, kg, k_row, k_plane);
                    page_block(e_cur[0], j * kKeyTile, d.n_c, cg, c_row[0], c_plane[0]);
                    page_block(e_cur[1], j * kKeyTile + 64, d.n_c, cg, c_row[1], c_plane[1]);
                    // The block that holds position Nk: its rows from Nk on exist in the page and may hold anything.
                    // As keys they are masked, but as latent rows they would meet their zero probabilities in the
                    // sum (0 x NaN), so this block goes through a barrier of this CTA, the thread clears those rows
                    // in shared memory, and only then arrives at the tile's barrier.
                    const int tail_h = (d.Nk & 63) ? (d.Nk - j * kKeyTile) >> 6 : -1;     // 0 or 1: the tile's half with that block
                    const bool tail = (tail_h == 0 || tail_h == 1) && c_row[tail_h & 1] < pm.page_size;
                    if (tail) {
                        ptx::mbar_expect_tx_cluster(bar, kKLoadBytes + kCLoadBytes / 2);
                        ptx::mbar_arrive_expect_tx(tail_bar, kCLoadBytes / 2);
                        ++tail_armed;
                    } else {
                        ptx::mbar_arrive_expect_tx_cluster(bar, kKLoadBytes + kCLoadBytes);
                    }
                    ptx::tma_load_3d_pair(k_s, &tm_k, bar, 0, k_row, k_plane);
                    if (DH == 128) ptx::tma_load_3d_pair(k_s + 8192, &tm_k, bar, 64, k_row, k_plane);
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const uint32_t hb = (tail && h == tail_h) ? tail_bar_addr : bar;
                        ptx::tma_load_3d_pair(c_s + h * 8192, &tm_c, hb, col0, c_row[h], c_plane[h]);
                        if (SLICE == 256)
                            ptx::tma_load_3d_pair(c_s + 16384 + h * 8192, &tm_c, hb, col0 + 64, c_row[h], c_plane[h]);
                    }
                    if (tail) {
                        ok = wait(tail_bar, (tail_armed - 1) & 1);
                        if (!ok) break;
                        const int live = d.Nk & 63;                       // rows of the block that are keys
                        const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
                        for (int grp = 0; grp < SLICE / 128; ++grp) {     // 64-column groups of this CTA: 128 bytes a row
                            uint4* z = reinterpret_cast<uint4*>(c_s + grp * 16384 + tail_h * 8192 + live * 128);
                            for (int i = 0; i < (64 - live) * 8; ++i) z[i] = zero;
                        }
                        ptx::fence_proxy_async_smem();                    // the MMAs read these rows through the async proxy
                        ptx::mbar_arrive_release_cluster(bar);
                    }
                }
            }
            if (*abort_flag && tail_armed > 0) ptx::mbar_wait_drain(tail_bar, (tail_armed - 1) & 1, drain_flag);
            if (*abort_flag && rank == 0) {
                // Unwinding: wait (bounded) for the copies that were armed, so that none lands after the CTA has
                // left.  At most the last two query tiles and the last three ring tiles can be outstanding (the
                // loads before them were consumed before their buffers were armed again), each on a barrier whose
                // earlier phases are complete, so a parity wait for its latest phase is unambiguous.
                for (int back = 1; back <= 2 && n_armed - back >= 0; ++back) {
                    const int m = n_armed - back;
                    ptx::mbar_wait_drain(&q_full[(m & 1) * 41], (m >> 1) & 1, drain_flag);
                }
                for (int back = 1; back <= kAttnStages && tj - back >= 0; ++back) {
                    const int jq = tj - back;
                    ptx::mbar_wait_drain(&full[jq % kAttnStages], (jq / kAttnStages) & 1, drain_flag);
                }
            }
        }
    } else if (warp == 21 || warp == 22) {
        // Two threads of the leader CTA feed the tensor pipe: one issues the score MMAs (S_u = Q K_u^T), the
        // other the sums (O += P_u C_u).  A single thread's instruction stream -- waits, descriptors, MMAs,
        // commits, one instruction every few cycles -- is what paced the pipe when one thread did both.
        // The two are ordered through barriers only: the scores of sub-tile u + 4 go into the buffer of
        // sub-tile u once its sum is COMPLETE (o_done), the sum of sub-tile u follows its probabilities
        // (p_full), which follow its scores (s_full).
        if (rank == 0 && ptx::elect_one()) {
            constexpr uint32_t idesc_qk = ptx::make_idesc_bf16(256, kSubKeys, 0, 0);   // both K-major
            constexpr uint32_t idesc_pv = ptx::make_idesc_bf16(256, SLICE, 0, 1);      // B = C, MN-major
            const uint32_t smem_base = ptx::smem_addr(smem);
            // descriptors differ in the start address only: base + (address >> 4)
            const uint64_t desc_kmajor = ptx::make_smem_desc(0, 16, 1024);
            const uint64_t desc_latent = ptx::make_smem_desc(0, 16384, 1024);
            bool ok = true;
            int u = 0;                  // sub-tiles so far over all items: buffer and group u & 3, ring tile u >> 1
            AttnItem w;
            for (int n = 0; ok && attn_item(d, n_kt, n_qp, n_slices, total, G, pr, n, &w); ++n) {
                const int n_sub = 2 * w.n_tiles;
                if (warp == 22) {
                    // ---- scores
                    const uint32_t q_lo = (smem_base + ((n & 1) ? kAttnOutOff : 0u)) >> 4;
                    for (int j = 0; j < n_sub && ok; ++j, ++u) {
                        const int tile = u >> 1, stage = tile % kAttnStages;
                        if (u >= kAttnGroups) ok = wait(&o_done[u & 3], ((u - kAttnGroups) >> 2) & 1);
                        if (ok && j == 0) ok = wait(&q_full[(n & 1) * 41], (n >> 1) & 1);
                        if (ok && (j & 1) == 0) ok = wait(&full[stage], (tile / kAttnStages) & 1);
                        if (!ok) break;
                        // the one tile of which the producers cleared rows (the block that holds position Nk): the
                        // peer's stores are ordered before its arrival by a release, taken here by an acquire fence
                        if (paged && (d.Nk & 63) != 0 && (j >> 1) == (d.Nk >> 7)) ptx::fence_acq_rel_cluster();
                        ptx::tc_fence_after_sync();
                        // this CTA's keys 32 (j & 1) .. of its 64 keys of the ring tile: 32 rows of 128 bytes further
                        // on; 32 bytes per k-step inside a 64-column half, the next half 16 KB (Q) / 8 KB (K) on
                        uint64_t dq = desc_kmajor + q_lo;
                        uint64_t dk = desc_kmajor + ((smem_base + kAttnRingOff + stage * kAttnStageBytes + (j & 1) * 4096) >> 4);
                        const uint32_t s_tmem = tmem_base + (u & 3) * kSubKeys;
#pragma unroll
                        for (int k8 = 0; k8 < DH / 16; ++k8) {
                            ptx::mma_ss_pair(s_tmem, dq, dk, idesc_qk, (uint32_t)k8);
                            const bool wrap = (k8 & 3) == 3;
                            dq += wrap ? (16384 - 96) >> 4 : 2;
                            dk += wrap ? (8192 - 96) >> 4 : 2;
                        }
                        ptx::tc_commit_pair(&s_full[u & 3], 3);
                    }
                } else {
                    // ---- sums
                    for (int j = 0; j < n_sub && ok; ++j, ++u) {
                        const int tile = u >> 1, stage = tile % kAttnStages, sub = j & 1;
                        ok = wait(&p_full[u & 3], (u >> 2) & 1);
                        if (ok && j == 0 && n > 0) ok = wait(o_free, (n - 1) & 1);
                        if (!ok) break;
                        ptx::tc_fence_after_sync();
                        // P columns 16 kk .. are the keys 32 sub + 16 (kk & 1) .. of CTA kk >> 1, i.e. rows
                        // 64 (kk >> 1) + 32 sub + 16 (kk & 1) .. of the 128-key latent tile (2 KB per 16 rows)
                        uint64_t dc = desc_latent + ((smem_base + kAttnRingOff + stage * kAttnStageBytes + kKHalfBytes + sub * 4096) >> 4);
                        uint32_t p_tmem = tmem_base + (u & 3) * kSubKeys;
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk) {
                            ptx::mma_ts_pair(tmem_o, p_tmem, dc, idesc_pv, (j > 0 || kk > 0) ? 1u : 0u);
                            p_tmem += 8;
                            dc += (kk == 1) ? (3 * 2048) >> 4 : 2048 >> 4;
                        }
                        ptx::tc_commit_pair(&o_done[u & 3], 3);
                        if (j + 1 == n_sub) ptx::tc_commit_pair(o_item, 3);   // for the epilogue warps
                        // both halves of the ring tile are used up (its scores were complete before these sums began)
                        if (sub == 1) ptx::tc_commit_pair(&empty[stage], 3);
                    }
                }
            }
            if (*abort_flag) {
                // Unwinding: the MMAs this thread has issued must be complete before tensor memory is freed.
                // A commit on a barrier that is used for nothing else completes when they all are.
                uint64_t* bar = &mma_drain[warp - 21];
                ptx::tc_commit_pair(bar, 1);
                ptx::mbar_wait_drain(bar, 0, drain_flag);
            }
        }
    } else if (warp < 4 * kAttnGroups) {
        // Four softmax groups of four warps (one per TMEM lane quarter), a query row per thread.  Group g
        // takes the sub-tiles u with u mod 4 = g (score buffer g).  Per sub-tile: (1) the row maximum of the
        // 64 scores; (2) the chain: take the running maximum that the previous group's thread of this row
        // published for the sub-tile before, raise it if this sub-tile exceeds it by more than 2^8, publish
        // it; (3) the exponentials, 32 keys at a time, P written over S; (4) rarely, O rescaled.  Step (2)
        // is all that orders the groups.
        const int wg = warp >> 2;
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const uint32_t lane_base = ((uint32_t)(quarter * 32) << 16);
        const float c_scale = d.scale * 1.4426950408889634f;
        const uint32_t p_full_leader = ptx::map_to_cta(ptx::smem_addr(&p_full[wg]), 0);
        const uint32_t s_tmem = tmem_base + lane_base + wg * kSubKeys;
        const int wg_prev = (wg + kAttnGroups - 1) & (kAttnGroups - 1);
        float* m_pub = xchg + wg * 128 + row;                 // written by this thread, read by the next group's
        const volatile float* m_in = xchg + wg_prev * 128 + row;
        uint64_t* chain_out = &chain[wg * 4 + quarter];
        uint64_t* chain_in = &chain[wg_prev * 4 + quarter];
        float2* xsum = reinterpret_cast<float2*>(smem + kAttnSumOff);
        const uint64_t cs2 = ptx::f32x2(c_scale, c_scale);
        // A wait that gives up raises the CTA's abort flag, after which every wait returns at once:
        // these warps then run their loops to the end all the same (on meaningless data).
        bool ok = true;
        int u = 0;                                  // sub-tiles so far, over all items
        AttnItem w, nxt;
        bool have = attn_item(d, n_kt, n_qp, n_slices, total, G, pr, 0, &w);
        for (int n = 0; have; ++n) {
            const bool have_next = attn_item(d, n_kt, n_qp, n_slices, total, G, pr, n + 1, &nxt);
            const int t = (2 * w.qp + (int)rank) * 128 + row;
            const int last_key = d.causal ? min(t + d.Nk - d.N, d.Nk - 1) : d.Nk - 1;
            const int n_sub = 2 * w.n_tiles;
            float m_own = -INFINITY, l = 0.f;       // m in scaled (log2) units; l: this group's share of the row sum, relative to m_own
            for (int j = 0; j < n_sub; ++j, ++u) {
                if ((u & (kAttnGroups - 1)) != wg) continue;
                // one warp of the group polls for the scores (on a scheduler of its own: group g's poller is its
                // warp of lane quarter g), the other three are woken through a named barrier
                if (quarter == wg) ok = __all_sync(0xffffffffu, wait(&s_full[wg], (u >> 2) & 1));
                wait_group_sync(1 + wg);
                ptx::tc_fence_after_sync();
                // columns 0 .. 31 of the buffer: keys key_a .. of the ring tile's first half (the leader CTA's),
                // columns 32 .. 63: keys key_b .. of its second half
                const int key_a = (j >> 1) * kKeyTile + (j & 1) * 32, key_b = key_a + 64;
                const bool boundary = key_b + 31 > last_key;
                uint32_t ra[32];
                // ---- (1) row maximum (the two 32-key halves in a rolled loop, like the exponentials below: the
                //      warps of a scheduler share a small instruction cache with the thread that issues the MMAs)
                float mx = -INFINITY;
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    ptx::tmem_ld32(s_tmem + c * 32, ra);
                    ptx::tmem_wait_ld();
                    if (boundary) mask_chunk(ra, c ? key_b : key_a, last_key);
                    mx = max_chunk(ra, mx);
                }
                ptx::tmem_ld32(s_tmem, ra);            // the first 32 scores again for step (3), under the chain
                const float m_tile = mx * c_scale;     // c_scale > 0
                // ---- (2) the chain of running maxima (every sub-tile but the very first waits for the one
                //      before it, every sub-tile but the very last signals the one after it: strict rotation)
                if (u > 0) ok = __all_sync(0xffffffffu, wait(chain_in, ((u - 1) >> 2) & 1));
                const float m_prev = (j == 0) ? -INFINITY : *m_in;
                const bool raise = m_tile > m_prev + 8.f;     // also true on the first live sub-tile (m_prev = -inf)
                const float m = raise ? m_tile : m_prev;
                *m_pub = m;
                __syncwarp();
                if (lane == 0 && (have_next || j + 1 < n_sub)) ptx::mbar_arrive(chain_out);
                if (m != m_own) {                     // this group's sum follows the maximum (other groups may have raised it)
                    l *= fast_exp2(m_own - m);        // m_own = -inf: l is 0 and stays 0
                    m_own = m;
                }
                // ---- (3) exponentials, 32 keys at a time (the scores are read from TMEM a second time: keeping
                //      all 64 in registers across the chain costs more in spills than the second load)
                const float neg_m = (m == -INFINITY) ? 0.f : -m;   // a fully masked row keeps p = 0
                const uint64_t nm2 = ptx::f32x2(neg_m, neg_m);
                uint64_t sum2[2] = {0ull, 0ull};         // two-wide fp32 arithmetic: half the issue slots
                uint32_t packed[16];
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    ptx::tmem_wait_ld();
                    if (boundary) mask_chunk(ra, c ? key_b : key_a, last_key);
                    softmax_chunk(ra, cs2, nm2, sum2, packed);
                    if (c == 0) ptx::tmem_ld32(s_tmem + 32, ra);
                    // P_u (bf16 pairs): 32 keys = 16 packed columns of the buffer, columns whose scores this thread
                    // has already loaded
                    ptx::tmem_st16(s_tmem + c * 16, packed);
                }
                float s0, s1;
                ptx::f32x2_split(ptx::add2(sum2[0], sum2[1]), s0, s1);
                l += s0 + s1;
                // ---- (4) O holds the sums of the sub-tiles before this one relative to m_prev: rescale it when
                //      the maximum was raised.  The sum of sub-tile u - 1 must be complete first; its barrier
                //      (one per buffer) completes once per four sub-tiles, and when the scores of sub-tile u exist
                //      the sum of sub-tile u - 4 is complete, so the phase waited for is the current or the last one.
                if (j > 0 && __any_sync(0xffffffffu, raise)) {
                    ok = __all_sync(0xffffffffu, wait(&o_done[(u - 1) & 3], ((u - 1) >> 2) & 1));
                    ptx::tc_fence_after_sync();
                    const float alpha = raise ? fast_exp2(m_prev - m) : 1.f;
                    const uint64_t a2 = ptx::f32x2(alpha, alpha);
#pragma unroll 1
                    for (int ch = 0; ch < SLICE / 32; ++ch) {
                        ptx::tmem_ld32(tmem_o + lane_base + ch * 32, ra);
                        ptx::tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; e += 2) {
                            float v0, v1;
                            ptx::f32x2_split(ptx::mul2(ptx::f32x2(__uint_as_float(ra[e]), __uint_as_float(ra[e + 1])), a2), v0, v1);
                            ra[e] = __float_as_uint(v0);
                            ra[e + 1] = __float_as_uint(v1);
                        }
                        ptx::tmem_st32(tmem_o + lane_base + ch * 32, ra);
                    }
                }
                ptx::tmem_wait_st();
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0 && !(withhold_first_arrive && u == 0 && quarter == 0 && rank == 0))
                    ptx::mbar_arrive_cluster(p_full_leader);
            }
            // ---- end of the item: (maximum, row sum) of this group go to the epilogue warps
            //      (double-buffered by item: the epilogue of item n reads them before it hands O
            //      back, which the sums of item n + 1 wait for, long before item n + 2 ends)
            xsum[((n & 1) * kAttnGroups + wg) * 128 + row] = make_float2(m_own, l);
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&epi_ready[(n & 1) * 24]);
            w = nxt;
            have = have_next;
        }
    } else if (warp < 4 * kAttnGroups + 4) {
        // 4 epilogue warps, one per TMEM lane quarter, a row per thread.  When the softmax groups have left their
        // (maximum, row sum) pairs (epi_ready) the row's normaliser is worked out; after the last sum of the item
        // (o_item: one completion per item, and the next cannot come before this item's O has been handed back) O is
        // read 16 columns at a time, the next 16 already on their way while the current ones are scaled, rounded to
        // bf16 and written straight to L with one 32-byte store per thread (a full sector of the thread's own row):
        // nothing between the read and the hand-back waits for a staging buffer or a store, so O is back with the
        // MMA threads after one pass over its columns.  (An earlier form staged 64-column boxes in shared memory
        // for TMA stores and held O for 2.7 us per item; handing it back sooner did not change the kernel's time,
        // which is set by the steady rate of the score-buffer loop, but this form needs no staging buffer.)
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const uint32_t lane_base = ((uint32_t)(quarter * 32) << 16);
        const uint32_t o_free_leader = ptx::map_to_cta(ptx::smem_addr(o_free), 0);
        const float2* xsum = reinterpret_cast<const float2*>(smem + kAttnSumOff);
        const bool poller = quarter == 2;    // one warp polls, the others are woken by it through a named barrier
        bool ok = true;      // as for the softmax warps: on a wait that gave up the loops run to their end
        AttnItem w;
        for (int n = 0; attn_item(d, n_kt, n_qp, n_slices, total, G, pr, n, &w); ++n) {
            if (poller) ok = __all_sync(0xffffffffu, wait(&epi_ready[(n & 1) * 24], (n >> 1) & 1, 200));
            wait_group_sync(6);
            // the groups' sums, each relative to the maximum its group saw last; O is relative to the largest
            float2 gs[kAttnGroups];
            float m_fin = -INFINITY;
#pragma unroll
            for (int g = 0; g < kAttnGroups; ++g) {
                gs[g] = xsum[((n & 1) * kAttnGroups + g) * 128 + row];
                m_fin = fmaxf(m_fin, gs[g].x);
            }
            float l_fin = 0.f;
#pragma unroll
            for (int g = 0; g < kAttnGroups; ++g)
                l_fin += gs[g].x == -INFINITY ? 0.f : gs[g].y * fast_exp2(gs[g].x - m_fin);
            const float inv_l = 1.f / l_fin;
            const uint64_t inv2 = ptx::f32x2(inv_l, inv_l);
            const int t = (2 * w.qp + (int)rank) * 128 + row;             // this thread's query row
            const int col0 = w.slice * SLICE;
            // narrow latent: the second half of the slice repeats the first and is not stored
            const int n_cols = narrow ? SLICE / 2 : SLICE;
            __nv_bfloat16* dst = l_out + ((size_t)(w.b * d.n_q + w.g) * d.N + (t < d.N ? t : 0)) * d.d_l + col0;
            const bool live = t < d.N;
            if (poller) ok = __all_sync(0xffffffffu, wait(o_item, n & 1, 64));
            wait_group_sync(6);
            ptx::tc_fence_after_sync();
            // every score MMA of the item is complete too: its query tile's buffer may take the tile of item n + 2
            if (warp == 4 * kAttnGroups && lane == 0) ptx::mbar_arrive(stage_free);
            uint32_t ra[16], rb[16];
            auto write_out = [&](const uint32_t (&r)[16], int c) {      // columns 16 c .. 16 c + 15 of the slice
                uint32_t pk[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    float v0, v1;
                    ptx::f32x2_split(ptx::mul2(ptx::f32x2(__uint_as_float(r[2 * e]), __uint_as_float(r[2 * e + 1])), inv2), v0, v1);
                    pk[e] = pack_bf16x2(v0, v1);
                }
                if (live && c * 16 < n_cols) ptx::st_global_256(dst + c * 16, pk);
            };
            constexpr int kChunks = SLICE / 16;
            ptx::tmem_ld16(tmem_o + lane_base, ra);
#pragma unroll 1
            for (int c = 0; c < kChunks; c += 2) {
                ptx::tmem_wait_ld();
                ptx::tmem_ld16(tmem_o + lane_base + (c + 1) * 16, rb);
                write_out(ra, c);
                ptx::tmem_wait_ld();
                if (c + 2 < kChunks) {
                    ptx::tmem_ld16(tmem_o + lane_base + (c + 2) * 16, ra);
                } else {                  // O has been read completely: the next item's sums may start
                    ptx::tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive_cluster(o_free_leader);
                }
                write_out(rb, c + 1);
            }
        }
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_arrive();     // neither CTA leaves (or frees TMEM) while the other may still signal it
    ptx::cluster_wait();
    if (warp == 21) ptx::tmem_dealloc_pair(tmem_base, 512);
    if (threadIdx.x == 0 && *abort_flag) raise_status(status_word, GTA_ERR_TIMEOUT);
}

// --------------------------------------------------------------------------- host side
gta_status_t sm100_attention_debug_wait(unsigned long long limit_ns, int withhold_first_arrive) {
    const unsigned long long lim = limit_ns ? limit_ns : ptx::kWaitLimitNs;
    const int sw = withhold_first_arrive ? 1 : 0;
    if (cudaMemcpyToSymbol(g_attn_wait_limit_ns, &lim, sizeof(lim)) != cudaSuccess ||
        cudaMemcpyToSymbol(g_attn_withhold_first_arrive, &sw, sizeof(sw)) != cudaSuccess) {
        cudaGetLastError();
        return GTA_ERR_CUDA;
    }
    return GTA_OK;
}

bool sm100_prefill_supported(const Dims& d, int dtype) {
    // the decoder + gate kernel cuts the output columns in blocks of at least 128 inside one attention map
    const bool blocks_ok = d.n_q > 0 && ((d.n_h / d.n_q) * d.d_h) % 128 == 0;
    return dtype == GTA_BF16 && (d.d_h == 128 || d.d_h == 64) && d.d_l % 128 == 0 && d.d_l <= 1024 &&
           d.H % 64 == 0 && d.N >= 1 && blocks_ok;
}

// One instantiation of the attention kernel: its occupancy (asked once per device) and its launch.
template <int DH, int SLICE>
static gta_status_t launch_attention(const Dims& d, const PageMap& pm, const CUtensorMap& tm_q, const CUtensorMap& tm_k,
                                     const CUtensorMap& tm_c, __nv_bfloat16* l_out, int32_t* status_word,
                                     cudaStream_t stream) {
    auto kern = sm100_attention_kernel<DH, SLICE>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAttnSmemTotal) != cudaSuccess)
        return GTA_ERR_CUDA;
    const int n_qt = (d.N + 127) / 128, n_qp = (n_qt + 1) / 2;
    const long long n_items = (long long)n_qp * (d.d_l * 2 == SLICE ? 1 : d.d_l / SLICE) * d.n_q * d.B;
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
    if (cudaLaunchKernelEx(&cfg, kern, tm_q, tm_k, tm_c, l_out, d, pm, status_word) != cudaSuccess) return GTA_ERR_CUDA;
    return cudaGetLastError() == cudaSuccess ? GTA_OK : GTA_ERR_CUDA;
}

// L[B, n_q, N, d_l] (bf16) = Softmax(scale Q K^T) C per attention map: the attention kernel alone.  d_l is a
// multiple of 128, or 64 (the narrow case of the comparison operators).
gta_status_t launch_sm100_attention(const Dims& d, const void* q, const void* k, const void* c, void* l_out,
                                    int32_t* status_word, cudaStream_t stream, const PageMap& pm) {
    CUtensorMap tm_q, tm_k, tm_c;
    __nv_bfloat16* l_bf16 = static_cast<__nv_bfloat16*>(l_out);
    const uint32_t box[3] = {64, 128, 1}, box_k[3] = {64, 64, 1};
    const uint64_t dq[3] = {(uint64_t)d.d_h, (uint64_t)d.N, (uint64_t)d.B * d.n_q};
    if (pm.table != nullptr) {
        // paged pools [n_pages, groups, page_size, width]: one plane per (page, group), blocks of 64 tokens
        if (pm.page_size % 64 != 0) return GTA_ERR_UNSUPPORTED;
        const uint64_t pk[3] = {(uint64_t)d.d_h, (uint64_t)pm.page_size, (uint64_t)pm.n_pages * d.n_k};
        const uint64_t pc[3] = {(uint64_t)d.d_l, (uint64_t)pm.page_size, (uint64_t)pm.n_pages * d.n_c};
        if (!make_bf16_map(&tm_q, q, 3, dq, box) || !make_bf16_map(&tm_k, k, 3, pk, box_k) ||
            !make_bf16_map(&tm_c, c, 3, pc, box_k))
            return GTA_ERR_CUDA;
    } else {
        // K / C: Nk of the S rows of a plane take part; the rest (the unused tail of a cache, which may hold
        // anything, NaN bit patterns included) lies outside the maps and reads as zeros
        const uint64_t dk[3] = {(uint64_t)d.d_h, (uint64_t)d.Nk, (uint64_t)d.B * d.n_k};
        const uint64_t dc[3] = {(uint64_t)d.d_l, (uint64_t)d.Nk, (uint64_t)d.B * d.n_c};
        const uint64_t ak[3] = {(uint64_t)d.d_h, (uint64_t)d.S, (uint64_t)d.B * d.n_k};
        const uint64_t ac[3] = {(uint64_t)d.d_l, (uint64_t)d.S, (uint64_t)d.B * d.n_c};
        if (!make_bf16_map(&tm_q, q, 3, dq, box) || !make_bf16_map(&tm_k, k, 3, dk, box_k, ak) ||
            !make_bf16_map(&tm_c, c, 3, dc, box, ac))
            return GTA_ERR_CUDA;
    }
    gta_status_t st;
    if (d.d_h == 128)
        st = d.d_l % 256 == 0 ? launch_attention<128, 256>(d, pm, tm_q, tm_k, tm_c, l_bf16, status_word, stream)
                              : launch_attention<128, 128>(d, pm, tm_q, tm_k, tm_c, l_bf16, status_word, stream);
    else
        st = d.d_l % 256 == 0 ? launch_attention<64, 256>(d, pm, tm_q, tm_k, tm_c, l_bf16, status_word, stream)
                              : launch_attention<64, 128>(d, pm, tm_q, tm_k, tm_c, l_bf16, status_word, stream);
    if (st != GTA_OK) return st;
    return cudaGetLastError() == cudaSuccess ? GTA_OK : GTA_ERR_CUDA;
}

gta_status_t launch_sm100_prefill(const Dims& d, const void* q, const void* k, const void* c, const void* x,
                                  const void* w_p, const void* w_g, void* out, void* workspace,
                                  int32_t* status_word, cudaStream_t stream, int stages, int* launches,
                                  const PageMap& pm) {
    if (stages & 1) {
        gta_status_t st = launch_sm100_attention(d, q, k, c, workspace, status_word, stream, pm);
        if (st != GTA_OK) return st;
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
