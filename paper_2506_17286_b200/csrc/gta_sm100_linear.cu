// tcgen05 / TMA linear maps of the attention layer around the operator (App. B.1.1):
//
//   input projections   [Q | K | C] = H_in [W_Q | W_K | W_C],  q and k then pass through RoPE and every
//                       column block goes straight to where the operator reads it: q to [B, n_q, N, d_h],
//                       k and c to rows pos0 + t of the caches (the prefill's bulk append);
//   output projection   u_t = W_O [o_{t,1} (.) g_{t,1}; ...]  (the operator's output times W_O).
//
// One kernel, C[M, n_cols] = A[M, K] W[K, n_cols] in bf16 with fp32 accumulation, two epilogues.
// Persistent CTA pairs (clusters of 2, tcgen05 cta_group::2, M = 256): a pair walks the (row tile,
// column block) units pr, pr + G, ...; a column block is 256 columns (128 at the ragged end).  Each
// CTA owns 128 of the unit's rows and stages its own A rows plus half of the unit's weight columns.
//   warp 0      TMA producer, 6-stage ring of {A tile 128 x 64, W tile 64 x block / 2}
//   warp 1      (leader CTA) MMA issuer; two accumulators of 256 TMEM columns alternate between
//               units, so the epilogue of unit n overlaps the MMAs of unit n + 1
//   warps 2-9   epilogue: TMEM -> registers -> (RoPE) -> bf16 -> global, one token row per thread
//
// RoPE (RoFormer, which the paper cites): the pairs are neighbouring elements (2 i, 2 i + 1) of a
// d_h-vector, rotated by the angle pos theta_i with theta_i = base^(-2 i / d_h).  A small kernel ahead
// of the projection writes (cos, sin) of every (position of the chunk, pair) to a table: the angle is
// formed and reduced to [-pi, pi] in double precision (theta_i comes from the host as doubles), so that
// long contexts do not lose the phase; sine and cosine are then single precision.  The projection's
// epilogue only loads its 16 pairs per 32-column piece (transcendentals inside it cost more than the
// MMAs of a unit: 75 us against 45 us on a 8192 x 2048 x 1536 projection).
#include "gta_sm100.cuh"

#include <cuda.h>
#include <math.h>

#include "sm100_ptx.cuh"
#include "tma_host.cuh"

namespace gta {

namespace {

constexpr int kLinStages = 6;
constexpr int kLinThreads = 352;    // warp 0 TMA, warp 1 MMA issue, warps 2-9 epilogue, warp 10 second MMA issuer (one-tile form)
constexpr int kTileM = 128;        // rows per CTA and unit
constexpr int kBlockK = 64;        // K elements per pipeline stage (one 128-byte swizzle row)
constexpr uint32_t kATileBytes = kTileM * kBlockK * 2;   // 16 KB
constexpr uint32_t kBGroupBytes = kBlockK * 64 * 2;      // 64 K-rows x 64 columns = 8 KB
constexpr uint32_t kStageBytes = kATileBytes + 2 * kBGroupBytes;   // 32 KB per CTA
constexpr uint32_t kBarOffset = kLinStages * kStageBytes;
constexpr uint32_t kLinSmemTotal = kBarOffset + 512 + 1024;        // barriers + alignment slack
constexpr int kMaxRopePairs = 64;  // d_h <= 128
// Without CTA pairs (at most 128 rows in all: a decode step): the A tile holds only the rows that exist,
// rounded up to the 8-row swizzle atom, which leaves room for a much deeper ring -- with one unit per CTA
// and few CTAs the bytes in flight per SM pace the kernel.  The MMA still reads 128 rows: the rows past the
// tile are whatever follows in shared memory, and only feed accumulator rows that are never stored.
constexpr int kMaxStages = 16;
constexpr uint32_t kSoloRingBytes = 200 * 1024;

struct LinArgs {
    int M, K, n_cols;        // C[M, n_cols] = A[M, K] W[K, n_cols]
    int block;               // columns per block: 256, 128 when there is a single 256-row tile, 64 without CTA pairs
    int n_stages;            // ring depth
    uint32_t a_bytes;        // bytes of an A tile in the ring
    int n_cb;                // column blocks (the last one possibly 128 wide)
    int n_units;             // row tiles (256 rows) x column blocks
    // Static schedule over G CTA pairs (or CTAs): every pair takes q = n_units / G whole units (unit pr + n G,
    // so that neighbouring pairs share a row tile); the r = n_units mod G left over are cut into two halves of
    // 128 columns when that makes the last round shorter (2 r <= G and every block is 256 wide), else handed
    // out whole.
    int q, r, split_tail;
    // plain epilogue
    __nv_bfloat16* c_out;    // [M, n_cols]
    // projection epilogue: row = b N + t
    Dims d;
    int pos0, S_cap;         // position of token 0 of the chunk; rows per cache plane
    __nv_bfloat16* q_out;    // [B, n_q, N, d_h]
    __nv_bfloat16* k_cache;  // [B, n_k, S_cap, d_h]
    __nv_bfloat16* c_cache;  // [B, n_c, S_cap, d_l]
    const float2* rope;      // [N, d_h / 2] (cos, sin) of position pos0 + t, pair i
    // one new token per sequence (N = 1): its position, or -1 for a sequence whose cache is full (nothing is
    // written for it); the table then has one row per sequence
    const int32_t* pos_seq;
    PageMap pm;              // table != nullptr: the caches are paged pools (decode step only)
};

struct RopeArgs {
    int pos0, n_pairs, n_tokens;
    double theta[kMaxRopePairs];
};

// one thread per (token of the chunk, pair)
__global__ void __launch_bounds__(256)
rope_table_kernel(const __grid_constant__ RopeArgs r, float2* __restrict__ table) {
    // launched with programmatic stream serialisation: the table may still be read by the kernel ahead
    ptx::grid_dependency_wait();
    ptx::grid_launch_dependents();
    const int idx = blockIdx.x * 256 + threadIdx.x;
    const int t = idx / r.n_pairs, i = idx - t * r.n_pairs;
    if (t >= r.n_tokens) return;
    double ang = (double)(r.pos0 + t) * r.theta[i];
    ang -= 6.283185307179586476925287 * rint(ang * 0.159154943091895335768884);
    float sn, cs;
    sincosf((float)ang, &sn, &cs);
    table[(size_t)t * r.n_pairs + i] = make_float2(cs, sn);
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// One decode step's bookkeeping, one CTA per sequence: the new token's position is the current length; the
// (cos, sin) row of that position; then the length advances.  A full cache leaves the length alone,
// raises the status word and marks the sequence with position -1.
__global__ void __launch_bounds__(kMaxRopePairs)
rope_decode_prep_kernel(const __grid_constant__ RopeArgs r, int S_cap, int32_t* __restrict__ seq_lens,
                        int32_t* __restrict__ pos_out, float2* __restrict__ table, int32_t* status_word) {
    // launched with programmatic stream serialisation: lengths, positions and table belong to the kernels ahead
    // in the stream until they are complete
    ptx::grid_dependency_wait();
    ptx::grid_launch_dependents();
    const int b = blockIdx.x, i = threadIdx.x;
    const int len = seq_lens[b];
    __syncthreads();   // every thread has read the old length before thread 0 rewrites it
    const bool ok = len >= 0 && len < S_cap;
    if (i < r.n_pairs) {
        double ang = (double)(ok ? len : 0) * r.theta[i];
        ang -= 6.283185307179586476925287 * rint(ang * 0.159154943091895335768884);
        float sn, cs;
        sincosf((float)ang, &sn, &cs);
        table[(size_t)b * r.n_pairs + i] = make_float2(cs, sn);
    }
    if (i == 0) {
        pos_out[b] = ok ? len : -1;
        if (ok) seq_lens[b] = len + 1;
        else raise_status(status_word, GTA_ERR_CACHE_FULL);
    }
}

// kProject: the epilogue of the input projections (RoPE + scatter); otherwise a plain row-major store
// kPair: CTA pairs (cta_group::2, M = 256); otherwise single CTAs (cta_group::1, M = 128) on 64-column units
template <bool kProject, bool kPair>
__global__ void __launch_bounds__(kLinThreads, 1)
sm100_linear_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_w,
                    const __grid_constant__ LinArgs a, int32_t* status_word) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    // ring: pairs keep {A, W} of a stage side by side; without pairs all A tiles come first, then all W tiles
    const int n_stages = kPair ? kLinStages : a.n_stages;
    const uint32_t a_stride = kPair ? kStageBytes : a.a_bytes;
    const uint32_t b_base = kPair ? kATileBytes : (uint32_t)n_stages * a.a_bytes;
    const uint32_t b_stride = kPair ? kStageBytes : kBGroupBytes;
    const uint32_t a_tile_bytes = kPair ? kATileBytes : a.a_bytes;
    const uint32_t bar_off = kPair ? kBarOffset : (uint32_t)n_stages * (a.a_bytes + kBGroupBytes);
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + bar_off);       // used in the leader CTA
    uint64_t* empty_bar = full_bar + kMaxStages;                             // both CTAs
    uint64_t* acc_full = empty_bar + kMaxStages;                             // [2] both CTAs
    uint64_t* acc_free = acc_full + 2;                                       // [2] leader CTA: 16 warps arrive
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_free + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile int* drain_flag = abort_flag + 1;   // never raised: lets the drain wait run to its limit

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = kPair ? ptx::cluster_ctarank() : 0u;          // 0 = leader
    const int G = kPair ? gridDim.x >> 1 : gridDim.x;                   // CTA pairs (or CTAs)
    const int pr = kPair ? blockIdx.x >> 1 : blockIdx.x;
    constexpr int kUnitRows = kPair ? 2 * kTileM : kTileM;
    const int n_items = a.q + ((a.split_tail ? pr < 2 * a.r : pr < a.r) ? 1 : 0);
    const int ks_total = a.K / kBlockK;
    // One-tile form: a single thread's instruction stream (wait, descriptors, four MMAs, commit per k-block) is what
    // paces a CTA there, so two threads issue -- the even and the odd k-blocks, into accumulators of their own that the
    // epilogue adds.
    const bool two_issuers = !kPair && ks_total >= 2;

    if (threadIdx.x == 0) {
        for (int s = 0; s < n_stages; ++s) { ptx::mbar_init(&full_bar[s], kPair ? 2 : 1); ptx::mbar_init(&empty_bar[s], 1); }
        for (int j = 0; j < 2; ++j) { ptx::mbar_init(&acc_full[j], two_issuers ? 2 : 1); ptx::mbar_init(&acc_free[j], kPair ? 16 : 8); }
        *abort_flag = 0;
        *drain_flag = 0;
        ptx::fence_mbar_init();
    }
    if (warp == 1) {
        if (kPair) ptx::tmem_alloc_pair(tmem_slot, 512);
        else ptx::tmem_alloc(tmem_slot, 512);
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (kPair) {
        ptx::cluster_arrive();     // the peer's barriers exist before anything is signalled to them
        ptx::cluster_wait();
    }
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // Launched with programmatic stream serialisation: the set-up above may have run while the kernel ahead
    // in the stream was draining.  Nothing of global memory is touched before that kernel is complete, and
    // only then may the kernel behind this one be scheduled.
    ptx::grid_dependency_wait();
    ptx::grid_launch_dependents();

    // unit n of this pair: column block cb (consecutive pairs share a row tile), first row, first column, width
    auto unit = [&](int n, int& row0, int& f0, int& nt) {
        int u, half = -1;
        if (n < a.q) u = pr + n * G;
        else if (a.split_tail) { u = G * a.q + (pr >> 1); half = pr & 1; }
        else u = G * a.q + pr;
        const int cb = u % a.n_cb;
        row0 = (u / a.n_cb) * kUnitRows;
        f0 = cb * a.block;
        nt = a.n_cols - f0 < a.block ? a.n_cols - f0 : a.block;
        if (half >= 0) { f0 += 128 * half; nt = 128; }
    };

    if (warp == 0) {
        if (ptx::elect_one()) {
            ptx::prefetch_tensormap(&tm_a);
            ptx::prefetch_tensormap(&tm_w);
            int it = 0, s = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int n = 0; n < n_items && ok; ++n) {
                int row0, f0, nt;
                unit(n, row0, f0, nt);
                const int r0 = row0 + (int)rank * kTileM;          // this CTA's rows
                const int n_grp = kPair ? nt / 128 : 1;             // 64-column groups this CTA stages
                const int fc = kPair ? f0 + (int)rank * (nt / 2) : f0;   // this CTA's first weight column
                const uint32_t tx = a_tile_bytes + (uint32_t)n_grp * kBGroupBytes;
                const uint32_t bar_base = kPair ? ptx::map_to_cta(ptx::smem_addr(&full_bar[0]), 0) : 0u;   // the leader's
                for (int ks = 0; ks < ks_total; ++ks, ++it, s = (s + 1 == n_stages) ? 0 : s + 1, ph ^= (s == 0)) {
                    ok = ptx::mbar_wait(&empty_bar[s], ph ^ 1, abort_flag);
                    if (!ok) break;
                    uint8_t* a_s = smem + s * a_stride;
                    uint8_t* b_s = smem + b_base + s * b_stride;
                    if (!kPair) {
                        ptx::mbar_arrive_expect_tx(&full_bar[s], tx);
                        ptx::tma_load_2d(a_s, &tm_a, &full_bar[s], ks * kBlockK, r0);
                        ptx::tma_load_2d(b_s, &tm_w, &full_bar[s], fc, ks * kBlockK);
                        continue;
                    }
                    const uint32_t bar = bar_base + (uint32_t)s * 8;
                    ptx::mbar_arrive_expect_tx_cluster(bar, tx);
                    ptx::tma_load_2d_pair(a_s, &tm_a, bar, ks * kBlockK, r0);
                    for (int grp = 0; grp < n_grp; ++grp)
                        ptx::tma_load_2d_pair(b_s + grp * kBGroupBytes, &tm_w, bar, fc + grp * 64, ks * kBlockK);
                }
            }
            if (*abort_flag && rank == 0) {   // drain: every armed stage either lands or the wait gives up
                for (int back = 1; back <= n_stages && it - back >= 0; ++back) {
                    const int kq = it - back;
                    ptx::mbar_wait_drain(&full_bar[kq % n_stages], (kq / n_stages) & 1, drain_flag);
                }
            }
        }
    } else if (!kPair && (warp == 1 || warp == 10)) {
        // one-tile form: issuer `me` takes the k-blocks it = me, me + 2, ... (all of them without a second issuer)
        const int me = warp == 1 ? 0 : 1, step = two_issuers ? 2 : 1;
        if ((me == 0 || two_issuers) && ptx::elect_one()) {
            const uint64_t desc_a0 = ptx::make_smem_desc(0, 16, 1024);
            const uint64_t desc_b0 = ptx::make_smem_desc(0, 64 * 128, 1024);
            const uint32_t smem_a = ptx::smem_addr(smem), smem_b = ptx::smem_addr(smem + b_base);
            bool ok = true;
            int it0 = 0;                 // first k-block of the unit in the ring's count
            for (int n = 0; n < n_items && ok; ++n, it0 += ks_total) {
                int row0, f0, nt;
                unit(n, row0, f0, nt);
                const uint32_t idesc = ptx::make_idesc_bf16(kTileM, nt, 0, 1);   // A K-major, W MN-major
                const uint32_t d_tmem = tmem_base + (uint32_t)(n & 1) * 256 + (uint32_t)me * 64;
                ok = ptx::mbar_wait(&acc_free[n & 1], ((n >> 1) & 1) ^ 1, abort_flag);
                bool first = true;
                int it = it0 + ((it0 + me) & (step - 1));
                int s = it % n_stages;                       // stage and phase kept as counters (no division per k-block)
                uint32_t ph = (uint32_t)(it / n_stages) & 1u;
                for (; it < it0 + ks_total && ok; it += step, s += step) {
                    if (s >= n_stages) { s -= n_stages; ph ^= 1u; }
                    ok = ptx::mbar_wait(&full_bar[s], ph, abort_flag);
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    const uint64_t a_desc = desc_a0 + ((smem_a + (uint32_t)s * a_stride) >> 4);
                    const uint64_t b_desc = desc_b0 + ((smem_b + (uint32_t)s * b_stride) >> 4);
#pragma unroll
                    for (int k4 = 0; k4 < kBlockK / 16; ++k4)
                        ptx::mma_ss(d_tmem, a_desc + 2 * k4, b_desc + k4 * ((16 * 128) >> 4), idesc, (first && k4 == 0) ? 0u : 1u);
                    first = false;
                    ptx::tc_commit(&empty_bar[s]);
                }
                if (ok) ptx::tc_commit(&acc_full[n & 1]);
            }
        }
    } else if (warp == 1) {
        if (rank == 0 && ptx::elect_one()) {
            int it = 0, s = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int n = 0; n < n_items && ok; ++n) {
                int row0, f0, nt;
                unit(n, row0, f0, nt);
                const uint32_t idesc = ptx::make_idesc_bf16(kUnitRows, nt, 0, 1);   // A K-major, W MN-major
                const uint32_t d_tmem = tmem_base + (uint32_t)(n & 1) * 256;
                // the accumulator about to be overwritten (unit n - 2) must have been read by both epilogues
                ok = ptx::mbar_wait(&acc_free[n & 1], ((n >> 1) & 1) ^ 1, abort_flag);
                for (int ks = 0; ks < ks_total && ok; ++ks, ++it, s = (s + 1 == n_stages) ? 0 : s + 1, ph ^= (s == 0)) {
                    ok = ptx::mbar_wait(&full_bar[s], ph, abort_flag);
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    const uint32_t a_addr = ptx::smem_addr(smem + s * a_stride);
                    const uint32_t b_addr = ptx::smem_addr(smem + b_base + s * b_stride);
#pragma unroll
                    for (int k4 = 0; k4 < kBlockK / 16; ++k4) {
                        const uint64_t a_desc = ptx::make_smem_desc(a_addr + k4 * 32, 16, 1024);
                        const uint64_t b_desc = ptx::make_smem_desc(b_addr + k4 * 16 * 128, 64 * 128, 1024);
                        if (kPair) ptx::mma_ss_pair(d_tmem, a_desc, b_desc, idesc, (ks == 0 && k4 == 0) ? 0u : 1u);
                        else ptx::mma_ss(d_tmem, a_desc, b_desc, idesc, (ks == 0 && k4 == 0) ? 0u : 1u);
                    }
                    if (kPair) {
                        ptx::tc_commit_pair(&empty_bar[s], 3);
                        if (ks == ks_total - 1) ptx::tc_commit_pair(&acc_full[n & 1], 3);
                    } else {
                        ptx::tc_commit(&empty_bar[s]);
                        if (ks == ks_total - 1) ptx::tc_commit(&acc_full[n & 1]);
                    }
                }
            }
        }
    } else if (warp >= 2 && warp < 10) {
        // epilogue: warp w may touch TMEM lanes [32 (w % 4), 32 (w % 4) + 32); the two warps of a
        // quarter take one half of the unit's columns each
        const int quarter = warp & 3;
        const int half = (warp - 2) >> 2;
        const int row_in_tile = quarter * 32 + lane;
        const uint32_t lane_base = ((uint32_t)(quarter * 32) << 16);
        const uint32_t acc_free_leader[2] = {kPair ? ptx::map_to_cta(ptx::smem_addr(&acc_free[0]), 0) : 0u,
                                             kPair ? ptx::map_to_cta(ptx::smem_addr(&acc_free[1]), 0) : 0u};
        const int Dq = a.d.n_q * a.d.d_h, Dk = a.d.n_k * a.d.d_h;
        bool ok = true;
        for (int n = 0; n < n_items && ok; ++n) {
            int row0, f0, nt;
            unit(n, row0, f0, nt);
            const int cols = nt / 2;                 // this warp's columns: 128, 64 or 32
            const int c0 = half * cols;
            const int row = row0 + (int)rank * kTileM + row_in_tile;
            bool live = row < a.M;
            const int b = kProject ? (live ? row / a.d.N : 0) : 0;
            const int t = kProject ? (live ? row - b * a.d.N : 0) : 0;
            int pos = a.pos0 + t, rope_row = t;
            if (kProject && a.pos_seq != nullptr) {
                pos = a.pos_seq[b];
                rope_row = b;
                live = live && pos >= 0;
                if (pos < 0) pos = 0;
            }
            const uint32_t acc = tmem_base + (uint32_t)(n & 1) * 256 + lane_base + c0;
            // (cos, sin) of the 16 pairs of piece ch, fetched one piece ahead of its use -- the first one before
            // the accumulator is even complete: they depend on the row and the columns only
            float4 rope_next[8];
            auto fetch_rope = [&](int ch) {
                const int col = f0 + c0 + ch * 32;
                if (!kProject || ch * 32 >= cols || col >= Dq + Dk) return;
                const int cc = col < Dq ? col : col - Dq;
                const int e0 = cc % a.d.d_h;
                const float4* rt = reinterpret_cast<const float4*>(a.rope + ((size_t)rope_row * (a.d.d_h >> 1) + (e0 >> 1)));
#pragma unroll
                for (int j2 = 0; j2 < 8; ++j2) rope_next[j2] = __ldg(rt + j2);
            };
            fetch_rope(0);
            ok = __all_sync(0xffffffffu, ptx::mbar_wait(&acc_full[n & 1], (n >> 1) & 1, abort_flag));
            if (!ok) break;
            ptx::tc_fence_after_sync();
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
                if (ch * 32 < cols) {
                    uint32_t v[32];
                    ptx::tmem_ld32(acc + ch * 32, v);
                    if (two_issuers) {       // the second issuer's share of the sum (64 columns further on)
                        uint32_t v2[32];
                        ptx::tmem_ld32(acc + 64 + ch * 32, v2);
                        ptx::tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e) v[e] = __float_as_uint(__uint_as_float(v[e]) + __uint_as_float(v2[e]));
                    }
                    float4 rope_cur[8];
#pragma unroll
                    for (int j2 = 0; j2 < 8; ++j2) rope_cur[j2] = rope_next[j2];
                    if (ch + 1 < 4) fetch_rope(ch + 1);
                    ptx::tmem_wait_ld();
                    const int col = f0 + c0 + ch * 32;     // first of these 32 output columns
                    __nv_bfloat16* dst;
                    if (!kProject) {
                        dst = a.c_out + (size_t)(live ? row : 0) * a.n_cols + col;
                    } else if (col < Dq + Dk) {
                        // a 32-column chunk lies inside one d_h-vector (d_h is a multiple of 64)
                        const bool is_q = col < Dq;
                        const int cc = is_q ? col : col - Dq;
                        const int g = cc / a.d.d_h, e0 = cc - g * a.d.d_h;
#pragma unroll
                        for (int j2 = 0; j2 < 8; ++j2) {      // two pairs per 16-byte table entry
                            const float4 r4 = rope_cur[j2];
                            const float x0 = __uint_as_float(v[4 * j2]), x1 = __uint_as_float(v[4 * j2 + 1]);
                            const float x2 = __uint_as_float(v[4 * j2 + 2]), x3 = __uint_as_float(v[4 * j2 + 3]);
                            v[4 * j2] = __float_as_uint(x0 * r4.x - x1 * r4.y);
                            v[4 * j2 + 1] = __float_as_uint(x0 * r4.y + x1 * r4.x);
                            v[4 * j2 + 2] = __float_as_uint(x2 * r4.z - x3 * r4.w);
                            v[4 * j2 + 3] = __float_as_uint(x2 * r4.w + x3 * r4.z);
                        }
                        if (is_q) {
                            dst = a.q_out + (((size_t)b * a.d.n_q + g) * a.d.N + t) * a.d.d_h + e0;
                        } else {
                            const long long kr = cache_row(a.pm, b, a.d.n_k, g, a.S_cap, pos, status_word);
                            live = live && kr >= 0;          // a block-table entry outside the pool: nothing is written
                            dst = a.k_cache + (size_t)(kr < 0 ? 0 : kr) * a.d.d_h + e0;
                        }
                    } else {
                        const int cc = col - Dq - Dk;
                        const int g = cc / a.d.d_l, e0 = cc - g * a.d.d_l;
                        const long long cr = cache_row(a.pm, b, a.d.n_c, g, a.S_cap, pos, status_word);
                        live = live && cr >= 0;
                        dst = a.c_cache + (size_t)(cr < 0 ? 0 : cr) * a.d.d_l + e0;
                    }
                    if (live) {
#pragma unroll
                        for (int w2 = 0; w2 < 2; ++w2) {      // 2 x 32 bytes: whole sectors
                            uint32_t ww[8];
#pragma unroll
                            for (int e = 0; e < 8; ++e)
                                ww[e] = pack_bf16x2(__uint_as_float(v[16 * w2 + 2 * e]), __uint_as_float(v[16 * w2 + 2 * e + 1]));
                            ptx::st_global_256(dst + w2 * 16, ww);
                        }
                    }
                }
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                if (kPair) ptx::mbar_arrive_cluster(acc_free_leader[n & 1]);
                else ptx::mbar_arrive(&acc_free[n & 1]);
            }
        }
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (kPair) {
        ptx::cluster_arrive();     // neither CTA leaves (or frees TMEM) while the other may still signal it
        ptx::cluster_wait();
    }
    if (warp == 1) {
        if (kPair) ptx::tmem_dealloc_pair(tmem_base, 512);
        else ptx::tmem_dealloc(tmem_base, 512);
    }
    if (threadIdx.x == 0 && *abort_flag) raise_status(status_word, GTA_ERR_TIMEOUT);
}

// SM count of the CURRENT device, looked up once per device ordinal and thread
int lin_sm_count() {
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

template <bool kProject>
gta_status_t launch_linear(const LinArgs& a, const void* a_ptr, const void* w_ptr, int32_t* status_word,
                           cudaStream_t stream) {
    CUtensorMap tm_a, tm_w;
    const bool solo = a.M <= kTileM;
    {
        const uint64_t dims[2] = {(uint64_t)a.K, (uint64_t)a.M};
        const uint32_t box[2] = {kBlockK, solo ? a.a_bytes / (kBlockK * 2) : (uint32_t)kTileM};
        if (!make_bf16_map(&tm_a, a_ptr, 2, dims, box)) return GTA_ERR_CUDA;
    }
    {
        const uint64_t dims[2] = {(uint64_t)a.n_cols, (uint64_t)a.K};
        const uint32_t box[2] = {64, kBlockK};
        if (!make_bf16_map(&tm_w, w_ptr, 2, dims, box)) return GTA_ERR_CUDA;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kLinThreads);
    cfg.stream = stream;
    if (solo) {   // 64-column units over as many SMs as there are units
        auto kern1 = sm100_linear_kernel<kProject, false>;
        const uint32_t smem_bytes = (uint32_t)a.n_stages * (a.a_bytes + kBGroupBytes) + 512 + 1024;
        if (cudaFuncSetAttribute(kern1, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes) != cudaSuccess)
            return GTA_ERR_CUDA;
        cfg.dynamicSmemBytes = smem_bytes;
        const int G1 = a.n_units < lin_sm_count() ? a.n_units : lin_sm_count();
        LinArgs a1 = a;
        a1.q = a.n_units / G1;
        a1.r = a.n_units % G1;
        a1.split_tail = 0;
        cfg.gridDim = dim3(G1);
        cudaLaunchAttribute attr1[1];
        attr1[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr1[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr1;
        cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, kern1, tm_a, tm_w, a1, status_word) != cudaSuccess) return GTA_ERR_CUDA;
        return cudaGetLastError() == cudaSuccess ? GTA_OK : GTA_ERR_CUDA;
    }
    auto kern = sm100_linear_kernel<kProject, true>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kLinSmemTotal) != cudaSuccess)
        return GTA_ERR_CUDA;
    cfg.dynamicSmemBytes = kLinSmemTotal;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;   // the occupancy query below takes the cluster attribute only
    // a persistent grid must be resident at once: as many pairs as the device can hold, asked once per device
    static thread_local int cached_dev = -1, cached_pairs = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return GTA_ERR_CUDA;
    if (dev != cached_dev) {
        cfg.gridDim = dim3(2 * (lin_sm_count() / 2));
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n < 1) return GTA_ERR_CUDA;
        cached_dev = dev;
        cached_pairs = n;
    }
    const int G = a.n_units < cached_pairs ? a.n_units : cached_pairs;
    LinArgs a2 = a;
    a2.q = a.n_units / G;
    a2.r = a.n_units % G;
    a2.split_tail = (a.block == 256 && a.n_cols % 256 == 0 && 2 * a2.r <= G) ? 1 : 0;
    cfg.gridDim = dim3(2 * G);
    cfg.numAttrs = 2;
    if (cudaLaunchKernelEx(&cfg, kern, tm_a, tm_w, a2, status_word) != cudaSuccess) return GTA_ERR_CUDA;
    return cudaGetLastError() == cudaSuccess ? GTA_OK : GTA_ERR_CUDA;
}

bool fill_common(LinArgs& a, long long M, int K, int n_cols) {
    if (M <= 0 || M > 0x3fffffffLL || K < kBlockK || K % kBlockK != 0 || n_cols < 128 || n_cols % 128 != 0) return false;
    a.M = (int)M;
    a.K = K;
    a.n_cols = n_cols;
    const bool solo = M <= kTileM;
    // a single row tile: narrower blocks keep more SMs busy
    a.block = solo ? 64 : (M <= 2 * kTileM ? 128 : 256);
    a.n_cb = (n_cols + a.block - 1) / a.block;
    a.n_stages = kLinStages;
    a.a_bytes = kATileBytes;
    if (solo) {
        a.a_bytes = (uint32_t)((M + 7) & ~7LL) * kBlockK * 2;
        a.n_stages = (int)(kSoloRingBytes / (a.a_bytes + kBGroupBytes));
        if (a.n_stages > kMaxStages) a.n_stages = kMaxStages;
        // the MMA reads 16 KB from every A tile: the W tiles behind the last one must cover that
        if ((uint32_t)a.n_stages * kBGroupBytes < kATileBytes) return false;
    }
    const long long unit_rows = solo ? kTileM : 2 * kTileM;
    const long long units = ((M + unit_rows - 1) / unit_rows) * a.n_cb;
    if (units > 0x3fffffffLL) return false;
    a.n_units = (int)units;
    return true;
}

}  // namespace

bool sm100_linear_supported(const Dims& d, int dtype) {
    if (dtype != GTA_BF16 || d.H % kBlockK != 0 || d.d_h % 64 != 0 || d.d_h > 2 * kMaxRopePairs || d.d_l % 64 != 0)
        return false;
    const int qkc = (d.n_q + d.n_k) * d.d_h + d.n_c * d.d_l;
    return qkc % 128 == 0 && d.H % 128 == 0 && (d.n_h * d.d_h) % kBlockK == 0;
}

size_t sm100_rope_table_bytes(const Dims& d) { return (size_t)d.N * (d.d_h / 2) * sizeof(float2); }

gta_status_t launch_sm100_project(const Dims& d, int pos0, int S_cap, double rope_base, const void* x,
                                  const void* w_qkc, void* q_out, void* k_cache, void* c_cache, void* rope_table,
                                  int32_t* status_word, cudaStream_t stream, const PageMap& pm) {
    LinArgs a = {};
    if (!fill_common(a, (long long)d.B * d.N, d.H, (d.n_q + d.n_k) * d.d_h + d.n_c * d.d_l)) return GTA_ERR_UNSUPPORTED;
    a.d = d;
    a.pos0 = pos0;
    a.S_cap = S_cap;
    a.q_out = static_cast<__nv_bfloat16*>(q_out);
    a.k_cache = static_cast<__nv_bfloat16*>(k_cache);
    a.c_cache = static_cast<__nv_bfloat16*>(c_cache);
    a.rope = static_cast<const float2*>(rope_table);
    a.pm = pm;
    RopeArgs r = {};
    r.pos0 = pos0;
    r.n_pairs = d.d_h / 2;
    for (int i = 0; i < r.n_pairs; ++i) r.theta[i] = pow(rope_base, -2.0 * i / d.d_h);
    r.n_tokens = d.N;
    {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((d.N * r.n_pairs + 255) / 256);
        cfg.blockDim = dim3(256);
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, rope_table_kernel, r, static_cast<float2*>(rope_table)) != cudaSuccess ||
            cudaGetLastError() != cudaSuccess)
            return GTA_ERR_CUDA;
    }
    return launch_linear<true>(a, x, w_qkc, status_word, stream);
}

size_t sm100_decode_prep_bytes(const Dims& d) {
    return (((size_t)d.B * (d.d_h / 2) * sizeof(float2) + 255) & ~(size_t)255) + (size_t)d.B * sizeof(int32_t);
}

gta_status_t launch_sm100_project_step(const Dims& d, int S_cap, double rope_base, const void* x_t, const void* w_qkc,
                                       void* q_out, void* k_cache, void* c_cache, int32_t* seq_lens, void* prep,
                                       int32_t* status_word, cudaStream_t stream, const PageMap& pm) {
    LinArgs a = {};
    a.pm = pm;
    Dims d1 = d;
    d1.N = 1;
    if (!fill_common(a, d.B, d.H, (d.n_q + d.n_k) * d.d_h + d.n_c * d.d_l)) return GTA_ERR_UNSUPPORTED;
    a.d = d1;
    a.S_cap = S_cap;
    a.q_out = static_cast<__nv_bfloat16*>(q_out);
    a.k_cache = static_cast<__nv_bfloat16*>(k_cache);
    a.c_cache = static_cast<__nv_bfloat16*>(c_cache);
    float2* table = static_cast<float2*>(prep);
    int32_t* pos = reinterpret_cast<int32_t*>(static_cast<char*>(prep) +
                                              (((size_t)d.B * (d.d_h / 2) * sizeof(float2) + 255) & ~(size_t)255));
    a.rope = table;
    a.pos_seq = pos;
    RopeArgs r = {};
    r.n_pairs = d.d_h / 2;
    for (int i = 0; i < r.n_pairs; ++i) r.theta[i] = pow(rope_base, -2.0 * i / d.d_h);
    {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(d.B);
        cfg.blockDim = dim3(kMaxRopePairs);
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, rope_decode_prep_kernel, r, S_cap, seq_lens, pos, table, status_word) !=
                cudaSuccess ||
            cudaGetLastError() != cudaSuccess)
            return GTA_ERR_CUDA;
    }
    return launch_linear<true>(a, x_t, w_qkc, status_word, stream);
}

gta_status_t launch_sm100_matmul(long long M, int K, int n_cols, const void* a_ptr, const void* w_ptr, void* c_out,
                                 int32_t* status_word, cudaStream_t stream) {
    LinArgs a = {};
    if (!fill_common(a, M, K, n_cols)) return GTA_ERR_UNSUPPORTED;
    a.c_out = static_cast<__nv_bfloat16*>(c_out);
    return launch_linear<false>(a, a_ptr, w_ptr, status_word, stream);
}

}  // namespace gta
