// tcgen05 / TMA decoder + gate kernel of the bf16 prefill path (d_h = 64 or 128):
//     out_i = (L_{q(i)} W_P,i) (.) sigmoid(X W_G,i)          (Sec. 3.3, reformulated equation)
//
// Persistent CTA pairs (clusters of 2, tcgen05 cta_group::2): a pair walks a static list of work
// items.  An item is a tile of 256 token rows x two heads of one attention map (256 output
// columns): each CTA of the pair owns 128 of the rows and stages its own A rows plus HALF of the
// item's weight columns, so a weight tile crosses L2 -> shared memory once per 256 rows.  What
// does not divide evenly over the pairs is cut into single-head items (128 columns) so that the
// last wave is short.  Roles in each CTA:
//   warp 0      TMA producer: 6-stage ring of {A tile 128 x 64, B tile 64 x NT/2}, gate operands
//               (X, W_G) first, then decoder operands (L, W_P); byte counts of both CTAs go to the
//               leader's barrier; it runs ahead into the next item.
//   warp 1      (leader CTA only) tcgen05.mma issuer, M = 256: acc_G (K = H) then acc_P (K = d_l),
//               side by side in each CTA's TMEM; completions are multicast to both CTAs' barriers.
//   warps 2-9   epilogue, two warps per TMEM lane quarter (one per head): as soon as acc_G is
//               complete they turn it into sigmoid gates held in registers (packed bf16) and hand
//               the columns back, so the MUFU work hides under the acc_P MMAs; when acc_P is
//               complete they multiply, round and store, while the next item's gate MMAs run.
//
// When all token rows fit one 128-row tile (a decode batch, a very short prompt) the second CTA of a
// pair would hold no rows at all, and a head per pair leaves most SMs idle while each pair spends
// its time on MMAs over padding.  That case runs the same kernel without pairs (template parameter
// kPair = false: plain clusters of one, cta_group::1, M = 128) on items of HALF a head (64
// columns), twice as many CTAs each with half the MMA time.
#include "gta_sm100.cuh"

#include <cuda.h>

#include "sm100_ptx.cuh"
#include "tma_host.cuh"

namespace gta {

namespace {

constexpr int kDecStages = 6;
constexpr int kDecThreads = 320;
constexpr int kTileM = 128;        // token rows per CTA and item
constexpr int kBlockK = 64;        // K elements per pipeline stage (one 128-byte swizzle row)
constexpr uint32_t kATileBytes = kTileM * kBlockK * 2;   // 16 KB
constexpr uint32_t kBGroupBytes = kBlockK * 64 * 2;      // 64 K-rows x 64 columns = 8 KB
constexpr uint32_t kStageBytes = kATileBytes + 2 * kBGroupBytes;   // 32 KB per CTA
constexpr uint32_t kBarOffset = kDecStages * kStageBytes;
constexpr uint32_t kBarBytes = 512;
constexpr uint32_t kDecSmemTotal = kBarOffset + kBarBytes + 1024;  // barriers + alignment slack
// Without CTA pairs (one row tile): the A tile holds only the rows that exist, rounded up to the
// 8-row swizzle atom, which leaves room for a much deeper ring -- with one item per CTA and few
// CTAs, the bytes in flight per SM are what paces the kernel.  The MMA still reads 128 rows: the
// rows past the tile are whatever follows in shared memory (other tiles), and only feed
// accumulator rows that are never stored.
constexpr int kMaxStages = 16;
constexpr uint32_t kSoloRingBytes = 200 * 1024;

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
// sigmoid(z) = 1/2 + 1/2 tanh(z / 2): one MUFU operation
__device__ __forceinline__ float sigmoid_tanh(float z) {
    float t;
    asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(0.5f * z));
    return fmaf(0.5f, t, 0.5f);
}

// Static schedule.  The output columns of a token (n_h d_h of them, head after head) are cut in
// blocks of 256 -- or 128 where the heads of an attention map do not fill a multiple of 256 -- that
// never straddle two maps.  U units (256 rows x column block) over G CTA pairs: every pair takes
// q = U / G whole units; the r = U mod G left over are cut in two halves (128 columns) when that
// makes the tail shorter (2 r <= G), else handed out whole.
struct Schedule {
    int n_hp;       // column blocks per row tile
    int pair;       // 1: a block is 256 columns (else 128; 64 without CTA pairs)
    int RT;         // 256-row tiles per sequence
    int q, r, split_tail;
    int n_stages;        // ring depth
    uint32_t a_bytes;    // bytes of an A tile in the ring
};

struct Item {
    int b, t0, f0, nt;   // batch entry, first token row, first output column (of n_h d_h), columns
};

__device__ __forceinline__ int items_of_pair(const Schedule& s, int pr) {
    if (s.split_tail) return s.q + ((pr < 2 * s.r) ? 1 : 0);
    return s.q + ((pr < s.r) ? 1 : 0);
}

template <bool kPair>
__device__ __forceinline__ Item item_of(const Schedule& s, int pr, int G, int n) {
    int u, half = -1;
    if (n < s.q) u = pr * s.q + n;
    else if (s.split_tail) { u = G * s.q + (pr >> 1); half = pr & 1; }
    else u = G * s.q + pr;
    Item it;
    const int hp = u % s.n_hp;
    const int rt = (u / s.n_hp) % s.RT;
    it.b = u / (s.n_hp * s.RT);
    if (!kPair) {            // 64 columns on one CTA
        it.t0 = rt * kTileM;
        it.f0 = hp * 64;
        it.nt = 64;
        return it;
    }
    it.t0 = rt * 2 * kTileM;
    if (s.pair) {
        it.f0 = 256 * hp + (half < 0 ? 0 : 128 * half);
        it.nt = half < 0 ? 256 : 128;
    } else {
        it.f0 = 128 * hp;
        it.nt = 128;
    }
    return it;
}

template <bool kPair>
__global__ void __launch_bounds__(kDecThreads, 1)
sm100_decoder_kernel(const __grid_constant__ CUtensorMap tm_l, const __grid_constant__ CUtensorMap tm_x,
                     const __grid_constant__ CUtensorMap tm_wp, const __grid_constant__ CUtensorMap tm_wg,
                     Dims d, Schedule sch, __nv_bfloat16* __restrict__ out, int32_t* status_word,
                     int32_t* step_lens, int step_batch, int step_cap) {
    // step_lens != nullptr (the fused append + decode step): once the kernel before this one is complete --
    // and with it every reader of the sequence lengths --, the producer thread of CTA 0 advances the length
    // of every sequence that had room for its new token.
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    // ring: pairs keep {A, B} of a stage side by side; without pairs all A tiles come first, then all B tiles
    const int n_stages = kPair ? kDecStages : sch.n_stages;
    const uint32_t a_stride = kPair ? kStageBytes : sch.a_bytes;
    const uint32_t b_base = kPair ? kATileBytes : (uint32_t)n_stages * sch.a_bytes;
    const uint32_t b_stride = kPair ? kStageBytes : kBGroupBytes;
    const uint32_t a_tile_bytes = kPair ? kATileBytes : sch.a_bytes;
    const uint32_t bar_off = kPair ? kBarOffset : (uint32_t)n_stages * (sch.a_bytes + kBGroupBytes);
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + bar_off);       // used in the leader CTA
    uint64_t* empty_bar = full_bar + kMaxStages;                             // both CTAs
    uint64_t* accg_full = empty_bar + kMaxStages;                            // both CTAs
    uint64_t* accp_full = accg_full + 1;                                     // both CTAs
    uint64_t* accg_free = accp_full + 1;                                     // leader CTA: 16 warps arrive
    uint64_t* accp_free = accg_free + 1;                                     // leader CTA
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(accp_free + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile int* drain_flag = abort_flag + 1;   // never raised: lets the drain wait run to its limit

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = kPair ? ptx::cluster_ctarank() : 0u;          // 0 = leader
    const int G = kPair ? gridDim.x >> 1 : gridDim.x;                   // CTA pairs (or CTAs)
    const int pr = kPair ? blockIdx.x >> 1 : blockIdx.x;                // this pair
    const int n_items = items_of_pair(sch, pr);
    const int ks_g = d.H / kBlockK, ks_p = d.d_l / kBlockK, ks_total = ks_g + ks_p;

    if (threadIdx.x == 0) {
        for (int s = 0; s < n_stages; ++s) { ptx::mbar_init(&full_bar[s], kPair ? 2 : 1); ptx::mbar_init(&empty_bar[s], 1); }
        ptx::mbar_init(accg_full, 1);
        ptx::mbar_init(accp_full, 1);
        ptx::mbar_init(accg_free, kPair ? 16 : 8);
        ptx::mbar_init(accp_free, kPair ? 16 : 8);
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
    const uint32_t tmem_p = tmem_base, tmem_g = tmem_base + 256;

    if (warp == 0) {
        if (ptx::elect_one()) {
            ptx::prefetch_tensormap(&tm_l); ptx::prefetch_tensormap(&tm_x);
            ptx::prefetch_tensormap(&tm_wp); ptx::prefetch_tensormap(&tm_wg);
            int it = 0;            // ring iteration, runs on across items
            int s = 0;             // its stage and phase, kept as counters (no division in the loop)
            uint32_t ph = 0;
            bool ok = true;
            bool l_ready = false;
            for (int n = 0; n < n_items && ok; ++n) {
                const Item w = item_of<kPair>(sch, pr, G, n);
                const int t0 = w.t0 + (int)rank * kTileM;          // this CTA's rows
                const int n_grp = kPair ? w.nt / 128 : w.nt / 64;  // 64-column groups this CTA stages
                const int col0 = (int)rank * (w.nt / 2);           // first of this CTA's columns inside the item
                const int fc = w.f0 + col0;                         // this CTA's first output column
                const int g = d.head_to_q(w.f0 / d.d_h);           // a block never straddles two maps
                // head and column inside it of the (up to two) 64-column groups this CTA stages
                const int wp_head[2] = {fc / d.d_h, (fc + 64) / d.d_h};
                const int wp_col[2] = {fc % d.d_h, (fc + 64) % d.d_h};
                const uint32_t tx = a_tile_bytes + (uint32_t)n_grp * kBGroupBytes;
                for (int ks = 0; ks < ks_total; ++ks, ++it, s = (s + 1 == n_stages) ? 0 : s + 1, ph ^= (s == 0)) {
                    ok = ptx::mbar_wait(&empty_bar[s], ph ^ 1, abort_flag);
                    if (!ok) break;
                    uint8_t* a_s = smem + s * a_stride;
                    uint8_t* b_s = smem + b_base + s * b_stride;
                    if (!kPair) {
                        uint64_t* bar = &full_bar[s];
                        ptx::mbar_arrive_expect_tx(bar, tx);
                        if (ks < ks_g) {
                            ptx::tma_load_3d(a_s, &tm_x, bar, ks * kBlockK, t0, w.b);
                            for (int grp = 0; grp < n_grp; ++grp)
                                ptx::tma_load_2d(b_s + grp * kBGroupBytes, &tm_wg, bar, fc + grp * 64, ks * kBlockK);
                        } else {
                            const int kk = ks - ks_g;
                            if (!l_ready) {
                                ptx::grid_dependency_wait();
                                l_ready = true;
                                if (step_lens != nullptr && blockIdx.x == 0)
                                    for (int sb = 0; sb < step_batch; ++sb) {
                                        const int len = step_lens[sb];
                                        if (len >= 0 && len < step_cap) step_lens[sb] = len + 1;
                                    }
                            }
                            ptx::tma_load_3d(a_s, &tm_l, bar, kk * kBlockK, t0, w.b * d.n_q + g);
                            for (int grp = 0; grp < n_grp; ++grp)
                                ptx::tma_load_3d(b_s + grp * kBGroupBytes, &tm_wp, bar, wp_col[grp], kk * kBlockK,
                                                 wp_head[grp]);
                        }
                        continue;
                    }
                    const uint32_t bar = ptx::map_to_cta(ptx::smem_addr(&full_bar[s]), 0);   // the leader's
                    ptx::mbar_arrive_expect_tx_cluster(bar, tx);
                    if (ks < ks_g) {
                        ptx::tma_load_3d_pair(a_s, &tm_x, bar, ks * kBlockK, t0, w.b);
                        for (int grp = 0; grp < n_grp; ++grp)
                            ptx::tma_load_2d_pair(b_s + grp * kBGroupBytes, &tm_wg, bar, fc + grp * 64, ks * kBlockK);
                    } else {
                        const int kk = ks - ks_g;
                        // L comes from the kernel before this one in the stream; this kernel is
                        // launched with programmatic serialisation, so the gate phase above (X, W_G
                        // only) may already have run while that kernel was draining
                        if (!l_ready) {
                                ptx::grid_dependency_wait();
                                l_ready = true;
                                if (step_lens != nullptr && blockIdx.x == 0)
                                    for (int sb = 0; sb < step_batch; ++sb) {
                                        const int len = step_lens[sb];
                                        if (len >= 0 && len < step_cap) step_lens[sb] = len + 1;
                                    }
                            }
                        ptx::tma_load_3d_pair(a_s, &tm_l, bar, kk * kBlockK, t0, w.b * d.n_q + g);
                        for (int grp = 0; grp < n_grp; ++grp)
                            ptx::tma_load_3d_pair(b_s + grp * kBGroupBytes, &tm_wp, bar, wp_col[grp], kk * kBlockK,
                                                  wp_head[grp]);
                    }
                }
            }
            if (*abort_flag && rank == 0) {   // drain: every armed stage either lands or the wait gives up
                for (int back = 1; back <= n_stages && it - back >= 0; ++back) {
                    const int kq = it - back;
                    ptx::mbar_wait_drain(&full_bar[kq % n_stages], (kq / n_stages) & 1, drain_flag);
                }
            }
        }
    } else if (warp == 1) {
        if (rank == 0 && ptx::elect_one()) {
            int it = 0, s = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int n = 0; n < n_items && ok; ++n) {
                const Item w = item_of<kPair>(sch, pr, G, n);
                const uint32_t idesc = ptx::make_idesc_bf16(kPair ? 2 * kTileM : kTileM, w.nt, 0, 1);   // A K-major, B MN-major
                for (int ks = 0; ks < ks_total; ++ks, ++it, s = (s + 1 == n_stages) ? 0 : s + 1, ph ^= (s == 0)) {
                    // the accumulator about to be overwritten must have been read by both epilogues
                    if (ks == 0) ok = ptx::mbar_wait(accg_free, (n & 1) ^ 1, abort_flag);
                    else if (ks == ks_g) ok = ptx::mbar_wait(accp_free, (n & 1) ^ 1, abort_flag);
                    if (!ok) break;
                    ok = ptx::mbar_wait(&full_bar[s], ph, abort_flag);
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    const uint32_t a_addr = ptx::smem_addr(smem + s * a_stride);
                    const uint32_t b_addr = ptx::smem_addr(smem + b_base + s * b_stride);
                    const uint32_t d_tmem = ks < ks_g ? tmem_g : tmem_p;
                    const bool first = (ks == 0) || (ks == ks_g);
#pragma unroll
                    for (int k4 = 0; k4 < kBlockK / 16; ++k4) {
                        const uint64_t a_desc = ptx::make_smem_desc(a_addr + k4 * 32, 16, 1024);
                        const uint64_t b_desc = ptx::make_smem_desc(b_addr + k4 * 16 * 128, 64 * 128, 1024);
                        if (kPair) ptx::mma_ss_pair(d_tmem, a_desc, b_desc, idesc, (first && k4 == 0) ? 0u : 1u);
                        else ptx::mma_ss(d_tmem, a_desc, b_desc, idesc, (first && k4 == 0) ? 0u : 1u);
                    }
                    if (kPair) {
                        ptx::tc_commit_pair(&empty_bar[s], 3);
                        if (ks == ks_g - 1) ptx::tc_commit_pair(accg_full, 3);
                        if (ks == ks_total - 1) ptx::tc_commit_pair(accp_full, 3);
                    } else {
                        ptx::tc_commit(&empty_bar[s]);
                        if (ks == ks_g - 1) ptx::tc_commit(accg_full);
                        if (ks == ks_total - 1) ptx::tc_commit(accp_full);
                    }
                }
            }
        }
    } else {
        // epilogue: warp w may touch TMEM lanes [32 (w % 4), 32 (w % 4) + 32); the two warps of a
        // quarter take one half of the item's columns each (= one head of a pair)
        const int quarter = warp & 3;
        const int half = (warp - 2) >> 2;
        const int row = quarter * 32 + lane;
        const uint32_t lane_base = ((uint32_t)(quarter * 32) << 16);
        const uint32_t accg_free_leader = ptx::map_to_cta(ptx::smem_addr(accg_free), 0);
        const uint32_t accp_free_leader = ptx::map_to_cta(ptx::smem_addr(accp_free), 0);
        bool ok = true;
        for (int n = 0; n < n_items && ok; ++n) {
            const Item w = item_of<kPair>(sch, pr, G, n);
            const int cols = w.nt / 2;               // this warp's columns: 128, 64 or 32
            const int c0 = half * cols;
            const int t = w.t0 + (int)rank * kTileM + row;
            uint32_t gate[64];                       // sigmoid gates, packed bf16 pairs
            ok = __all_sync(0xffffffffu, ptx::mbar_wait(accg_full, n & 1, abort_flag));
            if (!ok) break;
            ptx::tc_fence_after_sync();
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
                if (ch * 32 < cols) {
                    uint32_t z[32];
                    ptx::tmem_ld32(tmem_g + lane_base + c0 + ch * 32, z);
                    ptx::tmem_wait_ld();
#pragma unroll
                    for (int e = 0; e < 16; ++e)
                        gate[ch * 16 + e] = pack_bf16x2(sigmoid_tanh(__uint_as_float(z[2 * e])),
                                                        sigmoid_tanh(__uint_as_float(z[2 * e + 1])));
                }
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                if (kPair) ptx::mbar_arrive_cluster(accg_free_leader);
                else ptx::mbar_arrive(accg_free);
            }

            ok = __all_sync(0xffffffffu, ptx::mbar_wait(accp_full, n & 1, abort_flag));
            if (!ok) break;
            ptx::tc_fence_after_sync();
            // columns [c0, c0 + cols) of the item = output columns f0 + c0 .. of the token (head after head)
            __nv_bfloat16* o_row = out + ((size_t)w.b * d.N + (t < d.N ? t : 0)) * ((size_t)d.n_h * d.d_h) + w.f0 + c0;
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
                if (ch * 32 < cols) {
                    uint32_t p[32];
                    ptx::tmem_ld32(tmem_p + lane_base + c0 + ch * 32, p);
                    ptx::tmem_wait_ld();
                    uint32_t packed[16];
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        const uint32_t gg = gate[ch * 16 + e];
                        const float g0 = __uint_as_float(gg << 16), g1 = __uint_as_float(gg & 0xffff0000u);
                        packed[e] = pack_bf16x2(__uint_as_float(p[2 * e]) * g0, __uint_as_float(p[2 * e + 1]) * g1);
                    }
                    if (t < d.N) {
#pragma unroll
                        for (int v = 0; v < 2; ++v) {      // 2 x 32 bytes: whole sectors, half as many stores
                            const uint32_t ww[8] = {packed[8 * v], packed[8 * v + 1], packed[8 * v + 2], packed[8 * v + 3],
                                                    packed[8 * v + 4], packed[8 * v + 5], packed[8 * v + 6], packed[8 * v + 7]};
                            ptx::st_global_256(o_row + ch * 32 + v * 16, ww);
                        }
                    }
                }
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                if (kPair) ptx::mbar_arrive_cluster(accp_free_leader);
                else ptx::mbar_arrive(accp_free);
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

int sm_count() {
    static int n = [] {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0)
            v = 148;
        return v;
    }();
    return n;
}

}  // namespace

gta_status_t launch_sm100_decoder(const Dims& d, const void* l_bf16, const void* x, const void* w_p, const void* w_g,
                                  void* out, int32_t* status_word, cudaStream_t stream, int32_t* step_lens,
                                  int step_batch, int step_cap) {
    CUtensorMap tm_l, tm_x, tm_wp, tm_wg;
    const bool solo = d.N <= kTileM;                                    // one row tile: no CTA pairs
    const uint32_t a_rows = solo ? (uint32_t)((d.N + 7) & ~7) : kTileM; // rows of an A tile
    {
        const uint64_t dims[3] = {(uint64_t)d.d_l, (uint64_t)d.N, (uint64_t)d.B * d.n_q};
        const uint32_t box[3] = {kBlockK, a_rows, 1};
        if (!make_bf16_map(&tm_l, l_bf16, 3, dims, box)) return GTA_ERR_CUDA;
    }
    {
        const uint64_t dims[3] = {(uint64_t)d.H, (uint64_t)d.N, (uint64_t)d.B};
        const uint32_t box[3] = {kBlockK, a_rows, 1};
        if (!make_bf16_map(&tm_x, x, 3, dims, box)) return GTA_ERR_CUDA;
    }
    {
        const uint64_t dims[3] = {(uint64_t)d.d_h, (uint64_t)d.d_l, (uint64_t)d.n_h};
        const uint32_t box[3] = {64, kBlockK, 1};
        if (!make_bf16_map(&tm_wp, w_p, 3, dims, box)) return GTA_ERR_CUDA;
    }
    {
        const uint64_t dims[2] = {(uint64_t)d.n_h * d.d_h, (uint64_t)d.H};
        const uint32_t box[2] = {64, kBlockK};
        if (!make_bf16_map(&tm_wg, w_g, 2, dims, box)) return GTA_ERR_CUDA;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kDecThreads);
    cfg.dynamicSmemBytes = kDecSmemTotal;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    if (solo) {
        // half-head items over as many SMs as there are items
        Schedule s;
        s.a_bytes = a_rows * kBlockK * 2;
        s.n_stages = (int)(kSoloRingBytes / (s.a_bytes + kBGroupBytes));
        if (s.n_stages > kMaxStages) s.n_stages = kMaxStages;
        // the MMA reads 16 KB from every A tile: the B tiles behind the last one must cover that
        if ((uint32_t)s.n_stages * kBGroupBytes < kATileBytes) return GTA_ERR_UNSUPPORTED;
        const uint32_t smem_bytes = (uint32_t)s.n_stages * (s.a_bytes + kBGroupBytes) + kBarBytes + 1024;
        cfg.dynamicSmemBytes = smem_bytes;
        s.pair = 0;
        s.n_hp = d.n_h * d.d_h / 64;
        s.RT = 1;
        const long long U = (long long)d.B * s.n_hp;
        if (U > 0x3fffffffLL) return GTA_ERR_UNSUPPORTED;
        if (cudaFuncSetAttribute(sm100_decoder_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem_bytes) != cudaSuccess)
            return GTA_ERR_CUDA;
        const int G = U < sm_count() ? (int)U : sm_count();
        s.q = (int)(U / G);
        s.r = (int)(U % G);
        s.split_tail = 0;
        cfg.gridDim = dim3(G);
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, sm100_decoder_kernel<false>, tm_l, tm_x, tm_wp, tm_wg, d, s, (__nv_bfloat16*)out,
                               status_word, step_lens, step_batch, step_cap) != cudaSuccess)
            return GTA_ERR_CUDA;
        return cudaGetLastError() == cudaSuccess ? GTA_OK : GTA_ERR_CUDA;
    }
    Schedule s;
    s.n_stages = kDecStages;
    s.a_bytes = kATileBytes;
    const int map_cols = (d.n_h / d.n_q) * d.d_h;      // output columns of one attention map
    if (map_cols % 128 != 0) return GTA_ERR_UNSUPPORTED;
    s.pair = map_cols % 256 == 0 ? 1 : 0;
    s.n_hp = d.n_h * d.d_h / (s.pair ? 256 : 128);
    s.RT = (d.N + 2 * kTileM - 1) / (2 * kTileM);
    long long U = (long long)d.B * s.RT * s.n_hp;
    if (U > 0x3fffffffLL) return GTA_ERR_UNSUPPORTED;
    if (cudaFuncSetAttribute(sm100_decoder_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)kDecSmemTotal) != cudaSuccess)
        return GTA_ERR_CUDA;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;   // the occupancy query below takes the cluster attribute only
    // A persistent grid must be resident at once: as many pairs as the device can hold (not every
    // pair of SMs can host a cluster), asked once per device.
    static thread_local int cached_dev = -1, cached_pairs = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return GTA_ERR_CUDA;
    if (dev != cached_dev) {
        cfg.gridDim = dim3(2 * (sm_count() / 2));
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, sm100_decoder_kernel<true>, &cfg) != cudaSuccess || n < 1) return GTA_ERR_CUDA;
        cached_dev = dev;
        cached_pairs = n;
    }
    const int pairs = cached_pairs;
    if (s.pair && 2 * U <= pairs) {   // few units: 128-column blocks keep twice as many SMs busy
        s.pair = 0;
        s.n_hp *= 2;
        U *= 2;
    }
    const int G = U < pairs ? (int)U : pairs;
    s.q = (int)(U / G);
    s.r = (int)(U % G);
    s.split_tail = (s.pair && 2 * s.r <= G) ? 1 : 0;
    cfg.gridDim = dim3(2 * G);
    cfg.numAttrs = 2;
    if (cudaLaunchKernelEx(&cfg, sm100_decoder_kernel<true>, tm_l, tm_x, tm_wp, tm_wg, d, s, (__nv_bfloat16*)out,
                           status_word, step_lens, step_batch, step_cap) != cudaSuccess)
        return GTA_ERR_CUDA;
    return cudaGetLastError() == cudaSuccess ? GTA_OK : GTA_ERR_CUDA;
}

}  // namespace gta
