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
// One CTA = one 128-row query tile of one attention map x one 256-column slice of the latent
// (the 128 x d_l fp32 output does not fit the 512 TMEM columns next to the score tiles, so d_l is
// cut in slices of 256 and each slice CTA recomputes the scores).  Per 128-key tile j:
//   S_j = Q K_j^T            tcgen05.mma, smem x smem -> TMEM (two S buffers, ping-pong)
//   P_j = exp2(S_j c - m)    128 softmax threads, one row each; P_j (bf16) overwrites S_j in TMEM
//   O  += P_j C_j            tcgen05.mma, TMEM x smem (C is the MN-major B operand) -> TMEM
// The running maximum is only raised when it grows by more than 2^8 (the accumulators stay in
// range and O needs rescaling on few tiles); O is divided by the row sum at the end and written
// as bf16 to L[B, n_q, N, d_l].
constexpr int kAttnThreads = 192;
constexpr int kKeyTile = 128;
constexpr int kSlice = 256;
constexpr uint32_t kQBytes = 128 * 128 * 2;            // 32 KB
constexpr uint32_t kKStageBytes = kKeyTile * 128 * 2;  // 32 KB
constexpr uint32_t kCStageBytes = kKeyTile * kSlice * 2;  // 64 KB
constexpr uint32_t kAttnKOff = kQBytes;
constexpr uint32_t kAttnCOff = kAttnKOff + 2 * kKStageBytes;
constexpr uint32_t kAttnBarOff = kAttnCOff + 2 * kCStageBytes;
constexpr uint32_t kAttnSmemTotal = kAttnBarOff + 256 + 1024;

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__global__ void __launch_bounds__(kAttnThreads, 1)
sm100_attention_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                       const __grid_constant__ CUtensorMap tm_c, Dims d, __nv_bfloat16* __restrict__ o_lat,
                       int32_t* status_word) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kAttnBarOff);
    uint64_t* q_full = bars;            // 1
    uint64_t* k_full = bars + 1;        // 2
    uint64_t* k_empty = bars + 3;       // 2
    uint64_t* c_full = bars + 5;        // 2
    uint64_t* c_empty = bars + 7;       // 2
    uint64_t* s_full = bars + 9;        // 2
    uint64_t* p_full = bars + 11;       // 2
    uint64_t* o_done = bars + 13;       // 1
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 14);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile int* drain_flag = abort_flag + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // heaviest (latest) query tiles first
    const int n_slices = d.d_l / kSlice;
    const int n_qt = (d.N + 127) / 128;
    int bid = blockIdx.x;
    const int slice = bid % n_slices; bid /= n_slices;
    const int g = bid % d.n_q; bid /= d.n_q;
    const int b = bid % d.B; bid /= d.B;
    const int qi = n_qt - 1 - bid;
    const int q0 = qi * 128;
    const int kg = d.q_to_k(g), cg = d.q_to_c(g);
    const int n_tiles = d.causal ? qi + 1 : n_qt;

    if (threadIdx.x == 0) {
        ptx::mbar_init(q_full, 1);
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(&k_full[s], 1); ptx::mbar_init(&k_empty[s], 1);
            ptx::mbar_init(&c_full[s], 1); ptx::mbar_init(&c_empty[s], 1);
            ptx::mbar_init(&s_full[s], 1); ptx::mbar_init(&p_full[s], 128);
        }
        ptx::mbar_init(o_done, 1);
        *abort_flag = 0;
        *drain_flag = 0;
        ptx::fence_mbar_init();
    }
    if (warp == 1) ptx::tmem_alloc(tmem_slot, 512);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_o = tmem_base + 256;

    if (warp == 0) {
        if (ptx::elect_one()) {
            ptx::prefetch_tensormap(&tm_q); ptx::prefetch_tensormap(&tm_k); ptx::prefetch_tensormap(&tm_c);
            ptx::mbar_arrive_expect_tx(q_full, kQBytes);
            ptx::tma_load_3d(smem, &tm_q, q_full, 0, q0, b * d.n_q + g);
            ptx::tma_load_3d(smem + 16384, &tm_q, q_full, 64, q0, b * d.n_q + g);
            int j = 0;
            bool ok = true;
            for (; j < n_tiles && ok; ++j) {
                const int s = j & 1;
                const uint32_t ph = (j >> 1) & 1;
                ok = ptx::mbar_wait(&k_empty[s], ph ^ 1, abort_flag);
                if (!ok) break;
                uint8_t* k_s = smem + kAttnKOff + s * kKStageBytes;
                ptx::mbar_arrive_expect_tx(&k_full[s], kKStageBytes);
                ptx::tma_load_3d(k_s, &tm_k, &k_full[s], 0, j * kKeyTile, b * d.n_k + kg);
                ptx::tma_load_3d(k_s + 16384, &tm_k, &k_full[s], 64, j * kKeyTile, b * d.n_k + kg);
                ok = ptx::mbar_wait(&c_empty[s], ph ^ 1, abort_flag);
                if (!ok) { ++j; break; }
                uint8_t* c_s = smem + kAttnCOff + s * kCStageBytes;
                ptx::mbar_arrive_expect_tx(&c_full[s], kCStageBytes);
#pragma unroll
                for (int grp = 0; grp < kSlice / 64; ++grp)
                    ptx::tma_load_3d(c_s + grp * 16384, &tm_c, &c_full[s], slice * kSlice + grp * 64, j * kKeyTile,
                                     b * d.n_c + cg);
            }
            if (*abort_flag) {   // drain what was armed (bounded), so no copy lands after exit
                ptx::mbar_wait(q_full, 0, drain_flag);
                for (int back = 1; back <= 2 && j - back >= 0; ++back) {
                    const int jq = j - back;
                    ptx::mbar_wait(&k_full[jq & 1], (jq >> 1) & 1, drain_flag);
                    ptx::mbar_wait(&c_full[jq & 1], (jq >> 1) & 1, drain_flag);
                }
            }
        }
    } else if (warp == 1) {
        if (ptx::elect_one()) {
            constexpr uint32_t idesc_qk = ptx::make_idesc_bf16(128, kKeyTile, 0, 0);   // both K-major
            constexpr uint32_t idesc_pv = ptx::make_idesc_bf16(128, kSlice, 0, 1);     // B = C, MN-major
            const uint32_t q_addr = ptx::smem_addr(smem);
            auto issue_qk = [&](int j) {
                const uint32_t k_addr = ptx::smem_addr(smem + kAttnKOff + (j & 1) * kKStageBytes);
                const uint32_t s_tmem = tmem_base + (j & 1) * 128;
#pragma unroll
                for (int k8 = 0; k8 < 8; ++k8) {
                    const uint32_t off = (k8 >> 2) * 16384 + (k8 & 3) * 32;
                    ptx::mma_ss(s_tmem, ptx::make_smem_desc(q_addr + off, 16, 1024),
                                ptx::make_smem_desc(k_addr + off, 16, 1024), idesc_qk, k8 ? 1u : 0u);
                }
                ptx::tc_commit(&s_full[j & 1]);
                ptx::tc_commit(&k_empty[j & 1]);
            };
            bool ok = ptx::mbar_wait(q_full, 0, abort_flag) && ptx::mbar_wait(&k_full[0], 0, abort_flag);
            if (ok) {
                ptx::tc_fence_after_sync();
                issue_qk(0);
            }
            for (int j = 0; j < n_tiles && ok; ++j) {
                if (j + 1 < n_tiles) {
                    ok = ptx::mbar_wait(&k_full[(j + 1) & 1], ((j + 1) >> 1) & 1, abort_flag);
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    issue_qk(j + 1);
                }
                ok = ptx::mbar_wait(&p_full[j & 1], (j >> 1) & 1, abort_flag) &&
                     ptx::mbar_wait(&c_full[j & 1], (j >> 1) & 1, abort_flag);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint32_t c_addr = ptx::smem_addr(smem + kAttnCOff + (j & 1) * kCStageBytes);
                const uint32_t p_tmem = tmem_base + (j & 1) * 128;
#pragma unroll
                for (int k8 = 0; k8 < 8; ++k8)
                    ptx::mma_ts(tmem_o, p_tmem + k8 * 8, ptx::make_smem_desc(c_addr + k8 * 2048, 16384, 1024),
                                idesc_pv, (j > 0 || k8 > 0) ? 1u : 0u);
                ptx::tc_commit(o_done);
                ptx::tc_commit(&c_empty[j & 1]);
            }
        }
    } else {
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const int t = q0 + row;
        const uint32_t lane_base = ((uint32_t)(quarter * 32) << 16);
        const float c_scale = d.scale * 1.4426950408889634f;
        float m = -INFINITY, l = 0.f;
        bool ok = true;
        for (int j = 0; j < n_tiles && ok; ++j) {
            ok = __all_sync(0xffffffffu, ptx::mbar_wait(&s_full[j & 1], (j >> 1) & 1, abort_flag));
            if (!ok) break;   // warp-uniform: the TMEM instructions below are warp-collective
            ptx::tc_fence_after_sync();
            const uint32_t s_tmem = tmem_base + lane_base + (j & 1) * 128;
            float sv[128];
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
                uint32_t r[32];
                ptx::tmem_ld32(s_tmem + ch * 32, r);
                ptx::tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; ++e) sv[ch * 32 + e] = __uint_as_float(r[e]) * c_scale;
            }
            // mask: keys past the sequence end, and (causal) keys after the query, on boundary tiles
            const int key0 = j * kKeyTile;
            const int last_key = d.causal ? min(t, d.N - 1) : d.N - 1;
            if (key0 + kKeyTile - 1 > last_key) {
#pragma unroll
                for (int e = 0; e < 128; ++e)
                    if (key0 + e > last_key) sv[e] = -INFINITY;
            }
            float m_tile = sv[0];
#pragma unroll
            for (int e = 1; e < 128; ++e) m_tile = fmaxf(m_tile, sv[e]);
            float alpha = 1.f;
            bool raise = m_tile > m + 8.f;     // also true on the first tile (m = -inf)
            if (raise) {
                alpha = fast_exp2(m - m_tile);
                m = m_tile;
            }
            const float neg_m = (m == -INFINITY) ? 0.f : -m;   // a fully masked row keeps p = 0
            float sum = 0.f;
            uint32_t packed[64];
#pragma unroll
            for (int e = 0; e < 64; ++e) {
                const float p0 = fast_exp2(sv[2 * e] + neg_m);
                const float p1 = fast_exp2(sv[2 * e + 1] + neg_m);
                sum += p0 + p1;
                packed[e] = pack_bf16x2(p0, p1);
            }
            l = l * alpha + sum;
            // P_j (bf16 pairs) over the first 64 columns of S_j
            {
                uint32_t (*pk)[32] = reinterpret_cast<uint32_t (*)[32]>(packed);
                ptx::tmem_st32(s_tmem, pk[0]);
                ptx::tmem_st32(s_tmem + 32, pk[1]);
            }
            if (j > 0 && __any_sync(0xffffffffu, raise)) {
                ok = __all_sync(0xffffffffu, ptx::mbar_wait(o_done, (j - 1) & 1, abort_flag));
                if (!ok) break;
                ptx::tc_fence_after_sync();
#pragma unroll 1
                for (int ch = 0; ch < kSlice / 32; ++ch) {
                    uint32_t r[32];
                    ptx::tmem_ld32(tmem_o + lane_base + ch * 32, r);
                    ptx::tmem_wait_ld();
#pragma unroll
                    for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
                    ptx::tmem_st32(tmem_o + lane_base + ch * 32, r);
                }
            }
            ptx::tmem_wait_st();
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive(&p_full[j & 1]);
        }
        if (ok) ok = __all_sync(0xffffffffu, ptx::mbar_wait(o_done, (n_tiles - 1) & 1, abort_flag));
        if (ok) {
            ptx::tc_fence_after_sync();
            const float inv_l = 1.f / l;
            __nv_bfloat16* o_row = o_lat + (((size_t)b * d.n_q + g) * d.N + (t < d.N ? t : 0)) * d.d_l + slice * kSlice;
#pragma unroll 1
            for (int ch = 0; ch < kSlice / 32; ++ch) {
                uint32_t r[32];
                ptx::tmem_ld32(tmem_o + lane_base + ch * 32, r);
                ptx::tmem_wait_ld();
                if (t < d.N) {
                    uint4* dst = reinterpret_cast<uint4*>(o_row + ch * 32);
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        uint32_t w[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            w[e] = pack_bf16x2(__uint_as_float(r[8 * v + 2 * e]) * inv_l,
                                               __uint_as_float(r[8 * v + 2 * e + 1]) * inv_l);
                        dst[v] = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            }
        }
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) ptx::tmem_dealloc(tmem_base, 512);
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
        const uint32_t box[3] = {64, 128, 1};
        const uint64_t dq[3] = {(uint64_t)d.d_h, (uint64_t)d.N, (uint64_t)d.B * d.n_q};
        const uint64_t dk[3] = {(uint64_t)d.d_h, (uint64_t)d.N, (uint64_t)d.B * d.n_k};
        const uint64_t dc[3] = {(uint64_t)d.d_l, (uint64_t)d.N, (uint64_t)d.B * d.n_c};
        if (!make_bf16_map(&tm_q, q, 3, dq, box) || !make_bf16_map(&tm_k, k, 3, dk, box) || !make_bf16_map(&tm_c, c, 3, dc, box))
            return GTA_ERR_CUDA;
        if (cudaFuncSetAttribute(sm100_attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kAttnSmemTotal) != cudaSuccess)
            return GTA_ERR_CUDA;
        const int n_qt = (d.N + 127) / 128;
        const long long n_cta = (long long)n_qt * (d.d_l / kSlice) * d.n_q * d.B;
        if (n_cta > 0x7fffffffLL) return GTA_ERR_UNSUPPORTED;
        sm100_attention_kernel<<<(unsigned)n_cta, kAttnThreads, kAttnSmemTotal, stream>>>(
            tm_q, tm_k, tm_c, d, (__nv_bfloat16*)workspace, status_word);
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
