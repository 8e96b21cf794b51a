// tcgen05 / TMA (sm_100a) prefill path for bf16, d_h = 128.
//
//   sm100_decoder_kernel : out_i = (L_{q(i)} W_P,i) (.) sigmoid(X W_G,i)   (Sec. 3.3, reformulated
//       equation).  Two accumulators live in tensor memory side by side: acc_P (K loop over d_l)
//       and acc_G (K loop over H); the epilogue multiplies them through the sigmoid.  One CTA =
//       128 token rows x (1 or 2 heads); warp 0 issues TMA loads, warp 1 issues tcgen05.mma,
//       warps 2..5 run the epilogue out of tensor memory.
#include "gta_sm100.cuh"

#include <cuda.h>

#include "sm100_ptx.cuh"

namespace gta {

// --------------------------------------------------------------------------- host: tensor maps
namespace {

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// bf16 tensor, `rank` dims (innermost first), 128-byte swizzle, zero fill outside the tensor.
bool make_map(CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint32_t* box) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t gdim[5], gstride[5];
    cuuint32_t bx[5], estr[5];
    uint64_t stride = 2;
    for (int i = 0; i < rank; ++i) {
        gdim[i] = dims[i];
        bx[i] = box[i];
        estr[i] = 1;
        stride *= dims[i];
        if (i < rank - 1) gstride[i] = stride;   // byte stride of dimension i+1
    }
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gdim, gstride, bx, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// --------------------------------------------------------------------------- decoder + gate kernel
constexpr int kDecStages = 4;
constexpr int kDecThreads = 192;
constexpr int kTileM = 128;        // token rows per CTA
constexpr int kBlockK = 64;        // K elements per pipeline stage (one 128-byte swizzle row)
constexpr uint32_t kATileBytes = kTileM * kBlockK * 2;   // 16 KB
constexpr uint32_t kBGroupBytes = kBlockK * 64 * 2;      // 64 K-rows x 64 columns = 8 KB

template <int NT>
struct DecSmem {
    static constexpr uint32_t kBTileBytes = (NT / 64) * kBGroupBytes;
    static constexpr uint32_t kStageBytes = kATileBytes + kBTileBytes;
    static constexpr uint32_t kBarOffset = kDecStages * kStageBytes;
    static constexpr uint32_t kTotal = kBarOffset + 256 + 1024;   // barriers + alignment slack
};

__device__ __forceinline__ float fast_sigmoid(float z) { return __fdividef(1.f, 1.f + __expf(-z)); }

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

template <int NT>
__global__ void __launch_bounds__(kDecThreads, 1)
sm100_decoder_kernel(const __grid_constant__ CUtensorMap tm_l, const __grid_constant__ CUtensorMap tm_x,
                     const __grid_constant__ CUtensorMap tm_wp, const __grid_constant__ CUtensorMap tm_wg,
                     Dims d, __nv_bfloat16* __restrict__ out, int32_t* status_word) {
    using L = DecSmem<NT>;
    constexpr int HPC = NT / 128;   // heads per CTA
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + L::kBarOffset);
    uint64_t* empty_bar = full_bar + kDecStages;
    uint64_t* acc_bar = empty_bar + kDecStages;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_bar + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile int* drain_flag = abort_flag + 1;   // never raised: lets the drain wait run to its limit

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int i0 = blockIdx.x * HPC;            // first head of this CTA
    const int t0 = blockIdx.y * kTileM;         // first token row
    const int b = blockIdx.z;
    const int g = d.head_to_q(i0);
    const int ks_p = d.d_l / kBlockK, ks_total = ks_p + d.H / kBlockK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kDecStages; ++s) { ptx::mbar_init(&full_bar[s], 1); ptx::mbar_init(&empty_bar[s], 1); }
        ptx::mbar_init(acc_bar, 1);
        *abort_flag = 0;
        *drain_flag = 0;
        ptx::fence_mbar_init();
    }
    if (warp == 1) ptx::tmem_alloc(tmem_slot, 2 * NT);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (ptx::elect_one()) {
            ptx::prefetch_tensormap(&tm_l); ptx::prefetch_tensormap(&tm_x);
            ptx::prefetch_tensormap(&tm_wp); ptx::prefetch_tensormap(&tm_wg);
            int ks = 0;
            for (; ks < ks_total; ++ks) {
                const int s = ks % kDecStages;
                const uint32_t ph = (ks / kDecStages) & 1;
                if (!ptx::mbar_wait(&empty_bar[s], ph ^ 1, abort_flag)) break;
                uint8_t* a_s = smem + s * L::kStageBytes;
                uint8_t* b_s = a_s + kATileBytes;
                ptx::mbar_arrive_expect_tx(&full_bar[s], L::kStageBytes);
                if (ks < ks_p) {
                    ptx::tma_load_3d(a_s, &tm_l, &full_bar[s], ks * kBlockK, t0, b * d.n_q + g);
#pragma unroll
                    for (int grp = 0; grp < NT / 64; ++grp)
                        ptx::tma_load_3d(b_s + grp * kBGroupBytes, &tm_wp, &full_bar[s], (grp & 1) * 64, ks * kBlockK,
                                         i0 + (grp >> 1));
                } else {
                    const int kk = ks - ks_p;
                    ptx::tma_load_3d(a_s, &tm_x, &full_bar[s], kk * kBlockK, t0, b);
#pragma unroll
                    for (int grp = 0; grp < NT / 64; ++grp)
                        ptx::tma_load_2d(b_s + grp * kBGroupBytes, &tm_wg, &full_bar[s], i0 * 128 + grp * 64,
                                         kk * kBlockK);
                }
            }
            if (*abort_flag) {   // drain: every armed stage either lands or the wait gives up
                for (int back = 1; back <= kDecStages && ks - back >= 0; ++back) {
                    const int kq = ks - back;
                    ptx::mbar_wait(&full_bar[kq % kDecStages], (kq / kDecStages) & 1, drain_flag);
                }
            }
        }
    } else if (warp == 1) {
        if (ptx::elect_one()) {
            constexpr uint32_t idesc = ptx::make_idesc_bf16(kTileM, NT, 0, 1);   // A K-major, B MN-major
            for (int ks = 0; ks < ks_total; ++ks) {
                const int s = ks % kDecStages;
                const uint32_t ph = (ks / kDecStages) & 1;
                if (!ptx::mbar_wait(&full_bar[s], ph, abort_flag)) break;
                ptx::tc_fence_after_sync();
                const uint32_t a_addr = ptx::smem_addr(smem + s * L::kStageBytes);
                const uint32_t b_addr = a_addr + kATileBytes;
                const uint32_t d_tmem = tmem_base + (ks < ks_p ? 0 : NT);
                const bool first = (ks == 0) || (ks == ks_p);
#pragma unroll
                for (int k4 = 0; k4 < kBlockK / 16; ++k4) {
                    const uint64_t a_desc = ptx::make_smem_desc(a_addr + k4 * 32, 16, 1024);
                    const uint64_t b_desc = ptx::make_smem_desc(b_addr + k4 * 16 * 128, 64 * 128, 1024);
                    ptx::mma_ss(d_tmem, a_desc, b_desc, idesc, (first && k4 == 0) ? 0u : 1u);
                }
                ptx::tc_commit(&empty_bar[s]);
            }
            ptx::tc_commit(acc_bar);
        }
    } else {
        // epilogue: warp w may touch TMEM lanes [32 (w % 4), 32 (w % 4) + 32)
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const int t = t0 + row;
        if (ptx::mbar_wait(acc_bar, 0, abort_flag)) {
            ptx::tc_fence_after_sync();
            const uint32_t lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16);
            __nv_bfloat16* o_row = out + (((size_t)b * d.N + (t < d.N ? t : 0)) * d.n_h + i0) * 128;
#pragma unroll 1
            for (int chunk = 0; chunk < NT / 32; ++chunk) {
                uint32_t p[32], z[32];
                ptx::tmem_ld32(lane_base + chunk * 32, p);
                ptx::tmem_ld32(lane_base + NT + chunk * 32, z);
                ptx::tmem_wait_ld();
                uint32_t packed[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                    const float y0 = __uint_as_float(p[2 * e]) * fast_sigmoid(__uint_as_float(z[2 * e]));
                    const float y1 = __uint_as_float(p[2 * e + 1]) * fast_sigmoid(__uint_as_float(z[2 * e + 1]));
                    packed[e] = pack_bf16x2(y0, y1);
                }
                if (t < d.N) {
                    uint4* dst = reinterpret_cast<uint4*>(o_row + chunk * 32);
#pragma unroll
                    for (int v = 0; v < 4; ++v)
                        dst[v] = make_uint4(packed[4 * v], packed[4 * v + 1], packed[4 * v + 2], packed[4 * v + 3]);
                }
            }
        }
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) ptx::tmem_dealloc(tmem_base, 2 * NT);
    if (threadIdx.x == 0 && *abort_flag) raise_status(status_word, GTA_ERR_TIMEOUT);
}

// --------------------------------------------------------------------------- host side
bool sm100_prefill_supported(const Dims& d, int dtype) {
    return dtype == GTA_BF16 && d.d_h == 128 && d.d_l % 256 == 0 && d.d_l <= 1024 && d.H % 64 == 0 && d.N >= 1;
}

template <int NT>
static gta_status_t launch_decoder(const Dims& d, const CUtensorMap& tm_l, const CUtensorMap& tm_x,
                                   const CUtensorMap& tm_wp, const CUtensorMap& tm_wg, void* out,
                                   int32_t* status_word, cudaStream_t stream) {
    auto kern = sm100_decoder_kernel<NT>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DecSmem<NT>::kTotal) != cudaSuccess)
        return GTA_ERR_CUDA;
    dim3 grid(d.n_h / (NT / 128), (d.N + kTileM - 1) / kTileM, d.B);
    kern<<<grid, kDecThreads, DecSmem<NT>::kTotal, stream>>>(tm_l, tm_x, tm_wp, tm_wg, d, (__nv_bfloat16*)out, status_word);
    return cudaGetLastError() == cudaSuccess ? GTA_OK : GTA_ERR_CUDA;
}

gta_status_t launch_sm100_prefill(const Dims& d, const void* q, const void* k, const void* c, const void* x,
                                  const void* w_p, const void* w_g, void* out, void* workspace,
                                  int32_t* status_word, cudaStream_t stream, int stages, int* launches) {
    if (stages & 1) {
        if (launch_generic_attention_bf16(d, q, k, c, workspace, stream, launches) != cudaSuccess) return GTA_ERR_CUDA;
    }
    if (stages & 2) {
        CUtensorMap tm_l, tm_x, tm_wp, tm_wg;
        const int heads_per_map = d.n_h / d.n_q;
        const bool pair = heads_per_map % 2 == 0;
        {
            const uint64_t dims[3] = {(uint64_t)d.d_l, (uint64_t)d.N, (uint64_t)d.B * d.n_q};
            const uint32_t box[3] = {kBlockK, kTileM, 1};
            if (!make_map(&tm_l, workspace, 3, dims, box)) return GTA_ERR_CUDA;
        }
        {
            const uint64_t dims[3] = {(uint64_t)d.H, (uint64_t)d.N, (uint64_t)d.B};
            const uint32_t box[3] = {kBlockK, kTileM, 1};
            if (!make_map(&tm_x, x, 3, dims, box)) return GTA_ERR_CUDA;
        }
        {
            const uint64_t dims[3] = {(uint64_t)d.d_h, (uint64_t)d.d_l, (uint64_t)d.n_h};
            const uint32_t box[3] = {64, kBlockK, 1};
            if (!make_map(&tm_wp, w_p, 3, dims, box)) return GTA_ERR_CUDA;
        }
        {
            const uint64_t dims[2] = {(uint64_t)d.n_h * d.d_h, (uint64_t)d.H};
            const uint32_t box[2] = {64, kBlockK};
            if (!make_map(&tm_wg, w_g, 2, dims, box)) return GTA_ERR_CUDA;
        }
        gta_status_t st = pair ? launch_decoder<256>(d, tm_l, tm_x, tm_wp, tm_wg, out, status_word, stream)
                               : launch_decoder<128>(d, tm_l, tm_x, tm_wp, tm_wg, out, status_word, stream);
        if (st != GTA_OK) return st;
        *launches += 1;
    }
    return GTA_OK;
}

}  // namespace gta
