// C-ABI entry points: argument validation and dispatch to the kernel launchers.
#include <math.h>

#include "gta_common.cuh"
#include "gta_sm100.cuh"

namespace {

thread_local int g_last_launches = 0;

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

// Is the current device a Blackwell data-centre part (compute capability 10.x)?
gta_status_t check_device() {
    static thread_local int cached_dev = -1;
    static thread_local int cached_major = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return GTA_ERR_CUDA;
    if (dev != cached_dev) {
        int major = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
            return GTA_ERR_CUDA;
        cached_dev = dev;
        cached_major = major;
    }
    return cached_major == 10 ? GTA_OK : GTA_ERR_UNSUPPORTED;
}

// Shape checks common to all entry points.  `need_seq`: prefill uses shape->seq.
gta_status_t check_shape(const gta_shape_t* s, bool need_seq, gta::Dims* d) {
    if (!s) return GTA_ERR_INVALID_ARG;
    if (s->batch < 0 || (need_seq && s->seq < 0) || s->d_model < 1 || s->n_heads < 1 || s->n_q_groups < 1 ||
        s->n_k_groups < 1 || s->n_c_groups < 1 || s->head_dim < 1 || s->latent_dim < 1)
        return GTA_ERR_INVALID_ARG;
    if (s->n_heads % s->n_q_groups || s->n_q_groups % s->n_k_groups || s->n_q_groups % s->n_c_groups)
        return GTA_ERR_INVALID_ARG;
    if (s->dtype != GTA_F32 && s->dtype != GTA_BF16) return GTA_ERR_INVALID_ARG;
    if (s->causal != 0 && s->causal != 1) return GTA_ERR_INVALID_ARG;
    if (!(s->softmax_scale >= 0.f) || isinf(s->softmax_scale)) return GTA_ERR_INVALID_ARG;
    // rows are moved as 16-byte vectors
    if (s->head_dim % 8 || s->latent_dim % 8 || s->d_model % 8) return GTA_ERR_UNSUPPORTED;
    if (s->head_dim > 256 || s->batch > 65535 || s->n_q_groups > 65535 || s->n_heads > 65535)
        return GTA_ERR_UNSUPPORTED;
    d->B = s->batch; d->N = need_seq ? s->seq : 0; d->H = s->d_model; d->n_h = s->n_heads;
    d->n_q = s->n_q_groups; d->n_k = s->n_k_groups; d->n_c = s->n_c_groups;
    d->d_h = s->head_dim; d->d_l = s->latent_dim; d->causal = s->causal;
    d->scale = s->softmax_scale > 0.f ? s->softmax_scale : 1.0f / sqrtf((float)s->head_dim);
    d->Nk = d->N;
    d->S = d->N;
    return GTA_OK;
}

size_t elem_size(int dtype) { return dtype == GTA_F32 ? 4 : 2; }

}  // namespace

static gta_status_t prefill_impl(const gta_shape_t* shape, int32_t kv_len, int32_t kv_cap, const void* q,
                                 const void* k, const void* c, const void* x, const void* w_p, const void* w_g,
                                 void* out, void* workspace, size_t workspace_bytes, int32_t* status_word,
                                 void* cuda_stream, int32_t stages, const gta::PageMap& pm);
static gta_status_t decode_impl(const gta_shape_t* shape, const void* q, const void* k_cache, const void* c_cache,
                                const int32_t* seq_lens, int32_t S_cap, const void* x_t, const void* w_p,
                                const void* w_g, void* out, void* workspace, size_t workspace_bytes,
                                int32_t* status_word, void* cuda_stream, int32_t stages, const gta::PageMap& pm);
static gta_status_t append_impl(const gta_shape_t* shape, void* k_cache, void* c_cache, int32_t S_cap,
                                const void* k_new, const void* c_new, int32_t n_new, int32_t* seq_lens,
                                int32_t* status_word, void* cuda_stream, const gta::PageMap& pm);

// A block table is usable when it is there, 4-byte aligned, and the pool geometry is positive.
static bool page_args_ok(const int32_t* block_table, int32_t page_size, int32_t n_pages, int32_t max_pages) {
    return block_table && aligned(block_table, 4) && page_size > 0 && n_pages > 0 && max_pages > 0 &&
           (long long)page_size * max_pages <= INT32_MAX;
}

static gta::PageMap page_map(const int32_t* block_table, int32_t page_size, int32_t n_pages, int32_t max_pages) {
    gta::PageMap pm;
    pm.table = block_table;
    pm.page_size = page_size;
    pm.max_pages = max_pages;
    pm.n_pages = n_pages;
    return pm;
}

extern "C" {

const char* gta_status_string(gta_status_t status) {
    switch (status) {
        case GTA_OK: return "ok";
        case GTA_ERR_INVALID_ARG: return "invalid argument";
        case GTA_ERR_UNSUPPORTED: return "unsupported shape, dtype or device";
        case GTA_ERR_WORKSPACE: return "workspace missing or too small";
        case GTA_ERR_CUDA: return "CUDA call failed";
        case GTA_ERR_CACHE_FULL: return "cache full";
        case GTA_ERR_TIMEOUT: return "bounded device wait ran out";
        case GTA_ERR_STATIC_SCRATCH: return "problem exceeds the built-in scratch array of gta_decode_static";
        case GTA_ERR_BAD_PAGE: return "block-table entry outside the page pool";
    }
    return "unknown status";
}

int gta_version(void) { return 100; }

int gta_last_launch_count(void) { return g_last_launches; }

gta_status_t gta_debug_attention_wait(uint64_t limit_ns, int32_t withhold_first_arrive) {
    gta_status_t st = check_device();
    if (st != GTA_OK) return st;
    return gta::sm100_attention_debug_wait(limit_ns, withhold_first_arrive);
}

gta_status_t gta_debug_decode_wait(uint64_t limit_ns, int32_t withhold_first_arrive) {
    gta_status_t st = check_device();
    if (st != GTA_OK) return st;
    st = gta::decode_tc_debug_wait(limit_ns, withhold_first_arrive);
    if (st != GTA_OK) return st;
    return gta::decode_fp8_tc_debug_wait(limit_ns, withhold_first_arrive);
}

int gta_prefill_path(const gta_shape_t* shape) {
    gta::Dims d;
    if (check_shape(shape, true, &d) != GTA_OK) return 0;
    if (gta::sm100_prefill_supported(d, shape->dtype)) return 2;
    if (d.d_l > 1024) return 0;
    return 1;
}

size_t gta_prefill_workspace_bytes(const gta_shape_t* shape) {
    gta::Dims d;
    if (check_shape(shape, true, &d) != GTA_OK) return 0;
    // normalised latent attention output L[B, n_q, N, d_l]: fp32 on the plain-ALU path, bf16 on
    // the tensor-core path; sized for the larger so either path may run.
    size_t bytes = (size_t)d.B * d.n_q * d.N * d.d_l * sizeof(float);
    return bytes < 256 ? 256 : ((bytes + 255) & ~(size_t)255);
}

gta_status_t gta_prefill(const gta_shape_t* shape, const void* q, const void* k, const void* c,
                         const void* x, const void* w_p, const void* w_g, void* out, void* workspace,
                         size_t workspace_bytes, int32_t* status_word, void* cuda_stream) {
    return gta_prefill_stages(shape, q, k, c, x, w_p, w_g, out, workspace, workspace_bytes, status_word,
                              cuda_stream, 3);
}

gta_status_t gta_prefill_stages(const gta_shape_t* shape, const void* q, const void* k, const void* c,
                                const void* x, const void* w_p, const void* w_g, void* out, void* workspace,
                                size_t workspace_bytes, int32_t* status_word, void* cuda_stream,
                                int32_t stages) {
    if (!shape) return GTA_ERR_INVALID_ARG;
    return prefill_impl(shape, shape->seq, shape->seq, q, k, c, x, w_p, w_g, out, workspace, workspace_bytes,
                        status_word, cuda_stream, stages, gta::PageMap());
}

gta_status_t gta_prefill_chunk(const gta_shape_t* shape, int32_t kv_len, int32_t kv_cap, const void* q,
                               const void* k, const void* c, const void* x, const void* w_p, const void* w_g,
                               void* out, void* workspace, size_t workspace_bytes, int32_t* status_word,
                               void* cuda_stream) {
    if (!shape) return GTA_ERR_INVALID_ARG;
    if (kv_len < shape->seq || kv_cap < kv_len) return GTA_ERR_INVALID_ARG;
    return prefill_impl(shape, kv_len, kv_cap, q, k, c, x, w_p, w_g, out, workspace, workspace_bytes, status_word,
                        cuda_stream, 3, gta::PageMap());
}

gta_status_t gta_prefill_chunk_paged(const gta_shape_t* shape, int32_t kv_len, const void* q, const void* k_pool,
                                     const void* c_pool, const int32_t* block_table, int32_t page_size,
                                     int32_t n_pages, int32_t max_pages, const void* x, const void* w_p,
                                     const void* w_g, void* out, void* workspace, size_t workspace_bytes,
                                     int32_t* status_word, void* cuda_stream) {
    g_last_launches = 0;
    if (!shape) return GTA_ERR_INVALID_ARG;
    if (!page_args_ok(block_table, page_size, n_pages, max_pages)) return GTA_ERR_INVALID_ARG;
    if (kv_len < shape->seq || (long long)kv_len > (long long)page_size * max_pages) return GTA_ERR_INVALID_ARG;
    return prefill_impl(shape, kv_len, page_size * max_pages, q, k_pool, c_pool, x, w_p, w_g, out, workspace,
                        workspace_bytes, status_word, cuda_stream, 3,
                        page_map(block_table, page_size, n_pages, max_pages));
}

}  // extern "C"

static gta_status_t prefill_impl(const gta_shape_t* shape, int32_t kv_len, int32_t kv_cap, const void* q,
                                 const void* k, const void* c, const void* x, const void* w_p, const void* w_g,
                                 void* out, void* workspace, size_t workspace_bytes, int32_t* status_word,
                                 void* cuda_stream, int32_t stages, const gta::PageMap& pm) {
    g_last_launches = 0;
    if (stages < 1 || stages > 3) return GTA_ERR_INVALID_ARG;
    gta::Dims d;
    gta_status_t st = check_shape(shape, true, &d);
    if (st != GTA_OK) return st;
    d.Nk = kv_len;
    d.S = kv_cap;
    if (!q || !k || !c || !x || !w_p || !w_g || !out) return GTA_ERR_INVALID_ARG;
    if (!aligned(q, 16) || !aligned(k, 16) || !aligned(c, 16) || !aligned(x, 16) || !aligned(w_p, 16) ||
        !aligned(w_g, 16) || !aligned(out, 16) || !aligned(status_word, 4))
        return GTA_ERR_INVALID_ARG;
    const int path = gta_prefill_path(shape);
    if (path == 0) return GTA_ERR_UNSUPPORTED;
    if (d.B == 0 || d.N == 0) return GTA_OK;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < gta_prefill_workspace_bytes(shape))
        return GTA_ERR_WORKSPACE;
    if ((st = check_device()) != GTA_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int launches = 0;
    cudaError_t err;
    // paged pools: the tensor-core attention kernel loads blocks of 64 tokens, each inside one page
    if (path == 2 && (pm.table == nullptr || pm.page_size % 64 == 0)) {
        st = gta::launch_sm100_prefill(d, q, k, c, x, w_p, w_g, out, workspace, status_word, stream, stages, &launches,
                                       pm);
        if (st != GTA_OK) return st;
        err = cudaSuccess;
    } else {
        err = gta::launch_generic_prefill(d, shape->dtype, q, k, c, x, w_p, w_g, out,
                                          static_cast<float*>(workspace), stream, stages, &launches, pm, status_word);
    }
    if (err != cudaSuccess) return GTA_ERR_CUDA;
    g_last_launches = launches;
    return GTA_OK;
}

extern "C" {

size_t gta_decode_workspace_bytes(const gta_shape_t* shape, int32_t S_cap) {
    gta::Dims d;
    if (check_shape(shape, false, &d) != GTA_OK || S_cap < 0) return 0;
    return gta::decode_workspace_bytes(d, shape->dtype, S_cap);
}

gta_status_t gta_decode(const gta_shape_t* shape, const void* q, const void* k_cache, const void* c_cache,
                        const int32_t* seq_lens, int32_t S_cap, const void* x_t, const void* w_p,
                        const void* w_g, void* out, void* workspace, size_t workspace_bytes,
                        int32_t* status_word, void* cuda_stream) {
    return gta_decode_stages(shape, q, k_cache, c_cache, seq_lens, S_cap, x_t, w_p, w_g, out, workspace,
                             workspace_bytes, status_word, cuda_stream, 7);
}

gta_status_t gta_decode_stages(const gta_shape_t* shape, const void* q, const void* k_cache,
                               const void* c_cache, const int32_t* seq_lens, int32_t S_cap, const void* x_t,
                               const void* w_p, const void* w_g, void* out, void* workspace,
                               size_t workspace_bytes, int32_t* status_word, void* cuda_stream,
                               int32_t stages) {
    return decode_impl(shape, q, k_cache, c_cache, seq_lens, S_cap, x_t, w_p, w_g, out, workspace, workspace_bytes,
                       status_word, cuda_stream, stages, gta::PageMap());
}

size_t gta_decode_paged_workspace_bytes(const gta_shape_t* shape, int32_t page_size, int32_t max_pages) {
    gta::Dims d;
    if (check_shape(shape, false, &d) != GTA_OK || page_size <= 0 || max_pages <= 0 ||
        (long long)page_size * max_pages > INT32_MAX)
        return 0;
    return gta::decode_workspace_bytes(d, shape->dtype, page_size * max_pages, page_size);
}

gta_status_t gta_decode_paged(const gta_shape_t* shape, const void* q, const void* k_pool, const void* c_pool,
                              const int32_t* block_table, int32_t page_size, int32_t n_pages, int32_t max_pages,
                              const int32_t* seq_lens, const void* x_t, const void* w_p, const void* w_g,
                              void* out, void* workspace, size_t workspace_bytes, int32_t* status_word,
                              void* cuda_stream) {
    g_last_launches = 0;
    if (!page_args_ok(block_table, page_size, n_pages, max_pages)) return GTA_ERR_INVALID_ARG;
    return decode_impl(shape, q, k_pool, c_pool, seq_lens, page_size * max_pages, x_t, w_p, w_g, out, workspace,
                       workspace_bytes, status_word, cuda_stream, 7,
                       page_map(block_table, page_size, n_pages, max_pages));
}

gta_status_t gta_cache_append_paged(const gta_shape_t* shape, void* k_pool, void* c_pool,
                                    const int32_t* block_table, int32_t page_size, int32_t n_pages,
                                    int32_t max_pages, const void* k_new, const void* c_new, int32_t n_new,
                                    int32_t* seq_lens, int32_t* status_word, void* cuda_stream) {
    g_last_launches = 0;
    if (!page_args_ok(block_table, page_size, n_pages, max_pages)) return GTA_ERR_INVALID_ARG;
    return append_impl(shape, k_pool, c_pool, page_size * max_pages, k_new, c_new, n_new, seq_lens, status_word,
                       cuda_stream, page_map(block_table, page_size, n_pages, max_pages));
}

}  // extern "C"

// ---- whole attention layer (App. B.1.1): projections + RoPE + cache write, operator, output projection
static size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

extern "C" size_t gta_layer_prefill_workspace_bytes(const gta_shape_t* shape) {
    gta::Dims d;
    if (check_shape(shape, true, &d) != GTA_OK) return 0;
    const size_t es = elem_size(shape->dtype);
    const size_t q_bytes = align256((size_t)d.B * d.n_q * d.N * d.d_h * es);
    const size_t o_bytes = align256((size_t)d.B * d.N * d.n_h * d.d_h * es);
    return q_bytes + o_bytes + align256(gta::sm100_rope_table_bytes(d)) + gta_prefill_workspace_bytes(shape);
}

static gta_status_t layer_prefill_impl(const gta_shape_t* shape, int32_t pos0, int32_t S_cap, float rope_base,
                                       const void* x, const void* w_qkc, const void* w_p, const void* w_g,
                                       const void* w_o, void* k_cache, void* c_cache, void* u, void* workspace,
                                       size_t workspace_bytes, int32_t* status_word, void* cuda_stream,
                                       const gta::PageMap& pm);

extern "C" gta_status_t gta_layer_prefill(const gta_shape_t* shape, int32_t pos0, int32_t S_cap, float rope_base,
                                          const void* x, const void* w_qkc, const void* w_p, const void* w_g,
                                          const void* w_o, void* k_cache, void* c_cache, void* u, void* workspace,
                                          size_t workspace_bytes, int32_t* status_word, void* cuda_stream) {
    return layer_prefill_impl(shape, pos0, S_cap, rope_base, x, w_qkc, w_p, w_g, w_o, k_cache, c_cache, u, workspace,
                              workspace_bytes, status_word, cuda_stream, gta::PageMap());
}

extern "C" gta_status_t gta_layer_prefill_paged(const gta_shape_t* shape, int32_t pos0, float rope_base,
                                                const void* x, const void* w_qkc, const void* w_p, const void* w_g,
                                                const void* w_o, void* k_pool, void* c_pool,
                                                const int32_t* block_table, int32_t page_size, int32_t n_pages,
                                                int32_t max_pages, void* u, void* workspace, size_t workspace_bytes,
                                                int32_t* status_word, void* cuda_stream) {
    g_last_launches = 0;
    if (!page_args_ok(block_table, page_size, n_pages, max_pages)) return GTA_ERR_INVALID_ARG;
    return layer_prefill_impl(shape, pos0, page_size * max_pages, rope_base, x, w_qkc, w_p, w_g, w_o, k_pool, c_pool, u,
                              workspace, workspace_bytes, status_word, cuda_stream,
                              page_map(block_table, page_size, n_pages, max_pages));
}

static gta_status_t layer_prefill_impl(const gta_shape_t* shape, int32_t pos0, int32_t S_cap, float rope_base,
                                       const void* x, const void* w_qkc, const void* w_p, const void* w_g,
                                       const void* w_o, void* k_cache, void* c_cache, void* u, void* workspace,
                                       size_t workspace_bytes, int32_t* status_word, void* cuda_stream,
                                       const gta::PageMap& pm) {
    g_last_launches = 0;
    gta::Dims d;
    gta_status_t st = check_shape(shape, true, &d);
    if (st != GTA_OK) return st;
    if (pos0 < 0 || S_cap < 0 || (long long)pos0 + d.N > S_cap || !(rope_base > 1.0f)) return GTA_ERR_INVALID_ARG;
    if (!d.causal) return GTA_ERR_INVALID_ARG;      // a chunk written behind a cache is causal by construction
    if (!x || !w_qkc || !w_p || !w_g || !w_o || !k_cache || !c_cache || !u) return GTA_ERR_INVALID_ARG;
    if (!aligned(x, 16) || !aligned(w_qkc, 16) || !aligned(w_p, 16) || !aligned(w_g, 16) || !aligned(w_o, 16) ||
        !aligned(k_cache, 16) || !aligned(c_cache, 16) || !aligned(u, 16) || !aligned(status_word, 4))
        return GTA_ERR_INVALID_ARG;
    if (!gta::sm100_linear_supported(d, shape->dtype) || gta_prefill_path(shape) == 0) return GTA_ERR_UNSUPPORTED;
    if (d.B == 0 || d.N == 0) return GTA_OK;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < gta_layer_prefill_workspace_bytes(shape))
        return GTA_ERR_WORKSPACE;
    if ((st = check_device()) != GTA_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t es = elem_size(shape->dtype);
    char* ws = static_cast<char*>(workspace);
    void* q_ws = ws;
    void* o_ws = ws + align256((size_t)d.B * d.n_q * d.N * d.d_h * es);
    char* rope_ws = static_cast<char*>(o_ws) + align256((size_t)d.B * d.N * d.n_h * d.d_h * es);
    char* op_ws = rope_ws + align256(gta::sm100_rope_table_bytes(d));
    const size_t op_ws_bytes = workspace_bytes - (size_t)(op_ws - ws);
    st = gta::launch_sm100_project(d, pos0, S_cap, (double)rope_base, x, w_qkc, q_ws, k_cache, c_cache, rope_ws,
                                   status_word, stream, pm);
    if (st != GTA_OK) return st;
    // the chunk's queries against everything the caches now hold for these sequences
    st = prefill_impl(shape, pos0 + d.N, S_cap, q_ws, k_cache, c_cache, x, w_p, w_g, o_ws, op_ws, op_ws_bytes,
                      status_word, cuda_stream, 3, pm);
    if (st != GTA_OK) return st;
    const int op_launches = g_last_launches;
    st = gta::launch_sm100_matmul((long long)d.B * d.N, d.n_h * d.d_h, d.H, o_ws, w_o, u, status_word, stream);
    if (st != GTA_OK) return st;
    g_last_launches = op_launches + 3;
    return GTA_OK;
}

extern "C" size_t gta_layer_decode_workspace_bytes(const gta_shape_t* shape, int32_t S_cap) {
    gta::Dims d;
    if (check_shape(shape, false, &d) != GTA_OK || S_cap < 0) return 0;
    const size_t es = elem_size(shape->dtype);
    return align256((size_t)d.B * d.n_q * d.d_h * es) + align256((size_t)d.B * d.n_h * d.d_h * es) +
           align256(gta::sm100_decode_prep_bytes(d)) + gta::decode_workspace_bytes(d, shape->dtype, S_cap);
}

static gta_status_t layer_decode_impl(const gta_shape_t* shape, int32_t S_cap, float rope_base, const void* x_t,
                                      const void* w_qkc, const void* w_p, const void* w_g, const void* w_o,
                                      void* k_cache, void* c_cache, int32_t* seq_lens, void* u, void* workspace,
                                      size_t workspace_bytes, int32_t* status_word, void* cuda_stream,
                                      const gta::PageMap& pm);

extern "C" gta_status_t gta_layer_decode(const gta_shape_t* shape, int32_t S_cap, float rope_base, const void* x_t,
                                         const void* w_qkc, const void* w_p, const void* w_g, const void* w_o,
                                         void* k_cache, void* c_cache, int32_t* seq_lens, void* u, void* workspace,
                                         size_t workspace_bytes, int32_t* status_word, void* cuda_stream) {
    return layer_decode_impl(shape, S_cap, rope_base, x_t, w_qkc, w_p, w_g, w_o, k_cache, c_cache, seq_lens, u,
                             workspace, workspace_bytes, status_word, cuda_stream, gta::PageMap());
}

extern "C" size_t gta_layer_decode_paged_workspace_bytes(const gta_shape_t* shape, int32_t page_size,
                                                         int32_t max_pages) {
    gta::Dims d;
    if (check_shape(shape, false, &d) != GTA_OK || page_size <= 0 || max_pages <= 0 ||
        (long long)page_size * max_pages > INT32_MAX)
        return 0;
    const size_t es = elem_size(shape->dtype);
    return align256((size_t)d.B * d.n_q * d.d_h * es) + align256((size_t)d.B * d.n_h * d.d_h * es) +
           align256(gta::sm100_decode_prep_bytes(d)) +
           gta::decode_workspace_bytes(d, shape->dtype, page_size * max_pages, page_size);
}

extern "C" gta_status_t gta_layer_decode_paged(const gta_shape_t* shape, const int32_t* block_table,
                                               int32_t page_size, int32_t n_pages, int32_t max_pages,
                                               float rope_base, const void* x_t, const void* w_qkc, const void* w_p,
                                               const void* w_g, const void* w_o, void* k_pool, void* c_pool,
                                               int32_t* seq_lens, void* u, void* workspace, size_t workspace_bytes,
                                               int32_t* status_word, void* cuda_stream) {
    g_last_launches = 0;
    if (!page_args_ok(block_table, page_size, n_pages, max_pages)) return GTA_ERR_INVALID_ARG;
    return layer_decode_impl(shape, page_size * max_pages, rope_base, x_t, w_qkc, w_p, w_g, w_o, k_pool, c_pool,
                             seq_lens, u, workspace, workspace_bytes, status_word, cuda_stream,
                             page_map(block_table, page_size, n_pages, max_pages));
}

static gta_status_t layer_decode_impl(const gta_shape_t* shape, int32_t S_cap, float rope_base, const void* x_t,
                                      const void* w_qkc, const void* w_p, const void* w_g, const void* w_o,
                                      void* k_cache, void* c_cache, int32_t* seq_lens, void* u, void* workspace,
                                      size_t workspace_bytes, int32_t* status_word, void* cuda_stream,
                                      const gta::PageMap& pm) {
    g_last_launches = 0;
    gta::Dims d;
    gta_status_t st = check_shape(shape, false, &d);
    if (st != GTA_OK) return st;
    if (S_cap <= 0 || !(rope_base > 1.0f)) return GTA_ERR_INVALID_ARG;
    if (!x_t || !w_qkc || !w_p || !w_g || !w_o || !k_cache || !c_cache || !seq_lens || !u) return GTA_ERR_INVALID_ARG;
    if (!aligned(x_t, 16) || !aligned(w_qkc, 16) || !aligned(w_p, 16) || !aligned(w_g, 16) || !aligned(w_o, 16) ||
        !aligned(k_cache, 16) || !aligned(c_cache, 16) || !aligned(u, 16) || !aligned(seq_lens, 4) ||
        !aligned(status_word, 4))
        return GTA_ERR_INVALID_ARG;
    if (!gta::sm100_linear_supported(d, shape->dtype) || (size_t)d.d_l * elem_size(shape->dtype) > 4096)
        return GTA_ERR_UNSUPPORTED;
    if (d.B == 0) return GTA_OK;
    const size_t ws_need = pm.table ? gta_layer_decode_paged_workspace_bytes(shape, pm.page_size, pm.max_pages)
                                    : gta_layer_decode_workspace_bytes(shape, S_cap);
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < ws_need) return GTA_ERR_WORKSPACE;
    if ((st = check_device()) != GTA_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t es = elem_size(shape->dtype);
    char* ws = static_cast<char*>(workspace);
    char* q_ws = ws;
    char* o_ws = q_ws + align256((size_t)d.B * d.n_q * d.d_h * es);
    char* prep_ws = o_ws + align256((size_t)d.B * d.n_h * d.d_h * es);
    char* op_ws = prep_ws + align256(gta::sm100_decode_prep_bytes(d));
    const size_t op_ws_bytes = workspace_bytes - (size_t)(op_ws - ws);
    st = gta::launch_sm100_project_step(d, S_cap, (double)rope_base, x_t, w_qkc, q_ws, k_cache, c_cache, seq_lens,
                                        prep_ws, status_word, stream, pm);
    if (st != GTA_OK) return st;
    st = decode_impl(shape, q_ws, k_cache, c_cache, seq_lens, S_cap, x_t, w_p, w_g, o_ws, op_ws, op_ws_bytes,
                     status_word, cuda_stream, 7, pm);
    if (st != GTA_OK) return st;
    const int op_launches = g_last_launches;
    st = gta::launch_sm100_matmul(d.B, d.n_h * d.d_h, d.H, o_ws, w_o, u, status_word, stream);
    if (st != GTA_OK) return st;
    g_last_launches = op_launches + 3;
    return GTA_OK;
}

// Host-side checks of a decode call that need no workspace and no device: the shape, the pointers
// and their alignment, the limits of the kernels.  *empty is set when the batch is empty (nothing to do).
gta_status_t gta::decode_check_args(const gta_shape_t* shape, const void* q, const void* k_cache, const void* c_cache,
                                    const int32_t* seq_lens, int32_t S_cap, const void* x_t, const void* w_p,
                                    const void* w_g, const void* out, const int32_t* status_word, gta::Dims* d,
                                    bool* empty) {
    *empty = false;
    gta_status_t st = check_shape(shape, false, d);
    if (st != GTA_OK) return st;
    if (S_cap < 0) return GTA_ERR_INVALID_ARG;
    if (!q || !seq_lens || !x_t || !w_p || !w_g || !out) return GTA_ERR_INVALID_ARG;
    if (S_cap > 0 && (!k_cache || !c_cache)) return GTA_ERR_INVALID_ARG;
    if (!aligned(q, 16) || !aligned(k_cache, 16) || !aligned(c_cache, 16) || !aligned(x_t, 16) ||
        !aligned(w_p, 16) || !aligned(w_g, 16) || !aligned(out, 16) || !aligned(seq_lens, 4) ||
        !aligned(status_word, 4))
        return GTA_ERR_INVALID_ARG;
    // one latent row is spread over at most 256 threads, 16 bytes each
    if ((size_t)d->d_l * elem_size(shape->dtype) > 4096) return GTA_ERR_UNSUPPORTED;
    *empty = d->B == 0;
    return GTA_OK;
}

gta_status_t gta::check_current_device() { return check_device(); }

static gta_status_t decode_impl(const gta_shape_t* shape, const void* q, const void* k_cache, const void* c_cache,
                                const int32_t* seq_lens, int32_t S_cap, const void* x_t, const void* w_p,
                                const void* w_g, void* out, void* workspace, size_t workspace_bytes,
                                int32_t* status_word, void* cuda_stream, int32_t stages, const gta::PageMap& pm) {
    g_last_launches = 0;
    if (stages < 1 || stages > 7) return GTA_ERR_INVALID_ARG;
    gta::Dims d;
    bool empty = false;
    gta_status_t st = gta::decode_check_args(shape, q, k_cache, c_cache, seq_lens, S_cap, x_t, w_p, w_g, out,
                                             status_word, &d, &empty);
    if (st != GTA_OK) return st;
    if (empty) return GTA_OK;
    if (!workspace || !aligned(workspace, 256) ||
        workspace_bytes < gta::decode_workspace_bytes(d, shape->dtype, S_cap, pm.table ? pm.page_size : 0))
        return GTA_ERR_WORKSPACE;
    if ((st = check_device()) != GTA_OK) return st;
    int launches = 0;
    cudaError_t err = gta::launch_decode(d, shape->dtype, q, k_cache, c_cache, seq_lens, S_cap, x_t, w_p, w_g,
                                         out, workspace, status_word, static_cast<cudaStream_t>(cuda_stream),
                                         stages, &launches, pm);
    if (err != cudaSuccess) return GTA_ERR_CUDA;
    g_last_launches = launches;
    return GTA_OK;
}

extern "C" gta_status_t gta_cache_append(const gta_shape_t* shape, void* k_cache, void* c_cache, int32_t S_cap,
                                         const void* k_new, const void* c_new, int32_t n_new, int32_t* seq_lens,
                                         int32_t* status_word, void* cuda_stream) {
    return append_impl(shape, k_cache, c_cache, S_cap, k_new, c_new, n_new, seq_lens, status_word, cuda_stream,
                       gta::PageMap());
}

static gta_status_t append_impl(const gta_shape_t* shape, void* k_cache, void* c_cache, int32_t S_cap,
                                const void* k_new, const void* c_new, int32_t n_new, int32_t* seq_lens,
                                int32_t* status_word, void* cuda_stream, const gta::PageMap& pm) {
    g_last_launches = 0;
    gta::Dims d;
    gta_status_t st = check_shape(shape, false, &d);
    if (st != GTA_OK) return st;
    if (S_cap < 0 || n_new < 0) return GTA_ERR_INVALID_ARG;
    if (!k_cache || !c_cache || !k_new || !c_new || !seq_lens) return GTA_ERR_INVALID_ARG;
    if (!aligned(k_cache, 16) || !aligned(c_cache, 16) || !aligned(k_new, 16) || !aligned(c_new, 16) ||
        !aligned(seq_lens, 4) || !aligned(status_word, 4))
        return GTA_ERR_INVALID_ARG;
    if (d.B == 0 || n_new == 0) return GTA_OK;
    if ((st = check_device()) != GTA_OK) return st;
    int launches = 0;
    cudaError_t err = gta::launch_cache_append(d, (int)elem_size(shape->dtype), k_cache, c_cache, S_cap, k_new,
                                               c_new, n_new, seq_lens, status_word,
                                               static_cast<cudaStream_t>(cuda_stream), &launches, pm);
    if (err != cudaSuccess) return GTA_ERR_CUDA;
    g_last_launches = launches;
    return GTA_OK;
}

// ---- comparison operators of the paper (App. B.3, GQA; with one key / value head per query head, the MHA of
//      Sec. 3.1) on the same tensor-core attention kernel and the same stream / merge kernels
static gta_status_t gqa_check(const gta_shape_t* s, bool need_seq, float* scale) {
    if (!s) return GTA_ERR_INVALID_ARG;
    if (s->batch < 0 || (need_seq && s->seq < 0) || s->n_heads < 1 || s->n_k_groups < 1 || s->head_dim < 1)
        return GTA_ERR_INVALID_ARG;
    if (s->n_heads % s->n_k_groups) return GTA_ERR_INVALID_ARG;
    if (s->dtype != GTA_F32 && s->dtype != GTA_BF16) return GTA_ERR_INVALID_ARG;
    if (s->causal != 0 && s->causal != 1) return GTA_ERR_INVALID_ARG;
    if (!(s->softmax_scale >= 0.f) || isinf(s->softmax_scale)) return GTA_ERR_INVALID_ARG;
    if (s->dtype != GTA_BF16 || (s->head_dim != 64 && s->head_dim != 128) || s->batch > 65535 || s->n_heads > 65535)
        return GTA_ERR_UNSUPPORTED;
    *scale = s->softmax_scale > 0.f ? s->softmax_scale : 1.0f / sqrtf((float)s->head_dim);
    return GTA_OK;
}

extern "C" gta_status_t gta_ref_gqa_prefill(const gta_shape_t* shape, const void* q, const void* k, const void* v,
                                            void* out, int32_t* status_word, void* cuda_stream) {
    g_last_launches = 0;
    float scale = 0.f;
    gta_status_t st = gqa_check(shape, true, &scale);
    if (st != GTA_OK) return st;
    if (!q || !k || !v || !out) return GTA_ERR_INVALID_ARG;
    if (!aligned(q, 16) || !aligned(k, 16) || !aligned(v, 16) || !aligned(out, 16) || !aligned(status_word, 4))
        return GTA_ERR_INVALID_ARG;
    if (shape->batch == 0 || shape->seq == 0) return GTA_OK;
    if ((st = check_device()) != GTA_OK) return st;
    // one attention map per query head; the value heads take the place of the latent (d_h wide, one "latent
    // group" per key / value head); the attention kernel's normalised output is the operator's output
    gta::Dims d = {};
    d.B = shape->batch; d.N = shape->seq; d.H = 64; d.n_h = shape->n_heads; d.n_q = shape->n_heads;
    d.n_k = shape->n_k_groups; d.n_c = shape->n_k_groups; d.d_h = shape->head_dim; d.d_l = shape->head_dim;
    d.causal = shape->causal; d.scale = scale; d.Nk = d.N; d.S = d.N;
    st = gta::launch_sm100_attention(d, q, k, v, out, status_word, static_cast<cudaStream_t>(cuda_stream));
    if (st != GTA_OK) return st;
    g_last_launches = 1;
    return GTA_OK;
}

extern "C" size_t gta_ref_gqa_decode_workspace_bytes(const gta_shape_t* shape) {
    float scale = 0.f;
    if (gqa_check(shape, false, &scale) != GTA_OK) return 0;
    if (!gta::gqa_decode_supported(shape->batch, shape->n_heads, shape->n_k_groups, shape->head_dim, shape->dtype)) return 0;
    return gta::gqa_decode_workspace_bytes(shape->batch, shape->n_heads, shape->n_k_groups, shape->head_dim);
}

extern "C" gta_status_t gta_ref_gqa_decode(const gta_shape_t* shape, const void* q, const void* k_cache,
                                           const void* v_cache, const int32_t* seq_lens, int32_t S_cap, void* out,
                                           void* workspace, size_t workspace_bytes, int32_t* status_word,
                                           void* cuda_stream) {
    g_last_launches = 0;
    float scale = 0.f;
    gta_status_t st = gqa_check(shape, false, &scale);
    if (st != GTA_OK) return st;
    if (S_cap <= 0) return GTA_ERR_INVALID_ARG;
    if (!q || !k_cache || !v_cache || !seq_lens || !out) return GTA_ERR_INVALID_ARG;
    if (!aligned(q, 16) || !aligned(k_cache, 16) || !aligned(v_cache, 16) || !aligned(out, 16) ||
        !aligned(seq_lens, 4) || !aligned(status_word, 4))
        return GTA_ERR_INVALID_ARG;
    if (!gta::gqa_decode_supported(shape->batch, shape->n_heads, shape->n_k_groups, shape->head_dim, shape->dtype))
        return GTA_ERR_UNSUPPORTED;
    if (shape->batch == 0) return GTA_OK;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < gta_ref_gqa_decode_workspace_bytes(shape))
        return GTA_ERR_WORKSPACE;
    if ((st = check_device()) != GTA_OK) return st;
    int launches = 0;
    cudaError_t err = gta::launch_gqa_decode(shape->batch, shape->n_heads, shape->n_k_groups, shape->head_dim, scale, q,
                                             k_cache, v_cache, seq_lens, S_cap, out, workspace, status_word,
                                             static_cast<cudaStream_t>(cuda_stream), &launches);
    if (err != cudaSuccess) return GTA_ERR_CUDA;
    g_last_launches = launches;
    return GTA_OK;
}

// ---- 8-bit caches (e4m3 codes + one fp32 scale per cached row)
static gta_status_t fp8_check(const gta_shape_t* shape, gta::Dims* d) {
    gta_status_t st = check_shape(shape, false, d);
    if (st != GTA_OK) return st;
    if (d->d_h % 16 || d->d_l % 16 || d->d_l > 2048) return GTA_ERR_UNSUPPORTED;   // rows are read as 16-byte vectors of codes
    return GTA_OK;
}

// enough for either kernel family (which one runs also depends on the alignment of the scale arrays)
static size_t fp8_workspace(const gta::Dims& d, int dtype, int S_cap) {
    size_t need = gta::decode_fp8_workspace_bytes(d, S_cap);
    if (gta::decode_fp8_fast_supported(d, dtype, S_cap)) {
        const size_t fast = gta::decode_fp8_fast_workspace_bytes(d);
        need = fast > need ? fast : need;
    }
    return need;
}

extern "C" size_t gta_decode_fp8_workspace_bytes(const gta_shape_t* shape, int32_t S_cap) {
    gta::Dims d;
    if (fp8_check(shape, &d) != GTA_OK || S_cap < 0) return 0;
    return fp8_workspace(d, shape->dtype, S_cap);
}

extern "C" int gta_decode_fp8_path(const gta_shape_t* shape, int32_t S_cap) {
    gta::Dims d;
    if (fp8_check(shape, &d) != GTA_OK || S_cap <= 0) return 0;
    return gta::decode_fp8_fast_supported(d, shape->dtype, S_cap) ? 2 : 1;
}

extern "C" gta_status_t gta_cache_append_fp8(const gta_shape_t* shape, void* k_codes, void* c_codes, float* k_scales,
                                             float* c_scales, int32_t S_cap, const void* k_new, const void* c_new,
                                             int32_t n_new, int32_t* seq_lens, int32_t* status_word, void* cuda_stream) {
    g_last_launches = 0;
    gta::Dims d;
    gta_status_t st = fp8_check(shape, &d);
    if (st != GTA_OK) return st;
    if (S_cap < 0 || n_new < 0) return GTA_ERR_INVALID_ARG;
    if (!k_codes || !c_codes || !k_scales || !c_scales || !k_new || !c_new || !seq_lens) return GTA_ERR_INVALID_ARG;
    if (!aligned(k_codes, 16) || !aligned(c_codes, 16) || !aligned(k_scales, 4) || !aligned(c_scales, 4) ||
        !aligned(k_new, 16) || !aligned(c_new, 16) || !aligned(seq_lens, 4) || !aligned(status_word, 4))
        return GTA_ERR_INVALID_ARG;
    if (d.B == 0 || n_new == 0) return GTA_OK;
    if ((st = check_device()) != GTA_OK) return st;
    int launches = 0;
    cudaError_t err = gta::launch_cache_append_fp8(d, shape->dtype, k_codes, c_codes, k_scales, c_scales, S_cap, k_new,
                                                   c_new, n_new, seq_lens, status_word,
                                                   static_cast<cudaStream_t>(cuda_stream), &launches);
    if (err != cudaSuccess) return GTA_ERR_CUDA;
    g_last_launches = launches;
    return GTA_OK;
}

extern "C" gta_status_t gta_decode_fp8(const gta_shape_t* shape, const void* q, const void* k_codes, const void* c_codes,
                                       const float* k_scales, const float* c_scales, const int32_t* seq_lens,
                                       int32_t S_cap, const void* x_t, const void* w_p, const void* w_g, void* out,
                                       void* workspace, size_t workspace_bytes, int32_t* status_word,
                                       void* cuda_stream) {
    g_last_launches = 0;
    gta::Dims d;
    gta_status_t st = fp8_check(shape, &d);
    if (st != GTA_OK) return st;
    if (S_cap <= 0) return GTA_ERR_INVALID_ARG;
    if (!q || !k_codes || !c_codes || !k_scales || !c_scales || !seq_lens || !x_t || !w_p || !w_g || !out)
        return GTA_ERR_INVALID_ARG;
    if (!aligned(q, 16) || !aligned(k_codes, 16) || !aligned(c_codes, 16) || !aligned(k_scales, 4) ||
        !aligned(c_scales, 4) || !aligned(x_t, 16) || !aligned(w_p, 16) || !aligned(w_g, 16) || !aligned(out, 16) ||
        !aligned(seq_lens, 4) || !aligned(status_word, 4))
        return GTA_ERR_INVALID_ARG;
    if (d.B == 0) return GTA_OK;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < fp8_workspace(d, shape->dtype, S_cap))
        return GTA_ERR_WORKSPACE;
    if ((st = check_device()) != GTA_OK) return st;
    int launches = 0;
    cudaError_t err;
    // the streaming kernel copies the scale rows in 16-byte pieces
    if (gta::decode_fp8_fast_supported(d, shape->dtype, S_cap) && aligned(k_scales, 16) && aligned(c_scales, 16))
        err = gta::launch_decode_fp8_fast(d, q, k_codes, c_codes, k_scales, c_scales, seq_lens, S_cap, x_t, w_p, w_g, out,
                                          workspace, status_word, static_cast<cudaStream_t>(cuda_stream), &launches);
    else
        err = gta::launch_decode_fp8(d, shape->dtype, q, k_codes, c_codes, k_scales, c_scales, seq_lens, S_cap,
                                     x_t, w_p, w_g, out, workspace, status_word,
                                     static_cast<cudaStream_t>(cuda_stream), &launches);
    if (err != cudaSuccess) return GTA_ERR_CUDA;
    g_last_launches = launches;
    return GTA_OK;
}

// ---- caches in page-locked host memory
extern "C" size_t gta_decode_hostcache_workspace_bytes(const gta_shape_t* shape, int32_t S_cap) {
    gta::Dims d;
    if (check_shape(shape, false, &d) != GTA_OK || S_cap < 0) return 0;
    return gta::decode_plain_workspace_bytes(d, S_cap);
}

extern "C" gta_status_t gta_decode_hostcache(const gta_shape_t* shape, const void* q, const void* k_cache,
                                             const void* c_cache, const int32_t* seq_lens, int32_t S_cap,
                                             const void* x_t, const void* w_p, const void* w_g, void* out,
                                             void* workspace, size_t workspace_bytes, int32_t* status_word,
                                             void* cuda_stream) {
    g_last_launches = 0;
    gta::Dims d;
    bool empty = false;
    gta_status_t st = gta::decode_check_args(shape, q, k_cache, c_cache, seq_lens, S_cap, x_t, w_p, w_g, out, status_word,
                                             &d, &empty);
    if (st != GTA_OK) return st;
    if (empty) return GTA_OK;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < gta::decode_plain_workspace_bytes(d, S_cap))
        return GTA_ERR_WORKSPACE;
    if ((st = check_device()) != GTA_OK) return st;
    int launches = 0;
    cudaError_t err = gta::launch_decode_plain(d, shape->dtype, q, k_cache, c_cache, seq_lens, S_cap, x_t, w_p, w_g, out,
                                               workspace, status_word, static_cast<cudaStream_t>(cuda_stream), &launches);
    if (err != cudaSuccess) return GTA_ERR_CUDA;
    g_last_launches = launches;
    return GTA_OK;
}

// ---- append + decode in one call
extern "C" gta_status_t gta_decode_append(const gta_shape_t* shape, const void* q, void* k_cache, void* c_cache,
                                          const void* k_new, const void* c_new, int32_t* seq_lens, int32_t S_cap,
                                          const void* x_t, const void* w_p, const void* w_g, void* out, void* workspace,
                                          size_t workspace_bytes, int32_t* status_word, void* cuda_stream) {
    g_last_launches = 0;
    gta::Dims d;
    bool empty = false;
    gta_status_t st = gta::decode_check_args(shape, q, k_cache, c_cache, seq_lens, S_cap, x_t, w_p, w_g, out, status_word,
                                             &d, &empty);
    if (st != GTA_OK) return st;
    if (S_cap <= 0 || !k_new || !c_new || !aligned(k_new, 16) || !aligned(c_new, 16)) return GTA_ERR_INVALID_ARG;
    if (empty) return GTA_OK;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < gta::decode_workspace_bytes(d, shape->dtype, S_cap))
        return GTA_ERR_WORKSPACE;
    if ((st = check_device()) != GTA_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int launches = 0;
    cudaError_t err;
    if (gta::decode_fast_supported(d, shape->dtype, 0)) {
        // one pass: the stream kernel puts the new rows into the caches and attends over them, the lengths advance
        // in the last kernel of the step
        err = gta::launch_decode_fast(d, q, k_cache, c_cache, seq_lens, S_cap, x_t, w_p, w_g, out, workspace, status_word,
                                      stream, 7, &launches, gta::PageMap(), k_new, c_new);
    } else {
        err = gta::launch_cache_append(d, (int)elem_size(shape->dtype), k_cache, c_cache, S_cap, k_new, c_new, 1, seq_lens,
                                       status_word, stream, &launches);
        if (err == cudaSuccess)
            err = gta::launch_decode(d, shape->dtype, q, k_cache, c_cache, seq_lens, S_cap, x_t, w_p, w_g, out, workspace,
                                     status_word, stream, 7, &launches);
    }
    if (err != cudaSuccess) return GTA_ERR_CUDA;
    g_last_launches = launches;
    return GTA_OK;
}
