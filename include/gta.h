/*
 * gta.h — C ABI of the B200 (sm_100a) GTA attention operator library.
 *
 * GTA = Grouped-head latenT Attention.  One attention map is computed per query group
 * and shared by every head of the group; the probabilities are applied to a compressed
 * latent value tensor C (d_l wide) instead of per-head values; each head then decodes its
 * value with its own projection W_P,i and a sigmoid gate computed from the hidden state
 * of the query token (paper Sec. 3.2 "Input projections and grouping", "Nonlinear value
 * decoder", and Sec. 3.3 "Efficient attention computation", reformulated equation).
 *
 * Symbols (paper Sec. 3.2): B batch, N sequence length, H hidden size (d_model), n_h heads,
 * n_q / n_k / n_c query / key / latent groups, d_h head dim, d_l latent dim (d_l >= d_h).
 * Head -> group maps are contiguous blocks:
 *   q(i) = floor(i * n_q / n_h),  k(i) = floor(q(i) * n_k / n_q),  c(i) = floor(q(i) * n_c / n_q)
 * which needs n_q | n_h, n_k | n_q and n_c | n_q.
 *
 * General rules for every entry point
 *   - Every tensor pointer is a DEVICE pointer unless it says "host".  The caller owns all
 *     buffers; the library allocates no device memory and keeps no per-call state.
 *   - Tensors are dense, row-major, innermost dimension last, base address 16-byte aligned.
 *   - All work is enqueued on `cuda_stream` (a cudaStream_t cast to void*; NULL = the legacy
 *     default stream).  No call synchronises the device or the stream.
 *   - Errors the host can see (null pointer, misalignment, bad divisibility, unsupported
 *     sizes, workspace too small, not an sm_100 device) are returned as a status code before
 *     anything is launched.  Conditions only the device can see (a full cache, a bounded wait
 *     that ran out) are written to `*status_word`, a device int32 the caller zeroes and reads
 *     after its own synchronisation; kernels only ever raise it (atomic max) and it may be NULL.
 *   - No entry point aborts, traps or throws.
 */
#ifndef GTA_H_
#define GTA_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define GTA_API __attribute__((visibility("default")))
#else
#define GTA_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    GTA_OK = 0,
    GTA_ERR_INVALID_ARG = 1, /* null pointer, misaligned pointer, negative size, bad divisibility */
    GTA_ERR_UNSUPPORTED = 2, /* shape / dtype / device outside what the kernels cover */
    GTA_ERR_WORKSPACE = 3,   /* workspace missing or smaller than *_workspace_bytes() */
    GTA_ERR_CUDA = 4,        /* a CUDA runtime / driver call failed (launch, attribute, tensor map) */
    GTA_ERR_CACHE_FULL = 5,  /* device-side: an append would exceed S_cap for some sequence */
    GTA_ERR_TIMEOUT = 6,     /* device-side: a bounded wait inside a kernel ran out */
    GTA_ERR_STATIC_SCRATCH = 7, /* gta_decode_static: the problem needs more than GTA_STATIC_SCRATCH_BYTES */
    GTA_ERR_BAD_PAGE = 8     /* device-side: a block-table entry in use lies outside [0, n_pages) */
} gta_status_t;

typedef enum { GTA_F32 = 0, GTA_BF16 = 1 } gta_dtype_t;

typedef struct {
    int32_t batch;       /* B */
    int32_t seq;         /* prefill: N (query length = key length).  decode / append: ignored */
    int32_t d_model;     /* H: row length of x and number of rows of W_G */
    int32_t n_heads;     /* n_h */
    int32_t n_q_groups;  /* n_q: number of attention maps; must divide n_h */
    int32_t n_k_groups;  /* n_k: must divide n_q */
    int32_t n_c_groups;  /* n_c: must divide n_q */
    int32_t head_dim;    /* d_h */
    int32_t latent_dim;  /* d_l */
    int32_t causal;      /* 1: key j <= query t (diagonal included, App. B.1.1); 0: all keys */
    int32_t dtype;       /* gta_dtype_t; storage type of EVERY tensor argument */
    float softmax_scale; /* 0 => 1/sqrt(d_h) (Sec. 3.3) */
} gta_shape_t;

/*
 * gta_prefill — causal prefill of the whole operator (Sec. 3.3, reformulated equation, with
 * the causal sum of App. B.1.1):
 *   P_g   = Softmax(scale * Q_g K_{k(g)}^T)            one map per query group g
 *   L_g   = P_g C_{c(g)}                               [N, d_l]
 *   out_i = (L_{q(i)} W_P,i) (.) Sigmoid(X W_G,i)      per head i; the gate of row t uses x_t
 * The output projection W_O and RoPE are outside the operator (q, k arrive post-RoPE).
 *
 *   q   [B, n_q, N, d_h]      k   [B, n_k, N, d_h]      c  [B, n_c, N, d_l]
 *   x   [B, N, H]             w_p [n_h, d_l, d_h]       w_g [H, n_h*d_h]
 *   out [B, N, n_h, d_h]      (written; same dtype as the inputs, round-to-nearest-even)
 *   workspace: at least gta_prefill_workspace_bytes(shape) bytes, 256-byte aligned; holds
 *     the normalised latent attention output L between the two kernels; contents undefined
 *     afterwards.  Calls that share a workspace must be ordered on one stream.
 * Arithmetic: fp32 accumulation everywhere.  bf16 fast path (tcgen05 tensor cores) when
 * dtype = bf16, d_h = 64 or 128, d_l a multiple of 128 (at most 1024), H a multiple of 64 and
 * the heads of one attention map fill a multiple of 128 output columns ((n_h / n_q) d_h);
 * other shapes and fp32 run on the plain-ALU kernels of the same library (gta_prefill_path
 * tells which).  N = 0 or B = 0 is a no-op (GTA_OK).
 */
GTA_API size_t gta_prefill_workspace_bytes(const gta_shape_t *shape);
GTA_API gta_status_t gta_prefill(const gta_shape_t *shape, const void *q, const void *k, const void *c,
                         const void *x, const void *w_p, const void *w_g, void *out,
                         void *workspace, size_t workspace_bytes, int32_t *status_word,
                         void *cuda_stream);

/*
 * gta_prefill_chunk — gta_prefill for a chunk of queries against longer keys and latents that
 * already sit in a cache: the N = shape->seq query tokens are the LAST N of kv_len attended
 * positions, so with causal = 1 query t attends keys 0 .. t + kv_len - N (the causal sum of
 * App. B.1.1 over the whole sequence, restricted to the chunk's rows); row t of the result
 * equals row kv_len - N + t of gta_prefill over all kv_len tokens.
 *
 *   q   [B, n_q, N, d_h]          x   [B, N, H]        out [B, N, n_h, d_h]
 *   k   [B, n_k, kv_cap, d_h]     c   [B, n_c, kv_cap, d_l]    rows 0 .. kv_len-1 are read; the rows
 *   behind them may hold anything (uninitialised memory, NaN bit patterns): nothing of them reaches out
 *   N <= kv_len <= kv_cap (else GTA_ERR_INVALID_ARG); kv_len = kv_cap = N is gta_prefill.
 * Workspace, weights, arithmetic, paths and errors as for gta_prefill.
 */
GTA_API gta_status_t gta_prefill_chunk(const gta_shape_t *shape, int32_t kv_len, int32_t kv_cap,
                                       const void *q, const void *k, const void *c, const void *x,
                                       const void *w_p, const void *w_g, void *out, void *workspace,
                                       size_t workspace_bytes, int32_t *status_word, void *cuda_stream);

/*
 * gta_decode — one decode step (App. B.1.3): for every sequence b the new token's queries
 * attend the seq_lens[b] cached keys / latents (the new token's own entries included, i.e.
 * gta_cache_append has already run), then the decoder and gate of gta_prefill are applied
 * with x_t = hidden state of the new token.  Equals row seq_lens[b]-1 of gta_prefill.
 *
 *   q        [B, n_q, d_h]                 x_t [B, H]
 *   k_cache  [B, n_k, S_cap, d_h]          c_cache [B, n_c, S_cap, d_l]
 *   seq_lens device int32 [B], 0 <= seq_lens[b] <= S_cap (values above S_cap are clamped);
 *            a sequence with length 0 gets an all-zero output row; cache rows at and behind
 *            seq_lens[b] may hold anything (uninitialised memory, NaN bit patterns)
 *   w_p, w_g as in gta_prefill;  out [B, n_h, d_h]
 *   workspace: at least gta_decode_workspace_bytes(shape, S_cap) bytes, 256-byte aligned
 *     (split-KV partial results and gate partial sums).  The size follows the SM count of the
 *     device that is current when the function is asked, so ask with the device the call
 *     will run on (this holds for every *_workspace_bytes function of the decode family).
 * Needs d_h and d_l multiples of 8 (bf16) / 4 (fp32) so that rows are 16-byte vectors,
 * d_h <= 256, d_l <= 2048.  bf16 fast path (TMA-streamed caches, tensor-core decoder) when
 * d_h = 64 or 128, d_l = 128, 256, 512 or 1024, n_q <= 8, n_k = 1, 2, 4 or 8, H a
 * multiple of 64, B <= 512 and the heads of one attention map fill a multiple of 64 output
 * columns (128 for B > 128); everything else runs on the plain-ALU kernels.
 */
GTA_API size_t gta_decode_workspace_bytes(const gta_shape_t *shape, int32_t S_cap);
GTA_API gta_status_t gta_decode(const gta_shape_t *shape, const void *q, const void *k_cache,
                        const void *c_cache, const int32_t *seq_lens, int32_t S_cap,
                        const void *x_t, const void *w_p, const void *w_g, void *out,
                        void *workspace, size_t workspace_bytes, int32_t *status_word,
                        void *cuda_stream);

/*
 * gta_cache_append — write new keys and latents behind the live part of the caches (the
 * caches hold K and C of every past token: Sec. 3.3, last paragraph; App. B.1.3).  Pure
 * byte copy, bit-exact:
 *   for b with seq_lens[b] + n_new <= S_cap:
 *     k_cache[b, :, seq_lens[b] + n, :] = k_new[b, :, n, :]   n = 0 .. n_new-1   (c likewise)
 *     seq_lens[b] += n_new
 *   a sequence that would overflow is skipped entirely (cache and length unchanged) and
 *   *status_word is raised to GTA_ERR_CACHE_FULL.
 *
 *   k_cache [B, n_k, S_cap, d_h]  c_cache [B, n_c, S_cap, d_l]   (read-modify-write)
 *   k_new   [B, n_k, n_new, d_h]  c_new   [B, n_c, n_new, d_l]
 *   seq_lens device int32 [B] in/out.   n_new = 1 per decode step; n_new = N loads a prefill.
 * Rows must be multiples of 16 bytes (d_h, d_l multiples of 8 for bf16, 4 for fp32).
 */
GTA_API gta_status_t gta_cache_append(const gta_shape_t *shape, void *k_cache, void *c_cache,
                              int32_t S_cap, const void *k_new, const void *c_new,
                              int32_t n_new, int32_t *seq_lens, int32_t *status_word,
                              void *cuda_stream);

/*
 * gta_decode_paged / gta_cache_append_paged — gta_decode and gta_cache_append over a paged cache
 * (the paper keeps K and C of every past token, Sec. 3.3 last paragraph and App. B.1.3, and says
 * nothing on where the rows live: the operation is the same, only the addressing differs).
 * The rows of all sequences sit in two pools of fixed-size pages,
 *
 *   k_pool [n_pages, n_k, page_size, d_h]      c_pool [n_pages, n_c, page_size, d_l]
 *   block_table device int32 [B, max_pages]
 *
 * and cached token t of sequence b is row t % page_size of page block_table[b, t / page_size]
 * (the same page number in both pools).  The capacity of a sequence is page_size * max_pages
 * tokens, which takes the place of S_cap everywhere (length clamp, GTA_ERR_CACHE_FULL).  Only the
 * entries that cover live tokens (for the append: live and new tokens) are read; the others may
 * hold anything.  An entry in use outside [0, n_pages) raises *status_word to GTA_ERR_BAD_PAGE;
 * no memory outside the pools is touched, the affected sequences' results (or appended rows) are
 * unspecified.  The caller owns the block table and the assignment of pages; two sequences must
 * not append to the same page.
 *
 * Host-side errors: GTA_ERR_INVALID_ARG for a null or misaligned block table or a non-positive
 * page_size, n_pages or max_pages (or page_size * max_pages above INT32_MAX); otherwise as
 * gta_decode / gta_cache_append.  workspace: gta_decode_paged_workspace_bytes(shape, page_size,
 * max_pages).  The bf16 fast path of gta_decode applies when, in addition to its shape rules,
 * page_size is a multiple of 64; other page sizes run on the plain-ALU kernels.
 */
GTA_API size_t gta_decode_paged_workspace_bytes(const gta_shape_t *shape, int32_t page_size,
                                                int32_t max_pages);
GTA_API gta_status_t gta_decode_paged(const gta_shape_t *shape, const void *q, const void *k_pool,
                                      const void *c_pool, const int32_t *block_table,
                                      int32_t page_size, int32_t n_pages, int32_t max_pages,
                                      const int32_t *seq_lens, const void *x_t, const void *w_p,
                                      const void *w_g, void *out, void *workspace,
                                      size_t workspace_bytes, int32_t *status_word,
                                      void *cuda_stream);
GTA_API gta_status_t gta_cache_append_paged(const gta_shape_t *shape, void *k_pool, void *c_pool,
                                            const int32_t *block_table, int32_t page_size,
                                            int32_t n_pages, int32_t max_pages, const void *k_new,
                                            const void *c_new, int32_t n_new, int32_t *seq_lens,
                                            int32_t *status_word, void *cuda_stream);

/*
 * gta_prefill_chunk_paged — gta_prefill_chunk with the attended keys and latents in a paged cache (pools,
 * block table and their rules as in gta_decode_paged): attended position j of sequence b, 0 <= j < kv_len, is
 * row j % page_size of page block_table[b, j / page_size].  Every sequence has the same kv_len, with
 * N <= kv_len <= page_size * max_pages (else GTA_ERR_INVALID_ARG).  Only the block-table entries of
 * positions below kv_len are read; the rows of a sequence's last page behind kv_len, and every page no
 * such entry names, may hold anything (uninitialised memory, NaN bit patterns): nothing of them reaches
 * out.  An entry in use outside [0, n_pages) raises *status_word to GTA_ERR_BAD_PAGE; no memory outside
 * the pools is touched, and the keys of such a page take no part in the affected sequence's result
 * (they are left out of the softmax on the plain-ALU kernels and read as zero rows on the tensor-core
 * kernels, so that result is unspecified).
 * q, x, weights, out, workspace (gta_prefill_workspace_bytes), arithmetic and errors as for
 * gta_prefill_chunk; the tensor-core path applies when, in addition to gta_prefill's rules, page_size is
 * a multiple of 64, other page sizes run on the plain-ALU kernels.
 */
GTA_API gta_status_t gta_prefill_chunk_paged(const gta_shape_t *shape, int32_t kv_len, const void *q,
                                             const void *k_pool, const void *c_pool,
                                             const int32_t *block_table, int32_t page_size, int32_t n_pages,
                                             int32_t max_pages, const void *x, const void *w_p,
                                             const void *w_g, void *out, void *workspace,
                                             size_t workspace_bytes, int32_t *status_word,
                                             void *cuda_stream);

/*
 * gta_layer_prefill — the whole attention layer of App. B.1.1 for a chunk of N tokens per sequence
 * that starts at position pos0 (pos0 = 0: a prompt):
 *
 *   [q | k | c]_t = x_t W_qkc                 one matrix, columns = the n_q query groups (d_h each), then
 *                                             the n_k key groups (d_h each), then the n_c latent groups (d_l each)
 *   q, k <- RoPE(q, k; position pos0 + t)     per d_h-vector, pairs of neighbouring elements (2i, 2i+1)
 *                                             rotated by (pos0 + t) rope_base^(-2i/d_h)  (RoFormer, which the
 *                                             paper cites; the paper does not fix the pairing or the base)
 *   k_cache[b, :, pos0 + t, :] = k_t,  c_cache[b, :, pos0 + t, :] = c_t       (the prefill's bulk append)
 *   o_t = gta_prefill_chunk of the chunk's queries over cache rows 0 .. pos0 + N - 1, gated by x_t
 *   u_t = [o_{t,1}; ...; o_{t,n_h}] W_o
 *
 *   x [B, N, H]   w_qkc [H, (n_q + n_k) d_h + n_c d_l]   w_p, w_g as in gta_prefill   w_o [n_h d_h, H]
 *   k_cache [B, n_k, S_cap, d_h]   c_cache [B, n_c, S_cap, d_l]   (rows pos0 .. pos0 + N - 1 are written,
 *   rows below pos0 are read, rows above are left alone; no length vector is read or written)
 *   u [B, N, H]   workspace: gta_layer_prefill_workspace_bytes(shape), 256-byte aligned (q, the gated
 *   heads and the operator's own workspace).
 * q, k, c and the gated heads are rounded to the storage type where they are stored (the caches and
 * the workspace), as every tensor of the operator is.
 * bf16 only, on the tensor-core kernels: H a multiple of 128, d_h = 64 or 128, d_l a multiple of 64,
 * (n_q + n_k) d_h + n_c d_l a multiple of 128; otherwise GTA_ERR_UNSUPPORTED.  GTA_ERR_INVALID_ARG
 * also for pos0 < 0, pos0 + N > S_cap, rope_base <= 1 or a non-causal shape.
 */
GTA_API size_t gta_layer_prefill_workspace_bytes(const gta_shape_t *shape);
GTA_API gta_status_t gta_layer_prefill(const gta_shape_t *shape, int32_t pos0, int32_t S_cap,
                                       float rope_base, const void *x, const void *w_qkc,
                                       const void *w_p, const void *w_g, const void *w_o,
                                       void *k_cache, void *c_cache, void *u, void *workspace,
                                       size_t workspace_bytes, int32_t *status_word,
                                       void *cuda_stream);

/*
 * gta_layer_prefill_paged — gta_layer_prefill over a paged cache (pools, block table and their rules as in
 * gta_decode_paged; the capacity of a sequence, page_size * max_pages, takes the place of S_cap): the
 * chunk's keys and latents are written to the rows the block table assigns to positions
 * pos0 .. pos0 + N - 1, and the chunk attends positions 0 .. pos0 + N - 1 as gta_prefill_chunk_paged
 * does.  The block-table entries of positions below pos0 + N are read; a row whose entry lies outside
 * [0, n_pages) is not written and raises *status_word to GTA_ERR_BAD_PAGE.  The caller owns the
 * assignment of pages; two sequences must not be given the same page for the chunk's positions.
 * workspace: gta_layer_prefill_workspace_bytes(shape).  Shapes and errors as gta_layer_prefill, plus
 * GTA_ERR_INVALID_ARG for a bad block table or pool geometry.
 */
GTA_API gta_status_t gta_layer_prefill_paged(const gta_shape_t *shape, int32_t pos0, float rope_base,
                                             const void *x, const void *w_qkc, const void *w_p,
                                             const void *w_g, const void *w_o, void *k_pool,
                                             void *c_pool, const int32_t *block_table,
                                             int32_t page_size, int32_t n_pages, int32_t max_pages,
                                             void *u, void *workspace, size_t workspace_bytes,
                                             int32_t *status_word, void *cuda_stream);

/*
 * gta_layer_decode — one decode step of the whole attention layer (App. B.1.1 for the newest token;
 * cache handling as in App. B.1.3).  For every sequence b, with p = seq_lens[b] the new token's position:
 *
 *   [q | k | c] = x_t[b] W_qkc;  q, k <- RoPE(., position p)        (layouts and RoPE as in gta_layer_prefill)
 *   k_cache[b, :, p, :] = k,  c_cache[b, :, p, :] = c,  seq_lens[b] = p + 1
 *   o = gta_decode over the p + 1 cached tokens, gated by x_t[b];    u[b] = [o_1; ...; o_{n_h}] W_o
 *
 *   x_t [B, H]   u [B, H]   seq_lens device int32 [B] in/out   caches as in gta_decode
 *   workspace: gta_layer_decode_workspace_bytes(shape, S_cap), 256-byte aligned.
 * A sequence with seq_lens[b] outside [0, S_cap) is left as it is (no row written, length unchanged),
 * *status_word is raised to GTA_ERR_CACHE_FULL and its row of u is unspecified.
 * Shapes as gta_layer_prefill (bf16, tensor-core kernels); the decode itself runs on whichever kernel family
 * gta_decode picks for the shape.
 */
GTA_API size_t gta_layer_decode_workspace_bytes(const gta_shape_t *shape, int32_t S_cap);
GTA_API gta_status_t gta_layer_decode(const gta_shape_t *shape, int32_t S_cap, float rope_base,
                                      const void *x_t, const void *w_qkc, const void *w_p,
                                      const void *w_g, const void *w_o, void *k_cache, void *c_cache,
                                      int32_t *seq_lens, void *u, void *workspace,
                                      size_t workspace_bytes, int32_t *status_word, void *cuda_stream);

/*
 * gta_layer_decode_paged — gta_layer_decode over a paged cache (pools, block table and their rules as
 * in gta_decode_paged; the capacity of a sequence is page_size * max_pages).  The new token's key and
 * latent rows go to row p % page_size of page block_table[b, p / page_size], p = seq_lens[b]; an entry
 * outside [0, n_pages) raises GTA_ERR_BAD_PAGE and the row is not written.
 */
GTA_API size_t gta_layer_decode_paged_workspace_bytes(const gta_shape_t *shape, int32_t page_size,
                                                      int32_t max_pages);
GTA_API gta_status_t gta_layer_decode_paged(const gta_shape_t *shape, const int32_t *block_table,
                                            int32_t page_size, int32_t n_pages, int32_t max_pages,
                                            float rope_base, const void *x_t, const void *w_qkc,
                                            const void *w_p, const void *w_g, const void *w_o,
                                            void *k_pool, void *c_pool, int32_t *seq_lens, void *u,
                                            void *workspace, size_t workspace_bytes,
                                            int32_t *status_word, void *cuda_stream);

/*
 * gta_decode_static — gta_decode without a workspace argument (the paper has no counterpart: this
 * is a packaging variant of the same decode step, with the same arguments, results and errors).
 *
 * It is meant for hosts that cannot allocate device memory at the moment a decode step is due,
 * for example a serving process whose memory pool took the whole device at start-up, a plug-in
 * that may not use its host application's allocator, or a loop that cannot afford the device-
 * wide synchronisation an allocation implies.  The split-KV partial results go to a fixed array
 * of GTA_STATIC_SCRATCH_BYTES bytes that is part of the library image: every GPU on which the
 * library is used keeps that much memory until the process exits.  The call itself allocates
 * and frees nothing, on the host runtime or the device.
 *
 *   - A problem whose gta_decode_workspace_bytes() exceeds GTA_STATIC_SCRATCH_BYTES is refused
 *     with GTA_ERR_STATIC_SCRATCH before anything is launched (for the bf16 kernels the need
 *     grows with batch * n_q * d_l, not with the context length).
 *   - Arguments are checked exactly as gta_decode checks them (same order, same codes; an
 *     empty batch returns GTA_OK after those checks), then the size, then the device.
 *   - The first call on each device that gets past those checks looks up the array's device
 *     address (once, with that device current); make that first call outside any stream
 *     capture.
 *   - All calls on a device share the one array and find in it whatever the previous call left;
 *     the kernels write every word before they read it, so nothing needs clearing.  Two calls
 *     that may run on the GPU at the same time (different streams, no ordering) race on it:
 *     order them, or use gta_decode with separate workspaces.
 */
#define GTA_STATIC_SCRATCH_BYTES (16u << 20)
GTA_API gta_status_t gta_decode_static(const gta_shape_t *shape, const void *q, const void *k_cache,
                                       const void *c_cache, const int32_t *seq_lens, int32_t S_cap,
                                       const void *x_t, const void *w_p, const void *w_g, void *out,
                                       int32_t *status_word, void *cuda_stream);

/*
 * gta_decode_append — one decode step including the append of its token (App. B.1.3: the new
 * token's keys and latents join the caches, then its queries attend over all of them):
 * the same result, cache contents, lengths and status as
 *     gta_cache_append(shape, k_cache, c_cache, S_cap, k_new, c_new, 1, seq_lens, ...);
 *     gta_decode(shape, q, k_cache, c_cache, seq_lens, S_cap, x_t, w_p, w_g, out, ...);
 * bit for bit, in one call.  seq_lens (device int32 [B], in / out) does NOT count the new token
 * on entry and does on return; k_new [B, n_k, d_h], c_new [B, n_c, d_l]; a sequence whose cache
 * is full (or whose length is negative) keeps its cache and length, is attended over as it is,
 * and raises GTA_ERR_CACHE_FULL in the status word.  On the bf16 fast path of gta_decode the
 * append costs no kernel of its own: the CTA that streams the end of a sequence puts the new
 * rows over the corresponding rows of its shared-memory tile and writes them to the caches, and
 * the lengths advance in the last kernel of the step, after every reader of them is done.
 * Everywhere else the call runs the two calls above one after the other.  Workspace as for
 * gta_decode.
 */
GTA_API gta_status_t gta_decode_append(const gta_shape_t *shape, const void *q, void *k_cache, void *c_cache,
                                       const void *k_new, const void *c_new, int32_t *seq_lens, int32_t S_cap,
                                       const void *x_t, const void *w_p, const void *w_g, void *out,
                                       void *workspace, size_t workspace_bytes, int32_t *status_word,
                                       void *cuda_stream);

/*
 * gta_decode_hostcache — gta_decode with the K and C caches left in HOST memory (the setting of the paper's
 * offload experiments, Sec. 5.3 and App. C.2: the cache stays in host memory and crosses the host link
 * at every step, so the step is bound by the bytes of the cache all the more).  k_cache and c_cache are
 * addresses of page-locked host memory that the device can read directly (cudaHostAlloc / cudaMallocHost,
 * or cudaHostRegister'ed memory with its device pointer; on a system with unified addressing the host
 * pointer itself); layouts, lengths, all other arguments (device memory as before), result and errors
 * are those of gta_decode.  The cache is read in place with ordinary 16-byte loads by the plain-ALU
 * kernels, every live row exactly once per step: no staging copy and no device memory for the cache.
 * Pageable host memory is not accepted by the hardware: passing it is an error the library cannot
 * detect (the kernel faults).  The call also works on device-resident caches (it is then simply the
 * plain-ALU decode path).  workspace: gta_decode_hostcache_workspace_bytes(shape, S_cap).
 */
GTA_API size_t gta_decode_hostcache_workspace_bytes(const gta_shape_t *shape, int32_t S_cap);
GTA_API gta_status_t gta_decode_hostcache(const gta_shape_t *shape, const void *q, const void *k_cache,
                                          const void *c_cache, const int32_t *seq_lens, int32_t S_cap,
                                          const void *x_t, const void *w_p, const void *w_g, void *out,
                                          void *workspace, size_t workspace_bytes,
                                          int32_t *status_word, void *cuda_stream);

/*
 * 8-bit caches (the paper has no such format; Sec. 5.3 and App. C.2 only observe that the decode
 * step is bound by the bytes of the cache, the larger the context and the slower the memory the
 * more).  Reading taken here: K and C rows are kept as e4m3 codes (8-bit floats: 1 sign, 4
 * exponent, 3 mantissa bits, bias 7, no infinities, largest value 448) with ONE fp32 scale per
 * cached row (token and group):
 *     scale = max|row| / 448 (1 for an all-zero row),  code = round-to-nearest-even(x / scale),
 * both divisions in fp32, magnitudes saturating at 448; the operator runs on code * scale.
 *   k_codes uint8 [B, n_k, S_cap, d_h]   k_scales float [B, n_k, S_cap]
 *   c_codes uint8 [B, n_c, S_cap, d_l]   c_scales float [B, n_c, S_cap]
 * gta_cache_append_fp8 quantises k_new [B, n_k, n_new, d_h] / c_new [B, n_c, n_new, d_l] (in the
 * shape's dtype) into rows [len, len + n_new) and advances seq_lens, with the overflow rule of
 * gta_cache_append; codes and scales are bit-exact functions of the new rows.  gta_decode_fp8 is
 * gta_decode over such caches (q, x_t, w_p, w_g, out in the shape's dtype; rows at and behind
 * seq_lens[b] may hold anything).  Needs d_h and d_l multiples of 16, d_l <= 2048; contiguous
 * caches only.  gta_decode_fp8 has a streaming path (TMA ring, tensor-core MMAs on the e4m3 codes
 * themselves -- tcgen05 with the cached tokens as the MMA rows where every key group has 1, 2, 4 or 8
 * maps, warp-level MMAs otherwise --, query rows and probabilities carried as sums of
 * two e4m3 numbers, merge and tensor-core decoder kernels of gta_decode) for bf16 operator tensors with
 * d_h = 128, one latent group, d_l in {128, 256, 512, 1024}, at most 8 maps over 1, 2, 4 or 8 key groups,
 * S_cap a multiple of 4 and 16-byte aligned scale arrays; everything else, and the append, runs on the
 * plain-ALU kernels.
 * gta_decode_fp8_path says which (0 unsupported, 1 plain-ALU, 2 streaming, alignment aside).
 */
GTA_API size_t gta_decode_fp8_workspace_bytes(const gta_shape_t *shape, int32_t S_cap);
GTA_API int gta_decode_fp8_path(const gta_shape_t *shape, int32_t S_cap);
GTA_API gta_status_t gta_cache_append_fp8(const gta_shape_t *shape, void *k_codes, void *c_codes,
                                          float *k_scales, float *c_scales, int32_t S_cap,
                                          const void *k_new, const void *c_new, int32_t n_new,
                                          int32_t *seq_lens, int32_t *status_word, void *cuda_stream);
GTA_API gta_status_t gta_decode_fp8(const gta_shape_t *shape, const void *q, const void *k_codes,
                                    const void *c_codes, const float *k_scales, const float *c_scales,
                                    const int32_t *seq_lens, int32_t S_cap, const void *x_t,
                                    const void *w_p, const void *w_g, void *out, void *workspace,
                                    size_t workspace_bytes, int32_t *status_word, void *cuda_stream);

/*
 * Comparison operators of the paper, in the same harness: grouped-query attention (App. B.3, "GQA",
 * definition; with n_k_groups = n_heads it is the multi-head attention of Sec. 3.1), so that the
 * ratios the paper states analytically (Table 3; Sec. 4.3: 37.5 % of the attention cost, 30 % of
 * the cache at the 1B hyper-parameters) can be measured on the same kernels:
 *     o[b, i, t] = sum_{j <= t} Softmax_j(q[b, i, t] . k[b, kv(i), j] * scale) v[b, kv(i), j]
 * with kv(i) = floor(i * n_kv / n_h): contiguous blocks of query heads per key / value head, the
 * same reading as for the maps of GTA (App. B.3 prints i mod n_kv, which is this operator with
 * the query heads renumbered).  Of the shape only batch, seq (prefill), n_heads, n_k_groups (the
 * number of key / value heads), head_dim, causal, dtype and softmax_scale are read.
 *   gta_ref_gqa_prefill:  q [B, n_h, N, d_h]; k, v [B, n_kv, N, d_h]; out [B, n_h, N, d_h] (head-major).
 *   gta_ref_gqa_decode:   q [B, n_h, d_h]; k_cache, v_cache [B, n_kv, S_cap, d_h]; seq_lens device
 *     int32 [B] counting the new token (already in the caches); out [B, n_h, d_h]; a sequence of
 *     length 0 gives zeros.  workspace: gta_ref_gqa_decode_workspace_bytes(shape), 256-byte aligned.
 * bf16 with d_h = 64 or 128 only (decode also: at most 8 query heads per key / value head,
 * B * n_kv <= 512); anything else returns GTA_ERR_UNSUPPORTED.  Status word, stream and error
 * behaviour as for gta_prefill / gta_decode.
 */
GTA_API gta_status_t gta_ref_gqa_prefill(const gta_shape_t *shape, const void *q, const void *k, const void *v,
                                         void *out, int32_t *status_word, void *cuda_stream);
GTA_API size_t gta_ref_gqa_decode_workspace_bytes(const gta_shape_t *shape);
GTA_API gta_status_t gta_ref_gqa_decode(const gta_shape_t *shape, const void *q, const void *k_cache,
                                        const void *v_cache, const int32_t *seq_lens, int32_t S_cap,
                                        void *out, void *workspace, size_t workspace_bytes,
                                        int32_t *status_word, void *cuda_stream);

/*
 * Profiling aids (no counterpart in the paper): the same calls restricted to a subset of their
 * kernels, so that each kernel can be timed or captured alone.  `stages` is a bit mask;
 * gta_prefill_stages: 1 = attention kernel (writes L to the workspace), 2 = decoder + gate
 * kernel (reads L from the workspace); gta_decode_stages: 1 = gate partial sums, 2 = split-KV
 * cache kernel, 4 = merge + decoder.  A mask of all stages equals the plain call.  The
 * workspace must still hold what the skipped stages would have written.
 */
GTA_API gta_status_t gta_prefill_stages(const gta_shape_t *shape, const void *q, const void *k,
                                        const void *c, const void *x, const void *w_p, const void *w_g,
                                        void *out, void *workspace, size_t workspace_bytes,
                                        int32_t *status_word, void *cuda_stream, int32_t stages);
GTA_API gta_status_t gta_decode_stages(const gta_shape_t *shape, const void *q, const void *k_cache,
                                       const void *c_cache, const int32_t *seq_lens, int32_t S_cap,
                                       const void *x_t, const void *w_p, const void *w_g, void *out,
                                       void *workspace, size_t workspace_bytes, int32_t *status_word,
                                       void *cuda_stream, int32_t stages);

/* Host helpers. */
GTA_API const char *gta_status_string(gta_status_t status); /* static string, never NULL */
GTA_API int gta_version(void);                              /* major*10000 + minor*100 + patch */

/*
 * Which kernel family gta_prefill would use for `shape` on the current device:
 *   0 = invalid / unsupported, 1 = plain-ALU fp32 kernels, 2 = tcgen05 tensor-core kernels.
 */
GTA_API int gta_prefill_path(const gta_shape_t *shape);

/*
 * Number of kernel launches the last successful call of this thread enqueued (for
 * benchmark accounting; host-side counter only).
 */
GTA_API int gta_last_launch_count(void);

/*
 * Test hook (no counterpart in the paper).  Every wait inside the kernels is bounded: a thread
 * that waits longer than a time limit gives up, tells the other threads of its CTA and of its
 * cluster, the kernel unwinds (outstanding copies and MMAs are waited for, tensor memory is
 * freed), raises GTA_ERR_TIMEOUT in the status word and returns; the context stays usable.
 * This call lets a test exercise that path of the tensor-core attention kernel on a healthy
 * GPU: limit_ns replaces the limit of its waits (0 = the built-in two seconds), and with
 * withhold_first_arrive != 0 one softmax warp of every CTA pair keeps its first arrival to
 * itself, so that the first sum of every pair is never released and the limit runs out.
 * The settings live in device memory of the current device and hold for later launches on it
 * until they are changed back; the call synchronises the device.  Not for production use.
 */
GTA_API gta_status_t gta_debug_attention_wait(uint64_t limit_ns, int32_t withhold_first_arrive);

/*
 * The same test hook for the two decode stream kernels that keep their sums in tensor memory (bf16 caches and 8-bit
 * caches; App. B.1.3 is the step they compute): limit_ns replaces the limit of their waits (0 = the built-in two
 * seconds), and with withhold_first_arrive != 0 one warp of every CTA keeps its first "weights written" arrival to
 * itself, so that the thread that issues the sums runs into the limit; the kernel then unwinds as described above
 * (what it leaves in the workspace and in `out` is meaningless) and raises GTA_ERR_TIMEOUT.  Same lifetime of the
 * settings; the call synchronises the device.  Not for production use.
 */
GTA_API gta_status_t gta_debug_decode_wait(uint64_t limit_ns, int32_t withhold_first_arrive);

#ifdef __cplusplus
}
#endif
#endif /* GTA_H_ */
