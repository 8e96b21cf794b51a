"""Seeded synthetic inputs for the GTA operator (shared by the tests, the benchmark and the
smoke check; read by both the CUDA path and the CPU oracle).

This module holds NONE of the operator's arithmetic: it only draws random tensors with the
shapes, dtypes and value distributions of the five workloads, and lays them out the way the
C-ABI expects.  The upstream input projections (X W_Q, X W_K, X W_C — Sec. 3.2, first
equation) are applied here with plain torch matmuls so that Q, K and C carry the correlation
structure of a real layer; they are outside the operator.

Layouts (row-major): q [B, n_q, N, d_h], k [B, n_k, N, d_h], c [B, n_c, N, d_l], x [B, N, H],
w_p [n_h, d_l, d_h], w_g [H, n_h*d_h]; decode: q [B, n_q, d_h], caches [B, groups, S_cap, d],
x_t [B, H], seq_lens int32 [B].
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    kind: str          # "prefill" | "decode"
    dtype: str         # "f32" | "bf16"
    batch: int
    seq: int           # prefill: N; decode: fixed context (0 = ragged)
    d_model: int
    n_heads: int
    n_q: int
    n_k: int
    n_c: int
    d_h: int
    d_l: int
    ctx_min: int = 0   # ragged decode: context lengths uniform in [ctx_min, ctx_max]
    ctx_max: int = 0
    seed: int = 0

    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16


# The five workloads; "groups" of the workload statement = n_q = n_k, one latent group.
CONFIGS = {
    "c1_tiny_prefill_f32": Workload("c1_tiny_prefill_f32", "prefill", "f32", 1, 128, 256, 4, 2, 2, 1, 64, 128, seed=1001),
    "c2_prefill_bf16": Workload("c2_prefill_bf16", "prefill", "bf16", 4, 2048, 2048, 16, 4, 4, 1, 128, 512, seed=1002),
    "c3_decode_bf16": Workload("c3_decode_bf16", "decode", "bf16", 32, 4096, 2048, 16, 4, 4, 1, 128, 512, seed=1003),
    "c4_long_prefill_bf16": Workload("c4_long_prefill_bf16", "prefill", "bf16", 1, 16384, 4096, 32, 8, 8, 1, 128, 1024, seed=1004),
    "c5_ragged_decode_bf16": Workload("c5_ragged_decode_bf16", "decode", "bf16", 128, 0, 4096, 32, 8, 8, 1, 128, 1024,
                                      ctx_min=1024, ctx_max=32768, seed=1005),
    # beyond the five: the layer shape of the paper's 1B model (20 heads in 5 maps sharing one key
    # group and one latent group, d_h = 64, d_l = 128, H = 1280; cache 192 elements per token)
    "x1_gta1b_prefill_bf16": Workload("x1_gta1b_prefill_bf16", "prefill", "bf16", 8, 2048, 1280, 20, 5, 1, 1, 64, 128, seed=1011),
    "x2_gta1b_decode_bf16": Workload("x2_gta1b_decode_bf16", "decode", "bf16", 128, 8192, 1280, 20, 5, 1, 1, 64, 128, seed=1012),
}


def scaled(w: Workload, **changes) -> Workload:
    """A smaller (or otherwise altered) copy of a workload, for parity cases."""
    return replace(w, **changes)


def _randn(gen, shape, std=1.0):
    return torch.randn(shape, generator=gen, dtype=torch.float32) * std


def prefill_inputs(w: Workload, device="cpu", project: bool = True):
    """Dict of q, k, c, x, w_p, w_g in the workload dtype on `device`.

    x ~ N(0,1); weights ~ N(0, 1/fan_in).  With project=True, q/k/c are x times random
    N(0, 1/H) projection matrices (fp32 matmul, then cast); otherwise they are N(0,1).
    """
    assert w.kind == "prefill"
    gen = torch.Generator("cpu").manual_seed(w.seed)
    dt = w.torch_dtype()
    B, N, H = w.batch, w.seq, w.d_model
    x = _randn(gen, (B, N, H))
    w_p = _randn(gen, (w.n_heads, w.d_l, w.d_h), w.d_l ** -0.5)
    w_g = _randn(gen, (H, w.n_heads * w.d_h), H ** -0.5)
    dev = torch.device(device)

    def grouped(n_groups, d):
        if not project:
            return _randn(gen, (B, n_groups, N, d))
        w_in = _randn(gen, (H, n_groups * d), H ** -0.5).to(dev)
        y = (x.to(dev).reshape(B * N, H) @ w_in).reshape(B, N, n_groups, d)
        return y.permute(0, 2, 1, 3).contiguous()

    q = grouped(w.n_q, w.d_h)
    k = grouped(w.n_k, w.d_h)
    c = grouped(w.n_c, w.d_l)
    out = dict(q=q, k=k, c=c, x=x, w_p=w_p, w_g=w_g)
    return {name: t.to(dev).to(dt).contiguous() for name, t in out.items()}


def decode_seq_lens(w: Workload) -> torch.Tensor:
    """int32 [B] context lengths, counting the token being decoded."""
    gen = torch.Generator("cpu").manual_seed(w.seed + 7)
    if w.seq > 0:
        return torch.full((w.batch,), w.seq, dtype=torch.int32)
    return torch.randint(w.ctx_min, w.ctx_max + 1, (w.batch,), generator=gen, dtype=torch.int32)


def decode_inputs(w: Workload, device="cpu", s_cap: int | None = None, seq_lens=None):
    """Dict of q, k_cache, c_cache, seq_lens, s_cap, x_t, w_p, w_g (+ k_new, c_new for the
    next append).  Caches are N(0,1) everywhere (also beyond seq_lens, so that a kernel that
    reads past the live length is caught); they are drawn on `device`, one sequence at a
    time, from a generator seeded per sequence.
    """
    assert w.kind == "decode"
    gen = torch.Generator("cpu").manual_seed(w.seed)
    dt = w.torch_dtype()
    dev = torch.device(device)
    B, H = w.batch, w.d_model
    lens = decode_seq_lens(w) if seq_lens is None else torch.as_tensor(seq_lens, dtype=torch.int32)
    if s_cap is None:
        s_cap = int(lens.max().item()) + 64 if B > 0 else 64
    q = _randn(gen, (B, w.n_q, w.d_h))
    x_t = _randn(gen, (B, H))
    w_p = _randn(gen, (w.n_heads, w.d_l, w.d_h), w.d_l ** -0.5)
    w_g = _randn(gen, (H, w.n_heads * w.d_h), H ** -0.5)
    k_new = _randn(gen, (B, w.n_k, 1, w.d_h))
    c_new = _randn(gen, (B, w.n_c, 1, w.d_l))
    k_cache = torch.empty((B, w.n_k, s_cap, w.d_h), dtype=dt, device=dev)
    c_cache = torch.empty((B, w.n_c, s_cap, w.d_l), dtype=dt, device=dev)
    dgen = torch.Generator(dev)
    for b in range(B):
        dgen.manual_seed(w.seed * 4096 + b)
        k_cache[b] = torch.randn(k_cache.shape[1:], generator=dgen, dtype=torch.float32, device=dev).to(dt)
        c_cache[b] = torch.randn(c_cache.shape[1:], generator=dgen, dtype=torch.float32, device=dev).to(dt)
    small = dict(q=q, x_t=x_t, w_p=w_p, w_g=w_g, k_new=k_new, c_new=c_new)
    out = {name: t.to(dev).to(dt).contiguous() for name, t in small.items()}
    out.update(k_cache=k_cache, c_cache=c_cache, seq_lens=lens.to(dev), s_cap=s_cap)
    return out


def paginate(t: dict, page_size: int, seed: int = 0, spare_pages: int = 3) -> dict:
    """The decode inputs `t` (from decode_inputs) with the caches laid out as a paged pool.

    Adds k_pool [n_pages, n_k, page_size, d_h], c_pool [n_pages, n_c, page_size, d_l],
    block_table int32 [B, max_pages] and page_size; max_pages = ceil(s_cap / page_size), and token
    t of sequence b sits in row t % page_size of page block_table[b, t // page_size].  The pages of
    all sequences are dealt out by a seeded random permutation of the pool (`spare_pages` pages stay
    unassigned); rows no sequence maps to hold N(0,1) values.  Pure data movement.
    """
    k_cache, c_cache = t["k_cache"], t["c_cache"]
    B, n_k, s_cap, d_h = k_cache.shape
    n_c, d_l = c_cache.shape[1], c_cache.shape[3]
    dev, dt = k_cache.device, k_cache.dtype
    max_pages = max(1, -(-s_cap // page_size))
    n_pages = B * max_pages + spare_pages
    gen = torch.Generator("cpu").manual_seed(seed + 4242)
    table = torch.randperm(n_pages, generator=gen)[: B * max_pages].reshape(B, max_pages).to(torch.int32)
    dgen = torch.Generator(dev).manual_seed(seed + 4243)
    k_pool = torch.randn((n_pages, n_k, page_size, d_h), generator=dgen, dtype=torch.float32, device=dev).to(dt)
    c_pool = torch.randn((n_pages, n_c, page_size, d_l), generator=dgen, dtype=torch.float32, device=dev).to(dt)
    idx = table.to(dev).long()
    for b in range(B):
        for j in range(max_pages):
            lo, hi = j * page_size, min((j + 1) * page_size, s_cap)
            k_pool[idx[b, j], :, : hi - lo] = k_cache[b, :, lo:hi]
            c_pool[idx[b, j], :, : hi - lo] = c_cache[b, :, lo:hi]
    out = dict(t)
    out.update(k_pool=k_pool, c_pool=c_pool, block_table=table.to(dev).contiguous(), page_size=page_size,
               max_pages=max_pages, n_pages=n_pages)
    return out


def layer_inputs(w: Workload, device="cpu"):
    """Dict of x, w_qkc, w_p, w_g, w_o for the whole attention layer, in the workload dtype on `device`.

    x ~ N(0,1); w_qkc [H, (n_q + n_k) d_h + n_c d_l] ~ N(0, 1/H) (the query, key and latent projections side
    by side); w_p, w_g as in prefill_inputs; w_o [n_h d_h, H] ~ N(0, 1/(n_h d_h)).
    """
    assert w.kind == "prefill"
    gen = torch.Generator("cpu").manual_seed(w.seed + 17)
    dt = w.torch_dtype()
    H, D = w.d_model, w.n_heads * w.d_h
    out = dict(
        x=_randn(gen, (w.batch, w.seq, H)),
        w_qkc=_randn(gen, (H, (w.n_q + w.n_k) * w.d_h + w.n_c * w.d_l), H ** -0.5),
        w_p=_randn(gen, (w.n_heads, w.d_l, w.d_h), w.d_l ** -0.5),
        w_g=_randn(gen, (H, D), H ** -0.5),
        w_o=_randn(gen, (D, H), D ** -0.5),
    )
    dev = torch.device(device)
    return {name: t.to(dev).to(dt).contiguous() for name, t in out.items()}


def gqa_prefill_inputs(batch, n_heads, n_kv, seq, d_h, seed=0, device="cpu"):
    """q [B, n_h, N, d_h], k, v [B, n_kv, N, d_h] ~ N(0,1) in bf16 for the comparison operators (drawn on
    `device` from a generator seeded there: the full-size workloads are too large to draw on the host)."""
    dev = torch.device(device)
    gen = torch.Generator(dev).manual_seed(seed)

    def draw(*shape):
        return torch.randn(shape, generator=gen, dtype=torch.float32, device=dev).to(torch.bfloat16)

    return dict(q=draw(batch, n_heads, seq, d_h), k=draw(batch, n_kv, seq, d_h), v=draw(batch, n_kv, seq, d_h))


def gqa_decode_inputs(batch, n_heads, n_kv, d_h, seq_lens, s_cap=None, seed=0, device="cpu"):
    """q [B, n_h, d_h], k_cache, v_cache [B, n_kv, S_cap, d_h] ~ N(0,1) in bf16 (everywhere, also behind the
    live lengths), seq_lens int32 [B]."""
    dev = torch.device(device)
    gen = torch.Generator(dev).manual_seed(seed)
    lens = torch.as_tensor(seq_lens, dtype=torch.int32)
    if s_cap is None:
        s_cap = int(lens.max().item()) + 64

    def draw(*shape):
        return torch.randn(shape, generator=gen, dtype=torch.float32, device=dev).to(torch.bfloat16)

    return dict(q=draw(batch, n_heads, d_h), k_cache=draw(batch, n_kv, s_cap, d_h), v_cache=draw(batch, n_kv, s_cap, d_h),
                seq_lens=lens.to(dev), s_cap=s_cap)
