"""ctypes front end of the fp64 CPU oracle (``gta_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  It never touches the CUDA library and the CUDA
library never touches it.

Arrays may be numpy arrays (float32 / float64 / uint16 holding bf16 bit patterns)
or torch CPU tensors (float32 / float64 / bfloat16); values are handed to the C
code in their stored form and widened there, exactly, to double.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gta_oracle.c")
_LIB = os.path.join(_HERE, "libgta_oracle.so")

F32, BF16, F64 = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP) next to its source; returns the path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-ftree-vectorize", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


class _Shape(ctypes.Structure):
    _fields_ = [
        ("batch", ctypes.c_int32), ("seq", ctypes.c_int32), ("d_model", ctypes.c_int32),
        ("n_heads", ctypes.c_int32), ("n_q", ctypes.c_int32), ("n_k", ctypes.c_int32),
        ("n_c", ctypes.c_int32), ("d_h", ctypes.c_int32), ("d_l", ctypes.c_int32),
        ("causal", ctypes.c_int32), ("scale", ctypes.c_double),
    ]


@dataclass
class Shape:
    """Operator shape in the paper's symbols (Sec. 3.2): B, N, H, n_h, n_q, n_k, n_c, d_h, d_l."""
    batch: int
    seq: int
    d_model: int
    n_heads: int
    n_q: int
    n_k: int
    n_c: int
    d_h: int
    d_l: int
    causal: int = 1
    scale: float = 0.0

    def c(self) -> _Shape:
        return _Shape(self.batch, self.seq, self.d_model, self.n_heads, self.n_q, self.n_k,
                      self.n_c, self.d_h, self.d_l, self.causal, self.scale)


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        vp, i32, ip = ctypes.c_void_p, ctypes.c_int32, ctypes.POINTER(ctypes.c_int32)
        sp = ctypes.POINTER(_Shape)
        for name in ("gta_oracle_prefill", "gta_oracle_prefill_definition"):
            f = getattr(L, name)
            f.argtypes = [sp, i32, vp, vp, vp, vp, vp, vp, vp, i32, vp, i32]
            f.restype = i32
        L.gta_oracle_probs.argtypes = [sp, i32, vp, vp, vp]
        L.gta_oracle_probs.restype = i32
        L.gta_oracle_decode.argtypes = [sp, i32, vp, vp, vp, vp, i32, vp, vp, vp, vp, i32]
        L.gta_oracle_decode.restype = i32
        L.gta_oracle_cache_append.argtypes = [sp, i32, vp, vp, i32, vp, vp, i32, vp, ip]
        L.gta_oracle_cache_append.restype = i32
        L.gta_oracle_attention_cost.argtypes = [sp]
        L.gta_oracle_attention_cost.restype = ctypes.c_double
        L.gta_oracle_cache_elems.argtypes = [sp]
        L.gta_oracle_cache_elems.restype = ctypes.c_double
        L.gta_oracle_num_threads.restype = i32
        _lib = L
    return _lib


def _as_np(a):
    """torch CPU tensor or numpy array -> (contiguous numpy array, dtype code)."""
    if not isinstance(a, np.ndarray):
        import torch
        assert a.device.type == "cpu", "the oracle reads host memory only"
        a = a.contiguous()
        if a.dtype == torch.bfloat16:
            a = a.view(torch.int16).numpy().view(np.uint16)
        else:
            a = a.numpy()
    a = np.ascontiguousarray(a)
    code = {np.dtype(np.float32): F32, np.dtype(np.uint16): BF16, np.dtype(np.float64): F64}[a.dtype]
    return a, code


def _same_dtype(*arrs):
    conv = [_as_np(a) for a in arrs]
    codes = {c for _, c in conv}
    assert len(codes) == 1, "all operator tensors share one storage type"
    return [a for a, _ in conv], codes.pop()


def _ptr(a):
    return ctypes.c_void_p(a.ctypes.data)


def _check(rc, what):
    if rc != 0:
        raise RuntimeError(f"{what}: oracle returned {rc} (1 = bad argument, 2 = out of memory)")


def num_threads() -> int:
    return int(lib().gta_oracle_num_threads())


def prefill(shape: Shape, q, k, c, x, w_p, w_g, rows=None, n_threads: int = 0, definition=False):
    """out[B, R, n_h, d_h] (float64).  rows=None -> every position (R = N)."""
    (q, k, c, x, w_p, w_g), code = _same_dtype(q, k, c, x, w_p, w_g)
    s = shape
    assert q.size == s.batch * s.n_q * s.seq * s.d_h and k.size == s.batch * s.n_k * s.seq * s.d_h
    assert c.size == s.batch * s.n_c * s.seq * s.d_l and x.size == s.batch * s.seq * s.d_model
    assert w_p.size == s.n_heads * s.d_l * s.d_h and w_g.size == s.d_model * s.n_heads * s.d_h
    if rows is None:
        rows_np, n_rows, R = None, 0, s.seq
    else:
        rows_np = np.ascontiguousarray(np.asarray(rows, dtype=np.int32))
        n_rows = R = int(rows_np.size)
    out = np.zeros((s.batch, R, s.n_heads, s.d_h), dtype=np.float64)
    fn = lib().gta_oracle_prefill_definition if definition else lib().gta_oracle_prefill
    cs = s.c()
    rc = fn(ctypes.byref(cs), code, _ptr(q), _ptr(k), _ptr(c), _ptr(x), _ptr(w_p), _ptr(w_g),
            _ptr(rows_np) if rows_np is not None else None, n_rows, _ptr(out), n_threads)
    _check(rc, "prefill")
    return out


def probs(shape: Shape, q, k):
    """Attention probabilities [B, n_q, N, N] (float64); masked entries are 0."""
    (q, k), code = _same_dtype(q, k)
    s = shape
    out = np.zeros((s.batch, s.n_q, s.seq, s.seq), dtype=np.float64)
    cs = s.c()
    _check(lib().gta_oracle_probs(ctypes.byref(cs), code, _ptr(q), _ptr(k), _ptr(out)), "probs")
    return out


def decode(shape: Shape, q, k_cache, c_cache, seq_lens, s_cap: int, x_t, w_p, w_g, n_threads: int = 0):
    """out[B, n_h, d_h] (float64); seq_lens counts the new token, already appended."""
    (q, k_cache, c_cache, x_t, w_p, w_g), code = _same_dtype(q, k_cache, c_cache, x_t, w_p, w_g)
    s = shape
    assert k_cache.size == s.batch * s.n_k * s_cap * s.d_h
    assert c_cache.size == s.batch * s.n_c * s_cap * s.d_l
    lens = np.ascontiguousarray(np.asarray(seq_lens, dtype=np.int32))
    assert lens.size == s.batch
    out = np.zeros((s.batch, s.n_heads, s.d_h), dtype=np.float64)
    cs = s.c()
    rc = lib().gta_oracle_decode(ctypes.byref(cs), code, _ptr(q), _ptr(k_cache), _ptr(c_cache),
                                 _ptr(lens), s_cap, _ptr(x_t), _ptr(w_p), _ptr(w_g), _ptr(out),
                                 n_threads)
    _check(rc, "decode")
    return out


def cache_append(shape: Shape, k_cache, c_cache, s_cap: int, k_new, c_new, n_new: int, seq_lens):
    """Byte-exact append.  Returns (k_cache, c_cache, seq_lens, overflowed) as NEW numpy arrays."""
    (k_cache, c_cache, k_new, c_new), _ = _same_dtype(k_cache, c_cache, k_new, c_new)
    k_cache, c_cache = k_cache.copy(), c_cache.copy()
    lens = np.ascontiguousarray(np.asarray(seq_lens, dtype=np.int32)).copy()
    flag = ctypes.c_int32(0)
    cs = shape.c()
    rc = lib().gta_oracle_cache_append(ctypes.byref(cs), k_cache.dtype.itemsize, _ptr(k_cache),
                                       _ptr(c_cache), s_cap, _ptr(k_new), _ptr(c_new), n_new,
                                       _ptr(lens), ctypes.byref(flag))
    _check(rc, "cache_append")
    return k_cache, c_cache, lens, int(flag.value)


def paged_view(pool, block_table, page_size: int):
    """The contiguous cache [B, groups, max_pages * page_size, width] that a paged pool
    [n_pages, groups, page_size, width] and a block table [B, max_pages] describe: cached token t
    of sequence b is row t % page_size of page block_table[b, t // page_size] (the caches hold K
    and C of every past token, Sec. 3.3 last paragraph; paging changes where a row lives, not what
    it holds).  Rows under a negative entry stay zero.  Written token by token on purpose."""
    pool, _ = _as_np(pool)
    table = np.asarray(block_table, dtype=np.int64)
    n_seq, max_pages = table.shape
    groups, width = pool.shape[1], pool.shape[3]
    assert pool.shape[2] == page_size
    view = np.zeros((n_seq, groups, max_pages * page_size, width), dtype=pool.dtype)
    for b in range(n_seq):
        for t in range(max_pages * page_size):
            page = table[b, t // page_size]
            if page >= 0:
                view[b, :, t, :] = pool[page, :, t % page_size, :]
    return view


def decode_paged(shape: Shape, q, k_pool, c_pool, block_table, page_size: int, seq_lens, x_t, w_p, w_g,
                 n_threads: int = 0):
    """decode() over a paged cache: the pools are read through paged_view, nothing else changes."""
    k_cache = paged_view(k_pool, block_table, page_size)
    c_cache = paged_view(c_pool, block_table, page_size)
    q, _ = _as_np(q); x_t, _ = _as_np(x_t); w_p, _ = _as_np(w_p); w_g, _ = _as_np(w_g)
    return decode(shape, q, k_cache, c_cache, seq_lens, k_cache.shape[2], x_t, w_p, w_g, n_threads)


def cache_append_paged(k_pool, c_pool, block_table, page_size: int, k_new, c_new, seq_lens):
    """Byte-exact append into a paged cache: new row n of sequence b becomes cached token
    seq_lens[b] + n, i.e. row (seq_lens[b] + n) % page_size of the page the block table names for
    it; a sequence whose new rows would pass max_pages * page_size is skipped whole.  Returns
    (k_pool, c_pool, seq_lens, overflowed) as NEW numpy arrays."""
    (k_pool, c_pool, k_new, c_new), _ = _same_dtype(k_pool, c_pool, k_new, c_new)
    k_pool, c_pool = k_pool.copy(), c_pool.copy()
    table = np.asarray(block_table, dtype=np.int64)
    lens = np.asarray(seq_lens, dtype=np.int32).copy()
    n_new = k_new.shape[2]
    overflowed = 0
    for b in range(table.shape[0]):
        if lens[b] < 0 or lens[b] + n_new > table.shape[1] * page_size:
            overflowed = 1
            continue
        for n in range(n_new):
            t = int(lens[b]) + n
            page = table[b, t // page_size]
            k_pool[page, :, t % page_size, :] = k_new[b, :, n, :]
            c_pool[page, :, t % page_size, :] = c_new[b, :, n, :]
        lens[b] += n_new
    return k_pool, c_pool, lens, overflowed


def _to_f64(a):
    """Operator tensor in any accepted storage form -> float64 numpy array (exact widening)."""
    a, code = _as_np(a)
    if code == BF16:
        return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return a.astype(np.float64)


def round_to_storage(a, storage: int):
    """float64 array rounded to the storage type (round to nearest even), returned as float64: what a
    tensor holds after it has been written to a bf16 / fp32 buffer."""
    a = np.asarray(a, dtype=np.float64)
    if storage == F64:
        return a.copy()
    f = a.astype(np.float32)
    if storage == F32:
        return f.astype(np.float64)
    bits = f.view(np.uint32).astype(np.uint64)
    bits = ((bits + 0x7FFF + ((bits >> 16) & 1)) >> 16) << 16
    return bits.astype(np.uint32).view(np.float32).astype(np.float64)


def rope(v, positions, base: float = 10000.0):
    """Rotary position embedding of RoFormer (the RoPE the layer definition of App. B.1.1 applies to
    q and k): in a vector of even width d, elements (2i, 2i+1) form a pair that is rotated by the
    angle  position * base^(-2i/d).  v [..., N, d] float64, positions [N]."""
    v = np.asarray(v, dtype=np.float64)
    d = v.shape[-1]
    assert d % 2 == 0 and v.shape[-2] == len(positions)
    out = np.empty_like(v)
    for i in range(d // 2):
        theta = base ** (-2.0 * i / d)
        ang = np.asarray(positions, dtype=np.float64) * theta
        x0, x1 = v[..., 2 * i], v[..., 2 * i + 1]
        out[..., 2 * i] = x0 * np.cos(ang) - x1 * np.sin(ang)
        out[..., 2 * i + 1] = x0 * np.sin(ang) + x1 * np.cos(ang)
    return out


def layer_prefill(shape: Shape, x, w_qkc, w_p, w_g, w_o, rope_base: float = 10000.0, storage: int = BF16,
                  n_threads: int = 0, rows=None):
    """The attention layer of App. B.1.1 over a prompt (positions 0 .. N-1):
        q_t, k_t = RoPE(x_t W_Q), RoPE(x_t W_K);  c_t = x_t W_C        (W_qkc = [W_Q | W_K | W_C], groups
                                                                         side by side, d_h / d_h / d_l wide)
        o_t = the operator (prefill) on q, k, c, gated by x_t;          u_t = [o_t,1; ...; o_t,n_h] W_O
    Tensors that the layer stores between its steps (q, the K and C caches, the gated heads) are rounded
    to `storage` there; everything else is float64.  Returns dict(u, q, k, c, o) as float64 arrays:
    u [B, N, H], q [B, n_q, N, d_h], k [B, n_k, N, d_h], c [B, n_c, N, d_l], o [B, N, n_h, d_h].
    rows = a list of token positions: o and u are computed for those positions only ([B, R, ...])."""
    s = shape
    x64, w_qkc, w_o = _to_f64(x), _to_f64(w_qkc), _to_f64(w_o)
    B, N = s.batch, s.seq
    Dq, Dk, Dc = s.n_q * s.d_h, s.n_k * s.d_h, s.n_c * s.d_l
    assert x64.shape == (B, N, s.d_model) and w_qkc.shape == (s.d_model, Dq + Dk + Dc)
    assert w_o.shape == (s.n_heads * s.d_h, s.d_model)
    y = x64 @ w_qkc
    pos = np.arange(N)

    def grouped(cols, groups, width):
        return cols.reshape(B, N, groups, width).transpose(0, 2, 1, 3)

    q = round_to_storage(rope(grouped(y[..., :Dq], s.n_q, s.d_h), pos, rope_base), storage)
    k = round_to_storage(rope(grouped(y[..., Dq:Dq + Dk], s.n_k, s.d_h), pos, rope_base), storage)
    c = round_to_storage(grouped(y[..., Dq + Dk:], s.n_c, s.d_l), storage)
    o = prefill(s, np.ascontiguousarray(q), np.ascontiguousarray(k), np.ascontiguousarray(c), x64,
                _to_f64(w_p), _to_f64(w_g), rows=rows, n_threads=n_threads)
    o = round_to_storage(o, storage)
    u = o.reshape(B, o.shape[1], s.n_heads * s.d_h) @ w_o
    return dict(u=u, q=q, k=k, c=c, o=o)


def attention_cost(shape: Shape) -> float:
    """n_q (d_h + d_l) N^2 — Table 3, GTA row, 'Attention' column."""
    cs = shape.c()
    return float(lib().gta_oracle_attention_cost(ctypes.byref(cs)))


def cache_elems(shape: Shape) -> float:
    """(n_k d_h + n_c d_l) N — Table 3, GTA row, 'KV Cache per Layer' column."""
    cs = shape.c()
    return float(lib().gta_oracle_cache_elems(ctypes.byref(cs)))


# ----------------------------------------------------------------------------------------------
# Comparison operators of the paper: grouped-query attention (App. B.3 "GQA", definition) and, as its
# special case with one key / value head per query head, multi-head attention (Sec. 3.1).  Plain numpy in
# float64, one head and one batch entry at a time, straight from the definition.
def _kv_head(i: int, n_heads: int, n_kv: int, head_map: str) -> int:
    """Key / value head of query head i.  "mod": i mod n_kv, the map App. B.3 prints; "blocks": contiguous
    blocks of n_heads / n_kv query heads per key / value head (the same reading as for the maps of GTA).
    The two differ by a renumbering of the query heads only."""
    assert n_heads % n_kv == 0 and head_map in ("mod", "blocks")
    return i % n_kv if head_map == "mod" else i // (n_heads // n_kv)


def gqa_prefill(q, k, v, causal: bool = True, scale: float = 0.0, head_map: str = "blocks", rows=None):
    """o[b, i, t] = sum_{j <= t} Softmax_j(q[b, i, t] . k[b, kv(i), j] * scale) v[b, kv(i), j]   (App. B.3, GQA,
    attention equation; scale 0 means 1 / sqrt(d_h)).  q [B, n_h, N, d_h]; k, v [B, n_kv, N, d_h];
    returns float64 [B, n_h, N or len(rows), d_h] (head-major)."""
    q, k, v = _to_f64(q), _to_f64(k), _to_f64(v)
    B, n_h, N, d_h = q.shape
    n_kv = k.shape[1]
    assert k.shape == (B, n_kv, N, d_h) and v.shape == (B, n_kv, N, d_h)
    sc = scale if scale > 0 else 1.0 / np.sqrt(d_h)
    ts = list(range(N)) if rows is None else list(rows)
    out = np.zeros((B, n_h, len(ts), d_h))
    for b in range(B):
        for i in range(n_h):
            j = _kv_head(i, n_h, n_kv, head_map)
            for r, t in enumerate(ts):
                last = t if causal else N - 1
                s = (k[b, j, :last + 1] @ q[b, i, t]) * sc
                p = np.exp(s - s.max())
                out[b, i, r] = (p / p.sum()) @ v[b, j, :last + 1]
    return out


def gqa_decode(q, k_cache, v_cache, seq_lens, scale: float = 0.0, head_map: str = "blocks"):
    """One decode step of GQA (App. B.3, decode): the new token's query heads q [B, n_h, d_h] attend the
    seq_lens[b] cached keys / values (the new token's own included); an empty sequence gives zeros.
    k_cache, v_cache [B, n_kv, S_cap, d_h]; returns float64 [B, n_h, d_h]."""
    q, k_cache, v_cache = _to_f64(q), _to_f64(k_cache), _to_f64(v_cache)
    B, n_h, d_h = q.shape
    n_kv = k_cache.shape[1]
    sc = scale if scale > 0 else 1.0 / np.sqrt(d_h)
    out = np.zeros((B, n_h, d_h))
    for b in range(B):
        n = int(seq_lens[b])
        if n <= 0:
            continue
        for i in range(n_h):
            j = _kv_head(i, n_h, n_kv, head_map)
            s = (k_cache[b, j, :n] @ q[b, i]) * sc
            p = np.exp(s - s.max())
            out[b, i] = (p / p.sum()) @ v_cache[b, j, :n]
    return out


def gqa_attention_cost(n_heads: int, d_h: int, n: int) -> float:
    """2 n_h d_h N^2 — Table 3, GQA row, 'Attention' column (App. B.3 prefill)."""
    return 2.0 * n_heads * d_h * float(n) * float(n)


def gqa_cache_elems(n_kv: int, d_h: int, n: int) -> float:
    """2 n_k d_h N — Table 3, GQA row, 'KV Cache per Layer' column (App. B.3 decode)."""
    return 2.0 * n_kv * d_h * float(n)


# ----------------------------------------------------------------------------------------------
# Lower-precision caches (the direction of Sec. 5.3 / App. C.2: decode is bound by the bytes of the cache).
# Reading taken here, the paper fixing none: K and C rows are stored as 8-bit floats of the e4m3 format (1 sign,
# 4 exponent, 3 mantissa bits, bias 7, no infinities, largest finite value 448; the "fn" variant of the OCP 8-bit
# floating point specification) with ONE fp32 scale per cached row (token and group):
#     scale = max|row| / 448   (1 for an all-zero row),   code = round-to-nearest-even_e4m3(x / scale),
# both divisions in fp32, and the operator then runs unchanged on the dequantised values code * scale.
def e4m3_table():
    """Value of each of the 256 e4m3 codes, from the format's definition (codes 0x7f / 0xff are NaN)."""
    vals = np.zeros(256, dtype=np.float64)
    for code in range(256):
        sign = -1.0 if code & 0x80 else 1.0
        e, m = (code >> 3) & 0xF, code & 0x7
        if e == 0xF and m == 0x7:
            vals[code] = np.nan
        elif e == 0:
            vals[code] = sign * (m / 8.0) * 2.0 ** -6          # subnormal
        else:
            vals[code] = sign * (1.0 + m / 8.0) * 2.0 ** (e - 7)
    return vals


def round_to_e4m3(y):
    """fp32 values -> e4m3 codes (uint8): nearest representable value, ties to the even code, magnitudes above 448
    saturate to 448 (no infinities in this format)."""
    y = np.asarray(y, dtype=np.float32)
    mags = e4m3_table()[:0x7F]                        # the 127 finite non-negative values, ascending with the code
    a = np.minimum(np.abs(y).astype(np.float64), 448.0)
    hi = np.clip(np.searchsorted(mags, a, side="left"), 0, 0x7E)
    lo = np.maximum(hi - 1, 0)
    d_hi, d_lo = mags[hi] - a, a - mags[lo]
    pick_lo = (d_lo < d_hi) | ((d_lo == d_hi) & (lo % 2 == 0))
    code = np.where(pick_lo, lo, hi).astype(np.uint8)
    return code | np.where(np.signbit(y), 0x80, 0).astype(np.uint8)


def quantize_rows_e4m3(x):
    """Rows (last axis) of x -> (codes uint8 like x, scales float32 without the last axis)."""
    xf = _to_f64(x).astype(np.float32)                 # the stored values are exact in fp32 (bf16 / fp32 storage)
    amax = np.abs(xf).max(axis=-1)
    scale = np.where(amax > 0, amax / np.float32(448.0), np.float32(1.0)).astype(np.float32)
    return round_to_e4m3(xf / scale[..., None]), scale


def dequantize_e4m3(codes, scales):
    """float64 values code * scale."""
    return e4m3_table()[np.asarray(codes, dtype=np.uint8)] * np.asarray(scales, dtype=np.float64)[..., None]


def cache_append_fp8(k_codes, k_scales, c_codes, c_scales, k_new, c_new, seq_lens):
    """Quantising append: rows [len, len + n_new) of every group of sequence b take the codes and scales of
    k_new [B, n_k, n_new, d_h] / c_new [B, n_c, n_new, d_l]; a sequence whose rows do not fit is skipped (length
    unchanged).  Returns new arrays (k_codes, k_scales, c_codes, c_scales, seq_lens, overflowed)."""
    kc, ks, cc, cs = (np.array(a, copy=True) for a in (k_codes, k_scales, c_codes, c_scales))
    lens = np.array(seq_lens, dtype=np.int32, copy=True)
    kq, kqs = quantize_rows_e4m3(k_new)
    cq, cqs = quantize_rows_e4m3(c_new)
    n_new, cap, overflowed = kq.shape[2], kc.shape[2], 0
    for b in range(kc.shape[0]):
        if lens[b] < 0 or lens[b] + n_new > cap:
            overflowed = 1
            continue
        kc[b, :, lens[b]:lens[b] + n_new] = kq[b]; ks[b, :, lens[b]:lens[b] + n_new] = kqs[b]
        cc[b, :, lens[b]:lens[b] + n_new] = cq[b]; cs[b, :, lens[b]:lens[b] + n_new] = cqs[b]
        lens[b] += n_new
    return kc, ks, cc, cs, lens, overflowed


def decode_fp8(shape: Shape, q, k_codes, k_scales, c_codes, c_scales, seq_lens, x_t, w_p, w_g, n_threads: int = 0):
    """The decode step (App. B.1.3) over caches held as e4m3 codes + per-row scales: dequantise in float64, then
    the unchanged operator oracle.  Rows at and behind seq_lens[b] are never read (they are zeroed here first, so
    that NaN codes or scales there cannot leak through a 0 * NaN)."""
    s_cap = k_codes.shape[2]
    k = dequantize_e4m3(k_codes, k_scales)
    c = dequantize_e4m3(c_codes, c_scales)
    for b in range(shape.batch):
        n = max(0, min(int(seq_lens[b]), s_cap))
        k[b, :, n:] = 0.0
        c[b, :, n:] = 0.0
    return decode(shape, _to_f64(q), np.ascontiguousarray(k), np.ascontiguousarray(c), seq_lens, s_cap, _to_f64(x_t),
                  _to_f64(w_p), _to_f64(w_g), n_threads=n_threads)
