"""Thin ctypes binding of the C-ABI library (`include/gta.h`): argument marshalling only.

Every step of the operator runs inside the CUDA library; PyTorch is used for device memory,
streams and host<->device copies.  There is no CPU fallback: if `libgta_b200.so` has not been
built (``python -m paper_2506_17286_b200.build``) every entry point raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgta_b200.so")

GTA_OK, GTA_ERR_INVALID_ARG, GTA_ERR_UNSUPPORTED, GTA_ERR_WORKSPACE = 0, 1, 2, 3
GTA_ERR_CUDA, GTA_ERR_CACHE_FULL, GTA_ERR_TIMEOUT, GTA_ERR_STATIC_SCRATCH = 4, 5, 6, 7
GTA_ERR_BAD_PAGE = 8
STATIC_SCRATCH_BYTES = 16 << 20
GTA_F32, GTA_BF16 = 0, 1

EXPORTS = (
    "gta_prefill_workspace_bytes", "gta_prefill", "gta_decode_workspace_bytes", "gta_decode",
    "gta_cache_append", "gta_status_string", "gta_version", "gta_prefill_path", "gta_last_launch_count",
    "gta_prefill_stages", "gta_decode_stages", "gta_decode_static", "gta_prefill_chunk",
    "gta_decode_paged_workspace_bytes", "gta_decode_paged", "gta_cache_append_paged",
    "gta_layer_prefill_workspace_bytes", "gta_layer_prefill", "gta_layer_decode_workspace_bytes", "gta_layer_decode",
    "gta_layer_decode_paged_workspace_bytes", "gta_layer_decode_paged", "gta_debug_attention_wait",
    "gta_debug_decode_wait",
    "gta_ref_gqa_prefill", "gta_ref_gqa_decode_workspace_bytes", "gta_ref_gqa_decode",
    "gta_decode_fp8_workspace_bytes", "gta_cache_append_fp8", "gta_decode_fp8", "gta_decode_append",
    "gta_prefill_chunk_paged", "gta_layer_prefill_paged", "gta_decode_fp8_path",
    "gta_decode_hostcache_workspace_bytes", "gta_decode_hostcache",
)


class GtaShape(ctypes.Structure):
    """Mirror of gta_shape_t."""
    _fields_ = [
        ("batch", ctypes.c_int32), ("seq", ctypes.c_int32), ("d_model", ctypes.c_int32),
        ("n_heads", ctypes.c_int32), ("n_q_groups", ctypes.c_int32), ("n_k_groups", ctypes.c_int32),
        ("n_c_groups", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("latent_dim", ctypes.c_int32),
        ("causal", ctypes.c_int32), ("dtype", ctypes.c_int32), ("softmax_scale", ctypes.c_float),
    ]


class GtaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


_lib = None


def lib():
    """Load the shared library (once).  Raises if it is missing: there is no fallback."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} not found: build it with `python -m paper_2506_17286_b200.build` "
                "(the GTA operator has no CPU or PyTorch fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
        sp = ctypes.POINTER(GtaShape)
        L.gta_prefill_workspace_bytes.argtypes = [sp]
        L.gta_prefill_workspace_bytes.restype = sz
        L.gta_prefill.argtypes = [sp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp, vp]
        L.gta_prefill.restype = i32
        L.gta_prefill_stages.argtypes = [sp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp, vp, i32]
        L.gta_prefill_stages.restype = i32
        L.gta_prefill_chunk.argtypes = [sp, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp, vp]
        L.gta_prefill_chunk.restype = i32
        L.gta_prefill_chunk_paged.argtypes = [sp, i32, vp, vp, vp, vp, i32, i32, i32, vp, vp, vp, vp, vp, sz, vp, vp]
        L.gta_prefill_chunk_paged.restype = i32
        L.gta_layer_prefill_paged.argtypes = [sp, i32, ctypes.c_float, vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, vp,
                                              vp, sz, vp, vp]
        L.gta_layer_prefill_paged.restype = i32
        L.gta_decode_stages.argtypes = [sp, vp, vp, vp, vp, i32, vp, vp, vp, vp, vp, sz, vp, vp, i32]
        L.gta_decode_stages.restype = i32
        L.gta_decode_workspace_bytes.argtypes = [sp, i32]
        L.gta_decode_workspace_bytes.restype = sz
        L.gta_decode.argtypes = [sp, vp, vp, vp, vp, i32, vp, vp, vp, vp, vp, sz, vp, vp]
        L.gta_decode.restype = i32
        L.gta_decode_hostcache_workspace_bytes.argtypes = [sp, i32]
        L.gta_decode_hostcache_workspace_bytes.restype = sz
        L.gta_decode_hostcache.argtypes = [sp, vp, vp, vp, vp, i32, vp, vp, vp, vp, vp, sz, vp, vp]
        L.gta_decode_hostcache.restype = i32
        L.gta_decode_static.argtypes = [sp, vp, vp, vp, vp, i32, vp, vp, vp, vp, vp, vp]
        L.gta_decode_static.restype = i32
        L.gta_cache_append.argtypes = [sp, vp, vp, i32, vp, vp, i32, vp, vp, vp]
        L.gta_cache_append.restype = i32
        L.gta_decode_paged_workspace_bytes.argtypes = [sp, i32, i32]
        L.gta_decode_paged_workspace_bytes.restype = sz
        L.gta_decode_paged.argtypes = [sp, vp, vp, vp, vp, i32, i32, i32, vp, vp, vp, vp, vp, vp, sz, vp, vp]
        L.gta_decode_paged.restype = i32
        L.gta_cache_append_paged.argtypes = [sp, vp, vp, vp, i32, i32, i32, vp, vp, i32, vp, vp, vp]
        L.gta_cache_append_paged.restype = i32
        L.gta_layer_prefill_workspace_bytes.argtypes = [sp]
        L.gta_layer_prefill_workspace_bytes.restype = sz
        L.gta_layer_prefill.argtypes = [sp, i32, i32, ctypes.c_float, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp, vp]
        L.gta_layer_prefill.restype = i32
        L.gta_layer_decode_workspace_bytes.argtypes = [sp, i32]
        L.gta_layer_decode_workspace_bytes.restype = sz
        L.gta_layer_decode.argtypes = [sp, i32, ctypes.c_float, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp, vp]
        L.gta_layer_decode.restype = i32
        L.gta_layer_decode_paged_workspace_bytes.argtypes = [sp, i32, i32]
        L.gta_layer_decode_paged_workspace_bytes.restype = sz
        L.gta_layer_decode_paged.argtypes = [sp, vp, i32, i32, i32, ctypes.c_float, vp, vp, vp, vp, vp, vp, vp, vp, vp,
                                             vp, sz, vp, vp]
        L.gta_layer_decode_paged.restype = i32
        L.gta_status_string.argtypes = [i32]
        L.gta_status_string.restype = ctypes.c_char_p
        L.gta_version.restype = i32
        L.gta_prefill_path.argtypes = [sp]
        L.gta_prefill_path.restype = i32
        L.gta_last_launch_count.restype = i32
        L.gta_ref_gqa_prefill.argtypes = [sp, vp, vp, vp, vp, vp, vp]
        L.gta_ref_gqa_prefill.restype = i32
        L.gta_ref_gqa_decode_workspace_bytes.argtypes = [sp]
        L.gta_ref_gqa_decode_workspace_bytes.restype = sz
        L.gta_ref_gqa_decode.argtypes = [sp, vp, vp, vp, vp, i32, vp, vp, sz, vp, vp]
        L.gta_ref_gqa_decode.restype = i32
        L.gta_decode_fp8_workspace_bytes.argtypes = [sp, i32]
        L.gta_decode_fp8_workspace_bytes.restype = sz
        L.gta_decode_fp8_path.argtypes = [sp, i32]
        L.gta_decode_fp8_path.restype = i32
        L.gta_cache_append_fp8.argtypes = [sp, vp, vp, vp, vp, i32, vp, vp, i32, vp, vp, vp]
        L.gta_cache_append_fp8.restype = i32
        L.gta_decode_fp8.argtypes = [sp, vp, vp, vp, vp, vp, vp, i32, vp, vp, vp, vp, vp, sz, vp, vp]
        L.gta_decode_fp8.restype = i32
        L.gta_decode_append.argtypes = [sp, vp, vp, vp, vp, vp, vp, i32, vp, vp, vp, vp, vp, sz, vp, vp]
        L.gta_decode_append.restype = i32
        L.gta_debug_attention_wait.argtypes = [ctypes.c_uint64, i32]
        L.gta_debug_attention_wait.restype = i32
        L.gta_debug_decode_wait.argtypes = [ctypes.c_uint64, i32]
        L.gta_debug_decode_wait.restype = i32
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().gta_status_string(int(status)).decode()


def version() -> int:
    return int(lib().gta_version())


def debug_decode_wait(limit_ns: int = 0, withhold_first_arrive: bool = False) -> None:
    """Test hook of the tensor-memory decode stream kernels' bounded waits (see gta_debug_decode_wait in include/gta.h)."""
    st = lib().gta_debug_decode_wait(int(limit_ns), int(bool(withhold_first_arrive)))
    if st != GTA_OK:
        raise GtaError(st, "gta_debug_decode_wait")


def debug_attention_wait(limit_ns: int = 0, withhold_first_arrive: bool = False) -> None:
    """Test hook: time limit of the attention kernel's bounded waits (0 = built-in) and the switch that
    makes the first sum of every CTA pair wait in vain (see gta_debug_attention_wait in include/gta.h)."""
    st = lib().gta_debug_attention_wait(int(limit_ns), int(bool(withhold_first_arrive)))
    if st != GTA_OK:
        raise GtaError(st, "gta_debug_attention_wait")


def last_launch_count() -> int:
    return int(lib().gta_last_launch_count())


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return GTA_F32
    if t.dtype == torch.bfloat16:
        return GTA_BF16
    raise TypeError(f"unsupported dtype {t.dtype}: the library takes float32 or bfloat16")


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _check_tensors(*ts):
    dev, dt = ts[0].device, ts[0].dtype
    for t in ts:
        if t.device != dev or t.dtype != dt:
            raise ValueError("all operator tensors must share one device and one dtype")
        if not t.is_contiguous():
            raise ValueError("operator tensors must be contiguous")
        if t.device.type != "cuda":
            raise ValueError("operator tensors must live on a CUDA device")


def make_shape(*, batch, seq, d_model, n_heads, n_q, n_k, n_c, d_h, d_l, dtype, causal=True,
               softmax_scale=0.0) -> GtaShape:
    code = dtype if isinstance(dtype, int) else (GTA_F32 if dtype == torch.float32 else GTA_BF16)
    return GtaShape(batch, seq, d_model, n_heads, n_q, n_k, n_c, d_h, d_l, int(bool(causal)), code,
                    float(softmax_scale))


def prefill_workspace_bytes(shape: GtaShape) -> int:
    return int(lib().gta_prefill_workspace_bytes(ctypes.byref(shape)))


def decode_workspace_bytes(shape: GtaShape, s_cap: int) -> int:
    return int(lib().gta_decode_workspace_bytes(ctypes.byref(shape), int(s_cap)))


def prefill_path(shape: GtaShape) -> int:
    return int(lib().gta_prefill_path(ctypes.byref(shape)))


def _workspace(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)


def gta_prefill(q, k, c, x, w_p, w_g, *, causal=True, softmax_scale=0.0, out=None, workspace=None,
                status_word=None, stream=None, stages=3):
    """out[B, N, n_h, d_h] = GTA prefill.  q [B,n_q,N,d_h], k [B,n_k,N,d_h], c [B,n_c,N,d_l],
    x [B,N,H], w_p [n_h,d_l,d_h], w_g [H,n_h*d_h]; all on one CUDA device, one dtype."""
    _check_tensors(q, k, c, x, w_p, w_g)
    B, n_q, N, d_h = q.shape
    n_k, n_c, d_l = k.shape[1], c.shape[1], c.shape[3]
    n_h, H = w_p.shape[0], x.shape[2]
    if k.shape != (B, n_k, N, d_h) or c.shape != (B, n_c, N, d_l) or x.shape != (B, N, H) \
            or w_p.shape != (n_h, d_l, d_h) or w_g.shape != (H, n_h * d_h):
        raise ValueError("inconsistent operator tensor shapes")
    shape = make_shape(batch=B, seq=N, d_model=H, n_heads=n_h, n_q=n_q, n_k=n_k, n_c=n_c, d_h=d_h, d_l=d_l,
                       dtype=_dtype_code(q), causal=causal, softmax_scale=softmax_scale)
    if out is None:
        out = torch.empty((B, N, n_h, d_h), dtype=q.dtype, device=q.device)
    need = prefill_workspace_bytes(shape)
    if workspace is None:
        workspace = _workspace(need, q.device)
    args = (ctypes.byref(shape), _ptr(q), _ptr(k), _ptr(c), _ptr(x), _ptr(w_p), _ptr(w_g), _ptr(out),
            _ptr(workspace), workspace.numel() * workspace.element_size(), _ptr(status_word), _stream(stream))
    st = lib().gta_prefill(*args) if stages == 3 else lib().gta_prefill_stages(*args, stages)
    if st != GTA_OK:
        raise GtaError(st, "gta_prefill")
    return out


def gta_prefill_chunk(q, k, c, x, w_p, w_g, kv_len, *, causal=True, softmax_scale=0.0, out=None, workspace=None,
                      status_word=None, stream=None):
    """gta_prefill for the last N of kv_len positions.  q [B,n_q,N,d_h], x [B,N,H]; k [B,n_k,kv_cap,d_h],
    c [B,n_c,kv_cap,d_l] of which rows 0 .. kv_len-1 are attended."""
    _check_tensors(q, k, c, x, w_p, w_g)
    B, n_q, N, d_h = q.shape
    n_k, kv_cap, n_c, d_l = k.shape[1], k.shape[2], c.shape[1], c.shape[3]
    n_h, H = w_p.shape[0], x.shape[2]
    if k.shape != (B, n_k, kv_cap, d_h) or c.shape != (B, n_c, kv_cap, d_l) or x.shape != (B, N, H) \
            or w_p.shape != (n_h, d_l, d_h) or w_g.shape != (H, n_h * d_h):
        raise ValueError("inconsistent operator tensor shapes")
    shape = make_shape(batch=B, seq=N, d_model=H, n_heads=n_h, n_q=n_q, n_k=n_k, n_c=n_c, d_h=d_h, d_l=d_l,
                       dtype=_dtype_code(q), causal=causal, softmax_scale=softmax_scale)
    if out is None:
        out = torch.empty((B, N, n_h, d_h), dtype=q.dtype, device=q.device)
    need = prefill_workspace_bytes(shape)
    if workspace is None:
        workspace = _workspace(need, q.device)
    st = lib().gta_prefill_chunk(ctypes.byref(shape), int(kv_len), int(kv_cap), _ptr(q), _ptr(k), _ptr(c), _ptr(x),
                                 _ptr(w_p), _ptr(w_g), _ptr(out), _ptr(workspace),
                                 workspace.numel() * workspace.element_size(), _ptr(status_word), _stream(stream))
    if st != GTA_OK:
        raise GtaError(st, "gta_prefill_chunk")
    return out


def _check_pools(k_pool, c_pool, block_table):
    if block_table.dtype != torch.int32 or block_table.device != k_pool.device or not block_table.is_contiguous() \
            or block_table.dim() != 2:
        raise ValueError("block_table must be a contiguous int32 [B, max_pages] tensor on the pools' device")
    n_pages, n_k, page_size, d_h = k_pool.shape
    n_c, d_l = c_pool.shape[1], c_pool.shape[3]
    if c_pool.shape != (n_pages, n_c, page_size, d_l):
        raise ValueError("inconsistent pool tensor shapes")
    return n_pages, page_size, block_table.shape[1]


def gta_prefill_chunk_paged(q, k_pool, c_pool, block_table, x, w_p, w_g, kv_len, *, causal=True, softmax_scale=0.0,
                            out=None, workspace=None, status_word=None, stream=None):
    """gta_prefill_chunk over a paged cache: the N queries are the last N of kv_len positions, whose keys and
    latents are read from k_pool [n_pages,n_k,page_size,d_h], c_pool [n_pages,n_c,page_size,d_l] through
    block_table int32 [B,max_pages]."""
    _check_tensors(q, k_pool, c_pool, x, w_p, w_g)
    n_pages, page_size, max_pages = _check_pools(k_pool, c_pool, block_table)
    B, n_q, N, d_h = q.shape
    n_k, n_c, d_l = k_pool.shape[1], c_pool.shape[1], c_pool.shape[3]
    n_h, H = w_p.shape[0], x.shape[2]
    if k_pool.shape[3] != d_h or block_table.shape[0] != B or x.shape != (B, N, H) \
            or w_p.shape != (n_h, d_l, d_h) or w_g.shape != (H, n_h * d_h):
        raise ValueError("inconsistent operator tensor shapes")
    shape = make_shape(batch=B, seq=N, d_model=H, n_heads=n_h, n_q=n_q, n_k=n_k, n_c=n_c, d_h=d_h, d_l=d_l,
                       dtype=_dtype_code(q), causal=causal, softmax_scale=softmax_scale)
    if out is None:
        out = torch.empty((B, N, n_h, d_h), dtype=q.dtype, device=q.device)
    if workspace is None:
        workspace = _workspace(prefill_workspace_bytes(shape), q.device)
    st = lib().gta_prefill_chunk_paged(ctypes.byref(shape), int(kv_len), _ptr(q), _ptr(k_pool), _ptr(c_pool),
                                       _ptr(block_table), page_size, n_pages, max_pages, _ptr(x), _ptr(w_p),
                                       _ptr(w_g), _ptr(out), _ptr(workspace),
                                       workspace.numel() * workspace.element_size(), _ptr(status_word),
                                       _stream(stream))
    if st != GTA_OK:
        raise GtaError(st, "gta_prefill_chunk_paged")
    return out


def gta_layer_prefill_paged(x, w_qkc, w_p, w_g, w_o, k_pool, c_pool, block_table, *, pos0=0, rope_base=10000.0, n_q,
                            softmax_scale=0.0, out=None, workspace=None, status_word=None, stream=None):
    """gta_layer_prefill over a paged cache: the chunk's keys and latents are written to the pages that
    block_table assigns to positions pos0 .. pos0+N-1, and the chunk attends everything up to there."""
    _check_tensors(x, w_qkc, w_p, w_g, w_o, k_pool, c_pool)
    n_pages, page_size, max_pages = _check_pools(k_pool, c_pool, block_table)
    B, N, H = x.shape
    n_h, d_l, d_h = w_p.shape
    n_k, n_c = k_pool.shape[1], c_pool.shape[1]
    if k_pool.shape[3] != d_h or c_pool.shape[3] != d_l or block_table.shape[0] != B \
            or w_qkc.shape != (H, (n_q + n_k) * d_h + n_c * d_l) or w_g.shape != (H, n_h * d_h) \
            or w_o.shape != (n_h * d_h, H):
        raise ValueError("inconsistent layer tensor shapes")
    shape = make_shape(batch=B, seq=N, d_model=H, n_heads=n_h, n_q=n_q, n_k=n_k, n_c=n_c, d_h=d_h, d_l=d_l,
                       dtype=_dtype_code(x), causal=True, softmax_scale=softmax_scale)
    if out is None:
        out = torch.empty((B, N, H), dtype=x.dtype, device=x.device)
    if workspace is None:
        workspace = _workspace(layer_prefill_workspace_bytes(shape), x.device)
    st = lib().gta_layer_prefill_paged(ctypes.byref(shape), int(pos0), float(rope_base), _ptr(x), _ptr(w_qkc),
                                       _ptr(w_p), _ptr(w_g), _ptr(w_o), _ptr(k_pool), _ptr(c_pool),
                                       _ptr(block_table), page_size, n_pages, max_pages, _ptr(out), _ptr(workspace),
                                       workspace.numel() * workspace.element_size(), _ptr(status_word),
                                       _stream(stream))
    if st != GTA_OK:
        raise GtaError(st, "gta_layer_prefill_paged")
    return out


def layer_prefill_workspace_bytes(shape: GtaShape) -> int:
    return int(lib().gta_layer_prefill_workspace_bytes(ctypes.byref(shape)))


def gta_layer_prefill(x, w_qkc, w_p, w_g, w_o, k_cache, c_cache, *, pos0=0, rope_base=10000.0, n_q, softmax_scale=0.0,
                      out=None, workspace=None, status_word=None, stream=None):
    """u[B, N, H] = the whole attention layer for a chunk that starts at position pos0: projections + RoPE, keys
    and latents written to rows pos0 .. pos0+N-1 of the caches, the operator, the output projection.
    x [B,N,H], w_qkc [H,(n_q+n_k)d_h+n_c d_l], w_o [n_h d_h,H], k_cache [B,n_k,S_cap,d_h], c_cache [B,n_c,S_cap,d_l]."""
    _check_tensors(x, w_qkc, w_p, w_g, w_o, k_cache, c_cache)
    B, N, H = x.shape
    n_h, d_l, d_h = w_p.shape
    n_k, s_cap, n_c = k_cache.shape[1], k_cache.shape[2], c_cache.shape[1]
    if k_cache.shape != (B, n_k, s_cap, d_h) or c_cache.shape != (B, n_c, s_cap, d_l) \
            or w_qkc.shape != (H, (n_q + n_k) * d_h + n_c * d_l) or w_g.shape != (H, n_h * d_h) \
            or w_o.shape != (n_h * d_h, H):
        raise ValueError("inconsistent layer tensor shapes")
    shape = make_shape(batch=B, seq=N, d_model=H, n_heads=n_h, n_q=n_q, n_k=n_k, n_c=n_c, d_h=d_h, d_l=d_l,
                       dtype=_dtype_code(x), causal=True, softmax_scale=softmax_scale)
    if out is None:
        out = torch.empty((B, N, H), dtype=x.dtype, device=x.device)
    if workspace is None:
        workspace = _workspace(layer_prefill_workspace_bytes(shape), x.device)
    st = lib().gta_layer_prefill(ctypes.byref(shape), int(pos0), int(s_cap), float(rope_base), _ptr(x), _ptr(w_qkc),
                                 _ptr(w_p), _ptr(w_g), _ptr(w_o), _ptr(k_cache), _ptr(c_cache), _ptr(out),
                                 _ptr(workspace), workspace.numel() * workspace.element_size(), _ptr(status_word),
                                 _stream(stream))
    if st != GTA_OK:
        raise GtaError(st, "gta_layer_prefill")
    return out


def layer_decode_workspace_bytes(shape: GtaShape, s_cap: int) -> int:
    return int(lib().gta_layer_decode_workspace_bytes(ctypes.byref(shape), int(s_cap)))


def gta_layer_decode(x_t, w_qkc, w_p, w_g, w_o, k_cache, c_cache, seq_lens, *, rope_base=10000.0, n_q,
                     softmax_scale=0.0, out=None, workspace=None, status_word=None, stream=None):
    """u[B, H] = one decode step of the whole attention layer: the new token of every sequence is projected,
    rotated at position seq_lens[b], written to the caches (seq_lens advances), attended and projected by w_o."""
    _check_tensors(x_t, w_qkc, w_p, w_g, w_o, k_cache, c_cache)
    if seq_lens.dtype != torch.int32 or seq_lens.device != x_t.device or not seq_lens.is_contiguous():
        raise ValueError("seq_lens must be a contiguous int32 tensor on the operator's device")
    B, H = x_t.shape
    n_h, d_l, d_h = w_p.shape
    n_k, s_cap, n_c = k_cache.shape[1], k_cache.shape[2], c_cache.shape[1]
    if k_cache.shape != (B, n_k, s_cap, d_h) or c_cache.shape != (B, n_c, s_cap, d_l) \
            or w_qkc.shape != (H, (n_q + n_k) * d_h + n_c * d_l) or w_g.shape != (H, n_h * d_h) \
            or w_o.shape != (n_h * d_h, H) or seq_lens.shape != (B,):
        raise ValueError("inconsistent layer tensor shapes")
    shape = make_shape(batch=B, seq=0, d_model=H, n_heads=n_h, n_q=n_q, n_k=n_k, n_c=n_c, d_h=d_h, d_l=d_l,
                       dtype=_dtype_code(x_t), causal=True, softmax_scale=softmax_scale)
    if out is None:
        out = torch.empty((B, H), dtype=x_t.dtype, device=x_t.device)
    if workspace is None:
        workspace = _workspace(layer_decode_workspace_bytes(shape, s_cap), x_t.device)
    st = lib().gta_layer_decode(ctypes.byref(shape), int(s_cap), float(rope_base), _ptr(x_t), _ptr(w_qkc), _ptr(w_p),
                                _ptr(w_g), _ptr(w_o), _ptr(k_cache), _ptr(c_cache), _ptr(seq_lens), _ptr(out),
                                _ptr(workspace), workspace.numel() * workspace.element_size(), _ptr(status_word),
                                _stream(stream))
    if st != GTA_OK:
        raise GtaError(st, "gta_layer_decode")
    return out


def layer_decode_paged_workspace_bytes(shape: GtaShape, page_size: int, max_pages: int) -> int:
    return int(lib().gta_layer_decode_paged_workspace_bytes(ctypes.byref(shape), int(page_size), int(max_pages)))


def gta_layer_decode_paged(x_t, w_qkc, w_p, w_g, w_o, k_pool, c_pool, block_table, seq_lens, *, rope_base=10000.0,
                           n_q, softmax_scale=0.0, out=None, workspace=None, status_word=None, stream=None):
    """gta_layer_decode over a paged cache (pools and block table as in gta_decode_paged)."""
    _check_tensors(x_t, w_qkc, w_p, w_g, w_o, k_pool, c_pool)
    n_pages, page_size, max_pages = _check_paged(k_pool, c_pool, block_table, seq_lens)
    B, H = x_t.shape
    n_h, d_l, d_h = w_p.shape
    n_k, n_c = k_pool.shape[1], c_pool.shape[1]
    if k_pool.shape[3] != d_h or c_pool.shape[3] != d_l or block_table.shape[0] != B \
            or w_qkc.shape != (H, (n_q + n_k) * d_h + n_c * d_l) or w_g.shape != (H, n_h * d_h) \
            or w_o.shape != (n_h * d_h, H):
        raise ValueError("inconsistent layer tensor shapes")
    shape = make_shape(batch=B, seq=0, d_model=H, n_heads=n_h, n_q=n_q, n_k=n_k, n_c=n_c, d_h=d_h, d_l=d_l,
                       dtype=_dtype_code(x_t), causal=True, softmax_scale=softmax_scale)
    if out is None:
        out = torch.empty((B, H), dtype=x_t.dtype, device=x_t.device)
    if workspace is None:
        workspace = _workspace(layer_decode_paged_workspace_bytes(shape, page_size, max_pages), x_t.device)
    st = lib().gta_layer_decode_paged(ctypes.byref(shape), _ptr(block_table), page_size, n_pages, max_pages,
                                      float(rope_base), _ptr(x_t), _ptr(w_qkc), _ptr(w_p), _ptr(w_g), _ptr(w_o),
                                      _ptr(k_pool), _ptr(c_pool), _ptr(seq_lens), _ptr(out), _ptr(workspace),
                                      workspace.numel() * workspace.element_size(), _ptr(status_word), _stream(stream))
    if st != GTA_OK:
        raise GtaError(st, "gta_layer_decode_paged")
    return out


def decode_shape(q, k_cache, c_cache, x_t, w_p, causal=True, softmax_scale=0.0) -> GtaShape:
    B, n_q, d_h = q.shape
    return make_shape(batch=B, seq=0, d_model=x_t.shape[1], n_heads=w_p.shape[0], n_q=n_q,
                      n_k=k_cache.shape[1], n_c=c_cache.shape[1], d_h=d_h, d_l=c_cache.shape[3],
                      dtype=_dtype_code(q), causal=causal, softmax_scale=softmax_scale)


def gta_decode(q, k_cache, c_cache, seq_lens, x_t, w_p, w_g, *, softmax_scale=0.0, out=None, workspace=None,
               status_word=None, stream=None, stages=7):
    """out[B, n_h, d_h] = one decode step.  q [B,n_q,d_h], k_cache [B,n_k,S_cap,d_h],
    c_cache [B,n_c,S_cap,d_l], seq_lens int32 [B] (new token included), x_t [B,H]."""
    _check_tensors(q, k_cache, c_cache, x_t, w_p, w_g)
    if seq_lens.dtype != torch.int32 or seq_lens.device != q.device or not seq_lens.is_contiguous():
        raise ValueError("seq_lens must be a contiguous int32 tensor on the operator's device")
    B, n_q, d_h = q.shape
    s_cap = k_cache.shape[2]
    shape = decode_shape(q, k_cache, c_cache, x_t, w_p, softmax_scale=softmax_scale)
    n_h, d_l, H = shape.n_heads, shape.latent_dim, shape.d_model
    if k_cache.shape != (B, shape.n_k_groups, s_cap, d_h) or c_cache.shape != (B, shape.n_c_groups, s_cap, d_l) \
            or x_t.shape != (B, H) or w_p.shape != (n_h, d_l, d_h) or w_g.shape != (H, n_h * d_h) \
            or seq_lens.shape != (B,):
        raise ValueError("inconsistent operator tensor shapes")
    if out is None:
        out = torch.empty((B, n_h, d_h), dtype=q.dtype, device=q.device)
    if workspace is None:
        workspace = _workspace(decode_workspace_bytes(shape, s_cap), q.device)
    args = (ctypes.byref(shape), _ptr(q), _ptr(k_cache), _ptr(c_cache), _ptr(seq_lens), s_cap, _ptr(x_t),
            _ptr(w_p), _ptr(w_g), _ptr(out), _ptr(workspace), workspace.numel() * workspace.element_size(),
            _ptr(status_word), _stream(stream))
    st = lib().gta_decode(*args) if stages == 7 else lib().gta_decode_stages(*args, stages)
    if st != GTA_OK:
        raise GtaError(st, "gta_decode")
    return out


def decode_hostcache_workspace_bytes(shape: GtaShape, s_cap: int) -> int:
    return int(lib().gta_decode_hostcache_workspace_bytes(ctypes.byref(shape), int(s_cap)))


def gta_decode_hostcache(q, k_cache, c_cache, seq_lens, x_t, w_p, w_g, *, softmax_scale=0.0, out=None, workspace=None,
                         status_word=None, stream=None):
    """gta_decode with k_cache / c_cache in page-locked HOST memory (pinned CPU tensors, read in place over the
    host link; CUDA tensors are accepted too); everything else lives on the device."""
    _check_tensors(q, x_t, w_p, w_g)
    for t in (k_cache, c_cache):
        if t.dtype != q.dtype or not t.is_contiguous():
            raise ValueError("the caches must be contiguous and of the operator's dtype")
        if t.device.type == "cpu" and not t.is_pinned():
            raise ValueError("a cache in host memory must be page-locked (tensor.pin_memory())")
        if t.device.type == "cuda" and t.device != q.device:
            raise ValueError("a cache in device memory must live on the operator's device")
    if seq_lens.dtype != torch.int32 or seq_lens.device != q.device or not seq_lens.is_contiguous():
        raise ValueError("seq_lens must be a contiguous int32 tensor on the operator's device")
    B, n_q, d_h = q.shape
    s_cap = k_cache.shape[2]
    shape = decode_shape(q, k_cache, c_cache, x_t, w_p, softmax_scale=softmax_scale)
    n_h, d_l, H = shape.n_heads, shape.latent_dim, shape.d_model
    if k_cache.shape != (B, shape.n_k_groups, s_cap, d_h) or c_cache.shape != (B, shape.n_c_groups, s_cap, d_l) \
            or x_t.shape != (B, H) or w_p.shape != (n_h, d_l, d_h) or w_g.shape != (H, n_h * d_h) \
            or seq_lens.shape != (B,):
        raise ValueError("inconsistent operator tensor shapes")
    if out is None:
        out = torch.empty((B, n_h, d_h), dtype=q.dtype, device=q.device)
    if workspace is None:
        workspace = _workspace(decode_hostcache_workspace_bytes(shape, s_cap), q.device)
    st = lib().gta_decode_hostcache(ctypes.byref(shape), _ptr(q), _ptr(k_cache), _ptr(c_cache), _ptr(seq_lens), s_cap,
                                    _ptr(x_t), _ptr(w_p), _ptr(w_g), _ptr(out), _ptr(workspace),
                                    workspace.numel() * workspace.element_size(), _ptr(status_word), _stream(stream))
    if st != GTA_OK:
        raise GtaError(st, "gta_decode_hostcache")
    return out


def gta_decode_append(q, k_cache, c_cache, k_new, c_new, seq_lens, x_t, w_p, w_g, *, softmax_scale=0.0, out=None,
                      workspace=None, status_word=None, stream=None):
    """One decode step including the append of its token: k_new [B, n_k, 1, d_h] / c_new [B, n_c, 1, d_l] join the
    caches at row seq_lens[b], seq_lens advances, the new token's queries attend over everything."""
    _check_tensors(q, k_cache, c_cache, k_new, c_new, x_t, w_p, w_g)
    shape = decode_shape(q, k_cache, c_cache, x_t, w_p, softmax_scale=softmax_scale)
    B, n_k, s_cap, d_h = k_cache.shape
    if k_new.numel() != B * n_k * d_h or c_new.numel() != B * c_cache.shape[1] * c_cache.shape[3]:
        raise ValueError("k_new / c_new hold one row per sequence and group")
    if out is None:
        out = torch.empty((B, w_p.shape[0], d_h), dtype=q.dtype, device=q.device)
    if workspace is None:
        workspace = _workspace(decode_workspace_bytes(shape, s_cap), q.device)
    st = lib().gta_decode_append(ctypes.byref(shape), _ptr(q), _ptr(k_cache), _ptr(c_cache), _ptr(k_new), _ptr(c_new),
                                 _ptr(seq_lens), int(s_cap), _ptr(x_t), _ptr(w_p), _ptr(w_g), _ptr(out), _ptr(workspace),
                                 workspace.numel() * workspace.element_size(), _ptr(status_word), _stream(stream))
    if st != GTA_OK:
        raise GtaError(st, "gta_decode_append")
    return out


def gta_decode_static(q, k_cache, c_cache, seq_lens, x_t, w_p, w_g, *, softmax_scale=0.0, out=None,
                      status_word=None, stream=None):
    """gta_decode for callers that cannot allocate device memory (a pool that owns the whole
    device, a plug-in barred from the allocator, a loop that cannot take an allocation's device
    synchronisation): the split-KV scratch is a fixed STATIC_SCRATCH_BYTES array inside the
    library instead of a workspace tensor.  Pass `out`, and nothing is allocated at all.
    Raises GtaError(GTA_ERR_STATIC_SCRATCH) when the problem needs more than the array holds.
    Calls on one device share the array: order them on one stream."""
    _check_tensors(q, k_cache, c_cache, x_t, w_p, w_g)
    if seq_lens.dtype != torch.int32 or seq_lens.device != q.device or not seq_lens.is_contiguous():
        raise ValueError("seq_lens must be a contiguous int32 tensor on the operator's device")
    B, n_q, d_h = q.shape
    s_cap = k_cache.shape[2]
    shape = decode_shape(q, k_cache, c_cache, x_t, w_p, softmax_scale=softmax_scale)
    n_h, d_l, H = shape.n_heads, shape.latent_dim, shape.d_model
    if k_cache.shape != (B, shape.n_k_groups, s_cap, d_h) or c_cache.shape != (B, shape.n_c_groups, s_cap, d_l) \
            or x_t.shape != (B, H) or w_p.shape != (n_h, d_l, d_h) or w_g.shape != (H, n_h * d_h) \
            or seq_lens.shape != (B,):
        raise ValueError("inconsistent operator tensor shapes")
    if out is None:
        out = torch.empty((B, n_h, d_h), dtype=q.dtype, device=q.device)
    st = lib().gta_decode_static(ctypes.byref(shape), _ptr(q), _ptr(k_cache), _ptr(c_cache), _ptr(seq_lens), s_cap,
                                 _ptr(x_t), _ptr(w_p), _ptr(w_g), _ptr(out), _ptr(status_word), _stream(stream))
    if st != GTA_OK:
        raise GtaError(st, "gta_decode_static")
    return out


def gta_cache_append(k_cache, c_cache, k_new, c_new, seq_lens, *, status_word=None, stream=None):
    """In place: rows k_new [B,n_k,n_new,d_h] / c_new [B,n_c,n_new,d_l] go behind seq_lens[b] in the
    caches and seq_lens advances by n_new.  A full sequence is skipped and raises *status_word."""
    _check_tensors(k_cache, c_cache, k_new, c_new)
    if seq_lens.dtype != torch.int32 or seq_lens.device != k_cache.device or not seq_lens.is_contiguous():
        raise ValueError("seq_lens must be a contiguous int32 tensor on the caches' device")
    B, n_k, s_cap, d_h = k_cache.shape
    n_c, d_l = c_cache.shape[1], c_cache.shape[3]
    n_new = k_new.shape[2]
    if c_cache.shape != (B, n_c, s_cap, d_l) or k_new.shape != (B, n_k, n_new, d_h) \
            or c_new.shape != (B, n_c, n_new, d_l) or seq_lens.shape != (B,):
        raise ValueError("inconsistent cache tensor shapes")
    n_q = n_k * n_c // _gcd(n_k, n_c)   # any common multiple serves: append ignores the query groups
    shape = make_shape(batch=B, seq=0, d_model=8, n_heads=n_q, n_q=n_q, n_k=n_k, n_c=n_c, d_h=d_h, d_l=d_l,
                       dtype=_dtype_code(k_cache))
    st = lib().gta_cache_append(ctypes.byref(shape), _ptr(k_cache), _ptr(c_cache), s_cap, _ptr(k_new),
                                _ptr(c_new), n_new, _ptr(seq_lens), _ptr(status_word), _stream(stream))
    if st != GTA_OK:
        raise GtaError(st, "gta_cache_append")
    return seq_lens


def _check_paged(k_pool, c_pool, block_table, seq_lens):
    if block_table.dtype != torch.int32 or block_table.device != k_pool.device or not block_table.is_contiguous() \
            or block_table.dim() != 2:
        raise ValueError("block_table must be a contiguous int32 [B, max_pages] tensor on the pools' device")
    if seq_lens.dtype != torch.int32 or seq_lens.device != k_pool.device or not seq_lens.is_contiguous():
        raise ValueError("seq_lens must be a contiguous int32 tensor on the pools' device")
    n_pages, n_k, page_size, d_h = k_pool.shape
    n_c, d_l = c_pool.shape[1], c_pool.shape[3]
    if c_pool.shape != (n_pages, n_c, page_size, d_l) or seq_lens.shape != (block_table.shape[0],):
        raise ValueError("inconsistent pool tensor shapes")
    return n_pages, page_size, block_table.shape[1]


def decode_paged_workspace_bytes(shape: GtaShape, page_size: int, max_pages: int) -> int:
    return int(lib().gta_decode_paged_workspace_bytes(ctypes.byref(shape), int(page_size), int(max_pages)))


def gta_decode_paged(q, k_pool, c_pool, block_table, seq_lens, x_t, w_p, w_g, *, softmax_scale=0.0, out=None,
                     workspace=None, status_word=None, stream=None):
    """gta_decode over a paged cache.  k_pool [n_pages,n_k,page_size,d_h], c_pool [n_pages,n_c,page_size,d_l],
    block_table int32 [B,max_pages]: token t of sequence b is row t % page_size of page block_table[b, t // page_size]."""
    _check_tensors(q, k_pool, c_pool, x_t, w_p, w_g)
    n_pages, page_size, max_pages = _check_paged(k_pool, c_pool, block_table, seq_lens)
    B, n_q, d_h = q.shape
    shape = decode_shape(q, k_pool, c_pool, x_t, w_p, softmax_scale=softmax_scale)
    n_h, d_l, H = shape.n_heads, shape.latent_dim, shape.d_model
    if k_pool.shape[3] != d_h or x_t.shape != (B, H) or w_p.shape != (n_h, d_l, d_h) \
            or w_g.shape != (H, n_h * d_h) or block_table.shape[0] != B:
        raise ValueError("inconsistent operator tensor shapes")
    if out is None:
        out = torch.empty((B, n_h, d_h), dtype=q.dtype, device=q.device)
    if workspace is None:
        workspace = _workspace(decode_paged_workspace_bytes(shape, page_size, max_pages), q.device)
    st = lib().gta_decode_paged(ctypes.byref(shape), _ptr(q), _ptr(k_pool), _ptr(c_pool), _ptr(block_table),
                                page_size, n_pages, max_pages, _ptr(seq_lens), _ptr(x_t), _ptr(w_p), _ptr(w_g),
                                _ptr(out), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                _ptr(status_word), _stream(stream))
    if st != GTA_OK:
        raise GtaError(st, "gta_decode_paged")
    return out


def gta_cache_append_paged(k_pool, c_pool, block_table, k_new, c_new, seq_lens, *, status_word=None, stream=None):
    """gta_cache_append over a paged cache: the new rows go to the pages the block table names for positions
    seq_lens[b] .. seq_lens[b] + n_new - 1, and seq_lens advances by n_new."""
    _check_tensors(k_pool, c_pool, k_new, c_new)
    n_pages, page_size, max_pages = _check_paged(k_pool, c_pool, block_table, seq_lens)
    B = block_table.shape[0]
    n_k, d_h, n_c, d_l = k_pool.shape[1], k_pool.shape[3], c_pool.shape[1], c_pool.shape[3]
    n_new = k_new.shape[2]
    if k_new.shape != (B, n_k, n_new, d_h) or c_new.shape != (B, n_c, n_new, d_l):
        raise ValueError("inconsistent cache tensor shapes")
    n_q = n_k * n_c // _gcd(n_k, n_c)
    shape = make_shape(batch=B, seq=0, d_model=8, n_heads=n_q, n_q=n_q, n_k=n_k, n_c=n_c, d_h=d_h, d_l=d_l,
                       dtype=_dtype_code(k_pool))
    st = lib().gta_cache_append_paged(ctypes.byref(shape), _ptr(k_pool), _ptr(c_pool), _ptr(block_table), page_size,
                                      n_pages, max_pages, _ptr(k_new), _ptr(c_new), n_new, _ptr(seq_lens),
                                      _ptr(status_word), _stream(stream))
    if st != GTA_OK:
        raise GtaError(st, "gta_cache_append_paged")
    return seq_lens


def _check_fp8_caches(k_codes, c_codes, k_scales, c_scales):
    B, n_k, s_cap, d_h = k_codes.shape
    n_c, d_l = c_codes.shape[1], c_codes.shape[3]
    if k_codes.dtype != torch.uint8 or c_codes.dtype != torch.uint8 or k_scales.dtype != torch.float32 \
            or c_scales.dtype != torch.float32 or c_codes.shape != (B, n_c, s_cap, d_l) \
            or k_scales.shape != (B, n_k, s_cap) or c_scales.shape != (B, n_c, s_cap):
        raise ValueError("8-bit caches: codes uint8 [B, groups, S_cap, width], scales float32 [B, groups, S_cap]")
    for t in (k_codes, c_codes, k_scales, c_scales):
        if not t.is_contiguous() or t.device.type != "cuda":
            raise ValueError("cache tensors must be contiguous CUDA tensors")
    return B, n_k, n_c, s_cap, d_h, d_l


def gta_cache_append_fp8(k_codes, c_codes, k_scales, c_scales, k_new, c_new, seq_lens, *, status_word=None, stream=None):
    """Quantises k_new [B, n_k, n_new, d_h] / c_new [B, n_c, n_new, d_l] to e4m3 codes + per-row scales behind the
    live rows of the 8-bit caches and advances seq_lens."""
    B, n_k, n_c, s_cap, d_h, d_l = _check_fp8_caches(k_codes, c_codes, k_scales, c_scales)
    _check_tensors(k_new, c_new)
    n_new = k_new.shape[2]
    if k_new.shape != (B, n_k, n_new, d_h) or c_new.shape != (B, n_c, n_new, d_l):
        raise ValueError("inconsistent new-row shapes")
    n_q = n_k * n_c          # any map count that both group counts divide: the append does not look at it
    shape = make_shape(batch=B, seq=0, d_model=8, n_heads=n_q, n_q=n_q, n_k=n_k, n_c=n_c, d_h=d_h, d_l=d_l,
                       dtype=_dtype_code(k_new))
    st = lib().gta_cache_append_fp8(ctypes.byref(shape), _ptr(k_codes), _ptr(c_codes), _ptr(k_scales), _ptr(c_scales),
                                    int(s_cap), _ptr(k_new), _ptr(c_new), int(n_new), _ptr(seq_lens), _ptr(status_word),
                                    _stream(stream))
    if st != GTA_OK:
        raise GtaError(st, "gta_cache_append_fp8")
    return seq_lens


def decode_fp8_path(shape: GtaShape, s_cap: int) -> int:
    """0 unsupported, 1 plain-ALU kernels, 2 streaming kernels."""
    return int(lib().gta_decode_fp8_path(ctypes.byref(shape), int(s_cap)))


def decode_fp8_workspace_bytes(shape: GtaShape, s_cap: int) -> int:
    return int(lib().gta_decode_fp8_workspace_bytes(ctypes.byref(shape), int(s_cap)))


def gta_decode_fp8(q, k_codes, c_codes, k_scales, c_scales, seq_lens, x_t, w_p, w_g, *, softmax_scale=0.0, out=None,
                   workspace=None, status_word=None, stream=None):
    """gta_decode over 8-bit caches (e4m3 codes + one fp32 scale per cached row)."""
    B, n_k, n_c, s_cap, d_h, d_l = _check_fp8_caches(k_codes, c_codes, k_scales, c_scales)
    _check_tensors(q, x_t, w_p, w_g)
    n_q, n_h, H = q.shape[1], w_p.shape[0], x_t.shape[1]
    if q.shape != (B, n_q, d_h) or w_p.shape != (n_h, d_l, d_h) or w_g.shape != (H, n_h * d_h) or x_t.shape != (B, H):
        raise ValueError("inconsistent operator tensor shapes")
    shape = make_shape(batch=B, seq=0, d_model=H, n_heads=n_h, n_q=n_q, n_k=n_k, n_c=n_c, d_h=d_h, d_l=d_l,
                       dtype=_dtype_code(q), softmax_scale=softmax_scale)
    if out is None:
        out = torch.empty((B, n_h, d_h), dtype=q.dtype, device=q.device)
    if workspace is None:
        workspace = _workspace(decode_fp8_workspace_bytes(shape, s_cap), q.device)
    st = lib().gta_decode_fp8(ctypes.byref(shape), _ptr(q), _ptr(k_codes), _ptr(c_codes), _ptr(k_scales), _ptr(c_scales),
                              _ptr(seq_lens), int(s_cap), _ptr(x_t), _ptr(w_p), _ptr(w_g), _ptr(out), _ptr(workspace),
                              workspace.numel() * workspace.element_size(), _ptr(status_word), _stream(stream))
    if st != GTA_OK:
        raise GtaError(st, "gta_decode_fp8")
    return out


def gqa_shape(*, batch, seq, n_heads, n_kv, d_h, dtype, causal=True, softmax_scale=0.0) -> GtaShape:
    """Shape of the comparison operators: only batch, seq, n_heads, n_k (key / value heads), d_h are read."""
    return make_shape(batch=batch, seq=seq, d_model=8, n_heads=n_heads, n_q=n_heads, n_k=n_kv, n_c=n_kv, d_h=d_h,
                      d_l=d_h, dtype=dtype, causal=causal, softmax_scale=softmax_scale)


def gta_ref_gqa_prefill(q, k, v, *, causal=True, softmax_scale=0.0, out=None, status_word=None, stream=None):
    """Grouped-query attention (App. B.3 of the paper), the comparison operator: q [B, n_h, N, d_h],
    k, v [B, n_kv, N, d_h] -> out [B, n_h, N, d_h]."""
    _check_tensors(q, k, v)
    B, n_h, N, d_h = q.shape
    n_kv = k.shape[1]
    if k.shape != (B, n_kv, N, d_h) or v.shape != k.shape:
        raise ValueError("inconsistent tensor shapes")
    shape = gqa_shape(batch=B, seq=N, n_heads=n_h, n_kv=n_kv, d_h=d_h, dtype=_dtype_code(q), causal=causal,
                      softmax_scale=softmax_scale)
    if out is None:
        out = torch.empty((B, n_h, N, d_h), dtype=q.dtype, device=q.device)
    st = lib().gta_ref_gqa_prefill(ctypes.byref(shape), _ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(status_word),
                                   _stream(stream))
    if st != GTA_OK:
        raise GtaError(st, "gta_ref_gqa_prefill")
    return out


def gqa_decode_workspace_bytes(shape: GtaShape) -> int:
    return int(lib().gta_ref_gqa_decode_workspace_bytes(ctypes.byref(shape)))


def gta_ref_gqa_decode(q, k_cache, v_cache, seq_lens, *, softmax_scale=0.0, out=None, workspace=None, status_word=None,
                       stream=None):
    """One decode step of grouped-query attention: q [B, n_h, d_h], caches [B, n_kv, S_cap, d_h], seq_lens int32 [B]
    (counting the new token) -> out [B, n_h, d_h]."""
    _check_tensors(q, k_cache, v_cache)
    B, n_h, d_h = q.shape
    n_kv, s_cap = k_cache.shape[1], k_cache.shape[2]
    if k_cache.shape != (B, n_kv, s_cap, d_h) or v_cache.shape != k_cache.shape or seq_lens.shape != (B,) \
            or seq_lens.dtype != torch.int32:
        raise ValueError("inconsistent tensor shapes")
    shape = gqa_shape(batch=B, seq=0, n_heads=n_h, n_kv=n_kv, d_h=d_h, dtype=_dtype_code(q), softmax_scale=softmax_scale)
    if out is None:
        out = torch.empty((B, n_h, d_h), dtype=q.dtype, device=q.device)
    if workspace is None:
        workspace = _workspace(gqa_decode_workspace_bytes(shape), q.device)
    st = lib().gta_ref_gqa_decode(ctypes.byref(shape), _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(seq_lens), int(s_cap),
                                  _ptr(out), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                  _ptr(status_word), _stream(stream))
    if st != GTA_OK:
        raise GtaError(st, "gta_ref_gqa_decode")
    return out


def _gcd(a, b):
    while b:
        a, b = b, a % b
    return a
