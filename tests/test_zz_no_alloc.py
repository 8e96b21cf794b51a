"""gta_decode_static: the decode step for hosts that cannot allocate device memory (a memory
pool that owns the whole device, a plug-in barred from the allocator, a loop that cannot take
the device synchronisation of an allocation).  Its scratch is a fixed array inside the library,
so this file checks that it gives what gta_decode gives with a caller workspace, twice in a row
on different inputs (the second call finds the first call's leftovers in the array), and that a
problem beyond the array's size is refused on the host.  Collected last on purpose."""
import ctypes

import pytest
import torch

from paper_2506_17286_b200 import inputs as I
from tests.parity_utils import BF16_MAX_ABS, BF16_REL_L2


@pytest.fixture(scope="module")
def B():
    from paper_2506_17286_b200 import build, binding
    build.build()
    binding.lib()
    return binding


def test_oversize_problem_is_refused_on_the_host(B):
    """Needs no GPU: the size check comes before any CUDA call."""
    L = B.lib()
    buf = (ctypes.c_char * 1024)()
    p = ctypes.c_void_p((ctypes.addressof(buf) + 255) & ~255)   # aligned host address, never dereferenced
    big = B.make_shape(batch=4000, seq=0, d_model=4096, n_heads=32, n_q=8, n_k=8, n_c=1, d_h=128, d_l=1024,
                       dtype=B.GTA_F32)
    assert B.decode_workspace_bytes(big, 4096) > B.STATIC_SCRATCH_BYTES
    st = L.gta_decode_static(ctypes.byref(big), p, p, p, p, 4096, p, p, p, p, None, None)
    assert st == B.GTA_ERR_STATIC_SCRATCH
    assert "scratch" in B.status_string(st)
    bad = B.make_shape(batch=2, seq=0, d_model=64, n_heads=4, n_q=3, n_k=1, n_c=1, d_h=32, d_l=64, dtype=B.GTA_BF16)
    assert L.gta_decode_static(ctypes.byref(bad), p, p, p, p, 64, p, p, p, p, None, None) == B.GTA_ERR_INVALID_ARG


def test_bad_arguments_get_the_answer_gta_decode_gives(B):
    """Needs no GPU: every host-side refusal of gta_decode comes back unchanged from gta_decode_static, in the
    same order of checks, and an empty batch is a no-op only after its arguments were looked at."""
    L = B.lib()
    buf = (ctypes.c_char * 1024)()
    p = ctypes.c_void_p((ctypes.addressof(buf) + 255) & ~255)
    odd = ctypes.c_void_p(p.value + 2)
    good = B.make_shape(batch=2, seq=0, d_model=64, n_heads=4, n_q=2, n_k=2, n_c=1, d_h=32, d_l=64, dtype=B.GTA_BF16)

    def both(shape, ptrs=None, s_cap=64):
        a = list(ptrs or [p] * 9)             # q, k_cache, c_cache, seq_lens, x_t, w_p, w_g, out
        sp = ctypes.byref(shape) if shape is not None else None
        st_static = L.gta_decode_static(sp, a[0], a[1], a[2], a[3], s_cap, a[4], a[5], a[6], a[7], None, None)
        st_plain = L.gta_decode(sp, a[0], a[1], a[2], a[3], s_cap, a[4], a[5], a[6], a[7], p, 1 << 40, None, None)
        return st_static, st_plain

    def shape(**kw):
        base = dict(batch=2, seq=0, d_model=64, n_heads=4, n_q=2, n_k=2, n_c=1, d_h=32, d_l=64, dtype=B.GTA_BF16)
        base.update(kw)
        return B.make_shape(**base)

    for sh, ptrs, cap, want in [
        (None, None, 64, B.GTA_ERR_INVALID_ARG),
        (shape(n_q=3), None, 64, B.GTA_ERR_INVALID_ARG),                 # n_q does not divide n_h
        (shape(d_h=20), None, 64, B.GTA_ERR_UNSUPPORTED),                # rows are not 16-byte vectors
        (shape(batch=70000), None, 64, B.GTA_ERR_UNSUPPORTED),
        (shape(d_l=4096), None, 64, B.GTA_ERR_UNSUPPORTED),              # latent row wider than the kernels take
        (good, [None] + [p] * 8, 64, B.GTA_ERR_INVALID_ARG),             # null q
        (good, [odd] + [p] * 8, 64, B.GTA_ERR_INVALID_ARG),              # misaligned q
        (good, None, -1, B.GTA_ERR_INVALID_ARG),
        (shape(batch=0), [odd] + [p] * 8, 64, B.GTA_ERR_INVALID_ARG),    # empty batch: arguments still checked
        (shape(batch=0), None, 64, B.GTA_OK),
    ]:
        st_static, st_plain = both(sh, ptrs, cap)
        assert st_static == st_plain == want, (st_static, st_plain, want)


@pytest.mark.gpu
def test_static_scratch_decode_matches_workspace_decode_twice(B, oracle):
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from tests.parity_utils import assert_close, oracle_shape
    cases = [
        # dtype, B, H, n_h, n_q, n_k, n_c, d_h, d_l, lens, seed
        # the bf16 streaming kernels (split-KV slots, merged latents) ...
        ("bf16", 5, 256, 8, 4, 4, 1, 128, 512, [1, 63, 64, 65, 700], 21),
        ("bf16", 6, 256, 8, 4, 4, 1, 128, 512, [300, 2, 0, 511, 640, 17], 22),
        # ... and the plain-ALU kernels, which lay the scratch out differently (gate sums, per-chunk partials):
        # fp32, a latent width and a map count outside the streaming kernels
        ("f32", 3, 96, 6, 6, 3, 1, 32, 64, [100, 7, 260], 23),
        ("f32", 3, 96, 6, 6, 3, 1, 32, 64, [0, 300, 33], 24),
        ("bf16", 4, 128, 12, 12, 4, 2, 64, 64, [200, 0, 129, 5], 25),
        ("bf16", 4, 128, 12, 12, 4, 2, 64, 64, [7, 260, 33, 64], 26),
    ]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for dt, nb, H, n_h, n_q, n_k, n_c, d_h, d_l, lens, seed in cases:
        w = I.Workload("no_alloc", "decode", dt, nb, 0, H, n_h, n_q, n_k, n_c, d_h, d_l, seed=seed)
        t = I.decode_inputs(w, device="cuda", s_cap=max(lens) + 9, seq_lens=lens)
        args = (t["q"], t["k_cache"], t["c_cache"], t["seq_lens"], t["x_t"], t["w_p"], t["w_g"])
        want = B.gta_decode(*args, status_word=status)
        out = torch.full_like(want, float("nan"))
        got = B.gta_decode_static(*args, out=out, status_word=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        g, r = got.double(), want.double()
        assert torch.isfinite(g).all()
        rel = float((g - r).norm() / r.norm())
        tol_rel, tol_abs = (BF16_REL_L2, BF16_MAX_ABS) if dt == "bf16" else (1e-4, 1e-4 * float(r.abs().max()))
        assert rel <= tol_rel and float((g - r).abs().max()) <= tol_abs, (rel, lens)
        # same kernels, same launch shapes, same inputs: in fact bit-identical
        assert torch.equal(got, want)
        # and the answer is the operator's: the fp64 oracle on the same inputs
        cap = max(lens)
        ref = oracle.decode(oracle_shape(w, seq=0), t["q"].cpu(), t["k_cache"][:, :, :cap].contiguous().cpu(),
                            t["c_cache"][:, :, :cap].contiguous().cpu(), t["seq_lens"].cpu().numpy(), cap,
                            t["x_t"].cpu(), t["w_p"].cpu(), t["w_g"].cpu())
        assert_close(got, ref, w.torch_dtype(), f"gta_decode_static {dt} {lens}")
