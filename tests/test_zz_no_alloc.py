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


@pytest.mark.gpu
def test_static_scratch_decode_matches_workspace_decode_twice(B):
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    cases = [
        # B, H, n_h, n_q, n_k, n_c, d_h, d_l, lens, seed      (bf16 streaming kernels, then plain-ALU kernels)
        (5, 256, 8, 4, 4, 1, 128, 512, [1, 63, 64, 65, 700], 21),
        (6, 256, 8, 4, 4, 1, 128, 512, [300, 2, 0, 511, 640, 17], 22),
        (3, 128, 8, 4, 2, 2, 64, 128, [200, 5, 129], 23),
        (3, 128, 8, 4, 2, 2, 64, 128, [7, 260, 33], 24),
    ]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for nb, H, n_h, n_q, n_k, n_c, d_h, d_l, lens, seed in cases:
        w = I.Workload("no_alloc", "decode", "bf16", nb, 0, H, n_h, n_q, n_k, n_c, d_h, d_l, seed=seed)
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
        assert rel <= BF16_REL_L2 and float((g - r).abs().max()) <= BF16_MAX_ABS, (rel, lens)
        # same kernels, same launch shapes, same inputs: in fact bit-identical
        assert torch.equal(got, want)
