"""GPU parity of the decode step over caches that stay in page-locked HOST memory (gta_decode_hostcache): the
kernels read the cache rows in place over the host link; where a row lives does not change what the operator
computes, so the oracle is the decode oracle itself."""
import pytest
import torch

from paper_2506_17286_b200 import inputs as I
from tests.parity_utils import Guarded, assert_close, oracle_shape

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2506_17286_b200 import build, binding
    build.build()
    binding.lib()
    return binding


def _pinned(t):
    """A page-locked host copy; the rows behind the live lengths are overwritten with NaN by the caller."""
    h = torch.empty(t.shape, dtype=t.dtype, pin_memory=True)
    h.copy_(t)
    return h


def _case(B, oracle, w, lens, sample=None):
    cap = max(lens) + 5
    t = I.decode_inputs(w, device="cuda", s_cap=cap, seq_lens=lens)
    k_host, c_host = _pinned(t["k_cache"]), _pinned(t["c_cache"])
    for b, n in enumerate(lens):                         # what uninitialised memory may hold behind the live rows
        k_host[b, :, n:] = float("nan")
        c_host[b, :, n:] = float("nan")
    assert k_host.is_pinned() and c_host.is_pinned() and k_host.device.type == "cpu"
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    shape = B.decode_shape(t["q"], k_host, c_host, t["x_t"], t["w_p"])
    ws = Guarded((B.decode_hostcache_workspace_bytes(shape, cap),), torch.uint8)
    og = Guarded((w.batch, w.n_heads, w.d_h), w.torch_dtype())
    out = B.gta_decode_hostcache(t["q"], k_host, c_host, t["seq_lens"], t["x_t"], t["w_p"], t["w_g"], out=og.t,
                                 workspace=ws.t, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ws.check(w.name + " workspace"); og.check(w.name + " out")
    # the same call on device-resident copies of the same bytes: same kernels, same result bit for bit
    out_dev = B.gta_decode_hostcache(t["q"], k_host.cuda(), c_host.cuda(), t["seq_lens"], t["x_t"], t["w_p"], t["w_g"])
    torch.cuda.synchronize()
    assert torch.equal(out, out_dev)
    idx = list(range(w.batch)) if sample is None else sample
    sel = torch.as_tensor(idx, dtype=torch.long)
    sub_lens = [lens[i] for i in idx]
    sub_cap = max(sub_lens) if sub_lens else 0
    ws_ = I.scaled(w, batch=len(idx))
    want = oracle.decode(oracle_shape(ws_, seq=0), t["q"][sel.cuda()].cpu(),
                         t["k_cache"][sel.cuda()][:, :, :sub_cap].contiguous().cpu(),
                         t["c_cache"][sel.cuda()][:, :, :sub_cap].contiguous().cpu(), sub_lens, sub_cap,
                         t["x_t"][sel.cuda()].cpu(), t["w_p"].cpu(), t["w_g"].cpu())
    return assert_close(out[sel.cuda()], want, w.torch_dtype(), w.name)


HOST_CASES = [
    # name, dtype, B, H, n_h, n_q, n_k, n_c, d_h, d_l, lens
    ("bf16_ragged_c3_grouping", "bf16", 5, 256, 8, 4, 4, 1, 128, 512, [1, 63, 64, 65, 700]),
    ("bf16_empty_and_shared_keys", "bf16", 4, 128, 8, 4, 2, 2, 64, 128, [0, 512, 1, 300]),
    ("bf16_paper_1b_grouping", "bf16", 2, 1280, 20, 5, 1, 1, 64, 128, [333, 1000]),
    ("f32_general", "f32", 3, 96, 6, 6, 3, 1, 32, 64, [100, 7, 260]),
    # more maps on one key / latent group than one pass of the kernel holds (8): two passes, the second ragged
    ("bf16_twelve_maps_one_group", "bf16", 2, 128, 12, 12, 1, 1, 64, 128, [130, 77]),
    # three maps per latent group (a ragged pass of four) and key rows of two 16-byte vectors per lane
    ("f32_wide_heads_three_maps_per_latent", "f32", 2, 64, 6, 6, 2, 2, 256, 256, [50, 129]),
]


@pytest.mark.parametrize("case", HOST_CASES, ids=[c[0] for c in HOST_CASES])
def test_decode_over_caches_in_pinned_host_memory(B, oracle, case):
    name, dt, nb, H, n_h, n_q, n_k, n_c, d_h, d_l, lens = case
    w = I.Workload(name, "decode", dt, nb, 0, H, n_h, n_q, n_k, n_c, d_h, d_l, seed=81)
    _case(B, oracle, w, lens)


def test_decode_hostcache_config3_shape_sampled_sequences(B, oracle):
    """The decode workload's shape at a quarter of its context (67 MB of cache in host memory)."""
    w = I.CONFIGS["c3_decode_bf16"]
    _case(B, oracle, w, [1024] * w.batch, sample=[0, 13, 31])


def test_binding_refuses_pageable_host_memory(B):
    w = I.Workload("pageable", "decode", "bf16", 2, 0, 128, 4, 2, 2, 1, 64, 128, seed=82)
    t = I.decode_inputs(w, device="cuda", s_cap=40, seq_lens=[7, 30])
    with pytest.raises(ValueError, match="page-locked"):
        B.gta_decode_hostcache(t["q"], t["k_cache"].cpu(), t["c_cache"].cpu(), t["seq_lens"], t["x_t"], t["w_p"],
                               t["w_g"])
