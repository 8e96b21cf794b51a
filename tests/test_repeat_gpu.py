"""Run-to-run bit equality of every tensor-core / streaming path.  The kernels hand work between warps, CTAs of a
pair and consecutive kernels through barriers; a hand-off that is out of step shows up as an occasional wrong
tile, not as a wrong average, so each call is repeated many times on the same inputs and every result is
compared, bit for bit, with the first (whose parity against the oracle the other test files establish)."""
import pytest
import torch

from paper_2506_17286_b200 import inputs as I

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2506_17286_b200 import build, binding
    build.build()
    binding.lib()
    return binding


def _repeat(fn, n, what):
    first = None
    for rep in range(n):
        out = fn()
        torch.cuda.synchronize()
        outs = [o.clone() for o in (out if isinstance(out, (list, tuple)) else [out])]
        if first is None:
            first = outs
            continue
        for a, b in zip(outs, first):
            assert torch.equal(a.view(torch.uint8), b.view(torch.uint8)), f"{what}: run {rep} differs from run 0"


PREFILL = [
    # name, B, N, H, n_h, n_q, n_k, n_c, d_h, d_l   (more items than CTA pairs, long and short items mixed)
    ("two_slices", 4, 1024, 256, 8, 4, 4, 1, 128, 512),
    ("four_slices", 2, 768, 256, 8, 4, 4, 1, 128, 1024),
    ("paper_1b_grouping", 4, 1024, 1280, 20, 5, 1, 1, 64, 128),
    ("two_latent_groups", 3, 640, 256, 8, 4, 2, 2, 128, 256),
]


@pytest.mark.parametrize("case", PREFILL, ids=[c[0] for c in PREFILL])
def test_prefill_paths_repeat_bit_for_bit(B, case):
    name, nb, N, H, n_h, n_q, n_k, n_c, d_h, d_l = case
    w = I.Workload(name, "prefill", "bf16", nb, N, H, n_h, n_q, n_k, n_c, d_h, d_l, seed=5)
    t = I.prefill_inputs(w, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    _repeat(lambda: B.gta_prefill(t["q"], t["k"], t["c"], t["x"], t["w_p"], t["w_g"], status_word=status), 60, name)
    n_chunk = 300
    q, x = t["q"][:, :, -n_chunk:].contiguous(), t["x"][:, -n_chunk:].contiguous()
    _repeat(lambda: B.gta_prefill_chunk(q, t["k"], t["c"], x, t["w_p"], t["w_g"], N, status_word=status), 30,
            name + " chunk")
    pg = I.paginate(dict(k_cache=t["k"], c_cache=t["c"]), 64, seed=3)
    _repeat(lambda: B.gta_prefill_chunk_paged(q, pg["k_pool"], pg["c_pool"], pg["block_table"], x, t["w_p"], t["w_g"],
                                              N - 37, status_word=status), 30, name + " paged chunk")
    assert int(status.item()) == 0


def test_layer_prefill_repeats_bit_for_bit(B):
    w = I.Workload("layer", "prefill", "bf16", 2, 640, 512, 8, 4, 4, 1, 128, 512, seed=6)
    t = I.layer_inputs(w, device="cuda")
    k = torch.zeros(2, 4, 700, 128, dtype=torch.bfloat16, device="cuda")
    c = torch.zeros(2, 1, 700, 512, dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    _repeat(lambda: [B.gta_layer_prefill(t["x"], t["w_qkc"], t["w_p"], t["w_g"], t["w_o"], k, c, n_q=4,
                                         status_word=status), k, c], 40, "layer prefill")
    assert int(status.item()) == 0


DECODE = [
    # name, B, H, n_h, n_q, n_k, n_c, d_h, d_l, lens
    ("c3_grouping", 32, 2048, 16, 4, 4, 1, 128, 512, [1500 + 17 * i for i in range(32)]),
    ("paper_1b_grouping", 40, 1280, 20, 5, 1, 1, 64, 128, [(97 * i) % 3000 for i in range(40)]),
    ("eight_maps_dl1024", 16, 512, 16, 8, 8, 1, 128, 1024, [2000 - 100 * i for i in range(16)]),
]


@pytest.mark.parametrize("case", DECODE, ids=[c[0] for c in DECODE])
def test_decode_paths_repeat_bit_for_bit(B, case):
    name, nb, H, n_h, n_q, n_k, n_c, d_h, d_l, lens = case
    w = I.Workload(name, "decode", "bf16", nb, 0, H, n_h, n_q, n_k, n_c, d_h, d_l, seed=7)
    cap = (max(lens) + 68) // 4 * 4
    t = I.decode_inputs(w, device="cuda", s_cap=cap, seq_lens=lens)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    args = (t["x_t"], t["w_p"], t["w_g"])
    _repeat(lambda: B.gta_decode(t["q"], t["k_cache"], t["c_cache"], t["seq_lens"], *args, status_word=status), 80, name)
    k0, c0, l0 = t["k_cache"].clone(), t["c_cache"].clone(), t["seq_lens"].clone()

    def fused_step():
        t["k_cache"].copy_(k0); t["c_cache"].copy_(c0); t["seq_lens"].copy_(l0)
        out = B.gta_decode_append(t["q"], t["k_cache"], t["c_cache"], t["k_new"], t["c_new"], t["seq_lens"], *args,
                                  status_word=status)
        return [out, t["seq_lens"], t["k_cache"], t["c_cache"]]
    _repeat(fused_step, 30, name + " fused step")
    t["k_cache"].copy_(k0); t["c_cache"].copy_(c0); t["seq_lens"].copy_(l0)
    pg = I.paginate(t, 64, seed=1)
    _repeat(lambda: B.gta_decode_paged(t["q"], pg["k_pool"], pg["c_pool"], pg["block_table"], t["seq_lens"], *args,
                                       status_word=status), 30, name + " paged")
    if d_h == 128:      # the streaming kernel for 8-bit caches
        kq = torch.zeros((nb, n_k, cap, d_h), dtype=torch.uint8, device="cuda")
        cq = torch.zeros((nb, n_c, cap, d_l), dtype=torch.uint8, device="cuda")
        ks = torch.ones((nb, n_k, cap), device="cuda")
        cs = torch.ones((nb, n_c, cap), device="cuda")
        for b, n in enumerate(lens):
            if n:
                z = torch.zeros(1, dtype=torch.int32, device="cuda")
                B.gta_cache_append_fp8(kq[b:b + 1], cq[b:b + 1], ks[b:b + 1], cs[b:b + 1],
                                       t["k_cache"][b:b + 1, :, :n].contiguous(), t["c_cache"][b:b + 1, :, :n].contiguous(),
                                       z, status_word=status)
        _repeat(lambda: B.gta_decode_fp8(t["q"], kq, cq, ks, cs, l0, *args, status_word=status), 50, name + " 8-bit caches")
    assert int(status.item()) == 0


def test_comparison_operator_repeats_bit_for_bit(B):
    g = I.gqa_prefill_inputs(2, 8, 2, 512, 128, seed=9, device="cuda")
    _repeat(lambda: B.gta_ref_gqa_prefill(g["q"], g["k"], g["v"]), 40, "gqa prefill")
