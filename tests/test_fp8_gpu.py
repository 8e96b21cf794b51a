"""GPU parity of the 8-bit caches (e4m3 codes + one fp32 scale per cached row): the quantising append is a
bit-exact function of the new rows, the decode step over such caches matches the fp64 oracle on the dequantised
values within the bf16 bounds."""
import numpy as np
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


@pytest.mark.parametrize("dt", ["bf16", "f32"])
@pytest.mark.parametrize("n_new", [1, 3, 300])
def test_quantising_append_is_bit_exact(B, oracle, dt, n_new):
    tdt = torch.bfloat16 if dt == "bf16" else torch.float32
    nb, n_k, n_c, d_h, d_l, cap = 6, 4, 2, 64, 128, 512
    g = torch.Generator("cpu").manual_seed(31 + n_new)
    k_new = (torch.randn(nb, n_k, n_new, d_h, generator=g) * 3).to(tdt)
    c_new = torch.randn(nb, n_c, n_new, d_l, generator=g).to(tdt)
    k_new[0, 0, 0] = 0                                   # an all-zero row keeps scale 1
    c_new[1, 1, n_new - 1, 5] = 1000.0                   # one dominant element
    k_codes = torch.randint(0, 255, (nb, n_k, cap, d_h), generator=g, dtype=torch.uint8)
    c_codes = torch.randint(0, 255, (nb, n_c, cap, d_l), generator=g, dtype=torch.uint8)
    k_scales = torch.rand(nb, n_k, cap, generator=g)
    c_scales = torch.rand(nb, n_c, cap, generator=g)
    lens = torch.tensor([0, 1, cap - n_new, cap - n_new + 1, cap, 17], dtype=torch.int32)   # two do not fit
    want = oracle.cache_append_fp8(k_codes.numpy(), k_scales.numpy(), c_codes.numpy(), c_scales.numpy(), k_new, c_new,
                                   lens.numpy())
    dev = [t.cuda() for t in (k_codes, c_codes, k_scales, c_scales)]
    lens_d = lens.cuda()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.gta_cache_append_fp8(*dev, k_new.cuda(), c_new.cuda(), lens_d, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == B.GTA_ERR_CACHE_FULL
    assert lens_d.cpu().numpy().tolist() == want[4].tolist()
    for got, ref, what in zip(dev, (want[0], want[2], want[1], want[3]), ("k codes", "c codes", "k scales", "c scales")):
        g_ = got.cpu().numpy()
        if g_.dtype == np.float32:                       # compared as bit patterns
            assert np.array_equal(g_.view(np.uint32), np.asarray(ref, dtype=np.float32).view(np.uint32)), what
        else:
            # -0 and +0 are the same stored value as far as the operator goes, the codes 0x00 / 0x80 are not:
            # the cast keeps the sign of a value that rounds to zero, and so does the oracle
            assert np.array_equal(g_, ref), what


def _decode_case(B, oracle, w, lens, sample=None, cap=None, path=None, reshape_keys=None):
    nb = w.batch
    cap = cap or max(lens) + 7
    t = I.decode_inputs(w, device="cuda", s_cap=cap, seq_lens=lens)
    if reshape_keys is not None:
        reshape_keys(t)
    kq, ks = oracle.quantize_rows_e4m3(t["k_cache"].cpu())
    cq, cs = oracle.quantize_rows_e4m3(t["c_cache"].cpu())
    for b, n in enumerate(lens):                          # what uninitialised memory may hold behind the live rows
        kq[b, :, n:] = 0x7F; cq[b, :, n:] = 0xFF; ks[b, :, n:] = np.nan; cs[b, :, n:] = np.inf
    dev = [torch.from_numpy(a).cuda() for a in (kq, cq, ks, cs)]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    shape = B.decode_shape(t["q"], t["k_cache"], t["c_cache"], t["x_t"], t["w_p"])
    if path is not None:
        assert B.decode_fp8_path(shape, cap) == path
    ws = Guarded((B.decode_fp8_workspace_bytes(shape, cap),), torch.uint8)
    og = Guarded((nb, w.n_heads, w.d_h), w.torch_dtype())
    out = B.gta_decode_fp8(t["q"], *dev, t["seq_lens"], t["x_t"], t["w_p"], t["w_g"], out=og.t, workspace=ws.t,
                           status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ws.check("fp8 decode workspace"); og.check("fp8 decode out")
    idx = list(range(nb)) if sample is None else sample
    ws_ = I.scaled(w, batch=len(idx))
    want = oracle.decode_fp8(oracle_shape(ws_, seq=0), t["q"][idx].cpu(), kq[idx], ks[idx], cq[idx], cs[idx],
                             [lens[i] for i in idx], t["x_t"][idx].cpu(), t["w_p"].cpu(), t["w_g"].cpu())
    return assert_close(out[idx], want, w.torch_dtype(), w.name)


FP8_DECODE = [
    # name, dtype, B, H, n_h, n_q, n_k, n_c, d_h, d_l, lens
    ("bf16_ragged", "bf16", 5, 256, 8, 4, 4, 1, 128, 512, [1, 63, 64, 65, 700]),
    ("bf16_empty_and_shared_keys", "bf16", 4, 128, 8, 4, 2, 2, 64, 128, [0, 512, 1, 300]),
    ("bf16_paper_1b_shape", "bf16", 2, 1280, 20, 5, 1, 1, 64, 128, [333, 1000]),
    ("f32_general", "f32", 3, 96, 6, 6, 3, 1, 32, 64, [100, 7, 260]),
    ("bf16_dl1024_eight_maps", "bf16", 3, 512, 16, 8, 8, 1, 128, 1024, [257, 1, 1000]),
]


@pytest.mark.parametrize("case", FP8_DECODE, ids=[c[0] for c in FP8_DECODE])
def test_fp8_decode_small_shapes(B, oracle, case):
    name, dt, nb, H, n_h, n_q, n_k, n_c, d_h, d_l, lens = case
    w = I.Workload(name, "decode", dt, nb, 0, H, n_h, n_q, n_k, n_c, d_h, d_l, seed=61)
    _decode_case(B, oracle, w, lens)


FP8_STREAM = [
    # name, B, H, n_h, n_q, n_k, d_l, lens, cap  (bf16, d_h = 128, one latent group: the streaming kernels)
    ("ragged_64_token_subtiles", 5, 256, 8, 4, 4, 512, [1, 63, 64, 65, 700], 708),
    ("dl1024_eight_maps_32_token_subtiles", 3, 512, 16, 8, 8, 1024, [257, 1, 1000], 1004),
    ("dl128_five_maps_one_key_group", 2, 1280, 10, 5, 1, 128, [333, 1000], 1024),
    ("dl256_empty_sequences_shared_keys", 6, 256, 8, 4, 2, 256, [0, 512, 1, 0, 300, 33], 512),
    ("one_map_full_cache", 2, 128, 2, 1, 1, 256, [256, 255], 256),
    ("many_sequences", 150, 256, 8, 4, 4, 512, [((7 * i) % 130) for i in range(150)], 132),
    # the remaining (key groups, maps per group) instantiations of the tensor-memory kernel
    ("eight_maps_one_key_group_dl128", 4, 256, 8, 8, 1, 128, [640, 64, 129, 1], 640),
    ("eight_maps_two_key_groups_dl256", 3, 256, 8, 8, 2, 256, [500, 0, 191], 512),
    ("eight_maps_four_key_groups_dl512", 3, 256, 8, 8, 4, 512, [320, 65, 128], 320),
    ("two_maps_two_key_groups_dl128", 5, 128, 4, 2, 2, 128, [1, 2, 63, 300, 64], 304),
    ("two_maps_one_key_group_dl512", 2, 128, 4, 2, 1, 512, [200, 450], 452),
    ("four_maps_one_key_group_dl256", 3, 128, 8, 4, 1, 256, [1000, 7, 128], 1000),
    ("long_sequences_many_subtiles_per_cta", 2, 256, 8, 4, 4, 512, [20000, 12345], 20000),
    # 32-token sub-tiles (a token wider than 1 KB): four key groups on the rows of a score MMA, up to two such sets
    ("dl1024_eight_maps_four_key_groups", 3, 512, 16, 8, 4, 1024, [257, 1, 1000], 1004),
    ("dl1024_four_maps_four_key_groups", 3, 256, 8, 4, 4, 1024, [300, 31, 33], 304),
    ("dl1024_eight_maps_two_key_groups", 2, 256, 8, 8, 2, 1024, [129, 64], 132),
    ("dl1024_eight_maps_one_key_group", 2, 256, 8, 8, 1, 1024, [200, 95], 200),
    ("dl512_eight_key_groups", 3, 512, 16, 8, 8, 512, [100, 0, 333], 336),
    ("dl128_eight_key_groups", 2, 512, 8, 8, 8, 128, [70, 33], 72),
    ("dl256_eight_key_groups", 2, 512, 8, 8, 8, 256, [31, 260], 260),
    ("dl1024_one_map", 2, 128, 2, 1, 1, 1024, [150, 33], 152),
    ("dl1024_four_maps_one_key_group", 2, 128, 4, 4, 1, 1024, [64, 97], 100),
    ("dl1024_two_maps_two_key_groups", 2, 128, 4, 2, 2, 1024, [200, 32], 200),
    ("dl1024_four_maps_two_key_groups", 2, 128, 4, 4, 2, 1024, [129, 1], 132),
    ("batch_400_many_empty", 400, 256, 8, 4, 4, 512, [0 if i % 7 == 3 else 1 + (13 * i) % 70 for i in range(400)], 72),
    ("all_sequences_empty", 6, 256, 8, 4, 4, 512, [0, 0, 0, 0, 0, 0], 64),
]


@pytest.mark.parametrize("case", FP8_STREAM, ids=[c[0] for c in FP8_STREAM])
def test_fp8_decode_streaming_kernels(B, oracle, case):
    name, nb, H, n_h, n_q, n_k, d_l, lens, cap = case
    w = I.Workload(name, "decode", "bf16", nb, 0, H, n_h, n_q, n_k, 1, 128, d_l, seed=63)
    rel, mx = _decode_case(B, oracle, w, lens, cap=cap, path=2)
    print(f"\n{name}: rel-L2 {rel:.3e} max-abs {mx:.3e}")


@pytest.mark.parametrize("slope", [0.002, 0.02, -0.004])
def test_fp8_decode_scores_that_keep_rising_or_falling(B, oracle, slope):
    """Keys that point along their map's query with a length that grows (or shrinks) with the position: the reference
    maximum of the softmax is raised at almost every sub-tile (slope 0.002: by about two binary orders per sub-tile,
    0.02: by twenty) or set once and never again (negative slope), so the rescaling of the sums kept in tensor memory,
    the lag of the reference and weights that underflow are all exercised."""
    w = I.Workload("rising", "decode", "bf16", 3, 0, 256, 8, 4, 4, 1, 128, 512, seed=64)
    lens = [1000, 700, 130]

    def keys_along_queries(t):
        q = t["q"].float()                                   # [B, n_q, d_h]; one map per key group here
        pos = torch.arange(t["k_cache"].shape[2], device=q.device, dtype=torch.float32)
        length = slope * pos if slope > 0 else 4.0 + slope * pos
        noise = t["k_cache"].float() * 0.05
        t["k_cache"].copy_((q[:, :, None, :] * length[None, None, :, None] + noise).to(t["k_cache"].dtype))
    rel, mx = _decode_case(B, oracle, w, lens, cap=1000, path=2, reshape_keys=keys_along_queries)
    print(f"\nslope {slope}: rel-L2 {rel:.3e} max-abs {mx:.3e}")


def test_a_wait_that_runs_out_unwinds_the_fp8_stream_kernel(B, oracle):
    """One warp of every CTA keeps its first "weights written" arrival to itself and the waits give up after 2 ms:
    the call comes back with GTA_ERR_TIMEOUT, and the next ordinary call gives bit for bit what the call before gave."""
    w = I.Workload("timeout8", "decode", "bf16", 3, 0, 256, 8, 4, 4, 1, 128, 512, seed=65)
    lens, cap = [200, 64, 33], 208
    t = I.decode_inputs(w, device="cuda", s_cap=cap, seq_lens=lens)
    kq, ks = oracle.quantize_rows_e4m3(t["k_cache"].cpu())
    cq, cs = oracle.quantize_rows_e4m3(t["c_cache"].cpu())
    dev = [torch.from_numpy(a).cuda() for a in (kq, cq, ks, cs)]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    args = (t["q"], *dev, t["seq_lens"], t["x_t"], t["w_p"], t["w_g"])
    shape = B.decode_shape(t["q"], t["k_cache"], t["c_cache"], t["x_t"], t["w_p"])
    assert B.decode_fp8_path(shape, cap) == 2
    before = B.gta_decode_fp8(*args, status_word=status).clone()
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    B.debug_decode_wait(limit_ns=2_000_000, withhold_first_arrive=True)
    try:
        junk = B.gta_decode_fp8(*args, status_word=status)
        torch.cuda.synchronize()                      # returns: every wait is bounded
        assert int(status.item()) == B.GTA_ERR_TIMEOUT
        del junk
    finally:
        B.debug_decode_wait(limit_ns=0, withhold_first_arrive=False)
    status.zero_()
    after = B.gta_decode_fp8(*args, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(after.view(torch.int16), before.view(torch.int16))


def test_fp8_decode_config3_shape_sampled_sequences(B, oracle):
    w = I.CONFIGS["c3_decode_bf16"]
    rel, mx = _decode_case(B, oracle, w, [w.seq] * w.batch, sample=[0, 9, 31], cap=w.seq + 64, path=2)
    print(f"\nc3 shape over 8-bit caches: rel-L2 {rel:.3e} max-abs {mx:.3e}")


def test_fp8_decode_config5_shape_ragged_sampled_sequences(B, oracle):
    """The ragged workload's shape (8 maps over 8 key groups, d_l = 1024) at a tenth of its lengths."""
    w = I.scaled(I.CONFIGS["c5_ragged_decode_bf16"], batch=24)
    g = torch.Generator("cpu").manual_seed(5)
    lens = torch.randint(100, 3300, (24,), generator=g).tolist()
    _decode_case(B, oracle, w, lens, sample=[0, 11, 23], cap=3304, path=2)


def test_append_then_decode_over_fp8_caches(B, oracle):
    """The GPU's own quantising append feeds the GPU decode: the result is the oracle's on the oracle's append."""
    w = I.Workload("steps", "decode", "bf16", 3, 0, 128, 8, 4, 2, 1, 64, 256, seed=62)
    lens, cap = [5, 0, 130], 140
    t = I.decode_inputs(w, device="cuda", s_cap=cap, seq_lens=lens)
    kq = np.zeros((3, 2, cap, 64), np.uint8); ks = np.ones((3, 2, cap), np.float32)
    cq = np.zeros((3, 1, cap, 256), np.uint8); cs = np.ones((3, 1, cap), np.float32)
    dev = [torch.from_numpy(a).cuda() for a in (kq, cq, ks, cs)]
    lens_d = torch.zeros(3, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    # prefill-style bulk append of each sequence's history, one call per sequence (ragged lengths)
    for b, n in enumerate(lens):
        if n == 0:
            continue
        sub = [d_[b:b + 1] for d_ in dev]
        B.gta_cache_append_fp8(*sub, t["k_cache"][b:b + 1, :, :n].contiguous(), t["c_cache"][b:b + 1, :, :n].contiguous(),
                               lens_d[b:b + 1], status_word=status)
    # then one new token for all of them
    B.gta_cache_append_fp8(*dev, t["k_new"], t["c_new"], lens_d, status_word=status)
    out = B.gta_decode_fp8(t["q"], *dev, lens_d, t["x_t"], t["w_p"], t["w_g"], status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and lens_d.tolist() == [n + 1 for n in lens]
    k_hist, c_hist = t["k_cache"].cpu(), t["c_cache"].cpu()
    kq_r, ks_r, cq_r, cs_r = kq.copy(), ks.copy(), cq.copy(), cs.copy()
    for b, n in enumerate(lens):
        if n:
            a, s_ = oracle.quantize_rows_e4m3(k_hist[b, :, :n]); kq_r[b, :, :n] = a; ks_r[b, :, :n] = s_
            a, s_ = oracle.quantize_rows_e4m3(c_hist[b, :, :n]); cq_r[b, :, :n] = a; cs_r[b, :, :n] = s_
    kq_r, ks_r, cq_r, cs_r, lens_r, ov = oracle.cache_append_fp8(kq_r, ks_r, cq_r, cs_r, t["k_new"].cpu(), t["c_new"].cpu(),
                                                                  np.array(lens, np.int32))
    assert ov == 0
    assert np.array_equal(dev[0].cpu().numpy(), kq_r) and np.array_equal(dev[1].cpu().numpy(), cq_r)
    assert np.array_equal(dev[2].cpu().numpy().view(np.uint32), ks_r.view(np.uint32))
    want = oracle.decode_fp8(oracle_shape(w, seq=0), t["q"].cpu(), kq_r, ks_r, cq_r, cs_r, lens_r, t["x_t"].cpu(),
                             t["w_p"].cpu(), t["w_g"].cpu())
    assert_close(out, want, torch.bfloat16, "append then decode (fp8 caches)")
