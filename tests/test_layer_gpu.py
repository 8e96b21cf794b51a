"""GPU parity of the whole attention layer (projections + RoPE + cache write, operator, output projection)
against the fp64 oracle of App. B.1.1, element by element on identical seeded inputs."""
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


def _run_layer(B, w, t, chunks, s_cap, rope_base):
    """The layer chunk by chunk over caches that start out full of NaN (what uninitialised memory may hold);
    returns u, k_cache, c_cache."""
    k_cache = torch.full((w.batch, w.n_k, s_cap, w.d_h), float("nan"), device="cuda", dtype=torch.bfloat16)
    c_cache = torch.full((w.batch, w.n_c, s_cap, w.d_l), float("nan"), device="cuda", dtype=torch.bfloat16)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    us, pos0, guards = [], 0, []
    for n in chunks:
        x = t["x"][:, pos0:pos0 + n].contiguous()
        shape = B.make_shape(batch=w.batch, seq=n, d_model=w.d_model, n_heads=w.n_heads, n_q=w.n_q, n_k=w.n_k,
                             n_c=w.n_c, d_h=w.d_h, d_l=w.d_l, dtype=torch.bfloat16)
        ws = Guarded((B.layer_prefill_workspace_bytes(shape),), torch.uint8)
        ug = Guarded((w.batch, n, w.d_model), torch.bfloat16)
        us.append(B.gta_layer_prefill(x, t["w_qkc"], t["w_p"], t["w_g"], t["w_o"], k_cache, c_cache, pos0=pos0,
                                      rope_base=rope_base, n_q=w.n_q, workspace=ws.t, out=ug.t, status_word=status))
        guards += [ws, ug]
        pos0 += n
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for g in guards:
        g.check(w.name)
    # rows behind the last written position are untouched, everything before is written
    assert torch.isnan(k_cache[:, :, pos0:]).all() and torch.isnan(c_cache[:, :, pos0:]).all()
    assert not torch.isnan(k_cache[:, :, :pos0]).any() and not torch.isnan(c_cache[:, :, :pos0]).any()
    return torch.cat(us, dim=1), k_cache[:, :, :pos0], c_cache[:, :, :pos0]


def _layer_case(B, oracle, w, chunks=None, rope_base=10000.0, rows=None, sample=None):
    chunks = chunks or [w.seq]
    assert sum(chunks) == w.seq
    t = I.layer_inputs(w, device="cuda")
    u, k, c = _run_layer(B, w, t, chunks, w.seq + 40, rope_base)
    tc = {n: v.cpu() for n, v in t.items()}
    want = oracle.layer_prefill(oracle_shape(w), tc["x"], tc["w_qkc"], tc["w_p"], tc["w_g"], tc["w_o"],
                                rope_base=rope_base, rows=sample)
    # the caches hold the rounded RoPE'd projections: a value may land on the neighbouring bf16 number where fp32
    # and fp64 accumulation straddle a rounding boundary, nothing more
    for name, got, ref in (("k", k, want["k"]), ("c", c, want["c"])):
        g64 = got.double().cpu().numpy()
        # one bf16 step of the value, plus the fp32 accumulation error itself where the value is tiny
        # (a rotation can cancel: x0 cos - x1 sin near zero)
        step = np.abs(ref) * 2.0 ** -7 + 3e-5
        assert np.all(np.abs(g64 - ref) <= step), f"{name} cache differs by more than one bf16 step"
        assert np.mean(g64 != ref) < 2e-2, f"{name} cache: too many rounding flips"
    if sample is not None:      # the oracle computed these positions only
        return assert_close(u[:, torch.as_tensor(sample, device="cuda")], want["u"], torch.bfloat16, w.name)
    sel = slice(None) if rows is None else rows
    return assert_close(u[:, sel], want["u"][:, sel], torch.bfloat16, w.name)


LAYERS = [
    # name, B, N, H, n_h, n_q, n_k, n_c, d_h, d_l, chunks
    ("paper_1b_shape_small", 2, 300, 1280, 20, 5, 1, 1, 64, 128, None),
    ("c2_shape_small", 1, 384, 512, 8, 4, 4, 1, 128, 512, None),
    ("two_chunks", 2, 320, 256, 8, 4, 2, 2, 64, 128, [192, 128]),
    ("ragged_chunks_one_token_last", 1, 262, 256, 4, 2, 2, 1, 128, 256, [5, 256, 1]),
    ("odd_block_tail", 3, 130, 384, 6, 3, 3, 1, 64, 256, None),
]


@pytest.mark.parametrize("case", LAYERS, ids=[c[0] for c in LAYERS])
def test_layer_prefill_small_shapes(B, oracle, case):
    name, nb, N, H, n_h, n_q, n_k, n_c, d_h, d_l, chunks = case
    w = I.Workload(name, "prefill", "bf16", nb, N, H, n_h, n_q, n_k, n_c, d_h, d_l, seed=71)
    _layer_case(B, oracle, w, chunks=chunks)


def test_layer_prefill_other_rope_base_and_late_positions(B, oracle):
    """A chunk far into the context (positions 3000 ..): the phase of the fast pairs must survive."""
    w = I.Workload("late", "prefill", "bf16", 1, 3200, 256, 4, 2, 2, 1, 64, 128, seed=72)
    _layer_case(B, oracle, w, chunks=[3072, 128], rope_base=500000.0, rows=slice(3000, 3200))


def _sample_positions(N, n=24, seed=0):
    rng = np.random.default_rng(seed)
    fixed = [0, 1, 127, 128, 255, 256, N // 2, N - 2, N - 1]
    return sorted(set(fixed) | set(int(v) for v in rng.integers(0, N, n)))


@pytest.mark.parametrize("name", ["c2_prefill_bf16", "x1_gta1b_prefill_bf16", "c4_long_prefill_bf16"])
def test_layer_prefill_full_size_sampled_positions(B, oracle, name):
    w = I.CONFIGS[name]
    _layer_case(B, oracle, w, sample=_sample_positions(w.seq))


def _unrounded_case(B, oracle, w, sample=None):
    """u of gta_layer_prefill against the layer oracle with NO rounding anywhere (storage = float64): the
    definition of App. B.1.1 itself, whatever the kernels keep between their steps."""
    t = I.layer_inputs(w, device="cuda")
    u, _, _ = _run_layer(B, w, t, [w.seq], w.seq + 8, 10000.0)
    tc = {n: v.cpu() for n, v in t.items()}
    want = oracle.layer_prefill(oracle_shape(w), tc["x"], tc["w_qkc"], tc["w_p"], tc["w_g"], tc["w_o"], rows=sample,
                                storage=oracle.F64)
    got = u if sample is None else u[:, torch.as_tensor(sample, device="cuda")]
    rel, mx = assert_close(got, want["u"], torch.bfloat16, w.name + " (unrounded oracle)")
    print(f"\n{w.name}: u vs unrounded fp64 layer: rel-L2 {rel:.3e} max-abs {mx:.3e}")


@pytest.mark.parametrize("case", LAYERS, ids=[c[0] for c in LAYERS])
def test_layer_prefill_against_the_unrounded_definition_small(B, oracle, case):
    name, nb, N, H, n_h, n_q, n_k, n_c, d_h, d_l, _ = case
    _unrounded_case(B, oracle, I.Workload(name, "prefill", "bf16", nb, N, H, n_h, n_q, n_k, n_c, d_h, d_l, seed=74))


def test_layer_prefill_against_the_unrounded_definition_c2_sampled(B, oracle):
    w = I.CONFIGS["c2_prefill_bf16"]
    _unrounded_case(B, oracle, w, sample=_sample_positions(w.seq))


LAYER_STEPS = [
    # name, H, n_h, n_q, n_k, n_c, d_h, d_l, lens (tokens already cached per sequence)
    ("c3_shape_small", 512, 8, 4, 4, 1, 128, 512, [1, 63, 64, 200, 0]),
    ("paper_1b_shape", 1280, 20, 5, 1, 1, 64, 128, [130, 7]),
    ("two_latents_batch_20", 256, 8, 4, 2, 2, 64, 128, [(37 * i) % 150 for i in range(20)]),
    # more than 128 sequences: the one-token projections run on CTA pairs again (two row tiles)
    ("batch_150", 256, 8, 4, 2, 2, 64, 128, [(13 * i) % 90 for i in range(150)]),
]


@pytest.mark.parametrize("case", LAYER_STEPS, ids=[c[0] for c in LAYER_STEPS])
def test_layer_decode_step_equals_the_next_row_of_the_layer(B, oracle, case):
    """Caches filled by gta_layer_prefill (one call per sequence, ragged lengths), then one gta_layer_decode step:
    its output is row len_b of the layer oracle over len_b + 1 tokens, its cache rows the oracle's k / c there."""
    name, H, n_h, n_q, n_k, n_c, d_h, d_l, lens = case
    nb, cap = len(lens), max(lens) + 9
    w = I.Workload(name, "prefill", "bf16", nb, max(lens) + 1, H, n_h, n_q, n_k, n_c, d_h, d_l, seed=73)
    t = I.layer_inputs(w, device="cuda")          # x: the history of every sequence, the new token at row len_b
    k_cache = torch.full((nb, n_k, cap, d_h), float("nan"), device="cuda", dtype=torch.bfloat16)
    c_cache = torch.full((nb, n_c, cap, d_l), float("nan"), device="cuda", dtype=torch.bfloat16)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for b, n in enumerate(lens):
        if n > 0:
            B.gta_layer_prefill(t["x"][b:b + 1, :n].contiguous(), t["w_qkc"], t["w_p"], t["w_g"], t["w_o"],
                                k_cache[b:b + 1], c_cache[b:b + 1], n_q=n_q, status_word=status)
    k0, c0 = k_cache.clone(), c_cache.clone()
    seq_lens = torch.tensor(lens, dtype=torch.int32, device="cuda")
    idx = torch.arange(nb, device="cuda")
    x_t = t["x"][idx, seq_lens.long()].contiguous()
    shape = B.make_shape(batch=nb, seq=0, d_model=H, n_heads=n_h, n_q=n_q, n_k=n_k, n_c=n_c, d_h=d_h, d_l=d_l,
                         dtype=torch.bfloat16)
    ws = torch.full((B.layer_decode_workspace_bytes(shape, cap),), 0xFF, dtype=torch.uint8, device="cuda")
    # the same step over the same caches scattered into 64-token pages: bit-identical output and rows
    pg = I.paginate(dict(k_cache=k_cache, c_cache=c_cache), 64, seed=9)
    lens_p = seq_lens.clone()
    u_p = B.gta_layer_decode_paged(x_t, t["w_qkc"], t["w_p"], t["w_g"], t["w_o"], pg["k_pool"], pg["c_pool"],
                                   pg["block_table"], lens_p, n_q=n_q, status_word=status)
    u = B.gta_layer_decode(x_t, t["w_qkc"], t["w_p"], t["w_g"], t["w_o"], k_cache, c_cache, seq_lens, n_q=n_q,
                           workspace=ws, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert seq_lens.tolist() == [n + 1 for n in lens] and lens_p.tolist() == seq_lens.tolist()
    assert torch.equal(u_p.view(torch.int16), u.view(torch.int16))
    for b, n in enumerate(lens):
        page = int(pg["block_table"][b, n // 64])
        assert torch.equal(pg["k_pool"][page, :, n % 64].view(torch.int16), k_cache[b, :, n].view(torch.int16))
        assert torch.equal(pg["c_pool"][page, :, n % 64].view(torch.int16), c_cache[b, :, n].view(torch.int16))
    tc = {n: v.cpu() for n, v in t.items()}
    want_u = np.zeros((nb, H))
    for b, n in enumerate(lens):
        ws_b = I.scaled(w, batch=1, seq=n + 1)
        r = oracle.layer_prefill(oracle_shape(ws_b), tc["x"][b:b + 1, :n + 1], tc["w_qkc"], tc["w_p"], tc["w_g"],
                                 tc["w_o"], rows=[n])
        want_u[b] = r["u"][0, 0]
        for got, ref in ((k_cache[b, :, n], r["k"][0, :, n]), (c_cache[b, :, n], r["c"][0, :, n])):
            assert np.all(np.abs(got.double().cpu().numpy() - ref) <= np.abs(ref) * 2.0 ** -7 + 3e-5)
        # nothing but row n of this sequence's caches changed
        keep = torch.ones(cap, dtype=torch.bool, device="cuda")
        keep[n] = False
        assert torch.equal(k_cache[b][:, keep].view(torch.int16), k0[b][:, keep].view(torch.int16))
        assert torch.equal(c_cache[b][:, keep].view(torch.int16), c0[b][:, keep].view(torch.int16))
    assert_close(u, want_u, torch.bfloat16, name)


def test_layer_decode_full_cache_is_skipped_and_reported(B):
    w = I.Workload("full", "prefill", "bf16", 2, 8, 256, 4, 2, 2, 1, 64, 128, seed=2)
    t = I.layer_inputs(w, device="cuda")
    k = torch.zeros((2, 2, 8, 64), dtype=torch.bfloat16, device="cuda")
    c = torch.zeros((2, 1, 8, 128), dtype=torch.bfloat16, device="cuda")
    lens = torch.tensor([8, 3], dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.gta_layer_decode(t["x"][:, 0].contiguous(), t["w_qkc"], t["w_p"], t["w_g"], t["w_o"], k, c, lens, n_q=2,
                       status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == B.GTA_ERR_CACHE_FULL
    assert lens.tolist() == [8, 4]
    assert not k[0].any() and not c[0].any() and k[1, :, 3].any() and not k[1, :, 4:].any()


def test_layer_rejects_what_it_does_not_cover(B):
    w = I.Workload("bad", "prefill", "bf16", 1, 64, 256, 4, 2, 2, 1, 64, 128, seed=1)
    t = I.layer_inputs(w, device="cuda")
    k = torch.zeros((1, 2, 64, 64), dtype=torch.bfloat16, device="cuda")
    c = torch.zeros((1, 1, 64, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.GtaError) as e:     # chunk does not fit behind pos0
        B.gta_layer_prefill(t["x"], t["w_qkc"], t["w_p"], t["w_g"], t["w_o"], k, c, pos0=1, n_q=2)
    assert e.value.status == B.GTA_ERR_INVALID_ARG
    with pytest.raises(B.GtaError) as e:
        B.gta_layer_prefill(t["x"], t["w_qkc"], t["w_p"], t["w_g"], t["w_o"], k, c, rope_base=1.0, n_q=2)
    assert e.value.status == B.GTA_ERR_INVALID_ARG
    f = {n: v.float() for n, v in t.items()}
    with pytest.raises(B.GtaError) as e:     # fp32: not on the tensor-core kernels
        B.gta_layer_prefill(f["x"], f["w_qkc"], f["w_p"], f["w_g"], f["w_o"], k.float(), c.float(), n_q=2)
    assert e.value.status == B.GTA_ERR_UNSUPPORTED
