"""GPU parity: the CUDA library (through its C ABI) against the fp64 CPU oracle, element by
element on identical seeded inputs.  Sizes span several tiles plus ragged tails; the full-size
workloads are checked on sampled rows / sequences the oracle can compute one by one."""
import numpy as np
import pytest
import torch

from paper_2506_17286_b200 import inputs as I
from tests.parity_utils import Guarded, assert_close, cpu, oracle_shape

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2506_17286_b200 import build, binding
    build.build()
    binding.lib()
    return binding


def _prefill_case(B, oracle, w, causal=True, rows=None, scale=0.0, project=True):
    t = I.prefill_inputs(w, device="cuda", project=project)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    shape = B.make_shape(batch=w.batch, seq=w.seq, d_model=w.d_model, n_heads=w.n_heads, n_q=w.n_q, n_k=w.n_k,
                         n_c=w.n_c, d_h=w.d_h, d_l=w.d_l, dtype=w.torch_dtype())
    # a workspace full of NaN bit patterns: nothing may be read before the library wrote it; guard bands
    # around the workspace and the output: nothing may be written outside them
    ws = Guarded((B.prefill_workspace_bytes(shape),), torch.uint8)
    og = Guarded((w.batch, w.seq, w.n_heads, w.d_h), w.torch_dtype())
    out = B.gta_prefill(t["q"], t["k"], t["c"], t["x"], t["w_p"], t["w_g"], causal=causal,
                        softmax_scale=scale, status_word=status, workspace=ws.t, out=og.t)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ws.check(w.name + " workspace"); og.check(w.name + " out")
    tc = cpu(t)
    want = oracle.prefill(oracle_shape(w, causal=int(causal), scale=scale), tc["q"], tc["k"], tc["c"], tc["x"],
                          tc["w_p"], tc["w_g"], rows=rows)
    got = out if rows is None else out[:, torch.as_tensor(rows, device=out.device, dtype=torch.long)]
    return assert_close(got, want, w.torch_dtype(), w.name)


# --------------------------------------------------------------------------- prefill
def test_prefill_config1_tiny_fp32(B, oracle):
    _prefill_case(B, oracle, I.CONFIGS["c1_tiny_prefill_f32"])


SMALL_PREFILL = [
    # name, dtype, B, N, H, n_h, n_q, n_k, n_c, d_h, d_l
    ("bf16_tiles_ragged", "bf16", 2, 300, 256, 8, 4, 4, 1, 128, 512),
    ("bf16_two_slices_long", "bf16", 1, 640, 128, 4, 2, 2, 1, 128, 256),
    ("bf16_dl1024", "bf16", 1, 257, 192, 4, 2, 2, 1, 128, 1024),
    ("bf16_shared_keys_two_latents", "bf16", 2, 200, 128, 8, 4, 2, 2, 64, 128),
    ("bf16_paper_1b_shape", "bf16", 1, 160, 1280, 20, 5, 1, 1, 64, 128),
    ("f32_general", "f32", 2, 150, 96, 6, 6, 3, 1, 32, 64),
    ("f32_dh128", "f32", 1, 129, 64, 2, 1, 1, 1, 128, 256),
    # all rows in one 128-row tile: the decoder + gate kernel runs without CTA pairs on half-head items
    ("bf16_short_batch3_odd_heads", "bf16", 3, 100, 192, 6, 2, 2, 1, 128, 256),
    ("bf16_short_one_token", "bf16", 5, 1, 128, 4, 4, 4, 1, 128, 512),
    # head dimension 64 and 128-column latent slices on the tensor-core path
    ("bf16_dh64_dl256_long", "bf16", 2, 700, 192, 8, 2, 1, 1, 64, 256),
    ("bf16_dh128_dl128", "bf16", 1, 400, 128, 4, 2, 2, 1, 128, 128),
    ("bf16_dh64_dl384_two_latents", "bf16", 1, 300, 128, 4, 2, 2, 2, 64, 384),
]


@pytest.mark.parametrize("case", SMALL_PREFILL, ids=[c[0] for c in SMALL_PREFILL])
def test_prefill_small_shapes(B, oracle, case):
    name, dt, *dims = case
    w = I.Workload(name, "prefill", dt, *dims, seed=4242)
    _prefill_case(B, oracle, w)


@pytest.mark.parametrize("N", [1, 2, 127, 128, 129, 255, 256, 384])
def test_prefill_tile_boundaries_bf16(B, oracle, N):
    w = I.Workload(f"edge_{N}", "prefill", "bf16", 1, N, 128, 4, 2, 2, 1, 128, 256, seed=77 + N)
    _prefill_case(B, oracle, w)


def test_prefill_non_causal_and_explicit_scale(B, oracle):
    w = I.Workload("noncausal", "prefill", "bf16", 1, 200, 128, 4, 2, 2, 1, 128, 256, seed=5)
    _prefill_case(B, oracle, w, causal=False)
    _prefill_case(B, oracle, w, causal=True, scale=0.05)
    wf = I.Workload("noncausal_f32", "prefill", "f32", 1, 70, 64, 4, 2, 1, 1, 32, 64, seed=6)
    _prefill_case(B, oracle, wf, causal=False)


def test_prefill_is_deterministic_and_leaves_inputs_untouched(B):
    w = I.Workload("det", "prefill", "bf16", 2, 300, 256, 8, 4, 4, 1, 128, 512, seed=9)
    t = I.prefill_inputs(w, device="cuda")
    before = {k: v.clone() for k, v in t.items()}
    a = B.gta_prefill(t["q"], t["k"], t["c"], t["x"], t["w_p"], t["w_g"])
    b = B.gta_prefill(t["q"], t["k"], t["c"], t["x"], t["w_p"], t["w_g"])
    torch.cuda.synchronize()
    assert torch.equal(a, b)
    for k in t:
        assert torch.equal(t[k], before[k])


def test_prefill_repeated_runs_with_several_items_per_cta(B, oracle):
    """More work items than CTA pairs, short and long items mixed: a barrier wait that is out of step
    shows up as an occasional wrong query tile, so the call is repeated and every run is compared
    (rows of the second query tile included) and must be bit-identical to the first."""
    w = I.Workload("multi_item", "prefill", "bf16", 4, 1024, 256, 8, 4, 4, 1, 128, 512, seed=11)
    t = I.prefill_inputs(w, device="cuda")
    rows = sorted(set(range(120, 136)) | set(range(248, 264)) | {0, 1, 511, 512, 1022, 1023} | set(range(192, 256, 7)))
    tc = cpu(t)
    want = oracle.prefill(oracle_shape(w), tc["q"], tc["k"], tc["c"], tc["x"], tc["w_p"], tc["w_g"], rows=rows)
    sel = torch.as_tensor(rows, device="cuda", dtype=torch.long)
    first = None
    for rep in range(60):
        out = B.gta_prefill(t["q"], t["k"], t["c"], t["x"], t["w_p"], t["w_g"])
        torch.cuda.synchronize()
        assert_close(out[:, sel], want, torch.bfloat16, f"repeat {rep}")
        if first is None:
            first = out.clone()
        else:
            assert torch.equal(out, first), f"run {rep} differs from run 0"


def _sample_rows(N, n=48, seed=0):
    rng = np.random.default_rng(seed)
    fixed = {0, 1, 127, 128, 129, N // 2 - 1, N // 2, N - 129, N - 128, N - 2, N - 1}
    rows = sorted(r for r in fixed if 0 <= r < N)
    extra = rng.choice(N, size=max(0, n - len(rows)), replace=False).tolist()
    return sorted(set(rows) | set(extra))


def test_prefill_config2_full_size_sampled_rows(B, oracle):
    w = I.CONFIGS["c2_prefill_bf16"]
    _prefill_case(B, oracle, w, rows=_sample_rows(w.seq, 64, seed=2))


def test_prefill_config4_full_size_sampled_rows(B, oracle):
    w = I.CONFIGS["c4_long_prefill_bf16"]
    _prefill_case(B, oracle, w, rows=_sample_rows(w.seq, 40, seed=4))


def test_prefill_paper_1b_layer_shape_full_size_sampled_rows(B, oracle):
    # 20 heads in 5 maps over one key group and one latent group, d_h = 64, d_l = 128: the tensor-core
    # path with 64-wide heads, 128-column slices and several items per CTA pair
    w = I.CONFIGS["x1_gta1b_prefill_bf16"]
    _prefill_case(B, oracle, w, rows=_sample_rows(w.seq, 48, seed=11))


# --------------------------------------------------------------------------- chunked prefill
CHUNKS = [
    # name, dtype, B, kv_len, N (queries = the last N positions), kv_cap, H, n_h, n_q, n_k, n_c, d_h, d_l, causal
    ("bf16_chunk_mid", "bf16", 2, 700, 300, 768, 256, 8, 4, 4, 1, 128, 512, True),
    ("bf16_chunk_one_query", "bf16", 3, 513, 1, 513, 128, 4, 2, 2, 1, 128, 256, True),
    ("bf16_chunk_whole", "bf16", 1, 260, 260, 300, 128, 4, 2, 2, 1, 128, 256, True),
    ("bf16_chunk_dh64", "bf16", 2, 1000, 129, 1024, 192, 8, 2, 1, 1, 64, 128, True),
    ("bf16_chunk_non_causal", "bf16", 1, 400, 100, 400, 128, 4, 2, 2, 1, 128, 256, False),
    ("bf16_chunk_plain_alu_shape", "bf16", 2, 300, 77, 320, 128, 6, 6, 3, 1, 32, 64, True),
    ("f32_chunk", "f32", 1, 200, 50, 256, 96, 6, 6, 3, 1, 32, 64, True),
]


@pytest.mark.parametrize("case", CHUNKS, ids=[c[0] for c in CHUNKS])
def test_prefill_chunk_against_a_longer_cache(B, oracle, case):
    """The chunk's rows must equal the same rows of a prefill over all kv_len tokens (oracle); the
    cache rows past kv_len hold NaN (what uninitialised memory may hold) and must not reach the result."""
    name, dt, nb, kv_len, N, kv_cap, H, n_h, n_q, n_k, n_c, d_h, d_l, causal = case
    w = I.Workload(name, "prefill", dt, nb, kv_len, H, n_h, n_q, n_k, n_c, d_h, d_l, seed=321)
    t = I.prefill_inputs(w, device="cuda")
    first = kv_len - N
    gen = torch.Generator(device="cuda").manual_seed(5)
    k = torch.full((nb, n_k, kv_cap, d_h), float("nan"), device="cuda", dtype=w.torch_dtype())
    c = torch.full((nb, n_c, kv_cap, d_l), float("nan"), device="cuda", dtype=w.torch_dtype())
    k[:, :, :kv_len] = t["k"]
    c[:, :, :kv_len] = t["c"]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = B.gta_prefill_chunk(t["q"][:, :, first:].contiguous(), k, c, t["x"][:, first:].contiguous(), t["w_p"],
                              t["w_g"], kv_len, causal=causal, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    tc = cpu(t)
    rows = list(range(first, kv_len))
    want = oracle.prefill(oracle_shape(w, causal=int(causal)), tc["q"], tc["k"], tc["c"], tc["x"], tc["w_p"], tc["w_g"],
                          rows=rows)
    assert_close(out, want, w.torch_dtype(), name)


# --------------------------------------------------------------------------- decode
def _nan_behind_the_live_rows(t):
    """Cache rows at and past seq_lens[b] become NaN: what uninitialised memory may hold, and nothing of it may
    reach the result (a masked probability times NaN would)."""
    for b, n in enumerate(t["seq_lens"].cpu().tolist()):
        t["k_cache"][b, :, n:] = float("nan")
        t["c_cache"][b, :, n:] = float("nan")
    return t


def _decode_case(B, oracle, w, seq_lens=None, s_cap=None, sample=None):
    t = _nan_behind_the_live_rows(I.decode_inputs(w, device="cuda", s_cap=s_cap, seq_lens=seq_lens))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    shape = B.decode_shape(t["q"], t["k_cache"], t["c_cache"], t["x_t"], t["w_p"])
    ws = Guarded((B.decode_workspace_bytes(shape, t["s_cap"]),), torch.uint8)
    og = Guarded((w.batch, w.n_heads, w.d_h), w.torch_dtype())
    out = B.gta_decode(t["q"], t["k_cache"], t["c_cache"], t["seq_lens"], t["x_t"], t["w_p"], t["w_g"],
                       status_word=status, workspace=ws.t, out=og.t)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ws.check(w.name + " workspace"); og.check(w.name + " out")
    idx = list(range(w.batch)) if sample is None else sample
    sel = torch.as_tensor(idx, device="cuda", dtype=torch.long)
    lens = t["seq_lens"][sel].cpu().numpy()
    cap = int(lens.max()) if len(idx) else 0
    ws = I.scaled(w, batch=len(idx))
    want = oracle.decode(oracle_shape(ws, seq=0), t["q"][sel].cpu(), t["k_cache"][sel][:, :, :cap].contiguous().cpu(),
                         t["c_cache"][sel][:, :, :cap].contiguous().cpu(), lens, cap, t["x_t"][sel].cpu(),
                         t["w_p"].cpu(), t["w_g"].cpu())
    return assert_close(out[sel], want, w.torch_dtype(), w.name)


SMALL_DECODE = [
    # name, dtype, B, H, n_h, n_q, n_k, n_c, d_h, d_l, lens
    ("bf16_ragged", "bf16", 5, 256, 8, 4, 4, 1, 128, 512, [1, 63, 64, 65, 700]),
    ("bf16_empty_and_full", "bf16", 4, 128, 4, 2, 2, 1, 128, 256, [0, 512, 1, 300]),
    ("bf16_shared_keys_two_latents", "bf16", 3, 128, 8, 4, 2, 2, 64, 128, [200, 5, 129]),
    ("bf16_paper_1b_shape", "bf16", 2, 1280, 20, 5, 1, 1, 64, 128, [333, 1000]),
    ("bf16_eight_maps", "bf16", 9, 512, 16, 8, 8, 1, 128, 1024, [257, 256, 255, 1, 2, 1000, 64, 128, 511]),
    # the other (sub-tile, key groups, maps per group) instantiations of the tensor-memory stream kernel
    ("bf16_eight_maps_four_key_groups_dl512", "bf16", 4, 256, 16, 8, 4, 1, 128, 512, [700, 31, 32, 33]),
    ("bf16_four_maps_two_key_groups_dl512", "bf16", 5, 256, 8, 4, 2, 1, 128, 512, [1, 450, 0, 96, 65]),
    ("bf16_four_maps_one_key_group_dl512", "bf16", 3, 256, 8, 4, 1, 1, 128, 512, [500, 64, 17]),
    ("bf16_eight_maps_four_key_groups_dl1024", "bf16", 4, 256, 16, 8, 4, 1, 128, 1024, [300, 15, 16, 17]),
    ("bf16_eight_maps_two_key_groups_dl1024", "bf16", 3, 256, 16, 8, 2, 1, 128, 1024, [1, 129, 48]),
    ("bf16_eight_maps_one_key_group_dl1024", "bf16", 3, 256, 8, 8, 1, 1, 128, 1024, [200, 0, 33]),
    ("bf16_long_sequences_many_sub_tiles_per_cta", "bf16", 2, 256, 8, 4, 4, 1, 128, 512, [20000, 12345]),
    # 64-token sub-tiles (d_l = 256, one or two key groups: two key groups on the rows of a score MMA)
    ("bf16_eight_maps_one_key_group_dl256", "bf16", 3, 256, 8, 8, 1, 1, 128, 256, [500, 64, 65]),
    ("bf16_eight_maps_two_key_groups_dl256", "bf16", 4, 256, 8, 8, 2, 1, 128, 256, [63, 300, 0, 128]),
    ("bf16_four_maps_one_key_group_dl256", "bf16", 2, 128, 4, 4, 1, 1, 128, 256, [1000, 127]),
    ("bf16_eight_maps_four_key_groups_dl256", "bf16", 3, 256, 8, 8, 4, 1, 128, 256, [200, 31, 97]),
    ("bf16_eight_key_groups_dl256", "bf16", 3, 512, 8, 8, 8, 1, 128, 256, [100, 15, 49]),
    # the remaining groupings at d_l = 512 and 1024
    ("bf16_one_map_dl512", "bf16", 2, 128, 2, 1, 1, 1, 128, 512, [300, 33]),
    ("bf16_eight_maps_one_key_group_dl512", "bf16", 2, 256, 8, 8, 1, 1, 128, 512, [260, 95]),
    ("bf16_eight_maps_two_key_groups_dl512", "bf16", 2, 256, 8, 8, 2, 1, 128, 512, [64, 129]),
    ("bf16_eight_key_groups_dl512", "bf16", 3, 512, 8, 8, 8, 1, 128, 512, [100, 16, 47]),
    ("bf16_one_map_dl1024", "bf16", 2, 128, 2, 1, 1, 1, 128, 1024, [150, 17]),
    ("bf16_four_maps_two_key_groups_dl1024", "bf16", 2, 128, 4, 4, 2, 1, 128, 1024, [90, 33]),
    ("bf16_four_maps_four_key_groups_dl1024", "bf16", 2, 128, 4, 4, 4, 1, 128, 1024, [48, 200]),
    # more sequences than the stream kernel has threads (the prefix sum takes two per thread), many of them empty;
    # and a batch with nothing cached at all (no CTA has a sub-tile)
    ("bf16_batch_400_c3_grouping", "bf16", 400, 256, 8, 4, 4, 1, 128, 512, [0 if i % 7 == 3 else 1 + (13 * i) % 70 for i in range(400)]),
    ("bf16_all_sequences_empty_c3_grouping", "bf16", 6, 256, 8, 4, 4, 1, 128, 512, [0, 0, 0, 0, 0, 0]),
    ("f32_general", "f32", 3, 96, 6, 6, 3, 1, 32, 64, [100, 7, 260]),
    # more than 16 sequences: the finish goes through the merge kernel + the tensor-core decoder kernel
    # (without CTA pairs up to 128 sequences, with them above)
    ("bf16_batch_17", "bf16", 17, 192, 4, 2, 2, 1, 128, 256, [1 + (53 * i) % 400 for i in range(17)]),
    ("bf16_batch_128", "bf16", 128, 128, 4, 4, 4, 1, 128, 256, [(29 * i) % 150 for i in range(128)]),
    ("bf16_batch_200", "bf16", 200, 128, 4, 2, 2, 1, 128, 512, [1 + (31 * i) % 90 for i in range(200)]),
    ("bf16_batch_40", "bf16", 40, 256, 8, 4, 4, 1, 128, 512, [1 + (37 * i) % 300 for i in range(40)]),
    # head dimension 64, latent width 128, map counts that are no power of two, shared keys: the stream kernel's
    # other instantiations, finished by the merge kernel + the decoder kernel whatever the batch
    ("bf16_dh64_three_maps_batch_40", "bf16", 40, 192, 6, 3, 1, 1, 64, 128, [1 + (41 * i) % 700 for i in range(40)]),
    ("bf16_dh64_dl512_small_batch", "bf16", 3, 128, 8, 4, 2, 1, 64, 512, [70, 1, 513]),
    ("bf16_dh128_five_maps", "bf16", 7, 256, 10, 5, 1, 1, 128, 256, [300, 0, 64, 65, 1000, 17, 2]),
    ("bf16_two_latents_batch_20", "bf16", 20, 256, 8, 4, 4, 2, 128, 256, [1 + (67 * i) % 500 for i in range(20)]),
    ("bf16_four_latents_dl128", "bf16", 5, 128, 8, 8, 2, 4, 64, 128, [129, 1, 64, 400, 33]),
    ("bf16_batch_33_odd_heads", "bf16", 33, 128, 3, 1, 1, 1, 128, 256, [0 if i == 5 else 1 + (91 * i) % 500 for i in range(33)]),
]


@pytest.mark.parametrize("case", SMALL_DECODE, ids=[c[0] for c in SMALL_DECODE])
def test_decode_small_shapes(B, oracle, case):
    name, dt, nb, H, n_h, n_q, n_k, n_c, d_h, d_l, lens = case
    w = I.Workload(name, "decode", dt, nb, 0, H, n_h, n_q, n_k, n_c, d_h, d_l, seed=99)
    _decode_case(B, oracle, w, seq_lens=lens, s_cap=max(lens) + 13)


def test_decode_config3_full_size(B, oracle):
    _decode_case(B, oracle, I.CONFIGS["c3_decode_bf16"])


def test_decode_config5_full_size_sampled_sequences(B, oracle):
    w = I.CONFIGS["c5_ragged_decode_bf16"]
    lens = I.decode_seq_lens(w).numpy()
    order = np.argsort(lens)
    sample = sorted({int(order[0]), int(order[-1]), int(order[len(order) // 2]), 0, 1, 63, 127, int(order[1])})
    _decode_case(B, oracle, w, sample=sample)


def test_decode_equals_last_prefill_row_on_the_gpu(B):
    """Append the prefill's keys / latents to empty caches, decode the last token: both library
    paths must agree within the bf16 tolerance (and with the oracle through the other tests)."""
    w = I.Workload("p_vs_d", "prefill", "bf16", 3, 333, 256, 8, 4, 4, 1, 128, 512, seed=31)
    t = I.prefill_inputs(w, device="cuda")
    full = B.gta_prefill(t["q"], t["k"], t["c"], t["x"], t["w_p"], t["w_g"])
    cap = 400
    k_cache = torch.randn(w.batch, w.n_k, cap, w.d_h, device="cuda").to(torch.bfloat16)
    c_cache = torch.randn(w.batch, w.n_c, cap, w.d_l, device="cuda").to(torch.bfloat16)
    lens = torch.zeros(w.batch, dtype=torch.int32, device="cuda")
    B.gta_cache_append(k_cache, c_cache, t["k"][:, :, :-1].contiguous(), t["c"][:, :, :-1].contiguous(), lens)
    B.gta_cache_append(k_cache, c_cache, t["k"][:, :, -1:].contiguous(), t["c"][:, :, -1:].contiguous(), lens)
    assert lens.tolist() == [w.seq] * w.batch
    dec = B.gta_decode(t["q"][:, :, -1].contiguous(), k_cache, c_cache, lens, t["x"][:, -1].contiguous(),
                       t["w_p"], t["w_g"])
    torch.cuda.synchronize()
    assert_close(dec, full[:, -1].double().cpu().numpy(), torch.bfloat16, "decode vs prefill")


# --------------------------------------------------------------------------- cache append
@pytest.mark.parametrize("dt", ["bf16", "f32"])
@pytest.mark.parametrize("n_new", [1, 3, 700])
def test_cache_append_is_bit_exact(B, oracle, dt, n_new):
    tdt = torch.bfloat16 if dt == "bf16" else torch.float32
    nb, n_k, n_c, d_h, d_l, cap = 6, 4, 2, 64, 128, 1024
    g = torch.Generator("cpu").manual_seed(123 + n_new)
    k_cache = torch.randn(nb, n_k, cap, d_h, generator=g).to(tdt)
    c_cache = torch.randn(nb, n_c, cap, d_l, generator=g).to(tdt)
    k_new = torch.randn(nb, n_k, n_new, d_h, generator=g).to(tdt)
    c_new = torch.randn(nb, n_c, n_new, d_l, generator=g).to(tdt)
    lens = torch.tensor([0, 1, cap - n_new, cap - n_new + 1, cap, 17], dtype=torch.int32)  # two overflow
    shape = oracle.Shape(nb, 0, 8, 4, 4, n_k, n_c, d_h, d_l)
    wk, wc, wl, wov = oracle.cache_append(shape, k_cache, c_cache, cap, k_new, c_new, n_new, lens.numpy())
    assert wov == 1

    dk, dc, dl = k_cache.cuda(), c_cache.cuda(), lens.cuda()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.gta_cache_append(dk, dc, k_new.cuda(), c_new.cuda(), dl, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == B.GTA_ERR_CACHE_FULL
    assert dl.cpu().numpy().tolist() == wl.tolist()

    def bits(t):
        t = t.cpu().contiguous()
        return t.view(torch.int16).numpy().view(np.uint16) if t.dtype == torch.bfloat16 else t.numpy().view(np.uint32)

    want_k = wk if dt == "bf16" else wk.view(np.uint32)
    want_c = wc if dt == "bf16" else wc.view(np.uint32)
    assert np.array_equal(bits(dk), want_k.reshape(bits(dk).shape))
    assert np.array_equal(bits(dc), want_c.reshape(bits(dc).shape))


def test_append_then_decode_sequence_of_steps(B, oracle):
    """Three decode steps with appends in between track the oracle's cache model exactly."""
    w = I.Workload("steps", "decode", "bf16", 4, 0, 128, 4, 2, 2, 1, 128, 256, seed=55)
    lens0 = [10, 64, 0, 127]
    t = I.decode_inputs(w, device="cuda", s_cap=160, seq_lens=lens0)
    kc, cc, lens = t["k_cache"].clone(), t["c_cache"].clone(), t["seq_lens"].clone()
    hk, hc, hl = kc.cpu(), cc.cpu(), lens.cpu().numpy()
    g = torch.Generator("cpu").manual_seed(8)
    shape = oracle_shape(w, seq=0)
    for _ in range(3):
        k_new = torch.randn(w.batch, w.n_k, 1, w.d_h, generator=g).to(torch.bfloat16)
        c_new = torch.randn(w.batch, w.n_c, 1, w.d_l, generator=g).to(torch.bfloat16)
        q = torch.randn(w.batch, w.n_q, w.d_h, generator=g).to(torch.bfloat16)
        x_t = torch.randn(w.batch, w.d_model, generator=g).to(torch.bfloat16)
        B.gta_cache_append(kc, cc, k_new.cuda(), c_new.cuda(), lens)
        out = B.gta_decode(q.cuda(), kc, cc, lens, x_t.cuda(), t["w_p"], t["w_g"])
        nk, nc, hl, _ = oracle.cache_append(shape, hk, hc, 160, k_new, c_new, 1, hl)
        hk = torch.from_numpy(nk.view(np.int16)).view(torch.bfloat16).reshape(hk.shape)
        hc = torch.from_numpy(nc.view(np.int16)).view(torch.bfloat16).reshape(hc.shape)
        want = oracle.decode(shape, q, hk, hc, hl, 160, x_t, t["w_p"].cpu(), t["w_g"].cpu())
        torch.cuda.synchronize()
        assert lens.cpu().numpy().tolist() == hl.tolist()
        assert torch.equal(kc.cpu(), hk) and torch.equal(cc.cpu(), hc)
        assert_close(out, want, torch.bfloat16, "step")


# --------------------------------------------------------------------------- paged cache
def _paged_decode_case(B, oracle, w, page_size, seq_lens=None, s_cap=None, sample=None, holes=True):
    """gta_decode_paged against the oracle reading the same pools through the same block table."""
    t = I.paginate(_nan_behind_the_live_rows(I.decode_inputs(w, device="cuda", s_cap=s_cap, seq_lens=seq_lens)),
                   page_size, seed=w.seed)
    table = t["block_table"].clone()
    if holes:   # entries no live token maps to are never read: poison them
        lens_h = t["seq_lens"].cpu().tolist()
        for b, n in enumerate(lens_h):
            table[b, -(-n // page_size):] = -7
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    shape = B.decode_shape(t["q"], t["k_pool"], t["c_pool"], t["x_t"], t["w_p"])
    ws = torch.full((B.decode_paged_workspace_bytes(shape, page_size, t["max_pages"]),), 0xFF, dtype=torch.uint8,
                    device="cuda")
    out = B.gta_decode_paged(t["q"], t["k_pool"], t["c_pool"], table, t["seq_lens"], t["x_t"], t["w_p"], t["w_g"],
                             status_word=status, workspace=ws)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    idx = list(range(w.batch)) if sample is None else sample
    sel = torch.as_tensor(idx, device="cuda", dtype=torch.long)
    lens = t["seq_lens"][sel].cpu().numpy()
    # the oracle sees the pages of the sampled sequences only, renumbered (its view walks every entry)
    n_used = max(1, -(-int(lens.max()) // page_size)) if len(idx) else 1
    sub = t["block_table"][sel][:, :n_used].cpu().numpy()
    pages, inverse = np.unique(sub, return_inverse=True)
    pp = torch.as_tensor(pages, device="cuda", dtype=torch.long)
    want = oracle.decode_paged(oracle_shape(I.scaled(w, batch=len(idx)), seq=0), t["q"][sel].cpu(),
                               t["k_pool"][pp].cpu(), t["c_pool"][pp].cpu(), inverse.reshape(sub.shape), page_size,
                               lens, t["x_t"][sel].cpu(), t["w_p"].cpu(), t["w_g"].cpu())
    return assert_close(out[sel], want, w.torch_dtype(), w.name)


PAGED_DECODE = [
    # name, dtype, B, H, n_h, n_q, n_k, n_c, d_h, d_l, page_size, lens
    ("bf16_pages_of_64", "bf16", 6, 256, 8, 4, 4, 1, 128, 512, 64, [1, 63, 64, 65, 700, 0]),
    ("bf16_pages_of_128_batch_40", "bf16", 40, 256, 8, 4, 4, 1, 128, 512, 128, [1 + (37 * i) % 600 for i in range(40)]),
    ("bf16_pages_of_256_paper_1b_shape", "bf16", 3, 1280, 20, 5, 1, 1, 64, 128, 256, [333, 1000, 256]),
    ("bf16_pages_of_64_two_latents", "bf16", 5, 256, 8, 4, 4, 2, 128, 256, 64, [129, 1, 64, 400, 33]),
    # 16-token and 64-token sub-tiles of the tensor-memory stream kernel behind a block table
    ("bf16_pages_of_64_eight_key_groups_dl1024", "bf16", 4, 512, 8, 8, 8, 1, 128, 1024, 64, [257, 15, 64, 500]),
    ("bf16_pages_of_128_two_key_groups_dl256", "bf16", 4, 256, 8, 4, 2, 1, 128, 256, 128, [300, 0, 128, 65]),
    # page sizes the streaming kernel does not take (no multiple of 64), and fp32: the plain-ALU kernels
    ("bf16_pages_of_16", "bf16", 4, 128, 4, 2, 2, 1, 128, 256, 16, [0, 512, 1, 300]),
    ("bf16_pages_of_48", "bf16", 3, 128, 8, 4, 2, 2, 64, 128, 48, [200, 5, 129]),
    ("f32_pages_of_5", "f32", 3, 96, 6, 6, 3, 1, 32, 64, 5, [100, 7, 260]),
]


@pytest.mark.parametrize("case", PAGED_DECODE, ids=[c[0] for c in PAGED_DECODE])
def test_decode_paged_small_shapes(B, oracle, case):
    name, dt, nb, H, n_h, n_q, n_k, n_c, d_h, d_l, page_size, lens = case
    w = I.Workload(name, "decode", dt, nb, 0, H, n_h, n_q, n_k, n_c, d_h, d_l, seed=77)
    _paged_decode_case(B, oracle, w, page_size, seq_lens=lens, s_cap=max(lens) + 13)


def test_decode_paged_config3_full_size_sampled_sequences(B, oracle):
    w = I.CONFIGS["c3_decode_bf16"]
    _paged_decode_case(B, oracle, w, 64, sample=[0, w.batch // 2, w.batch - 1])


def test_decode_paged_is_bitwise_the_contiguous_decode_on_the_streaming_path(B):
    """Same kernels, same order of operations: only the tile addresses differ."""
    w = I.Workload("paged_vs_flat", "decode", "bf16", 9, 0, 256, 8, 4, 4, 1, 128, 512, seed=3)
    lens = [257, 256, 255, 1, 2, 1000, 64, 128, 511]
    t = I.paginate(I.decode_inputs(w, device="cuda", s_cap=1024, seq_lens=lens), 128, seed=1)
    flat = B.gta_decode(t["q"], t["k_cache"], t["c_cache"], t["seq_lens"], t["x_t"], t["w_p"], t["w_g"])
    paged = B.gta_decode_paged(t["q"], t["k_pool"], t["c_pool"], t["block_table"], t["seq_lens"], t["x_t"],
                               t["w_p"], t["w_g"])
    torch.cuda.synchronize()
    assert torch.equal(flat, paged)


@pytest.mark.parametrize("dt", ["bf16", "f32"])
@pytest.mark.parametrize("n_new", [1, 3, 200])
def test_cache_append_paged_is_bit_exact(B, oracle, dt, n_new):
    tdt = torch.bfloat16 if dt == "bf16" else torch.float32
    nb, n_k, n_c, d_h, d_l, page_size, max_pages = 6, 4, 2, 64, 128, 64, 5
    cap = page_size * max_pages
    g = torch.Generator("cpu").manual_seed(321 + n_new)
    n_pages = nb * max_pages + 4
    k_pool = torch.randn(n_pages, n_k, page_size, d_h, generator=g).to(tdt)
    c_pool = torch.randn(n_pages, n_c, page_size, d_l, generator=g).to(tdt)
    k_new = torch.randn(nb, n_k, n_new, d_h, generator=g).to(tdt)
    c_new = torch.randn(nb, n_c, n_new, d_l, generator=g).to(tdt)
    table = torch.randperm(n_pages, generator=g)[: nb * max_pages].reshape(nb, max_pages).to(torch.int32)
    # page boundaries inside the new rows, a full sequence and one that would overflow
    lens = torch.tensor([0, page_size - 1, cap - n_new, cap - n_new + 1, cap, 2 * page_size - 2], dtype=torch.int32)
    wk, wc, wl, wov = oracle.cache_append_paged(k_pool, c_pool, table.numpy(), page_size, k_new, c_new, lens.numpy())
    assert wov == 1

    dk, dc, dl = k_pool.cuda(), c_pool.cuda(), lens.cuda()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.gta_cache_append_paged(dk, dc, table.cuda(), k_new.cuda(), c_new.cuda(), dl, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == B.GTA_ERR_CACHE_FULL
    assert dl.cpu().numpy().tolist() == wl.tolist()

    def bits(t):
        t = t.cpu().contiguous()
        return t.view(torch.int16).numpy().view(np.uint16) if t.dtype == torch.bfloat16 else t.numpy().view(np.uint32)

    want_k = wk if dt == "bf16" else wk.view(np.uint32)
    want_c = wc if dt == "bf16" else wc.view(np.uint32)
    assert np.array_equal(bits(dk), want_k.reshape(bits(dk).shape))
    assert np.array_equal(bits(dc), want_c.reshape(bits(dc).shape))


def test_paged_append_then_decode_sequence_of_steps(B, oracle):
    """Decode steps over a paged cache, each after an append that may open a new page."""
    w = I.Workload("paged_steps", "decode", "bf16", 4, 0, 128, 4, 2, 2, 1, 128, 256, seed=56)
    page_size = 64
    t = I.paginate(I.decode_inputs(w, device="cuda", s_cap=192, seq_lens=[10, 63, 0, 127]), page_size, seed=2)
    kp, cp, lens, table = t["k_pool"].clone(), t["c_pool"].clone(), t["seq_lens"].clone(), t["block_table"]
    hk, hc, hl, ht = kp.cpu(), cp.cpu(), lens.cpu().numpy(), table.cpu().numpy()
    g = torch.Generator("cpu").manual_seed(9)
    shape = oracle_shape(w, seq=0)
    for _ in range(3):
        k_new = torch.randn(w.batch, w.n_k, 1, w.d_h, generator=g).to(torch.bfloat16)
        c_new = torch.randn(w.batch, w.n_c, 1, w.d_l, generator=g).to(torch.bfloat16)
        q = torch.randn(w.batch, w.n_q, w.d_h, generator=g).to(torch.bfloat16)
        x_t = torch.randn(w.batch, w.d_model, generator=g).to(torch.bfloat16)
        B.gta_cache_append_paged(kp, cp, table, k_new.cuda(), c_new.cuda(), lens)
        out = B.gta_decode_paged(q.cuda(), kp, cp, table, lens, x_t.cuda(), t["w_p"], t["w_g"])
        nk, nc, hl, _ = oracle.cache_append_paged(hk, hc, ht, page_size, k_new, c_new, hl)
        hk = torch.from_numpy(nk.view(np.int16)).view(torch.bfloat16).reshape(hk.shape)
        hc = torch.from_numpy(nc.view(np.int16)).view(torch.bfloat16).reshape(hc.shape)
        want = oracle.decode_paged(shape, q, hk, hc, ht, page_size, hl, x_t, t["w_p"].cpu(), t["w_g"].cpu())
        torch.cuda.synchronize()
        assert lens.cpu().numpy().tolist() == hl.tolist()
        assert torch.equal(kp.cpu(), hk) and torch.equal(cp.cpu(), hc)
        assert_close(out, want, torch.bfloat16, "paged step")


@pytest.mark.parametrize("page_size", [64, 16])
def test_block_table_entry_outside_the_pool_raises_the_status_word(B, page_size):
    """Both kernel families check the entries they use: the call completes, touches nothing outside the
    pools and reports GTA_ERR_BAD_PAGE."""
    w = I.Workload("bad_page", "decode", "bf16", 3, 0, 128, 4, 2, 2, 1, 128, 256, seed=4)
    t = I.paginate(I.decode_inputs(w, device="cuda", s_cap=256, seq_lens=[100, 200, 30]), page_size, seed=3)
    table = t["block_table"].clone()
    table[1, 1] = t["n_pages"] + 5
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = B.gta_decode_paged(t["q"], t["k_pool"], t["c_pool"], table, t["seq_lens"], t["x_t"], t["w_p"], t["w_g"],
                             status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == B.GTA_ERR_BAD_PAGE
    assert torch.isfinite(out.float()).all()
    # the append refuses the row as well: sequence 1's next token falls into the bad page when it starts there
    lens = torch.tensor([100, page_size, 30], dtype=torch.int32, device="cuda")
    status.zero_()
    before_k, before_c = t["k_pool"].clone(), t["c_pool"].clone()
    B.gta_cache_append_paged(t["k_pool"], t["c_pool"], table, t["k_new"], t["c_new"], lens, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == B.GTA_ERR_BAD_PAGE
    changed = (t["k_pool"] != before_k).flatten(1).any(1).sum().item()
    assert changed == 2   # the two good sequences wrote one row each, each in a page of its own


# --------------------------------------------------------------------------- bounded waits
def test_a_wait_that_runs_out_unwinds_the_attention_kernel(B, oracle):
    """With the test hook one softmax warp of every CTA pair keeps its first arrival to itself and the waits
    give up after 2 ms: the call must come back (no hang), report GTA_ERR_TIMEOUT in the status word, leave the
    context usable, and the next ordinary call must give bit for bit what the call before gave."""
    w = I.Workload("timeout", "prefill", "bf16", 1, 200, 128, 4, 1, 1, 1, 128, 256, seed=99)   # one item, two key tiles
    t = I.prefill_inputs(w, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    args = (t["q"], t["k"], t["c"], t["x"], t["w_p"], t["w_g"])
    before = B.gta_prefill(*args, status_word=status).clone()
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    B.debug_attention_wait(limit_ns=2_000_000, withhold_first_arrive=True)
    try:
        junk = B.gta_prefill(*args, status_word=status)
        torch.cuda.synchronize()                      # returns: every wait is bounded
        assert int(status.item()) == B.GTA_ERR_TIMEOUT
        del junk
    finally:
        B.debug_attention_wait(limit_ns=0, withhold_first_arrive=False)
    status.zero_()
    after = B.gta_prefill(*args, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(after.view(torch.int16), before.view(torch.int16))
    tc = cpu(t)
    want = oracle.prefill(oracle_shape(w), tc["q"], tc["k"], tc["c"], tc["x"], tc["w_p"], tc["w_g"])
    assert_close(after, want, torch.bfloat16, "after a timed-out call")


def test_a_wait_that_runs_out_unwinds_the_decode_stream_kernel(B, oracle):
    """The same for the decode stream kernel that keeps its sums in tensor memory: one warp of every CTA keeps its
    first "weights written" arrival to itself and the waits give up after 2 ms; the call comes back with
    GTA_ERR_TIMEOUT, and the next ordinary call gives bit for bit what the call before gave."""
    w = I.Workload("timeout", "decode", "bf16", 3, 0, 256, 8, 4, 4, 1, 128, 512, seed=98)
    lens = [200, 64, 33]
    t = I.decode_inputs(w, device="cuda", s_cap=208, seq_lens=lens)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    args = (t["q"], t["k_cache"], t["c_cache"], t["seq_lens"], t["x_t"], t["w_p"], t["w_g"])
    before = B.gta_decode(*args, status_word=status).clone()
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    B.debug_decode_wait(limit_ns=2_000_000, withhold_first_arrive=True)
    try:
        junk = B.gta_decode(*args, status_word=status)
        torch.cuda.synchronize()                      # returns: every wait is bounded
        assert int(status.item()) == B.GTA_ERR_TIMEOUT
        del junk
    finally:
        B.debug_decode_wait(limit_ns=0, withhold_first_arrive=False)
    status.zero_()
    after = B.gta_decode(*args, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(after.view(torch.int16), before.view(torch.int16))
    want = oracle.decode(oracle_shape(w, seq=0), t["q"].cpu(), t["k_cache"].cpu(), t["c_cache"].cpu(), lens, 208,
                         t["x_t"].cpu(), t["w_p"].cpu(), t["w_g"].cpu())
    assert_close(after, want, torch.bfloat16, "after a timed-out call")


# --------------------------------------------------------------------------- append + decode in one call
STEP_CASES = [
    # name, dtype, H, n_h, n_q, n_k, n_c, d_h, d_l, lens BEFORE the step, S_cap
    ("bf16_around_the_sub_tiles", "bf16", 256, 8, 4, 4, 1, 128, 512, [0, 1, 30, 31, 32, 33, 63, 64, 65, 700], 720),
    ("bf16_full_and_nearly_full", "bf16", 128, 4, 2, 2, 1, 128, 256, [128, 127, 5, 126], 128),
    ("bf16_two_latents_dh64", "bf16", 128, 8, 4, 2, 2, 64, 128, [200, 0, 129, 63, 64], 256),
    ("bf16_paper_1b_shape", "bf16", 1280, 20, 5, 1, 1, 64, 128, [333, 127, 128], 400),
    ("bf16_batch_40", "bf16", 256, 8, 4, 4, 1, 128, 512, [(37 * i) % 300 for i in range(40)], 320),
    # 16-token sub-tiles (eight key groups on the rows of one MMA), lengths around them, a full cache
    ("bf16_eight_key_groups_dl1024", "bf16", 512, 16, 8, 8, 1, 128, 1024, [0, 1, 14, 15, 16, 17, 31, 32, 300, 304], 304),
    ("bf16_two_maps_per_key_group_dl512", "bf16", 256, 16, 8, 4, 1, 128, 512, [95, 96, 97, 0, 640], 641),
    ("bf16_one_key_group_dl1024", "bf16", 256, 8, 8, 1, 1, 128, 1024, [47, 48, 200], 208),
    ("bf16_64_token_sub_tiles_dl256", "bf16", 256, 8, 8, 2, 1, 128, 256, [63, 64, 65, 0, 127, 128, 300], 301),
    ("bf16_eight_key_groups_dl256", "bf16", 512, 8, 8, 8, 1, 128, 256, [15, 16, 17, 100], 104),
    ("f32_plain_alu_kernels", "f32", 96, 6, 6, 3, 1, 32, 64, [100, 7, 0, 260], 261),
]


@pytest.mark.parametrize("case", STEP_CASES, ids=[c[0] for c in STEP_CASES])
def test_decode_append_equals_append_then_decode(B, oracle, case):
    name, dt, H, n_h, n_q, n_k, n_c, d_h, d_l, lens, cap = case
    w = I.Workload(name, "decode", dt, len(lens), 0, H, n_h, n_q, n_k, n_c, d_h, d_l, seed=83)
    t = I.decode_inputs(w, device="cuda", s_cap=cap, seq_lens=lens)
    status_a = torch.zeros(1, dtype=torch.int32, device="cuda")
    status_b = torch.zeros(1, dtype=torch.int32, device="cuda")
    # the two calls
    k_a, c_a, lens_a = t["k_cache"].clone(), t["c_cache"].clone(), t["seq_lens"].clone()
    B.gta_cache_append(k_a, c_a, t["k_new"], t["c_new"], lens_a, status_word=status_a)
    want = B.gta_decode(t["q"], k_a, c_a, lens_a, t["x_t"], t["w_p"], t["w_g"], status_word=status_a)
    # the one call, twice in a row on fresh copies (leftovers in the workspace must not matter)
    shape = B.decode_shape(t["q"], t["k_cache"], t["c_cache"], t["x_t"], t["w_p"])
    ws = Guarded((B.decode_workspace_bytes(shape, cap),), torch.uint8)
    for rep in range(2):
        k_b, c_b, lens_b = t["k_cache"].clone(), t["c_cache"].clone(), t["seq_lens"].clone()
        status_b.zero_()
        og = Guarded(tuple(want.shape), want.dtype)
        got = B.gta_decode_append(t["q"], k_b, c_b, t["k_new"], t["c_new"], lens_b, t["x_t"], t["w_p"], t["w_g"],
                                  out=og.t, workspace=ws.t, status_word=status_b)
        torch.cuda.synchronize()
        ws.check(name + " workspace"); og.check(name + " out")
        assert int(status_b.item()) == int(status_a.item())
        assert int(status_b.item()) == (B.GTA_ERR_CACHE_FULL if any(n >= cap for n in lens) else 0)
        assert lens_b.tolist() == lens_a.tolist() == [n + 1 if n < cap else n for n in lens]
        bits = torch.int16 if dt == "bf16" else torch.int32
        assert torch.equal(k_b.view(bits), k_a.view(bits)) and torch.equal(c_b.view(bits), c_a.view(bits))
        assert torch.equal(got.view(bits), want.view(bits))
    live = max(lens_a.tolist())
    ref = oracle.decode(oracle_shape(w, seq=0), t["q"].cpu(), k_a[:, :, :live].contiguous().cpu(),
                        c_a[:, :, :live].contiguous().cpu(), lens_a.cpu().numpy(), live, t["x_t"].cpu(), t["w_p"].cpu(),
                        t["w_g"].cpu())
    assert_close(got, ref, w.torch_dtype(), name)


def _step_full_size(B, oracle, w, sample):
    """The fused step as the benchmark times it (full size, lengths that do not count the new token yet): result on
    sampled sequences against the oracle over the caches WITH the new rows, the new rows bit for bit in every
    sequence's cache, the rows around them untouched, the lengths advanced."""
    t = I.decode_inputs(w, device="cuda")
    lens_after = t["seq_lens"].clone()
    lens = lens_after - 1                                   # the caches hold all tokens but the one being decoded
    pos = lens.long()
    ar = torch.arange(w.batch, device="cuda")
    k_before = t["k_cache"][ar, :, pos + 1].clone()         # the row behind the new one must stay as it is
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = B.gta_decode_append(t["q"], t["k_cache"], t["c_cache"], t["k_new"], t["c_new"], lens, t["x_t"], t["w_p"],
                              t["w_g"], status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.equal(lens, lens_after)
    assert torch.equal(t["k_cache"][ar, :, pos].view(torch.int16), t["k_new"][:, :, 0].view(torch.int16))
    assert torch.equal(t["c_cache"][ar, :, pos].view(torch.int16), t["c_new"][:, :, 0].view(torch.int16))
    assert torch.equal(t["k_cache"][ar, :, pos + 1].view(torch.int16), k_before.view(torch.int16))
    sel = torch.as_tensor(sample, device="cuda", dtype=torch.long)
    sub = lens_after[sel].cpu().numpy()
    cap = int(sub.max())
    want = oracle.decode(oracle_shape(I.scaled(w, batch=len(sample)), seq=0), t["q"][sel].cpu(),
                         t["k_cache"][sel][:, :, :cap].contiguous().cpu(), t["c_cache"][sel][:, :, :cap].contiguous().cpu(),
                         sub, cap, t["x_t"][sel].cpu(), t["w_p"].cpu(), t["w_g"].cpu())
    assert_close(out[sel], want, torch.bfloat16, w.name + " fused step")


def test_decode_append_config3_full_size_sampled_sequences(B, oracle):
    w = I.CONFIGS["c3_decode_bf16"]
    _step_full_size(B, oracle, w, [0, 7, 16, 31])


def test_decode_append_config5_full_size_sampled_sequences(B, oracle):
    w = I.CONFIGS["c5_ragged_decode_bf16"]
    lens = I.decode_seq_lens(w).numpy()
    order = np.argsort(lens)
    _step_full_size(B, oracle, w, sorted({int(order[0]), int(order[-1]), int(order[len(order) // 2]), 0, 127}))
