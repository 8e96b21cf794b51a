"""GPU parity of the comparison operators (grouped-query attention, App. B.3 of the paper; multi-head attention as
its special case) against their fp64 oracle, element by element on identical seeded inputs."""
import numpy as np
import pytest
import torch

from paper_2506_17286_b200 import inputs as I
from tests.parity_utils import Guarded, assert_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2506_17286_b200 import build, binding
    build.build()
    binding.lib()
    return binding


def _prefill_case(B, oracle, nb, n_h, n_kv, N, d_h, causal=True, scale=0.0, rows=None, seed=3):
    t = I.gqa_prefill_inputs(nb, n_h, n_kv, N, d_h, seed=seed, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    og = Guarded((nb, n_h, N, d_h), torch.bfloat16)
    out = B.gta_ref_gqa_prefill(t["q"], t["k"], t["v"], causal=causal, softmax_scale=scale, out=og.t, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    og.check("gqa prefill out")
    want = oracle.gqa_prefill(t["q"].cpu(), t["k"].cpu(), t["v"].cpu(), causal=causal, scale=scale, rows=rows)
    got = out if rows is None else out[:, :, torch.as_tensor(rows, device="cuda")]
    return assert_close(got, want, torch.bfloat16, f"gqa prefill {nb}x{n_h}/{n_kv}x{N}x{d_h}")


GQA_PREFILL = [
    # B, n_h, n_kv, N, d_h
    (2, 8, 2, 300, 128),
    (1, 20, 5, 333, 64),        # the 1B model's grouping, value heads of 64 columns (the narrow-latent mode)
    (1, 4, 4, 200, 128),        # one key / value head per query head: multi-head attention
    (3, 6, 1, 129, 64),         # one key / value head for all: multi-query attention
    (1, 2, 2, 1, 128),
]


@pytest.mark.parametrize("case", GQA_PREFILL, ids=[f"b{c[0]}_h{c[1]}_kv{c[2]}_n{c[3]}_d{c[4]}" for c in GQA_PREFILL])
def test_gqa_prefill_small_shapes(B, oracle, case):
    _prefill_case(B, oracle, *case)


def test_gqa_prefill_non_causal_and_explicit_scale(B, oracle):
    _prefill_case(B, oracle, 1, 4, 2, 200, 128, causal=False, scale=0.05)


def _sample_rows(N, n=24, seed=0):
    rng = np.random.default_rng(seed)
    fixed = [0, 1, 127, 128, 255, 256, N // 2, N - 2, N - 1]
    return sorted(set(fixed) | set(int(v) for v in rng.integers(0, N, n)))


@pytest.mark.parametrize("case", [(4, 16, 4, 2048, 128), (8, 20, 5, 2048, 64)], ids=["c2_shape", "gqa_1b_shape"])
def test_gqa_prefill_full_size_sampled_rows(B, oracle, case):
    _prefill_case(B, oracle, *case, rows=_sample_rows(case[3]))


def _decode_case(B, oracle, n_h, n_kv, d_h, lens, sample=None, seed=5):
    nb = len(lens)
    t = I.gqa_decode_inputs(nb, n_h, n_kv, d_h, lens, s_cap=max(lens) + 11, seed=seed, device="cuda")
    for b, n in enumerate(lens):      # what uninitialised memory may hold behind the live rows
        t["k_cache"][b, :, n:] = float("nan")
        t["v_cache"][b, :, n:] = float("nan")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    shape = B.gqa_shape(batch=nb, seq=0, n_heads=n_h, n_kv=n_kv, d_h=d_h, dtype=torch.bfloat16)
    ws = Guarded((B.gqa_decode_workspace_bytes(shape),), torch.uint8)
    og = Guarded((nb, n_h, d_h), torch.bfloat16)
    out = B.gta_ref_gqa_decode(t["q"], t["k_cache"], t["v_cache"], t["seq_lens"], out=og.t, workspace=ws.t,
                               status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ws.check("gqa decode workspace"); og.check("gqa decode out")
    idx = list(range(nb)) if sample is None else sample
    sel = torch.as_tensor(idx, device="cuda")
    cap = max(max(lens[i] for i in idx), 1)
    kc = torch.nan_to_num(t["k_cache"][sel][:, :, :cap]).cpu()
    vc = torch.nan_to_num(t["v_cache"][sel][:, :, :cap]).cpu()
    want = oracle.gqa_decode(t["q"][sel].cpu(), kc, vc, [lens[i] for i in idx])
    return assert_close(out[sel], want, torch.bfloat16, f"gqa decode {n_h}/{n_kv}x{d_h}")


GQA_DECODE = [
    # n_h, n_kv, d_h, lens
    (8, 2, 128, [1, 63, 64, 65, 700]),
    (20, 5, 64, [333, 0, 1000, 17]),
    (4, 4, 128, [300, 2, 511]),
    (8, 1, 64, [129, 64, 1]),
    (16, 4, 128, [1 + (37 * i) % 300 for i in range(40)]),
]


@pytest.mark.parametrize("case", GQA_DECODE, ids=[f"h{c[0]}_kv{c[1]}_d{c[2]}_b{len(c[3])}" for c in GQA_DECODE])
def test_gqa_decode_small_shapes(B, oracle, case):
    _decode_case(B, oracle, *case)


def test_gqa_decode_full_size_sampled_sequences(B, oracle):
    _decode_case(B, oracle, 16, 4, 128, [4096] * 32, sample=[0, 7, 31])                    # the c3 shape as GQA
    lens = [1024 + (977 * i) % 7000 for i in range(64)]
    _decode_case(B, oracle, 20, 5, 64, lens, sample=[0, 13, 63])                           # the 1B model's grouping


def test_gqa_rejects_what_it_does_not_cover(B):
    t = I.gqa_prefill_inputs(1, 4, 2, 64, 32, device="cuda")
    with pytest.raises(B.GtaError) as e:
        B.gta_ref_gqa_prefill(t["q"], t["k"], t["v"])
    assert e.value.status == B.GTA_ERR_UNSUPPORTED          # head dimension 32
    t = I.gqa_decode_inputs(2, 18, 2, 64, [5, 9], device="cuda")
    with pytest.raises(B.GtaError) as e:
        B.gta_ref_gqa_decode(t["q"], t["k_cache"], t["v_cache"], t["seq_lens"], workspace=torch.empty(1 << 20, dtype=torch.uint8, device="cuda"))
    assert e.value.status == B.GTA_ERR_UNSUPPORTED          # nine query heads per key / value head
