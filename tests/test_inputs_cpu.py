"""CPU checks of the seeded input generators that both the CUDA side and the oracle side read."""
import numpy as np
import torch

from paper_2506_17286_b200 import inputs as I


def _bits(t):
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def test_paginate_scatters_the_caches_without_changing_a_row(oracle):
    w = I.Workload("pg", "decode", "bf16", 3, 0, 64, 4, 2, 2, 1, 16, 32, seed=12)
    t = I.decode_inputs(w, s_cap=50, seq_lens=[7, 50, 0])
    p = I.paginate(t, 16, seed=4)
    assert p["max_pages"] == 4 and p["n_pages"] == 3 * 4 + 3
    table = p["block_table"].numpy()
    assert table.shape == (3, 4) and len(set(table.ravel().tolist())) == 12        # every page handed out once
    assert table.min() >= 0 and table.max() < p["n_pages"]
    # read back through the oracle's token-by-token view: the first s_cap rows are the caches, bit for bit
    kv = oracle.paged_view(p["k_pool"], table, 16)
    cv = oracle.paged_view(p["c_pool"], table, 16)
    assert np.array_equal(kv[:, :, :50], _bits(t["k_cache"])) and np.array_equal(cv[:, :, :50], _bits(t["c_cache"]))
    # same seed, same layout; another seed, another permutation
    assert torch.equal(I.paginate(t, 16, seed=4)["block_table"], p["block_table"])
    assert not torch.equal(I.paginate(t, 16, seed=5)["block_table"], p["block_table"])


def test_layer_inputs_shapes_and_determinism():
    w = I.Workload("li", "prefill", "bf16", 2, 5, 64, 4, 2, 1, 1, 16, 32, seed=3)
    a, b = I.layer_inputs(w), I.layer_inputs(w)
    assert a["x"].shape == (2, 5, 64) and a["w_qkc"].shape == (64, (2 + 1) * 16 + 32)
    assert a["w_p"].shape == (4, 32, 16) and a["w_g"].shape == (64, 64) and a["w_o"].shape == (64, 64)
    assert all(v.dtype == torch.bfloat16 for v in a.values())
    assert all(torch.equal(a[k], b[k]) for k in a)
    assert not torch.equal(I.layer_inputs(I.scaled(w, seed=4))["x"], a["x"])
