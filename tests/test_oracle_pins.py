"""CPU-only pins of the fp64 oracle against what the paper and the mathematics fix.

Every check compares the oracle with something that is not the oracle: a textbook attention
written here with numpy, an einsum restatement of the definition, closed forms of the softmax,
invariants (row sums, causality, batch independence, sharing inside a head group) and the
ratios / cache widths the paper prints.  A dropped term, a wrong head map, a transposed
operand, a missing sigmoid or an off-by-one in the causal bound fails at least one of them.
"""
import numpy as np
import pytest

from oracle.gta_oracle import Shape

RNG = np.random.default_rng(20250617)


def _rand(*shape, scale=1.0):
    return RNG.standard_normal(shape) * scale


def _inputs(s: Shape, n=None):
    n = s.seq if n is None else n
    return dict(
        q=_rand(s.batch, s.n_q, n, s.d_h), k=_rand(s.batch, s.n_k, n, s.d_h),
        c=_rand(s.batch, s.n_c, n, s.d_l), x=_rand(s.batch, n, s.d_model),
        w_p=_rand(s.n_heads, s.d_l, s.d_h, scale=s.d_l ** -0.5),
        w_g=_rand(s.d_model, s.n_heads * s.d_h, scale=s.d_model ** -0.5),
    )


def _softmax_np(s, axis=-1):
    e = np.exp(s - s.max(axis=axis, keepdims=True))
    return e / e.sum(axis=axis, keepdims=True)


def _einsum_gta(s: Shape, t):
    """Independent restatement of Sec. 3.2-3.3 with whole-matrix einsums (definition form)."""
    B, N, nh = s.batch, s.seq, s.n_heads
    scale = s.scale or s.d_h ** -0.5
    out = np.zeros((B, N, nh, s.d_h))
    mask = np.tril(np.ones((N, N), dtype=bool)) if s.causal else np.ones((N, N), dtype=bool)
    for i in range(nh):
        g = i * s.n_q // nh
        kg, cg = g * s.n_k // s.n_q, g * s.n_c // s.n_q
        S = np.einsum("btd,bjd->btj", t["q"][:, g], t["k"][:, kg]) * scale
        S = np.where(mask[None], S, -np.inf)
        P = _softmax_np(S)
        gate = 1.0 / (1.0 + np.exp(-np.einsum("bth,he->bte", t["x"], t["w_g"][:, i * s.d_h:(i + 1) * s.d_h])))
        V = np.einsum("bjl,le->bje", t["c"][:, cg], t["w_p"][i])            # C W_P
        Vt = V[:, None, :, :] * gate[:, :, None, :]                          # V^{(t)}[b,t,j,e]
        out[:, :, i, :] = np.einsum("btj,btje->bte", P, Vt)
    return out


# ---------------------------------------------------------------- P1: reduction to MHA
@pytest.mark.parametrize("causal", [1, 0])
def test_reduces_to_multi_head_attention(oracle, causal):
    """Group size 1, W_P = slice selector, W_G = 0  =>  0.5 * textbook MHA (sigmoid(0) = 1/2)."""
    nh, dh, N, B, H = 3, 8, 17, 2, 12
    s = Shape(B, N, H, nh, nh, nh, 1, dh, nh * dh, causal)
    t = _inputs(s)
    t["w_g"][:] = 0.0
    t["w_p"][:] = 0.0
    for i in range(nh):
        t["w_p"][i, i * dh:(i + 1) * dh, :] = np.eye(dh)
    got = oracle.prefill(s, **t)
    want = np.zeros_like(got)
    for b in range(B):
        for i in range(nh):
            S = t["q"][b, i] @ t["k"][b, i].T / np.sqrt(dh)
            if causal:
                S = np.where(np.tril(np.ones((N, N), dtype=bool)), S, -np.inf)
            want[b, :, i, :] = _softmax_np(S) @ t["c"][b, 0][:, i * dh:(i + 1) * dh]
    np.testing.assert_allclose(got, 0.5 * want, rtol=1e-12, atol=1e-14)


# ---------------------------------------------------------------- P2: softmax rows
def test_probability_rows_sum_to_one_and_respect_mask(oracle):
    s = Shape(2, 19, 8, 4, 2, 1, 1, 8, 16, 1)
    t = _inputs(s)
    P = oracle.probs(s, t["q"], t["k"])
    assert P.shape == (2, 2, 19, 19)
    np.testing.assert_allclose(P.sum(-1), 1.0, atol=1e-14)
    assert (P >= 0).all()
    assert np.all(np.triu(P, k=1) == 0.0)          # nothing above the diagonal
    assert np.all(np.diagonal(P, axis1=-2, axis2=-1) > 0)  # the diagonal is included
    # probabilities equal an independent softmax of the scaled scores
    S = np.einsum("bgtd,bjd->bgtj", t["q"], t["k"][:, 0]) / np.sqrt(8)
    S = np.where(np.tril(np.ones((19, 19), dtype=bool)), S, -np.inf)
    np.testing.assert_allclose(P, _softmax_np(S), rtol=1e-12, atol=1e-15)


# ---------------------------------------------------------------- P3: causality
def test_future_tokens_do_not_change_earlier_rows(oracle):
    s = Shape(1, 24, 16, 4, 2, 2, 1, 8, 16, 1)
    t = _inputs(s)
    base = oracle.prefill(s, **t)
    cut = 13
    t2 = {k: v.copy() for k, v in t.items()}
    for name in ("q", "k", "c"):
        t2[name][:, :, cut:, :] += _rand(*t2[name][:, :, cut:, :].shape)
    t2["x"][:, cut:, :] += 1.0
    pert = oracle.prefill(s, **t2)
    assert np.array_equal(base[:, :cut], pert[:, :cut])        # bit-identical
    assert not np.allclose(base[:, cut:], pert[:, cut:])
    # and the non-causal operator does depend on the future
    s0 = Shape(1, 24, 16, 4, 2, 2, 1, 8, 16, 0)
    assert not np.allclose(oracle.prefill(s0, **t)[:, :cut], oracle.prefill(s0, **t2)[:, :cut])


# ---------------------------------------------------------------- P4: decode == last prefill row
@pytest.mark.parametrize("n_k,n_c", [(4, 1), (2, 2), (1, 1)])
def test_decode_equals_last_prefill_row_after_append(oracle, n_k, n_c):
    B, N, cap = 3, 11, 16
    s = Shape(B, N, 24, 8, 4, n_k, n_c, 8, 16, 1)
    t = _inputs(s)
    full = oracle.prefill(s, **t)
    # load the first N-1 tokens into empty caches, then append token N-1 as a decode step would
    k_cache = _rand(B, n_k, cap, s.d_h)   # garbage beyond the live part must not matter
    c_cache = _rand(B, n_c, cap, s.d_l)
    lens = np.zeros(B, dtype=np.int32)
    k_cache, c_cache, lens, ov = oracle.cache_append(
        s, k_cache, c_cache, cap, t["k"][:, :, :N - 1].copy(), t["c"][:, :, :N - 1].copy(), N - 1, lens)
    assert ov == 0 and (lens == N - 1).all()
    k_cache, c_cache, lens, ov = oracle.cache_append(
        s, k_cache, c_cache, cap, t["k"][:, :, N - 1:].copy(), t["c"][:, :, N - 1:].copy(), 1, lens)
    assert ov == 0 and (lens == N).all()
    got = oracle.decode(s, t["q"][:, :, N - 1].copy(), k_cache, c_cache, lens, cap,
                        t["x"][:, N - 1].copy(), t["w_p"], t["w_g"])
    np.testing.assert_allclose(got, full[:, N - 1], rtol=1e-12, atol=1e-15)


def test_decode_ragged_lengths_and_empty_sequence(oracle):
    B, cap = 4, 12
    s = Shape(B, 0, 8, 4, 2, 2, 1, 4, 8, 1)
    lens = np.array([12, 1, 0, 5], dtype=np.int32)
    q, xt = _rand(B, 2, 4), _rand(B, 8)
    kc, cc = _rand(B, 2, cap, 4), _rand(B, 1, cap, 8)
    w_p, w_g = _rand(4, 8, 4), _rand(8, 16)
    got = oracle.decode(s, q, kc, cc, lens, cap, xt, w_p, w_g)
    assert np.all(got[2] == 0.0)
    # len == 1: attention is the identity on the single cached latent
    gate = 1 / (1 + np.exp(-(xt[1] @ w_g)))
    want = np.stack([cc[1, 0, 0] @ w_p[i] for i in range(4)]) * gate.reshape(4, 4)
    np.testing.assert_allclose(got[1], want, rtol=1e-12)
    # each sequence equals a one-sequence call (independence from the other lengths)
    for b in (0, 3):
        s1 = Shape(1, 0, 8, 4, 2, 2, 1, 4, 8, 1)
        one = oracle.decode(s1, q[b:b + 1], kc[b:b + 1], cc[b:b + 1], lens[b:b + 1], cap, xt[b:b + 1], w_p, w_g)
        assert np.array_equal(one[0], got[b])


# ---------------------------------------------------------------- P5 / P6: brute force, two forms
@pytest.mark.parametrize("shape", [
    Shape(2, 7, 6, 4, 2, 1, 1, 4, 8, 1),      # keys shared by both maps
    Shape(1, 8, 10, 8, 4, 2, 2, 4, 4, 1),     # two latent groups, d_l == d_h
    Shape(2, 5, 6, 6, 6, 3, 1, 2, 6, 0),      # non-causal, one head per map
    Shape(1, 1, 3, 2, 1, 1, 1, 2, 4, 1),      # single token
    Shape(1, 6, 4, 4, 2, 2, 1, 3, 5, 1, 0.37),  # explicit softmax scale
])
def test_matches_einsum_restatement_and_definition_form(oracle, shape):
    t = _inputs(shape)
    want = _einsum_gta(shape, t)
    got = oracle.prefill(shape, **t)
    got_def = oracle.prefill(shape, **t, definition=True)
    np.testing.assert_allclose(got, want, rtol=1e-11, atol=1e-14)
    np.testing.assert_allclose(got_def, want, rtol=1e-11, atol=1e-14)
    np.testing.assert_allclose(got, got_def, rtol=1e-11, atol=1e-14)     # P6
    rows = [shape.seq - 1, 0]
    sub = oracle.prefill(shape, **t, rows=rows)
    assert np.array_equal(sub, got[:, rows])


def test_gate_uses_the_query_token_not_the_key_token(oracle):
    """Changing x at position j changes row j only (the gate never follows the key index)."""
    s = Shape(1, 9, 8, 2, 1, 1, 1, 4, 8, 1)
    t = _inputs(s)
    base = oracle.prefill(s, **t)
    t["x"][0, 3] += 2.0
    pert = oracle.prefill(s, **t)
    changed = np.any(base != pert, axis=(0, 2, 3))
    assert changed.tolist() == [j == 3 for j in range(9)]


# ---------------------------------------------------------------- P7 / P8: closed forms
def test_uniform_attention_closed_form(oracle):
    s = Shape(2, 10, 8, 4, 2, 2, 1, 4, 8, 1)
    t = _inputs(s)
    t["q"][:] = 0.0
    got = oracle.prefill(s, **t)
    csum = np.cumsum(t["c"][:, 0], axis=1) / np.arange(1, 11)[None, :, None]   # running mean
    gate = 1 / (1 + np.exp(-(t["x"] @ t["w_g"]))).reshape(2, 10, 4, 4)
    want = np.einsum("btl,ile->btie", csum, t["w_p"]) * gate
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-15)


def test_one_hot_attention_closed_form(oracle):
    N, dh = 8, 8
    s = Shape(1, N, 6, 2, 1, 1, 1, dh, 12, 1)
    t = _inputs(s)
    perm = RNG.permutation(N)
    t["k"][0, 0] = 200.0 * np.eye(dh)[perm]              # key j points along axis perm[j]
    target = np.array([RNG.integers(0, tt + 1) for tt in range(N)])   # a visible key per row
    t["q"][0, 0] = np.eye(dh)[perm[target]] * np.sqrt(dh)
    got = oracle.prefill(s, **t)
    gate = 1 / (1 + np.exp(-(t["x"][0] @ t["w_g"]))).reshape(N, 2, dh)
    want = np.einsum("tl,ile->tie", t["c"][0, 0][target], t["w_p"]) * gate
    np.testing.assert_allclose(got[0], want, rtol=1e-10, atol=1e-12)


# ---------------------------------------------------------------- P9: sharing inside a group
def test_heads_of_one_map_share_probabilities(oracle):
    s = Shape(1, 12, 8, 4, 2, 2, 1, 4, 8, 1)
    t = _inputs(s)
    wg = t["w_g"].reshape(8, 4, 4)
    t["w_p"][1] = t["w_p"][0]; wg[:, 1] = wg[:, 0]        # heads 0,1: same map (group 0)
    t["w_p"][2] = t["w_p"][0]; wg[:, 2] = wg[:, 0]        # head 2: other map (group 1)
    t["w_g"] = wg.reshape(8, 16)
    out = oracle.prefill(s, **t)
    assert np.array_equal(out[:, :, 0], out[:, :, 1])
    assert not np.allclose(out[:, 1:, 0], out[:, 1:, 2])
    # head -> group map is by contiguous blocks: swapping query groups swaps head blocks
    t2 = dict(t); t2["q"] = t["q"][:, ::-1].copy(); t2["k"] = t["k"][:, ::-1].copy()
    out2 = oracle.prefill(s, **t2)
    assert np.array_equal(out2[:, :, 2], out[:, :, 0])


# ---------------------------------------------------------------- P10: printed cost figures
def test_cost_model_matches_printed_ratios(oracle):
    """Table 3 closed forms at the 1B hyper-parameters (App. A, model table) give the printed
    37.5 % attention cost and 30 % cache of GQA-1B; printed cache widths 192 / 320 / 384."""
    N = 2048
    gta_1b = Shape(1, N, 1280, 20, 5, 1, 1, 64, 128)
    gqa_attn = 2 * 20 * 64 * N * N            # 2 n_h d_h N^2
    gqa_cache = 2 * 5 * 64 * N                # 2 n_k d_h N with 5 KV heads
    assert oracle.attention_cost(gta_1b) / gqa_attn == pytest.approx(0.375, abs=1e-12)
    assert oracle.cache_elems(gta_1b) / gqa_cache == pytest.approx(0.30, abs=1e-12)
    assert oracle.cache_elems(Shape(1, 1, 768, 12, 3, 1, 1, 64, 128)) == 192      # GTA1
    assert oracle.cache_elems(Shape(1, 1, 1280, 20, 10, 1, 2, 64, 128)) == 320    # GTA4
    assert oracle.cache_elems(Shape(1, 1, 1280, 10, 5, 1, 1, 128, 256)) == 384    # d_h = 128 ablation
    assert 192 / 1536 == 0.125 and 320 / 2560 == 0.125 and 192 / 2560 == 0.075    # vs MHA


def test_weight_shapes_agree_with_printed_parameter_counts():
    """The printed parameter totals (in units of 2^20) fix the decoder shapes: W_P is n_h dense
    d_l x d_h blocks and W_G is H x n_h d_h."""
    M = 2.0 ** 20
    layers = 24
    # GTA1 - GQA at 160M: GQA has K,V = 2*3*64 columns; GTA1 has Q 3*64, K 64, C 128, W_P, W_G
    H, nh, dh, dl = 768, 12, 64, 128
    gqa = H * nh * dh + 2 * H * 3 * dh
    gta1 = H * 3 * dh + H * dh + H * dl + nh * dl * dh + H * nh * dh
    assert layers * (gta1 - gqa) / M == pytest.approx(160.75 - 158.50, abs=0.006)
    gta2 = gta1 + H * 3 * dh                                   # six query groups instead of three
    assert layers * (gta2 - gta1) / M == pytest.approx(164.13 - 160.75, abs=0.006)
    H, nh = 1280, 20
    gta3 = H * 5 * dh + H * dh + H * dl + nh * dl * dh + H * nh * dh
    gta4 = H * 10 * dh + H * dh + H * 2 * dl + nh * dl * dh + H * nh * dh
    assert layers * (gta4 - gta3) / M == pytest.approx(500.11 - 486.98, abs=0.006)


# ---------------------------------------------------------------- P12: independence
def test_batch_permutation_permutes_outputs(oracle):
    s = Shape(3, 6, 8, 4, 2, 1, 1, 4, 8, 1)
    t = _inputs(s)
    out = oracle.prefill(s, **t)
    perm = [2, 0, 1]
    t2 = {k: (v[perm].copy() if k in ("q", "k", "c", "x") else v) for k, v in t.items()}
    assert np.array_equal(oracle.prefill(s, **t2), out[perm])


# ---------------------------------------------------------------- storage types, append
def test_bf16_and_f32_storage_are_widened_exactly(oracle):
    import torch
    s = Shape(1, 9, 8, 4, 2, 2, 1, 4, 8, 1)
    t = {k: torch.from_numpy(v).to(torch.bfloat16) for k, v in _inputs(s).items()}
    out_bf = oracle.prefill(s, **t)
    out_f32 = oracle.prefill(s, **{k: v.float() for k, v in t.items()})
    out_f64 = oracle.prefill(s, **{k: v.double().numpy() for k, v in t.items()})
    assert np.array_equal(out_bf, out_f64) and np.array_equal(out_f32, out_f64)


def test_cache_append_is_a_byte_copy_with_overflow_skip(oracle):
    B, cap = 3, 6
    s = Shape(B, 0, 4, 2, 2, 2, 1, 4, 8, 1)
    kc = RNG.integers(0, 2 ** 16, (B, 2, cap, 4)).astype(np.uint16)
    cc = RNG.integers(0, 2 ** 16, (B, 1, cap, 8)).astype(np.uint16)
    kn = RNG.integers(0, 2 ** 16, (B, 2, 2, 4)).astype(np.uint16)
    cn = RNG.integers(0, 2 ** 16, (B, 1, 2, 8)).astype(np.uint16)
    lens = np.array([0, 4, 5], dtype=np.int32)          # the last one would overflow (5 + 2 > 6)
    k2, c2, l2, ov = oracle.cache_append(s, kc, cc, cap, kn, cn, 2, lens)
    assert ov == 1 and l2.tolist() == [2, 6, 5]
    want_k, want_c = kc.copy(), cc.copy()
    want_k[0, :, 0:2] = kn[0]; want_c[0, :, 0:2] = cn[0]
    want_k[1, :, 4:6] = kn[1]; want_c[1, :, 4:6] = cn[1]
    assert np.array_equal(k2, want_k) and np.array_equal(c2, want_c)
    assert np.array_equal(kc[2], k2[2]) and np.array_equal(cc[2], c2[2])


# --------------------------------------------------------------------------- paged cache
def _paged_problem(page_size, lens, seed=5):
    """A decode problem over contiguous caches plus the same caches scattered into a shuffled pool."""
    rng = np.random.default_rng(seed)
    B = len(lens)
    s = Shape(B, 0, 12, 4, 4, 2, 1, 8, 16, 1)
    max_pages = -(-max(max(lens), 1) // page_size) + 1
    cap = max_pages * page_size
    kc = rng.standard_normal((B, s.n_k, cap, s.d_h)); cc = rng.standard_normal((B, s.n_c, cap, s.d_l))
    n_pages = B * max_pages + 2
    table = rng.permutation(n_pages)[: B * max_pages].reshape(B, max_pages)
    kp = rng.standard_normal((n_pages, s.n_k, page_size, s.d_h)); cp = rng.standard_normal((n_pages, s.n_c, page_size, s.d_l))
    # scatter by slices (the oracle's view goes token by token: two different index computations)
    for b in range(B):
        for j in range(max_pages):
            kp[table[b, j]] = kc[b, :, j * page_size:(j + 1) * page_size]
            cp[table[b, j]] = cc[b, :, j * page_size:(j + 1) * page_size]
    rest = dict(q=rng.standard_normal((B, s.n_q, s.d_h)), x_t=rng.standard_normal((B, s.d_model)),
                w_p=rng.standard_normal((s.n_heads, s.d_l, s.d_h)) * 0.25,
                w_g=rng.standard_normal((s.d_model, s.n_heads * s.d_h)) * 0.3)
    return s, kc, cc, kp, cp, table, cap, rest


@pytest.mark.parametrize("page_size", [1, 4, 7])
def test_paged_decode_does_not_depend_on_where_the_pages_lie(oracle, page_size):
    lens = [0, 1, page_size, page_size + 1, 3 * page_size - 1, 19]
    s, kc, cc, kp, cp, table, cap, r = _paged_problem(page_size, lens)
    assert np.array_equal(oracle.paged_view(kp, table, page_size), kc)
    assert np.array_equal(oracle.paged_view(cp, table, page_size), cc)
    want = oracle.decode(s, r["q"], kc, cc, lens, cap, r["x_t"], r["w_p"], r["w_g"])
    got = oracle.decode_paged(s, r["q"], kp, cp, table, page_size, lens, r["x_t"], r["w_p"], r["w_g"])
    assert np.array_equal(got, want)
    # pages no live token maps to may be unassigned
    holes = table.copy()
    for b, n in enumerate(lens):
        holes[b, -(-n // page_size):] = -1
    got = oracle.decode_paged(s, r["q"], kp, cp, holes, page_size, lens, r["x_t"], r["w_p"], r["w_g"])
    assert np.array_equal(got, want)


@pytest.mark.parametrize("n_new", [1, 5])
def test_paged_append_equals_contiguous_append_seen_through_the_block_table(oracle, n_new):
    page_size, lens = 4, [0, 3, 4, 10, 17]
    s, kc, cc, kp, cp, table, cap, _ = _paged_problem(page_size, lens, seed=9)
    lens = np.array(lens, dtype=np.int32)
    lens[-1] = cap - n_new + 1                       # the last sequence would overflow
    rng = np.random.default_rng(3)
    kn = rng.standard_normal((len(lens), s.n_k, n_new, s.d_h)); cn = rng.standard_normal((len(lens), s.n_c, n_new, s.d_l))
    wk, wc, wl, wov = oracle.cache_append(s, kc, cc, cap, kn, cn, n_new, lens)
    gk, gc, gl, gov = oracle.cache_append_paged(kp, cp, table, page_size, kn, cn, lens)
    assert gov == wov == 1 and gl.tolist() == wl.tolist()
    assert np.array_equal(oracle.paged_view(gk, table, page_size), wk)
    assert np.array_equal(oracle.paged_view(gc, table, page_size), wc)
    # pages outside the block table are untouched
    unused = sorted(set(range(kp.shape[0])) - set(table.ravel().tolist()))
    assert np.array_equal(gk[unused], kp[unused]) and np.array_equal(gc[unused], cp[unused])


# --------------------------------------------------------------------------- whole layer (App. B.1.1)
def test_rope_is_a_rotation_that_depends_on_relative_position_only(oracle):
    d, n = 8, 6
    q = _rand(n, d); k = _rand(n, d)
    pos = np.arange(n)
    rq, rk = oracle.rope(q, pos), oracle.rope(k, pos)
    assert np.allclose(np.linalg.norm(rq, axis=-1), np.linalg.norm(q, axis=-1), rtol=1e-13)
    assert np.array_equal(rq[0], q[0])                                   # position 0: the identity
    # <RoPE(a, m), RoPE(b, n)> is a function of m - n: shift every position by 11
    rq2, rk2 = oracle.rope(q, pos + 11), oracle.rope(k, pos + 11)
    assert np.allclose(rq @ rk.T, rq2 @ rk2.T, rtol=0, atol=1e-12)
    # the complex form of the same definition: (x_{2i} + j x_{2i+1}) e^{j m theta_i}, theta_i = base^(-2i/d)
    z = (q[:, 0::2] + 1j * q[:, 1::2]) * np.exp(1j * pos[:, None] * 10000.0 ** (-np.arange(0, d, 2) / d)[None, :])
    assert np.allclose(rq[:, 0::2], z.real, atol=1e-13) and np.allclose(rq[:, 1::2], z.imag, atol=1e-13)
    # first pair turns by one radian per position; base changes every pair but the first
    e0 = np.zeros((n, d)); e0[:, 0] = 1.0
    r = oracle.rope(e0, pos, base=500.0)
    assert np.allclose(r[:, 0], np.cos(pos)) and np.allclose(r[:, 1], np.sin(pos)) and np.all(r[:, 2:] == 0)
    e2 = np.zeros((n, d)); e2[:, 2] = 1.0
    assert np.allclose(oracle.rope(e2, pos, base=500.0)[:, 3], np.sin(pos * 500.0 ** (-2 / d)))


def test_round_to_storage_is_round_to_nearest_even_bf16(oracle):
    F32, BF16 = 0, 1
    v = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 2.0 ** -7, 1.0 + 3 * 2.0 ** -8, -3.0 - 2.0 ** -7, 1e-3, 0.0])
    got = oracle.round_to_storage(v, BF16)
    # bf16 keeps 8 significant bits: ties go to the even neighbour
    want = np.array([1.0, 1.0, 1.0 + 2.0 ** -7, 1.0 + 2.0 ** -6, -3.0, got[5], 0.0])
    assert np.array_equal(got, want) and abs(got[5] - 1e-3) <= 1e-3 * 2.0 ** -9
    assert np.array_equal(oracle.round_to_storage(v, F32), v.astype(np.float32).astype(np.float64))


def test_layer_reduces_to_rotary_multi_head_attention_times_w_o(oracle):
    """n_q = n_k = n_c = n_h, W_P = identity (d_l = d_h), W_G = 0: u = 0.5 * MHA(RoPE(xW_Q), RoPE(xW_K), xW_C) W_O,
    checked against a textbook attention written here (no storage rounding: storage = float64)."""
    F64 = 2
    B, N, H, nh, dh = 2, 9, 12, 3, 4
    s = Shape(B, N, H, nh, nh, nh, nh, dh, dh, 1)
    x = _rand(B, N, H)
    w_qkc = _rand(H, 3 * nh * dh, scale=H ** -0.5)
    w_o = _rand(nh * dh, H, scale=0.3)
    w_p = np.broadcast_to(np.eye(dh), (nh, dh, dh)).copy()
    w_g = np.zeros((H, nh * dh))
    got = oracle.layer_prefill(s, x, w_qkc, w_p, w_g, w_o, rope_base=100.0, storage=F64)
    pos = np.arange(N)
    theta = 100.0 ** (-np.arange(0, dh, 2) / dh)

    def rot(v):   # [N, dh], written with the 2x2 rotation matrices
        out = np.zeros_like(v)
        for t in range(N):
            for i in range(dh // 2):
                c_, s_ = np.cos(pos[t] * theta[i]), np.sin(pos[t] * theta[i])
                out[t, 2 * i:2 * i + 2] = np.array([[c_, -s_], [s_, c_]]) @ v[t, 2 * i:2 * i + 2]
        return out

    want = np.zeros((B, N, H))
    for b in range(B):
        heads = []
        for h in range(nh):
            q = rot(x[b] @ w_qkc[:, h * dh:(h + 1) * dh])
            k = rot(x[b] @ w_qkc[:, (nh + h) * dh:(nh + h + 1) * dh])
            v = x[b] @ w_qkc[:, (2 * nh + h) * dh:(2 * nh + h + 1) * dh]
            sc = q @ k.T / np.sqrt(dh)
            sc[np.triu_indices(N, 1)] = -np.inf
            heads.append(0.5 * _softmax_np(sc) @ v)
        want[b] = np.concatenate(heads, axis=-1) @ w_o
    assert np.allclose(got["u"], want, rtol=1e-10, atol=1e-12)


def test_layer_is_the_operator_between_its_projections(oracle):
    """General grouping: the layer's u equals W_O applied to the operator oracle run on the layer's own q, k, c
    (which are the rounded RoPE'd projections), and the stored tensors are representable in bf16."""
    BF16 = 1
    s = Shape(2, 7, 16, 4, 2, 1, 1, 4, 8, 1)
    x = oracle.round_to_storage(_rand(s.batch, s.seq, s.d_model), BF16)
    w_qkc = oracle.round_to_storage(_rand(s.d_model, 2 * 4 + 4 + 8, scale=0.25), BF16)
    w_p = _rand(s.n_heads, s.d_l, s.d_h, scale=0.3); w_g = _rand(s.d_model, s.n_heads * s.d_h, scale=0.25)
    w_o = _rand(s.n_heads * s.d_h, s.d_model, scale=0.25)
    r = oracle.layer_prefill(s, x, w_qkc, w_p, w_g, w_o)
    for name in ("q", "k", "c", "o"):
        assert np.array_equal(oracle.round_to_storage(r[name], BF16), r[name])
    o = oracle.prefill(s, r["q"], r["k"], r["c"], x, w_p, w_g)
    assert np.allclose(r["u"], oracle.round_to_storage(o, BF16).reshape(2, 7, -1) @ w_o, rtol=1e-12, atol=1e-14)
    # c carries no position: token t's latent is x_t W_C whatever t is
    assert np.array_equal(r["c"][:, 0], oracle.round_to_storage(x @ w_qkc[:, 12:], BF16))
    # position 0 is not rotated
    assert np.array_equal(r["k"][:, 0, 0], oracle.round_to_storage(x[:, 0] @ w_qkc[:, 8:12], BF16))


def test_layer_widens_bf16_tensors_exactly(oracle):
    """The layer oracle fed bf16 torch tensors (what the GPU tests hand it) gives bit for bit what it gives
    for the same values as float64 arrays and as fp32 tensors; the widening is also checked against values
    written out by hand (2^-7 steps around 1, a subnormal-range number, negative zero)."""
    import torch
    s = Shape(2, 6, 16, 4, 2, 1, 1, 4, 8, 1)
    t = dict(x=_rand(s.batch, s.seq, s.d_model), w_qkc=_rand(s.d_model, 2 * 4 + 4 + 8, scale=0.25),
             w_p=_rand(s.n_heads, s.d_l, s.d_h, scale=0.3), w_g=_rand(s.d_model, s.n_heads * s.d_h, scale=0.25),
             w_o=_rand(s.n_heads * s.d_h, s.d_model, scale=0.25))
    tb = {k: torch.from_numpy(v).to(torch.bfloat16) for k, v in t.items()}
    for storage in (1, 2):      # rounded at the stored tensors, and not rounded at all
        r_bf = oracle.layer_prefill(s, **tb, storage=storage)
        r_f32 = oracle.layer_prefill(s, **{k: v.float() for k, v in tb.items()}, storage=storage)
        r_f64 = oracle.layer_prefill(s, **{k: v.double().numpy() for k, v in tb.items()}, storage=storage)
        for name in ("u", "q", "k", "c", "o"):
            assert np.array_equal(r_bf[name], r_f64[name]) and np.array_equal(r_f32[name], r_f64[name]), name
    bits = torch.from_numpy(np.array([0x3F80, 0x3F81, 0xBF81, 0x0001, 0x8000, 0x4049], dtype=np.uint16)
                            .view(np.int16)).view(torch.bfloat16)
    want = np.array([1.0, 1.0 + 2.0 ** -7, -(1.0 + 2.0 ** -7), 2.0 ** -133, -0.0, 3.140625])
    got = oracle._to_f64(bits)
    assert np.array_equal(got, want) and np.signbit(got[4])


# ---------------------------------------------------------------- comparison operators (App. B.3 GQA, Sec. 3.1 MHA)
def _mha_np(q, k, v, causal=True):
    """Textbook multi-head attention on whole matrices: q, k, v [B, n_h, N, d]."""
    d = q.shape[-1]
    s = np.einsum("bhtd,bhjd->bhtj", q, k) / np.sqrt(d)
    if causal:
        N = q.shape[2]
        s = np.where(np.tril(np.ones((N, N), dtype=bool))[None, None], s, -np.inf)
    return np.einsum("bhtj,bhjd->bhtd", _softmax_np(s), v)


@pytest.mark.parametrize("causal", [True, False])
def test_gqa_is_multi_head_attention_on_repeated_key_value_heads(oracle, causal):
    B, n_h, n_kv, N, d = 2, 6, 2, 11, 8
    q, k, v = _rand(B, n_h, N, d), _rand(B, n_kv, N, d), _rand(B, n_kv, N, d)
    got = oracle.gqa_prefill(q, k, v, causal=causal)
    rep = n_h // n_kv
    assert np.allclose(got, _mha_np(q, np.repeat(k, rep, axis=1), np.repeat(v, rep, axis=1), causal), rtol=1e-12, atol=1e-14)
    # the printed map i mod n_kv is the same operator with the query heads renumbered
    perm = [i for j in range(n_kv) for i in range(n_h) if i % n_kv == j]      # heads of kv head 0 first, ...
    got_mod = oracle.gqa_prefill(q, k, v, causal=causal, head_map="mod")
    assert np.allclose(got_mod[:, perm], oracle.gqa_prefill(q[:, perm], k, v, causal=causal), rtol=1e-12, atol=1e-14)
    # one key / value head per query head: multi-head attention itself, whichever map
    k1, v1 = _rand(B, n_h, N, d), _rand(B, n_h, N, d)
    for hm in ("blocks", "mod"):
        assert np.allclose(oracle.gqa_prefill(q, k1, v1, causal=causal, head_map=hm), _mha_np(q, k1, v1, causal),
                           rtol=1e-12, atol=1e-14)


def test_gqa_agrees_with_the_gta_oracle_where_the_two_operators_coincide(oracle):
    """GTA with one map per head, the latent holding the value heads side by side, selector decoders and a
    zero gate is 0.5 x GQA (sigmoid(0) = 1/2): the C oracle of the operator against the numpy comparison oracle."""
    B, n_h, n_kv, N, d = 2, 4, 2, 9, 4
    q, k, v = _rand(B, n_h, N, d), _rand(B, n_kv, N, d), _rand(B, n_kv, N, d)
    s = Shape(B, N, 8, n_h, n_h, n_kv, n_kv, d, d, 1)
    w_p = np.broadcast_to(np.eye(d), (n_h, d, d)).copy()
    got = oracle.prefill(s, q, k, v, _rand(B, N, 8), w_p, np.zeros((8, n_h * d)))       # [B, N, n_h, d]
    want = oracle.gqa_prefill(q, k, v)                                                  # [B, n_h, N, d]
    assert np.allclose(got.transpose(0, 2, 1, 3), 0.5 * want, rtol=1e-12, atol=1e-14)


def test_gqa_decode_is_the_last_prefill_row_and_skips_empty_sequences(oracle):
    B, n_h, n_kv, d, cap = 3, 4, 2, 8, 12
    lens = [7, 0, 12]
    kc, vc = _rand(B, n_kv, cap, d), _rand(B, n_kv, cap, d)
    q = _rand(B, n_h, d)
    got = oracle.gqa_decode(q, kc, vc, lens)
    assert not got[1].any()
    for b in (0, 2):
        n = lens[b]
        qq = np.zeros((1, n_h, n, d)); qq[0, :, n - 1] = q[b]
        full = oracle.gqa_prefill(qq, kc[b:b + 1, :, :n], vc[b:b + 1, :, :n])
        assert np.allclose(got[b], full[0, :, n - 1], rtol=1e-12, atol=1e-14)
    # rows of the cache behind the live length do not matter
    kc2, vc2 = kc.copy(), vc.copy()
    kc2[0, :, 7:] = np.nan; vc2[0, :, 7:] = np.nan
    assert np.array_equal(oracle.gqa_decode(q, kc2, vc2, lens)[0], got[0])


def test_gqa_cost_closed_forms_against_the_printed_ratios(oracle):
    """Table 3 rows of GQA and GTA at the 1B hyper-parameters: GTA-1B has 37.5 % of GQA-1B's attention cost and
    30 % of its cache (Sec. 4.3); GQA-1B caches 640 elements per token and layer, MHA 2560."""
    N = 2048
    gta_1b = Shape(1, N, 1280, 20, 5, 1, 1, 64, 128)
    assert oracle.attention_cost(gta_1b) / oracle.gqa_attention_cost(20, 64, N) == pytest.approx(0.375, abs=1e-12)
    assert oracle.cache_elems(gta_1b) / oracle.gqa_cache_elems(5, 64, N) == pytest.approx(0.30, abs=1e-12)
    assert oracle.gqa_cache_elems(5, 64, 1) == 640 and oracle.gqa_cache_elems(20, 64, 1) == 2560


# ---------------------------------------------------------------- 8-bit caches (e4m3 codes + one scale per row)
def test_e4m3_rounding_against_the_format_and_a_library_cast(oracle):
    """Values written out from the format's definition, ties to even, saturation at 448, and every fp32 value of a
    dense sweep against torch's own float8_e4m3fn cast (an independent implementation of the same format)."""
    import torch
    tab = oracle.e4m3_table()
    assert tab[0x7E] == 448.0 and tab[0x38] == 1.0 and tab[0x01] == 2.0 ** -9 and tab[0x08] == 2.0 ** -6
    assert tab[0xB8] == -1.0 and np.isnan(tab[0x7F]) and tab[0x3C] == 1.5
    r = oracle.round_to_e4m3
    assert r(np.float32(1.0)) == 0x38 and r(np.float32(-448.0)) == 0xFE and r(np.float32(1e9)) == 0x7E
    assert r(np.float32(1.0625)) == 0x38 and r(np.float32(1.1875)) == 0x3A      # ties: 1.0625 -> 1.0, 1.1875 -> 1.25
    assert r(np.float32(2.0 ** -10)) == 0x00 and r(np.float32(3 * 2.0 ** -10)) == 0x02   # ties among the subnormals
    y = np.concatenate([np.linspace(-460, 460, 200001), np.linspace(-0.05, 0.05, 50001), _rand(100000) * 30]).astype(np.float32)
    want = torch.from_numpy(np.clip(y, -448, 448)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = r(y)
    same = (got == want) | ((tab[got] == 0) & (tab[want] == 0))          # +0 / -0 of tiny negatives may differ in sign
    assert same.all()


def test_quantised_rows_are_within_half_a_step_and_all_zero_rows_keep_scale_one(oracle):
    x = _rand(3, 2, 5, 64)
    x[1, 0, 2] = 0.0
    codes, scales = oracle.quantize_rows_e4m3(x.astype(np.float32))
    assert codes.dtype == np.uint8 and scales.shape == (3, 2, 5) and scales[1, 0, 2] == 1.0
    back = oracle.dequantize_e4m3(codes, scales)
    amax = np.abs(x).max(axis=-1, keepdims=True)
    assert np.all(np.abs(back - x) <= np.maximum(np.abs(x) * 2.0 ** -4, amax / 448 * 2.0 ** -10) * 1.0001 + 1e-12)
    big = np.argmax(np.abs(x), axis=-1)                                  # the largest element of a row maps to +-448 exactly
    top = np.take_along_axis(oracle.e4m3_table()[codes], big[..., None], axis=-1)[..., 0]
    nz = amax[..., 0] > 0
    assert np.all(np.abs(top[nz]) == 448.0)


def test_fp8_decode_is_the_operator_on_the_dequantised_caches_and_append_skips_full_sequences(oracle):
    s = Shape(3, 0, 16, 4, 2, 2, 1, 8, 16, 1)
    cap = 9
    k, c = _rand(3, 2, cap, 8), _rand(3, 1, cap, 16)
    kq, ks = oracle.quantize_rows_e4m3(k.astype(np.float32))
    cq, cs = oracle.quantize_rows_e4m3(c.astype(np.float32))
    lens = np.array([4, 9, 0], dtype=np.int32)
    k_new, c_new = _rand(3, 2, 1, 8).astype(np.float32), _rand(3, 1, 1, 16).astype(np.float32)
    kq2, ks2, cq2, cs2, lens2, ov = oracle.cache_append_fp8(kq, ks, cq, cs, k_new, c_new, lens)
    assert ov == 1 and lens2.tolist() == [5, 9, 1]
    assert np.array_equal(kq2[1], kq[1]) and np.array_equal(cs2[1], cs[1])          # the full sequence is untouched
    nk, nks = oracle.quantize_rows_e4m3(k_new)
    assert np.array_equal(kq2[0, :, 4], nk[0, :, 0]) and np.array_equal(ks2[2, :, 0], nks[2, :, 0])
    assert np.array_equal(kq2[0, :, :4], kq[0, :, :4]) and np.array_equal(kq2[0, :, 5:], kq[0, :, 5:])
    t = dict(q=_rand(3, 2, 8), x_t=_rand(3, 16), w_p=_rand(4, 16, 8, scale=0.25), w_g=_rand(16, 32, scale=0.25))
    got = oracle.decode_fp8(s, t["q"], kq2, ks2, cq2, cs2, lens2, t["x_t"], t["w_p"], t["w_g"])
    want = oracle.decode(s, t["q"], oracle.dequantize_e4m3(kq2, ks2), oracle.dequantize_e4m3(cq2, cs2), lens2, cap,
                         t["x_t"], t["w_p"], t["w_g"])
    assert np.array_equal(got, want)
    # garbage (NaN codes and scales) behind the live rows does not matter
    kq3, ks3 = kq2.copy(), ks2.copy()
    kq3[0, :, 5:] = 0x7F; ks3[0, :, 5:] = np.nan
    assert np.array_equal(oracle.decode_fp8(s, t["q"], kq3, ks3, cq2, cs2, lens2, t["x_t"], t["w_p"], t["w_g"])[0], got[0])
