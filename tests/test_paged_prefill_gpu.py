"""GPU parity of prefill over a paged cache: gta_prefill_chunk_paged against the oracle's prefill over the rows
that the oracle's own reading of the block table (paged_view) finds in the pools, and gta_layer_prefill_paged
against the layer run over contiguous caches and against the layer oracle."""
import numpy as np
import pytest
import torch

from paper_2506_17286_b200 import inputs as I
from tests.parity_utils import Guarded, assert_close, cpu, oracle_shape

pytestmark = pytest.mark.gpu

GARBAGE_ENTRY = -12345      # block-table entries of positions that are not attended: never read


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2506_17286_b200 import build, binding
    build.build()
    binding.lib()
    return binding


def _pools(k, c, kv_len, page_size, seed, spare=3, extra_entries=2):
    """Pools and block table that hold rows 0 .. kv_len-1 of k [B,n_k,*,d_h] and c [B,n_c,*,d_l]: the pages are
    dealt out by a seeded permutation, every row no attended position maps to holds NaN (what uninitialised
    memory may hold), and the block-table entries behind the last page in use are garbage.  Data movement only."""
    nb, n_k, _, d_h = k.shape
    n_c, d_l = c.shape[1], c.shape[3]
    used = -(-kv_len // page_size)
    max_pages, n_pages = used + extra_entries, nb * used + spare
    gen = torch.Generator("cpu").manual_seed(seed)
    table = torch.full((nb, max_pages), GARBAGE_ENTRY, dtype=torch.int32)
    table[:, :used] = torch.randperm(n_pages, generator=gen)[: nb * used].reshape(nb, used).to(torch.int32)
    k_pool = torch.full((n_pages, n_k, page_size, d_h), float("nan"), device=k.device, dtype=k.dtype)
    c_pool = torch.full((n_pages, n_c, page_size, d_l), float("nan"), device=c.device, dtype=c.dtype)
    for b in range(nb):
        for j in range(used):
            lo, hi = j * page_size, min((j + 1) * page_size, kv_len)
            k_pool[table[b, j], :, : hi - lo] = k[b, :, lo:hi]
            c_pool[table[b, j], :, : hi - lo] = c[b, :, lo:hi]
    return k_pool, c_pool, table


def _oracle_rows(oracle, pool, table, page_size, kv_len):
    """The attended rows as the oracle reads them out of the pool through the block table (bf16 as raw bits);
    none of them is one of the NaN rows that surround the live ones."""
    rows = np.ascontiguousarray(oracle.paged_view(pool.cpu(), table.numpy(), page_size)[:, :, :kv_len])
    if rows.dtype == np.uint16:
        assert not ((rows & 0x7FFF) > 0x7F80).any()
    else:
        assert not np.isnan(rows).any()
    return rows


PAGED_CHUNKS = [
    # name, dtype, B, kv_len, N, page_size, H, n_h, n_q, n_k, n_c, d_h, d_l, causal
    # tensor-core kernels (page size a multiple of 64)
    ("p64_last_page_one_row", "bf16", 2, 705, 300, 64, 256, 8, 4, 4, 1, 128, 512, True),
    ("p128_last_page_one_row", "bf16", 2, 641, 641, 128, 256, 8, 4, 4, 1, 128, 512, True),
    ("p64_tail_in_second_half", "bf16", 1, 64 * 9 + 17, 200, 64, 128, 4, 2, 2, 1, 128, 256, True),
    ("p64_tail_in_first_half", "bf16", 3, 64 * 8 + 63, 77, 64, 128, 4, 2, 2, 1, 128, 256, True),
    ("p128_whole_pages", "bf16", 1, 512, 512, 128, 128, 4, 2, 2, 1, 128, 256, True),
    ("p192_one_query", "bf16", 2, 400, 1, 192, 128, 4, 2, 2, 1, 128, 256, True),
    ("p64_dh64_dl128", "bf16", 2, 1000, 129, 64, 192, 8, 2, 1, 1, 64, 128, True),
    ("p128_non_causal", "bf16", 1, 333, 100, 128, 128, 4, 2, 2, 1, 128, 256, False),
    ("p64_kv_shorter_than_a_page", "bf16", 2, 37, 37, 64, 128, 4, 2, 2, 1, 128, 256, True),
    # plain-ALU kernels: page sizes that are not multiples of 64, shapes outside the tensor-core path, fp32
    ("p16_plain_alu_page", "bf16", 2, 300, 120, 16, 128, 4, 2, 2, 1, 128, 256, True),
    ("p48_plain_alu_shape", "bf16", 2, 300, 77, 48, 128, 6, 6, 3, 1, 32, 64, True),
    ("p8_f32", "f32", 1, 201, 50, 8, 96, 6, 6, 3, 1, 32, 64, True),
]


@pytest.mark.parametrize("case", PAGED_CHUNKS, ids=[c[0] for c in PAGED_CHUNKS])
def test_prefill_chunk_paged(B, oracle, case):
    name, dt, nb, kv_len, N, page_size, H, n_h, n_q, n_k, n_c, d_h, d_l, causal = case
    w = I.Workload(name, "prefill", dt, nb, kv_len, H, n_h, n_q, n_k, n_c, d_h, d_l, seed=654)
    t = I.prefill_inputs(w, device="cuda")
    first = kv_len - N
    k_pool, c_pool, table = _pools(t["k"], t["c"], kv_len, page_size, seed=17)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    q = t["q"][:, :, first:].contiguous()
    x = t["x"][:, first:].contiguous()
    shape = B.make_shape(batch=nb, seq=N, d_model=H, n_heads=n_h, n_q=n_q, n_k=n_k, n_c=n_c, d_h=d_h, d_l=d_l,
                         dtype=w.torch_dtype(), causal=causal)
    ws = Guarded((B.prefill_workspace_bytes(shape),), torch.uint8)
    og = Guarded((nb, N, n_h, d_h), w.torch_dtype())
    out = B.gta_prefill_chunk_paged(q, k_pool, c_pool, table.cuda(), x, t["w_p"], t["w_g"], kv_len, causal=causal,
                                    status_word=status, workspace=ws.t, out=og.t)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ws.check(name + " workspace"); og.check(name + " out")
    # the oracle reads the pools through the same block table (garbage entries clamp to "no page": never attended)
    k_rows = _oracle_rows(oracle, k_pool, table, page_size, kv_len)
    c_rows = _oracle_rows(oracle, c_pool, table, page_size, kv_len)
    tc = cpu(t)
    want = oracle.prefill(oracle_shape(w, causal=int(causal)), tc["q"], k_rows, c_rows, tc["x"], tc["w_p"],
                          tc["w_g"], rows=list(range(first, kv_len)))
    assert_close(out, want, w.torch_dtype(), name)


def test_prefill_chunk_paged_is_bitwise_the_contiguous_chunk_on_the_tensor_core_path(B):
    """Same tiles, same order, same arithmetic: only the addresses of the loads differ."""
    w = I.Workload("paged_vs_flat_prefill", "prefill", "bf16", 2, 64 * 11 + 5, 256, 8, 4, 4, 1, 128, 512, seed=8)
    t = I.prefill_inputs(w, device="cuda")
    kv_len, N = w.seq, 400
    first = kv_len - N
    q, x = t["q"][:, :, first:].contiguous(), t["x"][:, first:].contiguous()
    flat = B.gta_prefill_chunk(q, t["k"], t["c"], x, t["w_p"], t["w_g"], kv_len)
    for page_size in (64, 128, 256):
        k_pool, c_pool, table = _pools(t["k"], t["c"], kv_len, page_size, seed=page_size)
        paged = B.gta_prefill_chunk_paged(q, k_pool, c_pool, table.cuda(), x, t["w_p"], t["w_g"], kv_len)
        torch.cuda.synchronize()
        assert torch.equal(flat, paged), page_size


def test_prefill_chunk_paged_full_size_c2_sampled_rows(B, oracle):
    """The benchmark's prefill shape with its keys and latents in 64-token pages."""
    w = I.CONFIGS["c2_prefill_bf16"]
    t = I.prefill_inputs(w, device="cuda")
    k_pool, c_pool, table = _pools(t["k"], t["c"], w.seq, 64, seed=3)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = B.gta_prefill_chunk_paged(t["q"], k_pool, c_pool, table.cuda(), t["x"], t["w_p"], t["w_g"], w.seq,
                                    status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    rng = np.random.default_rng(5)
    rows = sorted({0, 1, 63, 64, 127, 128, w.seq - 1} | {int(v) for v in rng.integers(0, w.seq, 40)})
    tc = cpu(t)
    want = oracle.prefill(oracle_shape(w), tc["q"], tc["k"], tc["c"], tc["x"], tc["w_p"], tc["w_g"], rows=rows)
    assert_close(out[:, torch.as_tensor(rows, device="cuda")], want, torch.bfloat16, w.name + " paged")


@pytest.mark.parametrize("page_size", [64, 16])
def test_prefill_chunk_paged_bad_page_is_reported_and_nothing_outside_the_pools_is_read(B, page_size):
    """An entry in use outside the pool: the status word says so, the call completes, and the sequences whose
    entries are sound get the result they get without the bad entry."""
    w = I.Workload("bad_page", "prefill", "bf16", 2, 300, 128, 4, 2, 2, 1, 128, 256, seed=31)
    t = I.prefill_inputs(w, device="cuda")
    k_pool, c_pool, table = _pools(t["k"], t["c"], w.seq, page_size, seed=1)
    good = B.gta_prefill_chunk_paged(t["q"], k_pool, c_pool, table.cuda(), t["x"], t["w_p"], t["w_g"], w.seq)
    bad = table.clone()
    bad[1, 1] = k_pool.shape[0] + 7
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = B.gta_prefill_chunk_paged(t["q"], k_pool, c_pool, bad.cuda(), t["x"], t["w_p"], t["w_g"], w.seq,
                                    status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == B.GTA_ERR_BAD_PAGE
    assert torch.equal(out[0], good[0])
    assert torch.isfinite(out.float()).all()


# --------------------------------------------------------------------------- whole layer over pages
def _layer_pools(w, page_size, chunks_total, seed):
    used = -(-chunks_total // page_size)
    max_pages, n_pages = used + 1, w.batch * used + 2
    gen = torch.Generator("cpu").manual_seed(seed)
    table = torch.full((w.batch, max_pages), GARBAGE_ENTRY, dtype=torch.int32)
    table[:, :used] = torch.randperm(n_pages, generator=gen)[: w.batch * used].reshape(w.batch, used).to(torch.int32)
    k_pool = torch.full((n_pages, w.n_k, page_size, w.d_h), float("nan"), device="cuda", dtype=torch.bfloat16)
    c_pool = torch.full((n_pages, w.n_c, page_size, w.d_l), float("nan"), device="cuda", dtype=torch.bfloat16)
    return k_pool, c_pool, table


LAYERS_PAGED = [
    # name, B, N, H, n_h, n_q, n_k, n_c, d_h, d_l, chunks, page_size
    ("two_chunks_p64", 2, 320, 256, 8, 4, 2, 2, 64, 128, [192, 128], 64),
    ("ragged_chunks_last_page_one_row_p128", 1, 257, 256, 4, 2, 2, 1, 128, 256, [5, 251, 1], 128),
    ("c2_shape_small_p64", 1, 384, 512, 8, 4, 4, 1, 128, 512, None, 64),
    ("plain_alu_page_p16", 2, 130, 256, 8, 4, 2, 2, 64, 128, [100, 30], 16),
]


@pytest.mark.parametrize("case", LAYERS_PAGED, ids=[c[0] for c in LAYERS_PAGED])
def test_layer_prefill_paged(B, oracle, case):
    name, nb, N, H, n_h, n_q, n_k, n_c, d_h, d_l, chunks, page_size = case
    chunks = chunks or [N]
    w = I.Workload(name, "prefill", "bf16", nb, N, H, n_h, n_q, n_k, n_c, d_h, d_l, seed=73)
    t = I.layer_inputs(w, device="cuda")
    k_pool, c_pool, table = _layer_pools(w, page_size, N, seed=9)
    k_flat = torch.full((nb, n_k, N + 9, d_h), float("nan"), device="cuda", dtype=torch.bfloat16)
    c_flat = torch.full((nb, n_c, N + 9, d_l), float("nan"), device="cuda", dtype=torch.bfloat16)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    us_p, us_f, pos0 = [], [], 0
    for n in chunks:
        x = t["x"][:, pos0:pos0 + n].contiguous()
        us_p.append(B.gta_layer_prefill_paged(x, t["w_qkc"], t["w_p"], t["w_g"], t["w_o"], k_pool, c_pool,
                                              table.cuda(), pos0=pos0, n_q=n_q, status_word=status))
        us_f.append(B.gta_layer_prefill(x, t["w_qkc"], t["w_p"], t["w_g"], t["w_o"], k_flat, c_flat, pos0=pos0,
                                        n_q=n_q, status_word=status))
        pos0 += n
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    u_p, u_f = torch.cat(us_p, dim=1), torch.cat(us_f, dim=1)
    # the pools, read through the table as the oracle reads them, hold exactly the rows of the contiguous caches;
    # every other row of the pools is untouched
    for pool, flat in ((k_pool, k_flat), (c_pool, c_flat)):
        view = oracle.paged_view(pool.cpu(), table.numpy(), page_size)          # raw bf16 bits
        assert np.array_equal(view[:, :, :N], flat[:, :, :N].contiguous().view(torch.int16).cpu().numpy().view(np.uint16))
        live = torch.zeros(pool.shape[0], page_size, dtype=torch.bool)
        for b in range(nb):
            for pos in range(N):
                live[table[b, pos // page_size], pos % page_size] = True
        dead = ~live.cuda()
        assert torch.isnan(pool.permute(0, 2, 1, 3)[dead]).all()
    if page_size % 64 == 0:
        assert torch.equal(u_p, u_f)           # same kernels, same tiles
    tc = {n_: v.cpu() for n_, v in t.items()}
    want = oracle.layer_prefill(oracle_shape(w), tc["x"], tc["w_qkc"], tc["w_p"], tc["w_g"], tc["w_o"])
    assert_close(u_p, want["u"], torch.bfloat16, name)
