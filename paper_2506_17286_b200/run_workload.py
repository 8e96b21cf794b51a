"""Run one named synthetic workload through the C-ABI library and print per-kernel device times.

    python -m paper_2506_17286_b200.run_workload c3_decode_bf16 [--iters 20] [--warmup 3]
           [--batch B] [--seq N] [--stages MASK] [--append] [--fp8] [--host-cache] [--page-size P] [--kv-len L]

A small, self-contained driver for timing or profiling one call at a time (the benchmark
times the whole step).  Times are CUDA-event times on the launching stream; between
iterations the inputs alternate between two independent sets, so a decode step never finds
its caches in L2.  `--batch` / `--seq` shrink the workload (e.g. for a profiler capture);
`--stages` restricts the call to some of its kernels (see gta_prefill_stages /
gta_decode_stages in include/gta.h).
"""
from __future__ import annotations

import argparse
import json
import statistics

import torch

from . import binding as G
from . import inputs as I


def _median(xs):
    return statistics.median(xs) if xs else 0.0


def run_prefill_chunk(w, iters, warmup, kv_len, page_size=0):
    """The last w.seq positions of a kv_len-token context as one chunk (gta_prefill_chunk; with a page size the
    keys and latents sit in a pool of pages dealt out in random order: gta_prefill_chunk_paged)."""
    dev = torch.device("cuda")
    t = I.prefill_inputs(w, device=dev)
    gen = torch.Generator(device=dev).manual_seed(w.seed)
    k = torch.randn((w.batch, w.n_k, kv_len, w.d_h), generator=gen, device=dev).to(w.torch_dtype())
    c = torch.randn((w.batch, w.n_c, kv_len, w.d_l), generator=gen, device=dev).to(w.torch_dtype())
    shape = G.make_shape(batch=w.batch, seq=w.seq, d_model=w.d_model, n_heads=w.n_heads, n_q=w.n_q, n_k=w.n_k,
                         n_c=w.n_c, d_h=w.d_h, d_l=w.d_l, dtype=w.torch_dtype())
    ws = torch.zeros(G.prefill_workspace_bytes(shape), dtype=torch.uint8, device=dev)
    out = torch.empty((w.batch, w.seq, w.n_heads, w.d_h), dtype=w.torch_dtype(), device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()

    if page_size > 0:
        pg = I.paginate(dict(k_cache=k, c_cache=c), page_size, seed=w.seed)
        k_pool, c_pool, table = pg["k_pool"], pg["c_pool"], pg["block_table"]

    def step():
        if page_size > 0:
            G.gta_prefill_chunk_paged(t["q"], k_pool, c_pool, table, t["x"], t["w_p"], t["w_g"], kv_len, out=out,
                                      workspace=ws, status_word=status)
        else:
            G.gta_prefill_chunk(t["q"], k, c, t["x"], t["w_p"], t["w_g"], kv_len, out=out, workspace=ws,
                                status_word=status)

    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    times = []
    for rep in range(3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(iters):
            step()
        e1.record(stream)
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1) / iters)
    assert int(status.item()) == 0, "device status word raised"
    return {"whole_call": _median(times), "kv_len": kv_len, "page_size": page_size}


def run_layer(w, iters, warmup):
    """The whole attention layer on the workload's shape (gta_layer_prefill, a prompt: pos0 = 0)."""
    dev = torch.device("cuda")
    t = I.layer_inputs(w, device=dev)
    shape = G.make_shape(batch=w.batch, seq=w.seq, d_model=w.d_model, n_heads=w.n_heads, n_q=w.n_q, n_k=w.n_k,
                         n_c=w.n_c, d_h=w.d_h, d_l=w.d_l, dtype=w.torch_dtype())
    ws = torch.zeros(G.layer_prefill_workspace_bytes(shape), dtype=torch.uint8, device=dev)
    k_cache = torch.zeros((w.batch, w.n_k, w.seq, w.d_h), dtype=w.torch_dtype(), device=dev)
    c_cache = torch.zeros((w.batch, w.n_c, w.seq, w.d_l), dtype=w.torch_dtype(), device=dev)
    u = torch.empty((w.batch, w.seq, w.d_model), dtype=w.torch_dtype(), device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()

    def step():
        G.gta_layer_prefill(t["x"], t["w_qkc"], t["w_p"], t["w_g"], t["w_o"], k_cache, c_cache, n_q=w.n_q, out=u,
                            workspace=ws, status_word=status)

    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    times = []
    for rep in range(3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(iters):
            step()
        e1.record(stream)
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1) / iters)
    assert int(status.item()) == 0, "device status word raised"
    M = w.batch * w.seq
    qkc = (w.n_q + w.n_k) * w.d_h + w.n_c * w.d_l
    D = w.n_heads * w.d_h
    # linear maps in full, attention over the causal half (as the operator's figures count it)
    flops = dict(project=2.0 * M * w.d_model * qkc, w_o=2.0 * M * D * w.d_model,
                 attention=w.batch * w.n_q * (w.d_h + w.d_l) * float(w.seq) * (w.seq + 1),
                 decoder=2.0 * M * w.n_heads * w.d_l * w.d_h, gate=2.0 * M * w.d_model * D)
    ms = _median(times)
    return {"whole_call": ms, "launches": G.last_launch_count(), "gflop": {k: v / 1e9 for k, v in flops.items()},
            "tflops": sum(flops.values()) / (ms * 1e-3) / 1e12}


def run_prefill(w, iters, warmup, stages):
    dev = torch.device("cuda")
    t = I.prefill_inputs(w, device=dev)
    shape = G.make_shape(batch=w.batch, seq=w.seq, d_model=w.d_model, n_heads=w.n_heads, n_q=w.n_q, n_k=w.n_k,
                         n_c=w.n_c, d_h=w.d_h, d_l=w.d_l, dtype=w.torch_dtype())
    ws = torch.zeros(G.prefill_workspace_bytes(shape), dtype=torch.uint8, device=dev)
    out = torch.empty((w.batch, w.seq, w.n_heads, w.d_h), dtype=w.torch_dtype(), device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()
    masks = [m for m in (1, 2) if stages & m]
    if len(masks) > 1:
        masks.append(3)
    times = {m: [] for m in masks}

    def step(m):
        G.gta_prefill(t["q"], t["k"], t["c"], t["x"], t["w_p"], t["w_g"], out=out, workspace=ws,
                      status_word=status, stages=m)

    # each stage mask: `iters` launches back to back between two events, three repeats, median
    for m in masks:
        for _ in range(warmup):
            step(m)
        torch.cuda.synchronize()
        for rep in range(3):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(iters):
                step(m)
            e1.record(stream)
            torch.cuda.synchronize()
            times[m].append(e0.elapsed_time(e1) / iters)
    assert int(status.item()) == 0, "device status word raised"
    names = {1: "attention", 2: "decoder_gate", 3: "whole_call"}
    return {names[m]: _median(v) for m, v in times.items()}


def run_decode_paged(w, iters, warmup, append, page_size):
    """The decode workload with its caches in a paged pool (gta_decode_paged, whole call only)."""
    dev = torch.device("cuda")
    sets = []
    for s in range(2):
        td = I.paginate(I.decode_inputs(I.scaled(w, seed=w.seed + s), device=dev), page_size, seed=w.seed + s)
        del td["k_cache"], td["c_cache"]
        td["lens0"] = td["seq_lens"].clone()
        sets.append(td)
    td = sets[0]
    shape = G.decode_shape(td["q"], td["k_pool"], td["c_pool"], td["x_t"], td["w_p"])
    ws = torch.zeros(G.decode_paged_workspace_bytes(shape, page_size, td["max_pages"]), dtype=torch.uint8, device=dev)
    out = torch.empty((w.batch, w.n_heads, w.d_h), dtype=w.torch_dtype(), device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()

    def step(it):
        td = sets[it % 2]
        if append:
            td["seq_lens"].copy_(td["lens0"] - 1)
            G.gta_cache_append_paged(td["k_pool"], td["c_pool"], td["block_table"], td["k_new"], td["c_new"],
                                     td["seq_lens"], status_word=status)
        G.gta_decode_paged(td["q"], td["k_pool"], td["c_pool"], td["block_table"], td["seq_lens"], td["x_t"],
                           td["w_p"], td["w_g"], out=out, workspace=ws, status_word=status)

    for it in range(warmup):
        step(it)
    torch.cuda.synchronize()
    times = []
    for rep in range(3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for it in range(iters):
            step(it)
        e1.record(stream)
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1) / iters)
    assert int(status.item()) == 0, "device status word raised"
    lens = sets[0]["lens0"].cpu().tolist()
    return {"whole_call": _median(times), "append_included": bool(append), "page_size": page_size,
            "launches": G.last_launch_count(),
            "cache_bytes": float(sum(lens)) * (w.n_k * w.d_h + w.n_c * w.d_l) * 2}


def run_layer_decode(w, iters, warmup):
    """One decode step of the whole attention layer per iteration (gta_layer_decode), two cache sets alternating;
    the lengths are put back before every step (a 4-byte-per-sequence copy inside the timed loop)."""
    dev = torch.device("cuda")
    wl = I.scaled(w, kind="prefill", seq=1)
    sets = []
    for s in range(2):
        td = I.decode_inputs(I.scaled(w, seed=w.seed + s), device=dev)
        td["lens0"] = td["seq_lens"].clone() - 1          # the step appends the new token itself
        td.update(I.layer_inputs(I.scaled(wl, seed=w.seed + s), device=dev))
        td["x_t"] = td["x"][:, 0].contiguous()
        sets.append(td)
    td = sets[0]
    shape = G.decode_shape(td["q"], td["k_cache"], td["c_cache"], td["x_t"], td["w_p"])
    ws = torch.zeros(G.layer_decode_workspace_bytes(shape, td["s_cap"]), dtype=torch.uint8, device=dev)
    u = torch.empty((w.batch, w.d_model), dtype=w.torch_dtype(), device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()

    def step(it):
        td = sets[it % 2]
        td["seq_lens"].copy_(td["lens0"])
        G.gta_layer_decode(td["x_t"], td["w_qkc"], td["w_p"], td["w_g"], td["w_o"], td["k_cache"], td["c_cache"],
                           td["seq_lens"], n_q=w.n_q, out=u, workspace=ws, status_word=status)

    for it in range(warmup):
        step(it)
    torch.cuda.synchronize()
    times = []
    for rep in range(3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for it in range(iters):
            step(it)
        e1.record(stream)
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1) / iters)
    assert int(status.item()) == 0, "device status word raised"
    lens = [n + 1 for n in sets[0]["lens0"].cpu().tolist()]
    qkc = (w.n_q + w.n_k) * w.d_h + w.n_c * w.d_l
    D = w.n_heads * w.d_h
    cache_bytes = float(sum(lens)) * (w.n_k * w.d_h + w.n_c * w.d_l) * 2
    weight_bytes = 2.0 * (w.d_model * qkc + w.n_heads * w.d_l * w.d_h + w.d_model * D + D * w.d_model)
    ms = _median(times)
    return {"whole_call": ms, "launches": G.last_launch_count(), "cache_bytes": cache_bytes,
            "weight_bytes": weight_bytes, "gbs": (cache_bytes + weight_bytes) / (ms * 1e-3) / 1e9}


def run_decode(w, iters, warmup, stages, append):
    dev = torch.device("cuda")
    sets = []
    for s in range(2):
        td = I.decode_inputs(I.scaled(w, seed=w.seed + s), device=dev)
        td["lens0"] = td["seq_lens"].clone()
        sets.append(td)
    shape = G.decode_shape(sets[0]["q"], sets[0]["k_cache"], sets[0]["c_cache"], sets[0]["x_t"], sets[0]["w_p"])
    ws = torch.zeros(G.decode_workspace_bytes(shape, sets[0]["s_cap"]), dtype=torch.uint8, device=dev)
    out = torch.empty((w.batch, w.n_heads, w.d_h), dtype=w.torch_dtype(), device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()
    masks = [m for m in (1, 2, 4) if stages & m]
    # a stage with no kernel on this path (e.g. the gate stage of the bf16 kernels) is not timed
    td = sets[0]
    live = []
    for m in masks:
        G.gta_decode(td["q"], td["k_cache"], td["c_cache"], td["seq_lens"], td["x_t"], td["w_p"], td["w_g"],
                     out=out, workspace=ws, status_word=status, stages=m)
        if G.last_launch_count() > 0:
            live.append(m)
    masks = live + ([sum(live)] if len(live) > 1 else [])
    times = {m: [] for m in masks}
    t_append = []

    def step(it, m):
        td = sets[it % 2]
        if append:
            td["seq_lens"].copy_(td["lens0"] - 1)
            G.gta_cache_append(td["k_cache"], td["c_cache"], td["k_new"], td["c_new"], td["seq_lens"],
                               status_word=status)
        G.gta_decode(td["q"], td["k_cache"], td["c_cache"], td["seq_lens"], td["x_t"], td["w_p"], td["w_g"],
                     out=out, workspace=ws, status_word=status, stages=m)

    # each stage mask: `iters` launches back to back between two events (launch gaps included,
    # host latency hidden behind the queue), repeated three times; the median repeat counts
    for m in masks:
        for it in range(warmup):
            step(it, m)
        torch.cuda.synchronize()
        for rep in range(3):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for it in range(iters):
                step(it, m)
            e1.record(stream)
            torch.cuda.synchronize()
            times[m].append(e0.elapsed_time(e1) / iters)
    assert int(status.item()) == 0, "device status word raised"
    names = {1: "gate", 2: "cache_stream", 4: "merge_decoder"}
    res = {names.get(m, "whole_call"): _median(v) for m, v in times.items()}
    res["append_included"] = bool(append)
    lens = sets[0]["lens0"].cpu().tolist()
    res["cache_bytes"] = float(sum(lens)) * (w.n_k * w.d_h + w.n_c * w.d_l) * 2
    return res


def run_decode_hostcache(w, iters, warmup):
    """gta_decode_hostcache: the caches stay in page-locked host memory and are read in place at every step."""
    dev = torch.device("cuda")
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    sets = []
    for s in range(2):
        td = I.decode_inputs(I.scaled(w, seed=w.seed + s), device=dev)
        for name in ("k_cache", "c_cache"):
            h = torch.empty(td[name].shape, dtype=td[name].dtype, pin_memory=True)
            h.copy_(td[name])
            td[name] = h
        sets.append(td)
    torch.cuda.synchronize()
    td = sets[0]
    shape = G.decode_shape(td["q"], td["k_cache"], td["c_cache"], td["x_t"], td["w_p"])
    ws = torch.zeros(G.decode_hostcache_workspace_bytes(shape, td["s_cap"]), dtype=torch.uint8, device=dev)
    out = torch.empty((w.batch, w.n_heads, w.d_h), dtype=w.torch_dtype(), device=dev)
    stream = torch.cuda.current_stream()

    def step(it):
        c = sets[it % 2]
        G.gta_decode_hostcache(c["q"], c["k_cache"], c["c_cache"], c["seq_lens"], c["x_t"], c["w_p"], c["w_g"], out=out,
                               workspace=ws, status_word=status)
    for it in range(warmup):
        step(it)
    torch.cuda.synchronize()
    times = []
    for rep in range(3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for it in range(iters):
            step(it)
        e1.record(stream)
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1) / iters)
    assert int(status.item()) == 0, "device status word raised"
    cache_bytes = float(td["seq_lens"].sum()) * (w.n_k * w.d_h + w.n_c * w.d_l) * td["k_cache"].element_size()
    ms = _median(times)
    return {"whole_call": ms, "launches": G.last_launch_count(), "cache_bytes": cache_bytes,
            "host_link_gbs": cache_bytes / (ms * 1e-3) / 1e9}


def run_decode_fp8(w, iters, warmup):
    """gta_decode_fp8 over caches quantised (outside the timed loop) by the library's own gta_cache_append_fp8."""
    dev = torch.device("cuda")
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    sets = []
    for s in range(2):
        td = I.decode_inputs(I.scaled(w, seed=w.seed + s), device=dev, s_cap=(w.seq or w.ctx_max) + 64)
        cap, nb = td["s_cap"], w.batch
        kq = torch.zeros((nb, w.n_k, cap, w.d_h), dtype=torch.uint8, device=dev)
        cq = torch.zeros((nb, w.n_c, cap, w.d_l), dtype=torch.uint8, device=dev)
        ks = torch.ones((nb, w.n_k, cap), dtype=torch.float32, device=dev)
        cs = torch.ones((nb, w.n_c, cap), dtype=torch.float32, device=dev)
        for b in range(nb):                      # sequence by sequence: the lengths may be ragged
            n = int(td["seq_lens"][b])
            if n == 0:
                continue
            zero = torch.zeros(1, dtype=torch.int32, device=dev)
            G.gta_cache_append_fp8(kq[b:b + 1], cq[b:b + 1], ks[b:b + 1], cs[b:b + 1],
                                   td["k_cache"][b:b + 1, :, :n].contiguous(), td["c_cache"][b:b + 1, :, :n].contiguous(),
                                   zero, status_word=status)
        sets.append(dict(kq=kq, cq=cq, ks=ks, cs=cs, lens=td["seq_lens"], q=td["q"], x_t=td["x_t"], w_p=td["w_p"],
                         w_g=td["w_g"], cap=cap))
        del td
    shape = G.make_shape(batch=w.batch, seq=0, d_model=w.d_model, n_heads=w.n_heads, n_q=w.n_q, n_k=w.n_k, n_c=w.n_c,
                         d_h=w.d_h, d_l=w.d_l, dtype=w.torch_dtype())
    cap = sets[0]["cap"]
    ws = torch.zeros(G.decode_fp8_workspace_bytes(shape, cap), dtype=torch.uint8, device=dev)
    out = torch.empty((w.batch, w.n_heads, w.d_h), dtype=w.torch_dtype(), device=dev)
    stream = torch.cuda.current_stream()

    def step(it):
        c = sets[it % 2]
        G.gta_decode_fp8(c["q"], c["kq"], c["cq"], c["ks"], c["cs"], c["lens"], c["x_t"], c["w_p"], c["w_g"], out=out,
                         workspace=ws, status_word=status)
    for it in range(warmup):
        step(it)
    torch.cuda.synchronize()
    times = []
    for rep in range(3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for it in range(iters):
            step(it)
        e1.record(stream)
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1) / iters)
    assert int(status.item()) == 0, "device status word raised"
    live = float(sets[0]["lens"].sum())
    cache_bytes = live * ((w.n_k * w.d_h + w.n_c * w.d_l) + 4 * (w.n_k + w.n_c))
    ms = _median(times)
    return {"whole_call": ms, "path": G.decode_fp8_path(shape, cap), "launches": G.last_launch_count(),
            "cache_bytes": cache_bytes, "cache_gbs": cache_bytes / (ms * 1e-3) / 1e9}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("workload", choices=sorted(I.CONFIGS))
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--seq", type=int, default=0)
    ap.add_argument("--stages", type=int, default=7)
    ap.add_argument("--append", action="store_true", help="decode: run gta_cache_append before every step")
    ap.add_argument("--kv-len", type=int, default=0,
                    help="prefill: treat the workload's tokens as the last chunk of a context of this length")
    ap.add_argument("--layer", action="store_true",
                    help="the whole attention layer (projections + RoPE + cache write, operator, W_O): "
                         "gta_layer_prefill on a prefill workload, gta_layer_decode on a decode workload")
    ap.add_argument("--host-cache", action="store_true",
                    help="decode: caches in page-locked host memory, read in place (gta_decode_hostcache)")
    ap.add_argument("--fp8", action="store_true",
                    help="decode: caches as e4m3 codes with one scale per cached row (gta_decode_fp8)")
    ap.add_argument("--page-size", type=int, default=0,
                    help="keep the caches in a paged pool with pages of this many tokens (decode, or a prefill chunk)")
    args = ap.parse_args()
    w = I.CONFIGS[args.workload]
    if args.batch:
        w = I.scaled(w, batch=args.batch)
    if args.seq:
        w = I.scaled(w, seq=args.seq) if w.kind == "prefill" or w.seq > 0 else I.scaled(w, ctx_max=args.seq)
    G.lib()
    torch.cuda.set_device(0)
    if w.kind == "prefill" and args.layer:
        res = run_layer(w, args.iters, args.warmup)
    elif w.kind == "prefill" and (args.kv_len > w.seq or args.page_size > 0):
        res = run_prefill_chunk(w, args.iters, args.warmup, max(args.kv_len, w.seq), args.page_size)
    elif w.kind == "prefill":
        res = run_prefill(w, args.iters, args.warmup, args.stages & 3)
    elif args.layer:
        res = run_layer_decode(w, args.iters, args.warmup)
    elif args.fp8:
        res = run_decode_fp8(w, args.iters, args.warmup)
    elif args.host_cache:
        res = run_decode_hostcache(w, args.iters, args.warmup)
    elif args.page_size > 0:
        res = run_decode_paged(w, args.iters, args.warmup, args.append, args.page_size)
    else:
        res = run_decode(w, args.iters, args.warmup, args.stages, args.append)
    print(json.dumps({"workload": w.name, "batch": w.batch, "seq": w.seq, "median_ms": res}))


if __name__ == "__main__":
    main()
