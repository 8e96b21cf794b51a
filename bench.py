#!/usr/bin/env python
"""Benchmark of the GTA operator library on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One *step* is one pass of the whole hot path over one synthetic batch:
  prefill leg : gta_prefill on workload c2 (B=4, N=2048, H=2048, 16 heads / 4 maps, d_h=128, d_l=512, bf16)
  decode leg  : gta_cache_append (one token per sequence) + gta_decode on workload c3
                (B=32, context 4096, same layer shape, bf16), rotating between two cache sets.
The headline `value` is prefill TFLOP/s (causal-useful flops / device time of the prefill legs);
the decode leg is reported under "decode" (tokens/s, HBM GB/s).  Inputs are resident in HBM for
`value`; "e2e" repeats the prefill through the public call with pinned HOST buffers, host->device
and device->host copies inside the timed region.  Prints ONE JSON line on rank 0.

With --gpus N > 1 (launched by torchrun, one rank per GPU) every rank runs an independent replica
of the step (the operator does not shard: no collective is on the path); times are the max over
ranks and `value` is the sum of the work of all ranks over that time.

--impl reference times the fp64 CPU oracle (the stand-in for a reference implementation, which
the paper does not ship) on a bounded sample of the same workload on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# dram__bytes_read.sum + dram__bytes_write.sum per launch on workload c2, from the ncu captures
# summarised under profiles/ (None once a kernel has changed since its counters were taken).
NCU_DRAM_BYTES_PER_LAUNCH = {"prefill_attention": 26.17e6, "prefill_decoder_gate": 127.71e6, "decode_stream": 272.99e6}

METRIC = "gta_prefill_tflops"
UNIT = "TFLOP/s"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# ----------------------------------------------------------------------------- work counters
def prefill_flops(w, rows=None):
    """Causal-useful flops of the operator (masked halves, recompute and padding not counted)."""
    if rows is None:
        pairs = w.seq * (w.seq + 1) // 2
        n_rows = w.seq
    else:
        pairs = sum(r + 1 for r in rows)
        n_rows = len(rows)
    attn = 2.0 * w.batch * w.n_q * pairs * (w.d_h + w.d_l)
    dec = 2.0 * w.batch * n_rows * w.n_heads * w.d_l * w.d_h
    gate = 2.0 * w.batch * n_rows * w.d_model * w.n_heads * w.d_h
    return dict(attention=attn, decoder=dec, gate=gate, total=attn + dec + gate)


def decode_bytes(w, lens, elem=2):
    cache = float(sum(int(l) for l in lens)) * (w.n_k * w.d_h + w.n_c * w.d_l) * elem
    weights = (w.n_heads * w.d_l * w.d_h + w.d_model * w.n_heads * w.d_h) * elem
    vectors = w.batch * (w.n_q * w.d_h + w.d_model + w.n_heads * w.d_h) * elem
    return dict(cache=cache, weights=float(weights), vectors=float(vectors), total=cache + weights + vectors)


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples nvidia-smi clocks / throttle reasons in the background (read-only queries)."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        self.lines, self.proc, self.thread = [], None, None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", gpu_id, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"], samples=0)
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        rows = [(ts, l) for ts, l in self.lines if t0 - 0.05 <= ts <= t1 + 0.15] or self.lines[-3:]
        for _, line in rows:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1])); mx.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


# ----------------------------------------------------------------------------- CPU oracle arm
_ORACLE_INPUTS = {}


def oracle_prefill_sample(w, n_rows, n_threads=0, batch_index=None):
    """Times the fp64 oracle, as it stands, on `n_rows` evenly spaced query rows of workload `w`
    (all heads; all batch entries, or only `batch_index`).  Returns (TFLOP/s of causal-useful
    flops, seconds, threads, description)."""
    from oracle import gta_oracle
    from paper_2506_17286_b200 import inputs as I
    gta_oracle.build()
    if w.name not in _ORACLE_INPUTS:
        _ORACLE_INPUTS[w.name] = I.prefill_inputs(w, device="cpu")
    t = _ORACLE_INPUTS[w.name]
    ws = w
    if batch_index is not None:
        b = batch_index % w.batch
        t = {k: (v[b:b + 1].contiguous() if k in ("q", "k", "c", "x") else v) for k, v in t.items()}
        ws = I.scaled(w, batch=1)
    n_rows = max(1, min(n_rows, w.seq))
    stride = max(1, w.seq // n_rows)
    rows = list(range(stride - 1, w.seq, stride))[:n_rows]
    shape = gta_oracle.Shape(ws.batch, ws.seq, ws.d_model, ws.n_heads, ws.n_q, ws.n_k, ws.n_c, ws.d_h, ws.d_l, 1, 0.0)
    t0 = time.perf_counter()
    gta_oracle.prefill(shape, t["q"], t["k"], t["c"], t["x"], t["w_p"], t["w_g"], rows=rows, n_threads=n_threads)
    dt = time.perf_counter() - t0
    flops = prefill_flops(ws, rows)["total"]
    threads = gta_oracle.num_threads() if n_threads <= 0 else n_threads
    desc = (f"{len(rows)} of {w.seq} query rows (every {stride}th) x {ws.batch} of {w.batch} sequences x "
            f"{w.n_heads} heads of {w.name}; fp64 oracle, time includes widening its inputs")
    return flops / dt / 1e12, dt, threads, desc


def run_reference(args):
    from paper_2506_17286_b200 import inputs as I
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    w = I.CONFIGS["c2_prefill_bf16"]
    # Each step is a bounded sample: one sequence, a few evenly spaced rows, sized so that the whole
    # run stays near 90 s of CPU time (about 0.12 s fixed + 5 ms per row on 8 cores).
    calls = max(1, args.warmup + args.steps)
    n_rows = int(max(1, min(256, (90.0 / calls - 0.12) / 0.005)))
    vals, secs, threads, desc = [], [], 0, ""
    for i in range(args.warmup + args.steps):
        v, dt, threads, desc = oracle_prefill_sample(w, n_rows, batch_index=i)
        if i >= args.warmup:
            vals.append(v); secs.append(dt)
    value = len(vals) / sum(1.0 / v for v in vals) if vals else 0.0     # total flops / total time
    ms = 1e3 * sum(secs) / len(secs) if secs else 0.0
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "sample_per_step": desc},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ----------------------------------------------------------------------------- ranks
def max_over_ranks(value, dist=None, device="cpu"):
    """The largest of `value` over all ranks of the default process group (every rank gets it); the
    value itself without a process group.  Times of a multi-GPU run are reduced with this."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(work_per_rank, world, ms):
    """Aggregate rate of `world` independent replicas that each did `work_per_rank` in `ms`
    milliseconds (the maximum over ranks): replicas only, no collective on the path."""
    return world * work_per_rank / (ms * 1e-3)


# ----------------------------------------------------------------------------- our arm
def run_ours(args):
    import torch
    from paper_2506_17286_b200 import binding as G
    from paper_2506_17286_b200 import inputs as I

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    G.lib()
    peaks = load_peaks()

    wp = I.CONFIGS["c2_prefill_bf16"]
    wd = I.CONFIGS["c3_decode_bf16"]
    # ---- prefill leg buffers
    tp = I.prefill_inputs(wp, device=dev)
    shape_p = G.make_shape(batch=wp.batch, seq=wp.seq, d_model=wp.d_model, n_heads=wp.n_heads, n_q=wp.n_q,
                           n_k=wp.n_k, n_c=wp.n_c, d_h=wp.d_h, d_l=wp.d_l, dtype=G.GTA_BF16)
    ws_p = torch.empty(G.prefill_workspace_bytes(shape_p), dtype=torch.uint8, device=dev)
    out_p = torch.empty((wp.batch, wp.seq, wp.n_heads, wp.d_h), dtype=torch.bfloat16, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    # ---- decode leg buffers: two cache sets, read alternately
    LENS_POOL = max(64, (max(args.steps, 20) + 1) // 2 + 8)   # length vectors per set: one per step of the longest loop
    sets = []
    for s in range(2):
        td = I.decode_inputs(I.scaled(wd, seed=wd.seed + s), device=dev, s_cap=wd.seq + 64)
        td["seq_lens"] -= 1            # the step's append brings the length back to wd.seq
        td["lens0"] = td["seq_lens"].clone()
        # One length vector per step, all set to wd.seq - 1 before a loop starts: the append of a step
        # advances its own vector, so no rewind copy sits between the steps of a timed region.
        td["pool"] = td["lens0"].unsqueeze(0).repeat(LENS_POOL, 1).contiguous()
        sets.append(td)
    shape_d = G.decode_shape(sets[0]["q"], sets[0]["k_cache"], sets[0]["c_cache"], sets[0]["x_t"], sets[0]["w_p"])
    ws_d = torch.empty(G.decode_workspace_bytes(shape_d, wd.seq + 64), dtype=torch.uint8, device=dev)
    out_d = torch.empty((wd.batch, wd.n_heads, wd.d_h), dtype=torch.bfloat16, device=dev)
    stream = torch.cuda.current_stream()
    launches = {"n": 0}

    def prefill_leg(ev_mid=None):
        if ev_mid is None:                # the call a user makes: both kernels, programmatically chained
            G.gta_prefill(tp["q"], tp["k"], tp["c"], tp["x"], tp["w_p"], tp["w_g"], out=out_p, workspace=ws_p,
                          status_word=status)
            launches["n"] += G.last_launch_count()
            return
        # kernel by kernel, with an event in between (the per-kernel loop below)
        G.gta_prefill(tp["q"], tp["k"], tp["c"], tp["x"], tp["w_p"], tp["w_g"], out=out_p, workspace=ws_p,
                      status_word=status, stages=1)
        launches["n"] += G.last_launch_count()
        ev_mid.record(stream)
        G.gta_prefill(tp["q"], tp["k"], tp["c"], tp["x"], tp["w_p"], tp["w_g"], out=out_p, workspace=ws_p,
                      status_word=status, stages=2)
        launches["n"] += G.last_launch_count()

    def reset_lens():
        for td in sets:
            td["pool"].copy_(td["lens0"].unsqueeze(0).expand(LENS_POOL, -1))

    def decode_leg(i, evs=None):
        td = sets[i % 2]
        lens = td["pool"][(i // 2) % LENS_POOL]            # this step's own length vector (wd.seq - 1)
        G.gta_cache_append(td["k_cache"], td["c_cache"], td["k_new"], td["c_new"], lens, status_word=status)
        launches["n"] += G.last_launch_count()
        if evs is not None:
            evs[0].record(stream)
        G.gta_decode(td["q"], td["k_cache"], td["c_cache"], lens, td["x_t"], td["w_p"], td["w_g"],
                     out=out_d, workspace=ws_d, status_word=status)
        launches["n"] += G.last_launch_count()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(args.warmup, 3)):
        prefill_leg(); decode_leg(i)
    barrier()

    K = args.steps
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(K)]
    gpu_id = str(local_rank)
    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        pass
    sampler = ClockSampler(gpu_id)
    time.sleep(0.8)                       # let nvidia-smi deliver its first samples
    for i in range(3):                    # keep the GPU warm after the sleep (untimed)
        prefill_leg(); decode_leg(i)
    reset_lens()
    launches["n"] = 0
    barrier()
    t_wall0 = time.time()
    e_start, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e_start.record(stream)
    for i in range(K):
        ev[i][0].record(stream)
        prefill_leg()
        ev[i][2].record(stream)
        decode_leg(i, (ev[i][3],))
        ev[i][4].record(stream)
    e_end.record(stream)
    barrier()
    t_wall1 = time.time()
    clocks = sampler.stop(t_wall0, t_wall1)
    n_launches = launches["n"]
    assert int(status.item()) == 0, "device status word raised during the benchmark"

    # ---- the same step once more with the prefill call split into its two kernels and an event
    #      between them: the per-kernel durations of the roofline (the event costs the programmatic
    #      overlap of the two kernels, which is why the loop above does not carry it)
    K_k = min(K, 400)
    evk = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K_k)]
    for i in range(3):
        prefill_leg(evk[0][1]); decode_leg(i)
    reset_lens()
    barrier()
    for i in range(K_k):
        evk[i][0].record(stream)
        prefill_leg(evk[i][1])
        evk[i][2].record(stream)
        decode_leg(i)
    barrier()
    assert int(status.item()) == 0, "device status word raised during the benchmark"

    # ---- decode leg alone, back to back (append + decode, alternating cache sets): the figure the
    #      decode roofline is quoted on; launch gaps between calls are inside the timed region
    K_d = max(K, 20)
    for i in range(3):
        decode_leg(i)
    reset_lens()
    barrier()
    d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    d0.record(stream)
    for i in range(K_d):
        decode_leg(i)
    d1.record(stream)
    barrier()
    t_decode_b2b = d0.elapsed_time(d1) / K_d
    assert int(status.item()) == 0, "device status word raised during the benchmark"
    # ---- the gta_decode call alone, back to back (no append; same alternation)
    for td in sets:
        td["seq_lens"].copy_(td["lens0"] + 1)

    def decode_call(i):
        td = sets[i % 2]
        G.gta_decode(td["q"], td["k_cache"], td["c_cache"], td["seq_lens"], td["x_t"], td["w_p"], td["w_g"],
                     out=out_d, workspace=ws_d, status_word=status)

    for i in range(3):
        decode_call(i)
    barrier()
    d2, d3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    d2.record(stream)
    for i in range(K_d):
        decode_call(i)
    d3.record(stream)
    barrier()
    t_decode_call = d2.elapsed_time(d3) / K_d
    assert int(status.item()) == 0, "device status word raised during the benchmark"
    # ---- the same call over a paged cache (pages of 64 tokens dealt out at random), back to back
    page_size = 64
    psets = [I.paginate(td, page_size, seed=wd.seed + i) for i, td in enumerate(sets)]
    ws_pg = torch.zeros(G.decode_paged_workspace_bytes(shape_d, page_size, psets[0]["max_pages"]), dtype=torch.uint8,
                        device=dev)

    def decode_paged_call(i):
        td = psets[i % 2]
        G.gta_decode_paged(td["q"], td["k_pool"], td["c_pool"], td["block_table"], td["seq_lens"], td["x_t"],
                           td["w_p"], td["w_g"], out=out_d, workspace=ws_pg, status_word=status)

    for i in range(3):
        decode_paged_call(i)
    barrier()
    d4, d5 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    d4.record(stream)
    for i in range(K_d):
        decode_paged_call(i)
    d5.record(stream)
    barrier()
    t_decode_paged = d4.elapsed_time(d5) / K_d
    assert int(status.item()) == 0, "device status word raised during the benchmark"
    del psets, ws_pg
    # ---- the whole attention layer on the prefill workload's shape (projections + RoPE + cache write, the
    #      operator, the output projection), back to back: context for the operator's figure, not part of `value`
    tl = I.layer_inputs(wp, device=dev)
    ws_l = torch.zeros(G.layer_prefill_workspace_bytes(shape_p), dtype=torch.uint8, device=dev)
    kc_l = torch.zeros((wp.batch, wp.n_k, wp.seq, wp.d_h), dtype=torch.bfloat16, device=dev)
    cc_l = torch.zeros((wp.batch, wp.n_c, wp.seq, wp.d_l), dtype=torch.bfloat16, device=dev)
    u_l = torch.empty((wp.batch, wp.seq, wp.d_model), dtype=torch.bfloat16, device=dev)

    def layer_call():
        G.gta_layer_prefill(tl["x"], tl["w_qkc"], tl["w_p"], tl["w_g"], tl["w_o"], kc_l, cc_l, n_q=wp.n_q, out=u_l,
                            workspace=ws_l, status_word=status)

    K_l = max(min(K, 200), 20)
    for i in range(3):
        layer_call()
    barrier()
    l0, l1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    l0.record(stream)
    for i in range(K_l):
        layer_call()
    l1.record(stream)
    barrier()
    t_layer = l0.elapsed_time(l1) / K_l
    assert int(status.item()) == 0, "device status word raised during the benchmark"
    del tl, ws_l, kc_l, cc_l, u_l
    # ---- one decode step of the whole layer on the decode workload's shape (projection of the new token + RoPE +
    #      cache row write + length update, gta_decode, W_O), two cache sets alternating; the lengths are put back
    #      before every step (a copy of 4 bytes per sequence inside the timed loop)
    wl_d = I.scaled(wd, kind="prefill", seq=1)
    tld = [I.layer_inputs(I.scaled(wl_d, seed=wd.seed + i), device=dev) for i in range(2)]
    for t_ in tld:
        t_["x_t"] = t_["x"][:, 0].contiguous()
    ws_ld = torch.zeros(G.layer_decode_workspace_bytes(shape_d, wd.seq + 64), dtype=torch.uint8, device=dev)
    u_ld = torch.empty((wd.batch, wd.d_model), dtype=torch.bfloat16, device=dev)

    def layer_decode_call(i):
        td, tl_ = sets[i % 2], tld[i % 2]
        td["seq_lens"].copy_(td["lens0"])
        G.gta_layer_decode(tl_["x_t"], tl_["w_qkc"], tl_["w_p"], tl_["w_g"], tl_["w_o"], td["k_cache"], td["c_cache"],
                           td["seq_lens"], n_q=wd.n_q, out=u_ld, workspace=ws_ld, status_word=status)

    for i in range(3):
        layer_decode_call(i)
    barrier()
    l2, l3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    l2.record(stream)
    for i in range(K_d):
        layer_decode_call(i)
    l3.record(stream)
    barrier()
    t_layer_decode = l2.elapsed_time(l3) / K_d
    assert int(status.item()) == 0, "device status word raised during the benchmark"
    del tld, ws_ld, u_ld

    total_ms = e_start.elapsed_time(e_end)
    t_attn = sum(e[0].elapsed_time(e[1]) for e in evk) / K_k
    t_dec_k = sum(e[1].elapsed_time(e[2]) for e in evk) / K_k
    t_prefill = sum(e[0].elapsed_time(e[2]) for e in ev) / K
    t_decode_leg = sum(e[2].elapsed_time(e[4]) for e in ev) / K
    t_decode = sum(e[3].elapsed_time(e[4]) for e in ev) / K

    def max_over_ranks_(v):
        return max_over_ranks(v, dist, dev)

    total_ms = max_over_ranks_(total_ms)
    t_attn, t_dec_k, t_prefill = max_over_ranks_(t_attn), max_over_ranks_(t_dec_k), max_over_ranks_(t_prefill)
    t_decode, t_decode_leg = max_over_ranks_(t_decode), max_over_ranks_(t_decode_leg)
    t_decode_b2b = max_over_ranks_(t_decode_b2b)
    t_decode_call = max_over_ranks_(t_decode_call)
    t_decode_paged = max_over_ranks_(t_decode_paged)
    t_layer = max_over_ranks_(t_layer)
    t_layer_decode = max_over_ranks_(t_layer_decode)

    fl = prefill_flops(wp)
    by = decode_bytes(wd, [wd.seq] * wd.batch)
    value = whole_job_rate(fl["total"], world, t_prefill) / 1e12
    path = G.prefill_path(shape_p)

    # ---- roofline of the dominant prefill kernel, and of the decode call
    kernels = [
        dict(kernel="prefill_attention", ms=t_attn, flops=fl["attention"]),
        dict(kernel="prefill_decoder_gate", ms=t_dec_k, flops=fl["decoder"] + fl["gate"]),
    ]
    dom = max(kernels, key=lambda k: k["ms"])
    peak_tf = peaks["bf16_tflops_sustained"]
    roofline = {
        "kernel": dom["kernel"], "bound": "tensor", "achieved": dom["flops"] / (dom["ms"] * 1e-3) / 1e12,
        "peak": peak_tf, "unit": "TFLOP/s", "traffic": NCU_DRAM_BYTES_PER_LAUNCH.get(dom["kernel"]),
        "peak_source": f"bf16_tflops_sustained of {peaks['source']} (kernel timed inside a long step)",
        "timing": f"CUDA events around each kernel in {K_k} further steps of the same loop (prefill call split "
                  "in two, which costs the programmatic overlap the timed region has)",
        "kernels": [dict(kernel=k["kernel"], ms=k["ms"], tflops=k["flops"] / (k["ms"] * 1e-3) / 1e12,
                         frac=k["flops"] / (k["ms"] * 1e-3) / 1e12 / peak_tf) for k in kernels],
        "whole_prefill_frac": fl["total"] / (t_prefill * 1e-3) / 1e12 / peak_tf,
        "whole_prefill_frac_of_burst_peak": fl["total"] / (t_prefill * 1e-3) / 1e12 / peaks["bf16_tflops"],
    }
    roofline["frac"] = roofline["achieved"] / roofline["peak"]
    decode = {
        "workload": wd.name, "step": "gta_cache_append + gta_decode, back to back, two cache sets alternating",
        "ms": t_decode_b2b, "tokens_per_s": world * wd.batch / (t_decode_b2b * 1e-3),
        "ms_decode_call": t_decode_call, "ms_in_step": t_decode_leg, "ms_in_step_decode_call_only": t_decode,
        "roofline": {"bound": "hbm", "achieved": by["total"] / (t_decode_call * 1e-3) / 1e9, "peak": peaks["hbm_gbs"],
                     "unit": "GB/s", "traffic": NCU_DRAM_BYTES_PER_LAUNCH.get("decode_stream"),
                     "peak_source": f"hbm_gbs of {peaks['source']}", "algorithmic_bytes": by["total"],
                     "note": "gta_decode calls back to back (all its kernels, launch gaps included); "
                             "bytes = live cache + weights + vectors",
                     "with_append": {"achieved": by["total"] / (t_decode_b2b * 1e-3) / 1e9,
                                     "frac": by["total"] / (t_decode_b2b * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                     "note": "loop of gta_cache_append + gta_decode (each step on its own "
                                             "length vector, prepared before the loop)"}},
    }
    decode["roofline"]["frac"] = decode["roofline"]["achieved"] / decode["roofline"]["peak"]
    M_l = wp.batch * wp.seq
    fl_layer = fl["total"] + 2.0 * M_l * wp.d_model * ((wp.n_q + wp.n_k) * wp.d_h + wp.n_c * wp.d_l) \
        + 2.0 * M_l * wp.n_heads * wp.d_h * wp.d_model
    layer = {"call": "gta_layer_prefill (X [W_Q|W_K|W_C] + RoPE + cache write, the operator, W_O), back to back",
             "ms": t_layer, "flops": fl_layer, "tflops": fl_layer / (t_layer * 1e-3) / 1e12,
             "frac_of_sustained_peak": fl_layer / (t_layer * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
             "frac_of_burst_peak": fl_layer / (t_layer * 1e-3) / 1e12 / peaks["bf16_tflops"]}
    lw_bytes = 2.0 * (wd.d_model * ((wd.n_q + wd.n_k) * wd.d_h + wd.n_c * wd.d_l) + wd.n_heads * wd.d_h * wd.d_model)
    layer["decode_step"] = {
        "call": "gta_layer_decode on the decode workload's shape, back to back", "ms": t_layer_decode,
        "tokens_per_s": world * wd.batch / (t_layer_decode * 1e-3),
        "algorithmic_bytes": by["total"] + lw_bytes,
        "achieved": (by["total"] + lw_bytes) / (t_layer_decode * 1e-3) / 1e9,
        "frac": (by["total"] + lw_bytes) / (t_layer_decode * 1e-3) / 1e9 / peaks["hbm_gbs"], "unit": "GB/s"}
    decode["paged"] = {"page_size": page_size, "ms_decode_call": t_decode_paged,
                       "achieved": by["total"] / (t_decode_paged * 1e-3) / 1e9,
                       "frac": by["total"] / (t_decode_paged * 1e-3) / 1e9 / peaks["hbm_gbs"],
                       "note": "gta_decode_paged back to back on the same caches scattered over a pool of 64-token "
                               "pages in random order"}

    # ---- end to end: pinned host buffers -> device -> gta_prefill -> pinned host buffer, every step.
    #      Copies and compute run on three streams with double-buffered device inputs and outputs, so
    #      that step i's upload, step i-1's call and step i-2's download overlap (PCIe is full duplex);
    #      the one-stream figure is reported beside it.
    names = ("q", "k", "c", "x")
    host_in = {n: tp[n].cpu().pin_memory() for n in names}
    dev_in = [{n: torch.empty_like(tp[n]) for n in names} for _ in range(2)]
    dev_out = [torch.empty_like(out_p) for _ in range(2)]
    host_out = [torch.empty(out_p.shape, dtype=out_p.dtype).pin_memory() for _ in range(2)]
    h2d = sum(host_in[n].numel() * host_in[n].element_size() for n in names)
    d2h = host_out[0].numel() * host_out[0].element_size()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()

    def e2e_serial_step():
        for n in names:
            dev_in[0][n].copy_(host_in[n], non_blocking=True)
        G.gta_prefill(dev_in[0]["q"], dev_in[0]["k"], dev_in[0]["c"], dev_in[0]["x"], tp["w_p"], tp["w_g"],
                      out=dev_out[0], workspace=ws_p, status_word=status)
        host_out[0].copy_(dev_out[0], non_blocking=True)

    def e2e_run(n_steps):
        ev_in = [torch.cuda.Event() for _ in range(n_steps)]
        ev_cmp = [torch.cuda.Event() for _ in range(n_steps)]
        ev_out = [torch.cuda.Event() for _ in range(n_steps)]
        for i in range(n_steps):
            sl = i % 2
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(ev_cmp[i - 2])       # the call that read this input set is done
                for n in names:
                    dev_in[sl][n].copy_(host_in[n], non_blocking=True)
                ev_in[i].record(s_in)
            stream.wait_event(ev_in[i])
            if i >= 2:
                stream.wait_event(ev_out[i - 2])          # the download of this output buffer is done
            G.gta_prefill(dev_in[sl]["q"], dev_in[sl]["k"], dev_in[sl]["c"], dev_in[sl]["x"], tp["w_p"], tp["w_g"],
                          out=dev_out[sl], workspace=ws_p, status_word=status)
            ev_cmp[i].record(stream)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_cmp[i])
                host_out[sl].copy_(dev_out[sl], non_blocking=True)
                ev_out[i].record(s_out)
        stream.wait_event(ev_out[n_steps - 1])
        if n_steps >= 2:
            stream.wait_event(ev_out[n_steps - 2])

    e2e_steps = min(K, 50)
    for _ in range(3):
        e2e_serial_step()
    barrier()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(e2e_steps):
        e2e_serial_step()
    b.record(stream)
    barrier()
    e2e_serial_ms = max_over_ranks_(a.elapsed_time(b) / e2e_steps)
    e2e_run(4)
    barrier()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    e2e_run(e2e_steps)
    b.record(stream)
    barrier()
    e2e_ms = max_over_ranks_(a.elapsed_time(b) / e2e_steps)
    assert int(status.item()) == 0, "device status word raised during the benchmark"
    e2e = {"value": world * fl["total"] / (e2e_ms * 1e-3) / 1e12, "unit": UNIT, "h2d_bytes_per_step": h2d,
           "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "steps": e2e_steps,
           "how": "upload, gta_prefill and download of consecutive steps overlapped on three streams",
           "one_stream": {"value": world * fl["total"] / (e2e_serial_ms * 1e-3) / 1e12, "ms_per_step": e2e_serial_ms}}

    # ---- CPU oracle baseline (rank 0, single-GPU run only)
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, dt, threads, desc = oracle_prefill_sample(wp, 512)
        cpu_baseline = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc,
                        "seconds": dt}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": args.warmup,
            "ms_per_step": total_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {
                "workload": wp.name, "decode_workload": wd.name, "prefill_path": {1: "plain-ALU", 2: "tcgen05"}.get(path),
                "step": "gta_prefill(c2) then gta_cache_append + gta_decode(c3)",
                "l2": "working set per step ~415 MB > 126 MB L2: the prefill leg touches 136 MB, the decode leg "
                      "streams 279 MB and alternates between two cache sets",
                "replicas": world, "parallelism": "replicas only (no collective on the path)",
            },
            "prefill": {"ms": t_prefill, "tokens_per_s": world * wp.batch * wp.seq / (t_prefill * 1e-3),
                        "flops": fl},
            "layer": layer, "decode": decode, "roofline": roofline, "e2e": e2e, "cpu_baseline": cpu_baseline,
            "gpu_launches": n_launches, "clocks": clocks,
        }
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
