#!/usr/bin/env python
"""Benchmark of the GTA operator library on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One *step* is one pass of the whole hot path over one synthetic batch:
  prefill leg : gta_prefill on workload c2 (B=4, N=2048, H=2048, 16 heads / 4 maps, d_h=128, d_l=512, bf16)
  decode leg  : gta_decode_append (the append of one token per sequence and the decode step in one call) on
                workload c3 (B=32, context 4096, same layer shape, bf16), rotating between two cache sets.
The headline `value` is prefill TFLOP/s (causal-useful flops / device time of the prefill legs);
the decode leg is reported under "decode" (tokens/s, HBM GB/s).  The two largest workloads are
timed in loops of their own and reported under "legs": c4 (one 16384-token prompt, d_l = 1024:
gta_prefill) and c5 (128 ragged sequences of 1024..32768 cached tokens: gta_decode_append
per step), each with its own roofline.  Inputs are resident in HBM for `value`; "e2e"
repeats the prefill through the public call with pinned HOST buffers, host->device and
device->host copies inside the timed region.  Prints ONE JSON line on rank 0.

The timed region is exactly --steps steps; it is repeated until at least MIN_TIMED_MS of device
time have been measured (every other loop likewise), and the median repetition is reported, so the
figures do not depend on --steps.  Tensor-bound fractions are given against both measured peaks
(cuBLAS burst and sustained); the headline denominator follows the clocks sampled during the loop
itself (burst when no sample shows the power cap and the median SM clock is within 5 % of the
maximum, sustained otherwise).

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

MIN_TIMED_MS = 500.0     # device time every timed loop is repeated up to, whatever --steps says

# Kernel -> source file whose hash ties a committed ncu capture to the code that was captured.
KERNEL_SOURCES = {
    "prefill_attention": "paper_2506_17286_b200/csrc/gta_sm100.cu",
    "prefill_decoder_gate": "paper_2506_17286_b200/csrc/gta_sm100_decoder.cu",
    "decode_stream": "paper_2506_17286_b200/csrc/gta_decode_tc.cu",
    "decode_stream_fp8": "paper_2506_17286_b200/csrc/gta_decode_fp8_tc.cu",
}


def load_traffic():
    """dram__bytes_read.sum + dram__bytes_write.sum per launch, read from the ncu summaries under
    profiles/: lines of the form
        traffic: kernel=<name> workload=<name> dram_bytes_per_launch=<number> source_sha256=<first 16 hex digits>
    A figure counts only while the kernel's source file still has that hash; otherwise it is None
    (the kernel has changed since its counters were taken)."""
    import glob
    import hashlib
    import re
    found = {}
    for path in sorted(glob.glob(os.path.join(ROOT, "profiles", "*.md"))):
        with open(path) as f:
            for m in re.finditer(r"traffic: kernel=(\w+) workload=(\w+) dram_bytes_per_launch=([0-9.eE+]+) "
                                 r"source_sha256=([0-9a-f]+)", f.read()):
                kernel, workload, nbytes, sha = m.group(1), m.group(2), float(m.group(3)), m.group(4)
                src = KERNEL_SOURCES.get(kernel)
                if not src or not os.path.exists(os.path.join(ROOT, src)):
                    continue
                with open(os.path.join(ROOT, src), "rb") as g:
                    now = hashlib.sha256(g.read()).hexdigest()
                if now.startswith(sha):
                    found[(kernel, workload)] = dict(bytes=nbytes, source="profiles/" + os.path.basename(path))
    return found

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

    def stop(self):
        if self.proc is None:
            return
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()

    def window(self, t0, t1):
        """Clocks and throttle reasons of the samples taken between wall-clock times t0 and t1."""
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"], samples=0)
        if t1 + 0.2 > time.time():
            time.sleep(0.2)               # let the last samples of the window arrive
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        rows = [(ts, l) for ts, l in list(self.lines) if t0 - 0.05 <= ts <= t1 + 0.15] or list(self.lines)[-3:]
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


def oracle_decode_sample(w, t, idx, n_threads=0):
    """Times the fp64 oracle's decode step, as it stands, on the sequences `idx` of the decode tensors `t`
    (copied to the host first, outside the timed part).  Returns a cpu_baseline record in tokens/s."""
    import torch
    from oracle import gta_oracle
    from paper_2506_17286_b200 import inputs as I
    gta_oracle.build()
    sel = torch.as_tensor(idx, dtype=torch.long, device=t["q"].device)
    lens = t["seq_lens"][sel].cpu().numpy()
    cap = int(lens.max())
    host = {n: t[n][sel].cpu() for n in ("q", "x_t")}
    k = t["k_cache"][sel][:, :, :cap].contiguous().cpu()
    c = t["c_cache"][sel][:, :, :cap].contiguous().cpu()
    ws = I.scaled(w, batch=len(idx))
    shape = gta_oracle.Shape(ws.batch, 0, ws.d_model, ws.n_heads, ws.n_q, ws.n_k, ws.n_c, ws.d_h, ws.d_l, 1, 0.0)
    t0 = time.perf_counter()
    gta_oracle.decode(shape, host["q"], k, c, lens, cap, host["x_t"], t["w_p"].cpu(), t["w_g"].cpu(),
                      n_threads=n_threads)
    dt = time.perf_counter() - t0
    threads = gta_oracle.num_threads() if n_threads <= 0 else n_threads
    nbytes = decode_bytes(ws, lens)["total"]
    return {"value": len(idx) / dt, "unit": "tokens/s", "gb_per_s": nbytes / dt / 1e9, "cores": threads,
            "kind": "oracle", "seconds": dt,
            "sample": f"{len(idx)} of {w.batch} sequences of {w.name} (contexts {sorted(int(v) for v in lens)}); fp64 "
                      "oracle, time includes widening its inputs"}


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
def tensor_peak(peaks, clk):
    """(peak TFLOP/s, its name) for a tensor-bound loop whose clock record is `clk`: the burst figure
    when the loop itself ran in burst conditions (no power-cap sample, median SM clock within 5 % of
    the maximum), the sustained figure otherwise."""
    burst = (clk.get("sm_mhz") is not None and clk.get("sm_max_mhz") and "sw_power_cap" not in clk["reasons"]
             and clk["sm_mhz"] >= 0.95 * clk["sm_max_mhz"])
    if burst:
        return peaks["bf16_tflops"], f"bf16_tflops (burst) of {peaks['source']}: no power cap in the loop's clock record"
    return (peaks["bf16_tflops_sustained"],
            f"bf16_tflops_sustained of {peaks['source']}: power cap or reduced SM clock in the loop's clock record")


def tensor_roofline(flops, ms, peaks, clk, **extra):
    tf = flops / (ms * 1e-3) / 1e12
    peak, why = tensor_peak(peaks, clk)
    r = {"bound": "tensor", "flops": flops, "ms": ms, "achieved": tf, "peak": peak, "unit": "TFLOP/s",
         "frac": tf / peak, "peak_source": why, "frac_of_burst_peak": tf / peaks["bf16_tflops"],
         "frac_of_sustained_peak": tf / peaks["bf16_tflops_sustained"],
         "ms_x_sm_mhz": ms * clk["sm_mhz"] if clk.get("sm_mhz") else None}
    r.update(extra)
    return r


def hbm_roofline(nbytes, ms, peaks, clk, **extra):
    gbs = nbytes / (ms * 1e-3) / 1e9
    r = {"bound": "hbm", "algorithmic_bytes": nbytes, "ms": ms, "achieved": gbs, "peak": peaks["hbm_gbs"],
         "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"], "peak_source": f"hbm_gbs of {peaks['source']}",
         "ms_x_sm_mhz": ms * clk["sm_mhz"] if clk.get("sm_mhz") else None}
    r.update(extra)
    return r


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
    global MIN_TIMED_MS
    MIN_TIMED_MS = float(args.min_timed_ms)
    peaks = load_peaks()
    traffic = load_traffic()
    stream = torch.cuda.current_stream()
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    launches = {"n": 0}

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def mx(v):
        return max_over_ranks(v, dist, dev)

    gpu_id = str(local_rank)
    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        pass
    sampler = ClockSampler(gpu_id)

    def timed_loop(step, n_iter, before_rep=None, min_ms=None, max_reps=400):
        """`n_iter` calls of step(i) between two CUDA events, repeated until `min_ms` of device time
        have been measured (at least 3 repetitions); `before_rep` runs untimed before each repetition.
        Returns (median ms per call over the repetitions, max over ranks; record of the loop)."""
        min_ms = MIN_TIMED_MS if min_ms is None else min(min_ms, MIN_TIMED_MS)
        if before_rep:
            before_rep()
        for i in range(3):
            step(i)
        barrier()
        reps, total, t0 = [], 0.0, time.time()
        while (total < min_ms or len(reps) < 3) and len(reps) < max_reps:
            if before_rep:
                before_rep()
                barrier()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for i in range(n_iter):
                step(i)
            b.record(stream)
            barrier()
            ms = a.elapsed_time(b)
            reps.append(ms / n_iter)
            total += ms
        t1 = time.time()
        assert int(status.item()) == 0, "device status word raised during the benchmark"
        clk = sampler.window(t0, t1)
        med = mx(statistics.median(reps))
        return med, {"ms": med, "ms_best": min(reps), "iters_per_rep": n_iter, "reps": len(reps),
                     "device_ms_total": total, "clocks": clk}

    wp = I.CONFIGS["c2_prefill_bf16"]
    wd = I.CONFIGS["c3_decode_bf16"]
    # ---- prefill leg buffers
    tp = I.prefill_inputs(wp, device=dev)
    shape_p = G.make_shape(batch=wp.batch, seq=wp.seq, d_model=wp.d_model, n_heads=wp.n_heads, n_q=wp.n_q,
                           n_k=wp.n_k, n_c=wp.n_c, d_h=wp.d_h, d_l=wp.d_l, dtype=G.GTA_BF16)
    ws_p = torch.empty(G.prefill_workspace_bytes(shape_p), dtype=torch.uint8, device=dev)
    out_p = torch.empty((wp.batch, wp.seq, wp.n_heads, wp.d_h), dtype=torch.bfloat16, device=dev)
    # ---- decode leg buffers: two cache sets, read alternately
    K = args.steps
    LENS_POOL = max(64, (max(K, 40) + 1) // 2 + 8)   # length vectors per set: one per step of the longest loop
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

    def prefill_leg(ev_mid=None):
        if ev_mid is None:                # the call a user makes: both kernels, programmatically chained
            G.gta_prefill(tp["q"], tp["k"], tp["c"], tp["x"], tp["w_p"], tp["w_g"], out=out_p, workspace=ws_p,
                          status_word=status)
            launches["n"] += G.last_launch_count()
            return
        # kernel by kernel, with an event in between (the per-kernel loop below)
        G.gta_prefill(tp["q"], tp["k"], tp["c"], tp["x"], tp["w_p"], tp["w_g"], out=out_p, workspace=ws_p,
                      status_word=status, stages=1)
        ev_mid.record(stream)
        G.gta_prefill(tp["q"], tp["k"], tp["c"], tp["x"], tp["w_p"], tp["w_g"], out=out_p, workspace=ws_p,
                      status_word=status, stages=2)

    def reset_lens():
        for td in sets:
            td["pool"].copy_(td["lens0"].unsqueeze(0).expand(LENS_POOL, -1))

    def decode_leg(i, ev=None):
        # one decode step including the append of its token (gta_decode_append: one call, no append kernel)
        td = sets[i % 2]
        lens = td["pool"][(i // 2) % LENS_POOL]            # this step's own length vector (wd.seq - 1)
        if ev is not None:
            ev.record(stream)
        G.gta_decode_append(td["q"], td["k_cache"], td["c_cache"], td["k_new"], td["c_new"], lens, td["x_t"], td["w_p"],
                            td["w_g"], out=out_d, workspace=ws_d, status_word=status)
        launches["n"] += G.last_launch_count()

    def decode_leg_two_calls(i):
        td = sets[i % 2]
        lens = td["pool"][(i // 2) % LENS_POOL]
        G.gta_cache_append(td["k_cache"], td["c_cache"], td["k_new"], td["c_new"], lens, status_word=status)
        G.gta_decode(td["q"], td["k_cache"], td["c_cache"], lens, td["x_t"], td["w_p"], td["w_g"],
                     out=out_d, workspace=ws_d, status_word=status)

    for i in range(max(args.warmup, 3)):
        prefill_leg(); decode_leg(i)
    barrier()
    time.sleep(0.6)                       # let nvidia-smi deliver its first samples
    for i in range(3):                    # keep the GPU warm after the sleep (untimed)
        prefill_leg(); decode_leg(i)

    # ---- the timed region: exactly K steps between a barrier + synchronize on both sides, repeated until
    #      MIN_TIMED_MS of device time have been measured; the median repetition is the one reported
    reps = []
    device_total = 0.0
    t_wall0 = time.time()
    while (device_total < MIN_TIMED_MS or len(reps) < 3) and len(reps) < 400:
        reset_lens()
        launches["n"] = 0
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(K)]
        barrier()
        e_start, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e_start.record(stream)
        for i in range(K):
            ev[i][0].record(stream)
            prefill_leg()
            ev[i][1].record(stream)
            decode_leg(i, ev[i][2])
            ev[i][3].record(stream)
        e_end.record(stream)
        barrier()
        total_ms = e_start.elapsed_time(e_end)
        device_total += total_ms
        reps.append(dict(total_ms=total_ms,
                         prefill=sum(e[0].elapsed_time(e[1]) for e in ev) / K,
                         decode_leg=sum(e[1].elapsed_time(e[3]) for e in ev) / K,
                         decode=sum(e[2].elapsed_time(e[3]) for e in ev) / K))
    t_wall1 = time.time()
    n_launches = launches["n"]
    assert int(status.item()) == 0, "device status word raised during the benchmark"
    clocks = sampler.window(t_wall0, t_wall1)
    n_reps = len(reps)
    total_ms = mx(statistics.median(r["total_ms"] for r in reps))
    t_prefill = mx(statistics.median(r["prefill"] for r in reps))
    t_decode_leg = mx(statistics.median(r["decode_leg"] for r in reps))
    t_decode = mx(statistics.median(r["decode"] for r in reps))

    # ---- the same step with the prefill call split into its two kernels and an event between them: the
    #      per-kernel durations (the event costs the programmatic overlap of the two kernels, which is why
    #      the loop above does not carry it)
    K_k = max(20, min(K, 200))
    acc = {"attn": [], "dec": []}

    def split_rep():
        evk = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K_k)]
        reset_lens()
        barrier()
        for i in range(K_k):
            evk[i][0].record(stream)
            prefill_leg(evk[i][1])
            evk[i][2].record(stream)
            decode_leg(i)
        barrier()
        acc["attn"].append(sum(e[0].elapsed_time(e[1]) for e in evk) / K_k)
        acc["dec"].append(sum(e[1].elapsed_time(e[2]) for e in evk) / K_k)
        return sum(e[0].elapsed_time(e[2]) for e in evk)

    split_rep()
    acc = {"attn": [], "dec": []}
    t0k, tot = time.time(), 0.0
    while tot < MIN_TIMED_MS or len(acc["attn"]) < 3:
        tot += split_rep()
    clk_k = sampler.window(t0k, time.time())
    t_attn, t_dec_k = mx(statistics.median(acc["attn"])), mx(statistics.median(acc["dec"]))
    assert int(status.item()) == 0, "device status word raised during the benchmark"

    if args.step_only:
        # the timed region alone (for a profiler's launch list of exactly the kernels of a step): a short line
        if rank == 0:
            fl_ = prefill_flops(wp)
            print(json.dumps({"metric": METRIC, "value": whole_job_rate(fl_["total"], world, t_prefill) / 1e12,
                              "unit": UNIT, "n_gpus": world, "steps": K, "warmup": args.warmup,
                              "ms_per_step": total_ms / K, "step_only": True,
                              "kernels_ms": {"prefill_attention": t_attn, "prefill_decoder_gate": t_dec_k,
                                             "decode_leg": t_decode_leg}, "gpu_launches": n_launches}))
        sampler.stop()
        if dist is not None:
            dist.destroy_process_group()
        return 0

    # ---- decode leg alone, back to back (append + decode, alternating cache sets): the figure the
    #      decode roofline is quoted on; launch gaps between calls are inside the timed region
    K_d = max(K, 40)
    t_decode_b2b, rec_decode_b2b = timed_loop(lambda i: decode_leg(i), K_d, before_rep=reset_lens)
    t_decode_two, rec_decode_two = timed_loop(decode_leg_two_calls, K_d, before_rep=reset_lens, min_ms=250.0)
    # ---- the gta_decode call alone, back to back (no append; same alternation)
    for td in sets:
        td["seq_lens"].copy_(td["lens0"] + 1)

    def decode_call(i):
        td = sets[i % 2]
        G.gta_decode(td["q"], td["k_cache"], td["c_cache"], td["seq_lens"], td["x_t"], td["w_p"], td["w_g"],
                     out=out_d, workspace=ws_d, status_word=status)

    t_decode_call, rec_decode_call = timed_loop(decode_call, K_d)
    # ---- the same call over a paged cache (pages of 64 tokens dealt out at random), back to back
    page_size = 64
    psets = [I.paginate(td, page_size, seed=wd.seed + i) for i, td in enumerate(sets)]
    ws_pg = torch.zeros(G.decode_paged_workspace_bytes(shape_d, page_size, psets[0]["max_pages"]), dtype=torch.uint8,
                        device=dev)

    def decode_paged_call(i):
        td = psets[i % 2]
        G.gta_decode_paged(td["q"], td["k_pool"], td["c_pool"], td["block_table"], td["seq_lens"], td["x_t"],
                           td["w_p"], td["w_g"], out=out_d, workspace=ws_pg, status_word=status)

    t_decode_paged, _ = timed_loop(decode_paged_call, K_d, min_ms=200.0)
    del psets, ws_pg
    # ---- the whole attention layer on the prefill workload's shape (projections + RoPE + cache write, the
    #      operator, the output projection), back to back: context for the operator's figure, not part of `value`
    tl = I.layer_inputs(wp, device=dev)
    ws_l = torch.zeros(G.layer_prefill_workspace_bytes(shape_p), dtype=torch.uint8, device=dev)
    kc_l = torch.zeros((wp.batch, wp.n_k, wp.seq, wp.d_h), dtype=torch.bfloat16, device=dev)
    cc_l = torch.zeros((wp.batch, wp.n_c, wp.seq, wp.d_l), dtype=torch.bfloat16, device=dev)
    u_l = torch.empty((wp.batch, wp.seq, wp.d_model), dtype=torch.bfloat16, device=dev)

    def layer_call(i):
        G.gta_layer_prefill(tl["x"], tl["w_qkc"], tl["w_p"], tl["w_g"], tl["w_o"], kc_l, cc_l, n_q=wp.n_q, out=u_l,
                            workspace=ws_l, status_word=status)

    t_layer, rec_layer = timed_loop(layer_call, max(min(K, 200), 20))
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

    t_layer_decode, rec_layer_decode = timed_loop(layer_decode_call, K_d)
    del tld, ws_ld, u_ld

    fl = prefill_flops(wp)
    by = decode_bytes(wd, [wd.seq] * wd.batch)
    value = whole_job_rate(fl["total"], world, t_prefill) / 1e12
    path = G.prefill_path(shape_p)

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

    e2e_steps = max(20, min(K, 50))
    for _ in range(3):
        e2e_serial_step()
    barrier()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(e2e_steps):
        e2e_serial_step()
    b.record(stream)
    barrier()
    e2e_serial_ms = mx(a.elapsed_time(b) / e2e_steps)
    e2e_run(4)
    barrier()
    e2e_reps, e2e_total = [], 0.0
    while e2e_total < MIN_TIMED_MS or len(e2e_reps) < 3:
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        e2e_run(e2e_steps)
        b.record(stream)
        barrier()
        e2e_total += a.elapsed_time(b)
        e2e_reps.append(a.elapsed_time(b) / e2e_steps)
    e2e_ms = mx(statistics.median(e2e_reps))
    assert int(status.item()) == 0, "device status word raised during the benchmark"
    e2e = {"value": world * fl["total"] / (e2e_ms * 1e-3) / 1e12, "unit": UNIT, "h2d_bytes_per_step": h2d,
           "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "steps": e2e_steps, "reps": len(e2e_reps),
           "how": "upload, gta_prefill and download of consecutive steps overlapped on three streams",
           "one_stream": {"value": world * fl["total"] / (e2e_serial_ms * 1e-3) / 1e12, "ms_per_step": e2e_serial_ms}}
    del host_in, dev_in, dev_out, host_out, tp, ws_p, out_p

    # ---- c4: one prompt of 16384 tokens, d_l = 1024 (gta_prefill back to back, then each kernel looped alone)
    w4 = I.CONFIGS["c4_long_prefill_bf16"]
    t4 = I.prefill_inputs(w4, device=dev)
    shape_4 = G.make_shape(batch=w4.batch, seq=w4.seq, d_model=w4.d_model, n_heads=w4.n_heads, n_q=w4.n_q,
                           n_k=w4.n_k, n_c=w4.n_c, d_h=w4.d_h, d_l=w4.d_l, dtype=G.GTA_BF16)
    ws_4 = torch.empty(G.prefill_workspace_bytes(shape_4), dtype=torch.uint8, device=dev)
    out_4 = torch.empty((w4.batch, w4.seq, w4.n_heads, w4.d_h), dtype=torch.bfloat16, device=dev)

    def c4_call(stages):
        def f(i):
            G.gta_prefill(t4["q"], t4["k"], t4["c"], t4["x"], t4["w_p"], t4["w_g"], out=out_4, workspace=ws_4,
                          status_word=status, stages=stages)
        return f

    t_c4, rec_c4 = timed_loop(c4_call(3), 10)
    t_c4_attn, rec_c4_attn = timed_loop(c4_call(1), 10, min_ms=250.0)
    t_c4_dec, rec_c4_dec = timed_loop(c4_call(2), 20, min_ms=250.0)
    fl4 = prefill_flops(w4)
    del t4, ws_4, out_4

    # ---- GTA against the paper's comparison operator (GQA, App. B.3) in the same harness: the ratios the paper
    #      states analytically (Table 3; Sec. 4.3: 37.5 % of the attention cost and 30 % of the cache at the 1B
    #      hyper-parameters), measured.  Prefill: the attention kernels alone (maps, softmax, latent / value sum) and
    #      GTA's whole operator (decoder + gate included, which GQA does not have); decode: one step, HBM-bound.
    def comparison(name, wl_gta, n_kv, ctx, dec_batch):
        """wl_gta: a GTA prefill workload; the GQA counterpart has the same heads, n_kv key / value heads, same d_h."""
        n_h, d_h, Bp, N = wl_gta.n_heads, wl_gta.d_h, wl_gta.batch, wl_gta.seq
        tg = I.prefill_inputs(wl_gta, device=dev)
        sh = G.make_shape(batch=Bp, seq=N, d_model=wl_gta.d_model, n_heads=n_h, n_q=wl_gta.n_q, n_k=wl_gta.n_k,
                          n_c=wl_gta.n_c, d_h=d_h, d_l=wl_gta.d_l, dtype=G.GTA_BF16)
        ws = torch.empty(G.prefill_workspace_bytes(sh), dtype=torch.uint8, device=dev)
        o = torch.empty((Bp, N, n_h, d_h), dtype=torch.bfloat16, device=dev)

        def gta_call(stages):
            return lambda i: G.gta_prefill(tg["q"], tg["k"], tg["c"], tg["x"], tg["w_p"], tg["w_g"], out=o, workspace=ws,
                                           status_word=status, stages=stages)
        t_gta_attn, _ = timed_loop(gta_call(1), 40, min_ms=150.0)
        t_gta_all, _ = timed_loop(gta_call(3), 40, min_ms=150.0)
        tq = I.gqa_prefill_inputs(Bp, n_h, n_kv, N, d_h, seed=wl_gta.seed, device=dev)
        oq = torch.empty((Bp, n_h, N, d_h), dtype=torch.bfloat16, device=dev)
        t_gqa_attn, _ = timed_loop(lambda i: G.gta_ref_gqa_prefill(tq["q"], tq["k"], tq["v"], out=oq, status_word=status),
                                   40, min_ms=150.0)
        pairs = N * (N + 1) // 2
        fl_gta = 2.0 * Bp * wl_gta.n_q * pairs * (d_h + wl_gta.d_l)
        fl_gqa = 2.0 * Bp * n_h * pairs * 2 * d_h
        del tg, ws, o, tq, oq
        # decode: dec_batch sequences of ctx cached tokens each, two cache sets alternating
        wd_g = I.scaled(wl_gta, kind="decode", batch=dec_batch, seq=ctx)
        sets_g = [I.decode_inputs(I.scaled(wd_g, seed=wd_g.seed + i), device=dev, s_cap=ctx + 64) for i in range(2)]
        sh_d = G.decode_shape(sets_g[0]["q"], sets_g[0]["k_cache"], sets_g[0]["c_cache"], sets_g[0]["x_t"], sets_g[0]["w_p"])
        ws_g = torch.empty(G.decode_workspace_bytes(sh_d, ctx + 64), dtype=torch.uint8, device=dev)
        o_g = torch.empty((dec_batch, n_h, d_h), dtype=torch.bfloat16, device=dev)

        def gta_dec(i):
            td = sets_g[i % 2]
            G.gta_decode(td["q"], td["k_cache"], td["c_cache"], td["seq_lens"], td["x_t"], td["w_p"], td["w_g"], out=o_g,
                         workspace=ws_g, status_word=status)
        t_gta_dec, _ = timed_loop(gta_dec, 40, min_ms=150.0)
        by_gta = decode_bytes(wd_g, [ctx] * dec_batch)
        del sets_g, ws_g, o_g
        sets_q = [I.gqa_decode_inputs(dec_batch, n_h, n_kv, d_h, [ctx] * dec_batch, s_cap=ctx + 64, seed=wd_g.seed + i,
                                      device=dev) for i in range(2)]
        sh_q = G.gqa_shape(batch=dec_batch, seq=0, n_heads=n_h, n_kv=n_kv, d_h=d_h, dtype=torch.bfloat16)
        ws_q = torch.empty(G.gqa_decode_workspace_bytes(sh_q), dtype=torch.uint8, device=dev)
        o_q = torch.empty((dec_batch, n_h, d_h), dtype=torch.bfloat16, device=dev)

        def gqa_dec(i):
            td = sets_q[i % 2]
            G.gta_ref_gqa_decode(td["q"], td["k_cache"], td["v_cache"], td["seq_lens"], out=o_q, workspace=ws_q,
                                 status_word=status)
        t_gqa_dec, _ = timed_loop(gqa_dec, 40, min_ms=150.0)
        cache_gta = (wl_gta.n_k * d_h + wl_gta.n_c * wl_gta.d_l)
        cache_gqa = 2 * n_kv * d_h
        by_gqa = float(dec_batch) * ctx * cache_gqa * 2 + 2.0 * dec_batch * n_h * d_h * 2
        del sets_q, ws_q, o_q
        return {
            "shape": f"{n_h} heads, d_h {d_h}; GTA: {wl_gta.n_q} maps, {wl_gta.n_k} key group(s), d_l {wl_gta.d_l}; "
                     f"GQA: {n_kv} key / value heads; prefill B={Bp}, N={N}; decode B={dec_batch}, context {ctx}",
            "prefill_attention": {
                "gta_ms": t_gta_attn, "gqa_ms": t_gqa_attn, "measured_time_ratio": t_gta_attn / t_gqa_attn,
                "analytic_cost_ratio": fl_gta / fl_gqa, "gta_tflops": fl_gta / (t_gta_attn * 1e-3) / 1e12,
                "gqa_tflops": fl_gqa / (t_gqa_attn * 1e-3) / 1e12,
                "note": "attention kernels alone: n_q (d_h + d_l) N^2 against 2 n_h d_h N^2 (Table 3, 'Attention')"},
            "prefill_operator": {"gta_ms_with_decoder_and_gate": t_gta_all, "ratio_to_gqa_attention": t_gta_all / t_gqa_attn,
                                 "note": "GTA's decoder and gate (2 d_h (d_l + H) flops per token and head) belong to "
                                         "its 'Linear' column; GQA's value projection, which they replace, is not "
                                         "timed here"},
            "decode_step": {
                "gta_ms": t_gta_dec, "gqa_ms": t_gqa_dec, "measured_time_ratio": t_gta_dec / t_gqa_dec,
                "cache_elements_per_token": {"gta": cache_gta, "gqa": cache_gqa, "ratio": cache_gta / cache_gqa},
                "gta_gbs": by_gta["total"] / (t_gta_dec * 1e-3) / 1e9, "gqa_gbs": by_gqa / (t_gqa_dec * 1e-3) / 1e9,
                "note": "GTA's step includes its decoder and gate (weights read once per step); GQA's is attention only. "
                        "The GQA step runs on the warp-level stream kernel; so does GTA's at d_h = 64, while at "
                        "d_h = 128 GTA's runs on the tcgen05 stream kernel (about 5 % faster on the same bytes): part "
                        "of that ratio is the kernel, not the operator"},
        }

    comparisons = {
        "gta_1b_vs_gqa_1b": comparison("1b", I.CONFIGS["x1_gta1b_prefill_bf16"], 5, 8192, 64),
        "c2_shape": comparison("c2", wp, 4, 4096, 32),
    }
    comparisons["paper"] = {"attention_cost_ratio_1b": 0.375, "cache_ratio_1b": 0.30,
                            "source": "Sec. 4.3 / Table 3 of the paper (analytic, GTA-1B against GQA-1B)"}

    # ---- 8-bit caches on the c3 shape: e4m3 codes + one fp32 scale per cached row (quantised on the device by the
    #      library's own append, outside the timed loop); the decode step runs on the streaming kernels
    def fp8_leg():
        ctx, nb = wd.seq, wd.batch
        caches = []
        for i in range(2):
            td = I.decode_inputs(I.scaled(wd, seed=wd.seed + 10 + i), device=dev, s_cap=ctx + 64)
            kq = torch.zeros((nb, wd.n_k, ctx + 64, wd.d_h), dtype=torch.uint8, device=dev)
            cq = torch.zeros((nb, wd.n_c, ctx + 64, wd.d_l), dtype=torch.uint8, device=dev)
            ks = torch.ones((nb, wd.n_k, ctx + 64), dtype=torch.float32, device=dev)
            cs = torch.ones((nb, wd.n_c, ctx + 64), dtype=torch.float32, device=dev)
            lens = torch.zeros(nb, dtype=torch.int32, device=dev)
            G.gta_cache_append_fp8(kq, cq, ks, cs, td["k_cache"][:, :, :ctx].contiguous(),
                                   td["c_cache"][:, :, :ctx].contiguous(), lens, status_word=status)
            caches.append(dict(kq=kq, cq=cq, ks=ks, cs=cs, lens=lens, q=td["q"], x_t=td["x_t"], w_p=td["w_p"], w_g=td["w_g"]))
        ws8 = torch.empty(G.decode_fp8_workspace_bytes(shape_d, ctx + 64), dtype=torch.uint8, device=dev)

        def call(i):
            c = caches[i % 2]
            G.gta_decode_fp8(c["q"], c["kq"], c["cq"], c["ks"], c["cs"], c["lens"], c["x_t"], c["w_p"], c["w_g"], out=out_d,
                             workspace=ws8, status_word=status)
        t8, rec8 = timed_loop(call, 20, min_ms=150.0)
        cache_bytes = float(nb) * ctx * ((wd.n_k * wd.d_h + wd.n_c * wd.d_l) + 4 * (wd.n_k + wd.n_c))
        nbytes = cache_bytes + by["weights"] + by["vectors"]
        r = hbm_roofline(nbytes, t8, peaks, rec8["clocks"],
                         note="gta_decode_fp8 back to back, two cache sets alternating; bytes = codes + scales of the live "
                              "rows + weights + vectors; tcgen05 streaming kernel (kind::f8f6f4, the cached tokens on the rows "
                              "of the MMAs), then the merge and decoder kernels of the bf16 step")
        r["path"] = G.decode_fp8_path(shape_d, ctx + 64)
        tr = traffic.get(("decode_stream_fp8", "c3"))
        r["traffic"] = tr["bytes"] if tr else None
        r["traffic_source"] = tr["source"] if tr else None
        r["cache_bytes_vs_bf16"] = cache_bytes / by["cache"]
        r["ms_vs_bf16_decode_call"] = t8 / t_decode_call
        return r

    fp8_cache = fp8_leg()

    # ---- the c3 shape with its caches left in page-locked host memory and read in place at every step (the setting
    #      of the paper's offload experiments): bound by the host link, not by HBM
    def offload_leg():
        ctx, nb = wd.seq, wd.batch
        sets = []
        for i in range(2):
            td = I.decode_inputs(I.scaled(wd, seed=wd.seed + 20 + i), device=dev, s_cap=ctx + 64)
            for name in ("k_cache", "c_cache"):
                h = torch.empty(td[name].shape, dtype=td[name].dtype, pin_memory=True)
                h.copy_(td[name])
                td[name] = h
            sets.append(td)
        torch.cuda.synchronize()
        wsh = torch.empty(G.decode_hostcache_workspace_bytes(shape_d, ctx + 64), dtype=torch.uint8, device=dev)

        def call(i):
            c = sets[i % 2]
            G.gta_decode_hostcache(c["q"], c["k_cache"], c["c_cache"], c["seq_lens"], c["x_t"], c["w_p"], c["w_g"],
                                   out=out_d, workspace=wsh, status_word=status)
        th, rech = timed_loop(call, 4, min_ms=100.0)
        return {"call": "gta_decode_hostcache back to back, two cache sets alternating", "ms": th,
                "cache_bytes_over_host_link": by["cache"], "host_link_gbs": by["cache"] / (th * 1e-3) / 1e9,
                "tokens_per_s": nb / (th * 1e-3), "ms_vs_device_resident_step": th / t_decode_call,
                "note": "bound by the host link (PCIe), so the step time follows the bytes of the cache per token: "
                        "(n_k d_h + n_c d_l) elements, Table 3 of the paper", "loop": rech}

    offloaded = offload_leg()

    # ---- c5: 128 ragged sequences (1024 .. 32768 cached tokens, 8.9 GB live), gta_cache_append + gta_decode per step
    w5 = I.CONFIGS["c5_ragged_decode_bf16"]
    t5 = I.decode_inputs(w5, device=dev)
    lens5 = t5["seq_lens"].clone()                       # counts the token being decoded
    N5 = 16
    pool5 = (lens5 - 1).unsqueeze(0).repeat(N5, 1).contiguous()
    shape_5 = G.decode_shape(t5["q"], t5["k_cache"], t5["c_cache"], t5["x_t"], t5["w_p"])
    ws_5 = torch.empty(G.decode_workspace_bytes(shape_5, t5["s_cap"]), dtype=torch.uint8, device=dev)
    out_5 = torch.empty((w5.batch, w5.n_heads, w5.d_h), dtype=torch.bfloat16, device=dev)

    def c5_reset():
        pool5.copy_((lens5 - 1).unsqueeze(0).expand(N5, -1))

    def c5_step(i):
        lens = pool5[i % N5]
        G.gta_decode_append(t5["q"], t5["k_cache"], t5["c_cache"], t5["k_new"], t5["c_new"], lens, t5["x_t"], t5["w_p"],
                            t5["w_g"], out=out_5, workspace=ws_5, status_word=status)

    def c5_call(i):
        G.gta_decode(t5["q"], t5["k_cache"], t5["c_cache"], lens5, t5["x_t"], t5["w_p"], t5["w_g"], out=out_5,
                     workspace=ws_5, status_word=status)

    t_c5, rec_c5 = timed_loop(c5_step, N5, before_rep=c5_reset)
    t_c5_call, rec_c5_call = timed_loop(c5_call, N5, min_ms=250.0)
    lens5_host = lens5.cpu().tolist()
    by5 = decode_bytes(w5, lens5_host)

    # ---- the same ragged step over 8-bit caches (quantised sequence by sequence by the library's own append,
    #      outside the timed loop)
    def fp8_ragged_leg():
        cap5, nb5 = (t5["s_cap"] + 3) // 4 * 4, w5.batch     # the streaming path copies scale rows in 16-byte pieces
        kq = torch.zeros((nb5, w5.n_k, cap5, w5.d_h), dtype=torch.uint8, device=dev)
        cq = torch.zeros((nb5, w5.n_c, cap5, w5.d_l), dtype=torch.uint8, device=dev)
        ks = torch.ones((nb5, w5.n_k, cap5), dtype=torch.float32, device=dev)
        cs = torch.ones((nb5, w5.n_c, cap5), dtype=torch.float32, device=dev)
        for b in range(nb5):
            n = int(lens5_host[b])
            zero = torch.zeros(1, dtype=torch.int32, device=dev)
            G.gta_cache_append_fp8(kq[b:b + 1], cq[b:b + 1], ks[b:b + 1], cs[b:b + 1],
                                   t5["k_cache"][b:b + 1, :, :n].contiguous(), t5["c_cache"][b:b + 1, :, :n].contiguous(),
                                   zero, status_word=status)
        ws8 = torch.empty(G.decode_fp8_workspace_bytes(shape_5, cap5), dtype=torch.uint8, device=dev)

        def call(i):
            G.gta_decode_fp8(t5["q"], kq, cq, ks, cs, lens5, t5["x_t"], t5["w_p"], t5["w_g"], out=out_5, workspace=ws8,
                             status_word=status)
        t8, rec8 = timed_loop(call, N5, min_ms=150.0)
        live = float(sum(lens5_host))
        cache_bytes = live * ((w5.n_k * w5.d_h + w5.n_c * w5.d_l) + 4 * (w5.n_k + w5.n_c))
        r = hbm_roofline(cache_bytes + by5["weights"] + by5["vectors"], t8, peaks, rec8["clocks"],
                         note="gta_decode_fp8 on the ragged workload, back to back (its 4.5 GB of codes and scales are far "
                              "larger than L2); bytes = codes + scales of the live rows + weights + vectors")
        r["path"] = G.decode_fp8_path(shape_5, cap5)
        r["ms_vs_bf16_decode_call"] = t8 / t_c5_call
        return r

    fp8_ragged = fp8_ragged_leg()
    append_bytes5 = 2.0 * w5.batch * (w5.n_k * w5.d_h + w5.n_c * w5.d_l) * 2      # read the new rows, write them
    sampler.stop()

    # ---- CPU oracle baselines (rank 0, single-GPU run only): bounded samples of each workload
    cpu_baseline, cpu_c3, cpu_c4, cpu_c5 = None, None, None, None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, dt, threads, desc = oracle_prefill_sample(wp, 512)
        cpu_baseline = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc, "seconds": dt}
        v, dt, threads, desc = oracle_prefill_sample(w4, 24)
        cpu_c4 = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc, "seconds": dt}
        cpu_c3 = oracle_decode_sample(wd, sets[0], list(range(8)))
        order = sorted(range(w5.batch), key=lambda b: lens5_host[b])
        cpu_c5 = oracle_decode_sample(w5, t5, [order[0], order[len(order) // 2], order[-1]])
    del t5, ws_5, out_5

    def with_traffic(r, kernel, workload, scale=1.0):
        tr = traffic.get((kernel, workload))
        r["traffic"] = tr["bytes"] * scale if tr else None
        r["traffic_source"] = tr["source"] if tr else None
        return r

    # ---- rooflines.  c2: each prefill kernel from the split loop, the whole call from the timed region.
    kernels = [
        with_traffic(tensor_roofline(fl["attention"], t_attn, peaks, clk_k, kernel="prefill_attention"),
                     "prefill_attention", "c2"),
        with_traffic(tensor_roofline(fl["decoder"] + fl["gate"], t_dec_k, peaks, clk_k, kernel="prefill_decoder_gate"),
                     "prefill_decoder_gate", "c2"),
    ]
    low = min(kernels, key=lambda k: k["frac"])
    roofline = dict(low)
    roofline.update({
        "why_this_kernel": "the prefill kernel furthest from its roofline (both are listed under kernels)",
        "timing": f"CUDA events around each kernel in further steps of the same loop ({K_k} steps per repetition; "
                  "the prefill call split in two, which costs the programmatic overlap the timed region has)",
        "kernels": kernels,
        "whole_prefill": tensor_roofline(fl["total"], t_prefill, peaks, clocks, call="gta_prefill inside the timed step"),
    })
    decode_roof = with_traffic(hbm_roofline(by["total"], t_decode_call, peaks, rec_decode_call["clocks"],
                                            note="gta_decode calls back to back (all its kernels, launch gaps "
                                                 "included); bytes = live cache + weights + vectors"),
                               "decode_stream", "c3")
    decode_roof["with_append"] = hbm_roofline(by["total"], t_decode_b2b, peaks, rec_decode_b2b["clocks"],
                                              note="loop of gta_decode_append, the step with the append of its token "
                                                   "in one call (each step on its own length vector, prepared "
                                                   "before the loop)")
    decode_roof["with_append_two_calls"] = hbm_roofline(by["total"], t_decode_two, peaks, rec_decode_two["clocks"],
                                                        note="the same step as gta_cache_append + gta_decode")
    decode = {
        "workload": wd.name, "step": "gta_decode_append (append + decode in one call), back to back, two cache sets alternating",
        "ms": t_decode_b2b, "tokens_per_s": world * wd.batch / (t_decode_b2b * 1e-3),
        "ms_decode_call": t_decode_call, "ms_in_step": t_decode_leg, "ms_in_step_decode_call_only": t_decode,
        "roofline": decode_roof, "cpu_baseline": cpu_c3,
        "paged": {"page_size": page_size, "ms_decode_call": t_decode_paged,
                  "achieved": by["total"] / (t_decode_paged * 1e-3) / 1e9,
                  "frac": by["total"] / (t_decode_paged * 1e-3) / 1e9 / peaks["hbm_gbs"],
                  "note": "gta_decode_paged back to back on the same caches scattered over a pool of 64-token "
                          "pages in random order"},
    }
    M_l = wp.batch * wp.seq
    fl_layer = fl["total"] + 2.0 * M_l * wp.d_model * ((wp.n_q + wp.n_k) * wp.d_h + wp.n_c * wp.d_l) \
        + 2.0 * M_l * wp.n_heads * wp.d_h * wp.d_model
    layer = tensor_roofline(fl_layer, t_layer, peaks, rec_layer["clocks"],
                            call="gta_layer_prefill (X [W_Q|W_K|W_C] + RoPE + cache write, the operator, W_O), "
                                 "back to back")
    lw_bytes = 2.0 * (wd.d_model * ((wd.n_q + wd.n_k) * wd.d_h + wd.n_c * wd.d_l) + wd.n_heads * wd.d_h * wd.d_model)
    layer["decode_step"] = hbm_roofline(by["total"] + lw_bytes, t_layer_decode, peaks, rec_layer_decode["clocks"],
                                        call="gta_layer_decode on the decode workload's shape, back to back",
                                        tokens_per_s=world * wd.batch / (t_layer_decode * 1e-3))
    legs = {
        "c2_prefill_bf16": {"call": "gta_prefill inside the timed step", "ms": t_prefill,
                            "tokens_per_s": world * wp.batch * wp.seq / (t_prefill * 1e-3),
                            "roofline": roofline["whole_prefill"], "cpu_baseline": cpu_baseline},
        "c3_decode_bf16": {"call": "gta_decode_append (append + decode in one call), back to back", "ms": t_decode_b2b,
                           "tokens_per_s": world * wd.batch / (t_decode_b2b * 1e-3),
                           "roofline": decode_roof["with_append"], "roofline_decode_call_only": decode_roof,
                           "cpu_baseline": cpu_c3},
        "c4_long_prefill_bf16": {
            "call": "gta_prefill back to back", "ms": t_c4, "tokens_per_s": world * w4.batch * w4.seq / (t_c4 * 1e-3),
            "flops": fl4, "loop": rec_c4,
            "roofline": tensor_roofline(fl4["total"], t_c4, peaks, rec_c4["clocks"]),
            "kernels": [tensor_roofline(fl4["attention"], t_c4_attn, peaks, rec_c4_attn["clocks"],
                                        kernel="prefill_attention", timing="looped alone"),
                        tensor_roofline(fl4["decoder"] + fl4["gate"], t_c4_dec, peaks, rec_c4_dec["clocks"],
                                        kernel="prefill_decoder_gate", timing="looped alone")],
            "cpu_baseline": cpu_c4},
        "c5_ragged_decode_bf16": {
            "call": "gta_decode_append per step (append + decode in one call), back to back (each step on its own length vector)",
            "ms": t_c5, "tokens_per_s": world * w5.batch / (t_c5 * 1e-3), "loop": rec_c5,
            "live_cache_bytes": by5["cache"], "mean_context": sum(lens5_host) / len(lens5_host),
            "roofline": hbm_roofline(by5["total"] + append_bytes5, t_c5, peaks, rec_c5["clocks"]),
            "roofline_decode_call_only": hbm_roofline(by5["total"], t_c5_call, peaks, rec_c5_call["clocks"]),
            "cpu_baseline": cpu_c5},
    }

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": args.warmup,
            "ms_per_step": total_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {
                "workload": wp.name, "decode_workload": wd.name, "also": [wd.name, w4.name, w5.name],
                "prefill_path": {1: "plain-ALU", 2: "tcgen05"}.get(path),
                "step": "gta_prefill(c2) then gta_decode_append(c3): the decode step with the append of its token",
                "l2": "working set per step ~415 MB > 126 MB L2: the prefill leg touches 136 MB, the decode leg "
                      "streams 279 MB and alternates between two cache sets",
                "timed_region": f"exactly {K} steps, repeated {n_reps} times ({device_total:.0f} ms of device time); "
                                "median repetition reported",
                "replicas": world, "parallelism": "replicas only (no collective on the path)",
            },
            "prefill": {"ms": t_prefill, "tokens_per_s": world * wp.batch * wp.seq / (t_prefill * 1e-3),
                        "flops": fl},
            "layer": layer, "decode": decode, "legs": legs, "comparison_with_gqa": comparisons, "fp8_cache_decode": fp8_cache, "fp8_cache_decode_ragged": fp8_ragged,
            "host_cache_decode": offloaded,
            "roofline": roofline,
            "e2e": e2e,
            "cpu_baseline": cpu_baseline, "gpu_launches": n_launches, "clocks": clocks,
        }
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--step-only", action="store_true",
                    help="run the timed region and the per-kernel loop only and print a short line (for a launch list)")
    ap.add_argument("--min-timed-ms", type=float, default=MIN_TIMED_MS,
                    help="device time every timed loop is repeated up to (lower it for a profiler's launch list)")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
