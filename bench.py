#!/usr/bin/env python
"""Benchmark of the LagKV compress pass on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]
                    [--variant lagkv|localkv|l2norm] [--storage bf16|fp16|fp8] [--layers N] [--tune w,t,s,c]
                    [--paged PAGE_ROWS]
    python bench.py --workload sweep --sweep [--sweep-B 1,8]   # one JSON line per (L, r, B) cell of the sweep
    python bench.py --workload decode_append --append          # the incremental pass, one triggering call per step
    python bench.py --workload decode_append --append --loop [--ragged]
                                                               # the whole decode: one call per appended token

A step is one whole compress pass (partition, lag statistics, normalise + std, softmax,
K+V sum, per-head top-k, compaction, sink and window copy) over every layer of one
synthetic cache, issued as ONE kernel launch with the layers folded into the batch
dimension.  The metric is compressed tokens*heads per second,
layers*B*H_kv*Ls / time-per-pass, with inputs resident in HBM; ``e2e`` is the same metric
with the cache starting and the compacted result ending in pinned host memory.  One JSON
line is printed by rank 0 (one per cell with ``--sweep``).  With N > 1 every rank compresses
its own cache of the same shape (independent sequences, no collective on the data path):
weak scaling.  ``--gpus N`` without a torchrun environment starts the N ranks itself.

Beside the contract's keys the default line carries
  ``sustained``     the same launch repeated back to back for at least two seconds with the SM
                    clock sampled every 20 ms: ms per step, median clock, time x clock, and ms
                    per step binned by clock, so that a short burst, single launches and a
                    power-capped run can be told apart;
  ``parity``        counters of a comparison with the float64 oracle on the first layer of the
                    cache, every partition (outside the timed region);
  ``cpu_baseline``  the oracle timed on all host cores, and on one thread.
"""
from __future__ import annotations

import argparse
import ctypes
import datetime
import hashlib
import json
import os
import socket
import statistics
import subprocess
import sys
import tempfile
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

METRIC = "compressed_tokens_heads_per_s"
UNIT = "tokens*heads/s"
DEFAULT_WORKLOAD = "llama8b_128k"
SWEEP_L = (64, 128, 256, 512, 1024, 2048)
SWEEP_R = (0.5, 0.25, 0.125, 0.0625)
TRAFFIC_JSON = ROOT / "profiles" / "ncu_traffic.json"


def algorithmic_bytes(w, L_R: int, variant: int = 0, elem_bytes: int = 2) -> int:
    """Every input row read once, every output row written once, index list written once.
    The L2-norm variant scores from K alone: of V only the L_R output rows are read."""
    units = w.layers * w.B * w.H
    row = w.D * elem_bytes
    if variant == 2:
        return units * (w.S * row + L_R * row + L_R * 2 * row + 4 * L_R)
    return units * ((w.S + L_R) * 2 * row + 4 * L_R)


def measured_peak():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            return float(json.loads(p.read_text())["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
        except Exception:
            pass
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


def kernel_source_hash(files) -> str:
    """Hash of the device source files a kernel is built from: a counter capture stays valid only
    while this does not change."""
    h = hashlib.sha256()
    for name in files:
        f = ROOT / "paper_2504_04704_b200" / "csrc" / name
        h.update(f.name.encode())
        h.update(f.read_bytes())
    return h.hexdigest()[:16]


def captured_traffic(key: str):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu capture recorded in
    profiles/ncu_traffic.json under ``key`` -- null when there is none, or when the kernel's
    source files have changed since the counters were taken."""
    try:
        rec = json.loads(TRAFFIC_JSON.read_text())[key]
        if rec["kernel_source_hash"] != kernel_source_hash(rec["source_files"]):
            return None
        return rec["traffic_bytes_per_launch"]
    except Exception:
        return None


class ClockSampler:
    """nvidia-smi clock / throttle samples taken while a timed region runs."""
    Q = ("timestamp,index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, gpu_index: int, period_ms: int = 20):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", str(period_ms),
                 "-i", str(gpu_index)], stdout=self.tmp, stderr=subprocess.DEVNULL)
        except OSError:
            pass

    def rows(self):
        """(unix time, sm MHz, max sm MHz, watts, [flags]) of every sample so far."""
        self.tmp.flush()
        out = []
        for r in Path(self.tmp.name).read_text().splitlines():
            f = [x.strip() for x in r.split(",")]
            if len(f) < 10:
                continue
            try:
                ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                out.append((ts, float(f[2]), float(f[3]), float(f[4]), f[6:10]))
            except ValueError:
                continue
        return out

    def summary(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        allrows = self.rows()
        inside = [r for r in allrows if t0 - 0.02 <= r[0] <= t1 + 0.02] or allrows[-3:]
        reasons = set()
        for _, _, _, _, fl in inside:
            for n, v in zip(self.NAMES, fl):
                if v.lower().startswith("active"):
                    reasons.add(n)
        sm = [r[1] for r in inside]
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max((r[2] for r in inside), default=None),
                "power_w_max": max((r[3] for r in inside), default=None), "reasons": sorted(reasons),
                "samples": len(inside)}

    def close(self):
        if self.proc is not None:
            self.proc.terminate()
            self.proc.wait()
            self.proc = None
        try:
            os.unlink(self.tmp.name)
        except OSError:
            pass


def time_oracle(w, layers_bits, seconds_target: float = 12.0, threads: int = 0):
    """The oracle as it stands, timed on the host cores: whole-layer passes over the given
    layers (bf16 bit patterns ``[B, H, Ls, D]``), cycled until ``seconds_target`` of CPU time."""
    from oracle import lagkv_oracle
    lagkv_oracle.build()
    all_cores = lagkv_oracle.num_threads()
    if threads:
        lagkv_oracle.set_threads(threads)
    k = lagkv_oracle.keep_count(w.ratio, w.lag)
    cores = lagkv_oracle.num_threads()
    passes, spent = 0, 0.0
    while spent < seconds_target:
        Kb, Vb = layers_bits[passes % len(layers_bits)]
        t0 = time.perf_counter()
        lagkv_oracle.compress(Kb, Vb, w.sink, w.lag, k, want_scores=False)
        spent += time.perf_counter() - t0
        passes += 1
    if threads:
        lagkv_oracle.set_threads(all_cores)
    th = passes * w.B * w.H * w.S
    return {"value": th / spent, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{passes} whole-layer passes cycling over {len(layers_bits)} of the {w.layers} layers of "
                      f"{w.name} (B={w.B}, H={w.H}, Ls={w.S}), {spent:.1f} s of float64 C with OpenMP",
            "seconds": spent, "tokens_heads": th}


def host_layers(w, count: int):
    """``count`` layers of the workload generated on the host (reference arm: no GPU needed)."""
    from paper_2504_04704_b200 import synth
    out = []
    for layer in range(min(count, w.layers)):
        K, V = synth.make_workload_layer(w, layer, device="cpu")
        out.append((synth.to_bits(K), synth.to_bits(V)))
    return out


def run_reference(args, w):
    """--impl reference: the CPU oracle on a bounded sample per step (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    per_step = args.cpu_seconds or max(1.0, min(20.0, 90.0 / max(1, args.steps + args.warmup)))
    layers_bits = host_layers(w, 2)
    vals = []
    last = None
    for i in range(args.warmup + args.steps):
        last = time_oracle(w, layers_bits, seconds_target=per_step)
        if i >= args.warmup:
            vals.append(last)
    tot_th = sum(v["tokens_heads"] for v in vals)
    tot_s = sum(v["seconds"] for v in vals)
    value = tot_th / tot_s
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * tot_s / len(vals),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "layers": w.layers, "B": w.B, "H_kv": w.H, "D": w.D, "Ls": w.S,
                   "sink": w.sink, "lag": w.lag, "keep_ratio": w.ratio,
                   "note": "each step times the CPU oracle on a bounded sample of whole layers"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": last["cores"], "kind": "oracle",
                         "sample": last["sample"]},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------ append
def append_alg_bytes(units, L, k, rem, D):
    """Per unit: the two partitions and the remainder are read once; k kept rows and the window
    (L + rem rows, moved down by L - k) are written once; k positions are recorded."""
    row = D * 2
    return units * ((2 * L + rem) * 2 * row + (k + L + rem) * 2 * row + 4 * k)


def run_append(args, w, binding, synth, dev, local):
    """Incremental pass (Section 2.2, bullets 2-4): every (sequence, layer) holds `Ls` stored rows =
    sink + kept rows + a window of L + rem rows, receives L - rem new rows and compresses one
    partition in place.  A step = two 4-byte-per-sequence length resets (so that every step
    triggers again on the same rows) + ONE launch.  Also times calls that skip."""
    import torch
    Bf, H, D, L, sink = w.layers * w.B, w.H, w.D, w.lag, w.sink
    plan = binding.Plan(Bf, H, D, sink, L, keep_ratio=w.ratio, device=local)
    if args.tune:
        t = [int(x) for x in args.tune.split(",")]
        plan.tune(warps=t[0], tile_rows=t[1], stages=t[2], ctas_per_sm=t[3])
    k = plan.k
    stat0 = sink + ((w.S - sink - L) // k) * k          # the workload's stored rows: sink + groups of k kept rows
    # ... + a window of L + (w.S - stat0 - L) rows; once the new rows fill the second partition
    # (rest = 2L, remainder 0) every sequence triggers
    rem = 0
    seq_trig = stat0 + 2 * L
    S_cap = seq_trig + 8
    K = torch.empty((Bf, H, S_cap, D), dtype=torch.bfloat16, device=dev)
    V = torch.empty_like(K)
    for layer in range(w.layers):
        sl = slice(layer * w.B, (layer + 1) * w.B)
        K[sl], V[sl] = synth.make_kv(w.B, H, S_cap, D, w.seed(layer), w.sigma_k, w.sigma_v, device=dev)
    seq0 = torch.full((Bf,), seq_trig, dtype=torch.int32, device=dev)
    stat0_t = torch.full((Bf,), stat0, dtype=torch.int32, device=dev)
    seq, stat = seq0.clone(), stat0_t.clone()
    ws = plan.new_workspace(1)

    def step():
        seq.copy_(seq0)
        stat.copy_(stat0_t)
        plan.compress_append(K, V, seq, stat, ws, max_new_chunks=1)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    assert plan.read_status(ws)[0] == 0 and int(stat[0]) == stat0 + k and int(seq[0]) == stat0 + k + L + rem
    sampler = ClockSampler(local)
    time.sleep(0.3)
    stream = torch.cuda.current_stream(dev)
    wall0 = time.time()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize()
    wall1 = time.time()
    time.sleep(0.05)
    clocks = sampler.summary(wall0, wall1)
    sampler.close()
    ms_step = e0.elapsed_time(e1) / args.steps
    # calls that find nothing to do (the lengths stay below the trigger)
    e0.record(stream)
    for _ in range(200):
        plan.compress_append(K, V, seq, stat, ws, max_new_chunks=1)
    e1.record(stream)
    torch.cuda.synchronize()
    ms_skip = e0.elapsed_time(e1) / 200
    assert plan.read_status(ws)[0] == 0
    units = Bf * H
    alg = append_alg_bytes(units, L, k, rem, D)
    achieved = alg / (ms_step * 1e-3) / 1e9
    peak, peak_src = measured_peak()
    print(json.dumps({
        "metric": METRIC, "value": units * (2 * L + rem) / (ms_step * 1e-3), "unit": UNIT, "n_gpus": 1,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "mode": "append: one triggering lagkv_compress_append call per step; value counts "
                   "the 2L + rem rows per (sequence, layer, head) that the call streams", "layers": w.layers, "B": w.B,
                   "H_kv": H, "D": D, "stored_rows": seq_trig, "static_rows": stat0, "sink": sink, "lag": L, "keep_k": k,
                   "l2": "%.2f GB touched per call, far larger than the 126 MB L2; no flush" % (alg / 1e9)},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": None if (args.layers or args.tune) else captured_traffic("decode_append"),
                     "peak_source": peak_src, "algorithmic_bytes_per_launch": alg, "kernel": "append"},
        "skip_call_ms": ms_skip, "clocks": clocks, "gpu_launches": args.steps,
    }))


def run_append_loop(args, w, binding, synth, dev, local):
    """The whole decode of the append workload: every (sequence, layer) starts with `Ls` stored rows
    (sink + kept rows + a window of L + 112 rows) and grows by 4096 tokens, ONE
    lagkv_compress_append call after every token.  Most calls find nothing to do and skip on the
    device; a sequence compresses one partition whenever 2L rows have gathered behind its static
    part.  Lockstep: all sequences trigger in the same 8 calls.  ``--ragged``: the windows start
    with different fill, so that the compressions spread over the calls.  Every call is bracketed
    by its own event pair; the token rows are written by plain torch copies outside those pairs."""
    import torch
    Bf, H, D, L, sink = w.layers * w.B, w.H, w.D, w.lag, w.sink
    plan = binding.Plan(Bf, H, D, sink, L, keep_ratio=w.ratio, device=local)
    k = plan.k
    grow = args.tokens
    stat0 = sink + ((w.S - sink - L) // k) * k
    if args.ragged:
        fill = (torch.arange(Bf, dtype=torch.int64) * 37) % L
    else:
        fill = torch.full((Bf,), w.S - stat0 - L, dtype=torch.int64)
    start = stat0 + L + fill
    # a sequence's stored length never exceeds its start + grow; the final one is what the lengths imply
    S_cap = int(start.max()) + 8 * k + 2 * L
    K = torch.empty((Bf, H, S_cap, D), dtype=torch.bfloat16, device=dev)
    V = torch.empty_like(K)
    for layer in range(w.layers):
        sl = slice(layer * w.B, (layer + 1) * w.B)
        K[sl], V[sl] = synth.make_kv(w.B, H, S_cap, D, w.seed(layer), w.sigma_k, w.sigma_v, device=dev)
    # token rows come from a small pool of fresh rows (their values only have to be new data)
    pool = 64
    Knew, Vnew = synth.make_kv(Bf, H, pool, D, w.seed(0) + 77, w.sigma_k, w.sigma_v, device=dev)
    seq = start.to(torch.int32).to(dev)
    stat = torch.full((Bf,), stat0, dtype=torch.int32, device=dev)
    ws = plan.new_workspace(1)
    bidx = torch.arange(Bf, device=dev)
    stream = torch.cuda.current_stream(dev)
    events = []
    for _ in range(3):                                   # warm-up: calls that skip
        plan.compress_append(K, V, seq, stat, ws, max_new_chunks=1)
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    time.sleep(0.2)
    wall0 = time.time()
    t_all0, t_all1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_all0.record(stream)
    for t in range(grow):
        pos = seq.long()
        K[bidx, :, pos] = Knew[:, :, t % pool]
        V[bidx, :, pos] = Vnew[:, :, t % pool]
        seq += 1
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        plan.compress_append(K, V, seq, stat, ws, max_new_chunks=1)
        b.record(stream)
        events.append((a, b))
    t_all1.record(stream)
    torch.cuda.synchronize()
    wall1 = time.time()
    time.sleep(0.05)
    clocks = sampler.summary(wall0, wall1)
    sampler.close()
    assert plan.read_status(ws)[0] == 0
    # host replay of the lengths (lagkv_lengths_after): which calls compressed, and how many sequences
    h_seq, h_stat = [int(x) for x in start], [stat0] * Bf
    compressing = [0] * grow
    for i in range(Bf):
        s_i, t_i = h_seq[i], h_stat[i]
        for t in range(grow):
            if s_i + 1 - t_i < 2 * L:        # below the trigger: nothing to ask the library
                s_i += 1
                continue
            s_i, nt = plan.lengths_after(s_i + 1, t_i)
            compressing[t] += nt != t_i
            t_i = nt
        h_seq[i], h_stat[i] = s_i, t_i
    assert seq.tolist() == h_seq and stat.tolist() == h_stat, "device lengths differ from lagkv_lengths_after"
    ms = [a.elapsed_time(b) for a, b in events]
    ms_calls = sum(ms)
    trig = [(m, c) for m, c in zip(ms, compressing) if c]
    skip = [m for m, c in zip(ms, compressing) if not c]
    comp_units = sum(compressing) * H
    # bytes of the compressing units only (a skipping unit reads two integers); remainder 0 at a trigger
    alg = append_alg_bytes(comp_units, L, k, 0, D)
    ms_trig = sum(m for m, _ in trig)
    peak, peak_src = measured_peak()
    achieved = alg / (ms_trig * 1e-3) / 1e9 if trig else 0.0
    print(json.dumps({
        "metric": METRIC, "value": Bf * H * grow / (ms_calls * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": grow,
        "warmup": 3, "ms_per_step": ms_calls / grow, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "mode": ("decode loop, ragged window offsets" if args.ragged else
                   "decode loop, lockstep") + ": one lagkv_compress_append call per appended token; value = "
                   "appended tokens x (sequence, layer, head) units / time inside the calls",
                   "layers": w.layers, "B": w.B, "H_kv": H, "D": D, "stored_rows_at_start": int(start.max()),
                   "static_rows": stat0, "sink": sink, "lag": L, "keep_k": k, "tokens": grow},
        "calls": {"total": grow, "compressing": len(trig), "skipping": len(skip),
                  "compressions": sum(compressing),
                  "ms_in_calls": ms_calls, "ms_in_compressing_calls": ms_trig,
                  "ms_per_compressing_call": (ms_trig / len(trig)) if trig else None,
                  "us_per_skipping_call": (1e3 * statistics.median(skip)) if skip else None,
                  "ms_whole_loop_with_token_writes": t_all0.elapsed_time(t_all1)},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": None, "peak_source": peak_src, "algorithmic_bytes": alg, "kernel": "append",
                     "note": "algorithmic bytes of the compressing units over the time of the calls in which "
                             "at least one sequence compresses"},
        "clocks": clocks, "gpu_launches": grow,
    }))


# ------------------------------------------------------------------------------ prefill
def time_prefill(torch, step, steps, stream, flush_l2, dev):
    """ms of ``steps`` launches: back to back when the inputs are far larger than L2, else one by
    one with a 256 MiB overwrite before each."""
    if not flush_l2:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            step()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)
    scrub = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in evs:
        scrub.fill_(1)
        a.record(stream)
        step()
        b.record(stream)
    torch.cuda.synchronize()
    return sum(a.elapsed_time(b) for a, b in evs)


def sustained_run(torch, step, stream, sampler, seconds=2.0, group=8):
    """The same launch back to back for at least ``seconds``; groups of ``group`` launches are
    bracketed by events and matched with the clock samples taken meanwhile."""
    marks = [torch.cuda.Event(enable_timing=True)]
    torch.cuda.synchronize()
    wall0 = time.time()
    marks[0].record(stream)
    while True:
        for _ in range(group):
            step()
        ev = torch.cuda.Event(enable_timing=True)
        ev.record(stream)
        marks.append(ev)
        if len(marks) % 8 == 0:          # keep the queue short so that wall time follows device time
            marks[-4].synchronize()
            if time.time() - wall0 >= seconds:
                break
    torch.cuda.synchronize()
    wall1 = time.time()
    time.sleep(0.05)
    offs = [marks[0].elapsed_time(m) for m in marks]            # ms since the start, per mark
    rows = [r for r in sampler.rows() if wall0 <= r[0] <= wall1]
    total_ms = offs[-1]
    nsteps = group * (len(marks) - 1)
    out = {"seconds": total_ms / 1e3, "steps": nsteps, "ms_per_step": total_ms / nsteps, "clock_samples": len(rows)}
    if rows:
        mhz = [r[1] for r in rows]
        out["sm_mhz_median"] = statistics.median(mhz)
        out["sm_mhz_min"], out["sm_mhz_max"] = min(mhz), max(mhz)
        out["power_w_max"] = max(r[3] for r in rows)
        out["ms_x_mhz"] = out["ms_per_step"] * out["sm_mhz_median"]
        reasons = set()
        for r in rows:
            for n, v in zip(ClockSampler.NAMES, r[4]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        out["reasons"] = sorted(reasons)
        bins = {}
        for g in range(len(marks) - 1):
            mid = wall0 + (offs[g] + offs[g + 1]) / 2e3
            clk = min(rows, key=lambda r: abs(r[0] - mid))[1]
            b = int(clk // 100) * 100
            bins.setdefault(b, []).append((offs[g + 1] - offs[g]) / group)
        out["ms_per_step_by_sm_mhz"] = {f"{b}-{b + 99}": {"ms": statistics.mean(v), "groups": len(v)}
                                        for b, v in sorted(bins.items())}
    return out


def parity_sample(torch, binding, synth, w, K, V, variant, store, local):
    """The first layer of the cache, every partition, against the float64 oracle (LagKV, bf16)."""
    sys.path.insert(0, str(ROOT / "tests"))
    import parity_util as pu
    from oracle import lagkv_oracle
    lagkv_oracle.build()
    plan = binding.Plan(w.B, w.H, w.D, w.sink, w.lag, keep_ratio=w.ratio, variant=variant, device=local, dtype=store)
    ws = plan.new_workspace()
    out = plan.compress_prefill(K[:w.B], V[:w.B], ws, want_scores=True)
    assert plan.read_status(ws)[0] == 0
    ref = lagkv_oracle.compress(synth.to_bits(K[:w.B]), synth.to_bits(V[:w.B]), w.sink, w.lag, plan.k,
                                want_rows=False)
    host = {"idx": out["idx"].cpu().numpy(), "scores": out["scores"].cpu().numpy()}
    res = pu.compare_with_oracle(ref, host, w.sink, w.lag, plan.k)
    import numpy as np
    take = host["idx"][..., None].astype(np.int64)
    res["rows_bit_exact"] = bool(
        np.array_equal(synth.to_bits(out["K_out"]), np.take_along_axis(synth.to_bits(K[:w.B]), take, axis=2)) and
        np.array_equal(synth.to_bits(out["V_out"]), np.take_along_axis(synth.to_bits(V[:w.B]), take, axis=2)))
    res["sample"] = f"layer 0 of {w.name}: all {res['partitions']} partitions"
    return res


def run_prefill(args, w, torch, binding, synth, shard, rank, world, local, dev, full=True):
    """One workload on this rank; returns the JSON line (rank 0) or None."""
    import torch.distributed as dist
    Bf = w.layers * w.B
    store = {"bf16": torch.bfloat16, "fp16": torch.float16, "fp8": torch.float8_e4m3fn}[args.storage]
    K = torch.empty((Bf, w.H, w.S, w.D), dtype=store, device=dev)
    V = torch.empty_like(K)
    for layer in range(w.layers):
        k_l, v_l = synth.make_kv(w.B, w.H, w.S, w.D, shard.rank_seed(w.seed(layer), rank), w.sigma_k, w.sigma_v,
                                 device=dev, dtype=store)
        K[layer * w.B:(layer + 1) * w.B], V[layer * w.B:(layer + 1) * w.B] = k_l, v_l
        del k_l, v_l
    variant = {"lagkv": 0, "localkv": 1, "l2norm": 2}[args.variant]
    plan = binding.Plan(Bf, w.H, w.D, w.sink, w.lag, keep_ratio=w.ratio, variant=variant, device=local, dtype=store)
    if args.tune:
        t = [int(x) for x in args.tune.split(",")]
        plan.tune(warps=t[0], tile_rows=t[1], stages=t[2], ctas_per_sm=t[3])
    ws = plan.new_workspace()
    L_R = plan.compressed_len(w.S)
    out = {"K_out": torch.empty((Bf, w.H, L_R, w.D), dtype=store, device=dev),
           "V_out": torch.empty((Bf, w.H, L_R, w.D), dtype=store, device=dev),
           "idx": torch.empty((Bf, w.H, L_R), dtype=torch.int32, device=dev)}
    info = plan.launch_info(w.S)
    step = lambda: plan.compress_prefill(K, V, ws, out=out)
    if args.paged:
        # the same cache cut into pages of args.paged rows, scattered over a pool in random order
        ps = args.paged
        nb = (w.S + ps - 1) // ps
        g = torch.Generator().manual_seed(1)
        perm = torch.randperm(Bf * nb, generator=g).reshape(Bf, nb).to(torch.int32).to(dev)
        pools = []
        for X in (K, V):
            pool = torch.empty((Bf * nb, w.H, ps, w.D), dtype=store, device=dev)
            padded = X if nb * ps == w.S else torch.nn.functional.pad(X, (0, 0, 0, nb * ps - w.S))
            for b in range(Bf):        # rows [j*ps, (j+1)*ps) of sequence b -> page perm[b, j]
                pool[perm[b].long()] = padded[b].reshape(w.H, nb, ps, w.D).permute(1, 0, 2, 3)
            pools.append(pool)
            del padded
        Kp, Vp = pools
        info = dict(info, kernel=info["paged_kernel"], note="launch shape of the paged call's kernel family")

        def step():
            rc = plan.lib.lagkv_compress_prefill_paged(
                plan.handle, binding._ptr(Kp), binding._ptr(Vp), ctypes.byref(lay), w.S, binding._ptr(out["K_out"]),
                binding._ptr(out["V_out"]), binding._ptr(out["idx"]), None, binding._ptr(ws), ws.numel(),
                binding._stream(dev))
            assert rc == 0, rc
        lay = plan._paged(Kp, perm, None)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    assert plan.read_status(ws)[0] == 0
    sampler = ClockSampler(local) if rank == 0 else None
    time.sleep(0.3 if rank == 0 else 0.0)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream(dev)
    input_bytes = 2 * K.numel() * K.element_size()
    flush_l2 = input_bytes < 4 * 126e6          # small caches would be served from the 126 MB L2
    wall0 = time.time()
    ms_total = time_prefill(torch, step, args.steps, stream, flush_l2, dev)
    wall1 = time.time()
    if world > 1:
        dist.barrier()
    ms_total = shard.max_over_ranks(ms_total, dev)
    time.sleep(0.05)
    clocks = sampler.summary(wall0, wall1) if sampler else None
    ms_step = ms_total / args.steps
    units_per_rank = w.layers * w.B * w.H * w.S
    value = shard.job_throughput(units_per_rank, world, ms_step)
    per_ms, sustained = None, None
    if full:
        # spread of single steps (outside the timed region: an event pair around every launch)
        scrub = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if flush_l2 else None
        per = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(20)]
        for a, b in per:
            if flush_l2:
                scrub.fill_(1)
            a.record(stream)
            step()
            b.record(stream)
        torch.cuda.synchronize()
        per_ms = sorted(a.elapsed_time(b) for a, b in per)
        del scrub
        if rank == 0 and not flush_l2 and args.sustained > 0:
            sustained = sustained_run(torch, step, stream, sampler, seconds=args.sustained)
    if sampler:
        sampler.close()
    status = plan.read_status(ws)
    assert status[0] == 0, f"device status {status}"

    # ---- end to end: host cache -> device -> compress -> compacted cache back on the host
    e2e = None
    if args.paged:      # check the timed launch's result against the contiguous call, then report the pass only
        ref = plan.compress_prefill(K, V, ws)
        assert torch.equal(ref["idx"], out["idx"]) and torch.equal(ref["K_out"], out["K_out"])
        assert torch.equal(ref["V_out"], out["V_out"])
        del ref
        full = False
    if full and not args.no_e2e and variant == 0 and args.storage == "bf16":
        chunk = max(1, min(4, w.layers)) * w.B
        while Bf % chunk:
            chunk -= 1
        del out
        hp = binding.HostPrefill(Bf, w.H, w.D, w.S, w.sink, w.lag, keep_ratio=w.ratio, chunk_B=chunk, device=local)
        Kh = torch.empty(K.shape, dtype=torch.bfloat16, pin_memory=True)
        Vh = torch.empty(V.shape, dtype=torch.bfloat16, pin_memory=True)
        Kh.copy_(K)
        Vh.copy_(V)
        Koh = torch.empty((Bf, w.H, L_R, w.D), dtype=torch.bfloat16, pin_memory=True)
        Voh = torch.empty((Bf, w.H, L_R, w.D), dtype=torch.bfloat16, pin_memory=True)
        Ih = torch.empty((Bf, w.H, L_R), dtype=torch.int32, pin_memory=True)
        hp.run(Kh, Vh, Koh, Voh, Ih)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record(stream)
        for _ in range(args.e2e_steps):
            hp.run(Kh, Vh, Koh, Voh, Ih)
        f1.record(stream)
        torch.cuda.synchronize()
        ms_e2e = f0.elapsed_time(f1) / args.e2e_steps
        ms_e2e = shard.max_over_ranks(ms_e2e, dev)
        e2e = {"value": shard.job_throughput(units_per_rank, world, ms_e2e), "unit": UNIT, "ms_per_step": ms_e2e,
               "h2d_bytes_per_step": hp.h2d_bytes, "d2h_bytes_per_step": hp.d2h_bytes, "steps": args.e2e_steps,
               "chunk_layers": chunk // w.B}
        del Kh, Vh, Koh, Voh, Ih, hp

    if rank != 0:
        return None
    peak, peak_src = measured_peak()
    alg = algorithmic_bytes(w, L_R, variant, 1 if args.storage == "fp8" else 2)
    achieved = alg / (ms_step * 1e-3) / 1e9
    captured = not args.layers and not args.tune and variant == 0 and args.storage == "bf16" and not args.paged
    traffic = captured_traffic(w.name) if captured else None   # counters of exactly this launch, else null
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "layers": w.layers, "B": w.B, "H_kv": w.H, "D": w.D, "Ls": w.S,
                   "sink": w.sink, "lag": w.lag, "keep_ratio": w.ratio, "keep_k": plan.k, "L_R": L_R,
                   "variant": args.variant, "paged": (f"pages of {args.paged} rows, random order" if args.paged else None),
                   "storage": args.storage, "parallelism": f"dp{world} (independent caches per rank, no collective)",
                   "launch": info,
                   "l2": ("inputs (%.2f GB per rank) are far larger than the 126 MB L2; no flush" % (input_bytes / 1e9))
                   if not flush_l2 else
                   ("inputs (%.3f GB per rank) would fit L2: every step is timed on its own and a 256 MiB buffer "
                    "is overwritten before each" % (input_bytes / 1e9))},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": traffic, "peak_source": peak_src, "algorithmic_bytes_per_launch": alg,
                     "frac_of_nominal_8TBs": achieved / 8000.0, "kernel": info["kernel"]},
        "clocks": clocks,
        "gpu_launches": args.steps * info["launches"],
    }
    if per_ms:
        line["single_steps_ms"] = {"median": per_ms[len(per_ms) // 2], "min": per_ms[0], "max": per_ms[-1],
                                   "n": len(per_ms),
                                   "note": "this rank, 20 launches timed one by one after the timed region"}
    if sustained:
        sustained["achieved_GBs"] = alg / (sustained["ms_per_step"] * 1e-3) / 1e9
        sustained["frac"] = sustained["achieved_GBs"] / peak
        line["sustained"] = sustained
    if e2e is not None:
        line["e2e"] = e2e
    if full and not args.no_cpu and world == 1 and variant == 0 and args.storage == "bf16":
        try:
            line["parity"] = parity_sample(torch, binding, synth, w, K, V, variant, store, local)
        except AssertionError as e:     # a bench line with a failed comparison must say so, not vanish
            line["parity"] = {"failed": str(e)[:300]}
        layers_bits = [(synth.to_bits(K[l * w.B:(l + 1) * w.B]), synth.to_bits(V[l * w.B:(l + 1) * w.B]))
                       for l in range(min(4, w.layers))]
        del K, V
        cb = time_oracle(w, layers_bits, seconds_target=args.cpu_seconds or 12.0)
        cb.pop("seconds"), cb.pop("tokens_heads")
        one = time_oracle(w, layers_bits[:1], seconds_target=(args.cpu_seconds or 12.0) / 3, threads=1)
        cb["single_thread_value"] = one["value"]
        line["cpu_baseline"] = cb
    return line


def run_sweep(args, w, torch, binding, synth, shard, rank, world, local, dev):
    """Config 4: Ls = 65536, sink = 4, one layer, every (L, r) cell, for each B asked for."""
    from dataclasses import replace
    cell = 0
    for L in SWEEP_L:
        for r in SWEEP_R:
            for B in [int(x) for x in args.sweep_B.split(",")]:
                wc = replace(w, lag=L, ratio=r, B=B, seed_base=w.seed_base + 100 * cell + B)
                line = run_prefill(args, wc, torch, binding, synth, shard, rank, world, local, dev, full=False)
                if line is not None:
                    line["config"]["cell"] = {"L": L, "r": r, "B": B}
                    print(json.dumps(line), flush=True)
            cell += 1


def respawn_under_torchrun(n: int) -> int:
    """--gpus N given without a torchrun environment: start the N ranks on this node."""
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), str(Path(__file__).resolve()), *sys.argv[1:]]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None, help="timed steps (default 100; 20 per cell with --sweep)")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (profiling a smaller case)")
    ap.add_argument("--tune", default="", help="warps,tile_rows,stages,ctas_per_sm override")
    ap.add_argument("--variant", default="lagkv", choices=["lagkv", "localkv", "l2norm"],
                    help="scoring variant of Section 4.3 (the headline metric is lagkv)")
    ap.add_argument("--storage", default="bf16", choices=["bf16", "fp16", "fp8"],
                    help="storage format of the caches (fp16, fp8 = e4m3: device-timed pass only)")
    ap.add_argument("--append", action="store_true",
                    help="time the incremental pass instead: every step is one lagkv_compress_append call in which "
                         "every sequence has just completed a partition and its lag partition (single GPU)")
    ap.add_argument("--loop", action="store_true", help="with --append: the whole decode, one call per appended token")
    ap.add_argument("--ragged", action="store_true", help="with --append --loop: per-sequence window offsets")
    ap.add_argument("--tokens", type=int, default=4096, help="with --append --loop: tokens appended per sequence")
    ap.add_argument("--sweep", action="store_true", help="with --workload sweep: every (L, r) cell, one line each")
    ap.add_argument("--sweep-B", default="1,8", help="batch sizes of the sweep")
    ap.add_argument("--paged", type=int, default=0, help="read the cache through a block table with pages of N rows")
    ap.add_argument("--sustained", type=float, default=2.0, help="seconds of the sustained run (0 = skip)")
    ap.add_argument("--cpu-seconds", type=float, default=0.0,
                    help="CPU time of the oracle sample (default: 12 s in the cpu_baseline leg, up to 20 s per step "
                         "of the reference arm)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=3)
    args = ap.parse_args()
    if args.steps is None:
        args.steps = 20 if args.sweep else 100

    from dataclasses import replace
    from paper_2504_04704_b200 import synth
    w = synth.WORKLOADS[args.workload]
    if args.layers:
        w = replace(w, layers=args.layers)
    if args.impl == "reference":
        return run_reference(args, w)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(respawn_under_torchrun(args.gpus))

    import torch
    import torch.distributed as dist
    import __graft_entry__
    from paper_2504_04704_b200 import binding, shard

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if rank == 0:
        __graft_entry__.build()
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist.barrier()
    binding.load_library()          # fails loudly if the CUDA library is missing
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)

    if args.append:
        if args.loop:
            return run_append_loop(args, w, binding, synth, dev, local)
        return run_append(args, w, binding, synth, dev, local)
    if args.sweep:
        run_sweep(args, w, torch, binding, synth, shard, rank, world, local, dev)
    else:
        line = run_prefill(args, w, torch, binding, synth, shard, rank, world, local, dev)
        if line is not None:
            print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
