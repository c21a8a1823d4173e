#!/usr/bin/env python
"""Benchmark of the LagKV prefill compress pass on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]
                    [--variant lagkv|localkv|l2norm] [--storage bf16|fp16] [--layers N] [--tune w,t,s,c]
    python bench.py --workload decode_append --append        # the incremental pass, one call per step

A step is one whole compress pass (partition, lag statistics, normalise + std, softmax,
K+V sum, per-head top-k, compaction, sink and window copy) over every layer of one
synthetic cache, issued as ONE kernel launch with the layers folded into the batch
dimension.  The metric is compressed tokens*heads per second,
layers*B*H_kv*Ls / time-per-pass, with inputs resident in HBM; ``e2e`` is the same metric
with the cache starting and the compacted result ending in pinned host memory.  One JSON
line is printed by rank 0.  With N > 1 every rank compresses its own cache of the same
shape (independent sequences, no collective on the data path): weak scaling.
"""
from __future__ import annotations

import argparse
import json
import os
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

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the stream kernel, from the ncu
# capture summarised under profiles/ (captured on a smaller case of the same kernel and
# scaled by processed units where noted there); None until captured.
NCU_TRAFFIC_BYTES = {"llama8b_128k": 21.7e9}
NCU_TRAFFIC_BYTES_APPEND = {"decode_append": 2.022e9}    # full-size launch captured directly (one-pass metrics)


def algorithmic_bytes(w, L_R: int, variant: int = 0) -> int:
    """Every input row read once, every output row written once, index list written once.
    The L2-norm variant scores from K alone: of V only the L_R output rows are read."""
    units = w.layers * w.B * w.H
    row = w.D * 2
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


class ClockSampler:
    """nvidia-smi clock / throttle samples taken while the timed region runs."""
    Q = ("timestamp,index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(gpu_index)], stdout=self.tmp, stderr=subprocess.DEVNULL)
        except OSError:
            pass

    def stop(self, t0: float, t1: float) -> dict:
        import datetime
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        time.sleep(0.15)
        self.proc.terminate()
        self.proc.wait()
        self.tmp.flush()
        rows = Path(self.tmp.name).read_text().splitlines()
        os.unlink(self.tmp.name)
        sm, smax, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        allrows = []
        for r in rows:
            f = [x.strip() for x in r.split(",")]
            if len(f) < 10:
                continue
            try:
                ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                rec = (ts, float(f[2]), float(f[3]), float(f[4]), f[6:10])
            except ValueError:
                continue
            allrows.append(rec)
        inside = [r for r in allrows if t0 - 0.05 <= r[0] <= t1 + 0.05] or allrows[-3:]
        for ts, a, b, p, fl in inside:
            sm.append(a)
            smax.append(b)
            power.append(p)
            for n, v in zip(names, fl):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None, "reasons": sorted(reasons), "samples": len(inside)}


def time_oracle(w, layers_bits, seconds_target: float = 12.0):
    """The oracle as it stands, timed on the host cores: whole-layer passes over the given
    layers (bf16 bit patterns ``[B, H, Ls, D]``), cycled until ``seconds_target`` of CPU time."""
    from oracle import lagkv_oracle
    lagkv_oracle.build()
    k = lagkv_oracle.keep_count(w.ratio, w.lag)
    cores = lagkv_oracle.num_threads()
    passes, spent = 0, 0.0
    while spent < seconds_target:
        Kb, Vb = layers_bits[passes % len(layers_bits)]
        t0 = time.perf_counter()
        lagkv_oracle.compress(Kb, Vb, w.sink, w.lag, k, want_scores=False)
        spent += time.perf_counter() - t0
        passes += 1
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
    per_step = max(1.0, min(20.0, 90.0 / max(1, args.steps + args.warmup)))
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
    clocks = sampler.stop(wall0, wall1)
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
    row = D * 2
    # per unit: the two partitions and the remainder are read once; k kept rows and the window
    # (L + rem rows, moved down by L - k) are written once; k positions are recorded
    alg = units * ((2 * L + rem) * 2 * row + (k + L + rem) * 2 * row + 4 * k)
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
                     "traffic": None if (args.layers or args.tune) else NCU_TRAFFIC_BYTES_APPEND.get(w.name),
                     "peak_source": peak_src, "algorithmic_bytes_per_launch": alg, "kernel": "lagkv_stream_kernel"},
        "skip_call_ms": ms_skip, "clocks": clocks, "gpu_launches": args.steps,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (profiling a smaller case)")
    ap.add_argument("--tune", default="", help="warps,tile_rows,stages,ctas_per_sm override")
    ap.add_argument("--variant", default="lagkv", choices=["lagkv", "localkv", "l2norm"],
                    help="scoring variant of Section 4.3 (the headline metric is lagkv)")
    ap.add_argument("--storage", default="bf16", choices=["bf16", "fp16"],
                    help="storage format of the caches (fp16: device-timed pass only)")
    ap.add_argument("--append", action="store_true",
                    help="time the incremental pass instead: every step is one lagkv_compress_append call in which "
                         "every sequence has just completed a partition and its lag partition (single GPU)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=3)
    args = ap.parse_args()

    from dataclasses import replace
    from paper_2504_04704_b200 import synth
    w = synth.WORKLOADS[args.workload]
    if args.layers:
        w = replace(w, layers=args.layers)
    if args.impl == "reference":
        return run_reference(args, w)

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
        return run_append(args, w, binding, synth, dev, local)

    # ---- this rank's cache: all layers folded into the batch dimension, resident in HBM
    Bf = w.layers * w.B
    store = torch.float16 if args.storage == "fp16" else torch.bfloat16
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
    input_bytes = 2 * K.numel() * 2
    flush_l2 = input_bytes < 4 * 126e6          # small caches would be served from the 126 MB L2
    wall0 = time.time()
    if not flush_l2:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.steps):
            step()
        e1.record(stream)
        torch.cuda.synchronize()
        ms_total = e0.elapsed_time(e1)
    else:   # time every step on its own and overwrite a buffer twice the size of L2 in between
        scrub = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        for a, b in evs:
            scrub.fill_(1)
            a.record(stream)
            step()
            b.record(stream)
        torch.cuda.synchronize()
        ms_total = sum(a.elapsed_time(b) for a, b in evs)
    wall1 = time.time()
    # spread of single steps (outside the timed region: an event pair around every launch)
    per = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(20)]
    for a, b in per:
        if flush_l2:
            scrub.fill_(1)
        a.record(stream)
        step()
        b.record(stream)
    torch.cuda.synchronize()
    per_ms = sorted(a.elapsed_time(b) for a, b in per)
    if world > 1:
        dist.barrier()
    status = plan.read_status(ws)
    assert status[0] == 0, f"device status {status}"
    ms_total = shard.max_over_ranks(ms_total, dev)
    clocks = sampler.stop(wall0, wall1) if sampler else None
    ms_step = ms_total / args.steps
    units_per_rank = w.layers * w.B * w.H * w.S
    value = shard.job_throughput(units_per_rank, world, ms_step)

    # ---- end to end: host cache -> device -> compress -> compacted cache back on the host
    e2e = None
    if not args.no_e2e and variant == 0 and args.storage == "bf16":
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
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_src = measured_peak()
    alg = algorithmic_bytes(w, L_R, variant)
    achieved = alg / (ms_step * 1e-3) / 1e9
    captured = not args.layers and not args.tune and variant == 0 and args.storage == "bf16"
    traffic = NCU_TRAFFIC_BYTES.get(w.name) if captured else None   # counters of exactly this launch, else null
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "single_steps_ms": {"median": per_ms[len(per_ms) // 2], "min": per_ms[0], "max": per_ms[-1], "n": len(per_ms),
                            "note": "this rank, 20 launches timed one by one after the timed region"},
        "config": {"workload": w.name, "layers": w.layers, "B": w.B, "H_kv": w.H, "D": w.D, "Ls": w.S,
                   "sink": w.sink, "lag": w.lag, "keep_ratio": w.ratio, "keep_k": plan.k, "L_R": L_R,
                   "variant": args.variant,
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
    if e2e is not None:
        line["e2e"] = e2e
    if not args.no_cpu and world == 1 and variant == 0 and args.storage == "bf16":
        layers_bits = [(synth.to_bits(K[l * w.B:(l + 1) * w.B]), synth.to_bits(V[l * w.B:(l + 1) * w.B]))
                       for l in range(min(4, w.layers))]
        del K, V
        cb = time_oracle(w, layers_bits)
        cb.pop("seconds"), cb.pop("tokens_heads")
        line["cpu_baseline"] = cb
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
