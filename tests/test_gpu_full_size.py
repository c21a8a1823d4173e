"""GPU parity at the full sizes of the benchmark configurations, in the launch configuration
``bench.py`` times (layers folded into the batch, planner defaults): properties that hold at any
size over the whole result, and EVERY partition's scores and kept indices against the float64
oracle, which replays the workload layer by layer (cell by cell for the sweep).  The counters
(largest score error, partitions whose index set differs, near-ties under both thresholds) are
printed and, when the environment names a folder in ``LAGKV_COUNTERS_DIR``, written to
``parity_counters.json`` there."""
import json
import os

import numpy as np
import pytest
import torch

import parity_util as pu
from paper_2504_04704_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    from paper_2504_04704_b200 import binding as b
    b.load_library()
    return b


def folded_cache(w, dev="cuda:0"):
    Bf = w.layers * w.B
    K = torch.empty((Bf, w.H, w.S, w.D), dtype=torch.bfloat16, device=dev)
    V = torch.empty_like(K)
    for layer in range(w.layers):
        K[layer * w.B:(layer + 1) * w.B], V[layer * w.B:(layer + 1) * w.B] = synth.make_workload_layer(w, layer, device=dev)
    return K, V


def oracle_all_partitions(oracle, K, V, out, sink, L, k, units_per_step):
    """The oracle over every (b, h, partition) of a folded cache, ``units_per_step`` sequences at a
    time so that the host copies stay small; returns the merged counters."""
    total = {}
    for b0 in range(0, K.shape[0], units_per_step):
        sl = slice(b0, min(K.shape[0], b0 + units_per_step))
        ref = oracle.compress(synth.to_bits(K[sl]), synth.to_bits(V[sl]), sink, L, k, want_rows=False)
        host = {"idx": out["idx"][sl].cpu().numpy(), "scores": out["scores"][sl].cpu().numpy()}
        pu.merge_counters(total, pu.compare_with_oracle(ref, host, sink, L, k))
        del ref, host
    return total


def record_counters(name, counters):
    print(f"{name}: {json.dumps(counters)}")
    root = os.environ.get("LAGKV_COUNTERS_DIR", "")
    if root and os.path.isdir(root):
        path = os.path.join(root, "parity_counters.json")
        allc = json.load(open(path)) if os.path.exists(path) else {}
        allc[name] = counters
        json.dump(allc, open(path, "w"), indent=1, sort_keys=True)


@pytest.mark.parametrize("name", ["llama8b_32k", "llama8b_128k"])
def test_full_size_prefill(binding, oracle, name):
    w = synth.WORKLOADS[name]
    K, V = folded_cache(w)
    plan = binding.Plan(w.layers * w.B, w.H, w.D, w.sink, w.lag, keep_ratio=w.ratio, device=0)
    ws = plan.new_workspace()
    out = plan.compress_prefill(K, V, ws, want_scores=True)
    st = plan.read_status(ws)
    assert st[0] == 0, st
    assert out["L_R"] == {"llama8b_32k": 9728, "llama8b_128k": 19968}[name]
    pu.check_structure(K, V, out, w.sink, w.lag, plan.k, w.S, chunk_units=32)
    counters = oracle_all_partitions(oracle, K, V, out, w.sink, w.lag, plan.k, units_per_step=w.B)
    assert counters["partitions"] == w.layers * w.B * w.H * ((w.S - w.sink) // w.lag - 1)
    counters.update(zero_range_channels=st[2], kernel=plan.launch_info(w.S)["kernel"])
    record_counters(name, counters)


@pytest.mark.parametrize("L,r,rows_only,D", [(1024, 0.25, False, 128), (2048, 0.125, True, 128), (256, 0.5, False, 128),
                                             (512, 0.25, True, 96), (512, 0.25, True, 256), (256, 0.125, True, 64)])
def test_repeated_runs_are_bit_identical(binding, L, r, rows_only, D):
    """The background copy warp and the final gather phase split the kept rows between them by
    timing; whatever the split, every output row must be written exactly as the index list
    says, run after run.  Outputs are poisoned before every run so that a row nobody wrote
    shows up; ``rows_only`` takes the path that parks positions in the output rows."""
    B, H, sink = 24, 8, 16
    S = sink + 18 * L + L // 2 + 3
    K, V = synth.make_kv(B, H, S, D, seed=L + D, device="cuda:0")
    plan = binding.Plan(B, H, D, sink, L, keep_ratio=r, device=0)
    assert plan.launch_info(S)["block"] == 384
    ws = plan.new_workspace()
    L_R = plan.compressed_len(S)
    first = None
    for run in range(12):
        out = {"K_out": torch.full((B, H, L_R, D), -1.0, dtype=torch.bfloat16, device="cuda:0"),
               "V_out": torch.full((B, H, L_R, D), -1.0, dtype=torch.bfloat16, device="cuda:0")}
        if not rows_only:
            out["idx"] = torch.full((B, H, L_R), -1, dtype=torch.int32, device="cuda:0")
        res = plan.compress_prefill(K, V, ws, out=out, want_idx=not rows_only)
        if first is None:
            first = res
            if not rows_only:
                pu.check_structure(K, V, res, sink, L, plan.k, S)
        else:
            assert torch.equal(res["K_out"], first["K_out"]) and torch.equal(res["V_out"], first["V_out"])
            if not rows_only:
                assert torch.equal(res["idx"], first["idx"])
    assert plan.read_status(ws)[0] == 0
    if rows_only:       # same rows as the run that also returns the positions
        full = plan.compress_prefill(K, V, ws)
        assert torch.equal(full["K_out"], first["K_out"]) and torch.equal(full["V_out"], first["V_out"])


CELLS = [(L, r) for L in (64, 128, 256, 512, 1024, 2048) for r in (0.5, 0.25, 0.125, 0.0625)]


@pytest.mark.parametrize("B", [1, 8])
def test_full_size_sweep(binding, oracle, B):
    """Config 4: Ls = 65536, sink = 4, every (L, r) cell, seed per cell."""
    w = synth.WORKLOADS["sweep"]
    total = {}
    for cell, (L, r) in enumerate(CELLS):
        K, V = synth.make_kv(B, w.H, w.S, w.D, seed=4000 + 100 * cell + B, device="cuda:0")
        plan = binding.Plan(B, w.H, w.D, w.sink, L, keep_ratio=r, device=0)
        assert plan.k == int(round(r * L))
        ws = plan.new_workspace()
        out = plan.compress_prefill(K, V, ws, want_scores=True)
        assert plan.read_status(ws)[0] == 0
        pu.check_structure(K, V, out, w.sink, L, plan.k, w.S)
        c = oracle_all_partitions(oracle, K, V, out, w.sink, L, plan.k, units_per_step=4)
        assert c["partitions"] == B * w.H * ((w.S - w.sink) // L - 1)
        pu.merge_counters(total, c)
        del K, V, out
    record_counters(f"sweep_B{B}", total)


def test_full_size_decode_append(binding, oracle):
    """Config 3: B = 16 sequences x 28 layers folded, 4 KV heads, L = 512, k = 128.  Every
    sequence starts with 16384 stored rows (16 sink + 123 x 128 kept + 624 window) and grows
    by 4096 tokens; the append entry point is called after every block of new tokens, which
    triggers 8 compressions of one partition each (after 400, 912, ... appended tokens) and
    skips otherwise.  Sampled sequences are replayed by the oracle."""
    w = synth.WORKLOADS["decode_append"]
    Bf, H, D, L, sink = w.layers * w.B, w.H, w.D, w.lag, w.sink
    plan = binding.Plan(Bf, H, D, sink, L, keep_ratio=w.ratio, device=0)
    k = plan.k
    start, grow = 16384, 4096
    S_cap = start + 8 * k + 2 * L            # the stored cache grows by k rows per trigger
    stat0 = sink + 123 * k
    assert start - stat0 == L + 112
    K = torch.empty((Bf, H, S_cap, D), dtype=torch.bfloat16, device="cuda:0")
    V = torch.empty_like(K)
    Knew = torch.empty((Bf, H, grow, D), dtype=torch.bfloat16, device="cuda:0")
    Vnew = torch.empty_like(Knew)
    for layer in range(w.layers):
        sl = slice(layer * w.B, (layer + 1) * w.B)
        k_l, v_l = synth.make_kv(w.B, H, start + grow, D, w.seed(layer), device="cuda:0")
        K[sl, :, :start], V[sl, :, :start] = k_l[:, :, :start], v_l[:, :, :start]
        Knew[sl], Vnew[sl] = k_l[:, :, start:], v_l[:, :, start:]
    seq = torch.full((Bf,), start, dtype=torch.int32, device="cuda:0")
    stat = torch.full((Bf,), stat0, dtype=torch.int32, device="cuda:0")
    ws = plan.new_workspace(1)
    rng = np.random.default_rng(3)
    sample = sorted({0, Bf - 1, *map(int, rng.integers(Bf, size=4))})
    ref = {b: (synth.to_bits(K[b:b + 1]), synth.to_bits(V[b:b + 1]), np.array([start]), np.array([stat0])) for b in sample}

    done, triggers, calls = 0, 0, 0
    blocks = [200, 200] + [256, 256] * 8          # 400, then 512 per trigger; ends at 4496 > 4096: clipped
    for step in blocks:
        step = min(step, grow - done)
        if step == 0:
            break
        cur = int(seq[0])                          # all sequences advance together in this workload
        K[:, :, cur:cur + step], V[:, :, cur:cur + step] = Knew[:, :, done:done + step], Vnew[:, :, done:done + step]
        seq += step
        before = int(stat[0])
        plan.compress_append(K, V, seq, stat, ws, max_new_chunks=1)
        calls += 1
        triggers += int(stat[0]) != before
        for b in sample:
            Kb, Vb, sb, tb = ref[b]
            c = int(sb[0])
            Kb[:, :, c:c + step] = synth.to_bits(Knew[b:b + 1, :, done:done + step])
            Vb[:, :, c:c + step] = synth.to_bits(Vnew[b:b + 1, :, done:done + step])
            Kb, Vb, sb, tb, _ = oracle.compress_append(Kb, Vb, sb + step, tb, L, k)
            ref[b] = (Kb, Vb, sb, tb)
        done += step
    assert plan.read_status(ws)[0] == 0
    assert done == grow and triggers == 8
    assert seq.tolist() == [stat0 + 8 * k + L + (start - stat0 - L + grow) % L] * Bf
    assert stat.tolist() == [stat0 + 8 * k] * Bf
    for b in sample:
        Kb, Vb, sb, tb = ref[b]
        m = int(sb[0])
        assert int(seq[b]) == m and int(stat[b]) == int(tb[0])
        np.testing.assert_array_equal(synth.to_bits(K[b:b + 1, :, :m]), Kb[:, :, :m])
        np.testing.assert_array_equal(synth.to_bits(V[b:b + 1, :, :m]), Vb[:, :, :m])
    print(f"decode_append: {calls} calls, {triggers} triggers, {len(sample)} sequences replayed by the oracle")


def test_full_size_decode_append_ragged(binding, oracle):
    """Config 3 with per-sequence window offsets: the 448 (sequence, layer) caches start with
    windows of different fill, so every call of the append entry point compresses some sequences
    and skips the others.  1024 tokens are appended in blocks of 64; sampled sequences are
    replayed by the oracle, and the number of compressions is the one the lengths imply."""
    w = synth.WORKLOADS["decode_append"]
    Bf, H, D, L, sink = w.layers * w.B, w.H, w.D, w.lag, w.sink
    plan = binding.Plan(Bf, H, D, sink, L, keep_ratio=w.ratio, device=0)
    k = plan.k
    stat0, grow, block = sink + 123 * k, 1024, 64
    fill = (torch.arange(Bf, dtype=torch.int64) * 37) % L                 # rows beyond one full partition
    start = stat0 + L + fill                                              # stored rows per sequence
    S_cap = int(start.max()) + grow + 8
    K = torch.empty((Bf, H, S_cap, D), dtype=torch.bfloat16, device="cuda:0")
    V = torch.empty_like(K)
    for layer in range(w.layers):
        sl = slice(layer * w.B, (layer + 1) * w.B)
        K[sl], V[sl] = synth.make_kv(w.B, H, S_cap, D, w.seed(layer) + 500, device="cuda:0")
    # rows [start_b + t] of the initial buffers are the tokens appended later: keep a copy of them
    idx_new = (start[:, None] + torch.arange(grow)[None, :]).to("cuda:0")                  # [Bf, grow]
    take = idx_new[:, None, :, None].expand(Bf, H, grow, D)
    Knew, Vnew = torch.gather(K, 2, take), torch.gather(V, 2, take)
    seq = start.to(torch.int32).to("cuda:0")
    stat = torch.full((Bf,), stat0, dtype=torch.int32, device="cuda:0")
    ws = plan.new_workspace(1)
    rng = np.random.default_rng(5)
    sample = sorted({0, Bf - 1, *map(int, rng.integers(Bf, size=4))})
    ref = {b: (synth.to_bits(K[b:b + 1]), synth.to_bits(V[b:b + 1]), np.array([int(start[b])]), np.array([stat0]))
           for b in sample}
    bidx = torch.arange(Bf, device="cuda:0")
    triggers = 0
    for done in range(0, grow, block):
        pos = seq.long()[:, None] + torch.arange(block, device="cuda:0")[None, :]          # where the new rows go
        K[bidx[:, None], :, pos] = Knew[:, :, done:done + block].permute(0, 2, 1, 3)
        V[bidx[:, None], :, pos] = Vnew[:, :, done:done + block].permute(0, 2, 1, 3)
        seq += block
        before = stat.clone()
        plan.compress_append(K, V, seq, stat, ws, max_new_chunks=1)
        triggers += int((stat != before).sum())
        for b in sample:
            Kb, Vb, sb, tb = ref[b]
            c = int(sb[0])
            Kb[:, :, c:c + block] = synth.to_bits(Knew[b:b + 1, :, done:done + block])
            Vb[:, :, c:c + block] = synth.to_bits(Vnew[b:b + 1, :, done:done + block])
            ref[b] = oracle.compress_append(Kb, Vb, sb + block, tb, L, k)[:4]
    assert plan.read_status(ws)[0] == 0
    want = int(((L + fill + grow) // L - 1).sum())                        # partitions completed per sequence
    assert triggers == want and 0 < triggers
    for b in sample:
        Kb, Vb, sb, tb = ref[b]
        m = int(sb[0])
        assert int(seq[b]) == m and int(stat[b]) == int(tb[0])
        np.testing.assert_array_equal(synth.to_bits(K[b:b + 1, :, :m]), Kb[:, :, :m])
        np.testing.assert_array_equal(synth.to_bits(V[b:b + 1, :, :m]), Vb[:, :, :m])
    print(f"decode_append ragged: {grow // block} calls, {triggers} compressions over {Bf} sequences")
