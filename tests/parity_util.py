"""Helpers shared by the GPU parity tests: checks of a prefill result on sampled
partitions (each recomputed by the oracle on its own) and properties that hold at any size."""
import numpy as np
import torch

from paper_2504_04704_b200 import synth

SCORE_ABS_TOL = 1e-4     # binding tolerance on scores
SCORE_REL_TOL = 1e-5     # tight: |gpu - oracle| <= SCORE_REL_TOL * (2 / L)


def compare_with_oracle(ref, out, sink, L, k, abs_tol=SCORE_ABS_TOL, rel_tol=SCORE_REL_TOL, l2norm=False):
    """Every partition of a prefill result against the oracle's (numpy arrays on both sides:
    ``ref`` from ``oracle.compress``, ``out`` with ``idx`` [B,H,L_R] and ``scores`` [B,H,n_c,L]).
    Asserts the bars of the parity tests and returns the counters:

      partitions            partitions compared
      max_abs / max_rel     largest |gpu - oracle| over all tokens, absolute and relative to the
                            mean score 2/L (for the L2-norm variant: relative to the score itself)
      mismatch_partitions   partitions whose kept index set differs from the oracle's
      near_tie_loose        partitions whose oracle k-th / (k+1)-th gap is below ``abs_tol``
      near_tie_tight        ... below twice the partition's own measured score error
      unexplained_*         mismatches that the respective threshold does not excuse (must be 0)
    """
    idx = out["idx"]
    B, H = idx.shape[:2]
    n_c = ref["n_c"]
    assert idx.shape[-1] == ref["L_R"]
    np.testing.assert_array_equal(idx[..., :sink], ref["idx"][..., :sink])
    np.testing.assert_array_equal(idx[..., sink + n_c * k:], ref["idx"][..., sink + n_c * k:])
    s32 = out["scores"].reshape(B, H, n_c, L)
    rs = ref["scores"].reshape(B, H, n_c, L)
    err = np.abs(s32.astype(np.float64) - rs)
    eps = err.max(-1)                                          # per partition
    max_abs = float(eps.max())
    if l2norm:
        max_rel = float((err / np.maximum(np.abs(rs), 1e-30)).max())
    else:
        max_rel = float(max_abs * L / 2.0)
        assert max_abs <= abs_tol, f"score error {max_abs}"
    assert max_rel <= rel_tol, f"relative score error {max_rel}"
    # the GPU's selection is the exact top-k (ties to the lower index) of its own fp32 scores
    base = (sink + np.arange(n_c) * L)[None, None, :, None]
    own = np.sort(np.argsort(-s32, axis=-1, kind="stable")[..., :k], axis=-1) + base
    got = idx[..., sink:sink + n_c * k].reshape(B, H, n_c, k)
    np.testing.assert_array_equal(got, own)
    # index sets against the oracle
    want = ref["idx"][..., sink:sink + n_c * k].reshape(B, H, n_c, k)
    res = {"partitions": int(B * H * n_c), "max_abs": max_abs, "max_rel": max_rel, "mismatch_partitions": 0,
           "near_tie_loose": 0, "near_tie_tight": 0, "unexplained_loose": 0, "unexplained_tight": 0}
    if k < L:
        part = np.partition(rs, L - k - 1, axis=-1)            # ascending: [L-k-1] = (k+1)-th largest
        kth1 = part[..., L - k - 1]
        kth = part[..., L - k:].min(-1)
        gap = kth - kth1
        res["near_tie_loose"] = int((gap < abs_tol).sum())
        res["near_tie_tight"] = int((gap < 2 * eps).sum())
        bad = np.argwhere((got != want).any(-1))
        res["mismatch_partitions"] = int(len(bad))
        for b, h, p in bad:
            if gap[b, h, p] >= abs_tol:
                res["unexplained_loose"] += 1
            diff = np.setxor1d(got[b, h, p], want[b, h, p]) - (sink + p * L)
            if np.any(np.abs(rs[b, h, p][diff] - kth[b, h, p]) > 2 * eps[b, h, p]):
                res["unexplained_tight"] += 1
    else:
        np.testing.assert_array_equal(got, want)
    assert res["unexplained_loose"] == 0 and res["unexplained_tight"] == 0, res
    return res


def merge_counters(total, res):
    """Accumulate the counters of ``compare_with_oracle`` over several calls."""
    if not total:
        total.update(res)
        return total
    for key in res:
        total[key] = max(total[key], res[key]) if key.startswith("max_") else total[key] + res[key]
    return total


def check_partition(oracle, Kcur, Vcur, Kref, Vref, gpu_scores, gpu_kept, k, ddof=1):
    """One partition: GPU fp32 scores and kept offsets (0..L-1, ascending) against the oracle.
    Returns True when the index sets agree exactly, False for an explained near-tie."""
    L = Kcur.shape[0]
    score, _, _ = oracle.partition_scores(synth.to_bits(Kcur), synth.to_bits(Vcur), synth.to_bits(Kref),
                                          synth.to_bits(Vref), ddof=ddof)
    err = np.abs(gpu_scores.astype(np.float64) - score)
    assert err.max() <= SCORE_ABS_TOL, f"score error {err.max()}"
    assert err.max() * L / 2.0 <= SCORE_REL_TOL, f"score error relative to 2/L: {err.max() * L / 2}"
    own = np.sort(np.argsort(-gpu_scores, kind="stable")[:k])
    np.testing.assert_array_equal(gpu_kept, own)            # exact top-k of the GPU's own scores
    want = oracle.topk(score, k)
    if np.array_equal(gpu_kept, want):
        return True
    srt = np.sort(score)[::-1]
    gap = srt[k - 1] - srt[k]
    assert gap < SCORE_ABS_TOL
    diff = np.setxor1d(gpu_kept, want)
    assert np.all(np.abs(score[diff] - srt[k - 1]) <= 2 * err.max()), "index mismatch not explained by score error"
    return False


def check_structure(K, V, out, sink, L, k, Ls, chunk_units=64):
    """Properties that hold at any size, evaluated on the device over the whole result:
    sink and window rows are iota, kept rows lie in their partition and ascend, there are
    exactly k per partition, and every output row is bit-identical to the row idx names."""
    B, H, S, D = K.shape[0], K.shape[1], Ls, K.shape[3]
    n = (Ls - sink) // L
    n_c = n - 1
    idx = out["idx"]
    L_R = idx.shape[-1]
    assert L_R == sink + n_c * k + L + (Ls - sink) % L
    dev = idx.device
    assert torch.equal(idx[..., :sink], torch.arange(sink, device=dev, dtype=torch.int32).expand(B, H, sink))
    win = torch.arange(sink + n_c * L, Ls, device=dev, dtype=torch.int32)
    assert torch.equal(idx[..., sink + n_c * k:], win.expand(B, H, win.numel()))
    kept = idx[..., sink:sink + n_c * k].reshape(B, H, n_c, k)
    lo = (sink + torch.arange(n_c, device=dev, dtype=torch.int32) * L).view(1, 1, n_c, 1)
    assert bool(((kept >= lo) & (kept < lo + L)).all())
    if k > 1:
        assert bool((kept[..., 1:] > kept[..., :-1]).all())
    for b0 in range(0, B, chunk_units):
        sl = slice(b0, min(B, b0 + chunk_units))
        take = idx[sl].long().unsqueeze(-1).expand(-1, -1, -1, D)
        assert torch.equal(out["K_out"][sl], torch.gather(K[sl, :, :Ls], 2, take))
        assert torch.equal(out["V_out"][sl], torch.gather(V[sl, :, :Ls], 2, take))
        del take
    if out.get("scores") is not None:
        tot = out["scores"].double().sum(-1)
        assert float((tot - 2.0).abs().max()) < 1e-4        # two softmaxes per partition


def check_samples(oracle, K, V, out, sink, L, k, Ls, samples, seed, ddof=1):
    """Recompute ``samples`` random (b, h, p) partitions with the oracle."""
    B, H = K.shape[0], K.shape[1]
    n_c = (Ls - sink) // L - 1
    rng = np.random.default_rng(seed)
    exact = 0
    picks = {(int(rng.integers(B)), int(rng.integers(H)), int(rng.integers(n_c))) for _ in range(samples)}
    picks |= {(0, 0, 0), (B - 1, H - 1, n_c - 1)}
    for b, h, p in sorted(picks):
        a = sink + p * L
        gs = out["scores"][b, h, p].cpu().numpy()
        gk = out["idx"][b, h, sink + p * k: sink + (p + 1) * k].cpu().numpy() - a
        exact += check_partition(oracle, K[b, h, a:a + L], V[b, h, a:a + L], K[b, h, a + L:a + 2 * L],
                                 V[b, h, a + L:a + 2 * L], gs, gk, k, ddof)
    return exact, len(picks)
