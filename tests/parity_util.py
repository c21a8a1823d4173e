"""Helpers shared by the GPU parity tests: checks of a prefill result on sampled
partitions (each recomputed by the oracle on its own) and properties that hold at any size."""
import numpy as np
import torch

from paper_2504_04704_b200 import synth

SCORE_ABS_TOL = 1e-4     # binding tolerance on scores
SCORE_REL_TOL = 2e-5     # tight: |gpu - oracle| <= SCORE_REL_TOL * (2 / L)


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
