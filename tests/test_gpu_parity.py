"""GPU parity: the CUDA library, called through its C ABI, against the float64 CPU oracle
on the same seeded bf16 inputs.

Bars:
  * per-token scores within 1e-4 absolute of the oracle (binding) and, tighter, within
    SCORE_REL_TOL of the mean score 2/L;
  * kept index sets identical to the oracle's, except partitions where the oracle's own
    k-th / (k+1)-th score gap is below the tolerance (counted, and additionally required
    to be explained by the measured score error: every token in the symmetric difference
    lies within 2*eps_p of the oracle's k-th score);
  * the GPU's selection is exactly the top-k (ties to the lower index) of the GPU's own
    fp32 scores -- bit-exact, no tolerance;
  * compacted K/V rows bit-exact given the indices; sink and window bit-identical.
"""
import functools

import numpy as np
import pytest
import torch

from paper_2504_04704_b200 import synth

pytestmark = pytest.mark.gpu

import parity_util as pu

SCORE_ABS_TOL = pu.SCORE_ABS_TOL     # binding tolerance on scores: 1e-4 absolute
SCORE_REL_TOL = pu.SCORE_REL_TOL     # tight: |gpu - oracle| <= 1e-5 * (2 / L)


@pytest.fixture(scope="module")
def binding():
    from paper_2504_04704_b200 import binding as b
    b.load_library()
    return b


def storage_of(oracle, dtype):
    """The oracle's name for a torch storage format."""
    return {torch.bfloat16: oracle.STORAGE_BF16, torch.float16: oracle.STORAGE_FP16,
            torch.float8_e4m3fn: oracle.STORAGE_FP8_E4M3}[dtype]


def check_against_oracle(oracle, Kb, Vb, sink, L, k, ddof, out, stats=None, variant=0, storage=0):
    """Compare a GPU prefill result ``out`` (numpy arrays) with the oracle on bit patterns."""
    ref = oracle.compress(Kb, Vb, sink, L, k, ddof=ddof, variant=variant, storage=storage)
    B, H, S, D = Kb.shape
    assert out["L_R"] == ref["L_R"]
    n_c = ref["n_c"]
    idx = out["idx"]
    # rows bit-exact given the GPU's own indices
    take = idx[..., None].astype(np.int64)
    np.testing.assert_array_equal(out["K_out"], np.take_along_axis(Kb, take, axis=2))
    np.testing.assert_array_equal(out["V_out"], np.take_along_axis(Vb, take, axis=2))
    if n_c == 0:
        np.testing.assert_array_equal(idx, ref["idx"])
        return {"mismatch_partitions": 0, "max_abs": 0.0, "max_rel": 0.0}
    res = pu.compare_with_oracle(ref, out, sink, L, k, abs_tol=SCORE_ABS_TOL, rel_tol=SCORE_REL_TOL)
    if stats is not None:
        stats.update(res)
    return res


def run_prefill(binding, oracle, B, H, D, S, sink, L, k, seed=0, ddof=1, tune=None, sigma_k=1.0, layout="bhsd",
                variant=0, dtype=torch.bfloat16):
    K, V = synth.make_kv(B, H, S, D, seed=seed, sigma_k=sigma_k, device="cuda:0", dtype=dtype)
    strides = (0, 0, 0)
    Kd, Vd = K, V
    if layout == "bshd":        # cache stored [B, S, H, D]; passed as a strided [B, H, S, D] view
        Kd = K.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
        Vd = V.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
        strides = (S * H * D, D, H * D)
    elif layout == "padded":    # rows padded to D + 8 elements
        Kp = torch.zeros((B, H, S, D + 8), dtype=dtype, device="cuda:0")
        Vp = torch.zeros_like(Kp)
        Kp[..., :D], Vp[..., :D] = K, V
        Kd, Vd = Kp, Vp
        strides = (H * S * (D + 8), S * (D + 8), D + 8)
    plan = binding.Plan(B, H, D, sink, L, keep_k=k, std_ddof=ddof, strides=strides, variant=variant, device=0,
                        dtype=dtype)
    if tune:
        plan.tune(**tune)
    ws = plan.new_workspace()
    out = plan.compress_prefill(Kd, Vd, ws, S_in=S, want_scores=True)
    st = plan.read_status(ws)
    assert st[0] == 0, f"device status {st}"
    host = {"L_R": out["L_R"], "idx": out["idx"].cpu().numpy(), "K_out": synth.to_bits(out["K_out"]),
            "V_out": synth.to_bits(out["V_out"]), "scores": out["scores"].cpu().numpy()}
    return check_against_oracle(oracle, synth.to_bits(K), synth.to_bits(V), sink, L, k, ddof, host, variant=variant,
                                storage=storage_of(oracle, dtype))


# ------------------------------------------------------------------------------- prefill
def test_config0_tiny_prefill(binding, oracle):
    """B=1, H=8, D=128, S=4096, sink=16, L=128, r=0.25, seed 0."""
    res = run_prefill(binding, oracle, 1, 8, 128, 4096, 16, 128, 32, seed=0)
    assert res["partitions"] == 8 * 30


@pytest.mark.parametrize("L,k,S_extra", [(64, 4, 60), (100, 25, 7), (72, 72, 0), (256, 1, 255), (512, 128, 3),
                                         (1024, 256, 1008), (2048, 256, 100), (37, 5, 36), (2, 1, 1)])
def test_prefill_lag_sweep(binding, oracle, L, k, S_extra):
    """Partition sizes across several tiles with ragged last tiles and remainders."""
    n = 5 if L >= 512 else 9
    run_prefill(binding, oracle, 2, 3, 128, 4 + n * L + S_extra, 4, L, k, seed=L)


@pytest.mark.parametrize("D", [64, 96, 128, 256])
@pytest.mark.parametrize("ddof", [0, 1])
def test_prefill_head_dims(binding, oracle, D, ddof):
    run_prefill(binding, oracle, 1, 4, D, 16 + 6 * 128 + 37, 16, 128, 32, seed=D + ddof, ddof=ddof)


@pytest.mark.parametrize("D,tile_rows", [(64, 32), (96, 32), (96, 16), (256, 16)])
@pytest.mark.parametrize("variant", [0, 1, 2])
def test_prefill_warp_specialised_head_dims(binding, oracle, D, tile_rows, variant):
    run = run_l2norm if variant == binding.VARIANT_L2NORM else functools.partial(run_prefill, variant=variant)
    run(binding, oracle, 2, 3, D, 16 + 5 * 256 + 201, 16, 256, 64, seed=D + tile_rows + variant,
        tune=dict(warps=12, tile_rows=tile_rows))


@pytest.mark.parametrize("layout", ["bshd", "padded"])
def test_prefill_strided_layouts(binding, oracle, layout):
    run_prefill(binding, oracle, 2, 4, 128, 8 + 4 * 96 + 11, 8, 96, 24, seed=3, layout=layout)


@pytest.mark.parametrize("warps,tile_rows,stages", [(8, 32, 3), (8, 32, 2), (4, 32, 4), (2, 32, 3), (8, 16, 4),
                                                    (4, 16, 2), (2, 16, 8), (12, 32, 2), (12, 16, 3), (12, 16, 2)])
def test_prefill_every_launch_shape(binding, oracle, warps, tile_rows, stages):
    run_prefill(binding, oracle, 1, 6, 128, 16 + 7 * 320 + 100, 16, 320, 80, seed=warps * 100 + tile_rows + stages,
                tune=dict(warps=warps, tile_rows=tile_rows, stages=stages, ctas_per_sm=1))


@pytest.mark.parametrize("warps,tile_rows,stages", [(2, 16, 3), (12, 32, 2)])
def test_prefill_many_units_ranges_start_mid_unit(binding, oracle, warps, tile_rows, stages):
    """More (b, h) units than CTAs and a partition count that does not divide evenly, so
    CTA ranges begin inside units and re-read a reference partition."""
    run_prefill(binding, oracle, 37, 5, 128, 3 + 6 * 64 + 5, 3, 64, 16, seed=77,
                tune=dict(warps=warps, tile_rows=tile_rows, stages=stages, ctas_per_sm=1))


@pytest.mark.parametrize("L,k,S_extra", [(64, 4, 60), (100, 25, 7), (72, 72, 0), (256, 1, 255), (37, 5, 36), (2, 1, 1)])
def test_prefill_warp_specialised_short_partitions(binding, oracle, L, k, S_extra):
    """The warp-specialised kernel forced onto partitions shorter than its default range
    (fewer tiles than streaming warps, ragged tiles, sink shorter than a copy chunk)."""
    run_prefill(binding, oracle, 2, 3, 128, 4 + 9 * L + S_extra, 4, L, k, seed=L + 1,
                tune=dict(warps=12, tile_rows=32, stages=2, ctas_per_sm=1))


@pytest.mark.parametrize("layout", ["bshd", "padded"])
def test_prefill_warp_specialised_strided(binding, oracle, layout):
    run_prefill(binding, oracle, 2, 4, 128, 40 + 4 * 300 + 111, 40, 300, 75, seed=4, layout=layout,
                tune=dict(warps=12, tile_rows=32, stages=2, ctas_per_sm=1))


@pytest.mark.parametrize("L,k", [(4096, 512), (8192, 1024), (8192, 8192), (6000, 7)])
def test_prefill_longest_partitions(binding, oracle, L, k):
    """Partitions up to the largest lag the plan accepts (8192): beyond what the warp-specialised
    kernel holds in shared memory, so the uniform kernel runs, with the selection in registers
    (L <= 5632 at 256 threads) or in shared memory (radix select)."""
    run_prefill(binding, oracle, 1, 2, 128, 16 + 3 * L + 77, 16, L, k, seed=L + k)


def test_prefill_heavy_outliers(binding, oracle):
    run_prefill(binding, oracle, 1, 8, 128, 16 + 8 * 256 + 200, 16, 256, 32, seed=5, sigma_k=1.5)


@pytest.mark.parametrize("warps", [0, 12, 100])
def test_prefill_sink_zero_and_minimal(binding, oracle, warps):
    """n = 2 (one compressed partition), no sink, no remainder, on every kernel family."""
    tune = dict(warps=warps, tile_rows=32, stages=2, ctas_per_sm=1) if warps else None
    run_prefill(binding, oracle, 1, 2, 128, 2 * 128, 0, 128, 32, seed=9, tune=tune)
    run_prefill(binding, oracle, 3, 2, 128, 5 + 2 * 128 + 127, 5, 128, 128, seed=10, tune=tune)   # k = L


def test_prefill_identity_when_too_short(binding, oracle):
    run_prefill(binding, oracle, 2, 2, 128, 16 + 2 * 128 - 1, 16, 128, 32, seed=11)


def test_constant_partition_ties_keep_first_k(binding, oracle):
    """All tokens of a partition identical: every score equals 2/L and the tie rule keeps
    the first k rows (exact, no tolerance)."""
    B, H, D, sink, L, k = 1, 2, 128, 4, 64, 16
    S = sink + 3 * L
    K, V = synth.make_kv(B, H, S, D, seed=13, device="cuda:0")
    K[:, :, sink:sink + L] = K[:, :, sink:sink + 1]
    V[:, :, sink:sink + L] = V[:, :, sink:sink + 1]
    plan = binding.Plan(B, H, D, sink, L, keep_k=k, device=0)
    ws = plan.new_workspace()
    out = plan.compress_prefill(K, V, ws, want_scores=True)
    assert plan.read_status(ws)[0] == 0
    idx = out["idx"].cpu().numpy()
    assert np.all(idx[..., sink:sink + k] == sink + np.arange(k))
    ref = oracle.compress(synth.to_bits(K), synth.to_bits(V), sink, L, k)
    np.testing.assert_array_equal(idx[..., :sink + k], ref["idx"][..., :sink + k])


def test_zero_range_channel(binding, oracle):
    """A reference channel that is constant over the lag partition contributes y = 0."""
    B, H, D, sink, L, k = 1, 2, 128, 4, 64, 16
    S = sink + 3 * L + 5
    K, V = synth.make_kv(B, H, S, D, seed=15, device="cuda:0")
    K[:, :, sink + L:sink + 2 * L, 7] = 1.5
    V[:, :, sink + L:sink + 2 * L, 100] = -0.25
    plan = binding.Plan(B, H, D, sink, L, keep_k=k, device=0)
    ws = plan.new_workspace()
    out = plan.compress_prefill(K, V, ws, want_scores=True)
    st = plan.read_status(ws)
    assert st[0] == 0 and st[2] >= 4      # two heads x (one K + one V channel)
    host = {"L_R": out["L_R"], "idx": out["idx"].cpu().numpy(), "K_out": synth.to_bits(out["K_out"]),
            "V_out": synth.to_bits(out["V_out"]), "scores": out["scores"].cpu().numpy()}
    check_against_oracle(oracle, synth.to_bits(K), synth.to_bits(V), sink, L, k, 1, host)


@pytest.mark.parametrize("warps", [0, 12, 100])
def test_indices_only_and_rows_only(binding, oracle, warps):
    B, H, D, sink, L, k = 1, 3, 128, 8, 128, 32
    S = sink + 4 * L + 17
    K, V = synth.make_kv(B, H, S, D, seed=17, device="cuda:0")
    plan = binding.Plan(B, H, D, sink, L, keep_k=k, device=0)
    if warps:
        plan.tune(warps=warps, tile_rows=32, stages=2, ctas_per_sm=1)
    ws = plan.new_workspace()
    full = plan.compress_prefill(K, V, ws)
    only_idx = plan.compress_prefill(K, V, ws, want_rows=False)
    only_rows = plan.compress_prefill(K, V, ws, want_idx=False)
    assert torch.equal(full["idx"], only_idx["idx"])
    assert torch.equal(full["K_out"], only_rows["K_out"]) and torch.equal(full["V_out"], only_rows["V_out"])
    assert plan.read_status(ws)[0] == 0


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16])
@pytest.mark.parametrize("D", [64, 96, 128, 256])
def test_rows_only_warp_specialised_every_head_dim(binding, oracle, D, dtype):
    """Rows without indices on the warp-specialised kernel: the kept positions are parked in the
    output rows themselves and read back by the copy warp and the final gather, whose lane-to-row
    mapping depends on head_dim.  Many slots per CTA, outputs poisoned before every run; the rows
    must equal those of the run that also returns indices, which is checked against the oracle."""
    B, H, sink, L, k = 8, 5, 16, 256, 64
    S = sink + 21 * L + 77                     # 40 units x 21 slots: five or six slots per CTA
    K, V = synth.make_kv(B, H, S, D, seed=300 + D, device="cuda:0", dtype=dtype)
    plan = binding.Plan(B, H, D, sink, L, keep_k=k, device=0, dtype=dtype)
    info = plan.launch_info(S)
    assert info["kernel"] == "lagkv_ws_kernel" and info["grid"] * 4 < B * H * 21
    ws = plan.new_workspace()
    full = plan.compress_prefill(K, V, ws, want_scores=True)
    assert plan.read_status(ws)[0] == 0
    host = {"L_R": full["L_R"], "idx": full["idx"].cpu().numpy(), "K_out": synth.to_bits(full["K_out"]),
            "V_out": synth.to_bits(full["V_out"]), "scores": full["scores"].cpu().numpy()}
    check_against_oracle(oracle, synth.to_bits(K), synth.to_bits(V), sink, L, k, 1, host,
                         storage=storage_of(oracle, dtype))
    L_R = full["L_R"]
    for run in range(6):
        out = {"K_out": torch.full((B, H, L_R, D), -3.0, dtype=dtype, device="cuda:0"),
               "V_out": torch.full((B, H, L_R, D), -3.0, dtype=dtype, device="cuda:0")}
        res = plan.compress_prefill(K, V, ws, out=out, want_idx=False)
        assert torch.equal(res["K_out"], full["K_out"]) and torch.equal(res["V_out"], full["V_out"]), f"run {run}"
    assert plan.read_status(ws)[0] == 0


def test_power_of_two_channel_rescale_is_bit_invariant(binding):
    """z -> 2^e_c z on every row (exact in bf16) leaves the normalised values, hence the fp32
    scores and the selection, bit-identical."""
    B, H, D, sink, L, k = 1, 4, 128, 0, 128, 32
    S = 5 * L
    K, V = synth.make_kv(B, H, S, D, seed=19, device="cuda:0")
    g = torch.Generator(device="cuda:0").manual_seed(1)
    e = torch.randint(-5, 6, (1, H, 1, D), generator=g, device="cuda:0").float()
    K2, V2 = (K.float() * torch.exp2(e)).to(torch.bfloat16), (V.float() * torch.exp2(-e)).to(torch.bfloat16)
    plan = binding.Plan(B, H, D, sink, L, keep_k=k, device=0)
    ws = plan.new_workspace()
    a = plan.compress_prefill(K, V, ws, want_scores=True)
    b = plan.compress_prefill(K2, V2, ws, want_scores=True)
    assert torch.equal(a["idx"], b["idx"])
    assert torch.equal(a["scores"], b["scores"])


# --------------------------------------------------------------------------- pair kernel
PAIRS = dict(warps=100, tile_rows=32, stages=2, ctas_per_sm=1)


@pytest.mark.parametrize("L,k,S_extra,B", [(64, 4, 60, 2), (64, 16, 0, 40), (100, 25, 7, 2), (72, 72, 0, 2), (128, 32, 100, 3),
                                           (256, 1, 255, 2), (512, 128, 3, 2), (500, 250, 499, 5), (37, 5, 36, 2),
                                           (2, 1, 1, 2)])
def test_pair_kernel_prefill(binding, oracle, L, k, S_extra, B):
    """The kernel for short partitions (four independent K/V warp pairs per CTA, selection by one
    warp): tile counts from 1 to 16 per partition, ragged tiles, remainders, idle pairs."""
    n = 5 if L >= 500 else 9
    run_prefill(binding, oracle, B, 3, 128, 4 + n * L + S_extra, 4, L, k, seed=L + 3, tune=PAIRS)


@pytest.mark.parametrize("D,tile_rows", [(64, 32), (96, 32), (256, 16), (128, 16)])
@pytest.mark.parametrize("ddof", [0, 1])
def test_pair_kernel_head_dims(binding, oracle, D, tile_rows, ddof):
    run_prefill(binding, oracle, 2, 4, D, 16 + 6 * 128 + 37, 16, 128, 32, seed=D + ddof + 1, ddof=ddof,
                tune=dict(PAIRS, tile_rows=tile_rows))


@pytest.mark.parametrize("layout", ["bshd", "padded"])
def test_pair_kernel_strided_and_many_units(binding, oracle, layout):
    run_prefill(binding, oracle, 37, 5, 128, 3 + 6 * 64 + 5, 3, 64, 16, seed=79, layout=layout, tune=PAIRS)


def test_pair_kernel_same_bits_as_other_kernels(binding):
    """Scores and selection do not depend on which kernel ran: bit-identical outputs from the
    pair kernel, the warp-specialised kernel and the uniform kernel."""
    B, H, D, sink, L, k = 3, 4, 128, 8, 256, 64
    S = sink + 7 * L + 99
    K, V = synth.make_kv(B, H, S, D, seed=81, device="cuda:0")
    outs = []
    for tune in (PAIRS, dict(warps=12, tile_rows=32, stages=2, ctas_per_sm=1), dict(warps=4, tile_rows=32, stages=2, ctas_per_sm=2),
                 dict(warps=2, tile_rows=16, stages=3, ctas_per_sm=4)):
        plan = binding.Plan(B, H, D, sink, L, keep_k=k, device=0)
        plan.tune(**tune)
        ws = plan.new_workspace()
        outs.append(plan.compress_prefill(K, V, ws, want_scores=True))
        assert plan.read_status(ws)[0] == 0
    for o in outs[1:]:
        assert torch.equal(o["scores"], outs[0]["scores"]) and torch.equal(o["idx"], outs[0]["idx"])
        assert torch.equal(o["K_out"], outs[0]["K_out"]) and torch.equal(o["V_out"], outs[0]["V_out"])
    with pytest.raises(binding.LagKVError):                  # one warp selects: L <= 512 only
        binding.Plan(1, 2, 128, 4, 1024, keep_k=16, device=0).tune(**PAIRS)


# ------------------------------------------------------------------------------ variants
@pytest.mark.parametrize("L,k,S_extra,B", [(64, 16, 60, 2), (100, 25, 7, 2), (256, 1, 255, 2), (512, 128, 3, 2),
                                           (1024, 256, 1008, 9), (2048, 256, 100, 1), (37, 5, 36, 2), (2, 1, 1, 2)])
def test_localkv_prefill(binding, oracle, L, k, S_extra, B):
    """LocalKV (Eq. 14, Eq. 15): min / max come from the partition that is being scored."""
    n = 5 if L >= 512 else 9
    run_prefill(binding, oracle, B, 3, 128, 4 + n * L + S_extra, 4, L, k, seed=L + 7, variant=binding.VARIANT_LOCALKV)


def test_localkv_many_units_and_minimal(binding, oracle):
    run_prefill(binding, oracle, 37, 5, 128, 3 + 6 * 64 + 5, 3, 64, 16, seed=78, variant=binding.VARIANT_LOCALKV)
    run_prefill(binding, oracle, 1, 2, 128, 2 * 128, 0, 128, 32, seed=10, variant=binding.VARIANT_LOCALKV)   # n = 2
    run_prefill(binding, oracle, 2, 4, 128, 40 + 4 * 300 + 111, 40, 300, 75, seed=4, layout="padded",
                variant=binding.VARIANT_LOCALKV)


L2_REL_TOL = 1e-5     # |gpu - oracle| <= L2_REL_TOL * |oracle| for the norm scores of Eq. 16


@pytest.mark.parametrize("L,k,S_extra,B", [(64, 16, 60, 2), (100, 25, 7, 2), (256, 1, 255, 2), (1024, 256, 1008, 9),
                                           (2048, 256, 100, 1), (37, 5, 36, 2)])
def test_l2norm_prefill(binding, oracle, L, k, S_extra, B):
    """L2-norm variant (Eq. 16): score = -||K row||, no softmax, V only gathered."""
    n = 5 if L >= 512 else 9
    run_l2norm(binding, oracle, B, 3, 128, 4 + n * L + S_extra, 4, L, k, seed=L + 9)


def run_l2norm(binding, oracle, B, H, D, S, sink, L, k, seed, tune=None, dtype=torch.bfloat16):
    K, V = synth.make_kv(B, H, S, D, seed=seed, device="cuda:0", dtype=dtype)
    plan = binding.Plan(B, H, D, sink, L, keep_k=k, variant=binding.VARIANT_L2NORM, device=0, dtype=dtype)
    if tune:
        plan.tune(**tune)
    ws = plan.new_workspace()
    out = plan.compress_prefill(K, V, ws, want_scores=True)
    assert plan.read_status(ws)[0] == 0
    Kb, Vb = synth.to_bits(K), synth.to_bits(V)
    ref = oracle.compress(Kb, Vb, sink, L, k, variant=oracle.VARIANT_L2NORM,
                          storage=storage_of(oracle, dtype))
    idx = out["idx"].cpu().numpy()
    n_c = ref["n_c"]
    assert out["L_R"] == ref["L_R"]
    take = idx[..., None].astype(np.int64)
    np.testing.assert_array_equal(synth.to_bits(out["K_out"]), np.take_along_axis(Kb, take, axis=2))
    np.testing.assert_array_equal(synth.to_bits(out["V_out"]), np.take_along_axis(Vb, take, axis=2))
    np.testing.assert_array_equal(idx[..., :sink], ref["idx"][..., :sink])
    np.testing.assert_array_equal(idx[..., sink + n_c * k:], ref["idx"][..., sink + n_c * k:])
    s32 = out["scores"].cpu().numpy()
    err = np.abs(s32.astype(np.float64) - ref["scores"])
    assert np.all(err <= L2_REL_TOL * np.abs(ref["scores"]))
    own = np.sort(np.argsort(-s32, axis=-1, kind="stable")[..., :k], axis=-1) + (sink + np.arange(n_c) * L)[None, None, :, None]
    got = idx[..., sink:sink + n_c * k].reshape(B, H, n_c, k)
    np.testing.assert_array_equal(got, own)
    want = ref["idx"][..., sink:sink + n_c * k].reshape(B, H, n_c, k)
    for b, h, p in np.argwhere((got != want).any(-1)):
        sc = ref["scores"][b, h, p]
        kth = np.sort(sc)[::-1][k - 1]
        diff = np.setxor1d(got[b, h, p], want[b, h, p]) - (sink + p * L)
        assert np.all(np.abs(sc[diff] - kth) <= 2 * err[b, h, p].max())


def test_variant_shapes(binding):
    """Variants run on the warp-specialised kernel and on the two uniform shapes compiled for
    them; other shapes are refused, and a partition too long for any of them refuses the plan."""
    plan = binding.Plan(1, 2, 128, 4, 64, keep_k=16, variant=binding.VARIANT_LOCALKV, device=0)
    plan.tune(warps=2, tile_rows=16, stages=2, ctas_per_sm=1)
    plan.tune(warps=12, tile_rows=32, stages=2, ctas_per_sm=1)
    with pytest.raises(binding.LagKVError) as e:
        plan.tune(warps=8, tile_rows=32, stages=2, ctas_per_sm=1)     # eight-warp CTAs: LagKV only
    assert e.value.code == binding.LAGKV_EUNSUPPORTED


# ------------------------------------------------------------------------------ fp16 caches
FP16_SHAPES = [(64, 16, 60, None), (128, 16, 100, "pairs"), (100, 25, 7, None), (256, 64, 255, None),
               (512, 128, 3, dict(warps=12, tile_rows=16)), (1024, 256, 1008, None), (2048, 256, 100, None),
               (1024, 128, 5, dict(warps=8, tile_rows=32))]


@pytest.mark.parametrize("L,k,S_extra,tune", FP16_SHAPES)
def test_fp16_prefill(binding, oracle, L, k, S_extra, tune):
    """IEEE fp16 caches through every kernel family, against the oracle reading the same bits as fp16."""
    tune = PAIRS if tune == "pairs" else tune
    B = 30 if tune is PAIRS else 2
    n = 5 if L >= 512 else 9
    run_prefill(binding, oracle, B, 3, 128, 4 + n * L + S_extra, 4, L, k, seed=L + 21, tune=tune, dtype=torch.float16)


@pytest.mark.parametrize("variant", [1, 2])
@pytest.mark.parametrize("L,k", [(64, 16), (512, 128)])
def test_fp16_variants(binding, oracle, variant, L, k):
    if variant == binding.VARIANT_L2NORM:
        run_l2norm(binding, oracle, 2, 3, 128, 4 + 6 * L + 9, 4, L, k, seed=L + variant, dtype=torch.float16)
    else:
        run_prefill(binding, oracle, 2, 3, 128, 4 + 6 * L + 9, 4, L, k, seed=L + variant, variant=variant,
                    dtype=torch.float16)


def test_fp16_append_and_layouts(binding, oracle):
    sink, L, k = 8, 96, 24
    stat = [sink, sink + 3 * k]
    seq = [stat[0] + 3 * L + 3, stat[1] + 2 * L]
    check_append(append_case(binding, oracle, 2, 3, 128, seq[0] + 9, sink, L, k, seq, stat, 2, seed=5,
                             dtype=torch.float16), 2)
    run_prefill(binding, oracle, 2, 4, 128, 40 + 4 * 300 + 111, 40, 300, 75, seed=4, layout="bshd", dtype=torch.float16)


def test_fp16_and_bf16_agree_on_values_both_hold(binding):
    """Values with at most 8 significant bits inside fp16's range: the two storage formats feed
    the same fp32 values into the same arithmetic, so scores and picks are bit-identical."""
    B, H, D, sink, L, k = 2, 3, 128, 4, 256, 64
    S = sink + 6 * L + 77
    K, V = synth.make_kv(B, H, S, D, seed=91, device="cuda:0")          # bf16: 8 significant bits
    K, V = K.clamp(-60000, 60000), V.clamp(-60000, 60000)
    K[K.abs() < 6.2e-5] = 0                                              # below fp16's normal range
    V[V.abs() < 6.2e-5] = 0
    Kh, Vh = K.to(torch.float16), V.to(torch.float16)
    assert torch.equal(Kh.float(), K.float()) and torch.equal(Vh.float(), V.float())
    res = []
    for dt, k_, v_ in ((torch.bfloat16, K, V), (torch.float16, Kh, Vh)):
        plan = binding.Plan(B, H, D, sink, L, keep_k=k, device=0, dtype=dt)
        ws = plan.new_workspace()
        res.append(plan.compress_prefill(k_, v_, ws, want_scores=True))
        assert plan.read_status(ws)[0] == 0
    assert torch.equal(res[0]["idx"], res[1]["idx"]) and torch.equal(res[0]["scores"], res[1]["scores"])
    assert torch.equal(res[0]["K_out"].float(), res[1]["K_out"].float())


@pytest.mark.parametrize("D", [64, 96, 256])
@pytest.mark.parametrize("L,k,tune", [(64, 16, None), (128, 16, "pairs"), (256, 64, None)])
def test_fp16_head_dims(binding, oracle, D, L, k, tune):
    tune = PAIRS if tune == "pairs" else tune
    if tune is PAIRS and D == 256:
        tune = dict(PAIRS, tile_rows=16)
    run_prefill(binding, oracle, 12 if tune else 2, 3, D, 4 + 7 * L + 33, 4, L, k, seed=D + L, tune=tune,
                dtype=torch.float16)


def test_fp16_append_head_dims(binding, oracle):
    for D in (64, 96, 256):
        sink, L, k = 8, 96, 24
        stat = [sink, sink + 3 * k]
        seq = [stat[0] + 3 * L + 3, stat[1] + 2 * L]
        check_append(append_case(binding, oracle, 2, 3, D, seq[0] + 9, sink, L, k, seq, stat, 2, seed=D,
                                 dtype=torch.float16), 2)


def test_fp16_tensor_type_is_checked(binding):
    plan = binding.Plan(1, 2, 128, 4, 64, device=0, dtype=torch.float16)
    K, V = synth.make_kv(1, 2, 300, 128, seed=1, device="cuda:0")
    with pytest.raises(TypeError):
        plan.compress_prefill(K, V, plan.new_workspace())                  # a bf16 tensor for an fp16 plan


# -------------------------------------------------------------------------------- gather
def test_gather(binding, oracle):
    B, H, D, S = 2, 3, 128, 500
    K, V = synth.make_kv(B, H, S, D, seed=21, device="cuda:0")
    g = torch.Generator(device="cuda:0").manual_seed(2)
    idx = torch.randint(0, S, (B, H, 77), generator=g, device="cuda:0", dtype=torch.int32)
    plan = binding.Plan(B, H, D, 4, 64, keep_k=16, device=0)
    ws = plan.new_workspace()
    Ko, Vo = plan.gather(K, V, idx, workspace=ws)
    np.testing.assert_array_equal(synth.to_bits(Ko), oracle.gather(synth.to_bits(K), idx.cpu().numpy()))
    np.testing.assert_array_equal(synth.to_bits(Vo), oracle.gather(synth.to_bits(V), idx.cpu().numpy()))
    assert plan.read_status(ws)[0] == 0
    Ko2, none = plan.gather(K, None, idx)
    assert none is None and torch.equal(Ko, Ko2)
    # an index outside [0, S) is skipped and reported, not dereferenced
    idx[0, 0, 3] = S
    plan.gather(K, V, idx, workspace=ws)
    assert plan.read_status(ws)[0] == binding.LAGKV_EINVAL


# ----------------------------------------------------------------------------- paged caches
def paginate(K, V, page_size, extra_pages=3, seed=0, pad=0):
    """Scatter contiguous caches ``[B, H, S, D]`` over pools ``[num_pages, H, page_size, D (+ pad)]`` in a
    random page order; returns (K_pool, V_pool, block_table [B, max_blocks] int32).  Unused pool
    rows hold a marker value; unused table entries name page 0 (never dereferenced)."""
    B, H, S, D = K.shape
    nb = (S + page_size - 1) // page_size
    g = torch.Generator().manual_seed(seed)
    num_pages = B * nb + extra_pages
    perm = torch.randperm(num_pages, generator=g)[:B * nb].reshape(B, nb).to(torch.int32)
    Kp = torch.full((num_pages, H, page_size, D + pad), 9.0, dtype=K.dtype, device=K.device)
    Vp = torch.full_like(Kp, 9.0)
    for b in range(B):
        for j in range(nb):
            r0, r1 = j * page_size, min(S, (j + 1) * page_size)
            Kp[perm[b, j], :, :r1 - r0, :D] = K[b, :, r0:r1]
            Vp[perm[b, j], :, :r1 - r0, :D] = V[b, :, r0:r1]
    table = torch.zeros((B, nb + 2), dtype=torch.int32)
    table[:, :nb] = perm
    return Kp, Vp, table.to(K.device)


def unpaginate(Kp, table, S, D):
    """The contiguous view ``[B, H, S, D]`` of a paged cache."""
    B, ps = table.shape[0], Kp.shape[2]
    nb = (S + ps - 1) // ps
    rows = Kp[table[:, :nb].long()]                       # [B, nb, H, ps, D+pad]
    return rows.permute(0, 2, 1, 3, 4).reshape(B, Kp.shape[1], nb * ps, -1)[:, :, :S, :D].contiguous()


@pytest.mark.parametrize("D,L,k,page,pad,dtype,variant", [
    (128, 128, 32, 16, 0, torch.bfloat16, 0), (128, 100, 25, 64, 0, torch.bfloat16, 0),
    (128, 512, 128, 128, 8, torch.bfloat16, 0), (128, 1024, 256, 32, 0, torch.float16, 0),
    (64, 64, 16, 16, 0, torch.bfloat16, 0), (96, 256, 64, 64, 0, torch.float16, 0), (256, 300, 75, 256, 0, torch.bfloat16, 0),
    (128, 128, 32, 32, 0, torch.bfloat16, 1), (128, 256, 64, 16, 0, torch.bfloat16, 2)])
def test_paged_prefill(binding, oracle, D, L, k, page, pad, dtype, variant):
    """Prefill from a paged cache (random page order, tiles straddling page boundaries because the
    sink is not a multiple of the tile height) equals the oracle on the contiguous cache."""
    B, H, sink = 3, 2, 20
    S = sink + 6 * L + L // 3
    K, V = synth.make_kv(B, H, S, D, seed=D + L + page, device="cuda:0", dtype=dtype)
    Kp, Vp, table = paginate(K, V, page, seed=L, pad=pad)
    plan = binding.Plan(B, H, D, sink, L, keep_k=k, variant=variant, device=0, dtype=dtype)
    ws = plan.new_workspace()
    strides = None if pad == 0 else (H * page * (D + pad), page * (D + pad), D + pad, page)
    out = plan.compress_prefill_paged(Kp, Vp, table, S, ws, want_scores=True, strides=strides)
    assert plan.read_status(ws)[0] == 0
    host = {"L_R": out["L_R"], "idx": out["idx"].cpu().numpy(), "K_out": synth.to_bits(out["K_out"]),
            "V_out": synth.to_bits(out["V_out"]), "scores": out["scores"].cpu().numpy()}
    storage = storage_of(oracle, dtype)
    if variant == 2:      # Eq. 16: relative tolerance on the norms; same picks as the contiguous call
        flat = binding.Plan(B, H, D, sink, L, keep_k=k, variant=variant, device=0, dtype=dtype)
        ref = flat.compress_prefill(K, V, ws, want_scores=True)
        assert torch.equal(ref["idx"], out["idx"]) and torch.equal(ref["K_out"], out["K_out"])
        assert torch.equal(ref["V_out"], out["V_out"]) and torch.equal(ref["scores"], out["scores"])
    else:
        check_against_oracle(oracle, synth.to_bits(K), synth.to_bits(V), sink, L, k, 1, host, variant=variant,
                             storage=storage)
    # the pools are read-only for a prefill
    Kp2, Vp2, _ = paginate(K, V, page, seed=L, pad=pad)
    assert torch.equal(Kp, Kp2) and torch.equal(Vp, Vp2)


@pytest.mark.parametrize("page,dtype", [(16, torch.bfloat16), (64, torch.float16), (1024, torch.bfloat16)])
def test_paged_prefill_warp_specialised_many_units(binding, page, dtype):
    """The warp-specialised kernel's paged twin with several slots per CTA and ranges that start
    inside a unit: rows, indices and scores are bit-identical to the contiguous call's, with and
    without the index output (positions parked in the output rows)."""
    B, H, D, sink, L, k = 8, 5, 128, 16, 256, 64
    S = sink + 21 * L + 77
    K, V = synth.make_kv(B, H, S, D, seed=page, device="cuda:0", dtype=dtype)
    Kp, Vp, table = paginate(K, V, page, seed=page + 1)
    plan = binding.Plan(B, H, D, sink, L, keep_k=k, device=0, dtype=dtype)
    assert plan.launch_info(S)["kernel"] == "lagkv_ws_kernel"
    ws = plan.new_workspace()
    ref = plan.compress_prefill(K, V, ws, want_scores=True)
    out = plan.compress_prefill_paged(Kp, Vp, table, S, ws, want_scores=True)
    assert plan.read_status(ws)[0] == 0
    for key in ("idx", "K_out", "V_out", "scores"):
        assert torch.equal(ref[key], out[key]), key
    lay = plan._paged(Kp, table, None)
    Ko = torch.full_like(ref["K_out"], -3.0)
    Vo = torch.full_like(ref["V_out"], -3.0)
    import ctypes
    rc = plan.lib.lagkv_compress_prefill_paged(plan.handle, binding._ptr(Kp), binding._ptr(Vp), ctypes.byref(lay), S,
                                               binding._ptr(Ko), binding._ptr(Vo), None, None, binding._ptr(ws),
                                               ws.numel(), binding._stream(torch.device("cuda", 0)))
    assert rc == 0 and plan.read_status(ws)[0] == 0
    assert torch.equal(Ko, ref["K_out"]) and torch.equal(Vo, ref["V_out"])


def test_paged_gather(binding, oracle):
    B, H, D, S, page = 2, 3, 128, 300, 32
    K, V = synth.make_kv(B, H, S, D, seed=44, device="cuda:0")
    Kp, Vp, table = paginate(K, V, page, seed=2)
    g = torch.Generator(device="cuda:0").manual_seed(1)
    idx = torch.randint(0, S, (B, H, 77), generator=g, device="cuda:0", dtype=torch.int32)
    plan = binding.Plan(B, H, D, 4, 64, keep_k=16, device=0)
    Ko, Vo = plan.gather_paged(Kp, Vp, table, idx, S)
    np.testing.assert_array_equal(synth.to_bits(Ko), oracle.gather(synth.to_bits(K), idx.cpu().numpy()))
    np.testing.assert_array_equal(synth.to_bits(Vo), oracle.gather(synth.to_bits(V), idx.cpu().numpy()))


def test_paged_prefill_identity_and_errors(binding, oracle):
    B, H, D, sink, L, k, page = 2, 2, 128, 8, 64, 16, 16
    S = sink + 2 * L - 1                                     # too short: identity
    K, V = synth.make_kv(B, H, S, D, seed=3, device="cuda:0")
    Kp, Vp, table = paginate(K, V, page, seed=1)
    plan = binding.Plan(B, H, D, sink, L, keep_k=k, device=0)
    ws = plan.new_workspace()
    out = plan.compress_prefill_paged(Kp, Vp, table, S, ws)
    assert out["L_R"] == S and torch.equal(out["K_out"], K) and torch.equal(out["V_out"], V)
    assert out["idx"][0, 0].tolist() == list(range(S))
    with pytest.raises(binding.LagKVError):                  # page size not a power of two
        plan.compress_prefill_paged(Kp, Vp, table, S, ws, strides=(0, 0, 0, 24))
    with pytest.raises(binding.LagKVError):                  # table too short for S_in rows
        plan.compress_prefill_paged(Kp, Vp, table[:, :2].contiguous(), S, ws)
    strided = binding.Plan(B, H, D, sink, L, keep_k=k, strides=(H * S * D, S * D, D), device=0)
    with pytest.raises(binding.LagKVError):                  # a plan with its own strides cannot take pages
        strided.compress_prefill_paged(Kp, Vp, table, S, ws)


@pytest.mark.parametrize("D,L,k,page,chunks,variant", [(128, 64, 16, 16, 3, 0), (128, 512, 128, 64, 1, 0),
                                                       (128, 96, 24, 32, 2, 0), (64, 128, 32, 128, 1, 0),
                                                       (256, 100, 10, 16, 2, 0), (128, 128, 32, 16, 2, 1),
                                                       (128, 128, 32, 64, 1, 2)])
def test_paged_append(binding, oracle, D, L, k, page, chunks, variant):
    """In-place append on a paged cache with a ragged batch (different lengths, one sequence
    skips): lengths, every valid row and the kept positions equal the oracle's replay on the
    contiguous cache; rows beyond a sequence's old length and pages of nobody stay untouched."""
    B, H, sink = 4, 3, 8
    stat = [sink, sink + 2 * k, sink + k, sink]
    seq = [stat[0] + (chunks + 1) * L + 3, stat[1] + (chunks + 1) * L, stat[2] + 2 * L + L - 1, stat[3] + 2 * L - 1]
    S = max(seq) + 5
    K, V = synth.make_kv(B, H, S, D, seed=D + L + page + chunks, device="cuda:0")
    Kp, Vp, table = paginate(K, V, page, seed=L + 1)
    Kp0, Vp0 = Kp.clone(), Vp.clone()
    plan = binding.Plan(B, H, D, sink, L, keep_k=k, variant=variant, device=0)
    ws = plan.new_workspace(chunks)
    seq_d = torch.tensor(seq, dtype=torch.int32, device="cuda:0")
    stat_d = torch.tensor(stat, dtype=torch.int32, device="cuda:0")
    idx_out = torch.full((B, H, chunks * k), -1, dtype=torch.int32, device="cuda:0")
    plan.compress_append_paged(Kp, Vp, table, seq_d, stat_d, ws, max_new_chunks=chunks, idx_out=idx_out)
    assert plan.read_status(ws)[0] == 0
    Kr, Vr, seq_r, stat_r, kept = oracle.compress_append(synth.to_bits(K), synth.to_bits(V), np.array(seq),
                                                         np.array(stat), L, k, variant=variant)
    assert seq_d.tolist() == seq_r.tolist() and stat_d.tolist() == stat_r.tolist()
    Kg, Vg = synth.to_bits(unpaginate(Kp, table, S, D)), synth.to_bits(unpaginate(Vp, table, S, D))
    Kb, Vb = synth.to_bits(K), synth.to_bits(V)
    for b in range(B):
        n = int(seq_r[b])
        np.testing.assert_array_equal(Kg[b, :, :n], Kr[b, :, :n])
        np.testing.assert_array_equal(Vg[b, :, :n], Vr[b, :, :n])
        np.testing.assert_array_equal(Kg[b, :, seq[b]:], Kb[b, :, seq[b]:])
        if kept[b].shape[1]:
            np.testing.assert_array_equal(idx_out[b, :, :kept[b].shape[1]].cpu().numpy(), kept[b])
    # pages that belong to no sequence, and the rows of a page behind the cache's end, are never written
    used = torch.zeros(Kp.shape[0], dtype=torch.bool)
    nb = (S + page - 1) // page
    used[table[:, :nb].cpu().long().flatten()] = True
    used = used.to("cuda:0")
    assert torch.equal(Kp[~used], Kp0[~used]) and torch.equal(Vp[~used], Vp0[~used])


# -------------------------------------------------------------------------------- append
def append_case(binding, oracle, B, H, D, S_cap, sink, L, k, seq, stat, max_chunks, seed, tune=None, give_idx=True,
                variant=0, dtype=torch.bfloat16):
    K, V = synth.make_kv(B, H, S_cap, D, seed=seed, device="cuda:0", dtype=dtype)
    Kb, Vb = synth.to_bits(K), synth.to_bits(V)
    seq_d = torch.tensor(seq, dtype=torch.int32, device="cuda:0")
    stat_d = torch.tensor(stat, dtype=torch.int32, device="cuda:0")
    plan = binding.Plan(B, H, D, sink, L, keep_k=k, variant=variant, device=0, dtype=dtype)
    if tune:
        plan.tune(**tune)
    ws = plan.new_workspace(max_chunks)
    idx_out = torch.full((B, H, max_chunks * k), -1, dtype=torch.int32, device="cuda:0") if give_idx else None
    plan.compress_append(K, V, seq_d, stat_d, ws, max_new_chunks=max_chunks, idx_out=idx_out)
    st = plan.read_status(ws)
    Kr, Vr, seq_r, stat_r, kept = oracle.compress_append(
        Kb, Vb, np.array(seq), np.array(stat), L, k, variant=variant,
        storage=storage_of(oracle, dtype))
    return dict(K=synth.to_bits(K), V=synth.to_bits(V), seq=seq_d.cpu().numpy(), stat=stat_d.cpu().numpy(),
                idx=None if idx_out is None else idx_out.cpu().numpy(), status=st,
                Kr=Kr, Vr=Vr, seq_r=seq_r, stat_r=stat_r, kept=kept, K0=Kb, V0=Vb)


def check_append(r, B):
    assert r["status"][0] == 0, r["status"]
    np.testing.assert_array_equal(r["seq"], r["seq_r"])
    np.testing.assert_array_equal(r["stat"], r["stat_r"])
    for b in range(B):
        n = int(r["seq_r"][b])
        np.testing.assert_array_equal(r["K"][b, :, :n], r["Kr"][b, :, :n])
        np.testing.assert_array_equal(r["V"][b, :, :n], r["Vr"][b, :, :n])
        if r["idx"] is not None and r["kept"][b].shape[1]:
            m = r["kept"][b].shape[1]
            np.testing.assert_array_equal(r["idx"][b, :, :m], r["kept"][b])


def test_append_single_chunk_ragged_batch(binding, oracle):
    """Decode-style trigger: some sequences just reached 2L of new rows, others not yet."""
    sink, L, k = 16, 128, 32
    stat = [16, 16 + 3 * k, 16, 16 + 7 * k]
    seq = [stat[0] + 2 * L, stat[1] + 2 * L + 5, stat[2] + 2 * L - 1, stat[3] + L]
    r = append_case(binding, oracle, 4, 3, 128, 1200, sink, L, k, seq, stat, 1, seed=31)
    check_append(r, 4)
    # skipped sequences are bit-identical everywhere
    np.testing.assert_array_equal(r["K"][2], r["K0"][2])
    np.testing.assert_array_equal(r["V"][3], r["V0"][3])
    # rows at and beyond the pre-call seq_len are never written
    for b in range(4):
        np.testing.assert_array_equal(r["K"][b, :, seq[b]:], r["K0"][b, :, seq[b]:])


CLUSTER = 101      # LAGKV_TUNE_APPEND_CLUSTER: 4 warps per CTA
CLUSTER8 = 102     # LAGKV_TUNE_APPEND_CLUSTER8: 8 warps per CTA (head_dim 128)


@pytest.mark.parametrize("code,splits,stages,ctas,D,L,k,dtype", [
    (CLUSTER, 1, 2, 2, 128, 64, 16, torch.bfloat16), (CLUSTER, 2, 2, 2, 128, 64, 16, torch.bfloat16),
    (CLUSTER, 4, 2, 2, 128, 72, 9, torch.bfloat16), (CLUSTER, 2, 3, 1, 128, 512, 128, torch.bfloat16),
    (CLUSTER, 4, 2, 3, 128, 512, 128, torch.float16), (CLUSTER, 1, 2, 1, 128, 512, 128, torch.bfloat16),
    (CLUSTER, 1, 2, 1, 128, 2048, 700, torch.bfloat16),     # pair of CTAs, window only partly resident
    (CLUSTER, 1, 2, 2, 128, 512, 128, torch.bfloat16),      # the same at L = 512 (two CTAs to an SM)
    (CLUSTER8, 1, 2, 1, 128, 512, 128, torch.bfloat16), (CLUSTER8, 2, 2, 1, 128, 1024, 256, torch.float16),
    (CLUSTER, 2, 2, 2, 64, 256, 64, torch.bfloat16), (CLUSTER, 4, 2, 1, 96, 200, 50, torch.float16),
    (CLUSTER, 2, 2, 1, 256, 256, 32, torch.bfloat16), (CLUSTER, 1, 2, 1, 256, 1024, 1, torch.float16),
    (CLUSTER, 2, 2, 2, 128, 37, 37, torch.bfloat16),        # k = L: nothing moves, only the lengths change
    (CLUSTER, 4, 2, 2, 128, 20, 3, torch.bfloat16),         # fewer tiles than row splits
])
def test_append_cluster_shapes(binding, oracle, code, splits, stages, ctas, D, L, k, dtype):
    """One-partition appends on every cluster shape: a ragged batch (some sequences trigger with and
    without a remainder, one skips, one asks for two partitions and is refused) against the
    oracle's replay, kept positions included."""
    sink = 8
    stat = [sink, sink + 3 * k, sink + k, sink, sink + 2 * k]
    seq = [stat[0] + 2 * L, stat[1] + 2 * L + L - 1, stat[2] + 2 * L + 5, stat[3] + 2 * L - 1, stat[4] + 3 * L]
    S_cap = max(seq) + 7
    B, H = 5, 3
    r = append_case(binding, oracle, B, H, D, S_cap, sink, L, k, seq, stat, 1, seed=L + k + splits, dtype=dtype,
                    tune=dict(warps=code, tile_rows=splits, stages=stages, ctas_per_sm=ctas))
    assert r["status"][0] == binding.LAGKV_ECAPACITY          # the last sequence needs two partitions
    for b in range(4):
        n = int(r["seq_r"][b])
        assert r["seq"][b] == r["seq_r"][b] and r["stat"][b] == r["stat_r"][b]
        np.testing.assert_array_equal(r["K"][b, :, :n], r["Kr"][b, :, :n])
        np.testing.assert_array_equal(r["V"][b, :, :n], r["Vr"][b, :, :n])
        np.testing.assert_array_equal(r["K"][b, :, seq[b]:], r["K0"][b, :, seq[b]:])     # nothing beyond the old length
        if r["kept"][b].shape[1]:
            np.testing.assert_array_equal(r["idx"][b, :, :k], r["kept"][b])
    assert r["seq"][3] == seq[3] and r["seq"][4] == seq[4] and r["stat"][4] == stat[4]
    np.testing.assert_array_equal(r["K"][3:], r["K0"][3:])
    np.testing.assert_array_equal(r["V"][3:], r["V0"][3:])


@pytest.mark.parametrize("splits,layout", [(1, "padded"), (2, "bshd"), (4, "padded")])
def test_append_cluster_strided(binding, oracle, splits, layout):
    """Cluster appends on caches whose rows are not contiguous: row-by-row copies everywhere."""
    B, H, D, sink, L, k = 3, 2, 128, 4, 96, 24
    stat = [sink, sink + k, sink]
    seq = [stat[0] + 2 * L + 11, stat[1] + 2 * L, stat[2] + L]
    S_cap = max(seq) + 3
    K, V = synth.make_kv(B, H, S_cap, D, seed=5 + splits, device="cuda:0")
    Kb, Vb = synth.to_bits(K), synth.to_bits(V)
    if layout == "bshd":
        Kd = K.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
        Vd = V.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
        strides = (S_cap * H * D, D, H * D)
    else:
        Kp = torch.zeros((B, H, S_cap, D + 8), dtype=torch.bfloat16, device="cuda:0")
        Vp = torch.zeros_like(Kp)
        Kp[..., :D], Vp[..., :D] = K, V
        Kd, Vd = Kp[..., :D], Vp[..., :D]
        strides = (H * S_cap * (D + 8), S_cap * (D + 8), D + 8)
    plan = binding.Plan(B, H, D, sink, L, keep_k=k, strides=strides, device=0)
    plan.tune(warps=CLUSTER, tile_rows=splits, stages=2, ctas_per_sm=2)
    ws = plan.new_workspace(1)
    seq_d = torch.tensor(seq, dtype=torch.int32, device="cuda:0")
    stat_d = torch.tensor(stat, dtype=torch.int32, device="cuda:0")
    plan.compress_append(Kd, Vd, seq_d, stat_d, ws, max_new_chunks=1)
    assert plan.read_status(ws)[0] == 0
    Kr, Vr, seq_r, stat_r, _ = oracle.compress_append(Kb, Vb, np.array(seq), np.array(stat), L, k)
    assert seq_d.tolist() == seq_r.tolist() and stat_d.tolist() == stat_r.tolist()
    Kg, Vg = synth.to_bits(Kd.contiguous()), synth.to_bits(Vd.contiguous())
    for b in range(B):
        n = int(seq_r[b])
        np.testing.assert_array_equal(Kg[b, :, :n], Kr[b, :, :n])
        np.testing.assert_array_equal(Vg[b, :, :n], Vr[b, :, :n])


@pytest.mark.parametrize("L,k,chunks", [(64, 16, 4), (96, 96, 2), (256, 1, 3), (512, 128, 2)])
def test_append_multi_chunk(binding, oracle, L, k, chunks):
    sink = 8
    stat = [sink, sink + 2 * k]
    seq = [stat[0] + (chunks + 1) * L + 3, stat[1] + (chunks + 1) * L + L - 1]
    r = append_case(binding, oracle, 2, 2, 128, seq[1] + 9, sink, L, k, seq, stat, chunks, seed=L + k,
                    give_idx=(L != 96))
    check_append(r, 2)


def test_ragged_batch_prefill_in_place(binding, oracle):
    """A batch of prompts of different lengths, compressed in place through the append entry
    point with static_len = sink: every sequence equals its own one-shot prefill (Eq. 7-12)."""
    sink, L, k, H, D = 16, 128, 32, 3, 128
    seq = [sink + 9 * L + 77, sink + 2 * L, sink + 2 * L - 1, sink + 5 * L, 40, sink + 12 * L + 127]
    B, S_cap = len(seq), max(seq) + 5
    K, V = synth.make_kv(B, H, S_cap, D, seed=77, device="cuda:0")
    Kb, Vb = synth.to_bits(K), synth.to_bits(V)
    seq_d = torch.tensor(seq, dtype=torch.int32, device="cuda:0")
    stat_d = torch.full((B,), sink, dtype=torch.int32, device="cuda:0")
    plan = binding.Plan(B, H, D, sink, L, keep_k=k, device=0)
    chunks = max((s - sink) // L - 1 for s in seq)
    ws = plan.new_workspace(chunks)
    idx_out = torch.full((B, H, chunks * k), -1, dtype=torch.int32, device="cuda:0")
    plan.compress_append(K, V, seq_d, stat_d, ws, max_new_chunks=chunks, idx_out=idx_out)
    assert plan.read_status(ws)[0] == 0
    Kn, Vn, idx = synth.to_bits(K), synth.to_bits(V), idx_out.cpu().numpy()
    for b in range(B):
        ref = oracle.compress(Kb[b:b + 1, :, :seq[b]], Vb[b:b + 1, :, :seq[b]], sink, L, k)
        L_R, n_c = ref["L_R"], ref["n_c"]
        assert int(seq_d[b]) == L_R and int(stat_d[b]) == sink + n_c * k
        mism = 0
        for h in range(H):
            got = idx[b, h, :n_c * k]
            want = ref["idx"][0, h, sink:sink + n_c * k]
            mism += int((got != want).any())
            src = np.concatenate([np.arange(sink), got, ref["idx"][0, h, sink + n_c * k:]]).astype(np.int64)
            np.testing.assert_array_equal(Kn[b, h, :L_R], Kb[b, h, src])
            np.testing.assert_array_equal(Vn[b, h, :L_R], Vb[b, h, src])
            assert np.all(idx[b, h, n_c * k:] == -1)
        assert mism == 0, f"sequence {b}: {mism} heads differ from the one-shot oracle"
        np.testing.assert_array_equal(Kn[b, :, seq[b]:], Kb[b, :, seq[b]:])


@pytest.mark.parametrize("layout", ["padded", "bshd"])
@pytest.mark.parametrize("L,k,chunks", [(96, 24, 2), (512, 128, 1)])
def test_append_strided_caches(binding, oracle, layout, L, k, chunks):
    """In-place append on caches whose rows are not contiguous: rows padded to D + 8 elements,
    and a [B, S, H, D] cache; the bytes outside the rows (the padding) stay untouched."""
    B, H, D, sink = 2, 3, 128, 8
    stat = [sink, sink + 2 * k]
    seq = [stat[0] + (chunks + 1) * L + 3, stat[1] + (chunks + 1) * L]
    S_cap = max(seq) + 9
    K, V = synth.make_kv(B, H, S_cap, D, seed=L + len(layout), device="cuda:0")
    Kb, Vb = synth.to_bits(K), synth.to_bits(V)
    if layout == "padded":
        Ks = torch.full((B, H, S_cap, D + 8), 7.0, dtype=torch.bfloat16, device="cuda:0")
        Vs = torch.full_like(Ks, 7.0)
        Ks[..., :D], Vs[..., :D] = K, V
        strides = (H * S_cap * (D + 8), S_cap * (D + 8), D + 8)
        view = lambda t: t[..., :D]
    else:
        Ks, Vs = K.permute(0, 2, 1, 3).contiguous(), V.permute(0, 2, 1, 3).contiguous()     # [B, S, H, D]
        strides = (S_cap * H * D, D, H * D)
        view = lambda t: t.permute(0, 2, 1, 3)
    seq_d = torch.tensor(seq, dtype=torch.int32, device="cuda:0")
    stat_d = torch.tensor(stat, dtype=torch.int32, device="cuda:0")
    plan = binding.Plan(B, H, D, sink, L, keep_k=k, strides=strides, device=0)
    ws = plan.new_workspace(chunks)
    rc = plan.lib.lagkv_compress_append(plan.handle, binding._ptr(Ks), binding._ptr(Vs), S_cap, binding._ptr(seq_d),
                                        binding._ptr(stat_d), chunks, None, None, binding._ptr(ws), ws.numel(),
                                        binding._stream(torch.device("cuda", 0)))
    assert rc == 0 and plan.read_status(ws)[0] == 0
    Kr, Vr, seq_r, stat_r, _ = oracle.compress_append(Kb, Vb, np.array(seq), np.array(stat), L, k)
    np.testing.assert_array_equal(seq_d.cpu().numpy(), seq_r)
    np.testing.assert_array_equal(stat_d.cpu().numpy(), stat_r)
    Kn, Vn = synth.to_bits(view(Ks).contiguous()), synth.to_bits(view(Vs).contiguous())
    for b in range(B):
        n = int(seq_r[b])
        np.testing.assert_array_equal(Kn[b, :, :n], Kr[b, :, :n])
        np.testing.assert_array_equal(Vn[b, :, :n], Vr[b, :, :n])
        np.testing.assert_array_equal(Kn[b, :, seq[b]:], Kb[b, :, seq[b]:])      # beyond the old length: untouched
    if layout == "padded":
        assert bool((Ks[..., D:] == 7.0).all()) and bool((Vs[..., D:] == 7.0).all())


def test_append_replays_from_a_cuda_graph(binding, oracle):
    """Decode loop: one captured launch, replayed after every appended token.  Which sequences
    compress is decided on the device from the lengths, so the graph never changes; the caches
    and lengths follow the oracle's token-by-token bookkeeping exactly."""
    B, H, D, sink, L, k, steps = 3, 2, 128, 8, 64, 16, 150
    S_cap = sink + 3 * L + 8
    seq0 = [sink + L + 5, sink + 2 * L - 1, 10]
    fresh_K, fresh_V = synth.make_kv(B, H, steps, D, seed=401, device="cuda:0")
    K, V = synth.make_kv(B, H, S_cap, D, seed=400, device="cuda:0")
    Kc, Vc = synth.to_bits(K), synth.to_bits(V)
    fK, fV = synth.to_bits(fresh_K), synth.to_bits(fresh_V)
    seq_ref, stat_ref = np.array(seq0, dtype=np.int64), np.full(B, sink, dtype=np.int64)
    seq = torch.tensor(seq0, dtype=torch.int32, device="cuda:0")
    stat = torch.full((B,), sink, dtype=torch.int32, device="cuda:0")
    plan = binding.Plan(B, H, D, sink, L, keep_k=k, device=0)
    ws = plan.new_workspace(1)
    bidx = torch.arange(B, device="cuda:0")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        plan.compress_append(K, V, seq, stat, ws, max_new_chunks=1)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(synth.to_bits(K), Kc)             # capturing ran nothing
    triggers = 0
    for t in range(steps):
        K[bidx, :, seq.long()] = fresh_K[:, :, t]                   # the model writes one new row per sequence
        V[bidx, :, seq.long()] = fresh_V[:, :, t]
        seq += 1
        graph.replay()
        for b in range(B):
            Kc[b, :, seq_ref[b]], Vc[b, :, seq_ref[b]] = fK[b, :, t], fV[b, :, t]
        seq_ref += 1
        triggers += int(((seq_ref - stat_ref) >= 2 * L).sum())
        Kc, Vc, seq_ref, stat_ref, _ = oracle.compress_append(Kc, Vc, seq_ref, stat_ref, L, k)
    torch.cuda.synchronize()
    assert plan.read_status(ws)[0] == 0 and triggers >= 5
    np.testing.assert_array_equal(seq.cpu().numpy(), seq_ref)
    np.testing.assert_array_equal(stat.cpu().numpy(), stat_ref)
    Kn, Vn = synth.to_bits(K), synth.to_bits(V)
    for b in range(B):
        n = int(seq_ref[b])
        np.testing.assert_array_equal(Kn[b, :, :n], Kc[b, :, :n])
        np.testing.assert_array_equal(Vn[b, :, :n], Vc[b, :, :n])


@pytest.mark.parametrize("variant", [1, 2])
@pytest.mark.parametrize("L,k,chunks", [(64, 16, 4), (256, 32, 3), (512, 128, 1)])
def test_append_variants(binding, oracle, variant, L, k, chunks):
    """LocalKV and L2-norm scoring in the incremental pass, ragged batch with a skipped sequence."""
    sink = 8
    stat = [sink, sink + 2 * k, sink]
    seq = [stat[0] + (chunks + 1) * L + 3, stat[1] + (chunks + 1) * L + L - 1, stat[2] + 2 * L - 1]
    r = append_case(binding, oracle, 3, 2, 128, seq[1] + 9, sink, L, k, seq, stat, chunks, seed=L + k + variant,
                    variant=variant)
    check_append(r, 3)
    np.testing.assert_array_equal(r["K"][2], r["K0"][2])


@pytest.mark.parametrize("variant", [1, 2])
def test_prefill_equals_incremental_variants(binding, variant):
    """Per variant: one-shot prefill (warp-specialised kernel) and block-wise appends (uniform
    kernel) end with the same cache, bit for bit."""
    B, H, D, sink, L, k = 2, 2, 128, 4, 256, 64
    total = sink + 2 * L + 3 * L + 11
    K, V = synth.make_kv(B, H, total, D, seed=52 + variant, device="cuda:0")
    plan = binding.Plan(B, H, D, sink, L, keep_k=k, variant=variant, device=0)
    assert plan.launch_info(total)["block"] == 384
    ws = plan.new_workspace(1)
    one = plan.compress_prefill(K, V, ws)
    Kc = torch.zeros((B, H, total, D), dtype=torch.bfloat16, device="cuda:0")
    Vc = torch.zeros_like(Kc)
    seq = torch.zeros((B,), dtype=torch.int32, device="cuda:0")
    stat = torch.full((B,), sink, dtype=torch.int32, device="cuda:0")
    pos = 0
    for step in [sink + 2 * L, 100, 156, 256, 200, 56 + 11]:
        s = int(seq[0])
        Kc[:, :, s:s + step], Vc[:, :, s:s + step] = K[:, :, pos:pos + step], V[:, :, pos:pos + step]
        seq += step
        pos += step
        plan.compress_append(Kc, Vc, seq, stat, ws, max_new_chunks=1)
    assert pos == total and plan.read_status(ws)[0] == 0
    assert seq.tolist() == [one["L_R"]] * B
    assert torch.equal(Kc[:, :, :one["L_R"]], one["K_out"]) and torch.equal(Vc[:, :, :one["L_R"]], one["V_out"])


@pytest.mark.parametrize("D", [64, 96, 256])
def test_append_head_dims(binding, oracle, D):
    sink, L, k = 8, 96, 24
    stat = [sink, sink + 3 * k]
    seq = [stat[0] + 3 * L + 3, stat[1] + 2 * L]
    r = append_case(binding, oracle, 2, 3, D, seq[0] + 9, sink, L, k, seq, stat, 2, seed=D)
    check_append(r, 2)


def test_append_capacity_error_leaves_sequence_alone(binding, oracle):
    sink, L, k = 4, 64, 16
    stat, seq = [4, 4], [4 + 2 * L, 4 + 4 * L]      # second sequence needs 3 chunks
    r = append_case(binding, oracle, 2, 2, 128, 300, sink, L, k, seq, stat, 1, seed=41)
    assert r["status"][0] == binding.LAGKV_ECAPACITY and r["status"][1] == 1
    np.testing.assert_array_equal(r["K"][1], r["K0"][1])
    assert r["seq"][1] == seq[1] and r["stat"][1] == stat[1]
    assert r["seq"][0] == r["seq_r"][0]
    np.testing.assert_array_equal(r["K"][0, :, :r["seq"][0]], r["Kr"][0, :, :r["seq"][0]])


def test_prefill_equals_incremental_on_gpu(binding, oracle):
    """One-shot prefill == prefill of S+2L rows followed by token-by-token appends with an
    append call after every token (most calls skip on the device)."""
    B, H, D, sink, L, k = 2, 2, 128, 4, 32, 8
    total = sink + 2 * L + 3 * L + 11
    K, V = synth.make_kv(B, H, total, D, seed=51, device="cuda:0")
    plan = binding.Plan(B, H, D, sink, L, keep_k=k, device=0)
    ws = plan.new_workspace(1)
    one = plan.compress_prefill(K, V, ws)
    Kc = torch.zeros((B, H, total, D), dtype=torch.bfloat16, device="cuda:0")
    Vc = torch.zeros_like(Kc)
    first = sink + 2 * L
    Kc[:, :, :first], Vc[:, :, :first] = K[:, :, :first], V[:, :, :first]
    seq = torch.full((B,), first, dtype=torch.int32, device="cuda:0")
    stat = torch.full((B,), sink, dtype=torch.int32, device="cuda:0")
    plan.compress_append(Kc, Vc, seq, stat, ws, max_new_chunks=1)
    for t in range(first, total):
        s = int(seq[0])
        Kc[:, :, s], Vc[:, :, s] = K[:, :, t], V[:, :, t]
        seq += 1
        plan.compress_append(Kc, Vc, seq, stat, ws, max_new_chunks=1)
    assert plan.read_status(ws)[0] == 0
    assert seq.tolist() == [one["L_R"]] * B
    assert stat.tolist() == [sink + 4 * k] * B
    assert torch.equal(Kc[:, :, :one["L_R"]], one["K_out"])
    assert torch.equal(Vc[:, :, :one["L_R"]], one["V_out"])


def test_chunked_prefill_driver_equals_one_shot(binding, oracle):
    """Chunk-by-chunk prefill (first S + 2L tokens, then L per step) ends with the same cache as
    one pass over the whole prompt, and with the oracle's."""
    B, H, D, sink, L, k = 2, 3, 128, 16, 128, 32
    total = sink + 2 * L + 5 * L + 77
    K, V = synth.make_kv(B, H, total, D, seed=61, device="cuda:0")
    drv = binding.ChunkedPrefill(B, H, D, sink, L, keep_k=k, device=0)
    drv.feed(K[:, :, :drv.first], V[:, :, :drv.first])
    pos = drv.first
    while pos < total:
        t = min(drv.step, total - pos)
        drv.feed(K[:, :, pos:pos + t], V[:, :, pos:pos + t])
        pos += t
        assert drv.rows <= sink + 3 * L + 6 * k            # the cache stays short all along
    assert drv.plan.read_status(drv.ws)[0] == 0
    ref = oracle.compress(synth.to_bits(K), synth.to_bits(V), sink, L, k)
    assert drv.rows == ref["L_R"] and drv.seq_len.tolist() == [ref["L_R"]] * B
    assert drv.static_len.tolist() == [drv.static] * B
    np.testing.assert_array_equal(synth.to_bits(drv.K[:, :, :drv.rows]), ref["K_out"])
    np.testing.assert_array_equal(synth.to_bits(drv.V[:, :, :drv.rows]), ref["V_out"])


@pytest.mark.parametrize("warps,L,k", [(0, 64, 16), (12, 256, 64), (100, 128, 16), (12, 2048, 256)])
def test_no_write_outside_the_output_buffers(binding, warps, L, k):
    """Guard zones before and after every output (rows, indices, scores) and around the
    workspace stay untouched; the inputs are not modified."""
    B, H, D, sink = 3, 2, 128, 8
    S = sink + 5 * L + L // 3
    K, V = synth.make_kv(B, H, S, D, seed=91, device="cuda:0")
    K0, V0 = K.clone(), V.clone()
    plan = binding.Plan(B, H, D, sink, L, keep_k=k, device=0)
    if warps:
        plan.tune(warps=warps, tile_rows=32, stages=2, ctas_per_sm=1)
    L_R, n_c, G = plan.compressed_len(S), (S - sink) // L - 1, 4096

    def guarded(numel, dtype, fill):
        buf = torch.full((numel + 2 * G,), fill, dtype=dtype, device="cuda:0")
        return buf, buf[G:G + numel]

    kb, ko = guarded(B * H * L_R * D, torch.bfloat16, 7.0)
    vb, vo = guarded(B * H * L_R * D, torch.bfloat16, 7.0)
    ib, io = guarded(B * H * L_R, torch.int32, -5)
    sb, so = guarded(B * H * n_c * L, torch.float32, -3.0)
    wb, wo = guarded(plan.workspace_bytes(), torch.uint8, 0)
    wb[:G] = 9
    wb[G + wo.numel():] = 9
    out = {"K_out": ko.view(B, H, L_R, D), "V_out": vo.view(B, H, L_R, D), "idx": io.view(B, H, L_R),
           "scores": so.view(B, H, n_c, L)}
    plan.compress_prefill(K, V, wo, out=out, want_scores=True)
    assert plan.read_status(wo)[0] == 0
    for buf, inner, fill in ((kb, ko, 7.0), (vb, vo, 7.0), (ib, io, -5), (sb, so, -3.0), (wb, wo, 9)):
        assert bool((buf[:G] == fill).all()) and bool((buf[G + inner.numel():] == fill).all())
    assert torch.equal(K, K0) and torch.equal(V, V0)
    take = out["idx"].long().unsqueeze(-1).expand(-1, -1, -1, D)
    assert torch.equal(out["K_out"], torch.gather(K, 2, take)) and torch.equal(out["V_out"], torch.gather(V, 2, take))


def test_append_state_is_cache_plus_two_lengths(binding):
    """Checkpoint / resume: the pass keeps no hidden state.  Copying (K, V, seq_len, static_len)
    after some appends and resuming on the copy with a new plan and workspace gives, bit for
    bit, what the uninterrupted run gives."""
    B, H, D, sink, L, k = 2, 2, 128, 4, 64, 16
    total = sink + 9 * L + 20
    Ksrc, Vsrc = synth.make_kv(B, H, total, D, seed=93, device="cuda:0")

    def feed(plan, ws, Kc, Vc, seq, stat, lo, hi, step=37):
        for pos in range(lo, hi, step):
            t = min(step, hi - pos)
            s = int(seq[0])
            Kc[:, :, s:s + t], Vc[:, :, s:s + t] = Ksrc[:, :, pos:pos + t], Vsrc[:, :, pos:pos + t]
            seq += t
            plan.compress_append(Kc, Vc, seq, stat, ws, max_new_chunks=1)

    def fresh():
        plan = binding.Plan(B, H, D, sink, L, keep_k=k, device=0)
        return plan, plan.new_workspace(1)

    Kc = torch.zeros((B, H, sink + 8 * k + 3 * L, D), dtype=torch.bfloat16, device="cuda:0")   # stored rows grow by k per partition
    Vc = torch.zeros_like(Kc)
    seq = torch.zeros((B,), dtype=torch.int32, device="cuda:0")
    stat = torch.full((B,), sink, dtype=torch.int32, device="cuda:0")
    plan, ws = fresh()
    half = sink + 4 * L + 11
    feed(plan, ws, Kc, Vc, seq, stat, 0, half)
    snap = [t.clone() for t in (Kc, Vc, seq, stat)]
    feed(plan, ws, Kc, Vc, seq, stat, half, total)
    plan2, ws2 = fresh()
    feed(plan2, ws2, *snap, half, total)
    assert plan.read_status(ws)[0] == 0 and plan2.read_status(ws2)[0] == 0
    for a, b in zip((Kc, Vc, seq, stat), snap):
        assert torch.equal(a, b)
    assert int(stat[0]) == sink + 8 * k


def test_append_writes_nothing_beyond_the_valid_rows(binding):
    """In-place append: rows at and beyond the pre-call length, other sequences' skipped caches
    and guard zones around the length arrays stay untouched."""
    B, H, D, sink, L, k = 3, 2, 128, 8, 128, 32
    S_cap = sink + 4 * L
    K, V = synth.make_kv(B, H, S_cap, D, seed=92, device="cuda:0")
    K0, V0 = K.clone(), V.clone()
    lens = torch.full((64,), -9, dtype=torch.int32, device="cuda:0")
    seq, stat = lens[16:16 + B], lens[40:40 + B]
    seq.copy_(torch.tensor([sink + 3 * L + 5, sink + 2 * L - 1, sink + 2 * L]))
    stat.fill_(sink)
    seq0 = seq.clone()
    plan = binding.Plan(B, H, D, sink, L, keep_k=k, device=0)
    ws = plan.new_workspace(2)
    plan.compress_append(K, V, seq, stat, ws, max_new_chunks=2)
    assert plan.read_status(ws)[0] == 0
    assert seq.tolist() == [sink + 2 * k + L + 5, sink + 2 * L - 1, sink + k + L]
    for b in range(B):
        n0 = int(seq0[b])
        assert torch.equal(K[b, :, n0:], K0[b, :, n0:]) and torch.equal(V[b, :, n0:], V0[b, :, n0:])
    assert torch.equal(K[1], K0[1]) and torch.equal(V[1], V0[1])           # the skipped sequence
    keep = torch.ones(64, dtype=torch.bool, device="cuda:0")
    keep[16:16 + B] = False
    keep[40:40 + B] = False
    assert bool((lens[keep] == -9).all())


def test_host_prefill_pipeline_matches_direct_call(binding, oracle):
    """The host end-to-end path (pinned host cache -> device chunks -> compress -> compacted rows
    and indices back on the host, three streams, two staging slots) returns what one direct
    call on the whole cache returns, and what the oracle says."""
    B, H, D, sink, L, k = 6, 2, 128, 16, 256, 64
    S = sink + 5 * L + 70
    K, V = synth.make_kv(B, H, S, D, seed=71, device="cuda:0")
    hp = binding.HostPrefill(B, H, D, S, sink, L, keep_k=k, chunk_B=2, device=0)
    Kh, Vh = K.cpu().pin_memory(), V.cpu().pin_memory()
    Ko = torch.zeros((B, H, hp.L_R, D), dtype=torch.bfloat16).pin_memory()
    Vo = torch.zeros_like(Ko).pin_memory()
    Io = torch.zeros((B, H, hp.L_R), dtype=torch.int32).pin_memory()
    for _ in range(2):                                       # the second run reuses both slots
        hp.run(Kh, Vh, Ko, Vo, Io)
    torch.cuda.synchronize()
    assert hp.h2d_bytes == 2 * K.numel() * 2 and hp.d2h_bytes == 2 * Ko.numel() * 2 + Io.numel() * 4
    plan = binding.Plan(B, H, D, sink, L, keep_k=k, device=0)
    direct = plan.compress_prefill(K, V, plan.new_workspace())
    assert torch.equal(Io, direct["idx"].cpu()) and torch.equal(Ko, direct["K_out"].cpu())
    assert torch.equal(Vo, direct["V_out"].cpu())
    ref = oracle.compress(synth.to_bits(K), synth.to_bits(V), sink, L, k)
    np.testing.assert_array_equal(Io.numpy(), ref["idx"])
    np.testing.assert_array_equal(synth.to_bits(Ko), ref["K_out"])
    assert hp.plan.read_status(hp.ws)[0] == 0
    # one chunk only, and a cache too short to compress (identity), through the same entry point
    for chunk_B, S2 in ((B, S), (3, sink + 2 * L - 1)):
        hp2 = binding.HostPrefill(B, H, D, S2, sink, L, keep_k=k, chunk_B=chunk_B, device=0)
        Kh2, Vh2 = Kh[:, :, :S2].contiguous().pin_memory(), Vh[:, :, :S2].contiguous().pin_memory()
        Ko2 = torch.zeros((B, H, hp2.L_R, D), dtype=torch.bfloat16).pin_memory()
        Vo2, Io2 = torch.zeros_like(Ko2).pin_memory(), torch.zeros((B, H, hp2.L_R), dtype=torch.int32).pin_memory()
        hp2.run(Kh2, Vh2, Ko2, Vo2, Io2)
        ref2 = oracle.compress(synth.to_bits(Kh2), synth.to_bits(Vh2), sink, L, k)
        np.testing.assert_array_equal(Io2.numpy(), ref2["idx"])
        np.testing.assert_array_equal(synth.to_bits(Ko2), ref2["K_out"])
        np.testing.assert_array_equal(synth.to_bits(Vo2), ref2["V_out"])
    # a staging buffer that is too small is refused before anything is enqueued
    rc = hp.plan.lib.lagkv_compress_prefill_host(
        hp.plan.handle, binding._ptr(Kh), binding._ptr(Vh), S, binding._ptr(Ko), binding._ptr(Vo), binding._ptr(Io), 2,
        binding._ptr(hp.staging), hp.staging.numel() - 256, binding._ptr(hp.ws), hp.ws.numel(),
        binding._stream(torch.device("cuda", 0)))
    assert rc == binding.LAGKV_EWORKSPACE
    assert hp.plan.lib.lagkv_host_staging_bytes(hp.plan.handle, S, B + 1) == 0      # more than the plan holds


def test_bounded_wait_gives_up_and_reports(binding):
    """Failure path without a fault: a wait on a barrier that nothing completes runs out after
    its limit, the status block says LAGKV_ETIMEOUT, and the same context goes on working."""
    import time
    plan = binding.Plan(1, 2, 128, 4, 64, keep_k=16, device=0)
    ws = plan.new_workspace()
    t0 = time.perf_counter()
    plan.selftest_bounded_wait(ws, limit_ms=50)
    st = plan.read_status(ws)
    dt = time.perf_counter() - t0
    assert st[0] == binding.LAGKV_ETIMEOUT and st[1] == -1
    assert 0.04 < dt < 1.0
    assert plan.read_status(ws)[0] == 0                      # reading cleared it
    K, V = synth.make_kv(1, 2, 4 + 3 * 64, 128, seed=2, device="cuda:0")
    out = plan.compress_prefill(K, V, ws)                    # the context is still usable
    assert plan.read_status(ws)[0] == 0 and out["L_R"] == 4 + 2 * 16 + 64


def test_plans_do_not_lower_each_others_limits(binding, oracle):
    """The dynamic shared memory limit is a property of the kernel function: a later plan that
    needs less (shorter partitions, shallower rings) must not stop an earlier plan's launches."""
    B, H, D, sink = 1, 2, 128, 16
    big = binding.Plan(B, H, D, sink, 2048, keep_k=256, device=0)
    small = binding.Plan(B, H, D, sink, 256, keep_k=64, device=0)          # same kernel, less shared memory
    for plan, L, k in ((big, 2048, 256), (small, 256, 64), (big, 2048, 256)):
        S = sink + 3 * L + 50
        K, V = synth.make_kv(B, H, S, D, seed=L, device="cuda:0")
        ws = plan.new_workspace()
        out = plan.compress_prefill(K, V, ws)
        assert plan.read_status(ws)[0] == 0
        ref = oracle.compress(synth.to_bits(K), synth.to_bits(V), sink, L, k, want_scores=False)
        np.testing.assert_array_equal(synth.to_bits(out["K_out"]), np.take_along_axis(
            synth.to_bits(K), out["idx"].cpu().numpy()[..., None].astype(np.int64), axis=2))
        assert out["L_R"] == ref["L_R"]
    # appends (three-stage rings) after a prefill plan of the same kernel with two stages
    a = binding.Plan(2, 2, D, 8, 96, keep_k=24, device=0)
    binding.Plan(2, 2, D, 8, 64, keep_k=16, device=0)
    Kc, Vc = synth.make_kv(2, 2, 8 + 3 * 96 + 20, D, seed=3, device="cuda:0")
    seq = torch.tensor([8 + 2 * 96 + 5, 8 + 3 * 96], dtype=torch.int32, device="cuda:0")
    stat = torch.full((2,), 8, dtype=torch.int32, device="cuda:0")
    wsa = a.new_workspace(2)
    a.compress_append(Kc, Vc, seq, stat, wsa, max_new_chunks=2)
    assert a.read_status(wsa)[0] == 0 and stat.tolist() == [8 + 24, 8 + 48]


# ----------------------------------------------------------------------- argument checks
def test_argument_errors(binding):
    with pytest.raises(binding.LagKVError) as e:
        binding.Plan(1, 1, 80, 4, 64, device=0)
    assert e.value.code == binding.LAGKV_EUNSUPPORTED
    with pytest.raises(binding.LagKVError) as e:
        binding.Plan(1, 1, 128, 4, 1, device=0)
    assert e.value.code == binding.LAGKV_EINVAL
    plan = binding.Plan(1, 2, 128, 4, 64, keep_k=16, device=0)
    K, V = synth.make_kv(1, 2, 300, 128, seed=1, device="cuda:0")
    small = torch.empty(16, dtype=torch.uint8, device="cuda:0")
    with pytest.raises(binding.LagKVError) as e:
        plan.compress_prefill(K, V, small)
    assert e.value.code == binding.LAGKV_EWORKSPACE
    ws = plan.new_workspace()
    with pytest.raises(binding.LagKVError) as e:      # misaligned cache pointer
        plan.compress_prefill(K.view(-1)[1:1 + 2 * 299 * 128].view(1, 2, 299, 128), V, ws, S_in=299)
    assert e.value.code == binding.LAGKV_EINVAL
    with pytest.raises(binding.LagKVError) as e:      # output aliases input
        plan.compress_prefill(K, V, ws, out={"K_out": K, "V_out": V})
    assert e.value.code == binding.LAGKV_EINVAL
    assert plan.read_status(ws)[0] == 0


def test_c_program_prefill_parity(binding, tmp_path):
    """No Python between the library and the oracle: a C program (tests/c_abi/prefill_parity.c)
    allocates with the CUDA runtime, calls the C ABI, and compares with the C oracle linked in."""
    import os
    import subprocess
    from pathlib import Path
    root = Path(__file__).resolve().parent.parent
    lib = Path(binding.LIB_PATH)
    cuda = Path(os.environ.get("CUDA_HOME", "/usr/local/cuda"))
    exe = tmp_path / "prefill_parity"
    subprocess.run(["gcc", "-std=c99", "-O2", "-Wall", "-Werror", "-fopenmp", f"-I{root / 'include'}", f"-I{cuda / 'include'}",
                    str(root / "tests" / "c_abi" / "prefill_parity.c"), str(root / "oracle" / "lagkv_oracle.c"),
                    "-o", str(exe), f"-L{lib.parent}", f"-l:{lib.name}", f"-Wl,-rpath,{lib.parent}",
                    f"-L{cuda / 'lib64'}", "-lcudart", f"-Wl,-rpath,{cuda / 'lib64'}", "-lm"], check=True)
    out = subprocess.run([str(exe)], capture_output=True, text=True)
    assert out.returncode == 0 and out.stdout.startswith("ok"), out.stdout + out.stderr


# ------------------------------------------------------------------------------- fp8 caches
FP8 = torch.float8_e4m3fn


@pytest.mark.parametrize("L,k,S_extra,tune,variant", [
    (64, 16, 60, None, 0), (100, 25, 7, None, 0), (128, 16, 100, dict(warps=100, tile_rows=32, stages=2, ctas_per_sm=1), 0),
    (128, 32, 0, dict(warps=100, tile_rows=16, stages=2, ctas_per_sm=1), 0), (256, 64, 255, None, 0), (512, 128, 3, dict(warps=12, tile_rows=16), 0),
    (1024, 256, 1008, None, 0), (2048, 256, 100, dict(warps=8, tile_rows=32, stages=3, ctas_per_sm=1), 0),
    (256, 1, 17, dict(warps=4, tile_rows=32, stages=3, ctas_per_sm=2), 0), (37, 5, 36, None, 0),
    (128, 32, 11, None, 1), (512, 128, 100, None, 1), (300, 75, 7, None, 2)])
def test_fp8_prefill(binding, oracle, L, k, S_extra, tune, variant):
    """fp8 (e4m3) caches through every kernel family and scoring variant: scores within the fp32
    bars of the oracle's reading of the same bytes, picks exact or explained, rows byte for byte."""
    n = 5 if L >= 512 else 9
    if variant == 2:
        run_l2norm(binding, oracle, 2, 3, 128, 4 + n * L + S_extra, 4, L, k, seed=L + 3, tune=tune, dtype=FP8)
    else:
        run_prefill(binding, oracle, 2, 3, 128, 4 + n * L + S_extra, 4, L, k, seed=L + k, tune=tune, variant=variant,
                    dtype=FP8)


def test_fp8_many_units_rows_only_and_paged(binding, oracle):
    """fp8 on the warp-specialised kernel with several slots per CTA: the run without indices (parked
    positions) and the run on a paged copy of the cache give the same bytes as the checked run."""
    B, H, D, sink, L, k = 8, 5, 128, 16, 256, 64
    S = sink + 21 * L + 77
    K, V = synth.make_kv(B, H, S, D, seed=88, device="cuda:0", dtype=FP8)
    plan = binding.Plan(B, H, D, sink, L, keep_k=k, device=0, dtype=FP8)
    assert plan.launch_info(S)["kernel"] == "lagkv_ws_kernel"
    ws = plan.new_workspace()
    full = plan.compress_prefill(K, V, ws, want_scores=True)
    host = {"L_R": full["L_R"], "idx": full["idx"].cpu().numpy(), "K_out": synth.to_bits(full["K_out"]),
            "V_out": synth.to_bits(full["V_out"]), "scores": full["scores"].cpu().numpy()}
    check_against_oracle(oracle, synth.to_bits(K), synth.to_bits(V), sink, L, k, 1, host,
                         storage=oracle.STORAGE_FP8_E4M3)
    u8 = lambda t: t.view(torch.uint8)
    rows = plan.compress_prefill(K, V, ws, want_idx=False)
    assert torch.equal(u8(rows["K_out"]), u8(full["K_out"])) and torch.equal(u8(rows["V_out"]), u8(full["V_out"]))
    Kp, Vp, table = paginate(u8(K), u8(V), 64, seed=3)
    paged = plan.compress_prefill_paged(Kp.view(FP8), Vp.view(FP8), table, S, ws, want_scores=True)
    assert plan.read_status(ws)[0] == 0
    assert torch.equal(paged["idx"], full["idx"]) and torch.equal(paged["scores"], full["scores"])
    assert torch.equal(u8(paged["K_out"]), u8(full["K_out"])) and torch.equal(u8(paged["V_out"]), u8(full["V_out"]))


@pytest.mark.parametrize("L,k,chunks,tune", [(64, 16, 3, None), (512, 128, 1, dict(warps=CLUSTER, tile_rows=2, stages=2, ctas_per_sm=2)),
                                             (512, 128, 1, dict(warps=4, tile_rows=32, stages=3, ctas_per_sm=2)),
                                             (96, 24, 1, dict(warps=CLUSTER, tile_rows=1, stages=2, ctas_per_sm=2))])
def test_fp8_append(binding, oracle, L, k, chunks, tune):
    sink = 8
    stat = [sink, sink + 2 * k, sink]
    seq = [stat[0] + (chunks + 1) * L + 3, stat[1] + (chunks + 1) * L, stat[2] + 2 * L - 1]
    r = append_case(binding, oracle, 3, 2, 128, max(seq) + 9, sink, L, k, seq, stat, chunks, seed=L + chunks, tune=tune,
                    dtype=FP8)
    check_append(r, 3)


def test_fp8_scores_do_not_depend_on_the_quantisation_scale(binding):
    """A power-of-two rescale of a whole fp8 cache (what a different per-tensor scale of the
    caller's quantiser amounts to) leaves scores and picks bit-identical: Eq. 9 cancels it."""
    B, H, D, sink, L, k = 2, 2, 128, 4, 128, 32
    S = sink + 6 * L + 9
    K, V = synth.make_kv(B, H, S, D, seed=5, device="cuda:0")                 # bf16 draws
    scale = 8.0 / float(K.float().abs().max())
    K8a, V8a = (K.float() * scale).to(FP8), (V.float() * scale).to(FP8)
    for t in (K8a, V8a):      # flush what would be subnormal (a rescale of those is not exact)
        t.view(torch.uint8)[(t.view(torch.uint8) & 0x78) == 0] = 0
    big = lambda t: (t.float() * 16.0).to(FP8)                                # exact: exponent + 4, far from both ends
    K8b, V8b = big(K8a), big(V8a)
    assert torch.equal(K8b.float(), K8a.float() * 16.0)
    plan = binding.Plan(B, H, D, sink, L, keep_k=k, device=0, dtype=FP8)
    ws = plan.new_workspace()
    a = plan.compress_prefill(K8a, V8a, ws, want_scores=True)
    b = plan.compress_prefill(K8b, V8b, ws, want_scores=True)
    assert torch.equal(a["scores"], b["scores"]) and torch.equal(a["idx"], b["idx"])


@pytest.mark.parametrize("D", [64, 96, 256])
@pytest.mark.parametrize("L,k,tune", [(64, 16, None), (128, 16, dict(warps=100, tile_rows=32, stages=2, ctas_per_sm=1)),
                                      (256, 64, None), (1024, 256, None)])
def test_fp8_head_dims(binding, oracle, D, L, k, tune):
    """fp8 rows of 64, 96 and 256 bytes on the uniform, pair and (where compiled) warp-specialised kernels."""
    n = 4 if L >= 512 else 7
    run_prefill(binding, oracle, 2, 3, D, 16 + n * L + 37, 16, L, k, seed=D + L, tune=tune, dtype=FP8)


@pytest.mark.parametrize("D", [64, 96, 256])
def test_fp8_append_head_dims(binding, oracle, D):
    """fp8 appends at the other head dims: several partitions (uniform kernel) and one (cluster)."""
    sink, L, k = 8, 128, 32
    for chunks in (2, 1):
        stat = [sink, sink + k]
        seq = [stat[0] + (chunks + 1) * L + 5, stat[1] + (chunks + 1) * L]
        r = append_case(binding, oracle, 2, 2, D, max(seq) + 9, sink, L, k, seq, stat, chunks, seed=D + chunks, dtype=FP8)
        check_append(r, 2)
