"""Pins for the float64 CPU oracle: everything here runs without a GPU.

The oracle is checked against things other than itself: hand-computed worked examples
(tests/golden), the closed form of Eq. 12, invariants that follow from Eq. 7-11,
special cases that reduce to numpy / scipy routines, an independent pure-Python brute
force, and the prefill == incremental equivalence of the recursive scheme.
"""
import math
from pathlib import Path

import numpy as np
import pytest
import scipy.special

from oracle import brute
from paper_2504_04704_b200 import synth

GOLDEN = Path(__file__).parent / "golden"


# ----------------------------------------------------------------------------- helpers
def read_case(name):
    case = {}
    for line in (GOLDEN / name).read_text().splitlines():
        if not line.strip() or line.startswith("#"):
            continue
        key, rest = line.split(None, 1)
        if key in ("K", "V"):
            case[key] = [[float(x) for x in row.split()] for row in rest.split("|")]
        else:
            vals = [float(x) for x in rest.split()]
            case[key] = vals if len(vals) > 1 or key.startswith(("s", "kept")) else vals[0]
    return case


def bits(x):
    """float array -> bf16 bit patterns; asserts the values are exactly representable."""
    x = np.asarray(x, dtype=np.float64)
    b = synth.f32_to_bits(x)
    assert np.array_equal(synth.bits_to_f64(b), x), "test value not representable in bf16"
    return b


def rand_bits(rng, shape, scale=1.0):
    """Random bf16 bit patterns (rounded normal draws)."""
    return synth.f32_to_bits(rng.standard_normal(shape) * scale)


def small_cache(seed, B=2, H=3, S=4 + 5 * 16 + 7, D=8):
    rng = np.random.default_rng(seed)
    return rand_bits(rng, (B, H, S, D)), rand_bits(rng, (B, H, S, D))


# --------------------------------------------------------------------- storage formats
def test_decode_every_bit_pattern(oracle):
    """The oracle's reading of all 65536 patterns: bf16 is the upper half of a binary32,
    fp16 is IEEE binary16 (held against numpy's float16)."""
    allbits = np.arange(65536, dtype=np.uint16)
    with np.errstate(invalid="ignore"):          # signalling NaN patterns
        want16 = allbits.view(np.float16).astype(np.float64)
        want_bf = (allbits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    for storage, want in ((oracle.STORAGE_FP16, want16), (oracle.STORAGE_BF16, want_bf)):
        got = oracle.decode(allbits, storage)
        assert np.array_equal(np.isnan(got), np.isnan(want))
        ok = ~np.isnan(want)
        assert np.array_equal(got[ok], want[ok]) and np.array_equal(np.signbit(got[ok]), np.signbit(want[ok]))


@pytest.mark.parametrize("ddof", [0, 1])
def test_fp16_storage_same_values_same_result(oracle, ddof):
    """Values that both formats hold exactly give the same scores and picks whichever format
    stores them, and the fp16 cache agrees with the pure-Python brute force on its values."""
    rng = np.random.default_rng(5 + ddof)
    S, L, D, k, n = 3, 8, 4, 3, 4
    Ls = S + n * L + 5
    Kf = rng.integers(-64, 65, (1, 1, Ls, D)) / 8.0      # multiples of 1/8 below 8: 7 significant bits
    Vf = rng.integers(-64, 65, (1, 1, Ls, D)) / 8.0
    Kb, Vb = bits(Kf), bits(Vf)
    Kh, Vh = Kf.astype(np.float16).view(np.uint16), Vf.astype(np.float16).view(np.uint16)
    assert np.array_equal(Kh.view(np.float16).astype(np.float64), Kf)
    a = oracle.compress(Kb, Vb, S, L, k, ddof=ddof)
    b = oracle.compress(Kh, Vh, S, L, k, ddof=ddof, storage=oracle.STORAGE_FP16)
    assert np.array_equal(a["idx"], b["idx"]) and np.array_equal(a["scores"], b["scores"])
    assert np.array_equal(b["K_out"], np.take_along_axis(Kh, b["idx"][..., None].astype(np.int64), axis=2))
    assert brute.compress_head(Kf[0, 0].tolist(), Vf[0, 0].tolist(), S, L, k, ddof) == b["idx"][0, 0].tolist()


def test_fp16_storage_values_only_fp16_holds(oracle):
    """Ten fraction bits: values that bf16 cannot hold, scored against numpy on the decoded values."""
    rng = np.random.default_rng(11)
    L, D = 16, 8
    h = (rng.standard_normal((4, L, D)) * 3).astype(np.float16)
    Kc, Vc, Kr, Vr = (x.view(np.uint16) for x in h)
    score, sK, sV = oracle.partition_scores(Kc, Vc, Kr, Vr, storage=oracle.STORAGE_FP16)
    f = h.astype(np.float64)
    parts = []
    for cur, ref in ((f[0], f[2]), (f[1], f[3])):
        y = (cur - ref.min(0)) / (ref.max(0) - ref.min(0))
        parts.append(scipy.special.softmax(np.std(y, axis=1, ddof=1)))
    want = parts[0] + parts[1]
    np.testing.assert_allclose(score, want, rtol=1e-12)
    np.testing.assert_allclose(sK, parts[0], rtol=1e-12)
    wrong = oracle.partition_scores(Kc, Vc, Kr, Vr)[0]              # the same bits read as bf16
    assert not np.allclose(wrong, want, rtol=1e-3)


def test_decode_fp8_every_byte(oracle):
    """The oracle's reading of all 256 fp8 (e4m3, finite-only) bytes against torch's conversion of
    the same bytes and against the format's definition: (-1)^s 2^(e-7) (1 + m/8), subnormals
    m/8 x 2^-6, no infinities, 0x7f and 0xff the only NaNs."""
    import torch
    allbytes = np.arange(256, dtype=np.uint8)
    got = oracle.decode(allbytes, oracle.STORAGE_FP8_E4M3)
    want = torch.from_numpy(allbytes.copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    assert np.isnan(got).sum() == 2 and np.isnan(got[0x7f]) and np.isnan(got[0xff])
    ok = ~np.isnan(want)
    assert np.array_equal(np.isnan(got), np.isnan(want))
    assert np.array_equal(got[ok], want[ok]) and np.array_equal(np.signbit(got[ok]), np.signbit(want[ok]))
    for byte, value in ((0x00, 0.0), (0x38, 1.0), (0x3c, 1.5), (0x40, 2.0), (0x7e, 448.0), (0x01, 2.0 ** -9),
                        (0x07, 7 * 2.0 ** -9), (0x08, 2.0 ** -6), (0xc0, -2.0), (0xfe, -448.0)):
        assert got[byte] == value, (hex(byte), got[byte], value)
    s, e, m = allbytes >> 7, (allbytes >> 3) & 15, allbytes & 7
    formula = np.where(e == 0, m / 8.0 * 2.0 ** -6, (1 + m / 8.0) * 2.0 ** (e.astype(np.float64) - 7)) * np.where(s == 1, -1.0, 1.0)
    assert np.array_equal(got[ok], formula[ok])


@pytest.mark.parametrize("ddof", [0, 1])
def test_fp8_storage_same_values_same_result(oracle, ddof):
    """Values that bf16 and fp8 both hold exactly (small integers and halves) give the same scores
    and picks whichever format stores them; the kept rows come back as the stored bytes."""
    import torch
    rng = np.random.default_rng(21 + ddof)
    S, L, D, k, n = 3, 8, 4, 3, 4
    Ls = S + n * L + 5
    Kf = rng.integers(-16, 17, (1, 1, Ls, D)) / 2.0      # multiples of 1/2 up to 8: at most 4 significant bits
    Vf = rng.integers(-16, 17, (1, 1, Ls, D)) / 2.0
    K8 = torch.from_numpy(Kf).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    V8 = torch.from_numpy(Vf).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(oracle.decode(K8, oracle.STORAGE_FP8_E4M3), Kf)
    a = oracle.compress(bits(Kf), bits(Vf), S, L, k, ddof=ddof)
    b = oracle.compress(K8, V8, S, L, k, ddof=ddof, storage=oracle.STORAGE_FP8_E4M3)
    assert np.array_equal(a["idx"], b["idx"]) and np.array_equal(a["scores"], b["scores"])
    assert b["K_out"].dtype == np.uint8
    assert np.array_equal(b["K_out"], np.take_along_axis(K8, b["idx"][..., None].astype(np.int64), axis=2))
    assert np.array_equal(b["V_out"], np.take_along_axis(V8, b["idx"][..., None].astype(np.int64), axis=2))
    assert brute.compress_head(Kf[0, 0].tolist(), Vf[0, 0].tolist(), S, L, k, ddof) == b["idx"][0, 0].tolist()


# ------------------------------------------------------------------ worked examples
@pytest.mark.parametrize("name", ["hand_case_1.txt", "hand_case_2.txt"])
@pytest.mark.parametrize("ddof", [0, 1])
def test_hand_cases(oracle, name, ddof):
    c = read_case(name)
    S, L, D, k = int(c["S"]), int(c["L"]), int(c["D"]), int(c["k"])
    K, V = np.array(c["K"]), np.array(c["V"])
    Kb, Vb = bits(K)[None, None], bits(V)[None, None]
    cur, ref = slice(S, S + L), slice(S + L, S + 2 * L)
    score, sK, sV = oracle.partition_scores(Kb[0, 0, cur], Vb[0, 0, cur], Kb[0, 0, ref],
                                            Vb[0, 0, ref], ddof=ddof)
    np.testing.assert_allclose(sK, c[f"sK_ddof{ddof}"], rtol=0, atol=1e-15)
    np.testing.assert_allclose(sV, c[f"sV_ddof{ddof}"], rtol=0, atol=1e-15)
    want_score = c.get("score", c.get(f"score_ddof{ddof}"))
    np.testing.assert_allclose(score, want_score, rtol=0, atol=1e-15)
    res = oracle.compress(Kb, Vb, S, L, k, ddof=ddof)
    assert res["L_R"] == len(c["kept_rows"]) == 4
    assert res["idx"][0, 0].tolist() == [int(v) for v in c["kept_rows"]]
    np.testing.assert_array_equal(res["K_out"][0, 0], Kb[0, 0][res["idx"][0, 0]])
    # the independent pure-Python statement agrees with the fixture too
    bs = brute.partition_score(K[cur].tolist(), V[cur].tolist(), K[ref].tolist(), V[ref].tolist(), ddof)
    np.testing.assert_allclose(bs, want_score, rtol=0, atol=1e-15)
    assert brute.compress_head(K.tolist(), V.tolist(), S, L, k, ddof) == res["idx"][0, 0].tolist()


# --------------------------------------------------------------------- Eq. 12 closed form
# (Ls, S, L, k) -> (n, rem, L_R): values worked out by hand from Eq. 12 for the
# benchmark configurations.
EQ12_TABLE = [
    ((4096, 16, 128, 32), (31, 112, 1216)),
    ((32768, 16, 1024, 256), (31, 1008, 9728)),
    ((131072, 16, 2048, 256), (63, 2032, 19968)),
    ((65536, 4, 64, 4), (1023, 60, 4216)),
    ((65536, 4, 2048, 1024), (31, 2044, 34816)),
    ((5, 1, 2, 1), (2, 0, 4)),
]


@pytest.mark.parametrize("args,want", EQ12_TABLE)
def test_eq12_table(oracle, args, want):
    Ls, S, L, k = args
    n, rem, L_R = want
    assert (Ls - S) // L == n and (Ls - S) % L == rem
    assert oracle.compressed_len(Ls, S, L, k) == L_R
    assert brute.lagkv_cache_len(Ls, S, L, k) == L_R


def test_skip_below_two_lags(oracle):
    # remark after Eq. 13: a sequence shorter than S + 2L is not compressed at all
    for Ls in (0, 5, 16 + 2 * 32 - 1):
        assert oracle.compressed_len(Ls, 16, 32, 8) == Ls
    assert oracle.compressed_len(16 + 2 * 32, 16, 32, 8) == 16 + 8 + 32
    K, V = small_cache(1, B=1, H=2, S=4 + 2 * 16 - 1)
    res = oracle.compress(K, V, 4, 16, 4)
    assert res["L_R"] == K.shape[2] and res["n_c"] == 0
    np.testing.assert_array_equal(res["K_out"], K)
    np.testing.assert_array_equal(res["V_out"], V)


def test_keep_count(oracle):
    assert oracle.keep_count(0.25, 128) == 32
    assert oracle.keep_count(0.125, 2048) == 256
    assert oracle.keep_count(0.0625, 64) == 4
    assert oracle.keep_count(0.167, 1024) == 172      # ceil(171.008)
    assert oracle.keep_count(1.0, 7) == 7
    assert oracle.keep_count(1e-9, 64) == 1
    assert oracle.keep_count(0.3, 10) == 3            # 0.3*10 = 3.0000000000000004 in binary


# ------------------------------------------------------------------ structural invariants
@pytest.mark.parametrize("seed,S,L,k,tail", [(0, 4, 16, 4, 7), (1, 0, 8, 3, 0), (2, 3, 5, 5, 4), (3, 1, 32, 1, 31)])
def test_structure(oracle, seed, S, L, k, tail):
    n = 4
    Ls = S + n * L + tail
    K, V = small_cache(seed, S=Ls)
    res = oracle.compress(K, V, S, L, k)
    idx = res["idx"]
    assert res["L_R"] == S + (n - 1) * k + L + tail == idx.shape[-1]
    for b in range(K.shape[0]):
        for h in range(K.shape[1]):
            row = idx[b, h]
            assert row[:S].tolist() == list(range(S))                      # sink untouched
            assert row[S + (n - 1) * k:].tolist() == list(range(S + (n - 1) * L, Ls))  # window
            assert np.all(np.diff(row) > 0)                                # order preserved
            for p in range(n - 1):
                part = row[S + p * k:S + (p + 1) * k]
                assert len(part) == k and part.min() >= S + p * L and part.max() < S + (p + 1) * L
            np.testing.assert_array_equal(res["K_out"][b, h], K[b, h][row])
            np.testing.assert_array_equal(res["V_out"][b, h], V[b, h][row])
    sc = res["scores"]
    np.testing.assert_allclose(sc.sum(-1), 2.0, rtol=0, atol=1e-12)        # two softmaxes
    assert sc.min() > 0 and sc.max() < 2


def test_keep_everything(oracle):
    K, V = small_cache(5, S=2 + 3 * 8 + 3)
    res = oracle.compress(K, V, 2, 8, 8)
    assert res["idx"][0, 0].tolist() == list(range(K.shape[2]))


# ------------------------------------------------------- reductions to library routines
def numpy_scores(Kc, Vc, Kr, Vr, ddof):
    out = []
    for cur, ref in ((Kc, Kr), (Vc, Vr)):
        cur, ref = synth.bits_to_f64(cur), synth.bits_to_f64(ref)
        y = (cur - ref.min(0)) / (ref.max(0) - ref.min(0))
        out.append(scipy.special.softmax(np.std(y, axis=1, ddof=ddof)))
    return out[0] + out[1], out[0], out[1]


@pytest.mark.parametrize("ddof", [0, 1])
@pytest.mark.parametrize("L,D", [(16, 8), (64, 128), (7, 3)])
def test_scores_vs_numpy_scipy(oracle, ddof, L, D):
    rng = np.random.default_rng(L * 1000 + D)
    Kc, Vc, Kr, Vr = (rand_bits(rng, (L, D), s) for s in (1.0, 3.0, 2.0, 0.5))
    got = oracle.partition_scores(Kc, Vc, Kr, Vr, ddof=ddof)
    want = numpy_scores(Kc, Vc, Kr, Vr, ddof)
    for g, w in zip(got, want):
        np.testing.assert_allclose(g, w, rtol=1e-12, atol=1e-15)


def test_ddof_matters(oracle):
    """The two std conventions give different scores: a mix-up cannot go unnoticed."""
    rng = np.random.default_rng(7)
    Kc, Vc, Kr, Vr = (rand_bits(rng, (16, 4)) for _ in range(4))
    s0 = oracle.partition_scores(Kc, Vc, Kr, Vr, ddof=0)[0]
    s1 = oracle.partition_scores(Kc, Vc, Kr, Vr, ddof=1)[0]
    assert np.abs(s0 - s1).max() > 1e-4


def test_topk_vs_stable_sort(oracle):
    rng = np.random.default_rng(11)
    for L, k in [(1, 1), (8, 3), (64, 16), (100, 99), (257, 31)]:
        score = rng.integers(0, 6, size=L).astype(np.float64)      # many exact ties
        want = np.sort(np.argsort(-score, kind="stable")[:k])
        np.testing.assert_array_equal(oracle.topk(score, k), want)
        assert brute.keep_indices(score.tolist(), k) == want.tolist()


def test_constant_partition_keeps_first_k(oracle):
    """All tokens of the current partition equal => every std equal => scores uniform
    2/L => the tie rule keeps the first k."""
    rng = np.random.default_rng(3)
    L, D, k = 16, 8, 5
    row_k, row_v = rand_bits(rng, (1, D)), rand_bits(rng, (1, D))
    Kc, Vc = np.repeat(row_k, L, 0), np.repeat(row_v, L, 0)
    Kr, Vr = rand_bits(rng, (L, D)), rand_bits(rng, (L, D))
    score = oracle.partition_scores(Kc, Vc, Kr, Vr)[0]
    np.testing.assert_allclose(score, 2.0 / L, rtol=1e-14)
    assert oracle.topk(score, k).tolist() == list(range(k))


def test_constant_v_reduces_to_k_std(oracle):
    """V constant over the partition => sV uniform => selection = top-k of std(K_norm)."""
    rng = np.random.default_rng(5)
    L, D, k = 32, 8, 6
    Kc, Kr, Vr = rand_bits(rng, (L, D)), rand_bits(rng, (L, D)), rand_bits(rng, (L, D))
    Vc = np.repeat(rand_bits(rng, (1, D)), L, 0)
    score, sK, sV = oracle.partition_scores(Kc, Vc, Kr, Vr)
    np.testing.assert_allclose(sV, 1.0 / L, rtol=1e-14)
    cur, ref = synth.bits_to_f64(Kc), synth.bits_to_f64(Kr)
    sd = np.std((cur - ref.min(0)) / (ref.max(0) - ref.min(0)), axis=1, ddof=1)
    want = np.sort(np.argsort(-sd, kind="stable")[:k])
    np.testing.assert_array_equal(oracle.topk(score, k), want)


def test_zero_range_channel_counts_as_zero(oracle):
    """A reference channel with max == min contributes y = 0 for every token."""
    rng = np.random.default_rng(9)
    L, D = 8, 4
    Kc, Vc, Kr, Vr = (rand_bits(rng, (L, D)) for _ in range(4))
    Kr[:, 2] = Kr[0, 2]
    cur, ref = synth.bits_to_f64(Kc), synth.bits_to_f64(Kr)
    rng_ = ref.max(0) - ref.min(0)
    y = np.where(rng_ > 0, (cur - ref.min(0)) / np.where(rng_ > 0, rng_, 1.0), 0.0)
    want = scipy.special.softmax(np.std(y, axis=1, ddof=1))
    np.testing.assert_allclose(oracle.partition_scores(Kc, Vc, Kr, Vr)[1], want, rtol=1e-12)


# ----------------------------------------------------------- what the reference may change
def test_reference_is_next_partition_only(oracle):
    """Scores of partition p depend on p (as current) and p+1 (as an unordered set of
    rows) and on nothing else."""
    S, L, k, n = 3, 16, 4, 4
    K, V = small_cache(21, B=1, H=1, S=S + n * L + 5)
    base = oracle.compress(K, V, S, L, k)["scores"][0, 0]
    rng = np.random.default_rng(0)
    # permuting the rows of partition 2 leaves partition 1's scores alone, changes 2's
    K2, V2 = K.copy(), V.copy()
    perm = rng.permutation(L)
    sl = slice(S + 2 * L, S + 3 * L)
    K2[0, 0, sl], V2[0, 0, sl] = K[0, 0, sl][perm], V[0, 0, sl][perm]
    got = oracle.compress(K2, V2, S, L, k)["scores"][0, 0]
    np.testing.assert_array_equal(got[0], base[0])
    np.testing.assert_allclose(got[1], base[1], rtol=1e-15)
    np.testing.assert_allclose(got[2], base[2][perm], rtol=1e-13)
    # rewriting partition 3 (the window) and the sink changes only partition 2's scores
    K3, V3 = K.copy(), V.copy()
    K3[0, 0, S + 3 * L:] = rand_bits(rng, K3[0, 0, S + 3 * L:].shape)
    K3[0, 0, :S] = rand_bits(rng, (S, K.shape[-1]))
    got = oracle.compress(K3, V3, S, L, k)["scores"][0, 0]
    np.testing.assert_array_equal(got[:2], base[:2])
    assert np.abs(got[2] - base[2]).max() > 1e-6
    # rewriting partition 0 changes only partition 0's scores
    K4 = K.copy()
    K4[0, 0, S:S + L] = rand_bits(rng, (L, K.shape[-1]))
    got = oracle.compress(K4, V, S, L, k)["scores"][0, 0]
    np.testing.assert_array_equal(got[1:], base[1:])
    assert np.abs(got[0] - base[0]).max() > 1e-6


def test_lag_direction(oracle):
    """The reference is the NEXT partition, not the previous one: scoring partition 0 of
    [A, B, ...] uses B; swapping in a different first partition must not change how B's
    statistics are applied.  Checked by building the expected scores with numpy."""
    S, L, k = 2, 8, 2
    K, V = small_cache(33, B=1, H=1, S=S + 3 * L)
    sc = oracle.compress(K, V, S, L, k)["scores"][0, 0]
    for p in range(2):
        cur, ref = slice(S + p * L, S + (p + 1) * L), slice(S + (p + 1) * L, S + (p + 2) * L)
        want = numpy_scores(K[0, 0, cur], V[0, 0, cur], K[0, 0, ref], V[0, 0, ref], 1)[0]
        np.testing.assert_allclose(sc[p], want, rtol=1e-12)


def test_affine_invariance_power_of_two(oracle):
    """z -> alpha_c * z with alpha_c a power of two, applied to the current and the
    reference partition alike, is exact in bf16 and must leave scores bit-identical."""
    rng = np.random.default_rng(17)
    L, D = 16, 8
    parts = [rand_bits(rng, (L, D)) for _ in range(4)]
    alpha = 2.0 ** rng.integers(-6, 7, size=D)
    scaled = [bits(synth.bits_to_f64(p) * alpha) for p in parts]
    a = oracle.partition_scores(*parts)
    b = oracle.partition_scores(*scaled)
    for x, y in zip(a, b):
        np.testing.assert_array_equal(x, y)


def test_affine_invariance_general_brute():
    """General per-channel affine maps (alpha_c > 0, any beta_c) leave Eq. 9 unchanged;
    checked on the pure-Python statement, which takes arbitrary floats."""
    rng = np.random.default_rng(19)
    L, D = 6, 4
    Kc, Vc, Kr, Vr = (rng.standard_normal((L, D)) for _ in range(4))
    al, be = rng.uniform(0.1, 5, D), rng.uniform(-3, 3, D)
    a = brute.partition_score(Kc.tolist(), Vc.tolist(), Kr.tolist(), Vr.tolist())
    b = brute.partition_score((Kc * al + be).tolist(), (Vc * al - be).tolist(),
                              (Kr * al + be).tolist(), (Vr * al - be).tolist())
    np.testing.assert_allclose(a, b, rtol=1e-10)
    # ... but rescaling the reference alone is NOT an invariance
    c = brute.partition_score(Kc.tolist(), Vc.tolist(), (Kr * al).tolist(), Vr.tolist())
    assert np.abs(np.array(a) - np.array(c)).max() > 1e-6


def test_channel_permutation(oracle):
    rng = np.random.default_rng(23)
    L, D = 16, 8
    parts = [rand_bits(rng, (L, D)) for _ in range(4)]
    perm = rng.permutation(D)
    a = oracle.partition_scores(*parts)[0]
    b = oracle.partition_scores(*[p[:, perm] for p in parts])[0]
    np.testing.assert_allclose(a, b, rtol=1e-13)


# -------------------------------------------------------------- brute force, tiny inputs
@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("ddof", [0, 1])
def test_c_oracle_vs_python_brute(oracle, seed, ddof):
    rng = np.random.default_rng(100 + seed)
    S, L, D = int(rng.integers(0, 5)), int(rng.integers(2, 9)), 4
    n, tail = int(rng.integers(2, 6)), int(rng.integers(0, L))
    k = int(rng.integers(1, L + 1))
    Ls = S + n * L + tail
    K, V = rand_bits(rng, (1, 1, Ls, D)), rand_bits(rng, (1, 1, Ls, D))
    res = oracle.compress(K, V, S, L, k, ddof=ddof)
    Kf, Vf = synth.bits_to_f64(K)[0, 0].tolist(), synth.bits_to_f64(V)[0, 0].tolist()
    assert brute.compress_head(Kf, Vf, S, L, k, ddof) == res["idx"][0, 0].tolist()
    for p in range(n - 1):
        a, b = S + p * L, S + (p + 1) * L
        want = brute.partition_score(Kf[a:b], Vf[a:b], Kf[b:b + L], Vf[b:b + L], ddof)
        np.testing.assert_allclose(res["scores"][0, 0, p], want, rtol=1e-12)


# --------------------------------------------------------------------------- recursion
@pytest.mark.parametrize("steps", [[1] * 40, [16] * 3, [5, 11, 3, 17, 4], [48]])
def test_prefill_equals_incremental(oracle, steps):
    """One pass over Ls tokens == a pass over the first S+2L tokens followed by appends in
    any step sizes with a pass after each (recursive application, Section 2.2)."""
    S, L, k, H, D = 3, 8, 3, 2, 8
    B = 2
    Ls = S + 2 * L + sum(steps)
    K, V = small_cache(41, B=B, H=H, S=Ls, D=D)
    one = oracle.compress(K, V, S, L, k)
    cap = Ls
    Kc, Vc = np.zeros((B, H, cap, D), np.uint16), np.zeros((B, H, cap, D), np.uint16)
    first = S + 2 * L
    Kc[:, :, :first], Vc[:, :, :first] = K[:, :, :first], V[:, :, :first]
    seq = np.full(B, first)
    stat = np.full(B, S)
    Kc, Vc, seq, stat, _ = oracle.compress_append(Kc, Vc, seq, stat, L, k)
    fed = first
    for st in steps:
        for b in range(B):
            Kc[b, :, seq[b]:seq[b] + st] = K[b, :, fed:fed + st]
            Vc[b, :, seq[b]:seq[b] + st] = V[b, :, fed:fed + st]
        seq = seq + st
        fed += st
        Kc, Vc, seq, stat, _ = oracle.compress_append(Kc, Vc, seq, stat, L, k)
    assert np.all(seq == one["L_R"])
    np.testing.assert_array_equal(Kc[:, :, :one["L_R"]], one["K_out"])
    np.testing.assert_array_equal(Vc[:, :, :one["L_R"]], one["V_out"])


def test_append_ragged_and_skip(oracle):
    """Sequences below 2L of new rows are left alone; others compress independently."""
    S, L, k, H, D = 2, 8, 2, 2, 8
    K, V = small_cache(43, B=3, H=H, S=64, D=D)
    seq = np.array([S + 2 * L - 1, S + 2 * L, S + 3 * L + 5])
    stat = np.array([S, S, S])
    Kn, Vn, seq2, stat2, kept = oracle.compress_append(K, V, seq, stat, L, k)
    assert seq2.tolist() == [S + 2 * L - 1, S + k + L, S + 2 * k + L + 5]
    assert stat2.tolist() == [S, S + k, S + 2 * k]
    np.testing.assert_array_equal(Kn[0], K[0])
    assert kept[0].shape == (H, 0) and kept[1].shape == (H, k) and kept[2].shape == (H, 2 * k)
    one = oracle.compress(K[2:3, :, :seq[2]], V[2:3, :, :seq[2]], S, L, k)
    np.testing.assert_array_equal(Kn[2, :, :seq2[2]], one["K_out"][0])


# ----------------------------------------------------------------------------- variants
def test_localkv_uses_own_statistics(oracle):
    rng = np.random.default_rng(29)
    L, D = 16, 8
    Kc, Vc, Kr, Vr = (rand_bits(rng, (L, D)) for _ in range(4))
    want = numpy_scores(Kc, Vc, Kc, Vc, 1)[0]
    np.testing.assert_allclose(oracle.partition_scores(Kc, Vc, Kc, Vc, variant=oracle.VARIANT_LOCALKV)[0],
                               want, rtol=1e-12)
    S, k = 2, 4
    K, V = small_cache(31, B=1, H=1, S=S + 3 * L)
    sc = oracle.compress(K, V, S, L, k, variant=oracle.VARIANT_LOCALKV)["scores"][0, 0]
    for p in range(2):
        cur = slice(S + p * L, S + (p + 1) * L)
        np.testing.assert_allclose(sc[p], numpy_scores(K[0, 0, cur], V[0, 0, cur], K[0, 0, cur], V[0, 0, cur], 1)[0],
                                   rtol=1e-12)
    # y lies in [0, 1] when a partition is normalised by itself
    assert sc.min() > 0


def test_l2norm_variant(oracle):
    rng = np.random.default_rng(37)
    L, D, k = 16, 8, 4
    Kc, Vc = rand_bits(rng, (L, D)), rand_bits(rng, (L, D))
    score = oracle.partition_scores(Kc, Vc, Kc, Vc, variant=oracle.VARIANT_L2NORM)[0]
    norms = np.linalg.norm(synth.bits_to_f64(Kc), axis=1)
    np.testing.assert_allclose(score, -norms, rtol=1e-14)
    np.testing.assert_array_equal(oracle.topk(score, k), np.sort(np.argsort(norms, kind="stable")[:k]))


def test_gather(oracle):
    rng = np.random.default_rng(39)
    X = rand_bits(rng, (2, 3, 20, 8))
    idx = rng.integers(0, 20, size=(2, 3, 11)).astype(np.int32)
    got = oracle.gather(X, idx)
    want = np.take_along_axis(X, idx[..., None].astype(np.int64), axis=2)
    np.testing.assert_array_equal(got, want)


def test_generator_is_seeded():
    a = synth.make_kv(1, 2, 64, 8, seed=5)
    b = synth.make_kv(1, 2, 64, 8, seed=5)
    c = synth.make_kv(1, 2, 64, 8, seed=6)
    assert np.array_equal(synth.to_bits(a[0]), synth.to_bits(b[0]))
    assert not np.array_equal(synth.to_bits(a[0]), synth.to_bits(c[0]))
    assert math.isfinite(float(a[1].float().abs().max()))
