"""The oracle's pins must have teeth: plant one plausible mistake at a time in a COPY of
the oracle's C source (text substitution, CPU only), rebuild it as a separate module and
check that at least one pin of test_oracle_pins.py fails for every planted mistake.

If the oracle's source changes so that a pattern no longer occurs, the test fails loudly
instead of silently testing nothing.
"""
import importlib.util
import shutil
import sys
from pathlib import Path

import pytest

import test_oracle_pins as pins

ORACLE_DIR = Path(__file__).resolve().parent.parent / "oracle"

MUTANTS = {
    "reference_is_self_not_next": ("? cur : cur + L;", "? cur + L : cur;"),
    "min_takes_larger": ("if (z < mn[c]) mn[c] = z;", "if (z > mn[c]) mn[c] = z;"),
    "range_multiplied": ("(z - mn[c]) / range", "(z - mn[c]) * range"),
    "ddof_ignored": ("(double)(D - ddof)", "(double)(D)"),
    "mean_not_divided": ("mean /= (double)D;", ";"),
    "variance_not_std": ("sd[t] = sqrt(ss / (double)(D - ddof));", "sd[t] = ss / (double)(D - ddof);"),
    "softmax_sign": ("out[t] = exp(sd[t] - top);", "out[t] = exp(top - sd[t]);"),
    "softmax_not_normalised": ("for (int64_t t = 0; t < L; ++t) out[t] /= denom;", ";"),
    "v_term_dropped": ("score[t] = a[t] + b[t];", "score[t] = a[t];"),
    "k_and_v_share_reference": ("tensor_score(Vcur, Vref,", "tensor_score(Vcur, Kref,"),
    "tie_to_higher_index": ("score[t] > score[best]) best = t;", "score[t] >= score[best]) best = t;"),
    "partition_count_rounded_up": ("int64_t n = rest / L;\n    int64_t rem", "int64_t n = (rest + L - 1) / L;\n    int64_t rem"),
    "l2_not_negated": ("score[t] = -sqrt(ss);", "score[t] = sqrt(ss);"),
    "fp16_exponent_bias": ("ldexp(1.0 + (double)frac / 1024.0, e - 15);", "ldexp(1.0 + (double)frac / 1024.0, e - 16);"),
    "fp16_subnormal_scale": ("ldexp((double)frac, -24);", "ldexp((double)frac, -25);"),
    "fp16_fraction_width": ("(double)frac / 1024.0", "(double)frac / 2048.0"),
    "fp8_exponent_bias": ("ldexp(1.0 + (double)frac / 8.0, e - 7);", "ldexp(1.0 + (double)frac / 8.0, e - 8);"),
    "fp8_subnormal_scale": ("ldexp((double)frac, -9);", "ldexp((double)frac, -10);"),
    "fp8_fraction_width": ("(double)frac / 8.0", "(double)frac / 16.0"),
    "fp8_has_infinities": ("else if (e == 15 && frac == 7)\n        v = NAN;", "else if (e == 15)\n        v = frac ? NAN : INFINITY;"),
    "fp8_flag_ignored": ("if (storage == LAGKV_ORACLE_FP8_E4M3) return fp8_e4m3_to_double(bits);", ""),
    "storage_flag_ignored": ("return storage == LAGKV_ORACLE_FP16 ? fp16_to_double(bits) : bf16_to_double(bits);",
                             "return bf16_to_double(bits);"),
}


# Mutants whose planted mistake makes the full pass index out of bounds run only the pins
# that do not execute it.
ONLY = {"partition_count_rounded_up": ("eq12",)}


def run_pins(mod, only=None):
    """Run a compact set of pins against oracle module ``mod``; return the names that failed."""
    checks = []
    for name in ("hand_case_1.txt", "hand_case_2.txt"):
        for ddof in (0, 1):
            checks.append((f"hand:{name}:{ddof}", lambda n=name, d=ddof: pins.test_hand_cases(mod, n, d)))
    for args, want in pins.EQ12_TABLE:
        checks.append((f"eq12:{args}", lambda a=args, w=want: pins.test_eq12_table(mod, a, w)))
    for ddof in (0, 1):
        checks.append((f"numpy:{ddof}", lambda d=ddof: pins.test_scores_vs_numpy_scipy(mod, d, 16, 8)))
    checks += [
        ("structure", lambda: pins.test_structure(mod, 0, 4, 16, 4, 7)),
        ("topk", lambda: pins.test_topk_vs_stable_sort(mod)),
        ("lag_direction", lambda: pins.test_lag_direction(mod)),
        ("reference_only", lambda: pins.test_reference_is_next_partition_only(mod)),
        ("constant_v", lambda: pins.test_constant_v_reduces_to_k_std(mod)),
        ("ddof_matters", lambda: pins.test_ddof_matters(mod)),
        ("l2", lambda: pins.test_l2norm_variant(mod)),
        ("brute", lambda: pins.test_c_oracle_vs_python_brute(mod, 0, 1)),
        ("decode", lambda: pins.test_decode_every_bit_pattern(mod)),
        ("fp16_same_values", lambda: pins.test_fp16_storage_same_values_same_result(mod, 1)),
        ("fp16_only", lambda: pins.test_fp16_storage_values_only_fp16_holds(mod)),
        ("fp8_decode", lambda: pins.test_decode_fp8_every_byte(mod)),
        ("fp8_same_values", lambda: pins.test_fp8_storage_same_values_same_result(mod, 1)),
    ]
    failed = []
    for name, fn in checks:
        if only is not None and not name.startswith(only):
            continue
        try:
            fn()
        except AssertionError:
            failed.append(name)
    return failed


def load_variant(tmp_path, tag, old=None, new=None):
    d = tmp_path / f"oracle_{tag}"
    d.mkdir()
    src = (ORACLE_DIR / "lagkv_oracle.c").read_text()
    if old is not None:
        assert src.count(old) == 1, f"pattern for mutant {tag!r} must occur exactly once in the oracle"
        src = src.replace(old, new)
    (d / "lagkv_oracle.c").write_text(src)
    shutil.copy(ORACLE_DIR / "lagkv_oracle.py", d / "lagkv_oracle.py")
    spec = importlib.util.spec_from_file_location(f"oracle_variant_{tag}", d / "lagkv_oracle.py")
    mod = importlib.util.module_from_spec(spec)
    sys.modules[spec.name] = mod
    spec.loader.exec_module(mod)
    mod.build()
    return mod


def test_unmodified_copy_passes_every_pin(tmp_path):
    assert run_pins(load_variant(tmp_path, "clean")) == []


@pytest.mark.parametrize("tag", sorted(MUTANTS))
def test_planted_mistake_is_caught(tmp_path, tag):
    old, new = MUTANTS[tag]
    failed = run_pins(load_variant(tmp_path, tag, old, new), ONLY.get(tag))
    assert failed, f"no pin noticed the planted mistake {tag!r}"
