"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol
the header declares, and its planner integers agree with Eq. 12 and the oracle."""
import ctypes
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def binding():
    import __graft_entry__ as g
    g.build()
    from paper_2504_04704_b200 import binding as b
    return b


def test_exports_match_header(binding):
    header = (ROOT / "include" / "lagkv.h").read_text()
    declared = set(re.findall(r"\b(lagkv_[a-z_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    lib = binding.load_library()
    for name in declared:
        assert getattr(lib, name) is not None


def test_no_torch_types_and_no_oracle_in_product():
    """The boundary is plain C; the product never touches the oracle."""
    header = (ROOT / "include" / "lagkv.h").read_text()
    assert "torch" not in header and "at::" not in header
    for path in (ROOT / "paper_2504_04704_b200").rglob("*"):
        if path.suffix in (".py", ".cu", ".cuh", ".h"):
            text = path.read_text()
            assert not re.search(r"^\s*(from|import)\s+oracle\b", text, re.M), f"{path} imports the oracle"
            assert "lagkv_oracle" not in text, f"{path} refers to the oracle library"


def test_status_strings(binding):
    assert binding.status_string(0) == "ok"
    assert "timed out" in binding.status_string(binding.LAGKV_ETIMEOUT)
    assert "sm_100a" in binding.version()


@pytest.mark.parametrize("Ls,S,L,k,want", [(4096, 16, 128, 32, 1216), (32768, 16, 1024, 256, 9728),
                                           (131072, 16, 2048, 256, 19968), (65536, 4, 64, 4, 4216),
                                           (65536, 4, 2048, 1024, 34816), (16 + 255, 16, 128, 32, 16 + 255)])
def test_planner_matches_eq12(binding, oracle, Ls, S, L, k, want):
    plan = binding.Plan(1, 8, 128, S, L, keep_k=k, device=-1)
    assert plan.compressed_len(Ls) == want == oracle.compressed_len(Ls, S, L, k)
    # a later pass over a partly compressed cache
    assert plan.compressed_len(Ls, S + 3 * k) == oracle.compressed_len(Ls, S + 3 * k, L, k)


@pytest.mark.parametrize("r,L", [(0.25, 128), (0.125, 2048), (0.0625, 64), (0.167, 1024), (0.3, 10), (1.0, 7), (1e-6, 64)])
def test_keep_count_matches_oracle(binding, oracle, r, L):
    assert binding.Plan(1, 1, 128, 0, L, keep_ratio=r, device=-1).k == oracle.keep_count(r, L)


def test_keep_for_target(binding, oracle):
    """Adaptive retention: the chosen k meets the target compression ratio and k-1 does not."""
    for Ls, S, L, C in [(16384, 16, 128, 0.25), (16384, 16, 128, 0.5), (16384, 16, 128, 0.875), (5000, 4, 512, 0.6)]:
        k = binding.lagkv_keep_for_target(Ls, S, L, C)
        ratio = lambda kk: 1 - oracle.compressed_len(Ls, S, L, kk) / Ls
        assert ratio(k) <= C + 1e-12
        assert k == 1 or ratio(k - 1) > C
    assert binding.lagkv_keep_for_target(100, 16, 128, 0.5) == 128    # too short to compress


def test_host_plan_rejects_bad_configs(binding):
    for kw in (dict(D=100), dict(lag=1), dict(lag=10000), dict(keep_ratio=0.0), dict(keep_ratio=1.5),
               dict(std_ddof=2), dict(strides=(-8, 0, 0)), dict(B=0), dict(sink=-1)):
        args = dict(B=1, H_kv=2, D=128, sink=4, lag=64, keep_ratio=0.25, device=-1)
        args.update(kw)
        with pytest.raises(binding.LagKVError):
            binding.Plan(**args)


def test_host_only_plan_refuses_launch(binding):
    plan = binding.Plan(1, 2, 128, 4, 64, device=-1)
    lib = binding.load_library()
    rc = lib.lagkv_compress_prefill(plan.handle, ctypes.c_void_p(256), ctypes.c_void_p(512), 300, None, None,
                                    None, None, ctypes.c_void_p(1024), 256, None)
    assert rc == binding.LAGKV_EINVAL


def test_launch_shapes_fit_the_sm(binding):
    for L in (64, 128, 256, 512, 1024, 2048, 4096, 8192):
        plan = binding.Plan(32, 8, 128, 16, L, device=-1)
        info = plan.launch_info(16 + 40 * L)
        assert info["smem"] <= 232448 and info["block"] in (64, 128, 256, 384) and info["grid"] >= 148
    plan = binding.Plan(1, 8, 128, 16, 128, device=-1)
    assert plan.launch_info(100)["smem"] == 0        # identity pass: plain copy kernel
    with pytest.raises(binding.LagKVError):
        plan.tune(warps=8, tile_rows=32, stages=8)   # 512 KiB of ring does not fit


def test_plain_c_program_links_and_runs(binding, tmp_path):
    """include/lagkv.h is valid strict C99 and a C program linked to the shared object gets the
    planner's integers (host-side calls only: no GPU needed)."""
    import subprocess
    lib = Path(binding.LIB_PATH)
    exe = tmp_path / "host_only"
    subprocess.run(["gcc", "-std=c99", "-pedantic", "-Wall", "-Wextra", "-Werror", f"-I{ROOT / 'include'}",
                    str(ROOT / "tests" / "c_abi" / "host_only.c"), "-o", str(exe), f"-L{lib.parent}",
                    f"-l:{lib.name}", f"-Wl,-rpath,{lib.parent}"], check=True)
    out = subprocess.run([str(exe)], capture_output=True, text=True)
    assert out.returncode == 0 and out.stdout.strip() == "ok", out.stderr
