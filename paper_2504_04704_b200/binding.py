"""ctypes binding of the C-ABI library declared in ``include/lagkv.h``.

Argument marshalling only: every step of the LagKV compress pass (Section 2.2 of
arXiv 2504.04704) runs inside the CUDA library.  PyTorch supplies device memory and the
current stream.  There is no CPU fallback: if ``liblagkv_b200.so`` has not been built
(``python -c "import __graft_entry__ as g; g.build()"``) the first call raises.

The functions carry the names of the C entry points (``lagkv_plan``,
``lagkv_compress_prefill``, ``lagkv_compress_append``, ``lagkv_gather`` ...); ``Plan`` is
a small convenience wrapper that owns the handle and allocates outputs with torch.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

LIB_PATH = Path(__file__).resolve().parent / "liblagkv_b200.so"

LAGKV_OK, LAGKV_EINVAL, LAGKV_EUNSUPPORTED, LAGKV_EWORKSPACE, LAGKV_ECUDA, LAGKV_ETIMEOUT, LAGKV_ECAPACITY = range(7)
LAGKV_ENOALLOC_LIMIT = 7
NOALLOC_SCRATCH_BYTES = 1048576
TUNE_PAIRS = 100          # lagkv_plan_tune(): the pair kernel for short partitions
VARIANT_LAGKV, VARIANT_LOCALKV, VARIANT_L2NORM = 0, 1, 2

# every symbol include/lagkv.h declares
EXPORTS = (
    "lagkv_plan", "lagkv_plan_destroy", "lagkv_keep_count", "lagkv_compressed_len",
    "lagkv_keep_for_target", "lagkv_lengths_after", "lagkv_workspace_bytes", "lagkv_workspace_init",
    "lagkv_compress_prefill", "lagkv_compress_prefill_host", "lagkv_host_staging_bytes",
    "lagkv_compress_append", "lagkv_compress_append_noalloc", "lagkv_compress_prefill_paged",
    "lagkv_compress_append_paged", "lagkv_gather", "lagkv_gather_paged",
    "lagkv_read_status",
    "lagkv_launch_info", "lagkv_plan_tune", "lagkv_selftest_bounded_wait", "lagkv_status_string", "lagkv_version",
)


class LagKVError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (status {code})")


class lagkv_config(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int32), ("H_kv", ctypes.c_int32), ("D", ctypes.c_int32),
        ("sink", ctypes.c_int32), ("lag", ctypes.c_int32),
        ("keep_ratio", ctypes.c_double),
        ("keep_k", ctypes.c_int32), ("std_ddof", ctypes.c_int32), ("variant", ctypes.c_int32),
        ("stride_b", ctypes.c_int64), ("stride_h", ctypes.c_int64), ("stride_s", ctypes.c_int64),
        ("device", ctypes.c_int32), ("dtype", ctypes.c_int32),
    ]


class lagkv_paged_layout(ctypes.Structure):
    _fields_ = [
        ("block_table", ctypes.c_void_p), ("max_blocks", ctypes.c_int32), ("page_size", ctypes.c_int32),
        ("stride_page", ctypes.c_int64), ("stride_h", ctypes.c_int64), ("stride_s", ctypes.c_int64),
    ]


_lib = None


def load_library() -> ctypes.CDLL:
    """Open the CUDA library; a missing build is an error, never a fallback."""
    global _lib
    if _lib is not None:
        return _lib
    if not LIB_PATH.exists():
        raise RuntimeError(
            f"{LIB_PATH} is missing: build the CUDA library first (__graft_entry__.build()); "
            "there is no CPU fallback for the LagKV compress pass")
    lib = ctypes.CDLL(str(LIB_PATH))
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    lib.lagkv_plan.restype = ctypes.c_int
    lib.lagkv_plan.argtypes = [ctypes.POINTER(lagkv_config), ctypes.POINTER(vp)]
    lib.lagkv_plan_destroy.restype = None
    lib.lagkv_plan_destroy.argtypes = [vp]
    lib.lagkv_keep_count.restype = i32
    lib.lagkv_keep_count.argtypes = [vp]
    lib.lagkv_compressed_len.restype = i64
    lib.lagkv_compressed_len.argtypes = [vp, i64, i64]
    lib.lagkv_lengths_after.restype = ctypes.c_int
    lib.lagkv_lengths_after.argtypes = [vp, i64, i64, ctypes.POINTER(i64), ctypes.POINTER(i64)]
    lib.lagkv_keep_for_target.restype = i32
    lib.lagkv_keep_for_target.argtypes = [i64, i32, i32, ctypes.c_double]
    lib.lagkv_workspace_bytes.restype = sz
    lib.lagkv_workspace_bytes.argtypes = [vp, i32]
    lib.lagkv_workspace_init.restype = ctypes.c_int
    lib.lagkv_workspace_init.argtypes = [vp, vp, sz, vp]
    lib.lagkv_compress_prefill.restype = ctypes.c_int
    lib.lagkv_compress_prefill.argtypes = [vp, vp, vp, i64, vp, vp, vp, vp, vp, sz, vp]
    lib.lagkv_host_staging_bytes.restype = sz
    lib.lagkv_host_staging_bytes.argtypes = [vp, i64, i32]
    lib.lagkv_compress_prefill_host.restype = ctypes.c_int
    lib.lagkv_compress_prefill_host.argtypes = [vp, vp, vp, i64, vp, vp, vp, i32, vp, sz, vp, sz, vp]
    lib.lagkv_compress_append.restype = ctypes.c_int
    lib.lagkv_compress_append.argtypes = [vp, vp, vp, i64, vp, vp, i32, vp, vp, vp, sz, vp]
    lib.lagkv_compress_append_noalloc.restype = ctypes.c_int
    lib.lagkv_compress_append_noalloc.argtypes = [vp, vp, vp, i64, vp, vp, i32, vp, vp, vp, vp]
    lib.lagkv_compress_prefill_paged.restype = ctypes.c_int
    lib.lagkv_compress_prefill_paged.argtypes = [vp, vp, vp, ctypes.POINTER(lagkv_paged_layout), i64, vp, vp, vp, vp, vp,
                                                 sz, vp]
    lib.lagkv_compress_append_paged.restype = ctypes.c_int
    lib.lagkv_compress_append_paged.argtypes = [vp, vp, vp, ctypes.POINTER(lagkv_paged_layout), vp, vp, i32, vp, vp, vp,
                                                sz, vp]
    lib.lagkv_gather_paged.restype = ctypes.c_int
    lib.lagkv_gather_paged.argtypes = [vp, vp, vp, ctypes.POINTER(lagkv_paged_layout), i64, vp, i64, vp, vp, vp, vp]
    lib.lagkv_gather.restype = ctypes.c_int
    lib.lagkv_gather.argtypes = [vp, vp, vp, i64, vp, i64, vp, vp, vp, vp]
    lib.lagkv_read_status.restype = ctypes.c_int
    lib.lagkv_read_status.argtypes = [vp, vp, vp, ctypes.POINTER(i32 * 4)]
    lib.lagkv_launch_info.restype = ctypes.c_int
    lib.lagkv_launch_info.argtypes = [vp, i64, ctypes.POINTER(i32 * 6)]
    lib.lagkv_plan_tune.restype = ctypes.c_int
    lib.lagkv_plan_tune.argtypes = [vp, i32, i32, i32, i32]
    lib.lagkv_selftest_bounded_wait.restype = ctypes.c_int
    lib.lagkv_selftest_bounded_wait.argtypes = [vp, vp, i32, vp]
    lib.lagkv_status_string.restype = ctypes.c_char_p
    lib.lagkv_status_string.argtypes = [ctypes.c_int]
    lib.lagkv_version.restype = ctypes.c_char_p
    lib.lagkv_version.argtypes = []
    _lib = lib
    return lib


def status_string(code: int) -> str:
    return load_library().lagkv_status_string(int(code)).decode()


def version() -> str:
    return load_library().lagkv_version().decode()


def _check(code: int, where: str) -> None:
    if code != LAGKV_OK:
        raise LagKVError(code, where)


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(device) -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream(device).cuda_stream)


def lagkv_keep_for_target(Ls: int, sink: int, lag: int, target_C: float) -> int:
    return int(load_library().lagkv_keep_for_target(int(Ls), int(sink), int(lag), float(target_C)))


DTYPE_BF16, DTYPE_FP16, DTYPE_FP8_E4M3 = 0, 1, 2
_DTYPES = {torch.bfloat16: DTYPE_BF16, torch.float16: DTYPE_FP16, torch.float8_e4m3fn: DTYPE_FP8_E4M3}


class Plan:
    """Owns a ``lagkv_plan_t``.  ``device=-1`` makes a host-only plan (integers and launch
    shapes only; it cannot launch)."""

    def __init__(self, B, H_kv, D, sink, lag, keep_ratio=0.25, keep_k=0, std_ddof=1,
                 variant=VARIANT_LAGKV, strides=(0, 0, 0), device=0, dtype=torch.bfloat16):
        lib = load_library()
        if dtype not in _DTYPES:
            raise TypeError("dtype must be torch.bfloat16, torch.float16 or torch.float8_e4m3fn")
        self.dtype = dtype
        self.cfg = lagkv_config(int(B), int(H_kv), int(D), int(sink), int(lag), float(keep_ratio), int(keep_k),
                                int(std_ddof), int(variant), int(strides[0]), int(strides[1]), int(strides[2]),
                                int(device), _DTYPES[dtype])
        self.handle = ctypes.c_void_p()
        _check(lib.lagkv_plan(ctypes.byref(self.cfg), ctypes.byref(self.handle)), "lagkv_plan")
        self.lib = lib
        self.device = int(device)
        self.k = int(lib.lagkv_keep_count(self.handle))

    def close(self):
        if getattr(self, "handle", None) is not None and self.handle.value:
            self.lib.lagkv_plan_destroy(self.handle)
            self.handle = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- host arithmetic
    def compressed_len(self, seq_len: int, static_len: int = -1) -> int:
        return int(self.lib.lagkv_compressed_len(self.handle, int(seq_len), int(static_len)))

    def lengths_after(self, seq_len: int, static_len: int = -1) -> tuple[int, int]:
        """``lagkv_lengths_after``: (seq_len, static_len) of a sequence after one pass."""
        a, b = ctypes.c_int64(), ctypes.c_int64()
        _check(self.lib.lagkv_lengths_after(self.handle, int(seq_len), int(static_len), ctypes.byref(a),
                                            ctypes.byref(b)), "lagkv_lengths_after")
        return int(a.value), int(b.value)

    def workspace_bytes(self, max_new_chunks: int = 0) -> int:
        return int(self.lib.lagkv_workspace_bytes(self.handle, int(max_new_chunks)))

    def launch_info(self, S_in: int) -> dict:
        info = (ctypes.c_int32 * 6)()
        _check(self.lib.lagkv_launch_info(self.handle, int(S_in), ctypes.byref(info)), "lagkv_launch_info")
        kernel = ("lagkv_copy_kernel", "lagkv_stream_kernel", "lagkv_ws_kernel", "lagkv_pair_kernel")[info[4]]
        names = ("lagkv_copy_kernel", "lagkv_stream_kernel", "lagkv_ws_kernel", "lagkv_pair_kernel")
        return {"grid": info[0], "block": info[1], "smem": info[2], "launches": info[3], "kernel": kernel,
                "paged_kernel": names[info[5]]}

    def tune(self, warps=0, tile_rows=0, stages=0, ctas_per_sm=0) -> None:
        _check(self.lib.lagkv_plan_tune(self.handle, int(warps), int(tile_rows), int(stages), int(ctas_per_sm)),
               "lagkv_plan_tune")

    # ---- device work
    def _dev(self):
        return torch.device("cuda", self.device)

    def new_workspace(self, max_new_chunks: int = 0) -> torch.Tensor:
        ws = torch.empty(self.workspace_bytes(max_new_chunks), dtype=torch.uint8, device=self._dev())
        _check(self.lib.lagkv_workspace_init(self.handle, _ptr(ws), ws.numel(), _stream(self._dev())),
               "lagkv_workspace_init")
        return ws

    def read_status(self, workspace) -> list[int]:
        """``lagkv_read_status``; ``workspace=None`` reads the library's built-in scratch."""
        st = (ctypes.c_int32 * 4)()
        rc = self.lib.lagkv_read_status(self.handle, _ptr(workspace), _stream(self._dev()), ctypes.byref(st))
        if rc == LAGKV_ECUDA or rc == LAGKV_EINVAL and st[0] != LAGKV_EINVAL:
            raise LagKVError(rc, "lagkv_read_status")
        return [int(v) for v in st]

    def selftest_bounded_wait(self, workspace: torch.Tensor, limit_ms: int = 50) -> None:
        """``lagkv_selftest_bounded_wait``: a wait that cannot succeed must end with LAGKV_ETIMEOUT."""
        _check(self.lib.lagkv_selftest_bounded_wait(self.handle, _ptr(workspace), int(limit_ms),
                                                    _stream(self._dev())), "lagkv_selftest_bounded_wait")

    def _check_cache(self, t: torch.Tensor, name: str):
        if t.dtype != self.dtype or not t.is_cuda or t.device.index != self.device:
            raise TypeError(f"{name} must be a {self.dtype} CUDA tensor on device {self.device}")

    def compress_prefill(self, K, V, workspace, S_in=None, want_rows=True, want_idx=True, want_scores=False,
                         out=None):
        """``lagkv_compress_prefill``.  K, V: ``[B, H, S_in, D]`` bf16 (any layout matching the
        plan's strides).  Returns dict with ``L_R`` and the requested ``K_out``, ``V_out``,
        ``idx``, ``scores`` tensors.  ``out`` may carry preallocated tensors of the same keys."""
        self._check_cache(K, "K")
        self._check_cache(V, "V")
        c = self.cfg
        S_in = int(K.shape[2] if S_in is None else S_in)
        L_R = self.compressed_len(S_in)
        rest = S_in - c.sink
        n_c = rest // c.lag - 1 if rest >= 2 * c.lag else 0
        dev = self._dev()
        out = dict(out or {})
        if want_rows:
            out.setdefault("K_out", torch.empty((c.B, c.H_kv, L_R, c.D), dtype=self.dtype, device=dev))
            out.setdefault("V_out", torch.empty((c.B, c.H_kv, L_R, c.D), dtype=self.dtype, device=dev))
        if want_idx:
            out.setdefault("idx", torch.empty((c.B, c.H_kv, L_R), dtype=torch.int32, device=dev))
        if want_scores:
            out.setdefault("scores", torch.empty((c.B, c.H_kv, n_c, c.lag), dtype=torch.float32, device=dev))
        rc = self.lib.lagkv_compress_prefill(
            self.handle, _ptr(K), _ptr(V), S_in, _ptr(out.get("K_out")), _ptr(out.get("V_out")),
            _ptr(out.get("idx")), _ptr(out.get("scores")), _ptr(workspace), workspace.numel(), _stream(dev))
        _check(rc, "lagkv_compress_prefill")
        out["L_R"], out["n_c"] = L_R, n_c
        return out

    def compress_append(self, K_cache, V_cache, seq_len, static_len, workspace, max_new_chunks=1,
                        idx_out=None, scores_out=None):
        """``lagkv_compress_append``: in place on ``[B, H, S_cap, D]`` caches; ``seq_len`` and
        ``static_len`` are int32 CUDA tensors ``[B]`` updated by the call."""
        self._check_cache(K_cache, "K_cache")
        self._check_cache(V_cache, "V_cache")
        for t, name in ((seq_len, "seq_len"), (static_len, "static_len")):
            if t.dtype != torch.int32 or not t.is_cuda or t.numel() != self.cfg.B or not t.is_contiguous():
                raise TypeError(f"{name} must be a contiguous int32 CUDA tensor [B]")
        dev = self._dev()
        rc = self.lib.lagkv_compress_append(
            self.handle, _ptr(K_cache), _ptr(V_cache), int(K_cache.shape[2]), _ptr(seq_len), _ptr(static_len),
            int(max_new_chunks), _ptr(idx_out), _ptr(scores_out), _ptr(workspace), workspace.numel(), _stream(dev))
        _check(rc, "lagkv_compress_append")

    def compress_append_noalloc(self, K_cache, V_cache, seq_len, static_len, max_new_chunks=1, idx_out=None,
                                scores_out=None, status_out=None):
        """``lagkv_compress_append_noalloc``: the append pass for callers that cannot hand over a
        workspace.  The library's own fixed scratch array is used instead; nothing is
        allocated here either (every tensor, ``status_out`` int32[4] included, is the
        caller's).  Raises ``LagKVError`` with ``LAGKV_ENOALLOC_LIMIT`` when the kept-position
        list would not fit the built-in array."""
        self._check_cache(K_cache, "K_cache")
        self._check_cache(V_cache, "V_cache")
        for t, name in ((seq_len, "seq_len"), (static_len, "static_len")):
            if t.dtype != torch.int32 or not t.is_cuda or t.numel() != self.cfg.B or not t.is_contiguous():
                raise TypeError(f"{name} must be a contiguous int32 CUDA tensor [B]")
        rc = self.lib.lagkv_compress_append_noalloc(
            self.handle, _ptr(K_cache), _ptr(V_cache), int(K_cache.shape[2]), _ptr(seq_len), _ptr(static_len),
            int(max_new_chunks), _ptr(idx_out), _ptr(scores_out), _ptr(status_out), _stream(self._dev()))
        _check(rc, "lagkv_compress_append_noalloc")

    def _paged(self, K_pool, block_table, strides):
        """``lagkv_paged_layout`` of a pool ``[num_pages, H, page_size, D]`` (or ``strides`` = (page, head,
        row) in elements for another arrangement) and an int32 CUDA table ``[B, max_blocks]``."""
        if block_table.dtype != torch.int32 or not block_table.is_cuda or not block_table.is_contiguous() or \
                block_table.dim() != 2 or block_table.shape[0] != self.cfg.B:
            raise TypeError("block_table must be a contiguous int32 CUDA tensor [B, max_blocks]")
        sp, sh, ss = strides[:3] if strides is not None else (0, 0, 0)
        page_size = int(K_pool.shape[2]) if strides is None else int(strides[3])
        return lagkv_paged_layout(block_table.data_ptr(), int(block_table.shape[1]), page_size, int(sp), int(sh), int(ss))

    def compress_prefill_paged(self, K_pool, V_pool, block_table, S_in, workspace, want_scores=False, strides=None):
        """``lagkv_compress_prefill_paged``: pools ``[num_pages, H, page_size, D]`` (``strides`` =
        (page, head, row, page_size) for another arrangement), table ``[B, max_blocks]``; the
        outputs are contiguous as for ``compress_prefill``."""
        self._check_cache(K_pool, "K_pool")
        self._check_cache(V_pool, "V_pool")
        lay = self._paged(K_pool, block_table, strides)
        c, dev = self.cfg, self._dev()
        L_R = self.compressed_len(S_in)
        rest = S_in - c.sink
        n_c = rest // c.lag - 1 if rest >= 2 * c.lag else 0
        out = {"K_out": torch.empty((c.B, c.H_kv, L_R, c.D), dtype=self.dtype, device=dev),
               "V_out": torch.empty((c.B, c.H_kv, L_R, c.D), dtype=self.dtype, device=dev),
               "idx": torch.empty((c.B, c.H_kv, L_R), dtype=torch.int32, device=dev)}
        if want_scores:
            out["scores"] = torch.empty((c.B, c.H_kv, n_c, c.lag), dtype=torch.float32, device=dev)
        rc = self.lib.lagkv_compress_prefill_paged(
            self.handle, _ptr(K_pool), _ptr(V_pool), ctypes.byref(lay), int(S_in), _ptr(out["K_out"]),
            _ptr(out["V_out"]), _ptr(out["idx"]), _ptr(out.get("scores")), _ptr(workspace), workspace.numel(),
            _stream(dev))
        _check(rc, "lagkv_compress_prefill_paged")
        out["L_R"], out["n_c"] = L_R, n_c
        return out

    def compress_append_paged(self, K_pool, V_pool, block_table, seq_len, static_len, workspace, max_new_chunks=1,
                              idx_out=None, scores_out=None, strides=None):
        """``lagkv_compress_append_paged``: in place inside the sequences' own pages."""
        self._check_cache(K_pool, "K_pool")
        self._check_cache(V_pool, "V_pool")
        lay = self._paged(K_pool, block_table, strides)
        rc = self.lib.lagkv_compress_append_paged(
            self.handle, _ptr(K_pool), _ptr(V_pool), ctypes.byref(lay), _ptr(seq_len), _ptr(static_len),
            int(max_new_chunks), _ptr(idx_out), _ptr(scores_out), _ptr(workspace), workspace.numel(),
            _stream(self._dev()))
        _check(rc, "lagkv_compress_append_paged")

    def gather_paged(self, K_pool, V_pool, block_table, idx, S_in, workspace=None, strides=None):
        """``lagkv_gather_paged``: rows ``idx`` ``[B, H, n_idx]`` of a paged cache."""
        self._check_cache(K_pool, "K_pool")
        lay = self._paged(K_pool, block_table, strides)
        c, dev = self.cfg, self._dev()
        n_idx = int(idx.shape[-1])
        K_out = torch.empty((c.B, c.H_kv, n_idx, c.D), dtype=self.dtype, device=dev)
        V_out = None if V_pool is None else torch.empty_like(K_out)
        rc = self.lib.lagkv_gather_paged(self.handle, _ptr(K_pool), _ptr(V_pool), ctypes.byref(lay), int(S_in), _ptr(idx),
                                         n_idx, _ptr(K_out), _ptr(V_out), _ptr(workspace), _stream(dev))
        _check(rc, "lagkv_gather_paged")
        return K_out, V_out

    def gather(self, K, V, idx, workspace=None, S_in=None):
        """``lagkv_gather``: rows ``idx`` ``[B, H, n_idx]`` int32 of K (and V, may be None)."""
        self._check_cache(K, "K")
        c = self.cfg
        dev = self._dev()
        if idx.dtype != torch.int32 or not idx.is_cuda or not idx.is_contiguous():
            raise TypeError("idx must be a contiguous int32 CUDA tensor")
        n_idx = int(idx.shape[-1])
        S_in = int(K.shape[2] if S_in is None else S_in)
        K_out = torch.empty((c.B, c.H_kv, n_idx, c.D), dtype=self.dtype, device=dev)
        V_out = None if V is None else torch.empty_like(K_out)
        rc = self.lib.lagkv_gather(self.handle, _ptr(K), _ptr(V), S_in, _ptr(idx), n_idx, _ptr(K_out), _ptr(V_out),
                                   _ptr(workspace), _stream(dev))
        _check(rc, "lagkv_gather")
        return K_out, V_out


# ---- C-named thin functions ---------------------------------------------------------------
def lagkv_plan(**kw) -> Plan:
    return Plan(**kw)


def lagkv_plan_destroy(plan: Plan) -> None:
    plan.close()


def lagkv_compress_prefill(plan: Plan, K, V, workspace, **kw):
    return plan.compress_prefill(K, V, workspace, **kw)


def lagkv_compress_append(plan: Plan, K_cache, V_cache, seq_len, static_len, workspace, **kw):
    return plan.compress_append(K_cache, V_cache, seq_len, static_len, workspace, **kw)


def lagkv_compress_append_noalloc(plan: Plan, K_cache, V_cache, seq_len, static_len, **kw):
    return plan.compress_append_noalloc(K_cache, V_cache, seq_len, static_len, **kw)


def lagkv_gather(plan: Plan, K, V, idx, **kw):
    return plan.gather(K, V, idx, **kw)


class ChunkedPrefill:
    """Chunk-by-chunk compression during prefill (Section 4.2 of the paper: the first S + 2L
    tokens, then L tokens per step, compressing between steps) on top of
    ``lagkv_compress_append``.  The caller's model produces K/V rows chunk by chunk; ``feed``
    appends them to the caches held here and runs the append pass, so the caches never grow
    beyond ``capacity`` rows.  All sequences advance together."""

    def __init__(self, B, H_kv, D, sink, lag, keep_ratio=0.25, keep_k=0, std_ddof=1, capacity=None, device=0,
                 variant=VARIANT_LAGKV, dtype=torch.bfloat16):
        self.plan = Plan(B, H_kv, D, sink, lag, keep_ratio=keep_ratio, keep_k=keep_k, std_ddof=std_ddof, device=device,
                         variant=variant, dtype=dtype)
        dev = self.plan._dev()
        self.first = sink + 2 * lag                     # tokens of the first step
        self.step = lag                                 # tokens of every later step
        self.capacity = int(capacity if capacity is not None else sink + 4 * lag)
        self.K = torch.zeros((B, H_kv, self.capacity, D), dtype=dtype, device=dev)
        self.V = torch.zeros_like(self.K)
        self.seq_len = torch.zeros((B,), dtype=torch.int32, device=dev)
        self.static_len = torch.full((B,), sink, dtype=torch.int32, device=dev)
        self.ws = self.plan.new_workspace(2)
        self.rows = 0                                   # stored rows (host mirror of seq_len, all equal)
        self.static = sink                              # host mirror of static_len

    def feed(self, K_new, V_new, check_status: bool = False) -> None:
        """Append ``[B, H, t, D]`` new rows (any t that fits) and compress.  The host mirrors of
        the two lengths come from the library (``lagkv_lengths_after``), so no read-back is
        needed between steps; ``check_status`` synchronises and raises on a device-side error
        (without it, call ``status()`` at the end of the prompt)."""
        t = int(K_new.shape[2])
        if self.rows + t > self.capacity:
            raise ValueError("chunk does not fit the cache capacity")
        # more partitions than the workspace was sized for would be refused on the device
        if (self.rows + t - self.static) // self.plan.cfg.lag - 1 > 2:
            raise ValueError("chunk completes more than two partitions at once")
        self.K[:, :, self.rows:self.rows + t] = K_new
        self.V[:, :, self.rows:self.rows + t] = V_new
        self.seq_len += t
        self.rows += t
        self.plan.compress_append(self.K, self.V, self.seq_len, self.static_len, self.ws, max_new_chunks=2)
        self.rows, self.static = self.plan.lengths_after(self.rows, self.static)
        if check_status:
            self.status()

    def status(self) -> None:
        """Synchronise and raise if any append since the last check recorded a device-side error."""
        st = self.plan.read_status(self.ws)
        if st[0] != LAGKV_OK:
            raise LagKVError(st[0], "lagkv_compress_append (device status)")


class HostPrefill:
    """Prefill compression of a cache that lives in pinned HOST memory: ``lagkv_compress_prefill_host``.

    The library cuts the ``[B, H, S_in, D]`` host cache into chunks of ``chunk_B`` sequences (or
    layers folded into B), copies each chunk to the device staging buffer held here, compresses
    it and copies the compacted rows and indices back, on three streams with two staging slots
    so that copies in both directions overlap the kernel.  This class only owns the staging
    buffer and the workspace and marshals the call.
    """

    def __init__(self, B, H_kv, D, S_in, sink, lag, keep_ratio=0.25, keep_k=0, std_ddof=1, chunk_B=1, device=0):
        if B % chunk_B:
            raise ValueError("B must be a multiple of chunk_B")
        self.B, self.chunk_B, self.S_in = int(B), int(chunk_B), int(S_in)
        self.plan = Plan(B, H_kv, D, sink, lag, keep_ratio=keep_ratio, keep_k=keep_k, std_ddof=std_ddof, device=device)
        dev = self.plan._dev()
        self.L_R = self.plan.compressed_len(S_in)
        self.ws = self.plan.new_workspace()
        nbytes = int(self.plan.lib.lagkv_host_staging_bytes(self.plan.handle, self.S_in, self.chunk_B))
        if nbytes == 0:
            raise LagKVError(LAGKV_EINVAL, "lagkv_host_staging_bytes")
        self.staging = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        self.h2d_bytes = 2 * B * H_kv * S_in * D * 2
        self.d2h_bytes = 2 * B * H_kv * self.L_R * D * 2 + B * H_kv * self.L_R * 4

    def run(self, K_host, V_host, K_out_host, V_out_host, idx_host, wait: bool = True) -> None:
        """All five tensors are contiguous (pinned) host tensors.  The call only enqueues; with
        ``wait`` it returns after the last copy has landed."""
        want = {"K_host": (K_host, (self.B, self.plan.cfg.H_kv, self.S_in, self.plan.cfg.D), torch.bfloat16),
                "V_host": (V_host, (self.B, self.plan.cfg.H_kv, self.S_in, self.plan.cfg.D), torch.bfloat16),
                "K_out_host": (K_out_host, (self.B, self.plan.cfg.H_kv, self.L_R, self.plan.cfg.D), torch.bfloat16),
                "V_out_host": (V_out_host, (self.B, self.plan.cfg.H_kv, self.L_R, self.plan.cfg.D), torch.bfloat16),
                "idx_host": (idx_host, (self.B, self.plan.cfg.H_kv, self.L_R), torch.int32)}
        for name, (t, shape, dt) in want.items():
            if t.is_cuda or t.dtype != dt or tuple(t.shape) != shape or not t.is_contiguous():
                raise TypeError(f"{name} must be a contiguous host tensor {shape} of {dt}")
        dev = self.plan._dev()
        rc = self.plan.lib.lagkv_compress_prefill_host(
            self.plan.handle, _ptr(K_host), _ptr(V_host), self.S_in, _ptr(K_out_host), _ptr(V_out_host),
            _ptr(idx_host), self.chunk_B, _ptr(self.staging), self.staging.numel(), _ptr(self.ws), self.ws.numel(),
            _stream(dev))
        _check(rc, "lagkv_compress_prefill_host")
        if wait:
            torch.cuda.current_stream(dev).synchronize()
