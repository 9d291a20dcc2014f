"""Thin ctypes binding of ``libtriattn.so`` (the C ABI of ``include/tri_attention.h``).

Argument marshalling only: torch tensors provide device memory and the current stream, every
step of the compression round runs in the library's CUDA kernels.  There is no fallback: if the
shared library is missing, or a call returns an error status, an exception is raised.
"""
from __future__ import annotations

import ctypes
import dataclasses
import os
import subprocess
from pathlib import Path
from typing import Optional, Sequence

import torch

_PKG = Path(__file__).resolve().parent
_ROOT = _PKG.parent
LIB_PATH = _PKG / "lib" / "libtriattn.so"
SOURCES = [_PKG / "csrc" / "tri_api.cu"]
HEADERS = [_ROOT / "include" / "tri_attention.h", _PKG / "csrc" / "tri_common.cuh", _PKG / "csrc" / "tri_score.cuh",
           _PKG / "csrc" / "tri_score_pre.cuh", _PKG / "csrc" / "tri_score_tma.cuh", _PKG / "csrc" / "tri_score_umma.cuh", _PKG / "csrc" / "tri_calib.cuh", _PKG / "csrc" / "tri_calib_tma.cuh",
           _PKG / "csrc" / "tri_select.cuh", _PKG / "csrc" / "tri_compact.cuh"]

EXPORTS = ["tri_create", "tri_destroy", "tri_workspace_bytes", "tri_score", "tri_select", "tri_compact",
           "tri_compress", "tri_select_budgets", "tri_compress_budgets", "tri_compress_windowed", "tri_compress_host", "tri_score_static", "tri_score_static_bytes", "tri_compress_launches", "tri_set_pipeline", "tri_set_score_kernel", "tri_last_cuda_error",
           "tri_profile_begin", "tri_profile_read", "tri_profile_end",
           "tri_calib_state_bytes", "tri_calib_workspace_bytes", "tri_calib_reset", "tri_calib_accumulate",
           "tri_calib_finalize", "tri_selftest_bounded_wait"]

STATUS = {0: "TRI_OK", 1: "TRI_ERR_INVALID_ARG", 2: "TRI_ERR_UNSUPPORTED", 3: "TRI_ERR_WORKSPACE",
          4: "TRI_ERR_CUDA", 5: "TRI_ERR_DEVICE_CHECK", 6: "TRI_ERR_TIMEOUT"}

DEFAULT_OFFSETS = tuple(1 << j for j in range(17))   # D = {1, 2, 4, ..., 2^16} (Section 4.2)


class TriError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        self.code = code
        super().__init__(f"{where}: {STATUS.get(code, code)}" + (f" ({detail})" if detail else ""))


def build(force: bool = False, verbose: bool = False) -> Path:
    """Compile the library for sm_100a with nvcc (works without a GPU)."""
    deps = SOURCES + HEADERS
    if not force and LIB_PATH.exists() and all(LIB_PATH.stat().st_mtime >= d.stat().st_mtime for d in deps):
        return LIB_PATH
    LIB_PATH.parent.mkdir(parents=True, exist_ok=True)
    tmp = LIB_PATH.with_suffix(f".tmp{os.getpid()}.so")
    cmd = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-I", str(_ROOT / "include"), "-shared", "-Xcompiler", "-fPIC", "-o", str(tmp)]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [str(s) for s in SOURCES]
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIB_PATH)
    return LIB_PATH


class _ModelDesc(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32), ("group_size", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("rope_theta", ctypes.c_double), ("pair_layout", ctypes.c_int32),
                ("n_offsets", ctypes.c_int32), ("offsets", ctypes.c_void_p), ("norm_variant", ctypes.c_int32)]


class _CacheView(ctypes.Structure):
    _fields_ = [("k", ctypes.c_void_p), ("v", ctypes.c_void_p), ("k_kind", ctypes.c_int32), ("paged", ctypes.c_int32),
                ("stride_layer", ctypes.c_int64), ("stride_seq", ctypes.c_int64), ("stride_head", ctypes.c_int64),
                ("stride_tok", ctypes.c_int64), ("page_table", ctypes.c_void_p),
                ("max_pages_per_seq", ctypes.c_int32), ("page_size", ctypes.c_int32), ("n_pages", ctypes.c_int32),
                ("stride_page", ctypes.c_int64), ("stride_slot", ctypes.c_int64), ("seq_lens", ctypes.c_void_p),
                ("positions", ctypes.c_void_p), ("n_max", ctypes.c_int32)]


_lib = None


def lib():
    """The loaded shared library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not LIB_PATH.exists():
        raise RuntimeError(f"{LIB_PATH} is missing: build it with paper_2604_04921_b200.binding.build() "
                           "(or __graft_entry__.build()); the compression round has no other implementation")
    L = ctypes.CDLL(str(LIB_PATH))
    P, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
    VP = ctypes.POINTER(_CacheView)
    L.tri_create.argtypes = [ctypes.POINTER(_ModelDesc), P, P, ctypes.POINTER(P)]
    L.tri_create.restype = ctypes.c_int
    L.tri_destroy.argtypes = [P]
    L.tri_destroy.restype = ctypes.c_int
    L.tri_workspace_bytes.argtypes = [P, i32, i32, i32]
    L.tri_workspace_bytes.restype = sz
    L.tri_score.argtypes = [P, VP, i32, P, P, P, P, sz, P]
    L.tri_score.restype = ctypes.c_int
    L.tri_score_static.argtypes = [P, VP, i32, P, P, P, P]
    L.tri_score_static.restype = ctypes.c_int
    L.tri_score_static_bytes.argtypes = [P, i32, i32]
    L.tri_score_static_bytes.restype = sz
    L.tri_select.argtypes = [P, P, P, i32, i32, i32, P, P, P, sz, P]
    L.tri_select.restype = ctypes.c_int
    L.tri_compact.argtypes = [P, VP, P, P, i32, i32, VP, P, P]
    L.tri_compact.restype = ctypes.c_int
    L.tri_compress.argtypes = [P, VP, i32, P, i32, VP, P, P, P, P, P, sz, P]
    L.tri_compress.restype = ctypes.c_int
    L.tri_select_budgets.argtypes = [P, P, P, i32, i32, i32, P, P, P, P]
    L.tri_select_budgets.restype = ctypes.c_int
    L.tri_compress_budgets.argtypes = [P, VP, i32, P, i32, P, VP, P, P, P, P, P, sz, P]
    L.tri_compress_budgets.restype = ctypes.c_int
    L.tri_compress_windowed.argtypes = [P, VP, i32, P, i32, P, i32, i32, VP, P, P, P, P, P, sz, P]
    L.tri_compress_windowed.restype = ctypes.c_int
    L.tri_compress_host.argtypes = [P, VP, VP, i32, P, P, i32, VP, VP, P, P, P, sz, P]
    L.tri_compress_host.restype = ctypes.c_int
    L.tri_compress_launches.argtypes = [P, VP, i32, VP]
    L.tri_set_pipeline.argtypes = [P, i32]
    L.tri_set_pipeline.restype = ctypes.c_int
    L.tri_set_score_kernel.argtypes = [P, i32]
    L.tri_set_score_kernel.restype = ctypes.c_int
    L.tri_compress_launches.restype = i32
    for fn in (L.tri_profile_begin, L.tri_profile_end):
        fn.argtypes = [P]
        fn.restype = ctypes.c_int
    L.tri_profile_read.argtypes = [P, P]
    L.tri_profile_read.restype = ctypes.c_int
    i64 = ctypes.c_int64
    L.tri_calib_state_bytes.argtypes = [i32]
    L.tri_calib_state_bytes.restype = sz
    L.tri_calib_workspace_bytes.argtypes = [i32, i64]
    L.tri_calib_workspace_bytes.restype = sz
    L.tri_calib_reset.argtypes = [P, i32, P]
    L.tri_calib_reset.restype = ctypes.c_int
    L.tri_calib_accumulate.argtypes = [P, i32, i64, i32, i64, i64, i32, P, P, sz, P]
    L.tri_calib_accumulate.restype = ctypes.c_int
    L.tri_calib_finalize.argtypes = [P, i32, i32, P, P, P, P]
    L.tri_calib_finalize.restype = ctypes.c_int
    L.tri_selftest_bounded_wait.argtypes = [P, P]
    L.tri_selftest_bounded_wait.restype = ctypes.c_int
    L.tri_last_cuda_error.argtypes = []
    L.tri_last_cuda_error.restype = ctypes.c_char_p
    _lib = L
    return L


def _check(code: int, where: str):
    if code != 0:
        detail = lib().tri_last_cuda_error().decode() if code == 4 else ""
        raise TriError(code, where, detail)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


@dataclasses.dataclass
class CacheView:
    """K/V cache as torch tensors plus the layout the C ABI needs.

    contiguous: k, v [L, S, H, N, 128];  paged: k, v [L, P, H, page_size, 128] + page_table [S, max_pages].
    """
    k: torch.Tensor
    v: Optional[torch.Tensor]
    seq_lens: Optional[torch.Tensor] = None       # [S] int32
    positions: Optional[torch.Tensor] = None      # [L, S, H, n_max] int32
    page_table: Optional[torch.Tensor] = None     # [S, max_pages] int32
    n_max: Optional[int] = None
    pre_rope: bool = False                        # bf16 keys are pre-RoPE vectors (k_kind 2); fp32 keys always are

    def c_view(self) -> _CacheView:
        k = self.k
        assert k.dim() == 5 and k.shape[-1] == 128 and k.stride(-1) == 1
        fp8 = k.dtype == torch.float8_e4m3fn                 # e4m3 keys come with e4m3 values (k_kind 3)
        if self.v is not None:
            assert self.v.shape == k.shape and self.v.stride() == k.stride()
            assert self.v.dtype == (torch.float8_e4m3fn if fp8 else torch.bfloat16)
        assert k.dtype in (torch.bfloat16, torch.float32, torch.float8_e4m3fn)
        cv = _CacheView()
        cv.k = k.data_ptr()
        cv.v = self.v.data_ptr() if self.v is not None else None
        cv.k_kind = 3 if fp8 else ((2 if self.pre_rope else 0) if k.dtype == torch.bfloat16 else 1)
        if self.page_table is None:
            cv.paged = 0
            cv.stride_layer, cv.stride_seq, cv.stride_head, cv.stride_tok = k.stride()[:4]
            cv.n_max = k.shape[3] if self.n_max is None else self.n_max
        else:
            pt = self.page_table
            assert pt.dtype == torch.int32 and pt.is_contiguous()
            cv.paged = 1
            cv.stride_layer, cv.stride_page, cv.stride_head, cv.stride_slot = k.stride()[:4]
            cv.page_table = pt.data_ptr()
            cv.max_pages_per_seq = pt.shape[1]
            cv.page_size = k.shape[3]
            cv.n_pages = k.shape[1]
            cv.n_max = pt.shape[1] * k.shape[3] if self.n_max is None else self.n_max
        if self.seq_lens is not None:
            assert self.seq_lens.dtype == torch.int32 and self.seq_lens.is_contiguous()
            cv.seq_lens = self.seq_lens.data_ptr()
        if self.positions is not None:
            assert self.positions.dtype == torch.int32 and self.positions.is_contiguous()
            assert self.positions.shape[-1] == cv.n_max
            cv.positions = self.positions.data_ptr()
        return cv


class TriContext:
    """Per-model context: calibration statistics of Section 4.1 and the offset set of Section 4.2."""

    def __init__(self, n_layers: int, n_kv_heads: int, group_size: int, q_center: torch.Tensor,
                 q_mean_norm: torch.Tensor, rope_theta: float = 1e6, offsets: Sequence[int] = DEFAULT_OFFSETS,
                 pair_layout: int = 0, norm_variant: int = 0, head_dim: int = 128):
        L = lib()
        self.n_layers, self.n_kv_heads, self.group_size = n_layers, n_kv_heads, group_size
        qc = q_center.detach().to("cpu", torch.float32).contiguous()
        qn = q_mean_norm.detach().to("cpu", torch.float32).contiguous()
        assert qc.shape == (n_layers, n_kv_heads * group_size, head_dim), qc.shape
        assert qn.shape == (n_layers, n_kv_heads * group_size, head_dim // 2), qn.shape
        offs = (ctypes.c_int64 * len(offsets))(*[int(o) for o in offsets])
        d = _ModelDesc(n_layers, n_kv_heads, group_size, head_dim, float(rope_theta), pair_layout, len(offsets),
                       ctypes.cast(offs, ctypes.c_void_p), norm_variant)
        h = ctypes.c_void_p()
        self._h = None
        _check(L.tri_create(ctypes.byref(d), qc.data_ptr(), qn.data_ptr(), ctypes.byref(h)), "tri_create")
        self._h = h

    def close(self):
        if self._h is not None:
            lib().tri_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def units(self, S: int) -> int:
        return self.n_layers * S * self.n_kv_heads

    def workspace_bytes(self, S: int, n_max: int, budget: int) -> int:
        return int(lib().tri_workspace_bytes(self._h, S, n_max, budget))

    def workspace(self, S: int, n_max: int, budget: int, device="cuda") -> torch.Tensor:
        return torch.empty(self.workspace_bytes(S, n_max, budget), dtype=torch.uint8, device=device)

    # -- the four calls of the round --------------------------------------------------------
    def score(self, src: CacheView, cur_pos: torch.Tensor, scores: torch.Tensor, ws: torch.Tensor,
              raw: Optional[torch.Tensor] = None):
        S = cur_pos.shape[0]
        cv = src.c_view()
        assert cur_pos.dtype == torch.int64 and scores.dtype == torch.float32 and scores.is_contiguous()
        assert scores.numel() == self.units(S) * cv.n_max
        if raw is not None:
            assert raw.dtype == torch.float32 and raw.is_contiguous()
            assert raw.numel() == self.units(S) * cv.n_max * self.group_size
        _check(lib().tri_score(self._h, ctypes.byref(cv), S, _ptr(cur_pos), _ptr(scores), _ptr(raw), _ptr(ws),
                               ws.numel(), _stream()), "tri_score")

    STATIC_SCRATCH_BYTES = 16 * 1024 * 1024

    def score_static_bytes(self, S: int, n_max: int) -> int:
        """Bytes of the built-in array score_static would use for this shape."""
        return int(lib().tri_score_static_bytes(self._h, S, n_max))

    def score_static(self, src: CacheView, cur_pos: torch.Tensor, scores: torch.Tensor,
                     raw: Optional[torch.Tensor] = None):
        """tri_score_static: like score() but with no workspace tensor -- the library's built-in
        16 MiB device array is the scratch.  For callers that cannot obtain device memory at call
        time (an engine whose page pool owns all of HBM, a plug-in barred from the host's allocator).
        This method creates no torch tensor.  Shapes that need more scratch raise TriError(3) with
        both sizes in the message.  Calls share that array: do not let two of them overlap on the GPU.
        Make the first call on a device during set-up (it looks up the array's address)."""
        S = cur_pos.shape[0]
        cv = src.c_view()
        assert cur_pos.dtype == torch.int64 and scores.dtype == torch.float32 and scores.is_contiguous()
        assert scores.numel() == self.units(S) * cv.n_max
        if raw is not None:
            assert raw.dtype == torch.float32 and raw.is_contiguous()
            assert raw.numel() == self.units(S) * cv.n_max * self.group_size
        code = lib().tri_score_static(self._h, ctypes.byref(cv), S, _ptr(cur_pos), _ptr(scores), _ptr(raw), _stream())
        if code == 3:
            raise TriError(code, "tri_score_static", lib().tri_last_cuda_error().decode())
        _check(code, "tri_score_static")

    def select(self, scores: torch.Tensor, seq_lens: torch.Tensor, n_max: int, budget: int,
               kept_idx: torch.Tensor, kept_cnt: torch.Tensor, ws: Optional[torch.Tensor] = None,
               unit_budgets: Optional[torch.Tensor] = None):
        S = seq_lens.shape[0]
        assert scores.dtype == torch.float32 and scores.is_contiguous() and scores.numel() == self.units(S) * n_max
        assert kept_idx.dtype == torch.int32 and kept_idx.numel() == self.units(S) * budget
        assert kept_cnt.dtype == torch.int32 and kept_cnt.numel() == self.units(S)
        if unit_budgets is not None:
            assert unit_budgets.dtype == torch.int32 and unit_budgets.numel() == self.units(S) and unit_budgets.is_contiguous()
            _check(lib().tri_select_budgets(self._h, _ptr(scores), _ptr(seq_lens), S, n_max, budget, _ptr(unit_budgets),
                                            _ptr(kept_idx), _ptr(kept_cnt), _stream()), "tri_select_budgets")
            return
        _check(lib().tri_select(self._h, _ptr(scores), _ptr(seq_lens), S, n_max, budget, _ptr(kept_idx),
                                _ptr(kept_cnt), _ptr(ws), 0 if ws is None else ws.numel(), _stream()), "tri_select")

    def compact(self, src: CacheView, kept_idx: torch.Tensor, kept_cnt: torch.Tensor, S: int, budget: int,
                dst: CacheView, new_seq_lens: Optional[torch.Tensor] = None):
        cs, cd = src.c_view(), dst.c_view()
        assert kept_idx.dtype == torch.int32 and kept_idx.numel() == self.units(S) * budget
        assert kept_cnt.dtype == torch.int32 and kept_cnt.numel() == self.units(S)
        _check(lib().tri_compact(self._h, ctypes.byref(cs), _ptr(kept_idx), _ptr(kept_cnt), S, budget,
                                 ctypes.byref(cd), _ptr(new_seq_lens), _stream()), "tri_compact")

    def compress(self, src: CacheView, cur_pos: torch.Tensor, budget: int, dst: CacheView, ws: torch.Tensor,
                 kept_idx: Optional[torch.Tensor] = None, kept_cnt: Optional[torch.Tensor] = None,
                 new_seq_lens: Optional[torch.Tensor] = None, device_status: Optional[torch.Tensor] = None,
                 unit_budgets: Optional[torch.Tensor] = None):
        S = cur_pos.shape[0]
        cs, cd = src.c_view(), dst.c_view()
        assert cur_pos.dtype == torch.int64
        if kept_idx is not None:
            assert kept_idx.dtype == torch.int32 and kept_idx.numel() == self.units(S) * budget
        if kept_cnt is not None:
            assert kept_cnt.dtype == torch.int32 and kept_cnt.numel() == self.units(S)
        if unit_budgets is not None:
            assert unit_budgets.dtype == torch.int32 and unit_budgets.numel() == self.units(S) and unit_budgets.is_contiguous()
            _check(lib().tri_compress_budgets(self._h, ctypes.byref(cs), S, _ptr(cur_pos), budget, _ptr(unit_budgets),
                                              ctypes.byref(cd), _ptr(kept_idx), _ptr(kept_cnt), _ptr(new_seq_lens),
                                              _ptr(device_status), _ptr(ws), ws.numel(), _stream()), "tri_compress_budgets")
            return
        _check(lib().tri_compress(self._h, ctypes.byref(cs), S, _ptr(cur_pos), budget, ctypes.byref(cd),
                                  _ptr(kept_idx), _ptr(kept_cnt), _ptr(new_seq_lens), _ptr(device_status),
                                  _ptr(ws), ws.numel(), _stream()), "tri_compress")

    def compress_windowed(self, src: CacheView, cur_pos: torch.Tensor, budget: int, decoded: torch.Tensor, step: int,
                          beta: int, dst: CacheView, ws: torch.Tensor, kept_idx: Optional[torch.Tensor] = None,
                          kept_cnt: Optional[torch.Tensor] = None, new_seq_lens: Optional[torch.Tensor] = None,
                          device_status: Optional[torch.Tensor] = None):
        """tri_compress behind the device-side window trigger: sequences whose counter reaches beta and whose cache
        exceeds the budget are compressed, the others are left alone."""
        S = cur_pos.shape[0]
        cs, cd = src.c_view(), dst.c_view()
        assert cur_pos.dtype == torch.int64 and decoded.dtype == torch.int32 and decoded.numel() == S
        _check(lib().tri_compress_windowed(self._h, ctypes.byref(cs), S, _ptr(cur_pos), budget, _ptr(decoded), step, beta,
                                           ctypes.byref(cd), _ptr(kept_idx), _ptr(kept_cnt), _ptr(new_seq_lens),
                                           _ptr(device_status), _ptr(ws), ws.numel(), _stream()), "tri_compress_windowed")

    def compress_host(self, src_host: CacheView, src_dev: CacheView, cur_pos_host: torch.Tensor,
                      cur_pos_dev: torch.Tensor, budget: int, dst_host: CacheView, dst_dev: CacheView,
                      kept_cnt_host: torch.Tensor, kept_cnt_dev: torch.Tensor, ws: torch.Tensor):
        S = cur_pos_host.shape[0]
        a, b, c, d = src_host.c_view(), src_dev.c_view(), dst_host.c_view(), dst_dev.c_view()
        _check(lib().tri_compress_host(self._h, ctypes.byref(a), ctypes.byref(b), S, _ptr(cur_pos_host),
                                       _ptr(cur_pos_dev), budget, ctypes.byref(c), ctypes.byref(d),
                                       _ptr(kept_cnt_host), _ptr(kept_cnt_dev), _ptr(ws), ws.numel(), _stream()),
               "tri_compress_host")

    KERNELS = ("fold_phasors", "score", "normalize", "select", "compact")

    def profile_begin(self):
        _check(lib().tri_profile_begin(self._h), "tri_profile_begin")

    def profile_read(self):
        """Durations (ms) of the 5 kernels of the last compress() call; waits for that call."""
        ms = (ctypes.c_float * 5)()
        _check(lib().tri_profile_read(self._h, ctypes.cast(ms, ctypes.c_void_p)), "tri_profile_read")
        return dict(zip(self.KERNELS, [float(x) for x in ms]))

    def profile_end(self):
        _check(lib().tri_profile_end(self._h), "tri_profile_end")

    def compress_launches(self, src: CacheView, S: int, dst: CacheView) -> int:
        a, b = src.c_view(), dst.c_view()
        return int(lib().tri_compress_launches(self._h, ctypes.byref(a), S, ctypes.byref(b)))

    def set_score_kernel(self, which: int):
        """0: tcgen05 scoring kernel (default); 1: mma.sync scoring kernel.  Call before workspace()."""
        _check(lib().tri_set_score_kernel(self._h, which), "tri_set_score_kernel")

    def set_pipeline(self, ranges: int):
        """0: ranges chosen per call (default); 1: the whole round on the caller's stream; n: n unit ranges with
        selection and compaction on the context's side stream."""
        _check(lib().tri_set_pipeline(self._h, ranges), "tri_set_pipeline")


class Calibrator:
    """Streaming calibration statistics of one layer's query heads (Section 4.1): feed chunks of pre-RoPE
    queries [T, n_heads, 128] (bf16 or fp32) with add(), read E[q_f], E|q_f| and R_f with result()."""

    def __init__(self, n_heads: int, pair_layout: int = 0, device="cuda"):
        self.n_heads, self.pair_layout, self.device = n_heads, pair_layout, torch.device(device)
        self.state = torch.empty(lib().tri_calib_state_bytes(n_heads) // 8, dtype=torch.float64, device=self.device)
        self._ws = None
        self.reset()

    def reset(self):
        _check(lib().tri_calib_reset(_ptr(self.state), self.n_heads, _stream()), "tri_calib_reset")

    def add(self, q: torch.Tensor):
        assert q.dim() == 3 and q.shape[1] == self.n_heads and q.shape[2] == 128 and q.stride(2) == 1
        assert q.dtype in (torch.bfloat16, torch.float32) and q.device == self.state.device
        T = q.shape[0]
        need = int(lib().tri_calib_workspace_bytes(self.n_heads, T))
        if self._ws is None or self._ws.numel() * 8 < need:
            self._ws = torch.empty((need + 7) // 8, dtype=torch.float64, device=self.device)
        _check(lib().tri_calib_accumulate(_ptr(q), 0 if q.dtype == torch.bfloat16 else 1, T, self.n_heads, q.stride(0),
                                          q.stride(1), self.pair_layout, _ptr(self.state), _ptr(self._ws),
                                          self._ws.numel() * 8, _stream()), "tri_calib_accumulate")

    def result(self):
        """(q_center [n_heads, 128], q_mean_norm [n_heads, 64], mrl [n_heads, 64]) as fp32 device tensors."""
        qc = torch.empty(self.n_heads, 128, dtype=torch.float32, device=self.device)
        qn = torch.empty(self.n_heads, 64, dtype=torch.float32, device=self.device)
        r = torch.empty(self.n_heads, 64, dtype=torch.float32, device=self.device)
        _check(lib().tri_calib_finalize(_ptr(self.state), self.n_heads, self.pair_layout, _ptr(qc), _ptr(qn), _ptr(r),
                                        _stream()), "tri_calib_finalize")
        return qc, qn, r
