"""float64 CPU oracle for the TriAttention KV-compression round (ctypes front end).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the benchmark's
CPU-baseline / reference legs, never by the CUDA library or its Python binding.  All
arithmetic lives in ``tri_oracle.c`` (plain C, double precision, the paper's formulas
term by term); this module only compiles it with gcc and marshals numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "tri_oracle.c"
_LIB = _HERE / "libtri_oracle.so"
_lib = None

#: Future-offset set of Section 4.2: D = {1, 2, 4, ..., 2^16} (17 offsets).
DEFAULT_OFFSETS = np.array([1 << j for j in range(17)], dtype=np.int64)


def build(force: bool = False) -> Path:
    """Compile ``tri_oracle.c`` into a shared object next to it (gcc -O2 -fopenmp)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", str(tmp), str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(str(build()))
    c_d, c_i, c_i64 = ctypes.c_double, ctypes.c_int, ctypes.c_int64
    P = ctypes.c_void_p
    lib.tri_oracle_omega.argtypes = [c_d, c_i, P]
    lib.tri_oracle_omega.restype = None
    lib.tri_oracle_bf16_to_f64.argtypes = [P, c_i64, P]
    lib.tri_oracle_bf16_to_f64.restype = None
    lib.tri_oracle_unrotate.argtypes = [P, P, c_i64, c_i, c_d, c_i, P]
    lib.tri_oracle_unrotate.restype = None
    lib.tri_oracle_s_trig.argtypes = [P, P, c_i, c_d, c_i, c_d]
    lib.tri_oracle_s_trig.restype = c_d
    lib.tri_oracle_s_norm.argtypes = [P, P, P, c_i, c_i, c_i]
    lib.tri_oracle_s_norm.restype = c_d
    lib.tri_oracle_score_raw.argtypes = [P, P, c_i64, c_i, c_i64, P, P, c_i, P, c_i, c_d, c_i, c_i, P]
    lib.tri_oracle_score_raw.restype = None
    lib.tri_oracle_normalize.argtypes = [P, c_i, c_i64, P, P]
    lib.tri_oracle_normalize.restype = None
    lib.tri_oracle_select.argtypes = [P, c_i64, c_i64, P]
    lib.tri_oracle_select.restype = c_i64
    lib.tri_oracle_compact.argtypes = [P, c_i64, P, c_i64, P]
    lib.tri_oracle_compact.restype = None
    lib.tri_oracle_unit_bf16.argtypes = [P, P, c_i64, c_i, c_i64, P, P, c_i, P, c_i, c_d, c_i, c_i,
                                         c_i64, P, P, P]
    lib.tri_oracle_unit_bf16.restype = c_i64
    lib.tri_oracle_unit_e4m3.argtypes = lib.tri_oracle_unit_bf16.argtypes
    lib.tri_oracle_unit_e4m3.restype = c_i64
    lib.tri_oracle_e4m3_to_f64.argtypes = [P, c_i64, P]
    lib.tri_oracle_e4m3_to_f64.restype = None
    lib.tri_oracle_calibrate.argtypes = [P, c_i64, c_i, c_i, P, P, P]
    lib.tri_oracle_calibrate.restype = None
    lib.tri_oracle_num_threads.argtypes = []
    lib.tri_oracle_num_threads.restype = c_i
    _lib = lib
    return lib


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _i64(a):
    return np.ascontiguousarray(a, dtype=np.int64)


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def num_threads() -> int:
    return int(_load().tri_oracle_num_threads())


def omega(theta: float, d: int) -> np.ndarray:
    out = np.empty(d // 2, dtype=np.float64)
    _load().tri_oracle_omega(float(theta), int(d), _p(out))
    return out


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    out = np.empty(bits.shape, dtype=np.float64)
    _load().tri_oracle_bf16_to_f64(_p(bits), bits.size, _p(out))
    return out


def unrotate(k_post, pos, theta: float, layout: int = 0) -> np.ndarray:
    k_post = _f64(k_post)
    pos = _i64(pos)
    N, d = k_post.shape
    assert pos.shape == (N,)
    out = np.empty_like(k_post)
    _load().tri_oracle_unrotate(_p(k_post), _p(pos), N, d, float(theta), int(layout), _p(out))
    return out


def s_trig(k_pre, q_center, theta: float, Delta: float, layout: int = 0) -> float:
    k_pre, q_center = _f64(k_pre), _f64(q_center)
    return float(_load().tri_oracle_s_trig(_p(k_pre), _p(q_center), k_pre.shape[-1], float(theta),
                                           int(layout), float(Delta)))


def s_norm(k_pre, q_center, q_mean_norm, layout: int = 0, variant: int = 0) -> float:
    k_pre, q_center, q_mean_norm = _f64(k_pre), _f64(q_center), _f64(q_mean_norm)
    return float(_load().tri_oracle_s_norm(_p(k_pre), _p(q_center), _p(q_mean_norm), k_pre.shape[-1],
                                           int(layout), int(variant)))


def score_raw(k_pre, pos, p_q: int, q_center, q_mean_norm, offsets=DEFAULT_OFFSETS, theta: float = 1e6,
              layout: int = 0, norm_variant: int = 0) -> np.ndarray:
    """S~^(g)(k) for one unit: returns raw[G, N]."""
    k_pre, pos = _f64(k_pre), _i64(pos)
    q_center, q_mean_norm, offsets = _f64(q_center), _f64(q_mean_norm), _i64(offsets)
    N, d = k_pre.shape
    G = q_center.shape[0]
    assert q_center.shape == (G, d) and q_mean_norm.shape == (G, d // 2) and pos.shape == (N,)
    raw = np.empty((G, N), dtype=np.float64)
    _load().tri_oracle_score_raw(_p(k_pre), _p(pos), N, d, int(p_q), _p(q_center), _p(q_mean_norm), G,
                                 _p(offsets), offsets.size, float(theta), int(layout), int(norm_variant),
                                 _p(raw))
    return raw


def normalize(raw):
    """GQA z-score + max: returns (zscore[G, N], s_final[N])."""
    raw = _f64(raw)
    G, N = raw.shape
    z = np.empty((G, N), dtype=np.float64)
    s = np.empty(N, dtype=np.float64)
    _load().tri_oracle_normalize(_p(raw), G, N, _p(z), _p(s))
    return z, s


def select(s_final, B: int) -> np.ndarray:
    s_final = _f64(s_final)
    N = s_final.shape[0]
    idx = np.empty(max(min(N, int(B)), 0), dtype=np.int32)
    cnt = _load().tri_oracle_select(_p(s_final), N, int(B), _p(idx))
    assert cnt == idx.size
    return idx


def compact(rows: np.ndarray, kept_idx) -> np.ndarray:
    """Gather rows[kept_idx] as opaque byte records (bit copies)."""
    rows = np.ascontiguousarray(rows)
    kept_idx = np.ascontiguousarray(kept_idx, dtype=np.int32)
    row_bytes = rows.strides[0] if rows.ndim > 1 else rows.itemsize
    out = np.empty((kept_idx.size,) + rows.shape[1:], dtype=rows.dtype)
    _load().tri_oracle_compact(_p(rows), row_bytes, _p(kept_idx), kept_idx.size, _p(out))
    return out


def unit_bf16(k_post_bits, pos, p_q: int, q_center, q_mean_norm, B: int, offsets=DEFAULT_OFFSETS,
              theta: float = 1e6, layout: int = 0, norm_variant: int = 0):
    """Whole round for one unit cached post-RoPE in bf16 (given as uint16 bit patterns).

    Returns (raw[G, N], s_final[N], kept_idx[min(B, N)]).
    """
    k_post_bits = np.ascontiguousarray(k_post_bits, dtype=np.uint16)
    pos = _i64(pos)
    q_center, q_mean_norm, offsets = _f64(q_center), _f64(q_mean_norm), _i64(offsets)
    N, d = k_post_bits.shape
    G = q_center.shape[0]
    assert q_center.shape == (G, d) and q_mean_norm.shape == (G, d // 2) and pos.shape == (N,)
    raw = np.empty((G, N), dtype=np.float64)
    s = np.empty(N, dtype=np.float64)
    idx = np.empty(max(min(N, int(B)), 0), dtype=np.int32)
    cnt = _load().tri_oracle_unit_bf16(_p(k_post_bits), _p(pos), N, d, int(p_q), _p(q_center),
                                       _p(q_mean_norm), G, _p(offsets), offsets.size, float(theta),
                                       int(layout), int(norm_variant), int(B), _p(raw), _p(s), _p(idx))
    assert cnt == idx.size
    return raw, s, idx


def e4m3_to_f64(bits: np.ndarray) -> np.ndarray:
    """e4m3 bit patterns (uint8) -> the values they encode."""
    bits = np.ascontiguousarray(bits, dtype=np.uint8)
    out = np.empty(bits.shape, dtype=np.float64)
    _load().tri_oracle_e4m3_to_f64(_p(bits), bits.size, _p(out))
    return out


def unit_e4m3(k_post_bits, pos, p_q: int, q_center, q_mean_norm, B: int, offsets=DEFAULT_OFFSETS,
              theta: float = 1e6, layout: int = 0, norm_variant: int = 0):
    """unit_bf16 for a unit cached post-RoPE in e4m3 (given as uint8 bit patterns)."""
    k_post_bits = np.ascontiguousarray(k_post_bits, dtype=np.uint8)
    pos = _i64(pos)
    q_center, q_mean_norm, offsets = _f64(q_center), _f64(q_mean_norm), _i64(offsets)
    N, d = k_post_bits.shape
    G = q_center.shape[0]
    assert q_center.shape == (G, d) and q_mean_norm.shape == (G, d // 2) and pos.shape == (N,)
    raw = np.empty((G, N), dtype=np.float64)
    s = np.empty(N, dtype=np.float64)
    idx = np.empty(max(min(N, int(B)), 0), dtype=np.int32)
    cnt = _load().tri_oracle_unit_e4m3(_p(k_post_bits), _p(pos), N, d, int(p_q), _p(q_center),
                                       _p(q_mean_norm), G, _p(offsets), offsets.size, float(theta),
                                       int(layout), int(norm_variant), int(B), _p(raw), _p(s), _p(idx))
    assert cnt == idx.size
    return raw, s, idx


def calibrate(q, layout: int = 0):
    """Calibration statistics of one query head from its pre-RoPE queries q[T, d]:
    returns (center[d], mean_norm[d/2], mrl[d/2]) = (E[q_f], E|q_f|, R_f)."""
    q = _f64(q)
    T, d = q.shape
    center = np.empty(d, dtype=np.float64)
    mean_norm = np.empty(d // 2, dtype=np.float64)
    mrl = np.empty(d // 2, dtype=np.float64)
    _load().tri_oracle_calibrate(_p(q), T, d, int(layout), _p(center), _p(mean_norm), _p(mrl))
    return center, mean_norm, mrl
