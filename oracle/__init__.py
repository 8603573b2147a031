"""ctypes front end of the CPU oracle  --  TEST INFRASTRUCTURE, not product code.

Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It builds `civic_oracle.c` with gcc on first use and exposes its functions
on numpy arrays.  Nothing here touches CUDA or the product package.
"""

from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "civic_oracle.c")
_LIB = os.path.join(_HERE, "libcivic_oracle.so")

OK, ERR_ARG, ERR_K_RANGE, ERR_FLOOR_EXCEEDS_K, ERR_INDEX, ERR_NOMEM = range(6)


class OracleError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"{where}: oracle status {code}")
        self.code = code


def build(force: bool = False, defines: Sequence[str] = (), out: Optional[str] = None) -> str:
    """Compile the oracle (gcc -O2, OpenMP for the K/V unit loop). Returns the .so path.

    `defines`/`out` let a test build a deliberately broken copy (a planted mistake) to
    show that the pins notice it.
    """
    out = out or _LIB
    if not force and os.path.exists(out) and os.path.getmtime(out) >= os.path.getmtime(_SRC):
        return out
    cmd = ["gcc", "-std=gnu11", "-O2", "-fPIC", "-shared", "-fopenmp", "-Wall", "-Wextra",
           *[f"-D{d}" for d in defines], "-o", out, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return out


def _bind(path: str) -> ctypes.CDLL:
    lib = ctypes.CDLL(path)
    i32, f32p, i32p, vp, sz = (ctypes.c_int, ctypes.POINTER(ctypes.c_float),
                               ctypes.POINTER(ctypes.c_int32), ctypes.c_void_p, ctypes.c_size_t)
    vpp = ctypes.POINTER(ctypes.c_void_p)
    lib.oracle_score_cmp.argtypes = [ctypes.c_float, ctypes.c_float]
    lib.oracle_score_cmp.restype = i32
    lib.oracle_reserved_count.argtypes = [i32] * 6
    lib.oracle_reserved_count.restype = ctypes.c_int64
    lib.oracle_select.argtypes = [f32p, i32, i32, i32, i32, i32, i32, i32, i32, i32p]
    lib.oracle_select.restype = i32
    lib.oracle_compact.argtypes = [vp, sz, i32p, i32p, i32, i32, i32, vp, i32p]
    lib.oracle_compact.restype = i32
    lib.oracle_seq_indices.argtypes = [i32p, i32, i32, i32, i32, i32, i32p]
    lib.oracle_seq_indices.restype = i32
    lib.oracle_compact_kv.argtypes = [vpp, vpp, vpp, vpp, i32, i32, i32, i32, sz, i32p]
    lib.oracle_compact_kv.restype = i32
    lib.oracle_set_threads.argtypes = [i32]
    lib.oracle_set_threads.restype = i32
    return lib


_lib: Optional[ctypes.CDLL] = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = _bind(build())
    return _lib


def load_variant(defines: Sequence[str], tag: str) -> "Oracle":
    """An oracle built with extra -D flags (used to plant mistakes in tests)."""
    path = os.path.join(_HERE, f"libcivic_oracle_{tag}.so")
    return Oracle(_bind(build(force=True, defines=defines, out=path)))


def _f32p(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_float))


def _i32p(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)) if a is not None else None


def _check(rc: int, where: str) -> None:
    if rc != OK:
        raise OracleError(rc, where)


class Oracle:
    """The oracle's functions on numpy arrays."""

    def __init__(self, handle: Optional[ctypes.CDLL] = None):
        self._h = handle

    @property
    def h(self) -> ctypes.CDLL:
        return self._h if self._h is not None else lib()

    def score_cmp(self, a: float, b: float) -> int:
        return int(self.h.oracle_score_cmp(ctypes.c_float(a), ctypes.c_float(b)))

    def score_cmp_bits(self, a_bits: int, b_bits: int) -> int:
        a = np.array([a_bits], dtype=np.uint32).view(np.float32)
        b = np.array([b_bits], dtype=np.uint32).view(np.float32)
        fa, fb = ctypes.c_float(), ctypes.c_float()
        ctypes.memmove(ctypes.byref(fa), a.ctypes.data, 4)
        ctypes.memmove(ctypes.byref(fb), b.ctypes.data, 4)
        return int(self.h.oracle_score_cmp(fa, fb))

    def reserved_count(self, t, h, w, region_h, region_w, m) -> int:
        return int(self.h.oracle_reserved_count(t, h, w, region_h, region_w, m))

    def select(self, scores: np.ndarray, t: int, h: int, w: int, region_h: int, region_w: int,
               m: int, k: int) -> np.ndarray:
        """scores fp32 [n_seg, n] -> ascending keep indices int32 [n_seg, k]."""
        scores = np.ascontiguousarray(scores, dtype=np.float32)
        assert scores.ndim == 2 and scores.shape[1] == t * h * w
        out = np.full((scores.shape[0], max(k, 0)), -1, dtype=np.int32)
        _check(self.h.oracle_select(_f32p(scores), scores.shape[0], t, h, w, region_h, region_w,
                                    m, k, _i32p(out)), "oracle_select")
        return out

    def compact(self, hidden: Optional[np.ndarray], pos_ids: Optional[np.ndarray],
                keep_idx: np.ndarray):
        """hidden [n_seg, n, row] (any dtype, rows are bytes), pos_ids int32 [n_seg, n, 3]."""
        keep_idx = np.ascontiguousarray(keep_idx, dtype=np.int32)
        n_seg, k = keep_idx.shape
        h_out = p_out = None
        n = None
        row_bytes = 0
        if hidden is not None:
            hidden = np.ascontiguousarray(hidden)
            assert hidden.ndim == 3 and hidden.shape[0] == n_seg
            n = hidden.shape[1]
            row_bytes = hidden.shape[2] * hidden.itemsize
            h_out = np.zeros((n_seg, k, hidden.shape[2]), dtype=hidden.dtype)
        if pos_ids is not None:
            pos_ids = np.ascontiguousarray(pos_ids, dtype=np.int32)
            assert pos_ids.shape[0] == n_seg and pos_ids.shape[2] == 3
            assert n is None or n == pos_ids.shape[1]
            n = pos_ids.shape[1]
            p_out = np.zeros((n_seg, k, 3), dtype=np.int32)
        _check(self.h.oracle_compact(
            hidden.ctypes.data if hidden is not None else None, row_bytes, _i32p(pos_ids),
            _i32p(keep_idx), n_seg, n, k,
            h_out.ctypes.data if h_out is not None else None, _i32p(p_out)), "oracle_compact")
        return h_out, p_out

    def seq_indices(self, keep_idx: np.ndarray, seq_len: int, vis_start: int, n_vis: int) -> np.ndarray:
        keep_idx = np.ascontiguousarray(keep_idx, dtype=np.int32)
        n_seq, k = keep_idx.shape
        out = np.full((n_seq, seq_len - n_vis + k), -1, dtype=np.int32)
        _check(self.h.oracle_seq_indices(_i32p(keep_idx), n_seq, k, seq_len, vis_start, n_vis,
                                         _i32p(out)), "oracle_seq_indices")
        return out

    def compact_kv(self, k_src: Sequence[np.ndarray], v_src: Sequence[np.ndarray],
                   seq_idx: np.ndarray):
        """Per layer K and V as [n_seq, seq_len, row] arrays -> lists of [n_seq, s_out, row]."""
        seq_idx = np.ascontiguousarray(seq_idx, dtype=np.int32)
        n_seq, s_out = seq_idx.shape
        n_layers = len(k_src)
        assert len(v_src) == n_layers
        k_src = [np.ascontiguousarray(a) for a in k_src]
        v_src = [np.ascontiguousarray(a) for a in v_src]
        if n_layers:
            a0 = k_src[0]
            assert a0.ndim == 3 and a0.shape[0] == n_seq
            seq_len, row, dt = a0.shape[1], a0.shape[2], a0.dtype
            assert all(a.shape == a0.shape and a.dtype == dt for a in k_src + v_src)
        else:
            seq_len, row, dt = 0, 0, np.uint8
        k_dst = [np.zeros((n_seq, s_out, row), dtype=dt) for _ in range(n_layers)]
        v_dst = [np.zeros((n_seq, s_out, row), dtype=dt) for _ in range(n_layers)]

        def table(arrs):
            return (ctypes.c_void_p * max(n_layers, 1))(*[a.ctypes.data for a in arrs])

        _check(self.h.oracle_compact_kv(table(k_src), table(v_src), table(k_dst), table(v_dst),
                                        n_layers, n_seq, seq_len, s_out,
                                        row * np.dtype(dt).itemsize, _i32p(seq_idx)),
               "oracle_compact_kv")
        return k_dst, v_dst

    def set_threads(self, n: int) -> int:
        return int(self.h.oracle_set_threads(n))


default = Oracle()
