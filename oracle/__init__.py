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
    lib.oracle_merge_embeddings.argtypes = [vp, vp, sz, i32p, i32, i32, i32, i32, i32, vp]
    lib.oracle_merge_embeddings.restype = i32
    lib.oracle_compact_pos_planes.argtypes = [i32p, i32, i32, i32, i32p, i32, i32p]
    lib.oracle_compact_pos_planes.restype = i32
    lib.oracle_compact_kv_heads.argtypes = [vpp, vpp, vpp, vpp, i32, i32, i32, i32, i32, sz, i32p]
    lib.oracle_compact_kv_heads.restype = i32
    lib.oracle_compact_kv_paged.argtypes = [vpp, vpp, vpp, vpp, i32, i32, i32, i32, sz, i32p, i32p,
                                            i32, i32, i32]
    lib.oracle_compact_kv_paged.restype = i32
    lib.oracle_floor_from_ratio.argtypes = [i32] * 4
    lib.oracle_floor_from_ratio.restype = ctypes.c_int64
    lib.oracle_select_ragged.argtypes = [f32p, i32, i32p, i32p, i32p]
    lib.oracle_select_ragged.restype = i32
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

    def merge_embeddings(self, text: np.ndarray, visual: np.ndarray, keep_idx: np.ndarray,
                         vis_start: int) -> np.ndarray:
        """text [n_seq, seq_len, row], visual [n_seq, n_vis, row] -> [n_seq, seq_len - n_vis + k, row]."""
        text, visual = np.ascontiguousarray(text), np.ascontiguousarray(visual)
        keep_idx = np.ascontiguousarray(keep_idx, dtype=np.int32)
        n_seq, seq_len, row = text.shape
        n_vis, k = visual.shape[1], keep_idx.shape[1]
        assert visual.shape == (n_seq, n_vis, row) and visual.dtype == text.dtype
        out = np.zeros((n_seq, seq_len - n_vis + k, row), dtype=text.dtype)
        _check(self.h.oracle_merge_embeddings(text.ctypes.data, visual.ctypes.data, row * text.itemsize,
                                              _i32p(keep_idx), n_seq, seq_len, vis_start, n_vis, k,
                                              out.ctypes.data), "oracle_merge_embeddings")
        return out

    def compact_pos_planes(self, pos: np.ndarray, seq_idx: np.ndarray) -> np.ndarray:
        """pos int32 [n_planes, n_seq, seq_len], seq_idx [n_seq, s_out] -> [n_planes, n_seq, s_out]."""
        pos = np.ascontiguousarray(pos, dtype=np.int32)
        seq_idx = np.ascontiguousarray(seq_idx, dtype=np.int32)
        n_planes, n_seq, seq_len = pos.shape
        s_out = seq_idx.shape[1]
        out = np.full((n_planes, n_seq, s_out), -1, dtype=np.int32)
        _check(self.h.oracle_compact_pos_planes(_i32p(pos), n_planes, n_seq, seq_len, _i32p(seq_idx),
                                                s_out, _i32p(out)), "oracle_compact_pos_planes")
        return out

    def compact_kv_heads(self, k_src: Sequence[np.ndarray], v_src: Sequence[np.ndarray],
                         seq_idx: np.ndarray):
        """Per layer K and V as [n_seq, n_heads, seq_len, d] -> lists of [n_seq, n_heads, s_out, d]."""
        seq_idx = np.ascontiguousarray(seq_idx, dtype=np.int32)
        n_seq, s_out = seq_idx.shape
        n_layers = len(k_src)
        k_src = [np.ascontiguousarray(a) for a in k_src]
        v_src = [np.ascontiguousarray(a) for a in v_src]
        a0 = k_src[0]
        _, n_heads, seq_len, d = a0.shape
        assert all(a.shape == a0.shape and a.dtype == a0.dtype for a in k_src + v_src)
        k_dst = [np.zeros((n_seq, n_heads, s_out, d), dtype=a0.dtype) for _ in range(n_layers)]
        v_dst = [np.zeros((n_seq, n_heads, s_out, d), dtype=a0.dtype) for _ in range(n_layers)]
        table = lambda arrs: (ctypes.c_void_p * n_layers)(*[a.ctypes.data for a in arrs])
        _check(self.h.oracle_compact_kv_heads(table(k_src), table(v_src), table(k_dst), table(v_dst),
                                              n_layers, n_seq, n_heads, seq_len, s_out,
                                              d * a0.itemsize, _i32p(seq_idx)), "oracle_compact_kv_heads")
        return k_dst, v_dst

    def compact_kv_paged(self, k_src: Sequence[np.ndarray], v_src: Sequence[np.ndarray],
                         seq_idx: np.ndarray, block_table: np.ndarray, page_size: int,
                         k_cache: Sequence[np.ndarray], v_cache: Sequence[np.ndarray]) -> None:
        """Writes the kept rows of src [n_seq, seq_len, row] into caches [n_pages, page_size, row]
        (modified in place) through block_table int32 [n_seq, max_pages_per_seq]."""
        seq_idx = np.ascontiguousarray(seq_idx, dtype=np.int32)
        block_table = np.ascontiguousarray(block_table, dtype=np.int32)
        n_seq, s_out = seq_idx.shape
        n_layers = len(k_src)
        k_src = [np.ascontiguousarray(a) for a in k_src]
        v_src = [np.ascontiguousarray(a) for a in v_src]
        a0, c0 = k_src[0], k_cache[0]
        seq_len, row = a0.shape[1], a0.shape[2]
        assert all(c.flags.c_contiguous and c.shape == c0.shape and c.dtype == a0.dtype
                   for c in list(k_cache) + list(v_cache))
        assert c0.shape[1] == page_size and c0.shape[2] == row and block_table.shape[0] == n_seq
        table = lambda arrs: (ctypes.c_void_p * n_layers)(*[a.ctypes.data for a in arrs])
        _check(self.h.oracle_compact_kv_paged(table(k_src), table(v_src), table(k_cache), table(v_cache),
                                              n_layers, n_seq, seq_len, s_out, row * a0.itemsize,
                                              _i32p(seq_idx), _i32p(block_table), block_table.shape[1],
                                              page_size, c0.shape[0]), "oracle_compact_kv_paged")

    def floor_from_ratio(self, region_h: int, region_w: int, num: int, den: int) -> int:
        return int(self.h.oracle_floor_from_ratio(region_h, region_w, num, den))

    def select_ragged(self, scores: np.ndarray, descs: Sequence[Sequence[int]]):
        """scores fp32 [sum n] concatenated, descs [(t, h, w, region_h, region_w, m, k)] ->
        (segment-local keep indices [sum k], the same tokens numbered over the concatenation)."""
        scores = np.ascontiguousarray(scores, dtype=np.float32).reshape(-1)
        d = np.ascontiguousarray(np.asarray(descs, dtype=np.int32).reshape(-1, 7))
        assert scores.size == int(sum(int(r[0]) * int(r[1]) * int(r[2]) for r in d))
        total_k = int(d[:, 6].sum()) if len(d) else 0
        keep = np.full(total_k, -1, dtype=np.int32)
        flat = np.full(total_k, -1, dtype=np.int32)
        _check(self.h.oracle_select_ragged(_f32p(scores), len(d), _i32p(d), _i32p(keep), _i32p(flat)),
               "oracle_select_ragged")
        return keep, flat

    def set_threads(self, n: int) -> int:
        return int(self.h.oracle_set_threads(n))


default = Oracle()
