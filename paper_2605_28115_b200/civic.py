"""Thin ctypes binding of libcivic.so: argument marshalling only.

Every step of the path runs inside the CUDA library; torch is used for device memory and
streams.  The functions carry the names of the C entry points (include/civic.h).  There is
no CPU fallback: if the library cannot be loaded, or a tensor is neither on a CUDA device
nor in pinned host memory (which the GPU reads and writes directly over PCIe), the call raises.
"""

from __future__ import annotations

import ctypes
import dataclasses
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcivic.so")

CIVIC_OK = 0
STATUS_NAMES = ("CIVIC_OK", "CIVIC_ERR_INVALID_ARG", "CIVIC_ERR_K_RANGE", "CIVIC_ERR_FLOOR_EXCEEDS_K",
                "CIVIC_ERR_ALIGNMENT", "CIVIC_ERR_UNSUPPORTED", "CIVIC_ERR_CUDA", "CIVIC_ERR_WORKSPACE")

# every symbol include/civic.h declares
EXPORTS = ("civic_select", "civic_select_max_tokens", "civic_reserved_count", "civic_compact",
           "civic_seq_indices", "civic_compact_kv", "civic_status_string", "civic_last_cuda_error",
           "civic_launch_count", "civic_select_seq", "civic_set_programmatic_launch",
           "civic_compact_kv_heads", "civic_compact_kv_paged", "civic_merge_embeddings",
           "civic_compact_pos_planes", "civic_select_large", "civic_select_workspace_bytes",
           "civic_select_ragged", "civic_floor_from_ratio",
           "civic_select_large_static", "civic_select_static_scratch_bytes",
           "civic_anchor_aggregate", "civic_anchor_aggregate_workspace_bytes",
           "civic_kv_compressed_attention", "civic_kv_compressed_attention_workspace_bytes",
           "civic_set_index_check", "civic_validate_indices", "civic_selftest_bounded_wait",
           "civic_anchor_prepared_bytes", "civic_anchor_prepare", "civic_anchor_aggregate_prepared",
           "civic_kv_attention_prepared_bytes", "civic_kv_attention_prepare", "civic_kv_compressed_attention_prepared")

INDEX_FAULTS = ("CIVIC_INDEX_OK", "CIVIC_INDEX_OUT_OF_RANGE", "CIVIC_INDEX_NOT_ASCENDING", "CIVIC_INDEX_BAD_PAGE")


class CivicError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"{where}: {name}{(' (' + detail + ')') if detail else ''}")
        self.status = status


class SelectDesc(ctypes.Structure):
    """civic_select_desc_t"""
    _fields_ = [("t", ctypes.c_int32), ("h", ctypes.c_int32), ("w", ctypes.c_int32),
                ("region_h", ctypes.c_int32), ("region_w", ctypes.c_int32),
                ("floor_per_region", ctypes.c_int32), ("k", ctypes.c_int32)]


_lib: Optional[ctypes.CDLL] = None


def load(path: Optional[str] = None) -> ctypes.CDLL:
    """Load libcivic.so (built in-tree by paper_2605_28115_b200.build). Raises if missing."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    path = path or LIB_PATH
    if not os.path.exists(path):
        raise RuntimeError(f"{path} not found: build it with `python -m paper_2605_28115_b200.build` "
                           "(there is no fallback implementation)")
    lib = ctypes.CDLL(path)
    vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
    vpp = ctypes.POINTER(ctypes.c_void_p)
    lib.civic_select.argtypes = [vp, i32, ctypes.POINTER(SelectDesc), vp, vp]
    lib.civic_select.restype = ctypes.c_int
    lib.civic_select_max_tokens.argtypes = []
    lib.civic_select_max_tokens.restype = i32
    lib.civic_reserved_count.argtypes = [ctypes.POINTER(SelectDesc)]
    lib.civic_reserved_count.restype = ctypes.c_int64
    lib.civic_compact.argtypes = [vp, sz, vp, vp, i32, i32, i32, vp, vp, vp]
    lib.civic_compact.restype = ctypes.c_int
    lib.civic_seq_indices.argtypes = [vp, i32, i32, i32, i32, i32, vp, vp]
    lib.civic_seq_indices.restype = ctypes.c_int
    lib.civic_compact_kv.argtypes = [vpp, vpp, vpp, vpp, i32, i32, i32, i32, sz, vp, vp]
    lib.civic_compact_kv.restype = ctypes.c_int
    lib.civic_status_string.argtypes = [ctypes.c_int]
    lib.civic_status_string.restype = ctypes.c_char_p
    lib.civic_last_cuda_error.argtypes = []
    lib.civic_last_cuda_error.restype = ctypes.c_char_p
    lib.civic_launch_count.argtypes = []
    lib.civic_launch_count.restype = ctypes.c_uint64
    lib.civic_select_seq.argtypes = [vp, i32, ctypes.POINTER(SelectDesc), i32, i32, vp, vp, vp]
    lib.civic_select_seq.restype = ctypes.c_int
    lib.civic_set_programmatic_launch.argtypes = [i32]
    lib.civic_set_programmatic_launch.restype = i32
    lib.civic_compact_kv_heads.argtypes = [vpp, vpp, vpp, vpp, i32, i32, i32, i32, i32, sz, vp, vp]
    lib.civic_compact_kv_heads.restype = ctypes.c_int
    lib.civic_compact_kv_paged.argtypes = [vpp, vpp, vpp, vpp, i32, i32, i32, i32, sz, vp, vp, i32, i32,
                                           i32, vp]
    lib.civic_compact_kv_paged.restype = ctypes.c_int
    lib.civic_merge_embeddings.argtypes = [vp, vp, sz, vp, i32, i32, i32, i32, i32, vp, vp]
    lib.civic_merge_embeddings.restype = ctypes.c_int
    lib.civic_compact_pos_planes.argtypes = [vp, i32, i32, i32, vp, i32, vp, vp]
    lib.civic_compact_pos_planes.restype = ctypes.c_int
    lib.civic_select_large.argtypes = [vp, i32, ctypes.POINTER(SelectDesc), vp, vp, sz, i32, vp]
    lib.civic_select_large.restype = ctypes.c_int
    lib.civic_select_workspace_bytes.argtypes = [ctypes.POINTER(SelectDesc), i32, i32]
    lib.civic_select_workspace_bytes.restype = sz
    lib.civic_select_ragged.argtypes = [vp, i32, ctypes.POINTER(SelectDesc), vp, vp, vp]
    lib.civic_select_ragged.restype = ctypes.c_int
    lib.civic_floor_from_ratio.argtypes = [i32, i32, i32, i32]
    lib.civic_floor_from_ratio.restype = i32
    lib.civic_select_large_static.argtypes = [vp, i32, ctypes.POINTER(SelectDesc), vp, i32, vp]
    lib.civic_select_large_static.restype = ctypes.c_int
    lib.civic_select_static_scratch_bytes.argtypes = []
    lib.civic_select_static_scratch_bytes.restype = sz
    lib.civic_anchor_aggregate.argtypes = [vp, vp, i32, i32, i32, i32, ctypes.c_float, vp, vp, vp, sz, vp, vp]
    lib.civic_anchor_aggregate.restype = ctypes.c_int
    lib.civic_anchor_aggregate_workspace_bytes.argtypes = [i32, i32, i32, i32]
    lib.civic_anchor_aggregate_workspace_bytes.restype = sz
    lib.civic_kv_compressed_attention.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, i32, vp, vp, sz, vp, vp]
    lib.civic_kv_compressed_attention.restype = ctypes.c_int
    lib.civic_kv_compressed_attention_workspace_bytes.argtypes = [i32, i32, i32, i32, i32]
    lib.civic_kv_compressed_attention_workspace_bytes.restype = sz
    lib.civic_anchor_prepared_bytes.argtypes = [i32, i32]
    lib.civic_anchor_prepared_bytes.restype = sz
    lib.civic_anchor_prepare.argtypes = [vp, i32, i32, vp, sz, vp]
    lib.civic_anchor_prepare.restype = ctypes.c_int
    lib.civic_anchor_aggregate_prepared.argtypes = [vp, vp, i32, i32, i32, i32, ctypes.c_float, vp, vp, vp, sz, vp, vp]
    lib.civic_anchor_aggregate_prepared.restype = ctypes.c_int
    lib.civic_kv_attention_prepared_bytes.argtypes = [i32, i32]
    lib.civic_kv_attention_prepared_bytes.restype = sz
    lib.civic_kv_attention_prepare.argtypes = [vp, i32, i32, vp, sz, vp]
    lib.civic_kv_attention_prepare.restype = ctypes.c_int
    lib.civic_kv_compressed_attention_prepared.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, i32, vp, vp, sz, vp, vp]
    lib.civic_kv_compressed_attention_prepared.restype = ctypes.c_int
    lib.civic_set_index_check.argtypes = [vp]
    lib.civic_set_index_check.restype = ctypes.c_int
    lib.civic_validate_indices.argtypes = [vp, i32, i32, i32, i32, vp, vp]
    lib.civic_validate_indices.restype = ctypes.c_int
    lib.civic_selftest_bounded_wait.argtypes = [ctypes.c_uint64, vp, vp]
    lib.civic_selftest_bounded_wait.restype = ctypes.c_int
    _lib = lib
    return lib


def _check(status: int, where: str) -> None:
    if status != CIVIC_OK:
        detail = load().civic_last_cuda_error().decode() if status == 6 else ""
        raise CivicError(status, where, detail)


def _dev_ptr(x: Optional[torch.Tensor], what: str, dtype: Optional[torch.dtype] = None) -> Optional[int]:
    if x is None:
        return None
    if not (x.is_cuda or x.is_pinned()):
        raise ValueError(f"{what} must be a CUDA tensor or pinned (device-mapped) host memory: "
                         "the kernels run on the GPU only, there is no CPU path")
    if not x.is_contiguous():
        raise ValueError(f"{what} must be contiguous")
    if dtype is not None and x.dtype != dtype:
        raise ValueError(f"{what} must be {dtype}, got {x.dtype}")
    return x.data_ptr()


def _device_of(*tensors) -> torch.device:
    """The CUDA device to launch on: that of the first CUDA tensor, else the current device."""
    for t in tensors:
        if t is not None and t.is_cuda:
            return t.device
    return torch.device("cuda", torch.cuda.current_device())


_raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    """cudaStream_t of `stream`, or of torch's current stream on the current device."""
    if stream is not None:
        return stream.cuda_stream
    if _raw_stream is not None:  # same value as current_stream().cuda_stream without building a Stream object
        return _raw_stream(torch.cuda.current_device())
    return torch.cuda.current_stream().cuda_stream


class _on_device:
    """Makes `device` current for the duration of a call; does nothing when it already is (the
    common case, and several microseconds cheaper than torch.cuda.device)."""

    __slots__ = ("index", "ctx")

    def __init__(self, device: torch.device):
        self.index = device.index if device.index is not None else torch.cuda.current_device()
        self.ctx = None

    def __enter__(self):
        if torch.cuda.current_device() != self.index:
            self.ctx = torch.cuda.device(self.index)
            self.ctx.__enter__()

    def __exit__(self, *exc):
        if self.ctx is not None:
            self.ctx.__exit__(*exc)


def launch_count() -> int:
    return int(load().civic_launch_count())


def select_max_tokens() -> int:
    return int(load().civic_select_max_tokens())


def reserved_count(desc: SelectDesc) -> int:
    return int(load().civic_reserved_count(ctypes.byref(desc)))


def civic_select(scores: torch.Tensor, desc: SelectDesc, keep_idx: Optional[torch.Tensor] = None,
                 stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """scores fp32 [n_seg, n] (CUDA) -> ascending keep indices int32 [n_seg, k]."""
    if scores.dim() != 2 or scores.shape[1] != desc.t * desc.h * desc.w:
        raise ValueError("scores must be [n_seg, t*h*w]")
    n_seg = scores.shape[0]
    if keep_idx is None:
        keep_idx = torch.empty((n_seg, max(desc.k, 0)), dtype=torch.int32, device=_device_of(scores))
    elif tuple(keep_idx.shape) != (n_seg, desc.k):
        raise ValueError("keep_idx must be [n_seg, k]")
    args = (_dev_ptr(scores, "scores", torch.float32), n_seg, ctypes.byref(desc),
            _dev_ptr(keep_idx, "keep_idx", torch.int32))
    with _on_device(_device_of(scores, keep_idx)):
        _check(load().civic_select(*args, _stream_ptr(stream)), "civic_select")
    return keep_idx


def civic_select_seq(scores: torch.Tensor, desc: SelectDesc, seq_len: int, vis_start: int,
                     keep_idx: Optional[torch.Tensor] = None, seq_idx: Optional[torch.Tensor] = None,
                     stream: Optional[torch.cuda.Stream] = None):
    """civic_select and civic_seq_indices in one launch: -> (keep_idx [n_seq, k], seq_idx [n_seq, seq_len-n+k])."""
    n = desc.t * desc.h * desc.w
    if scores.dim() != 2 or scores.shape[1] != n:
        raise ValueError("scores must be [n_seq, t*h*w]")
    n_seq = scores.shape[0]
    s_out = seq_len - n + desc.k
    dev = _device_of(scores)
    if keep_idx is None:
        keep_idx = torch.empty((n_seq, max(desc.k, 0)), dtype=torch.int32, device=dev)
    elif tuple(keep_idx.shape) != (n_seq, desc.k):
        raise ValueError("keep_idx must be [n_seq, k]")
    if seq_idx is None:
        seq_idx = torch.empty((n_seq, max(s_out, 0)), dtype=torch.int32, device=dev)
    elif tuple(seq_idx.shape) != (n_seq, s_out):
        raise ValueError("seq_idx must be [n_seq, seq_len - n + k]")
    args = (_dev_ptr(scores, "scores", torch.float32), n_seq, ctypes.byref(desc), seq_len, vis_start,
            _dev_ptr(keep_idx, "keep_idx", torch.int32), _dev_ptr(seq_idx, "seq_idx", torch.int32))
    with _on_device(_device_of(scores, keep_idx)):
        _check(load().civic_select_seq(*args, _stream_ptr(stream)), "civic_select_seq")
    return keep_idx, seq_idx


def select_workspace_bytes(desc: SelectDesc, n_seg: int, chunk_tokens: int = 0) -> int:
    return int(load().civic_select_workspace_bytes(ctypes.byref(desc), n_seg, chunk_tokens))


def civic_select_large(scores: torch.Tensor, desc: SelectDesc, keep_idx: Optional[torch.Tensor] = None,
                       workspace: Optional[torch.Tensor] = None, chunk_tokens: int = 0,
                       stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """civic_select for segments of any size: many thread blocks per segment, scratch in `workspace`
    (a uint8 CUDA tensor of at least select_workspace_bytes(...) bytes; allocated here if omitted)."""
    if scores.dim() != 2 or scores.shape[1] != desc.t * desc.h * desc.w:
        raise ValueError("scores must be [n_seg, t*h*w]")
    n_seg = scores.shape[0]
    dev = _device_of(scores)
    if keep_idx is None:
        keep_idx = torch.empty((n_seg, max(desc.k, 0)), dtype=torch.int32, device=dev)
    elif tuple(keep_idx.shape) != (n_seg, desc.k):
        raise ValueError("keep_idx must be [n_seg, k]")
    if workspace is None:
        workspace = torch.empty(max(select_workspace_bytes(desc, n_seg, chunk_tokens), 256),
                                dtype=torch.uint8, device=dev)
    args = (_dev_ptr(scores, "scores", torch.float32), n_seg, ctypes.byref(desc),
            _dev_ptr(keep_idx, "keep_idx", torch.int32), _dev_ptr(workspace, "workspace", torch.uint8),
            workspace.numel(), chunk_tokens)
    with _on_device(dev):
        _check(load().civic_select_large(*args, _stream_ptr(stream)), "civic_select_large")
    return keep_idx


def select_static_scratch_bytes() -> int:
    return int(load().civic_select_static_scratch_bytes())


def civic_select_large_static(scores: torch.Tensor, desc: SelectDesc, keep_idx: torch.Tensor,
                              chunk_tokens: int = 0, stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """civic_select_large with the scratch built into the library (at most
    select_static_scratch_bytes()): for callers that may not allocate device memory, so the
    output tensor is required and nothing is allocated here either.  Calls that can overlap on
    one GPU race on the shared scratch; keep them in one stream."""
    if scores.dim() != 2 or scores.shape[1] != desc.t * desc.h * desc.w:
        raise ValueError("scores must be [n_seg, t*h*w]")
    n_seg = scores.shape[0]
    if tuple(keep_idx.shape) != (n_seg, desc.k):
        raise ValueError("keep_idx must be [n_seg, k]")
    args = (_dev_ptr(scores, "scores", torch.float32), n_seg, ctypes.byref(desc),
            _dev_ptr(keep_idx, "keep_idx", torch.int32), chunk_tokens)
    with _on_device(_device_of(scores)):
        _check(load().civic_select_large_static(*args, _stream_ptr(stream)), "civic_select_large_static")
    return keep_idx


def floor_from_ratio(region_h: int, region_w: int, num: int, den: int) -> int:
    """Smallest floor_per_region m with m >= (num/den) * region_h * region_w; -1 on bad arguments."""
    return int(load().civic_floor_from_ratio(region_h, region_w, num, den))


def civic_select_ragged(scores: torch.Tensor, descs: Sequence[SelectDesc],
                        keep_idx: Optional[torch.Tensor] = None, flat_idx: Optional[torch.Tensor] = None,
                        want_flat: bool = True, stream: Optional[torch.cuda.Stream] = None):
    """scores fp32 [sum n] (segments concatenated), one SelectDesc per segment ->
    (segment-local keep indices int32 [sum k], the same tokens numbered over the concatenation or None)."""
    total_n = sum(d.t * d.h * d.w for d in descs)
    total_k = sum(max(d.k, 0) for d in descs)
    if scores.dim() != 1 or scores.shape[0] != total_n:
        raise ValueError("scores must be the 1-D concatenation of all segments")
    dev = _device_of(scores)
    if keep_idx is None:
        keep_idx = torch.empty((total_k,), dtype=torch.int32, device=dev)
    elif tuple(keep_idx.shape) != (total_k,):
        raise ValueError("keep_idx must be [sum k]")
    if flat_idx is None and want_flat:
        flat_idx = torch.empty((total_k,), dtype=torch.int32, device=dev)
    elif flat_idx is not None and tuple(flat_idx.shape) != (total_k,):
        raise ValueError("flat_idx must be [sum k]")
    table = (SelectDesc * max(len(descs), 1))(*descs)
    args = (_dev_ptr(scores, "scores", torch.float32), len(descs), table,
            _dev_ptr(keep_idx, "keep_idx", torch.int32), _dev_ptr(flat_idx, "flat_idx", torch.int32))
    with _on_device(dev):
        _check(load().civic_select_ragged(*args, _stream_ptr(stream)), "civic_select_ragged")
    return keep_idx, flat_idx


def set_programmatic_launch(enable: bool) -> bool:
    """Switch programmatic dependent launch on or off (process-wide); returns the old setting."""
    return bool(load().civic_set_programmatic_launch(1 if enable else 0))


def civic_compact(hidden: Optional[torch.Tensor], pos_ids: Optional[torch.Tensor], keep_idx: torch.Tensor,
                  hidden_out: Optional[torch.Tensor] = None, pos_out: Optional[torch.Tensor] = None,
                  stream: Optional[torch.cuda.Stream] = None):
    """hidden [n_seg, n, D] (any dtype), pos_ids int32 [n_seg, n, 3] -> ([n_seg, k, D], [n_seg, k, 3])."""
    n_seg, k = keep_idx.shape
    n = None
    row_bytes = 0
    if hidden is not None:
        if hidden.dim() != 3 or hidden.shape[0] != n_seg:
            raise ValueError("hidden must be [n_seg, n, D]")
        n = hidden.shape[1]
        row_bytes = hidden.shape[2] * hidden.element_size()
        if hidden_out is None:
            hidden_out = torch.empty((n_seg, k, hidden.shape[2]), dtype=hidden.dtype, device=_device_of(keep_idx, hidden))
        elif tuple(hidden_out.shape) != (n_seg, k, hidden.shape[2]) or hidden_out.dtype != hidden.dtype:
            raise ValueError("hidden_out must be [n_seg, k, D] of hidden's dtype")
    if pos_ids is not None:
        if pos_ids.dim() != 3 or pos_ids.shape[0] != n_seg or pos_ids.shape[2] != 3:
            raise ValueError("pos_ids must be [n_seg, n, 3]")
        if n is not None and pos_ids.shape[1] != n:
            raise ValueError("hidden and pos_ids disagree on n")
        n = pos_ids.shape[1]
        if pos_out is None:
            pos_out = torch.empty((n_seg, k, 3), dtype=torch.int32, device=_device_of(keep_idx, pos_ids))
        elif tuple(pos_out.shape) != (n_seg, k, 3):
            raise ValueError("pos_out must be [n_seg, k, 3]")
    if n is None:
        raise ValueError("nothing to compact")
    args = (_dev_ptr(hidden, "hidden"), row_bytes, _dev_ptr(pos_ids, "pos_ids", torch.int32),
            _dev_ptr(keep_idx, "keep_idx", torch.int32), n_seg, n, k,
            _dev_ptr(hidden_out, "hidden_out"), _dev_ptr(pos_out, "pos_out", torch.int32))
    with _on_device(_device_of(keep_idx, hidden, pos_ids)):
        _check(load().civic_compact(*args, _stream_ptr(stream)), "civic_compact")
    return hidden_out, pos_out


def civic_seq_indices(keep_idx: torch.Tensor, seq_len: int, vis_start: int, n_vis: int,
                      seq_idx: Optional[torch.Tensor] = None,
                      stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """keep_idx int32 [n_seq, k] -> kept positions of the full sequence int32 [n_seq, seq_len-n_vis+k]."""
    n_seq, k = keep_idx.shape
    s_out = seq_len - n_vis + k
    if seq_idx is None:
        seq_idx = torch.empty((n_seq, max(s_out, 0)), dtype=torch.int32, device=_device_of(keep_idx))
    elif tuple(seq_idx.shape) != (n_seq, s_out):
        raise ValueError("seq_idx must be [n_seq, seq_len - n_vis + k]")
    args = (_dev_ptr(keep_idx, "keep_idx", torch.int32), n_seq, k, seq_len, vis_start, n_vis,
            _dev_ptr(seq_idx, "seq_idx", torch.int32))
    with _on_device(_device_of(keep_idx, seq_idx)):
        _check(load().civic_seq_indices(*args, _stream_ptr(stream)), "civic_seq_indices")
    return seq_idx


@dataclasses.dataclass
class KVTables:
    """Host pointer tables for civic_compact_kv, built once per set of cache tensors."""
    k_src: ctypes.Array
    v_src: ctypes.Array
    k_dst: ctypes.Array
    v_dst: ctypes.Array
    n_layers: int
    n_seq: int
    seq_len: int
    s_out: int
    row_bytes: int
    keepalive: tuple


def kv_tables(k_src: Sequence[torch.Tensor], v_src: Sequence[torch.Tensor],
              k_dst: Sequence[torch.Tensor], v_dst: Sequence[torch.Tensor]) -> KVTables:
    """Marshal per-layer tensors ([n_seq, seq_len, ...] -> [n_seq, s_out, ...]) into pointer tables."""
    n_layers = len(k_src)
    if not (len(v_src) == len(k_dst) == len(v_dst) == n_layers):
        raise ValueError("the four tensor lists must have one entry per layer")
    if n_layers == 0:
        raise ValueError("no layers")
    src_shape, dst_shape = tuple(k_src[0].shape), tuple(k_dst[0].shape)
    for a in list(k_src) + list(v_src):
        if tuple(a.shape) != src_shape or a.dtype != k_src[0].dtype:
            raise ValueError("all source tensors must share shape and dtype")
    for a in list(k_dst) + list(v_dst):
        if tuple(a.shape) != dst_shape or a.dtype != k_src[0].dtype:
            raise ValueError("all destination tensors must share shape and dtype")
    if len(src_shape) < 3 or src_shape[0] != dst_shape[0] or src_shape[2:] != dst_shape[2:]:
        raise ValueError("source [n_seq, seq_len, ...] and destination [n_seq, s_out, ...] disagree")
    row_elems = 1
    for d in src_shape[2:]:
        row_elems *= d

    def table(ts, what):
        return (ctypes.c_void_p * n_layers)(*[_dev_ptr(t, what) for t in ts])

    return KVTables(table(k_src, "k_src"), table(v_src, "v_src"), table(k_dst, "k_dst"),
                    table(v_dst, "v_dst"), n_layers, src_shape[0], src_shape[1], dst_shape[1],
                    row_elems * k_src[0].element_size(),
                    (tuple(k_src), tuple(v_src), tuple(k_dst), tuple(v_dst)))


def civic_compact_kv(tables: KVTables, seq_idx: torch.Tensor,
                     stream: Optional[torch.cuda.Stream] = None) -> None:
    """k_dst[l][s, j] = k_src[l][s, seq_idx[s, j]] (and V) for every layer, one launch."""
    if tuple(seq_idx.shape) != (tables.n_seq, tables.s_out):
        raise ValueError("seq_idx must be [n_seq, s_out]")
    idx_ptr = _dev_ptr(seq_idx, "seq_idx", torch.int32)
    with _on_device(_device_of(seq_idx, *tables.keepalive[0], *tables.keepalive[2])):
        _check(load().civic_compact_kv(tables.k_src, tables.v_src, tables.k_dst, tables.v_dst,
                                       tables.n_layers, tables.n_seq, tables.seq_len, tables.s_out,
                                       tables.row_bytes, idx_ptr, _stream_ptr(stream)),
               "civic_compact_kv")


def _table(ts: Sequence[torch.Tensor], what: str) -> ctypes.Array:
    return (ctypes.c_void_p * len(ts))(*[_dev_ptr(t, what) for t in ts])


def _same(ts: Sequence[torch.Tensor], what: str):
    shape, dtype = tuple(ts[0].shape), ts[0].dtype
    for t in ts:
        if tuple(t.shape) != shape or t.dtype != dtype:
            raise ValueError(f"all {what} tensors must share shape and dtype")
    return shape, dtype


@dataclasses.dataclass
class KVHeadsTables:
    """Host pointer tables for civic_compact_kv_heads, built once per set of cache tensors."""
    tables: tuple
    n_layers: int
    n_seq: int
    n_heads: int
    seq_len: int
    s_out: int
    head_bytes: int
    keepalive: tuple


def kv_heads_tables(k_src: Sequence[torch.Tensor], v_src: Sequence[torch.Tensor],
                    k_dst: Sequence[torch.Tensor], v_dst: Sequence[torch.Tensor]) -> KVHeadsTables:
    """Marshal head-major per-layer tensors ([n_seq, n_heads, seq_len, d] -> [n_seq, n_heads, s_out, d])."""
    n_layers = len(k_src)
    if n_layers == 0 or not (len(v_src) == len(k_dst) == len(v_dst) == n_layers):
        raise ValueError("the four tensor lists must have one entry per layer")
    src_shape, dtype = _same(list(k_src) + list(v_src), "source")
    dst_shape, dst_dtype = _same(list(k_dst) + list(v_dst), "destination")
    if len(src_shape) != 4 or len(dst_shape) != 4 or dst_dtype != dtype or \
            src_shape[:2] != dst_shape[:2] or src_shape[3] != dst_shape[3]:
        raise ValueError("source [n_seq, n_heads, seq_len, d] and destination [n_seq, n_heads, s_out, d] disagree")
    n_seq, n_heads, seq_len, d = src_shape
    return KVHeadsTables((_table(k_src, "k_src"), _table(v_src, "v_src"), _table(k_dst, "k_dst"),
                          _table(v_dst, "v_dst")), n_layers, n_seq, n_heads, seq_len, dst_shape[2],
                         d * k_src[0].element_size(),
                         (tuple(k_src), tuple(v_src), tuple(k_dst), tuple(v_dst)))


def civic_compact_kv_heads(tables: KVHeadsTables, seq_idx: torch.Tensor,
                           stream: Optional[torch.cuda.Stream] = None) -> None:
    """Head-major caches: k_dst[l][s, h, j] = k_src[l][s, h, seq_idx[s, j]] (and V), every layer."""
    t = tables
    if tuple(seq_idx.shape) != (t.n_seq, t.s_out):
        raise ValueError("seq_idx must be [n_seq, s_out]")
    idx_ptr = _dev_ptr(seq_idx, "seq_idx", torch.int32)
    with _on_device(_device_of(seq_idx, t.keepalive[0][0], t.keepalive[2][0])):
        _check(load().civic_compact_kv_heads(*t.tables, t.n_layers, t.n_seq, t.n_heads, t.seq_len, t.s_out,
                                             t.head_bytes, idx_ptr, _stream_ptr(stream)),
               "civic_compact_kv_heads")


@dataclasses.dataclass
class KVPagedTables:
    """Host pointer tables for civic_compact_kv_paged, built once per set of cache tensors."""
    tables: tuple
    n_layers: int
    n_seq: int
    seq_len: int
    row_bytes: int
    n_pages: int
    page_size: int
    keepalive: tuple


def kv_paged_tables(k_src: Sequence[torch.Tensor], v_src: Sequence[torch.Tensor],
                    k_cache: Sequence[torch.Tensor], v_cache: Sequence[torch.Tensor]) -> KVPagedTables:
    """Marshal token-major sources [n_seq, seq_len, ...] and paged caches [n_pages, page_size, ...]."""
    n_layers = len(k_src)
    if n_layers == 0 or not (len(v_src) == len(k_cache) == len(v_cache) == n_layers):
        raise ValueError("the four tensor lists must have one entry per layer")
    src_shape, dtype = _same(list(k_src) + list(v_src), "source")
    cache_shape, cache_dtype = _same(list(k_cache) + list(v_cache), "cache")
    if len(src_shape) < 3 or len(cache_shape) != len(src_shape) or cache_dtype != dtype or \
            src_shape[2:] != cache_shape[2:]:
        raise ValueError("source [n_seq, seq_len, ...] and cache [n_pages, page_size, ...] disagree")
    row_elems = 1
    for d in src_shape[2:]:
        row_elems *= d
    return KVPagedTables((_table(k_src, "k_src"), _table(v_src, "v_src"), _table(k_cache, "k_cache"),
                          _table(v_cache, "v_cache")), n_layers, src_shape[0], src_shape[1],
                         row_elems * k_src[0].element_size(), cache_shape[0], cache_shape[1],
                         (tuple(k_src), tuple(v_src), tuple(k_cache), tuple(v_cache)))


def civic_compact_kv_paged(tables: KVPagedTables, seq_idx: torch.Tensor, block_table: torch.Tensor,
                           stream: Optional[torch.cuda.Stream] = None) -> None:
    """Kept rows of every layer's K and V into the paged caches through block_table int32
    [n_seq, max_pages_per_seq]: compact position j -> page block_table[s, j // page_size], slot j % page_size."""
    t = tables
    if seq_idx.dim() != 2 or seq_idx.shape[0] != t.n_seq:
        raise ValueError("seq_idx must be [n_seq, s_out]")
    if block_table.dim() != 2 or block_table.shape[0] != t.n_seq:
        raise ValueError("block_table must be [n_seq, max_pages_per_seq]")
    idx_ptr = _dev_ptr(seq_idx, "seq_idx", torch.int32)
    tab_ptr = _dev_ptr(block_table, "block_table", torch.int32)
    with _on_device(_device_of(seq_idx, t.keepalive[0][0], t.keepalive[2][0])):
        _check(load().civic_compact_kv_paged(*t.tables, t.n_layers, t.n_seq, t.seq_len, seq_idx.shape[1],
                                             t.row_bytes, idx_ptr, tab_ptr, block_table.shape[1],
                                             t.page_size, t.n_pages, _stream_ptr(stream)),
               "civic_compact_kv_paged")


def civic_merge_embeddings(text: torch.Tensor, visual: torch.Tensor, keep_idx: torch.Tensor,
                           vis_start: int, merged: Optional[torch.Tensor] = None,
                           stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """text [n_seq, seq_len, D], dense visual [n_seq, n_vis, D], keep_idx [n_seq, k] ->
    merged [n_seq, seq_len - n_vis + k, D] (Eq. 13)."""
    if text.dim() != 3 or visual.dim() != 3 or text.shape[0] != visual.shape[0] or \
            text.shape[2] != visual.shape[2] or text.dtype != visual.dtype:
        raise ValueError("text [n_seq, seq_len, D] and visual [n_seq, n_vis, D] disagree")
    n_seq, seq_len, dim = text.shape
    n_vis = visual.shape[1]
    if keep_idx.dim() != 2 or keep_idx.shape[0] != n_seq:
        raise ValueError("keep_idx must be [n_seq, k]")
    k = keep_idx.shape[1]
    s_out = seq_len - n_vis + k
    if merged is None:
        merged = torch.empty((n_seq, max(s_out, 0), dim), dtype=text.dtype, device=_device_of(keep_idx, text))
    elif tuple(merged.shape) != (n_seq, s_out, dim) or merged.dtype != text.dtype:
        raise ValueError("merged must be [n_seq, seq_len - n_vis + k, D] of text's dtype")
    args = (_dev_ptr(text, "text"), _dev_ptr(visual, "visual"), dim * text.element_size(),
            _dev_ptr(keep_idx, "keep_idx", torch.int32), n_seq, seq_len, vis_start, n_vis, k,
            _dev_ptr(merged, "merged"))
    with _on_device(_device_of(keep_idx, text, visual)):
        _check(load().civic_merge_embeddings(*args, _stream_ptr(stream)), "civic_merge_embeddings")
    return merged


def civic_compact_pos_planes(pos: torch.Tensor, seq_idx: torch.Tensor,
                             pos_out: Optional[torch.Tensor] = None,
                             stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """pos int32 [n_planes, n_seq, seq_len], seq_idx [n_seq, s_out] -> [n_planes, n_seq, s_out]."""
    if pos.dim() != 3 or seq_idx.dim() != 2 or pos.shape[1] != seq_idx.shape[0]:
        raise ValueError("pos must be [n_planes, n_seq, seq_len] and seq_idx [n_seq, s_out]")
    n_planes, n_seq, seq_len = pos.shape
    s_out = seq_idx.shape[1]
    if pos_out is None:
        pos_out = torch.empty((n_planes, n_seq, s_out), dtype=torch.int32, device=_device_of(seq_idx, pos))
    elif tuple(pos_out.shape) != (n_planes, n_seq, s_out):
        raise ValueError("pos_out must be [n_planes, n_seq, s_out]")
    args = (_dev_ptr(pos, "pos", torch.int32), n_planes, n_seq, seq_len,
            _dev_ptr(seq_idx, "seq_idx", torch.int32), s_out, _dev_ptr(pos_out, "pos_out", torch.int32))
    with _on_device(_device_of(seq_idx, pos)):
        _check(load().civic_compact_pos_planes(*args, _stream_ptr(stream)), "civic_compact_pos_planes")
    return pos_out


def anchor_aggregate_workspace_bytes(n_img: int, t_e: int, m_e: int, d_v: int) -> int:
    return int(load().civic_anchor_aggregate_workspace_bytes(n_img, t_e, m_e, d_v))


@dataclasses.dataclass
class PreparedAnchors:
    """Q_A = Norm(LN(A)) in bf16 and its row sums, written once by civic_anchor_prepare."""
    buffer: torch.Tensor
    m_e: int
    d_v: int


def civic_anchor_prepare(anchors: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> PreparedAnchors:
    """anchors fp32 [m_e, d_v] -> the per-model constants of Eq. 8, for civic_anchor_aggregate(x0, prepared, ...)."""
    if anchors.dim() != 2:
        raise ValueError("anchors must be [m_e, d_v]")
    m_e, d_v = anchors.shape
    need = int(load().civic_anchor_prepared_bytes(m_e, d_v))
    if need == 0:
        raise CivicError(5, "civic_anchor_prepared_bytes")
    buf = torch.empty(need, dtype=torch.uint8, device=_device_of(anchors))
    with _on_device(_device_of(anchors)):
        _check(load().civic_anchor_prepare(_dev_ptr(anchors, "anchors", torch.float32), m_e, d_v,
                                           _dev_ptr(buf, "prepared"), need, _stream_ptr(stream)), "civic_anchor_prepare")
    return PreparedAnchors(buf, m_e, d_v)


def civic_anchor_aggregate(x0: torch.Tensor, anchors, tau: float,
                           z0: Optional[torch.Tensor] = None, token_mass: Optional[torch.Tensor] = None,
                           want_mass: bool = True, workspace: Optional[torch.Tensor] = None,
                           device_status: Optional[torch.Tensor] = None,
                           stream: Optional[torch.cuda.Stream] = None):
    """Eq. 8: x0 bf16 [n_img, t_e, d_v], anchors fp32 [m_e, d_v] (or PreparedAnchors) ->
    (z0 bf16 [n_img, m_e, d_v], token mass fp32 [n_img, t_e] or None, device_status int32 [1]: 0 after a clean run)."""
    prepared = anchors if isinstance(anchors, PreparedAnchors) else None
    if prepared is not None:
        if x0.dim() != 3 or prepared.d_v != x0.shape[2]:
            raise ValueError("x0 must be [n_img, t_e, d_v] with the prepared anchors' d_v")
        m_e = prepared.m_e
    else:
        if x0.dim() != 3 or anchors.dim() != 2 or anchors.shape[1] != x0.shape[2]:
            raise ValueError("x0 must be [n_img, t_e, d_v] and anchors [m_e, d_v]")
        m_e = anchors.shape[0]
    n_img, t_e, d_v = x0.shape
    dev = _device_of(x0)
    if z0 is None:
        z0 = torch.empty((n_img, m_e, d_v), dtype=torch.bfloat16, device=dev)
    elif tuple(z0.shape) != (n_img, m_e, d_v):
        raise ValueError("z0 must be [n_img, m_e, d_v]")
    if token_mass is None and want_mass:
        token_mass = torch.empty((n_img, t_e), dtype=torch.float32, device=dev)
    elif token_mass is not None and tuple(token_mass.shape) != (n_img, t_e):
        raise ValueError("token_mass must be [n_img, t_e]")
    if workspace is None:
        workspace = torch.empty(max(anchor_aggregate_workspace_bytes(n_img, t_e, m_e, d_v), 256),
                                dtype=torch.uint8, device=dev)
    if device_status is None:
        device_status = torch.empty((1,), dtype=torch.int32, device=dev)
    a_ptr = _dev_ptr(prepared.buffer, "prepared") if prepared is not None else _dev_ptr(anchors, "anchors", torch.float32)
    args = (_dev_ptr(x0, "x0", torch.bfloat16), a_ptr, n_img, t_e, m_e, d_v,
            ctypes.c_float(tau), _dev_ptr(z0, "z0", torch.bfloat16), _dev_ptr(token_mass, "token_mass", torch.float32),
            _dev_ptr(workspace, "workspace", torch.uint8), workspace.numel(),
            _dev_ptr(device_status, "device_status", torch.int32))
    fn = load().civic_anchor_aggregate_prepared if prepared is not None else load().civic_anchor_aggregate
    with _on_device(dev):
        _check(fn(*args, _stream_ptr(stream)), "civic_anchor_aggregate")
    return z0, token_mass, device_status


def kv_compressed_attention_workspace_bytes(n_img: int, m_e: int, n_heads: int, head_dim: int, s: int) -> int:
    return int(load().civic_kv_compressed_attention_workspace_bytes(n_img, m_e, n_heads, head_dim, s))


@dataclasses.dataclass
class PreparedAssignment:
    """R in bf16 and its column sums, written once by civic_kv_attention_prepare."""
    buffer: torch.Tensor
    m_e: int
    s: int


def civic_kv_attention_prepare(r: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> PreparedAssignment:
    """r fp32 [m_e, s] -> the per-model constants of Eq. 9, for civic_kv_compressed_attention(q, k, v, prepared, ...)."""
    if r.dim() != 2:
        raise ValueError("r must be [m_e, s]")
    m_e, s = r.shape
    need = int(load().civic_kv_attention_prepared_bytes(m_e, s))
    if need == 0:
        raise CivicError(5, "civic_kv_attention_prepared_bytes")
    buf = torch.empty(need, dtype=torch.uint8, device=_device_of(r))
    with _on_device(_device_of(r)):
        _check(load().civic_kv_attention_prepare(_dev_ptr(r, "r", torch.float32), m_e, s, _dev_ptr(buf, "prepared"), need,
                                                 _stream_ptr(stream)), "civic_kv_attention_prepare")
    return PreparedAssignment(buf, m_e, s)


def civic_kv_compressed_attention(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, r, n_heads: int,
                                  out: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                                  device_status: Optional[torch.Tensor] = None,
                                  stream: Optional[torch.cuda.Stream] = None):
    """Eq. 9 for projected q, k, v bf16 [n_img, m_e, n_heads * d] and the assignment r fp32 [m_e, s] (or a
    PreparedAssignment) -> (attention output bf16 [n_img, m_e, n_heads * d], device_status int32 [1]: 0 after a clean run)."""
    prepared = r if isinstance(r, PreparedAssignment) else None
    r_rows, r_cols = (prepared.m_e, prepared.s) if prepared is not None else (tuple(r.shape) if r.dim() == 2 else (-1, -1))
    if q.dim() != 3 or q.shape != k.shape or q.shape != v.shape or r_rows != q.shape[1]:
        raise ValueError("q, k, v must be [n_img, m_e, D] and r [m_e, s]")
    n_img, m_e, dim = q.shape
    if dim % n_heads:
        raise ValueError("the feature dimension must be a multiple of n_heads")
    head_dim, s = dim // n_heads, r_cols
    dev = _device_of(q)
    if out is None:
        out = torch.empty_like(q)
    elif out.shape != q.shape:
        raise ValueError("out must have q's shape")
    if workspace is None:
        workspace = torch.empty(max(kv_compressed_attention_workspace_bytes(n_img, m_e, n_heads, head_dim, s), 256),
                                dtype=torch.uint8, device=dev)
    if device_status is None:
        device_status = torch.empty((1,), dtype=torch.int32, device=dev)
    r_ptr = _dev_ptr(prepared.buffer, "prepared") if prepared is not None else _dev_ptr(r, "r", torch.float32)
    args = (_dev_ptr(q, "q", torch.bfloat16), _dev_ptr(k, "k", torch.bfloat16), _dev_ptr(v, "v", torch.bfloat16),
            r_ptr, n_img, m_e, n_heads, head_dim, s, _dev_ptr(out, "out", torch.bfloat16),
            _dev_ptr(workspace, "workspace", torch.uint8), workspace.numel(),
            _dev_ptr(device_status, "device_status", torch.int32))
    fn = load().civic_kv_compressed_attention_prepared if prepared is not None else load().civic_kv_compressed_attention
    with _on_device(dev):
        _check(fn(*args, _stream_ptr(stream)), "civic_kv_compressed_attention")
    return out, device_status


class index_check:
    """Context manager: inside it this thread's compaction calls validate their index arrays on the
    device and record the first fault in `record` (int32 [4] on the device: code, row, position,
    value; see INDEX_FAULTS).  The record is not cleared here."""

    def __init__(self, record: torch.Tensor):
        if record.numel() < 4:
            raise ValueError("the fault record must hold 4 int32")
        self.ptr = _dev_ptr(record, "record", torch.int32)
        self.keepalive = record

    def __enter__(self):
        _check(load().civic_set_index_check(self.ptr), "civic_set_index_check")
        return self

    def __exit__(self, *exc):
        load().civic_set_index_check(None)


def civic_validate_indices(idx: torch.Tensor, limit: int, record: torch.Tensor, require_ascending: bool = True,
                           stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """idx int32 [n_rows, row_len]: every value in [0, limit), rows strictly ascending if asked;
    the first fault found goes to `record` (int32 [4], sticky)."""
    if idx.dim() != 2 or record.numel() < 4:
        raise ValueError("idx must be [n_rows, row_len] and the record hold 4 int32")
    args = (_dev_ptr(idx, "idx", torch.int32), idx.shape[0], idx.shape[1], limit, 1 if require_ascending else 0,
            _dev_ptr(record, "record", torch.int32))
    with _on_device(_device_of(idx, record)):
        _check(load().civic_validate_indices(*args, _stream_ptr(stream)), "civic_validate_indices")
    return record


def civic_selftest_bounded_wait(limit_cycles: int, record: torch.Tensor,
                                stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """Runs the kernels' bounded wait on a barrier nobody signals; record int32 [2] -> (time-out code, 1)."""
    if record.numel() < 2:
        raise ValueError("the record must hold 2 int32")
    with _on_device(_device_of(record)):
        _check(load().civic_selftest_bounded_wait(limit_cycles, _dev_ptr(record, "record", torch.int32),
                                                  _stream_ptr(stream)), "civic_selftest_bounded_wait")
    return record
