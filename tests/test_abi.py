"""The C-ABI library: loads without a GPU, exports what include/civic.h declares, and
rejects bad arguments on the host before anything is launched."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
from paper_2605_28115_b200 import build, civic

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return civic.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "civic.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(civic_[a-z_]+)\s*\(", text)))


def test_exports_match_header(lib):
    names = declared_functions()
    assert sorted(civic.EXPORTS) == names
    for name in names:
        assert getattr(lib, name) is not None


def test_status_strings(lib):
    for code, name in enumerate(civic.STATUS_NAMES):
        assert lib.civic_status_string(code).decode() == name
    assert lib.civic_status_string(99).decode() == "CIVIC_ERR_UNKNOWN"
    assert lib.civic_last_cuda_error().decode() == ""


def test_max_tokens_covers_workloads(lib):
    assert lib.civic_select_max_tokens() >= 3136
    assert lib.civic_select_max_tokens() <= 65535


def test_reserved_count_matches_region_enumeration(lib):
    rng = np.random.default_rng(0)
    for _ in range(300):
        t, h, w = (int(rng.integers(1, 5)), int(rng.integers(1, 40)), int(rng.integers(1, 40)))
        rh, rw, m = int(rng.integers(1, 9)), int(rng.integers(1, 9)), int(rng.integers(0, 20))
        d = civic.SelectDesc(t, h, w, rh, rw, m, 0)
        assert civic.reserved_count(d) == oracle.default.reserved_count(t, h, w, rh, rw, m)
    assert civic.reserved_count(civic.SelectDesc(1, 4, 4, 0, 1, 1, 1)) == -1


def _select_status(lib, desc, n_seg=1, scores=0x1000, out=0x2000):
    return lib.civic_select(scores, n_seg, ctypes.byref(desc), out, None)


def test_select_validation_happens_on_host(lib):
    D = civic.SelectDesc
    before = lib.civic_launch_count()
    assert _select_status(lib, D(1, 4, 4, 2, 2, 1, 17)) == 2  # k > n
    assert _select_status(lib, D(1, 4, 4, 2, 2, 1, -1)) == 2
    assert _select_status(lib, D(1, 4, 4, 2, 2, 1, 3)) == 3  # floor needs 4
    assert _select_status(lib, D(1, 4, 4, 2, 2, 5, 15)) == 3
    assert _select_status(lib, D(0, 4, 4, 2, 2, 1, 3)) == 1
    assert _select_status(lib, D(1, 4, 4, 2, 0, 1, 3)) == 1
    assert _select_status(lib, D(1, 4, 4, 2, 2, -1, 3)) == 1
    assert _select_status(lib, D(1, 4, 4, 2, 2, 1, 8), n_seg=-1) == 1
    assert _select_status(lib, D(1, 4, 4, 2, 2, 1, 8), scores=None) == 1
    assert _select_status(lib, D(1, 4, 4, 2, 2, 1, 8), out=None) == 1
    assert _select_status(lib, D(1, 4, 4, 2, 2, 1, 8), scores=0x1002) == 4
    assert _select_status(lib, D(1, 4, 4, 2, 2, 1, 8), scores=0x1000, out=0x1010) == 1  # overlap
    assert _select_status(lib, D(1, 300, 300, 2, 2, 0, 8)) == 5  # 90000 tokens > one block
    assert _select_status(lib, D(2, 40000, 40000, 2, 2, 0, 8)) == 5
    assert lib.civic_select(None, 1, None, None, None) == 1
    # nothing to do: OK without touching the device
    assert _select_status(lib, D(1, 4, 4, 2, 2, 0, 0)) == 0
    assert _select_status(lib, D(1, 4, 4, 2, 2, 1, 8), n_seg=0) == 0
    assert lib.civic_launch_count() == before


def test_compact_validation(lib):
    f = lib.civic_compact
    before = lib.civic_launch_count()
    assert f(0x10000, 64, None, 0x100, 1, 8, 9, 0x20000, None, None) == 2  # k > n
    assert f(0x10000, 64, None, 0x100, 1, 8, 4, None, None, None) == 1  # hidden without out
    assert f(None, 64, 0x10000, 0x100, 1, 8, 4, None, None, None) == 1  # pos without out
    assert f(0x10000, 6, None, 0x100, 1, 8, 4, 0x20000, None, None) == 4  # row not multiple of 4
    assert f(0x10002, 64, None, 0x100, 1, 8, 4, 0x20000, None, None) == 4
    assert f(0x10000, 64, None, 0x100, 1, 8, 4, 0x10100, None, None) == 1  # overlap
    assert f(0x10000, 64, None, None, 1, 8, 4, 0x20000, None, None) == 1  # no indices
    assert f(0x10000, 64, None, 0x100, -1, 8, 4, 0x20000, None, None) == 1
    assert f(0x10000, 64, None, 0x100, 0, 8, 4, 0x20000, None, None) == 0
    assert f(0x10000, 64, None, 0x100, 1, 8, 0, 0x20000, None, None) == 0
    assert lib.civic_launch_count() == before


def test_seq_indices_validation(lib):
    f = lib.civic_seq_indices
    assert f(0x100, 1, 5, 20, 3, 12, None, None) == 1
    assert f(0x100, 1, 13, 20, 3, 12, 0x1000, None) == 2  # k > n_vis
    assert f(0x100, 1, 5, 20, 10, 12, 0x1000, None) == 1  # span runs past the end
    assert f(0x100, 1, 5, 20, -1, 12, 0x1000, None) == 1
    assert f(0x100, 0, 5, 20, 3, 12, 0x1000, None) == 0


def test_select_seq_validation(lib):
    D = civic.SelectDesc
    f = lambda d, seq_len, vis_start, n_seq=1, scores=0x1000, keep=0x2000, seq=0x3000: \
        lib.civic_select_seq(scores, n_seq, ctypes.byref(d), seq_len, vis_start, keep, seq, None)
    before = lib.civic_launch_count()
    assert f(D(1, 4, 4, 2, 2, 1, 8), 15, 0) == 1  # visual span longer than the sequence
    assert f(D(1, 4, 4, 2, 2, 1, 8), 20, 5) == 1  # span runs past the end
    assert f(D(1, 4, 4, 2, 2, 1, 8), 20, -1) == 1
    assert f(D(1, 4, 4, 2, 2, 1, 17), 20, 2) == 2
    assert f(D(1, 4, 4, 2, 2, 1, 3), 20, 2) == 3
    assert f(D(1, 4, 4, 2, 2, 1, 8), 20, 2, seq=None) == 1
    assert f(D(1, 4, 4, 2, 2, 1, 8), 20, 2, seq=0x3002) == 4
    assert f(D(1, 4, 4, 2, 2, 1, 8), 20, 2, seq=0x2010) == 1  # seq_idx overlaps keep_idx
    assert f(D(1, 4, 4, 2, 2, 1, 8), 20, 2, n_seq=0) == 0
    assert lib.civic_launch_count() == before
    assert lib.civic_set_programmatic_launch(1) == 1  # on by default, setter returns the old value


def test_compact_kv_validation(lib):
    f = lib.civic_compact_kv
    P = ctypes.c_void_p * 2
    ks, vs = P(0x100000, 0x200000), P(0x300000, 0x400000)
    kd, vd = P(0x500000, 0x600000), P(0x700000, 0x800000)
    assert f(ks, vs, kd, vd, 2, 2, 16, 17, 64, 0x10, None) == 2  # s_out > seq_len
    assert f(ks, vs, kd, vd, 2, 2, 16, 8, 0, 0x10, None) == 1
    assert f(ks, vs, kd, vd, 2, 2, 16, 8, 6, 0x10, None) == 4
    assert f(ks, vs, kd, vd, 2, 2, 16, 8, 64, None, None) == 1
    assert f(None, vs, kd, vd, 2, 2, 16, 8, 64, 0x10, None) == 1
    assert f(ks, vs, ks, vd, 2, 2, 16, 8, 64, 0x10, None) == 1  # destination is a source
    assert f(ks, vs, kd, kd, 2, 2, 16, 8, 64, 0x10, None) == 1  # two destinations coincide
    assert f(ks, vs, P(0x500000, None), vd, 2, 2, 16, 8, 64, 0x10, None) == 1
    assert f(ks, vs, kd, vd, 0, 2, 16, 8, 64, 0x10, None) == 0
    assert f(ks, vs, kd, vd, -1, 2, 16, 8, 64, 0x10, None) == 1


def test_select_large_validation(lib):
    D = civic.SelectDesc
    f = lambda d, n_seg=1, scores=0x100000, keep=0x200000, ws=0x300000, ws_bytes=1 << 30, chunk=0: \
        lib.civic_select_large(scores, n_seg, ctypes.byref(d), keep, ws, ws_bytes, chunk, None)
    before = lib.civic_launch_count()
    d = D(8, 40, 40, 4, 4, 1, 4000)
    need = lib.civic_select_workspace_bytes(ctypes.byref(d), 2, 0)
    # 2 segments: histograms + scalars, per-chunk counts, one flag byte per token, 256-byte sections
    assert need >= 2 * (3 * 2048 + 16) * 4 + 2 * 12800 and need % 256 == 0
    assert lib.civic_select_workspace_bytes(ctypes.byref(D(8, 40, 40, 0, 4, 1, 4000)), 2, 0) == 0
    assert lib.civic_select_workspace_bytes(ctypes.byref(d), 2, 100) == 0  # region row of 160 tokens
    assert f(d, ws=None) == 7
    assert f(d, ws_bytes=need // 2 - 1) == 7  # one segment needs about half
    assert f(d, ws=0x300010) == 4
    assert f(d, chunk=100) == 5
    assert f(d, chunk=-1) == 1
    assert f(D(8, 40, 40, 4, 4, 1, 12801)) == 2
    assert f(D(8, 40, 40, 4, 4, 1, 799)) == 3
    assert f(d, scores=None) == 1
    assert f(d, keep=0x300100) == 1  # output inside the workspace
    assert f(d, n_seg=0) == 0
    assert f(D(8, 40, 40, 4, 4, 0, 0)) == 0
    assert f(D(1, 4, 70000, 4, 4, 1, 70000)) == 5  # one region row holds 280000 tokens
    assert lib.civic_launch_count() == before
    assert lib.civic_status_string(7).decode() == "CIVIC_ERR_WORKSPACE"


def test_select_ragged_validation(lib):
    D = civic.SelectDesc
    arr = lambda *ds: (D * len(ds))(*ds)
    f = lambda descs, n, scores=0x100000, keep=0x200000, flat=0x300000: \
        lib.civic_select_ragged(scores, n, descs, keep, flat, None)
    before = lib.civic_launch_count()
    good = arr(D(1, 4, 4, 2, 2, 1, 8), D(2, 3, 5, 1, 5, 0, 7))
    assert f(good, 2, scores=None) == 1
    assert f(good, 2, keep=None) == 1
    assert f(arr(D(1, 4, 4, 2, 2, 1, 8), D(1, 4, 4, 2, 2, 1, 17)), 2) == 2
    assert f(arr(D(1, 4, 4, 2, 2, 1, 8), D(1, 4, 4, 2, 2, 1, 3)), 2) == 3
    assert f(arr(D(1, 4, 4, 2, 2, 1, 8), D(1, 0, 4, 2, 2, 1, 3)), 2) == 1
    assert f(arr(D(1, 4, 4, 2, 2, 1, 8), D(1, 300, 300, 2, 2, 0, 3)), 2) == 5
    assert f(good, 2, flat=0x200004) == 1  # flat_idx overlaps keep_idx
    assert f(good, 2, keep=0x200002) == 4
    assert f(None, 1) == 1
    assert f(good, 0) == 0
    assert f(arr(D(1, 4, 4, 2, 2, 0, 0), D(2, 3, 5, 1, 5, 0, 0)), 2) == 0  # nothing kept anywhere
    assert lib.civic_launch_count() == before
    assert lib.civic_floor_from_ratio(4, 4, 1, 5) == 4 and lib.civic_floor_from_ratio(4, 4, 0, 1) == 0
    assert lib.civic_floor_from_ratio(4, 4, 1, 0) == -1


def test_adjacent_calls_validation(lib):
    P = ctypes.c_void_p * 2
    ks, vs = P(0x100000, 0x200000), P(0x300000, 0x400000)
    kd, vd = P(0x500000, 0x600000), P(0x700000, 0x800000)
    before = lib.civic_launch_count()
    h = lib.civic_compact_kv_heads
    assert h(ks, vs, kd, vd, 2, 2, 4, 16, 17, 64, 0x10, None) == 2  # s_out > seq_len
    assert h(ks, vs, kd, vd, 2, 2, 4, 16, 8, 6, 0x10, None) == 4
    assert h(ks, vs, kd, vd, 2, 2, -1, 16, 8, 64, 0x10, None) == 1
    assert h(ks, vs, ks, vd, 2, 2, 4, 16, 8, 64, 0x10, None) == 1  # destination is a source
    assert h(ks, vs, kd, vd, 2, 2, 4, 16, 8, 64, None, None) == 1
    assert h(ks, vs, kd, vd, 2, 2, 0, 16, 8, 64, 0x10, None) == 0
    g = lib.civic_compact_kv_paged
    assert g(ks, vs, kd, vd, 2, 2, 16, 8, 64, 0x10, 0x40, 1, 4, 100, None) == 1  # 1 page of 4 < 8 rows
    assert g(ks, vs, kd, vd, 2, 2, 16, 8, 64, 0x10, 0x40, 2, 0, 100, None) == 1  # page size 0
    assert g(ks, vs, kd, vd, 2, 2, 16, 8, 64, 0x10, None, 2, 4, 100, None) == 1  # no block table
    assert g(ks, vs, kd, vd, 2, 2, 16, 17, 64, 0x10, 0x40, 8, 4, 100, None) == 2
    assert g(ks, vs, kd, vd, 2, 2, 16, 8, 64, 0x10, 0x42, 2, 4, 100, None) == 4
    assert g(ks, vs, kd, vd, 2, 0, 16, 8, 64, 0x10, 0x40, 2, 4, 100, None) == 0
    m = lib.civic_merge_embeddings
    assert m(0x10000, 0x20000, 64, 0x100, 1, 20, 3, 12, 13, 0x30000, None) == 2  # k > n_vis
    assert m(0x10000, 0x20000, 64, 0x100, 1, 20, 10, 12, 5, 0x30000, None) == 1  # span past the end
    assert m(0x10000, 0x20000, 6, 0x100, 1, 20, 3, 12, 5, 0x30000, None) == 4
    assert m(0x10000, 0x20000, 64, 0x100, 1, 20, 3, 12, 5, 0x10100, None) == 1  # output overlaps text
    assert m(0x10000, None, 64, 0x100, 1, 20, 3, 12, 5, 0x30000, None) == 1
    assert m(0x10000, 0x20000, 64, 0x100, 0, 20, 3, 12, 5, 0x30000, None) == 0
    q = lib.civic_compact_pos_planes
    assert q(0x10000, 3, 2, 20, 0x100, 21, 0x30000, None) == 2
    assert q(0x10000, 3, 2, 20, 0x100, 5, None, None) == 1
    assert q(0x10000, 3, 2, 20, 0x100, 5, 0x10010, None) == 1  # overlap
    assert q(0x10000, 0, 2, 20, 0x100, 5, 0x30000, None) == 0
    assert lib.civic_launch_count() == before


def test_anchor_aggregate_validation(lib):
    f = lambda n_img=1, t_e=100, m_e=10, d_v=128, tau=0.1, x=0x100000, a=0x200000, z=0x300000, mass=None, \
        ws=0x1000000, ws_bytes=1 << 30, status=0x400000: \
        lib.civic_anchor_aggregate(x, a, n_img, t_e, m_e, d_v, ctypes.c_float(tau), z, mass, ws, ws_bytes, status, None)
    before = lib.civic_launch_count()
    assert f(d_v=100) == 5 and f(d_v=0) == 1 and f(t_e=0) == 1 and f(m_e=0) == 1
    assert f(tau=0.01) == 5 and f(tau=float("nan")) == 5
    assert f(x=None) == 1 and f(status=None) == 1 and f(x=0x100008) == 4
    assert f(ws=None) == 7 and f(ws_bytes=1000) == 7 and f(ws=0x1000010) == 4
    assert f(z=0x100100) == 1  # output overlaps the tokens
    assert f(n_img=0) == 0
    assert civic.anchor_aggregate_workspace_bytes(1, 100, 10, 100) == 0
    need = civic.anchor_aggregate_workspace_bytes(2, 100, 10, 128)
    assert need >= 10 * 128 * 2 + 2 * 100 * 8 + 2 * 10 * 104 * 2 and need % 256 == 0
    assert lib.civic_launch_count() == before


def test_kv_compressed_attention_validation(lib):
    f = lambda n_img=1, m_e=100, heads=2, d=64, s=128, q=0x100000, k=0x200000, v=0x300000, r=0x400000, \
        out=0x500000, ws=0x1000000, ws_bytes=1 << 30, status=0x600000: \
        lib.civic_kv_compressed_attention(q, k, v, r, n_img, m_e, heads, d, s, out, ws, ws_bytes, status, None)
    before = lib.civic_launch_count()
    assert f(d=68) == 5 and f(s=100) == 5 and f(s=576) == 5 and f(d=256) == 5 and f(d=136) == 5
    assert f(m_e=0) == 1 and f(heads=0) == 1 and f(q=None) == 1 and f(status=None) == 1
    assert f(k=0x200008) == 4 and f(ws=0x1000010) == 4
    assert f(ws=None) == 7 and f(ws_bytes=100) == 7
    assert f(out=0x100040) == 1  # output overlaps q
    assert f(n_img=0) == 0
    assert lib.civic_kv_compressed_attention_workspace_bytes(1, 100, 2, 68, 128) == 0
    need = lib.civic_kv_compressed_attention_workspace_bytes(2, 100, 2, 64, 128)
    assert need >= 100 * 128 * 2 + 128 * 4 + 2 * 2 * 128 * 128 * 2 and need % 256 == 0
    # the paper's shapes are accepted: 72-wide heads (stored 80 wide), 512 anchors, both with 128-wide heads
    wide = lib.civic_kv_compressed_attention_workspace_bytes(2, 100, 2, 72, 128)
    assert wide >= 2 * 2 * 128 * (2 * 80) * 2 and wide % 256 == 0
    assert lib.civic_kv_compressed_attention_workspace_bytes(1, 100, 16, 64, 512) > 0
    assert lib.civic_kv_compressed_attention_workspace_bytes(1, 100, 8, 128, 512) > 0
    assert lib.civic_launch_count() == before


def test_prepared_constants_validation(lib):
    before = lib.civic_launch_count()
    assert lib.civic_anchor_prepared_bytes(10, 100) == 0  # d_v not a multiple of 64
    need = lib.civic_anchor_prepared_bytes(10, 128)
    assert need >= 10 * 128 * 2 + 10 * 4 and need % 256 == 0
    f = lib.civic_anchor_prepare
    assert f(None, 10, 128, 0x200000, need, None) == 1
    assert f(0x100000, 10, 128, None, need, None) == 1
    assert f(0x100000, 10, 128, 0x200010, need, None) == 4
    assert f(0x100000, 10, 128, 0x200000, need - 1, None) == 7
    assert f(0x100000, 10, 100, 0x200000, need, None) == 5
    assert f(0x100000, 10, 128, 0x100100, need, None) == 1  # output inside the anchors
    g = lambda x=0x100000, prep=0x200000, ws=0x1000000, ws_bytes=1 << 30, status=0x400000, z=0x300000: \
        lib.civic_anchor_aggregate_prepared(x, prep, 1, 100, 10, 128, ctypes.c_float(0.1), z, None, ws, ws_bytes, status, None)
    assert g(prep=None) == 1 and g(prep=0x200010) == 4 and g(ws_bytes=10) == 7 and g(z=0x200000) == 1
    assert lib.civic_kv_attention_prepared_bytes(100, 100) == 0
    need = lib.civic_kv_attention_prepared_bytes(100, 128)
    assert need >= 100 * 128 * 2 + 128 * 4 and need % 256 == 0
    h = lib.civic_kv_attention_prepare
    assert h(None, 100, 128, 0x200000, need, None) == 1 and h(0x100000, 100, 128, 0x200000, need - 1, None) == 7
    assert h(0x100000, 100, 100, 0x200000, need, None) == 5 and h(0x100000, 100, 128, 0x200008, need, None) == 4
    k = lambda prep=0x400000, out=0x500000, ws_bytes=1 << 30: lib.civic_kv_compressed_attention_prepared(
        0x100000, 0x200000, 0x300000, prep, 1, 100, 2, 64, 128, out, 0x1000000, ws_bytes, 0x600000, None)
    assert k(prep=None) == 1 and k(prep=0x400010) == 4 and k(ws_bytes=10) == 7 and k(out=0x400000) == 1
    assert lib.civic_launch_count() == before


def test_binding_refuses_cpu_tensors():
    import torch

    d = civic.SelectDesc(1, 4, 4, 2, 2, 1, 8)
    with pytest.raises(ValueError, match="CUDA tensor or pinned"):
        civic.civic_select(torch.zeros(1, 16), d, keep_idx=torch.zeros(1, 8, dtype=torch.int32))


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(RuntimeError, match="no fallback"):
        civic.load(str(tmp_path / "libcivic.so"))


def test_index_check_entries_validate_on_host(lib):
    before = lib.civic_launch_count()
    assert lib.civic_set_index_check(0x1002) == 4
    assert lib.civic_set_index_check(0x1000) == 0
    assert lib.civic_set_index_check(None) == 0
    f = lib.civic_validate_indices
    assert f(0x1000, -1, 4, 10, 1, 0x9000, None) == 1
    assert f(0x1000, 2, 4, -1, 1, 0x9000, None) == 1
    assert f(None, 2, 4, 10, 1, 0x9000, None) == 1
    assert f(0x1000, 2, 4, 10, 1, None, None) == 1
    assert f(0x1002, 2, 4, 10, 1, 0x9000, None) == 4
    assert f(0x1000, 2, 4, 10, 1, 0x1010, None) == 1  # the record inside the index array
    assert f(0x1000, 0, 4, 10, 1, None, None) == 0    # nothing to check
    g = lib.civic_selftest_bounded_wait
    assert g(0, 0x1000, None) == 1 and g(1 << 25, 0x1000, None) == 1 and g(100, None, None) == 1
    assert g(100, 0x1002, None) == 4
    assert lib.civic_launch_count() == before
