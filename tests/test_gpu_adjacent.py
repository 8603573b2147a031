"""CUDA path against the CPU oracle for the steps next to the core path: Eq. 13 merge,
plane-major position ids, head-major and paged K/V (needs a B200)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_28115_b200 import build, civic
from paper_2605_28115_b200 import workloads as W
from tests.test_gpu_parity import CANARY, DEV, bits16, padded

pytestmark = pytest.mark.gpu

O = oracle.default


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    civic.load()


def sorted_choice(rng, n, k, rows):
    if k == 0:
        return np.zeros((rows, 0), np.int32)
    return np.stack([np.sort(rng.choice(n, k, replace=False)) for _ in range(rows)]).astype(np.int32)


# ------------------------------------------------------------------ Eq. 13 merge

@pytest.mark.parametrize("n_seq,seq_len,vis_start,n_vis,k,row_elems", [
    (2, 20, 3, 12, 5, 8), (3, 12, 0, 12, 4, 6), (1, 15, 5, 10, 10, 4), (2, 9, 9, 0, 0, 2),
    (2, 30, 23, 7, 0, 10), (3, 70, 9, 40, 13, 1032), (2, 300, 17, 256, 85, 4096), (2, 50, 5, 40, 20, 2)])
def test_merge_embeddings_small(n_seq, seq_len, vis_start, n_vis, k, row_elems):
    rng = np.random.default_rng(n_seq * 1000 + seq_len)
    text = rng.integers(-30000, 30000, (n_seq, seq_len, row_elems)).astype(np.int16)
    visual = rng.integers(-30000, 30000, (n_seq, n_vis, row_elems)).astype(np.int16)
    keep = sorted_choice(rng, n_vis, k, n_seq)
    want = O.merge_embeddings(text, visual, keep, vis_start)
    out, chk = padded((n_seq, seq_len - n_vis + k, row_elems), torch.int16, 77)
    civic.civic_merge_embeddings(torch.from_numpy(text).to(DEV), torch.from_numpy(visual).to(DEV),
                                 torch.from_numpy(keep).to(DEV), vis_start, merged=out)
    assert np.array_equal(out.cpu().numpy(), want)
    chk()


def test_merge_embeddings_c3_full_size():
    """The benchmark's sequence shape: 16 x (16 text + 1024 visual + 48 text) rows of 8 KB."""
    wl = W.C3
    keep = O.select(W.scores(wl), wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, wl.k)
    visual = W.hidden(wl, DEV)
    text = W.payload_bf16((wl.n_seg, wl.seq_len, wl.hidden_dim), wl.seed + 700, DEV)
    W.stamp_rows(visual, wl.hidden_dim)
    W.stamp_rows(text, wl.hidden_dim)
    out, chk = padded((wl.n_seg, wl.s_out, wl.hidden_dim), torch.bfloat16, 5.0)
    civic.civic_merge_embeddings(text, visual, torch.from_numpy(keep).to(DEV), wl.text_before, merged=out)
    want = O.merge_embeddings(bits16(text), bits16(visual), keep, wl.text_before)
    assert np.array_equal(bits16(out), want)
    chk()
    assert out.shape[1] == wl.text_before + wl.text_after + wl.k  # Eq. 13: L + M_p rows


# ------------------------------------------------------------------ plane-major position ids

@pytest.mark.parametrize("n_planes,n_seq,seq_len,s_out", [(3, 2, 17, 6), (3, 4, 40, 40), (1, 1, 5, 1),
                                                          (4, 2, 9, 0), (3, 16, 1088, 405), (3, 4, 3136, 1045)])
def test_pos_planes(n_planes, n_seq, seq_len, s_out):
    rng = np.random.default_rng(seq_len)
    pos = rng.integers(-3, 50000, (n_planes, n_seq, seq_len)).astype(np.int32)
    idx = sorted_choice(rng, seq_len, s_out, n_seq)
    want = O.compact_pos_planes(pos, idx)
    out, chk = padded((n_planes, n_seq, s_out), torch.int32, CANARY)
    civic.civic_compact_pos_planes(torch.from_numpy(pos).to(DEV), torch.from_numpy(idx).to(DEV), pos_out=out)
    assert np.array_equal(out.cpu().numpy(), want)
    chk()


# ------------------------------------------------------------------ head-major K/V

def run_kv_heads(n_layers, n_seq, n_heads, seq_len, s_out, d, dtype=torch.int16, seed=0, idx=None):
    rng = np.random.default_rng(seed + seq_len)
    np_dt = np.int16 if dtype == torch.int16 else np.int32
    ks = [rng.integers(-30000, 30000, (n_seq, n_heads, seq_len, d)).astype(np_dt) for _ in range(n_layers)]
    vs = [rng.integers(-30000, 30000, (n_seq, n_heads, seq_len, d)).astype(np_dt) for _ in range(n_layers)]
    if idx is None:
        idx = sorted_choice(rng, seq_len, s_out, n_seq)
    want_k, want_v = O.compact_kv_heads(ks, vs, idx)
    outs = [padded((n_seq, n_heads, s_out, d), dtype, 99) for _ in range(2 * n_layers)]
    kd, vd = [o[0] for o in outs[:n_layers]], [o[0] for o in outs[n_layers:]]
    tables = civic.kv_heads_tables([torch.from_numpy(a).to(DEV) for a in ks],
                                   [torch.from_numpy(a).to(DEV) for a in vs], kd, vd)
    civic.civic_compact_kv_heads(tables, torch.from_numpy(idx).to(DEV))
    for l in range(n_layers):
        assert np.array_equal(kd[l].cpu().numpy(), want_k[l]), f"K layer {l}"
        assert np.array_equal(vd[l].cpu().numpy(), want_v[l]), f"V layer {l}"
    for _, chk in outs:
        chk()


def test_kv_heads_small_and_odd():
    run_kv_heads(2, 3, 4, 23, 9, 128)            # 256-byte pieces: eight to a warp tile
    run_kv_heads(1, 2, 3, 50, 17, 24)            # 48-byte pieces: 42 to a tile, two idle vectors
    run_kv_heads(2, 2, 2, 31, 31, 6)             # 12-byte pieces: 4-byte vector path
    run_kv_heads(1, 1, 5, 40, 13, 2)             # 4-byte pieces
    run_kv_heads(1, 2, 2, 20, 7, 1536)           # 3 KB pieces: long-row path
    run_kv_heads(1, 1, 1, 9, 9, 8, dtype=torch.int32)
    run_kv_heads(3, 2, 8, 77, 0, 128)            # nothing kept


def test_kv_heads_more_layers_than_one_launch():
    run_kv_heads(83, 1, 2, 19, 6, 16)


@pytest.mark.parametrize("wl", [W.C3.replace(n_layers=4), W.C5_THIRD.replace(n_layers=3)], ids=lambda w: w.name)
def test_kv_heads_workload_shapes(wl):
    """Benchmark sequence shapes with 8 heads of 128 bf16 (256-byte pieces), selection from the oracle."""
    keep = O.select(W.scores(wl), wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, wl.k)
    idx = O.seq_indices(keep, wl.seq_len, wl.text_before, wl.n)
    run_kv_heads(wl.n_layers, wl.n_seg, wl.kv_heads, wl.seq_len, wl.s_out, wl.head_dim, idx=idx)


# ------------------------------------------------------------------ paged K/V

def run_kv_paged(n_layers, n_seq, seq_len, s_out, row_elems, page, seed=0, idx=None):
    rng = np.random.default_rng(seed + seq_len + page)
    per_seq = -(-s_out // page) + 1
    n_pages = n_seq * per_seq + 3
    table = rng.permutation(n_pages)[: n_seq * per_seq].reshape(n_seq, per_seq).astype(np.int32)
    ks = [rng.integers(-30000, 30000, (n_seq, seq_len, row_elems)).astype(np.int16) for _ in range(n_layers)]
    vs = [rng.integers(-30000, 30000, (n_seq, seq_len, row_elems)).astype(np.int16) for _ in range(n_layers)]
    if idx is None:
        idx = sorted_choice(rng, seq_len, s_out, n_seq)
    old_k = [rng.integers(-9, 9, (n_pages, page, row_elems)).astype(np.int16) for _ in range(n_layers)]
    old_v = [rng.integers(-9, 9, (n_pages, page, row_elems)).astype(np.int16) for _ in range(n_layers)]
    want_k, want_v = [a.copy() for a in old_k], [a.copy() for a in old_v]
    O.compact_kv_paged(ks, vs, idx, table, page, want_k, want_v)
    outs = [padded((n_pages, page, row_elems), torch.int16, 99) for _ in range(2 * n_layers)]
    kc, vc = [o[0] for o in outs[:n_layers]], [o[0] for o in outs[n_layers:]]
    for dst, src in zip(kc + vc, old_k + old_v):
        dst.copy_(torch.from_numpy(src))
    tables = civic.kv_paged_tables([torch.from_numpy(a).to(DEV) for a in ks],
                                   [torch.from_numpy(a).to(DEV) for a in vs], kc, vc)
    civic.civic_compact_kv_paged(tables, torch.from_numpy(idx).to(DEV), torch.from_numpy(table).to(DEV))
    for l in range(n_layers):
        assert np.array_equal(kc[l].cpu().numpy(), want_k[l]), f"K cache layer {l}"
        assert np.array_equal(vc[l].cpu().numpy(), want_v[l]), f"V cache layer {l}"
    for _, chk in outs:
        chk()


def test_kv_paged_small_and_odd():
    run_kv_paged(2, 3, 29, 13, 1024, 4)    # 2 KB rows, ragged last page
    run_kv_paged(1, 2, 16, 16, 1024, 16)   # exactly one full page per sequence
    run_kv_paged(2, 2, 21, 7, 6, 1)        # page size 1, 12-byte rows
    run_kv_paged(1, 1, 10, 10, 2, 3)
    run_kv_paged(1, 3, 40, 11, 128, 5)     # 256-byte rows: several rows per warp tile
    run_kv_paged(2, 2, 33, 0, 64, 8)       # nothing kept: cache untouched
    run_kv_paged(1, 2, 64, 50, 2048, 16)   # 4 KB rows: two tiles per row


@pytest.mark.parametrize("wl", [W.C3.replace(n_layers=4), W.C5_HALF.replace(n_layers=2)], ids=lambda w: w.name)
def test_kv_paged_workload_shapes(wl):
    keep = O.select(W.scores(wl), wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, wl.k)
    idx = O.seq_indices(keep, wl.seq_len, wl.text_before, wl.n)
    run_kv_paged(wl.n_layers, wl.n_seg, wl.seq_len, wl.s_out, wl.kv_heads * wl.head_dim, 16, idx=idx)


def test_small_rows_take_the_packed_path_in_the_core_calls():
    """civic_compact / civic_compact_kv with rows shorter than a warp tile (packed several to a tile)."""
    rng = np.random.default_rng(3)
    for n_seg, n, k, row_elems in [(3, 300, 101, 8), (2, 90, 31, 24), (1, 500, 499, 2), (4, 64, 9, 256)]:
        hidden = rng.integers(-30000, 30000, (n_seg, n, row_elems)).astype(np.int16)
        pos = rng.integers(0, 999, (n_seg, n, 3)).astype(np.int32)
        keep = sorted_choice(rng, n, k, n_seg)
        want_h, want_p = O.compact(hidden, pos, keep)
        h_out, chk_h = padded((n_seg, k, row_elems), torch.int16, 77)
        p_out, chk_p = padded((n_seg, k, 3), torch.int32, CANARY)
        civic.civic_compact(torch.from_numpy(hidden).to(DEV), torch.from_numpy(pos).to(DEV),
                            torch.from_numpy(keep).to(DEV), hidden_out=h_out, pos_out=p_out)
        assert np.array_equal(h_out.cpu().numpy(), want_h) and np.array_equal(p_out.cpu().numpy(), want_p)
        chk_h()
        chk_p()
