"""Device-side validation of index arrays (needs a B200).

A compaction call reads its indices on the device, so a wrong entry is invisible to the host-side
validation.  With a fault record set (civic_set_index_check) the kernels test every index they
use: the offending row is neither read nor written and the record names it.  Each case plants ONE
bad entry in otherwise valid indices and checks
  * the record: (code, row, position, value) of the planted entry;
  * every other output row: equal to the oracle's result bit for bit;
  * the offending output row: still the canary the buffer was filled with (not written);
  * the padding around the outputs: intact.
The planted values point far outside the source tensors; no case is ever run without the check.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_28115_b200 import build, civic
from tests.test_gpu_parity import CANARY, DEV, padded

pytestmark = pytest.mark.gpu

O = oracle.default
FILL = 0x5A5A  # int16 canary of the payload outputs


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    civic.load()


def new_record():
    return torch.zeros(4, dtype=torch.int32, device=DEV)


def sorted_rows(rng, n, k, rows):
    return np.stack([np.sort(rng.choice(n, k, replace=False)) for _ in range(rows)]).astype(np.int32)


def assert_rows(got, want, skip, fill):
    """got == want except the rows in `skip` ((row, position) pairs), which still hold the canary."""
    mask = np.ones(got.shape[:2], bool)
    for r, j in skip:
        mask[r, j] = False
        assert np.all(got[r, j] == fill), f"row {(r, j)} with a bad index was written"
    assert np.array_equal(got[mask], want[mask])


BAD_VALUES = [-1, -2 ** 31, 50, 2 ** 31 - 1, 10 ** 6]  # n = 50 in the cases below


@pytest.mark.parametrize("bad", BAD_VALUES)
@pytest.mark.parametrize("row_elems", [8, 2, 1032])  # packed rows, 4-byte path, tiled rows
def test_compact_skips_and_reports_a_bad_index(bad, row_elems):
    rng = np.random.default_rng(abs(bad) % 1000 + row_elems)
    n_seg, n, k = 3, 50, 17
    hidden = rng.integers(-30000, 30000, (n_seg, n, row_elems)).astype(np.int16)
    pos = rng.integers(0, 99999, (n_seg, n, 3)).astype(np.int32)
    keep = sorted_rows(rng, n, k, n_seg)
    want_h, want_p = O.compact(hidden, pos, keep)
    planted = keep.copy()
    planted[1, 5] = bad
    rec = new_record()
    h_out, chk_h = padded((n_seg, k, row_elems), torch.int16, FILL)
    p_out, chk_p = padded((n_seg, k, 3), torch.int32, CANARY)
    with civic.index_check(rec):
        civic.civic_compact(torch.from_numpy(hidden).to(DEV), torch.from_numpy(pos).to(DEV),
                            torch.from_numpy(planted).to(DEV), hidden_out=h_out, pos_out=p_out)
    torch.cuda.synchronize()
    assert rec.cpu().tolist() == [1, 1, 5, bad]
    assert_rows(h_out.cpu().numpy(), want_h, [(1, 5)], FILL)
    assert_rows(p_out.cpu().numpy(), want_p, [(1, 5)], CANARY)
    chk_h()
    chk_p()


def test_check_on_valid_indices_changes_nothing_and_is_off_by_default():
    rng = np.random.default_rng(3)
    n_seg, n, k, row_elems = 2, 64, 20, 16
    hidden = rng.integers(-30000, 30000, (n_seg, n, row_elems)).astype(np.int16)
    keep = sorted_rows(rng, n, k, n_seg)
    want, _ = O.compact(hidden, None, keep)
    rec = new_record()
    with civic.index_check(rec):
        got, _ = civic.civic_compact(torch.from_numpy(hidden).to(DEV), None, torch.from_numpy(keep).to(DEV))
    assert rec.cpu().tolist() == [0, 0, 0, 0]
    assert np.array_equal(got.cpu().numpy(), want)
    # outside the context the record is no longer used: a later (valid) call leaves it alone
    rec.fill_(9)
    civic.civic_compact(torch.from_numpy(hidden).to(DEV), None, torch.from_numpy(keep).to(DEV))
    assert rec.cpu().tolist() == [9, 9, 9, 9]


@pytest.mark.parametrize("layout", ["token_major", "head_major", "paged"])
def test_kv_layouts_skip_and_report(layout):
    rng = np.random.default_rng(len(layout))
    n_layers, n_seq, seq_len, s_out, heads, d = 3, 2, 40, 13, 4, 16
    row = heads * d
    idx = sorted_rows(rng, seq_len, s_out, n_seq)
    ks = [rng.integers(-30000, 30000, (n_seq, seq_len, row)).astype(np.int16) for _ in range(n_layers)]
    vs = [rng.integers(-30000, 30000, (n_seq, seq_len, row)).astype(np.int16) for _ in range(n_layers)]
    want_k, want_v = O.compact_kv(ks, vs, idx)
    planted = idx.copy()
    planted[0, 7] = seq_len + 3
    rec = new_record()
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
    outs, checks = [], []
    if layout == "head_major":
        src = lambda a: dev(a.reshape(n_seq, seq_len, heads, d).transpose(0, 2, 1, 3))
        shape = (n_seq, heads, s_out, d)
    else:
        src = dev
        shape = (n_seq, s_out, row)
    page = 4
    per_seq = -(-s_out // page)
    if layout == "paged":
        shape = (n_seq * per_seq, page, row)
        table = rng.permutation(n_seq * per_seq).astype(np.int32).reshape(n_seq, per_seq)
    for _ in range(2 * n_layers):
        o, c = padded(shape, torch.int16, FILL)
        outs.append(o)
        checks.append(c)
    k_dst, v_dst = outs[:n_layers], outs[n_layers:]
    k_src, v_src = [src(a) for a in ks], [src(a) for a in vs]
    with civic.index_check(rec):
        if layout == "token_major":
            civic.civic_compact_kv(civic.kv_tables(k_src, v_src, k_dst, v_dst), dev(planted))
        elif layout == "head_major":
            civic.civic_compact_kv_heads(civic.kv_heads_tables(k_src, v_src, k_dst, v_dst), dev(planted))
        else:
            civic.civic_compact_kv_paged(civic.kv_paged_tables(k_src, v_src, k_dst, v_dst), dev(planted), dev(table))
    torch.cuda.synchronize()
    assert rec.cpu().tolist() == [1, 0, 7, seq_len + 3]
    for got_l, want_l in list(zip(k_dst, want_k)) + list(zip(v_dst, want_v)):
        got = got_l.cpu().numpy()
        if layout == "head_major":
            got = got.transpose(0, 2, 1, 3).reshape(n_seq, s_out, row)
        elif layout == "paged":
            flat = got.reshape(-1, row)
            slots = (table[:, np.arange(s_out) // page] * page + np.arange(s_out) % page)
            used = np.zeros(flat.shape[0], bool)
            used[slots.reshape(-1)] = True
            assert np.all(flat[~used] == FILL), "a slot outside the block table's range was written"
            got = flat[slots]
        assert_rows(got, want_l, [(0, 7)], FILL)
    for c in checks:
        c()


def test_paged_cache_bad_page_is_not_written():
    rng = np.random.default_rng(12)
    n_seq, seq_len, s_out, row, page = 2, 30, 10, 32, 4
    per_seq = -(-s_out // page)
    n_pages = n_seq * per_seq
    idx = sorted_rows(rng, seq_len, s_out, n_seq)
    ks = [rng.integers(-30000, 30000, (n_seq, seq_len, row)).astype(np.int16)]
    vs = [rng.integers(-30000, 30000, (n_seq, seq_len, row)).astype(np.int16)]
    table = rng.permutation(n_pages).astype(np.int32).reshape(n_seq, per_seq)
    want_k = [np.full((n_pages, page, row), FILL, np.int16)]
    want_v = [np.full((n_pages, page, row), FILL, np.int16)]
    O.compact_kv_paged(ks, vs, idx, table, page, want_k, want_v)
    lost = table[1, 2]  # the page of compact positions 8 and 9 of sequence 1
    want_k[0][lost] = FILL
    want_v[0][lost] = FILL
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
    for bad in (-1, n_pages, 2 ** 30):
        planted = table.copy()
        planted[1, 2] = bad
        rec = new_record()
        kc, chk_k = padded((n_pages, page, row), torch.int16, FILL)
        vc, chk_v = padded((n_pages, page, row), torch.int16, FILL)
        with civic.index_check(rec):
            civic.civic_compact_kv_paged(civic.kv_paged_tables([dev(ks[0])], [dev(vs[0])], [kc], [vc]), dev(idx),
                                         dev(planted))
        torch.cuda.synchronize()
        assert rec.cpu().tolist() == [3, 1, 2, bad]
        # every other row is in place; the rows of the bad page went nowhere
        assert np.array_equal(kc.cpu().numpy(), want_k[0])
        assert np.array_equal(vc.cpu().numpy(), want_v[0])
        chk_k()
        chk_v()


def test_merge_and_pos_planes_skip_and_report():
    rng = np.random.default_rng(21)
    n_seq, seq_len, vis_start, n_vis, k, row_elems = 2, 30, 4, 20, 7, 8
    text = rng.integers(-30000, 30000, (n_seq, seq_len, row_elems)).astype(np.int16)
    visual = rng.integers(-30000, 30000, (n_seq, n_vis, row_elems)).astype(np.int16)
    keep = sorted_rows(rng, n_vis, k, n_seq)
    want = O.merge_embeddings(text, visual, keep, vis_start)
    planted = keep.copy()
    planted[1, 0] = n_vis  # one past the end of the visual span
    rec = new_record()
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
    out, chk = padded((n_seq, seq_len - n_vis + k, row_elems), torch.int16, FILL)
    with civic.index_check(rec):
        civic.civic_merge_embeddings(dev(text), dev(visual), dev(planted), vis_start, merged=out)
    torch.cuda.synchronize()
    assert rec.cpu().tolist() == [1, 1, 0, n_vis]
    assert_rows(out.cpu().numpy(), want, [(1, vis_start)], FILL)
    chk()

    n_planes, s_out = 3, 11
    pos = rng.integers(0, 9999, (n_planes, n_seq, seq_len)).astype(np.int32)
    idx = sorted_rows(rng, seq_len, s_out, n_seq)
    want_p = O.compact_pos_planes(pos, idx)
    planted = idx.copy()
    planted[0, 10] = -7
    rec = new_record()
    p_out, chk = padded((n_planes, n_seq, s_out), torch.int32, CANARY)
    with civic.index_check(rec):
        civic.civic_compact_pos_planes(dev(pos), dev(planted), pos_out=p_out)
    torch.cuda.synchronize()
    assert rec.cpu().tolist() == [1, 0, 10, -7]
    got = p_out.cpu().numpy()
    assert np.all(got[:, 0, 10] == CANARY)
    got[:, 0, 10] = want_p[:, 0, 10]
    assert np.array_equal(got, want_p)
    chk()


def test_validate_indices():
    rng = np.random.default_rng(33)
    n_rows, row_len, limit = 5, 40, 300
    idx = sorted_rows(rng, limit, row_len, n_rows)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
    rec = new_record()
    civic.civic_validate_indices(dev(idx), limit, rec)
    assert rec.cpu().tolist() == [0, 0, 0, 0]
    # the indices the selection itself writes are valid
    s = torch.from_numpy(rng.random((3, 1024)).astype(np.float32)).to(DEV)
    keep, seq = civic.civic_select_seq(s, civic.SelectDesc(1, 32, 32, 4, 4, 1, 341), 1088, 16)
    civic.civic_validate_indices(keep, 1024, rec)
    civic.civic_validate_indices(seq, 1088, rec)
    assert rec.cpu().tolist() == [0, 0, 0, 0]
    # out of range: negative, == limit
    for bad in (-1, limit, 2 ** 31 - 1):
        planted = idx.copy()
        planted[3, 39] = bad
        rec = new_record()
        civic.civic_validate_indices(dev(planted), limit, rec, require_ascending=False)
        assert rec.cpu().tolist() == [1, 3, 39, bad]
    # a swapped pair and a repeated entry are "not ascending": the record names the second of the pair
    planted = idx.copy()
    planted[2, 10], planted[2, 11] = idx[2, 11], idx[2, 10]
    rec = new_record()
    civic.civic_validate_indices(dev(planted), limit, rec)
    assert rec.cpu().tolist() == [2, 2, 11, int(planted[2, 11])]
    rec = new_record()
    civic.civic_validate_indices(dev(planted), limit, rec, require_ascending=False)
    assert rec.cpu().tolist() == [0, 0, 0, 0]
    planted = idx.copy()
    planted[4, 1] = planted[4, 0]
    rec = new_record()
    civic.civic_validate_indices(dev(planted), limit, rec)
    assert rec.cpu().tolist() == [2, 4, 1, int(planted[4, 0])]
    # sticky: a second fault does not replace the first; a clean array does not clear it
    civic.civic_validate_indices(dev(idx), limit, rec)
    assert rec.cpu().tolist()[0] == 2
    # empty arrays enqueue nothing
    before = civic.launch_count()
    civic.civic_validate_indices(torch.zeros((0, 7), dtype=torch.int32, device=DEV), 5, rec)
    assert civic.launch_count() == before
