"""CUDA path against the CPU oracle, bit for bit, through the C ABI (needs a B200)."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2605_28115_b200 import build, civic
from paper_2605_28115_b200 import workloads as W

pytestmark = pytest.mark.gpu

O = oracle.default
DEV = "cuda:0"
CANARY = -0x5A5A5A5B


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    civic.load()


def gpu_select(scores_np, t, h, w, rh, rw, m, k):
    """Runs civic_select into a canary-padded buffer and checks the padding afterwards."""
    n_seg = scores_np.shape[0]
    s = torch.from_numpy(np.ascontiguousarray(scores_np)).to(DEV)
    pad = 64
    buf = torch.full((n_seg * k + 2 * pad,), CANARY, dtype=torch.int32, device=DEV)
    out = buf[pad:pad + n_seg * k].view(n_seg, k)
    civic.civic_select(s, civic.SelectDesc(t, h, w, rh, rw, m, k), keep_idx=out)
    torch.cuda.synchronize()
    host = buf.cpu().numpy()
    assert np.all(host[:pad] == CANARY) and np.all(host[pad + n_seg * k:] == CANARY), "wrote outside keep_idx"
    return host[pad:pad + n_seg * k].reshape(n_seg, k)


def assert_select_parity(scores_np, t, h, w, rh, rw, m, k):
    want = O.select(scores_np, t, h, w, rh, rw, m, k)
    got = gpu_select(scores_np, t, h, w, rh, rw, m, k)
    if not np.array_equal(got, want):
        bad = np.argwhere(got != want)[0]
        raise AssertionError(f"select mismatch at {tuple(bad)}: got {got[tuple(bad)]}, want {want[tuple(bad)]} "
                             f"(grid {(t, h, w)}, region {(rh, rw)}, m={m}, k={k})")


# ------------------------------------------------------------------ select

@pytest.mark.parametrize("wl", W.ALL, ids=lambda wl: wl.name)
def test_select_workloads(wl):
    assert_select_parity(W.scores(wl), wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, wl.k)


@pytest.mark.parametrize("wl", W.ALL, ids=lambda wl: wl.name)
def test_select_workloads_variants(wl):
    s = W.scores(wl)
    n_res = O.reserved_count(wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m)
    # plain top-K, the tightest budget (only the floor), one more, everything, two per region
    assert_select_parity(s, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, 0, wl.k)
    assert_select_parity(s, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, n_res)
    assert_select_parity(s, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, n_res + 1)
    assert_select_parity(s, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, wl.n)
    assert_select_parity(s, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, 2, max(wl.k, 2 * wl.n_regions))
    # forced-active floor: scores concentrated in one corner
    ramp = np.arange(wl.n, dtype=np.float32)[None].repeat(wl.n_seg, 0)
    assert_select_parity(ramp, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, wl.k)
    assert_select_parity(-ramp, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, wl.k)


def test_select_random_shapes():
    rng = np.random.default_rng(101)
    for trial in range(120):
        t = int(rng.integers(1, 5))
        h = int(rng.integers(1, 50))
        w = int(rng.integers(1, 50))
        rh = int(rng.integers(1, min(h, 9) + 1))
        rw = int(rng.integers(1, min(w, 9) + 1))
        m = int(rng.integers(0, 4))
        n = t * h * w
        n_res = O.reserved_count(t, h, w, rh, rw, m)
        k = int(rng.integers(n_res, n + 1))
        n_seg = int(rng.integers(1, 4))
        kind = trial % 4
        if kind == 0:
            s = rng.random((n_seg, n))
        elif kind == 1:
            s = rng.integers(0, 5, (n_seg, n))  # heavy ties
        elif kind == 2:
            s = rng.standard_normal((n_seg, n)) * 1e3  # both signs
        else:
            s = np.exp(rng.standard_normal((n_seg, n)) * 8)  # wide exponent range
        assert_select_parity(s.astype(np.float32), t, h, w, rh, rw, m, k)


def test_select_all_equal_and_degenerate_regions():
    s = np.ones((2, 7 * 9), dtype=np.float32)
    for m, k in [(0, 10), (1, 20), (3, 40)]:
        assert_select_parity(s, 1, 7, 9, 3, 4, m, k)
    # one region covering the whole grid, 1x1 regions, m larger than the region
    r = np.random.default_rng(1).random((1, 12 * 12)).astype(np.float32)
    assert_select_parity(r, 1, 12, 12, 12, 12, 5, 30)
    assert_select_parity(r, 1, 12, 12, 1, 1, 1, 144)
    assert_select_parity(r, 1, 12, 12, 5, 5, 40, 144)
    assert_select_parity(r, 1, 12, 12, 5, 5, 4, 9 * 4 + 3)
    # single token
    assert_select_parity(np.zeros((3, 1), np.float32), 1, 1, 1, 1, 1, 1, 1)


def test_select_floor_of_one_by_slots_and_by_tile_walk():
    """m = 1 beyond one token per thread: large tiles take the regions' maxima through shared-memory slots,
    small tiles are walked by one thread each; both with ragged edge tiles and with ties inside the tiles."""
    rng = np.random.default_rng(7)
    for t, h, w, rh, rw in [(1, 40, 45, 10, 10), (2, 30, 33, 9, 8), (1, 40, 45, 3, 3), (3, 25, 31, 8, 8), (1, 50, 50, 7, 9)]:
        n = t * h * w
        n_res = O.reserved_count(t, h, w, rh, rw, 1)
        for s in (rng.random((2, n)), rng.integers(0, 4, (2, n)), np.exp(rng.standard_normal((2, n)) * 6)):
            for k in (n_res, n_res + 1, (n + n_res) // 2):
                assert_select_parity(s.astype(np.float32), t, h, w, rh, rw, 1, k)


def test_select_threshold_decided_by_the_leading_digits():
    """Keys built so that the radix search can stop after its first, second or third digit (the threshold bin
    is wanted whole), with several different keys inside the bins that are taken whole."""
    rng = np.random.default_rng(31)
    n = 24 * 24
    for low_bits in (24, 16, 8, 0):  # key bits below the digit that decides
        # a few well separated groups in the leading bits, arbitrary bits below
        lead = rng.integers(1, 40, size=(2, n)).astype(np.uint32)
        low = rng.integers(0, 1 << low_bits, size=(2, n)).astype(np.uint32) if low_bits else np.zeros((2, n), np.uint32)
        bits = (np.uint32(0x30000000) + (lead << np.uint32(low_bits)) + low).astype(np.uint32)
        s = bits.view(np.float32)
        assert np.all(np.isfinite(s))
        counts = np.bincount(lead[0], minlength=40)
        above = int(counts[20:].sum())  # exactly the tokens of the groups 20..39 of segment 0: whole bins
        for m, k in [(0, max(above, 1)), (0, 7), (1, 36 + 50), (2, 300), (0, n - 1)]:
            assert_select_parity(s, 1, 24, 24, 4, 4, m, k)
    # powers of four: every token alone in its leading-digit bin, any K stops after the first digit
    p4 = (4.0 ** -np.arange(60, dtype=np.float64)).astype(np.float32)[None, :]
    for k in (1, 17, 59, 60):
        assert_select_parity(np.ascontiguousarray(p4[:, ::-1]), 1, 6, 10, 2, 5, 0, k)
        assert_select_parity(p4, 1, 6, 10, 2, 5, 1, max(k, 6))


def test_select_special_values():
    specials = np.array([0x80000000, 0x00000000, 0x7F800000, 0xFF800000, 0x00000001, 0x80000001,
                         0x7FC00000, 0xFFC00000, 0x7F800001, 0xFF800001, 0x7FFFFFFF, 0xFFFFFFFF,
                         0x3F800000, 0xBF800000, 0x007FFFFF, 0x807FFFFF], dtype=np.uint32)
    rng = np.random.default_rng(5)
    bits = rng.choice(specials, size=(3, 8 * 8)).astype(np.uint32)
    s = bits.view(np.float32)
    for m, k in [(0, 0), (0, 1), (0, 17), (0, 64), (1, 16), (1, 33), (2, 40)]:
        if k == 0:
            continue
        assert_select_parity(s, 1, 8, 8, 2, 2, m, k)
    # arbitrary bit patterns
    bits = rng.integers(0, 2 ** 32, size=(2, 1000), dtype=np.uint64).astype(np.uint32)
    assert_select_parity(bits.view(np.float32), 1, 25, 40, 5, 8, 1, 333)


def test_select_largest_segment():
    n_max = civic.select_max_tokens()
    h = 64
    w = n_max // h
    rng = np.random.default_rng(9)
    s = np.floor(rng.random((2, h * w)) * 4096).astype(np.float32)  # ties too
    assert_select_parity(s, 1, h, w, 8, 8, 1, (h * w) // 3)
    assert_select_parity(s, 1, h, w, 8, 8, 0, (h * w) // 2)
    with pytest.raises(civic.CivicError, match="UNSUPPORTED"):
        civic.civic_select(torch.zeros((1, 300 * 300), device=DEV), civic.SelectDesc(1, 300, 300, 2, 2, 0, 5))


def test_select_many_segments_and_determinism():
    wl = W.C2.replace(n_seg=300)
    s = W.scores(wl)
    a = gpu_select(s, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, 1, wl.k)
    b = gpu_select(s, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, 1, wl.k)
    assert np.array_equal(a, b)
    assert np.array_equal(a, O.select(s, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, 1, wl.k))


# ------------------------------------------------------------------ compaction

def bits16(x: torch.Tensor) -> np.ndarray:
    return x.contiguous().view(torch.int16).cpu().numpy()


def padded(shape, dtype, fill):
    """A tensor carved out of a larger canary-filled buffer, plus a checker for the padding."""
    numel = int(np.prod(shape))
    pad = 256
    buf = torch.full((numel + 2 * pad,), fill, dtype=dtype, device=DEV)
    view = buf[pad:pad + numel].view(*shape)

    def check():
        host = buf.cpu()
        assert bool((host[:pad] == fill).all()) and bool((host[pad + numel:] == fill).all()), \
            "wrote outside the output buffer"

    return view, check


@pytest.mark.parametrize("wl", [W.C1, W.C2, W.C3, W.C4, W.C5_HALF, W.C5_THIRD, W.C5_QUARTER], ids=lambda wl: wl.name)
def test_compact_workloads(wl):
    s = W.scores(wl)
    keep = O.select(s, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, wl.k)
    hidden = W.hidden(wl, DEV)
    W.stamp_rows(hidden, wl.hidden_dim)
    pos = W.pos_ids(wl)
    h_out, chk_h = padded((wl.n_seg, wl.k, wl.hidden_dim), torch.bfloat16, 7.0)
    p_out, chk_p = padded((wl.n_seg, wl.k, 3), torch.int32, CANARY)
    civic.civic_compact(hidden, torch.from_numpy(pos).to(DEV), torch.from_numpy(keep).to(DEV),
                        hidden_out=h_out, pos_out=p_out)
    torch.cuda.synchronize()
    want_h, want_p = O.compact(bits16(hidden), pos, keep)
    assert np.array_equal(bits16(h_out), want_h)
    assert np.array_equal(p_out.cpu().numpy(), want_p)
    chk_h()
    chk_p()


def test_compact_odd_rows_and_optional_payloads():
    rng = np.random.default_rng(77)
    for n_seg, n, k, row_elems, dtype in [(3, 50, 17, 6, torch.int16), (2, 33, 33, 2, torch.int16),
                                          (1, 9, 1, 10, torch.int32), (5, 130, 64, 136, torch.int16),
                                          (2, 70, 23, 1, torch.int32), (2, 40, 11, 1032, torch.int16)]:
        np_dt = np.int16 if dtype == torch.int16 else np.int32
        hidden = rng.integers(-30000, 30000, (n_seg, n, row_elems)).astype(np_dt)
        pos = rng.integers(-9, 99999, (n_seg, n, 3)).astype(np.int32)
        keep = np.stack([np.sort(rng.choice(n, k, replace=False)) for _ in range(n_seg)]).astype(np.int32)
        want_h, want_p = O.compact(hidden, pos, keep)
        dh, dp, dk = (torch.from_numpy(a).to(DEV) for a in (hidden, pos, keep))
        h_out, chk_h = padded((n_seg, k, row_elems), dtype, 77)
        p_out, chk_p = padded((n_seg, k, 3), torch.int32, CANARY)
        civic.civic_compact(dh, dp, dk, hidden_out=h_out, pos_out=p_out)
        assert np.array_equal(h_out.cpu().numpy(), want_h)
        assert np.array_equal(p_out.cpu().numpy(), want_p)
        chk_h()
        chk_p()
        only_h, none = civic.civic_compact(dh, None, dk)
        assert none is None and np.array_equal(only_h.cpu().numpy(), want_h)
        none, only_p = civic.civic_compact(None, dp, dk)
        assert none is None and np.array_equal(only_p.cpu().numpy(), want_p)
    # a misaligned (4-byte aligned only) hidden buffer must still be exact
    base = torch.from_numpy(rng.integers(-30000, 30000, 3 * 20 * 8 + 2).astype(np.int16)).to(DEV)
    hid = base[2:].view(3, 20, 8)
    keep = np.stack([np.sort(rng.choice(20, 7, replace=False)) for _ in range(3)]).astype(np.int32)
    got, _ = civic.civic_compact(hid, None, torch.from_numpy(keep).to(DEV))
    want, _ = O.compact(hid.cpu().numpy(), None, keep)
    assert np.array_equal(got.cpu().numpy(), want)


def test_seq_indices():
    rng = np.random.default_rng(55)
    for n_seq, seq_len, vis_start, n_vis, k in [(3, 20, 3, 12, 5), (2, 12, 0, 12, 4), (4, 15, 5, 10, 10),
                                                (2, 9, 9, 0, 0), (1, 30, 0, 7, 0), (16, 1088, 16, 1024, 341),
                                                (4, 3136, 0, 3136, 1045)]:
        keep = (np.stack([np.sort(rng.choice(n_vis, k, replace=False)) for _ in range(n_seq)]).astype(np.int32)
                if n_vis else np.zeros((n_seq, 0), np.int32))
        want = O.seq_indices(keep, seq_len, vis_start, n_vis)
        out, chk = padded((n_seq, seq_len - n_vis + k), torch.int32, CANARY)
        civic.civic_seq_indices(torch.from_numpy(keep).to(DEV), seq_len, vis_start, n_vis, seq_idx=out)
        assert np.array_equal(out.cpu().numpy(), want)
        chk()


def test_select_seq_fused_matches_the_two_calls():
    """One launch writes keep_idx and seq_idx; both equal the oracle's select and sequence indices."""
    rng = np.random.default_rng(808)
    cases = [(W.C3, 16, 48), (W.C3.replace(n_seg=3), 0, 0), (W.C5_THIRD, 5, 0), (W.C4, 0, 7),
             (W.C1, 3, 2)]
    for wl, before, after in cases:
        s = W.scores(wl)
        seq_len = before + wl.n + after
        for k in (wl.k, O.reserved_count(wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m), wl.n):
            want_keep = O.select(s, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, k)
            want_seq = O.seq_indices(want_keep, seq_len, before, wl.n)
            keep, chk_k = padded((wl.n_seg, k), torch.int32, CANARY)
            seq, chk_s = padded((wl.n_seg, seq_len - wl.n + k), torch.int32, CANARY)
            desc = civic.SelectDesc(wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, k)
            civic.civic_select_seq(torch.from_numpy(s).to(DEV), desc, seq_len, before, keep_idx=keep, seq_idx=seq)
            assert np.array_equal(keep.cpu().numpy(), want_keep)
            assert np.array_equal(seq.cpu().numpy(), want_seq)
            chk_k()
            chk_s()
    # k = 0: only text survives
    s = rng.random((2, 6 * 6)).astype(np.float32)
    keep, seq = civic.civic_select_seq(torch.from_numpy(s).to(DEV), civic.SelectDesc(1, 6, 6, 2, 2, 0, 0), 41, 2)
    assert keep.shape == (2, 0)
    assert np.array_equal(seq.cpu().numpy(), O.seq_indices(np.zeros((2, 0), np.int32), 41, 2, 36))


def test_plain_launches_give_the_same_results():
    """Programmatic dependent launch switched off: same bytes."""
    wl = W.C3.replace(n_seg=3, n_layers=2)
    old = civic.set_programmatic_launch(False)
    try:
        assert old is True
        run_kv(wl)
    finally:
        civic.set_programmatic_launch(True)
    run_kv(wl)


def run_kv(wl, layers_on_host=True):
    """select -> seq_indices -> compact_kv on the GPU; oracle on the host copy of the same inputs."""
    s = W.scores(wl)
    keep_o = O.select(s, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, wl.k)
    idx_o = O.seq_indices(keep_o, wl.seq_len, wl.text_before, wl.n)
    desc = civic.SelectDesc(wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, wl.k)
    keep = civic.civic_select(torch.from_numpy(s).to(DEV), desc)
    idx = civic.civic_seq_indices(keep, wl.seq_len, wl.text_before, wl.n)
    assert np.array_equal(keep.cpu().numpy(), keep_o)
    assert np.array_equal(idx.cpu().numpy(), idx_o)
    ks = [W.kv_layer(wl, l, 0, DEV) for l in range(wl.n_layers)]
    vs = [W.kv_layer(wl, l, 1, DEV) for l in range(wl.n_layers)]
    for x in ks + vs:
        W.stamp_rows(x, wl.kv_heads * wl.head_dim)
    shape = (wl.n_seg, wl.s_out, wl.kv_heads, wl.head_dim)
    outs = [padded(shape, torch.bfloat16, 3.0) for _ in range(2 * wl.n_layers)]
    kd = [o[0] for o in outs[:wl.n_layers]]
    vd = [o[0] for o in outs[wl.n_layers:]]
    civic.civic_compact_kv(civic.kv_tables(ks, vs, kd, vd), idx)
    torch.cuda.synchronize()
    row = wl.kv_heads * wl.head_dim
    flat = lambda x: bits16(x).reshape(wl.n_seg, -1, row)
    want_k, want_v = O.compact_kv([flat(x) for x in ks], [flat(x) for x in vs], idx_o)
    for l in range(wl.n_layers):
        assert np.array_equal(flat(kd[l]), want_k[l]), f"K layer {l}"
        assert np.array_equal(flat(vd[l]), want_v[l]), f"V layer {l}"
    for _, chk in outs:
        chk()
    return sum(x.numel() * 2 for x in kd + vd), sum(x.numel() * 2 for x in ks + vs)


def test_compact_kv_small():
    # several tiles and a ragged tail: 3 layers, 405 and 1045 output rows
    run_kv(W.C3.replace(n_seg=3, n_layers=3))
    run_kv(W.C5_THIRD.replace(n_seg=2, n_layers=2))
    # tiny rows, odd sizes
    run_kv(W.C1.replace(n_layers=2, kv_heads=1, head_dim=6, text_before=5, text_after=3))
    run_kv(W.C1.replace(n_layers=1, kv_heads=3, head_dim=40, text_before=0, text_after=1))


def test_compact_kv_more_layers_than_one_launch():
    run_kv(W.C1.replace(n_layers=83, kv_heads=2, head_dim=16, text_before=2, text_after=2))


@pytest.mark.parametrize("wl", [W.C3, W.C5_HALF, W.C5_THIRD, W.C5_QUARTER], ids=lambda wl: wl.name)
def test_compact_kv_full_size(wl):
    """Full benchmark sizes, every output byte compared; Eq. 14's cache ratio holds exactly."""
    compact_bytes, dense_bytes = run_kv(wl)
    L = wl.text_before + wl.text_after
    assert compact_bytes * (L + wl.n) == dense_bytes * (L + wl.k)
    assert 2 * compact_bytes == W.kv_algorithmic_bytes(wl)


def test_pinned_host_buffers_zero_copy():
    """Payload sources and results in pinned host memory: the kernels read and write them
    directly; results must still equal the oracle's."""
    wl = W.C3.replace(n_seg=3, n_layers=2)
    s = W.scores(wl)
    keep_o = O.select(s, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, wl.k)
    idx_o = O.seq_indices(keep_o, wl.seq_len, wl.text_before, wl.n)
    pin = lambda x: torch.empty(x.shape, dtype=x.dtype, pin_memory=True).copy_(x)
    keep = torch.from_numpy(keep_o).to(DEV)
    idx = torch.from_numpy(idx_o).to(DEV)
    hidden = pin(W.hidden(wl, "cpu"))
    pos = W.pos_ids(wl)
    h_out = torch.zeros((wl.n_seg, wl.k, wl.hidden_dim), dtype=torch.bfloat16).pin_memory()
    p_out = torch.zeros((wl.n_seg, wl.k, 3), dtype=torch.int32).pin_memory()
    civic.civic_compact(hidden, pin(torch.from_numpy(pos)), keep, hidden_out=h_out, pos_out=p_out)
    ks = [pin(W.kv_layer(wl, l, 0, "cpu")) for l in range(wl.n_layers)]
    vs = [pin(W.kv_layer(wl, l, 1, "cpu")) for l in range(wl.n_layers)]
    shape = (wl.n_seg, wl.s_out, wl.kv_heads, wl.head_dim)
    kd = [torch.zeros(shape, dtype=torch.bfloat16).pin_memory() for _ in ks]
    vd = [torch.zeros(shape, dtype=torch.bfloat16).pin_memory() for _ in vs]
    civic.civic_compact_kv(civic.kv_tables(ks, vs, kd, vd), idx)
    torch.cuda.synchronize()
    want_h, want_p = O.compact(bits16(hidden), pos, keep_o)
    assert np.array_equal(bits16(h_out), want_h) and np.array_equal(p_out.numpy(), want_p)
    row = wl.kv_heads * wl.head_dim
    flat = lambda x: bits16(x).reshape(wl.n_seg, -1, row)
    want_k, want_v = O.compact_kv([flat(x) for x in ks], [flat(x) for x in vs], idx_o)
    for l in range(wl.n_layers):
        assert np.array_equal(flat(kd[l]), want_k[l]) and np.array_equal(flat(vd[l]), want_v[l])
    with pytest.raises(ValueError, match="pinned"):
        civic.civic_compact(W.hidden(wl, "cpu"), None, keep)
