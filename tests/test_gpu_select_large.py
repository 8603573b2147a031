"""Many-block selection (civic_select_large) against the CPU oracle, bit for bit (needs a B200)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_28115_b200 import build, civic
from paper_2605_28115_b200 import workloads as W
from tests.test_gpu_parity import CANARY, DEV

pytestmark = pytest.mark.gpu

O = oracle.default


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    civic.load()


def gpu_select_large(scores_np, t, h, w, rh, rw, m, k, chunk_tokens=0):
    """civic_select_large with canary-padded output and a workspace of exactly the advertised size,
    itself followed by a canary."""
    n_seg = scores_np.shape[0]
    desc = civic.SelectDesc(t, h, w, rh, rw, m, k)
    s = torch.from_numpy(np.ascontiguousarray(scores_np)).to(DEV)
    pad = 64
    buf = torch.full((n_seg * k + 2 * pad,), CANARY, dtype=torch.int32, device=DEV)
    out = buf[pad:pad + n_seg * k].view(n_seg, k)
    need = civic.select_workspace_bytes(desc, n_seg, chunk_tokens)
    assert need > 0
    ws_buf = torch.full((need + 512,), 0xA5, dtype=torch.uint8, device=DEV)
    civic.civic_select_large(s, desc, keep_idx=out, workspace=ws_buf[:need], chunk_tokens=chunk_tokens)
    torch.cuda.synchronize()
    host = buf.cpu().numpy()
    assert np.all(host[:pad] == CANARY) and np.all(host[pad + n_seg * k:] == CANARY), "wrote outside keep_idx"
    assert bool((ws_buf[need:] == 0xA5).all()), "wrote past the advertised workspace size"
    return host[pad:pad + n_seg * k].reshape(n_seg, k)


def assert_parity(scores_np, t, h, w, rh, rw, m, k, chunk_tokens=0):
    want = O.select(scores_np, t, h, w, rh, rw, m, k)
    got = gpu_select_large(scores_np, t, h, w, rh, rw, m, k, chunk_tokens)
    if not np.array_equal(got, want):
        bad = np.argwhere(got != want)[0]
        raise AssertionError(f"mismatch at {tuple(bad)}: got {got[tuple(bad)]}, want {want[tuple(bad)]} "
                             f"(grid {(t, h, w)}, region {(rh, rw)}, m={m}, k={k}, chunk {chunk_tokens})")


@pytest.mark.parametrize("wl", W.ALL, ids=lambda wl: wl.name)
def test_workloads_in_small_chunks(wl):
    """The benchmark workloads cut into many chunks per segment (one or a few region rows each)."""
    s = W.scores(wl)
    row = min(wl.region_h, wl.h) * wl.w
    n_res = O.reserved_count(wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m)
    for chunk in (row, 3 * row, 0):
        assert_parity(s, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, wl.k, chunk)
    assert_parity(s, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, 0, wl.k, row)
    assert_parity(s, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, n_res, 2 * row)
    assert_parity(s, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, wl.n, row)
    assert_parity(s, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, 2, max(wl.k, 2 * wl.n_regions), 2 * row)


def test_random_shapes_in_small_chunks():
    rng = np.random.default_rng(202)
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
        chunk = min(rh, h) * w * int(rng.integers(1, 4))
        assert_parity(s.astype(np.float32), t, h, w, rh, rw, m, k, chunk)


def test_special_values_and_all_equal():
    specials = np.array([0x80000000, 0x00000000, 0x7F800000, 0xFF800000, 0x00000001, 0x80000001,
                         0x7FC00000, 0xFFC00000, 0x7F800001, 0xFF800001, 0x7FFFFFFF, 0xFFFFFFFF,
                         0x3F800000, 0xBF800000, 0x007FFFFF, 0x807FFFFF], dtype=np.uint32)
    rng = np.random.default_rng(6)
    s = rng.choice(specials, size=(3, 8 * 8)).astype(np.uint32).view(np.float32)
    for m, k in [(0, 1), (0, 17), (0, 64), (1, 16), (1, 33), (2, 40)]:
        assert_parity(s, 1, 8, 8, 2, 2, m, k, 16)
    bits = rng.integers(0, 2 ** 32, size=(2, 1000), dtype=np.uint64).astype(np.uint32)
    assert_parity(bits.view(np.float32), 1, 25, 40, 5, 8, 1, 333, 200)
    ones = np.ones((2, 7 * 9), dtype=np.float32)
    for m, k in [(0, 10), (1, 20), (3, 40)]:
        assert_parity(ones, 1, 7, 9, 3, 4, m, k, 27)


@pytest.mark.parametrize("t,h,w,rh,rw,m,frac,kind", [
    (64, 56, 56, 4, 4, 1, 3, "quant"),      # 200 704 tokens: a 128-frame clip at 56x56
    (96, 48, 40, 4, 4, 2, 2, "lognormal"),  # 184 320 tokens, two reserved per tile
    (250, 64, 64, 8, 8, 1, 4, "uniform"),   # 1 024 000 tokens
    (3, 181, 211, 7, 5, 1, 3, "quant"),     # ragged tiles on both edges, 114 573 tokens
])
def test_long_videos(t, h, w, rh, rw, m, frac, kind):
    rng = np.random.default_rng(t * 1000 + h)
    n = t * h * w
    u = rng.random((2, n))
    s = {"quant": np.floor(u * 256) / 256, "lognormal": np.exp(rng.standard_normal((2, n))), "uniform": u}[kind]
    assert_parity(s.astype(np.float32), t, h, w, rh, rw, m, n // frac)


def test_default_chunking_takes_one_launch_of_block_clusters():
    """Segments up to 16 K tokens (and batches of larger ones) with the library's own chunking: one launch, a
    cluster of four blocks per segment."""
    rng = np.random.default_rng(77)
    specials = np.array([0x80000000, 0x00000000, 0x7F800000, 0xFF800000, 0x00000001, 0x80000001, 0x7FC00000,
                         0xFFC00000, 0x3F800000, 0xBF800000], dtype=np.uint32).view(np.float32)
    done = 0
    for trial in range(200):
        t = int(rng.integers(1, 7))
        h = int(rng.integers(4, 90))
        w = int(rng.integers(4, 90))
        rh = int(rng.integers(1, 12))
        rw = int(rng.integers(1, 12))
        m = int(rng.integers(0, 4))
        n = t * h * w
        if n > 16384 or done == 48:
            continue
        done += 1
        n_res = O.reserved_count(t, h, w, rh, rw, m)
        k = [n_res, n, int(rng.integers(n_res, n + 1))][done % 3] if done % 5 == 0 else int(rng.integers(n_res, n + 1))
        n_seg = int(rng.integers(1, 4))
        kind = done % 4
        if kind == 0:
            s = rng.random((n_seg, n))
        elif kind == 1:
            s = rng.integers(0, 5, (n_seg, n))  # heavy ties: the threshold class spans the blocks
        elif kind == 2:
            s = rng.choice(specials, size=(n_seg, n))
        else:
            s = np.exp(rng.standard_normal((n_seg, n)) * 8)  # wide exponent range
        before = civic.launch_count()
        assert_parity(np.asarray(s, dtype=np.float32), t, h, w, rh, rw, m, k)
        assert civic.launch_count() - before == (1 if k > 0 else 0), (t, h, w, rh, rw, m, k)
    assert done == 48
    # two region rows for a cluster of four blocks: the last two blocks hold nothing
    s = rng.random((2, 64 * 128)).astype(np.float32)
    before = civic.launch_count()
    assert_parity(s, 1, 64, 128, 32, 16, 1, 3000)
    assert civic.launch_count() - before == 1
    # all scores equal: every kept token beyond the floor is a tie split by index across the blocks
    ones = np.ones((2, 3 * 60 * 70), dtype=np.float32)
    for m, k in [(0, 1), (1, 5000), (2, 12600)]:
        assert_parity(ones, 3, 60, 70, 6, 7, m, k)
    # a batch of mid-sized segments (more tokens than one wave of small blocks): still one launch
    s = np.floor(rng.random((8, 16 * 56 * 56)) * 256).astype(np.float32)
    before = civic.launch_count()
    assert_parity(s, 16, 56, 56, 4, 4, 1, 16 * 56 * 56 // 3)
    assert civic.launch_count() - before == 1


def test_agrees_with_the_one_block_kernel_at_its_largest_segment():
    n_max = civic.select_max_tokens()
    h = 64
    w = n_max // h
    rng = np.random.default_rng(10)
    s = np.floor(rng.random((2, h * w)) * 4096).astype(np.float32)
    desc = civic.SelectDesc(1, h, w, 8, 8, 1, (h * w) // 3)
    d = torch.from_numpy(s).to(DEV)
    a = civic.civic_select(d, desc)
    b = civic.civic_select_large(d, desc)
    assert torch.equal(a, b)
    assert np.array_equal(b.cpu().numpy(), O.select(s, 1, h, w, 8, 8, 1, (h * w) // 3))


def test_workspace_errors_and_reuse():
    desc = civic.SelectDesc(4, 40, 40, 4, 4, 1, 2000)
    s = torch.rand((2, 6400), device=DEV)
    need = civic.select_workspace_bytes(desc, 2)
    ws = torch.empty(need, dtype=torch.uint8, device=DEV)
    with pytest.raises(civic.CivicError, match="WORKSPACE"):
        civic.civic_select_large(s, desc, workspace=ws[: need - 256])
    with pytest.raises(civic.CivicError, match="ALIGNMENT"):
        civic.civic_select_large(s, desc, workspace=torch.empty(need + 64, dtype=torch.uint8, device=DEV)[16:])
    with pytest.raises(civic.CivicError, match="UNSUPPORTED"):  # a region row of 160 tokens > 100
        civic.civic_select_large(s, desc, workspace=ws, chunk_tokens=100)
    # the same workspace, dirty from the previous call, serves the next one
    want = O.select(s.cpu().numpy(), 4, 40, 40, 4, 4, 1, 2000)
    for _ in range(3):
        got = civic.civic_select_large(s, desc, workspace=ws)
        assert np.array_equal(got.cpu().numpy(), want)


# ------------------------------------------------------------------ ragged batches

def run_ragged(descs, parts):
    scores = np.concatenate(parts).astype(np.float32)
    want_keep, want_flat = O.select_ragged(scores, descs)
    total_k = len(want_keep)
    pad = 64
    bufs = [torch.full((total_k + 2 * pad,), CANARY, dtype=torch.int32, device=DEV) for _ in range(2)]
    keep, flat = (b[pad:pad + total_k] for b in bufs)
    civic.civic_select_ragged(torch.from_numpy(scores).to(DEV), [civic.SelectDesc(*d) for d in descs],
                              keep_idx=keep, flat_idx=flat)
    assert np.array_equal(keep.cpu().numpy(), want_keep)
    assert np.array_equal(flat.cpu().numpy(), want_flat)
    for b in bufs:
        host = b.cpu().numpy()
        assert np.all(host[:pad] == CANARY) and np.all(host[pad + total_k:] == CANARY)
    return scores, want_keep, want_flat


def test_ragged_random_batches():
    rng = np.random.default_rng(303)
    for trial in range(25):
        descs, parts = [], []
        for _ in range(int(rng.integers(1, 9))):
            t, h, w = int(rng.integers(1, 4)), int(rng.integers(1, 40)), int(rng.integers(1, 40))
            rh, rw = int(rng.integers(1, min(h, 8) + 1)), int(rng.integers(1, min(w, 8) + 1))
            m = int(rng.integers(0, 3))
            n = t * h * w
            k = int(rng.integers(O.reserved_count(t, h, w, rh, rw, m), n + 1))
            descs.append((t, h, w, rh, rw, m, k))
            parts.append(rng.integers(0, 6, n) if trial % 2 else rng.random(n))
        run_ragged(descs, parts)


def test_ragged_mixed_workloads_compacts_in_one_call():
    """Images and a video of the benchmark shapes in one batch, budgets differing per segment
    (one of them from a Min-Keep-Ratio floor); the flat indices compact the whole batch at once."""
    m_ratio = civic.floor_from_ratio(4, 4, 1, 5)
    assert m_ratio == O.floor_from_ratio(4, 4, 1, 5) == 4
    shapes = [(W.C1, 65, 1), (W.C2, 341, 1), (W.C4, 1045, 1), (W.C5_THIRD, 1500, m_ratio), (W.C2, 0, 0),
              (W.C2, 512, 2)]
    descs = [(wl.t, wl.h, wl.w, wl.region_h, wl.region_w, m, k) for wl, k, m in shapes]
    parts = [W.scores(wl, seg=i % wl.n_seg) for i, (wl, _, _) in enumerate(shapes)]
    scores, keep, flat = run_ragged(descs, parts)
    total_n, total_k = len(scores), len(keep)
    rng = np.random.default_rng(1)
    hidden = rng.integers(-30000, 30000, (1, total_n, 64)).astype(np.int16)
    pos = rng.integers(0, 99, (1, total_n, 3)).astype(np.int32)
    h_out, p_out = civic.civic_compact(torch.from_numpy(hidden).to(DEV), torch.from_numpy(pos).to(DEV),
                                       torch.from_numpy(flat[None]).to(DEV))
    want_h, want_p = O.compact(hidden, pos, flat[None])
    assert np.array_equal(h_out.cpu().numpy(), want_h) and np.array_equal(p_out.cpu().numpy(), want_p)
    assert h_out.shape == (1, total_k, 64)


def test_ragged_more_segments_than_one_launch():
    rng = np.random.default_rng(304)
    descs = [(1, 6, 7, 2, 3, 1, int(rng.integers(9, 42))) for _ in range(150)]
    run_ragged(descs, [rng.random(42) for _ in descs])


def test_floor_from_ratio_matches_the_oracle():
    for rh in range(1, 7):
        for rw in range(1, 7):
            for den in range(1, 9):
                for num in range(0, den + 1):
                    assert civic.floor_from_ratio(rh, rw, num, den) == O.floor_from_ratio(rh, rw, num, den)
    assert civic.floor_from_ratio(4, 4, 3, 2) == -1
    # Table 2's ratios on the benchmark's 4x4 tiles, run through the selection
    wl = W.C5_HALF
    s = W.scores(wl)
    for num, den in [(0, 1), (1, 5), (1, 2)]:
        m = civic.floor_from_ratio(wl.region_h, wl.region_w, num, den)
        k = max(wl.k, m * wl.n_regions)
        want = O.select(s, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, m, k)
        got = civic.civic_select(torch.from_numpy(s).to(DEV), civic.SelectDesc(wl.t, wl.h, wl.w, wl.region_h, wl.region_w, m, k))
        assert np.array_equal(got.cpu().numpy(), want)
