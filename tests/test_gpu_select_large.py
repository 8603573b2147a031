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
