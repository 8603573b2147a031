"""Compact visual aggregation (Eq. 8) on the tensor cores against the fp64 oracle (needs a B200).

Tolerance, from the arithmetic of the CUDA path (inputs are bf16 tokens and fp32 anchors, the same
for both sides):
  * the normalised anchors are rounded to bf16 (relative 2^-9 per element) and the products are
    accumulated in fp32 over d_v terms, so a cosine is off by at most
        d_cos = 2^-9 + d_v * 2^-24        (Cauchy-Schwarz: sum |q_j k_j| <= 1);
  * a weight exp(cos / tau) / sum is then off by at most the factor exp(2 d_cos / tau), and its
    bf16 rounding (numerator and the sum of the rounded values) adds 2 * 2^-9:
        eps_w = exp(2 d_cos / tau) - 1 + 2^-8;
  * Z_0 = W_A X_0 inherits eps_w relative to sum_i W_A[m, i] |x_i|, plus 2^-9 |Z_0| for the bf16
    result:   |Z_gpu - Z_oracle| <= eps_w * (W_A |X_0|) + 2^-9 |Z_0|   element by element;
  * the token mass (a column sum of W_A) inherits eps_w relatively.
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import aggregate as OA
from paper_2605_28115_b200 import build, civic

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
BOUND_SHARE = 0.5  # regression bar: the largest error as a share of the derived bound


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    civic.load()


def eps_w(tau, d_v):
    d_cos = 2.0 ** -9 + d_v * 2.0 ** -24
    return np.expm1(2 * d_cos / tau) + 2.0 ** -8


def inputs(n_img, t_e, m_e, d_v, seed, scale=1.5, offset=0.7):
    g = torch.Generator().manual_seed(seed)
    x = (torch.randn((n_img, t_e, d_v), generator=g) * scale + offset).to(torch.bfloat16)
    a = torch.randn((m_e, d_v), generator=g)
    return x, a


def check(x, a, tau):
    n_img, t_e, d_v = x.shape
    m_e = a.shape[0]
    pad = 256
    zbuf = torch.full((n_img * m_e * d_v + 2 * pad,), 7.0, dtype=torch.bfloat16, device=DEV)
    mbuf = torch.full((n_img * t_e + 2 * pad,), -3.0, dtype=torch.float32, device=DEV)
    z = zbuf[pad:pad + n_img * m_e * d_v].view(n_img, m_e, d_v)
    mass = mbuf[pad:pad + n_img * t_e].view(n_img, t_e)
    need = civic.anchor_aggregate_workspace_bytes(n_img, t_e, m_e, d_v)
    ws = torch.full((need + 512,), 0xA5, dtype=torch.uint8, device=DEV)
    _, _, status = civic.civic_anchor_aggregate(x.to(DEV), a.to(DEV), tau, z0=z, token_mass=mass, workspace=ws[:need])
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "a wait inside the kernels ran into its time limit"
    assert bool((zbuf[:pad] == 7.0).all()) and bool((zbuf[pad + z.numel():] == 7.0).all()), "wrote outside z0"
    assert bool((mbuf[:pad] == -3.0).all()) and bool((mbuf[pad + mass.numel():] == -3.0).all())
    assert bool((ws[need:] == 0xA5).all()), "wrote past the advertised workspace size"

    x64, a64 = x.double().numpy(), a.double().numpy()
    z_o, mass_o = OA.anchor_aggregate_batch(x64, a64, tau)
    e = eps_w(tau, d_v)
    z_g = z.float().cpu().numpy().astype(np.float64)
    worst = 0.0
    for i in range(n_img):
        w = OA.aggregation_weights(x64[i], a64, tau)
        bound = e * (w @ np.abs(x64[i])) + 2.0 ** -9 * np.abs(z_o[i])
        share = np.abs(z_g[i] - z_o[i]) / np.maximum(bound, 1e-300)
        assert np.all(share <= 1.0), (i, float(share.max()))
        worst = max(worst, float(share.max()))
    mass_share = np.abs(mass.cpu().numpy() - mass_o) / (e * mass_o + 1e-30)
    assert np.all(mass_share <= 1.0)
    worst = max(worst, float(mass_share.max()))
    # the bound is a worst case; an accuracy regression that stays inside it is still seen here
    assert worst <= BOUND_SHARE, f"largest error is {worst:.2f} of the bound (bar {BOUND_SHARE})"
    return z, mass


@pytest.mark.parametrize("n_img,t_e,m_e,d_v,tau", [
    (1, 200, 130, 128, 0.1),     # two anchor tiles, two token tiles, ragged on both
    (2, 197, 65, 64, 0.05),      # t_e not a multiple of 8: padded leading dimension of W_A
    (3, 333, 257, 192, 0.07),    # 192-wide feature tile
    (2, 1000, 300, 320, 0.2),    # feature tile of 256 running past d_v
    (2, 1024, 512, 1024, 0.1),
    (1, 50, 1, 64, 1.0),         # a single anchor
    (1, 1, 5, 128, 0.5),         # a single dense token: every anchor returns it
    (2, 3136, 341, 1280, 0.025), # the smallest supported temperature
])
def test_against_oracle(n_img, t_e, m_e, d_v, tau):
    x, a = inputs(n_img, t_e, m_e, d_v, seed=t_e + m_e)
    check(x, a, tau)


def test_benchmark_shape_one_image():
    """4096 patches of 1152 features (a 896x896 image), 1024 anchors."""
    x, a = inputs(1, 4096, 1024, 1152, seed=5)
    check(x, a, 0.07)


def test_many_tiles_ragged_everywhere():
    """More pair tiles than resident pairs in the anchor direction, ragged token and anchor edges."""
    x, a = inputs(2, 9001, 1500, 320, seed=13)
    check(x, a, 0.05)


def test_structure_and_degenerate_tokens():
    x, a = inputs(2, 300, 40, 128, seed=9)
    x[0, 17] = 2.5        # a token with all features equal has no direction: logit 0, as in the oracle
    x[1, :, :] = x[1, 0]  # an image of identical tokens: every anchor returns that token
    z, mass = check(x, a, 0.1)
    assert torch.allclose(z[1].float().cpu(), x[1, :40].float(), atol=0, rtol=2.0 ** -7)
    assert abs(float(mass.sum()) - 2 * 40) < 1e-2 * 80  # every anchor hands out one unit per image
    # deterministic: same bits on a second run
    z2, mass2, _ = civic.civic_anchor_aggregate(x.to(DEV), a.to(DEV), 0.1)
    assert torch.equal(z2, z) and torch.equal(mass2, mass)


def test_token_mass_feeds_the_selection():
    """Aggregate -> token mass -> civic_select: the scores produced on the GPU select the same
    tokens as the oracle's selection on the same score bits."""
    import oracle

    x, a = inputs(2, 32 * 32, 64, 128, seed=11)
    _, mass, status = civic.civic_anchor_aggregate(x.to(DEV), a.to(DEV), 0.1)
    desc = civic.SelectDesc(1, 32, 32, 4, 4, 1, 341)
    keep = civic.civic_select(mass, desc)
    assert int(status.item()) == 0
    want = oracle.default.select(mass.cpu().numpy(), 1, 32, 32, 4, 4, 1, 341)
    assert np.array_equal(keep.cpu().numpy(), want)


def test_a_wait_that_never_gets_its_signal_ends_with_a_status():
    """The kernels' bounded wait, run on a barrier nobody signals (no copy, no tensor-core work in
    flight): it comes back within a millisecond with the time-out code in the device word, the
    block's second waiter leaves through the stop flag, and the next ordinary call on the same
    stream is still right."""
    rec = torch.full((2,), -1, dtype=torch.int32, device=DEV)
    civic.civic_selftest_bounded_wait(1 << 16, rec)  # first call: module load, not timed
    torch.cuda.synchronize()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    rec.fill_(-1)
    start.record()
    civic.civic_selftest_bounded_wait(1 << 16, rec)
    end.record()
    x, a = inputs(1, 200, 130, 128, seed=330)
    check(x, a, 0.1)  # enqueued behind the self-test on the same stream
    assert rec.cpu().tolist() == [1, 1]  # kAggTimeoutFull; the flag released the second waiter
    assert start.elapsed_time(end) < 1.0, "the wait did not stop at its limit (2^16 cycles = 33 us)"
    lib = civic.load()
    assert lib.civic_selftest_bounded_wait(0, rec.data_ptr(), None) == 1
    assert lib.civic_selftest_bounded_wait(1 << 25, rec.data_ptr(), None) == 1
    assert lib.civic_selftest_bounded_wait(100, None, None) == 1


def test_prepared_anchors_give_the_same_bits():
    """Q_A prepared once (civic_anchor_prepare) and reused: bit-identical to the plain call."""
    x, a = inputs(2, 333, 257, 192, seed=77)
    z, mass = check(x, a, 0.07)
    prepared = civic.civic_anchor_prepare(a.to(DEV))
    for _ in range(2):
        z2, mass2, status = civic.civic_anchor_aggregate(x.to(DEV), prepared, 0.07)
        assert int(status.item()) == 0
        assert torch.equal(z2, z) and torch.equal(mass2, mass)
