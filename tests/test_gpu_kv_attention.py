"""KV-compressed visual attention (Eq. 9) on the tensor cores against the fp64 oracle (needs a B200).

Tolerance, from the arithmetic of the CUDA path (bf16 inputs, the same for both sides):
  * K_c and V_c are weighted averages taken with bf16-rounded weights (relative 2^-9), accumulated in
    fp32 and rounded to bf16 (2^-9): each is off by at most 2^-8 of the same average of absolute values;
  * a logit q . k_c / sqrt(d) is therefore off by at most lam = 2^-8 * max (|q| . |K_c|) / sqrt(d), a
    softmax weight by the factor exp(2 lam); the weights are cut (not rounded) to bf16, each losing a
    fraction in [0, 2^-8], and normalised by the sum of the cut weights, which loses a fraction in the
    same range: a normalised weight moves by at most the factor 1 / (1 - 2^-8):
        eps_w = exp(2 lam) - 1 + 2^-8 (1 + 2^-7);
  * out = W V_c inherits eps_w from the weights and 2^-8 from V_c, relative to W |V_c|, plus 2^-9 |out|
    for the bf16 result:   |out_gpu - out_oracle| <= (eps_w + 2^-8) (W |V_c|) + 2^-9 |out|.
"""
import numpy as np
import pytest
import torch

from oracle import aggregate as OA
from paper_2605_28115_b200 import build, civic

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
BOUND_SHARE = 0.5


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    civic.load()


def inputs(n_img, m_e, heads, d, s, seed):
    g = torch.Generator().manual_seed(seed)
    dim = heads * d
    q, k, v = ((torch.randn((n_img, m_e, dim), generator=g) * 1.2).to(torch.bfloat16) for _ in range(3))
    # a soft assignment: every token spreads over the anchors with a few dominant ones
    r = torch.softmax(torch.randn((m_e, s), generator=g) * 3.0, dim=1)
    return q, k, v, r


def check(q, k, v, r, heads):
    n_img, m_e, dim = q.shape
    d, s = dim // heads, r.shape[1]
    pad = 256
    buf = torch.full((q.numel() + 2 * pad,), 7.0, dtype=torch.bfloat16, device=DEV)
    out = buf[pad:pad + q.numel()].view(q.shape)
    need = civic.kv_compressed_attention_workspace_bytes(n_img, m_e, heads, d, s)
    assert need > 0
    ws = torch.full((need + 512,), 0xA5, dtype=torch.uint8, device=DEV)
    _, status = civic.civic_kv_compressed_attention(q.to(DEV), k.to(DEV), v.to(DEV), r.to(DEV), heads, out=out,
                                                    workspace=ws[:need])
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "a wait inside the kernels ran into its time limit"
    assert bool((buf[:pad] == 7.0).all()) and bool((buf[pad + q.numel():] == 7.0).all()), "wrote outside out"
    assert bool((ws[need:] == 0xA5).all()), "wrote past the advertised workspace size"
    got = out.float().cpu().numpy().astype(np.float64)
    r64 = r.double().numpy()
    rbar = OA.column_normalize(r64)
    worst = 0.0
    for i in range(n_img):
        q64, k64, v64 = (a[i].double().numpy() for a in (q, k, v))
        want, k_c, v_c = OA.kv_compressed_attention(q64, k64, v64, r64, heads)
        abs_kc, abs_vc = rbar.T @ np.abs(k64), rbar.T @ np.abs(v64)
        for h in range(heads):
            c = slice(h * d, (h + 1) * d)
            lam = 2.0 ** -8 * np.max(np.abs(q64[:, c]) @ abs_kc[:, c].T) / np.sqrt(d)
            eps_w = np.expm1(2 * lam) + 2.0 ** -8 * (1 + 2.0 ** -7)
            logits = q64[:, c] @ k_c[:, c].T / np.sqrt(d)
            w = np.exp(logits - logits.max(axis=1, keepdims=True))
            w /= w.sum(axis=1, keepdims=True)
            bound = (eps_w + 2.0 ** -8) * (w @ abs_vc[:, c]) + 2.0 ** -9 * np.abs(want[:, c])
            err = np.abs(got[i][:, c] - want[:, c])
            assert np.all(err <= bound), (i, h, float(np.max(err / bound)))
            worst = max(worst, float(np.max(err / bound)))
    # The bound is a worst case; measured, the kernels use about a fifth of it.  Half of it is the
    # regression bar: a change that loses accuracy inside the bound is still seen.
    assert worst <= BOUND_SHARE, f"largest error is {worst:.2f} of the bound (bar {BOUND_SHARE})"
    return out, worst


@pytest.mark.parametrize("n_img,m_e,heads,d,s", [
    (2, 300, 2, 64, 128),    # three query tiles, the last ragged
    (1, 130, 3, 64, 64),     # one block of memory anchors, 192 features (192-wide compression tile)
    (2, 256, 2, 128, 128),   # head dimension 128: two 64-column blocks per operand
    (1, 100, 1, 64, 192),    # three blocks of anchors
    (1, 200, 1, 128, 256),   # the largest shared-memory footprint
    (1, 1024, 16, 64, 256),  # Qwen3-VL-2B-shaped vision layer: 1024 compact tokens, 16 heads of 64, 256 anchors
    (10, 700, 16, 64, 64),   # more (head, image) pairs than SMs: blocks walk three query tiles, the last ragged
    (5, 1100, 32, 64, 128),  # nine query tiles in three blocks per pair
    (20, 520, 8, 128, 128),  # five tiles per block with 128-wide heads: both Q slots reused twice
    (3, 300, 50, 128, 256),  # the largest shared-memory footprint (one block per SM), three tiles per block
    (2, 150, 80, 64, 192),   # 192 anchors (P and O share 256 TMEM columns with S), two tiles per block
    (1, 5, 2, 64, 64),       # fewer queries than one warp's 32 rows: one partly filled store box, three skipped
    (2, 33, 3, 128, 128),    # one row into the second warp's box
    (1, 129, 1, 64, 256),    # one row into the second query tile
    (2, 300, 16, 72, 256),   # 72-wide heads (1152-wide towers with 16 heads): stored 80 wide, O written 64 + 8 columns
    (1, 200, 3, 72, 64),     # the same with one block of anchors; the last head's second box runs past the tensor
    (2, 300, 16, 64, 512),   # Table 2's 512 anchors: S fills all of tensor memory, the first chain is two MMAs wide
    (1, 260, 8, 128, 512),   # 512 anchors, 128-wide heads: K_c resident, V_c streamed per query tile, one Q slot
    (1, 140, 4, 128, 320),   # five blocks of anchors, streamed
    (1, 150, 5, 64, 448),    # seven blocks of anchors, resident
    (1, 100, 3, 40, 128),    # a head narrower than one box: K = 48, the output a single plain box of 40 columns
    (1, 100, 3, 96, 128),    # 64 + 32 columns
    (2, 130, 2, 112, 192),   # 64 + 48 columns
    (1, 70, 5, 8, 64),       # the narrowest head
    (1, 90, 2, 120, 256),    # 128-wide storage of a 120-wide head
    (2, 1300, 8, 128, 512),  # streamed V_c with more tiles than SMs: blocks walk two tiles, some across two heads
    (1, 700, 30, 128, 320),  # the same with five blocks of anchors and one K_c slot reloaded per head
    (40, 128, 4, 64, 256),   # one query tile per (head, image): every tile of a block starts a new pair
])
def test_against_oracle(n_img, m_e, heads, d, s):
    q, k, v, r = inputs(n_img, m_e, heads, d, s, seed=m_e + s)
    check(q, k, v, r, heads)


def test_identity_assignment_is_dense_attention_and_deterministic():
    """S = M_e = 128 and R = identity: nothing is compressed (the oracle's pin, here on the GPU)."""
    q, k, v, _ = inputs(1, 128, 2, 64, 128, seed=3)
    out, _ = check(q, k, v, torch.eye(128), 2)
    want = torch.nn.functional.scaled_dot_product_attention(
        q.float().view(1, 128, 2, 64).transpose(1, 2), k.float().view(1, 128, 2, 64).transpose(1, 2),
        v.float().view(1, 128, 2, 64).transpose(1, 2)).transpose(1, 2).reshape(1, 128, 128)
    assert torch.allclose(out.float().cpu(), want, atol=0.03, rtol=0.03)
    out2, _ = civic.civic_kv_compressed_attention(q.to(DEV), k.to(DEV), v.to(DEV), torch.eye(128, device=DEV), 2)
    assert torch.equal(out2, out)


@pytest.mark.parametrize("n_img,m_e,heads,d,s", [(2, 300, 4, 64, 128), (1, 200, 16, 72, 256), (1, 260, 2, 128, 512)])
def test_prepared_assignment_gives_the_same_bits(n_img, m_e, heads, d, s):
    """R converted once (civic_kv_attention_prepare) and reused: bit-identical to the plain call, twice."""
    q, k, v, r = inputs(n_img, m_e, heads, d, s, seed=m_e + s + 1)
    plain, _ = check(q, k, v, r, heads)
    prepared = civic.civic_kv_attention_prepare(r.to(DEV))
    for _ in range(2):
        status = torch.full((1,), 77, dtype=torch.int32, device=DEV)  # the call itself clears it
        got, status = civic.civic_kv_compressed_attention(q.to(DEV), k.to(DEV), v.to(DEV), prepared, heads,
                                                          device_status=status)
        assert int(status.item()) == 0
        assert torch.equal(got, plain)
