"""The calls chained on one stream without any synchronisation in between, as a serving stack would
issue them: Eq. 8 aggregation -> token mass as scores -> selection with sequence indices -> Eq. 13
merge, plane-major position ids and the K/V cache of the kept positions (needs a B200)."""
import numpy as np
import pytest
import torch

import oracle
from oracle import aggregate as OA
from paper_2605_28115_b200 import build, civic

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
O = oracle.default


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    civic.load()


def test_aggregate_select_compact_chain():
    g = torch.Generator().manual_seed(77)
    n_img, grid, d_v, m_e = 3, 24, 128, 96
    n = grid * grid  # one dense token per grid cell
    k, text_before, text_after, layers, row = 200, 5, 9, 3, 64
    seq_len = text_before + n + text_after
    x0 = (torch.randn((n_img, n, d_v), generator=g) + 0.3).to(torch.bfloat16).to(DEV)
    anchors = torch.randn((m_e, d_v), generator=g).to(DEV)
    text = torch.randn((n_img, seq_len, d_v), generator=g).to(torch.bfloat16).to(DEV)
    pos = torch.randint(0, 1000, (3, n_img, seq_len), generator=g, dtype=torch.int32).to(DEV)
    ks = [torch.randn((n_img, seq_len, row), generator=g).to(torch.bfloat16).to(DEV) for _ in range(layers)]
    vs = [torch.randn((n_img, seq_len, row), generator=g).to(torch.bfloat16).to(DEV) for _ in range(layers)]
    kd = [torch.empty((n_img, seq_len - n + k, row), dtype=torch.bfloat16, device=DEV) for _ in range(layers)]
    vd = [torch.empty((n_img, seq_len - n + k, row), dtype=torch.bfloat16, device=DEV) for _ in range(layers)]
    desc = civic.SelectDesc(1, grid, grid, 4, 4, 1, k)

    # ---- the chain: nothing here waits for the GPU
    z0, mass, status = civic.civic_anchor_aggregate(x0, anchors, 0.1)
    keep, seq_idx = civic.civic_select_seq(mass, desc, seq_len, text_before)
    merged = civic.civic_merge_embeddings(text, x0, keep, text_before)
    pos_c = civic.civic_compact_pos_planes(pos, seq_idx)
    civic.civic_compact_kv(civic.kv_tables(ks, vs, kd, vd), seq_idx)
    torch.cuda.synchronize()
    assert int(status.item()) == 0

    # ---- every stage against the oracle, fed with the previous stage's GPU result
    mass_h = mass.cpu().numpy()
    _, mass_o = OA.anchor_aggregate_batch(x0.double().cpu().numpy(), anchors.double().cpu().numpy(), 0.1)
    assert np.allclose(mass_h, mass_o, rtol=0.1)
    keep_o = O.select(mass_h, 1, grid, grid, 4, 4, 1, k)
    idx_o = O.seq_indices(keep_o, seq_len, text_before, n)
    assert np.array_equal(keep.cpu().numpy(), keep_o) and np.array_equal(seq_idx.cpu().numpy(), idx_o)
    bits = lambda t: t.contiguous().view(torch.int16).cpu().numpy()
    assert np.array_equal(bits(merged), O.merge_embeddings(bits(text), bits(x0), keep_o, text_before))
    assert np.array_equal(pos_c.cpu().numpy(), O.compact_pos_planes(pos.cpu().numpy(), idx_o))
    want_k, want_v = O.compact_kv([bits(a) for a in ks], [bits(a) for a in vs], idx_o)
    for l in range(layers):
        assert np.array_equal(bits(kd[l]), want_k[l]) and np.array_equal(bits(vd[l]), want_v[l])
    assert merged.shape[1] == text_before + text_after + k  # Eq. 13: L + M_p rows


def test_aggregation_feeds_kv_compressed_attention_on_one_vision_width():
    """Eq. 8 and Eq. 9 on ONE model shape, chained on a stream: a 1152-wide vision tower with 16 heads
    of 72.  Z_0 from the aggregation is projected (plain GEMMs: the caller's BLAS, here torch) to Q, K,
    V of the compact encoder layer, which attends through 256 memory anchors with prepared constants."""
    from tests.test_gpu_aggregate import check as check_aggregate
    from tests.test_gpu_kv_attention import check as check_attention

    g = torch.Generator().manual_seed(1152)
    n_img, t_e, m_e, d_v, heads, s = 2, 1024, 256, 1152, 16, 256
    x0 = (torch.randn((n_img, t_e, d_v), generator=g) * 1.5 + 0.7).to(torch.bfloat16)
    anchors = torch.randn((m_e, d_v), generator=g)
    w_q, w_k, w_v = (torch.randn((d_v, d_v), generator=g).mul_(d_v ** -0.5).to(torch.bfloat16).to(DEV) for _ in range(3))
    r = torch.softmax(torch.randn((m_e, s), generator=g) * 3.0, dim=1)

    prepared_a = civic.civic_anchor_prepare(anchors.to(DEV))
    prepared_r = civic.civic_kv_attention_prepare(r.to(DEV))
    z0, _, st1 = civic.civic_anchor_aggregate(x0.to(DEV), prepared_a, 0.07, want_mass=False)
    q, k, v = (torch.matmul(z0, w) for w in (w_q, w_k, w_v))
    out, st2 = civic.civic_kv_compressed_attention(q, k, v, prepared_r, heads)
    torch.cuda.synchronize()
    assert int(st1.item()) == 0 and int(st2.item()) == 0

    # every stage against the oracle, the second fed with the first stage's GPU result
    z_plain, _ = check_aggregate(x0, anchors, 0.07)
    assert torch.equal(z_plain, z0)
    out_plain, _ = check_attention(q.cpu(), k.cpu(), v.cpu(), r, heads)
    assert torch.equal(out_plain, out)
