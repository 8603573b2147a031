"""Pins for the CPU oracle: facts fixed by the paper, the benchmark definition and plain
mathematics, each checked WITHOUT re-using the oracle's own formulation.

Every function takes the oracle object under test and raises AssertionError on a
mismatch, so the same pins run against the real oracle (must pass) and against copies
with a planted mistake (at least one pin must fail).
"""

from __future__ import annotations

import itertools
import math

import numpy as np

from paper_2605_28115_b200 import workloads as W


# ---------------------------------------------------------------- helpers (test side)

def region_ids(t, h, w, rh, rw):
    """Region id of every token, row-major (t, h, w); regions never span t."""
    tt, hh, ww = np.meshgrid(np.arange(t), np.arange(h), np.arange(w), indexing="ij")
    n_rh, n_rw = math.ceil(h / rh), math.ceil(w / rw)
    return ((tt * n_rh + hh // rh) * n_rw + ww // rw).reshape(-1)


def rank_of(scores):
    """rank[i] = position of token i when tokens are listed best first
    (higher score first, equal scores: lower index first).  Finite scores only."""
    order = sorted(range(len(scores)), key=lambda i: (-float(scores[i]), i))
    rank = np.empty(len(scores), dtype=np.int64)
    rank[order] = np.arange(len(scores))
    return rank


def floor_need(reg, m):
    sizes = np.bincount(reg)
    return np.minimum(sizes, m)


# ---------------------------------------------------------------- total order on fp32

def _f(bits):
    return np.array([bits], dtype=np.uint32).view(np.float32)[0]


# ascending under IEEE-754 totalOrder, written out by hand
TOTAL_ORDER_LADDER = [
    0xFFFFFFFF,  # -qNaN, largest payload
    0xFFC00000,  # -qNaN
    0xFF800001,  # -sNaN, smallest payload
    0xFF800000,  # -inf
    0xFF7FFFFF,  # -FLT_MAX
    0xBF800000,  # -1
    0x80800000,  # -FLT_MIN (normal)
    0x807FFFFF,  # largest-magnitude negative subnormal
    0x80000001,  # smallest-magnitude negative subnormal
    0x80000000,  # -0
    0x00000000,  # +0
    0x00000001,  # smallest subnormal
    0x007FFFFF,  # largest subnormal
    0x00800000,  # FLT_MIN
    0x3F800000,  # 1
    0x3F800001,  # nextafter(1)
    0x7F7FFFFF,  # FLT_MAX
    0x7F800000,  # +inf
    0x7F800001,  # +sNaN, smallest payload
    0x7FC00000,  # +qNaN
    0x7FFFFFFF,  # +qNaN, largest payload
]


def pin_total_order(o):
    lad = TOTAL_ORDER_LADDER
    for i, a in enumerate(lad):
        for j, b in enumerate(lad):
            want = (i > j) - (i < j)
            got = o.score_cmp_bits(a, b)
            assert got == want, f"cmp({a:#010x},{b:#010x}) = {got}, want {want}"
    # finite values: must agree with ordinary comparison
    rng = np.random.default_rng(7)
    vals = rng.standard_normal(200).astype(np.float32)
    for a, b in zip(vals[:-1], vals[1:]):
        assert o.score_cmp(float(a), float(b)) == int(a > b) - int(a < b)


def pin_special_values_in_select(o):
    """-0 < +0, infinities, subnormals and NaNs take part in the selection in totalOrder."""
    bits = np.array([0x80000000, 0x00000000, 0x7F800000, 0xFF800000, 0x00000001, 0x80000001,
                     0x7FC00000, 0xFFC00000, 0x3F800000, 0x3F800000], dtype=np.uint32)
    s = bits.view(np.float32)[None]
    # best first: +NaN(6) +inf(2) 1.0(8) 1.0(9) sub(4) +0(1) -0(0) -sub(5) -inf(3) -NaN(7)
    best_first = [6, 2, 8, 9, 4, 1, 0, 5, 3, 7]
    for k in range(0, 11):
        got = o.select(s, 1, 1, 10, 1, 10, 0, k)[0]
        assert list(got) == sorted(best_first[:k]), (k, got)


# ---------------------------------------------------------------- selection pins

def pin_plain_topk_is_stable_argsort(o):
    """floor m = 0 reduces to the library routine: first K of a stable descending argsort."""
    for wl in (W.C1, W.C2, W.C5_THIRD):
        s = W.scores(wl)
        got = o.select(s, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, 0, wl.k)
        for b in range(wl.n_seg):
            want = np.sort(np.argsort(-s[b].astype(np.float64), kind="stable")[: wl.k])
            assert np.array_equal(got[b], want), (wl.name, b)
    # K = 0 and K = n
    s = W.scores(W.C1)
    assert o.select(s, 1, 14, 14, 2, 2, 0, 0).shape == (1, 0)
    assert np.array_equal(o.select(s, 1, 14, 14, 2, 2, 0, 196)[0], np.arange(196))
    assert np.array_equal(o.select(s, 1, 14, 14, 2, 2, 1, 196)[0], np.arange(196))


def best_feasible_subset(scores, reg, m, k):
    """Brute force over all K-subsets: among those meeting the floor in every region,
    the one whose best-first rank vector is lexicographically smallest."""
    n = len(scores)
    rank = rank_of(scores)
    need = floor_need(reg, m)
    best, best_key = None, None
    for sub in itertools.combinations(range(n), k):
        cnt = np.bincount(reg[list(sub)], minlength=len(need))
        if np.any(cnt < need):
            continue
        key = sorted(rank[list(sub)])
        if best_key is None or key < best_key:
            best, best_key = sub, key
    return best


def pin_bruteforce_tiny(o, trials=60):
    """On tiny grids the oracle's set is the optimum found by exhaustive search."""
    rng = np.random.default_rng(11)
    shapes = [(1, 3, 4, 2, 2), (2, 2, 3, 1, 2), (1, 3, 3, 2, 2), (1, 2, 5, 2, 3), (3, 2, 2, 2, 2),
              (1, 4, 3, 3, 2)]
    for trial in range(trials):
        t, h, w, rh, rw = shapes[trial % len(shapes)]
        n = t * h * w
        reg = region_ids(t, h, w, rh, rw)
        m = int(rng.integers(0, 3))
        n_res = int(floor_need(reg, m).sum())
        k = int(rng.integers(n_res, n + 1))
        if trial % 2:
            s = rng.integers(0, 3, n).astype(np.float32)  # heavy ties
        else:
            s = rng.random(n).astype(np.float32)
        got = o.select(s[None], t, h, w, rh, rw, m, k)[0]
        want = best_feasible_subset(s, reg, m, k)
        assert want is not None
        assert list(got) == list(want), (trial, (t, h, w, rh, rw, m, k), s, got, want)


def pin_full_sort_tiny(o):
    """m = 0 on tiny grids: all tie patterns of up to 6 tokens against a full sort."""
    for n in range(1, 7):
        for pattern in itertools.product(range(3), repeat=n):
            s = np.array(pattern, dtype=np.float32)
            order = sorted(range(n), key=lambda i: (-pattern[i], i))
            for k in (0, 1, n // 2, n):
                got = o.select(s[None], 1, 1, n, 1, 1, 0, k)[0]
                assert list(got) == sorted(order[:k]), (pattern, k)


def check_invariants(scores, t, h, w, rh, rw, m, k, keep):
    """Size-independent properties of a correct selection (finite scores)."""
    n = t * h * w
    keep = np.asarray(keep)
    assert keep.shape == (k,), "output length must be exactly K"
    assert np.all(keep[1:] > keep[:-1]), "indices must be strictly ascending (source order)"
    if k:
        assert keep[0] >= 0 and keep[-1] < n
    reg = region_ids(t, h, w, rh, rw)
    need = floor_need(reg, m)
    mask = np.zeros(n, dtype=bool)
    mask[keep] = True
    cnt = np.bincount(reg[mask], minlength=len(need))
    assert np.all(cnt >= need), "retention floor violated in some region"
    # exchange optimality: no dropped token d may beat a kept token x when swapping them
    # keeps the floor satisfied (same region, or x's region has a spare token)
    rank = rank_of(scores)
    dropped = np.nonzero(~mask)[0]
    if len(dropped) == 0 or k == 0:
        return
    spare = cnt[reg[keep]] - 1 >= need[reg[keep]]
    d_rank = rank[dropped][:, None]
    x_rank = rank[keep][None, :]
    same = reg[dropped][:, None] == reg[keep][None, :]
    bad = (d_rank < x_rank) & (same | spare[None, :])
    assert not bad.any(), "a dropped token beats a kept token it could replace"


def pin_invariants_on_workloads(o):
    for wl in W.ALL:
        s = W.scores(wl)
        got = o.select(s, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, wl.k)
        for b in range(wl.n_seg):
            check_invariants(s[b], wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, wl.k, got[b])


def pin_invariants_random(o, trials=150):
    rng = np.random.default_rng(5)
    for trial in range(trials):
        t = int(rng.integers(1, 4))
        h = int(rng.integers(1, 13))
        w = int(rng.integers(1, 13))
        rh = int(rng.integers(1, h + 1))
        rw = int(rng.integers(1, w + 1))
        m = int(rng.integers(0, 4))
        n = t * h * w
        n_res = int(floor_need(region_ids(t, h, w, rh, rw), m).sum())
        k = int(rng.integers(n_res, n + 1))
        kind = trial % 3
        if kind == 0:
            s = rng.random(n)
        elif kind == 1:
            s = rng.integers(0, 4, n)
        else:
            s = -np.abs(rng.standard_normal(n))  # negative scores
        s = s.astype(np.float32)
        got = o.select(s[None], t, h, w, rh, rw, m, k)[0]
        check_invariants(s, t, h, w, rh, rw, m, k, got)


def pin_floor_inactive(o):
    """If plain top-K already meets the floor in every region, the floor changes nothing."""
    rng = np.random.default_rng(3)
    hits = 0
    for trial in range(200):
        h, w, rh, rw = 6, 6, 3, 3
        s = rng.random(36).astype(np.float32)
        k = int(rng.integers(8, 30))
        plain = np.sort(np.argsort(-s.astype(np.float64), kind="stable")[:k])
        reg = region_ids(1, h, w, rh, rw)
        if np.all(np.bincount(reg[plain], minlength=4) >= 1):
            hits += 1
            got = o.select(s[None], 1, h, w, rh, rw, 1, k)[0]
            assert np.array_equal(got, plain), trial
    assert hits > 20


def repair_select(scores, reg, k):
    """A second formulation for floor m = 1: take plain top-K, then while some region is
    empty add its best token and evict the worst kept token whose removal empties no region."""
    n = len(scores)
    order = sorted(range(n), key=lambda i: (-float(scores[i]), i))
    rank = {tok: r for r, tok in enumerate(order)}
    kept = set(order[:k])
    n_reg = int(reg.max()) + 1
    while True:
        cnt = np.bincount(reg[sorted(kept)], minlength=n_reg) if kept else np.zeros(n_reg, int)
        empty = [r for r in range(n_reg) if cnt[r] == 0]
        if not empty:
            break
        r = empty[0]
        best = min((i for i in range(n) if reg[i] == r), key=lambda i: rank[i])
        kept.add(best)
        cnt[r] += 1
        evictable = [x for x in kept if cnt[reg[x]] >= 2]
        kept.remove(max(evictable, key=lambda i: rank[i]))
    return sorted(kept)


def pin_repair_formulation(o, trials=300):
    rng = np.random.default_rng(19)
    for trial in range(trials):
        h = int(rng.integers(2, 9))
        w = int(rng.integers(2, 9))
        rh = int(rng.integers(1, 4))
        rw = int(rng.integers(1, 4))
        reg = region_ids(1, h, w, rh, rw)
        n_reg = int(reg.max()) + 1
        n = h * w
        k = int(rng.integers(n_reg, n + 1))
        s = (rng.random(n) if trial % 2 else rng.integers(0, 5, n)).astype(np.float32)
        got = o.select(s[None], 1, h, w, rh, rw, 1, k)[0]
        assert list(got) == repair_select(s, reg, k), trial


def pin_hand_worked_example(o):
    """A 2x4 grid small enough to do by hand.  Regions are 2x2 (left: tokens 0,1,4,5; right:
    2,3,6,7).  Scores: left block 9,8,7,6 / right block 1,2,2,0.
         idx: 0 1 2 3
              4 5 6 7
    m=1, K=3: reserve 0 (left best) and 3?  right block scores: t2=1, t3=2, t6=2, t7=0 ->
    best is 3 (2.0, lower index than 6).  Fill 1 more from the rest: token 1 (8.0).
    -> {0,1,3}.  Plain top-3 would be {0,1,4}."""
    s = np.array([[9, 8, 1, 2, 7, 6, 2, 0]], dtype=np.float32)
    assert list(o.select(s, 1, 2, 4, 2, 2, 1, 3)[0]) == [0, 1, 3]
    assert list(o.select(s, 1, 2, 4, 2, 2, 0, 3)[0]) == [0, 1, 4]
    # m=2, K=5: reserve {0,1} and {3,6}; fill one: 4 (7.0) -> {0,1,3,4,6}
    assert list(o.select(s, 1, 2, 4, 2, 2, 2, 5)[0]) == [0, 1, 3, 4, 6]
    # two temporal slices of 1x4, regions 1x2, m=1, K=4: every region keeps exactly its best
    s2 = np.array([[1, 5, 5, 2, 0, 0, 3, 4]], dtype=np.float32)
    assert list(o.select(s2, 2, 1, 4, 1, 2, 1, 4)[0]) == [1, 2, 4, 7]
    # the same scores as ONE 2x4 slice with 2x2 regions differ: left {0,1,4,5}->1, right->2
    assert list(o.select(s2, 1, 2, 4, 2, 2, 1, 2)[0]) == [1, 2]


def pin_error_codes(o):
    import oracle as O

    s = np.zeros((1, 16), dtype=np.float32)
    for args, code in [((1, 4, 4, 2, 2, 1, 17), O.ERR_K_RANGE), ((1, 4, 4, 2, 2, 1, -1), O.ERR_K_RANGE),
                       ((1, 4, 4, 2, 2, 1, 3), O.ERR_FLOOR_EXCEEDS_K),
                       ((1, 4, 4, 2, 2, 5, 15), O.ERR_FLOOR_EXCEEDS_K),
                       ((1, 4, 4, 0, 2, 1, 4), O.ERR_ARG)]:
        try:
            o.select(s, *args)
        except O.OracleError as e:
            assert e.code == code, (args, e.code)
        else:
            raise AssertionError(f"no error for {args}")
    assert o.reserved_count(1, 5, 5, 2, 2, 3) == 4 * 3 + 2 * 2 + 2 * 2 + 1


# ---------------------------------------------------------------- compaction pins

def pin_compact_is_take(o):
    """Row gather equals numpy's own indexing, byte for byte; positions are copied, not renumbered."""
    rng = np.random.default_rng(23)
    n_seg, n, k, row = 3, 37, 11, 24
    hidden = rng.integers(0, 2 ** 16, (n_seg, n, row), dtype=np.uint16)
    pos = rng.integers(-5, 1000, (n_seg, n, 3)).astype(np.int32)
    keep = np.stack([np.sort(rng.choice(n, k, replace=False)) for _ in range(n_seg)]).astype(np.int32)
    h_out, p_out = o.compact(hidden, pos, keep)
    for b in range(n_seg):
        assert h_out[b].tobytes() == hidden[b][keep[b]].tobytes()
        assert np.array_equal(p_out[b], pos[b][keep[b]])
    h_only, none = o.compact(hidden, None, keep)
    assert none is None and h_only.tobytes() == h_out.tobytes()
    none, p_only = o.compact(None, pos, keep)
    assert none is None and np.array_equal(p_only, p_out)


def pin_seq_indices(o):
    """Text positions always survive; the result is the sorted union (library routine)."""
    rng = np.random.default_rng(29)
    for seq_len, vis_start, n_vis, k in [(20, 3, 12, 5), (12, 0, 12, 4), (15, 5, 10, 10), (9, 9, 0, 0),
                                         (30, 0, 7, 0), (1088, 16, 1024, 341)]:
        keep = np.stack([np.sort(rng.choice(n_vis, k, replace=False)) for _ in range(3)]).astype(np.int32) \
            if n_vis else np.zeros((3, 0), np.int32)
        got = o.seq_indices(keep, seq_len, vis_start, n_vis)
        text = np.concatenate([np.arange(vis_start), np.arange(vis_start + n_vis, seq_len)])
        for b in range(3):
            want = np.union1d(text, keep[b] + vis_start)
            assert np.array_equal(got[b], want)
            assert len(got[b]) == seq_len - n_vis + k


def pin_compact_kv_is_take(o):
    rng = np.random.default_rng(31)
    n_layers, n_seq, seq_len, s_out, row = 3, 2, 29, 13, 16
    ks = [rng.integers(0, 2 ** 16, (n_seq, seq_len, row), dtype=np.uint16) for _ in range(n_layers)]
    vs = [rng.integers(0, 2 ** 16, (n_seq, seq_len, row), dtype=np.uint16) for _ in range(n_layers)]
    idx = np.stack([np.sort(rng.choice(seq_len, s_out, replace=False)) for _ in range(n_seq)]).astype(np.int32)
    kd, vd = o.compact_kv(ks, vs, idx)
    for l in range(n_layers):
        for b in range(n_seq):
            assert kd[l][b].tobytes() == ks[l][b][idx[b]].tobytes()
            assert vd[l][b].tobytes() == vs[l][b][idx[b]].tobytes()


def read_golden(path):
    out = {}
    with open(path) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                key, val = line.split()
                out[key] = float(val)
    return out


def pin_cache_ratio(o, golden_path):
    """Eq. 14: compact cache / dense cache = (L + M_p) / (L + T_p), exactly, and Table 1's
    printed cache sizes follow that proportionality to the printed precision."""
    g = read_golden(golden_path)
    tok = g["civic_prefill_tokens"] / g["dense_prefill_tokens"]
    mb = g["civic_kv_cache_mb"] / g["dense_kv_cache_mb"]
    assert abs(tok - mb) < 5e-4
    assert abs(g["visiontrim_prefill_tokens"] / g["dense_prefill_tokens"]
               - g["visiontrim_kv_cache_mb"] / g["dense_kv_cache_mb"]) < 5e-4
    wl = W.C3.replace(n_seg=2, n_layers=2)
    L, T_p, M_p = wl.text_before + wl.text_after, wl.n, wl.k
    s = W.scores(wl)
    keep = o.select(s, wl.t, wl.h, wl.w, wl.region_h, wl.region_w, wl.floor_m, wl.k)
    idx = o.seq_indices(keep, wl.seq_len, wl.text_before, wl.n)
    rng = np.random.default_rng(1)
    ks = [rng.integers(0, 2 ** 16, (wl.n_seg, wl.seq_len, 8), dtype=np.uint16) for _ in range(2)]
    kd, vd = o.compact_kv(ks, ks, idx)
    dense = sum(a.nbytes for a in ks)
    compact = sum(a.nbytes for a in kd)
    assert compact * (L + T_p) == dense * (L + M_p)
    assert (L + M_p, L + T_p) == (405, 1088)


# ---------------------------------------------------------------- adjacent steps

def _sorted_choice(rng, n, k, rows):
    return np.stack([np.sort(rng.choice(n, k, replace=False)) for _ in range(rows)]).astype(np.int32) \
        if k else np.zeros((rows, 0), np.int32)


def pin_merge_embeddings(o):
    """Eq. 13: text rows with the visual span replaced by the kept visual rows -- numpy's own
    concatenate; the length is L + M_p; keeping everything is the dense merge (Eq. 1); and the
    compact merge is the dense merge with the dropped rows taken out (sequence indices)."""
    rng = np.random.default_rng(37)
    for n_seq, seq_len, vis_start, n_vis, k, row in [(2, 20, 3, 12, 5, 8), (3, 12, 0, 12, 4, 6),
                                                     (1, 15, 5, 10, 10, 4), (2, 9, 9, 0, 0, 2),
                                                     (2, 30, 23, 7, 0, 10), (2, 40, 4, 30, 11, 34)]:
        text = rng.integers(0, 2 ** 16, (n_seq, seq_len, row), dtype=np.uint16)
        visual = rng.integers(0, 2 ** 16, (n_seq, n_vis, row), dtype=np.uint16)
        keep = _sorted_choice(rng, n_vis, k, n_seq)
        got = o.merge_embeddings(text, visual, keep, vis_start)
        assert got.shape == (n_seq, seq_len - n_vis + k, row)
        dense = text.copy()
        dense[:, vis_start:vis_start + n_vis] = visual
        idx = o.seq_indices(keep, seq_len, vis_start, n_vis)
        for b in range(n_seq):
            want = np.concatenate([text[b, :vis_start], visual[b][keep[b]], text[b, vis_start + n_vis:]])
            assert got[b].tobytes() == want.tobytes()
            assert got[b].tobytes() == dense[b][idx[b]].tobytes()
        everything = np.tile(np.arange(n_vis, dtype=np.int32), (n_seq, 1))
        assert o.merge_embeddings(text, visual, everything, vis_start).tobytes() == dense.tobytes()


def pin_pos_planes(o):
    """Plane-major position ids: numpy's take_along_axis; agrees with the row layout [.., 3]."""
    rng = np.random.default_rng(41)
    for n_planes, n_seq, seq_len, s_out in [(3, 2, 17, 6), (3, 4, 40, 40), (1, 1, 5, 1), (4, 2, 9, 0)]:
        pos = rng.integers(-3, 5000, (n_planes, n_seq, seq_len)).astype(np.int32)
        idx = _sorted_choice(rng, seq_len, s_out, n_seq)
        got = o.compact_pos_planes(pos, idx)
        want = np.take_along_axis(pos, np.broadcast_to(idx[None], (n_planes, n_seq, s_out)), axis=2)
        assert np.array_equal(got, want)
        if n_planes == 3 and s_out:
            _, rows = o.compact(None, np.ascontiguousarray(pos.transpose(1, 2, 0)), idx)
            assert np.array_equal(got, rows.transpose(2, 0, 1))


def pin_kv_heads(o):
    """Head-major K/V: numpy indexing on the token axis, and the transposed token-major result."""
    rng = np.random.default_rng(43)
    n_layers, n_seq, n_heads, seq_len, s_out, d = 2, 3, 4, 23, 9, 6
    ks = [rng.integers(0, 2 ** 16, (n_seq, n_heads, seq_len, d), dtype=np.uint16) for _ in range(n_layers)]
    vs = [rng.integers(0, 2 ** 16, (n_seq, n_heads, seq_len, d), dtype=np.uint16) for _ in range(n_layers)]
    idx = _sorted_choice(rng, seq_len, s_out, n_seq)
    kd, vd = o.compact_kv_heads(ks, vs, idx)
    tok = lambda a: np.ascontiguousarray(a.transpose(0, 2, 1, 3)).reshape(n_seq, a.shape[2], n_heads * d)
    kt, vt = o.compact_kv([tok(a) for a in ks], [tok(a) for a in vs], idx)
    for l in range(n_layers):
        for b in range(n_seq):
            assert kd[l][b].tobytes() == ks[l][b][:, idx[b]].tobytes()
            assert vd[l][b].tobytes() == vs[l][b][:, idx[b]].tobytes()
        assert np.array_equal(tok(kd[l]), kt[l]) and np.array_equal(tok(vd[l]), vt[l])


def pin_kv_paged(o):
    """Paged destination: reading the cache back through the block table gives the kept rows;
    every other slot keeps its old contents; page size 1 with an identity table is the
    contiguous compaction."""
    rng = np.random.default_rng(47)
    for n_seq, seq_len, s_out, row, page in [(3, 29, 13, 8, 4), (2, 16, 16, 4, 16), (2, 21, 7, 6, 1),
                                            (1, 10, 10, 2, 3)]:
        n_layers = 2
        per_seq = -(-s_out // page) + 1  # one spare table entry per sequence, never used
        n_pages = n_seq * per_seq + 3
        table = rng.permutation(n_pages)[: n_seq * per_seq].reshape(n_seq, per_seq).astype(np.int32)
        ks = [rng.integers(0, 2 ** 15, (n_seq, seq_len, row), dtype=np.uint16) for _ in range(n_layers)]
        vs = [rng.integers(0, 2 ** 15, (n_seq, seq_len, row), dtype=np.uint16) for _ in range(n_layers)]
        idx = _sorted_choice(rng, seq_len, s_out, n_seq)
        kc = [np.full((n_pages, page, row), 0xFFFF, dtype=np.uint16) for _ in range(n_layers)]
        vc = [np.full((n_pages, page, row), 0xFFFE, dtype=np.uint16) for _ in range(n_layers)]
        o.compact_kv_paged(ks, vs, idx, table, page, kc, vc)
        for l in range(n_layers):
            written = np.zeros((n_pages, page), dtype=bool)
            for b in range(n_seq):
                for j in range(s_out):
                    pg, slot = table[b, j // page], j % page
                    assert np.array_equal(kc[l][pg, slot], ks[l][b, idx[b, j]])
                    assert np.array_equal(vc[l][pg, slot], vs[l][b, idx[b, j]])
                    written[pg, slot] = True
            assert np.all(kc[l][~written] == 0xFFFF) and np.all(vc[l][~written] == 0xFFFE)
    # page size 1, identity table: the contiguous compaction
    n_seq, seq_len, s_out, row = 2, 19, 8, 4
    ks = [rng.integers(0, 2 ** 15, (n_seq, seq_len, row), dtype=np.uint16)]
    idx = _sorted_choice(rng, seq_len, s_out, n_seq)
    table = np.arange(n_seq * s_out, dtype=np.int32).reshape(n_seq, s_out)
    kc = [np.zeros((n_seq * s_out, 1, row), dtype=np.uint16)]
    vc = [np.zeros((n_seq * s_out, 1, row), dtype=np.uint16)]
    o.compact_kv_paged(ks, ks, idx, table, 1, kc, vc)
    kd, _ = o.compact_kv(ks, ks, idx)
    assert kc[0].tobytes() == kd[0].tobytes() and vc[0].tobytes() == kd[0].tobytes()


def pin_floor_from_ratio(o):
    """Table 2's Min Keep Ratio values on the benchmark's tiles: exact rational ceiling."""
    from fractions import Fraction

    assert [o.floor_from_ratio(4, 4, n, d) for n, d in [(0, 1), (1, 5), (1, 2)]] == [0, 4, 8]
    assert [o.floor_from_ratio(2, 2, n, d) for n, d in [(0, 1), (1, 5), (1, 2)]] == [0, 1, 2]
    for rh in range(1, 7):
        for rw in range(1, 7):
            for den in range(1, 9):
                for num in range(0, den + 1):
                    assert o.floor_from_ratio(rh, rw, num, den) == math.ceil(Fraction(num, den) * rh * rw)
    assert o.floor_from_ratio(4, 4, 1, 1) == 16
    assert o.floor_from_ratio(4, 4, 3, 2) == -1 and o.floor_from_ratio(0, 4, 1, 2) == -1


def pin_select_ragged(o):
    """A ragged batch is the per-segment selection laid end to end: invariants hold segment by
    segment, offsets follow numpy's cumulative sums, and tiny segments match the brute force."""
    rng = np.random.default_rng(53)
    for trial in range(12):
        descs, parts = [], []
        for _ in range(int(rng.integers(1, 6))):
            t, h, w = int(rng.integers(1, 3)), int(rng.integers(1, 7)), int(rng.integers(1, 7))
            rh, rw = int(rng.integers(1, h + 1)), int(rng.integers(1, w + 1))
            m = int(rng.integers(0, 3))
            n = t * h * w
            n_res = int(floor_need(region_ids(t, h, w, rh, rw), m).sum())
            k = int(rng.integers(n_res, n + 1))
            descs.append((t, h, w, rh, rw, m, k))
            parts.append((rng.integers(0, 4, n) if trial % 2 else rng.random(n)).astype(np.float32))
        scores = np.concatenate(parts)
        keep, flat = o.select_ragged(scores, descs)
        tok0 = np.concatenate([[0], np.cumsum([d[0] * d[1] * d[2] for d in descs])])
        out0 = np.concatenate([[0], np.cumsum([d[6] for d in descs])])
        assert len(keep) == out0[-1] and len(flat) == out0[-1]
        for s, (d, part) in enumerate(zip(descs, parts)):
            mine = keep[out0[s]:out0[s + 1]]
            check_invariants(part, *d, mine)
            assert np.array_equal(flat[out0[s]:out0[s + 1]], mine + tok0[s])
            if len(part) <= 10:
                want = best_feasible_subset(part, region_ids(*d[:5]), d[5], d[6])
                assert list(mine) == list(want)
        if len(flat):
            assert np.all(np.diff(flat) > 0), "tokens of the concatenation stay in source order"


ALL_SELECT_PINS = [pin_total_order, pin_special_values_in_select, pin_plain_topk_is_stable_argsort,
                   pin_bruteforce_tiny, pin_full_sort_tiny, pin_invariants_on_workloads,
                   pin_invariants_random, pin_floor_inactive, pin_repair_formulation,
                   pin_hand_worked_example, pin_error_codes]
ALL_COMPACT_PINS = [pin_compact_is_take, pin_seq_indices, pin_compact_kv_is_take]
ALL_ADJACENT_PINS = [pin_merge_embeddings, pin_pos_planes, pin_kv_heads, pin_kv_paged, pin_floor_from_ratio,
                     pin_select_ragged]
