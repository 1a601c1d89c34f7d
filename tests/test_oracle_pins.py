"""Pins for the CPU oracle: every oracle function is checked against something
other than itself -- numbers the paper prints, closed forms, invariants,
special cases that reduce to a library routine, finite differences, brute
force.  CPU only."""
import itertools

import numpy as np
import pytest
import torch

from oracle import cowa_oracle as orc

RNG = np.random.default_rng(1234)


# ---------------------------------------------------------------- windows/mask

def test_paper_token_budgets(golden):
    # Final-query support of every head equals the printed budget
    # (table "Per-Query Token Budgets"); w_sink=1, w_near=1023, H_k=8.
    for n, budget in golden("paper_token_budgets.txt"):
        n, budget = int(n), int(budget)
        ws = orc.default_windows(n, 8, 1, 1023)
        for w in ws:
            assert w[0] + w[1] + w[3] == budget or n == 1024
            row = orc.visible_mask(n, n, w, rows=[n - 1])
            assert int(row.sum()) == budget


@pytest.mark.parametrize("sink,near", [(1, 1023), (128, 896), (512, 512)])
def test_paper_mean_support(golden, sink, near):
    # s-bar printed in the scaling-law appendix; independent of how the
    # shared 1024 tokens are divided between sink and near.
    for n, sbar in golden("paper_mean_support.txt"):
        n = int(n)
        if n > 4096 and (sink, near) != (1, 1023):
            continue  # the 32K count is done once (it walks 8 x 32768^2 pairs)
        ws = orc.default_windows(n, 8, sink, near)
        total = sum(int(orc.support_sizes(n, n, w).sum()) for w in ws)
        assert round(total / (8 * n), 2) == sbar


def test_fullattn_mean_support():
    # Dense causal: s-bar = (n + 1) / 2.
    n = 777
    w = (0, n, 0, 0)
    assert orc.support_sizes(n, n, w).mean() == (n + 1) / 2


def test_coverage_layout_fractions(golden):
    # Fraction of the long-range span [sink, N - near) of the final query that
    # some head sees, for the m-unique-window layouts over 8 heads.
    n, sink, near = 8192, 1, 1023
    for m, pct in golden("paper_coverage_layouts.txt"):
        ws = orc.duplicated_windows(n, 8, sink, near, int(m))
        seen = np.zeros(n, dtype=bool)
        for w in ws:
            seen |= orc.visible_mask(n, n, w, rows=[n - 1])[0]
        span = seen[sink:n - near]
        assert 100.0 * span.mean() == pct


@pytest.mark.parametrize("n_q,n_k,h_k,sink,near", [
    (257, 257, 8, 3, 17), (64, 300, 4, 0, 5), (1, 513, 8, 16, 33),
    (100, 100, 3, 7, 1), (90, 90, 8, 40, 60), (129, 200, 5, 2, 190), (50, 50, 16, 4, 4),
])
def test_mask_invariants(n_q, n_k, h_k, sink, near):
    ws = orc.default_windows(n_k, h_k, sink, near)
    delta = orc.causal_distance(n_q, n_k)
    causal = delta >= 0
    masks = [orc.visible_mask(n_q, n_k, w) for w in ws]
    # collective coverage: union over heads = causal prefix, for every query
    union = np.zeros_like(causal)
    for m in masks:
        assert not (m & ~causal).any()
        union |= m
    assert (union == causal).all()
    # shared windows identical across heads; long bands pairwise disjoint in distance
    i_k = np.arange(n_k)[None, :]
    shared = causal & ((delta < near) | (i_k < sink))
    longs = []
    for m, w in zip(masks, ws):
        assert ((m & shared) == shared).all()
        assert (w[0], w[1]) == (sink, near)
        longs.append((w[1] + w[2], w[1] + w[2] + w[3]))
    for (a0, a1), (b0, b1) in itertools.combinations(longs, 2):
        assert min(a1, b1) <= max(a0, b0)  # empty intersection of [a0,a1) and [b0,b1)
    # the bands tile [near, near + L) without holes
    span = max(n_k - sink - near, 0)
    assert longs[0][0] == near and longs[-1][1] == near + span
    for (a0, a1), (b0, b1) in zip(longs, longs[1:]):
        assert a1 == b0
    # closed form at the final query when sink + near <= N_k
    total = sum(int(m[n_q - 1].sum()) for m in masks)
    if sink + near <= n_k:
        assert total == h_k * (sink + near) + span
    else:
        assert total == h_k * n_k


def test_mask_brute_force():
    # element-by-element loops straight from the three window definitions
    n_q, n_k = 23, 41
    for w in [(3, 4, 5, 6), (0, 1, 0, 0), (2, 7, 0, 9), (50, 3, 2, 2), (1, 2, 30, 100)]:
        m = orc.visible_mask(n_q, n_k, w)
        for iq in range(n_q):
            for ik in range(n_k):
                d = iq + (n_k - n_q) - ik
                near = 0 <= d < w[1]
                sink = ik < w[0] and d >= 0
                far = w[1] + w[2] <= d < w[1] + w[2] + w[3]
                assert m[iq, ik] == (near or sink or far)
        # the mask restricted to chosen rows and key columns is the same predicate on that sub-rectangle
        rows, cols = np.array([0, 5, 22]), np.array([40, 0, 7, 8, 33])
        assert (orc.visible_mask(n_q, n_k, w, rows, cols) == m[np.ix_(rows, cols)]).all()


def test_breakpoints_floor_and_global_index():
    # floor rule with L not divisible by H_k, L < H_k, and TP sharding
    ws = orc.default_windows(1000 + 5 + 10, 8, 5, 10)  # L = 1000
    assert [w[2] for w in ws] == [0, 125, 250, 375, 500, 625, 750, 875]
    ws = orc.default_windows(30 + 3, 8, 1, 2)  # L = 30
    b = [(h * 30) // 8 for h in range(9)]
    assert [(w[2], w[3]) for w in ws] == [(b[h], b[h + 1] - b[h]) for h in range(8)]
    ws = orc.default_windows(8, 8, 2, 3)  # L = 3 < H_k: zero-width bands allowed
    assert sum(w[3] for w in ws) == 3 and min(w[3] for w in ws) == 0
    full = orc.default_windows(5000, 8, 16, 100)
    for tp in (2, 4, 8):
        loc = 8 // tp
        got = []
        for r in range(tp):
            got += orc.default_windows(5000, 8, 16, 100, hk_offset=r * loc, hk_local=loc)
        assert got == full


# ---------------------------------------------------------------- forward

# ---------------------------------------------------------------- equal-area breakpoints

@pytest.mark.parametrize("n_q,n_k,h_k,sink,near", [
    (90, 90, 4, 3, 10), (64, 150, 3, 5, 7), (200, 200, 8, 0, 1), (1, 77, 5, 2, 6), (120, 120, 2, 100, 30),
])
def test_equal_area_windows_balance_and_coverage(n_q, n_k, h_k, sink, near):
    ws = orc.equal_area_windows(n_q, n_k, h_k, sink, near)
    span = max(n_k - sink - near, 0)
    # same shape as the default pattern: shared sink/near, bands tile [0, L) in order without gaps
    assert [w[:2] for w in ws] == [(sink, near)] * h_k
    assert ws[0][2] == 0 and all(ws[h][2] + ws[h][3] == ws[h + 1][2] for h in range(h_k - 1))
    assert ws[-1][2] + ws[-1][3] == span
    # hence the heads still cover the whole causal prefix together (Eq. fwa_collective_coverage)
    union = np.zeros((n_q, n_k), dtype=bool)
    for w in ws:
        union |= orc.visible_mask(n_q, n_k, w)
    iq, ik = np.meshgrid(np.arange(n_q), np.arange(n_k), indexing="ij")
    assert np.array_equal(union, iq + (n_k - n_q) - ik >= 0)
    if span == 0:
        return
    # brute force on the explicit masks: the pairs a band adds outside sink and near window, per head
    # and cumulatively; every breakpoint is the first offset whose cumulative count reaches h/H of the total
    delta = iq + (n_k - n_q) - ik
    outside = (delta >= near) & (ik >= sink)
    per_offset = np.array([int((outside & (delta == near + x)).sum()) for x in range(span)])
    cum = np.concatenate([[0], np.cumsum(per_offset)])
    for h, w in enumerate(ws):
        b = w[2]
        assert h_k * cum[b] >= h * cum[-1]
        assert b == 0 or h_k * cum[b - 1] < h * cum[-1]
    areas = [int(cum[w[2] + w[3]] - cum[w[2]]) for w in ws]
    assert sum(areas) == cum[-1]
    assert max(areas) - min(areas) <= 2 * per_offset.max()  # balanced to within the heaviest diagonals


def test_equal_area_windows_special_cases():
    # one query (decode): every offset weighs 1, so equal area is equal width, b_h = ceil(h L / H)
    n_k, h_k, sink, near = 1000, 7, 11, 40
    span = n_k - sink - near
    ws = orc.equal_area_windows(1, n_k, h_k, sink, near)
    assert [w[2] for w in ws] == [-(-h * span // h_k) for h in range(h_k)]
    # square causal case: offsets weigh L, L-1, ..., 1 (a triangle); cutting a triangle into H equal
    # areas from its long side puts the cuts at L (1 - sqrt(1 - h/H))
    n, h_k = 40000, 8
    ws = orc.equal_area_windows(n, n, h_k, 0, 1)
    span = n - 1
    for h, w in enumerate(ws):
        assert abs(w[2] - span * (1.0 - np.sqrt(1.0 - h / h_k))) <= 1.0
    # global head indexing: a rank's tuples are a slice of the global list
    full = orc.equal_area_windows(500, 800, 6, 9, 20)
    assert orc.equal_area_windows(500, 800, 6, 9, 20, hk_offset=2, hk_local=3) == full[2:5]
    # sink + near already cover everything: no bands
    assert orc.equal_area_windows(50, 50, 4, 30, 30) == [(30, 30, 0, 0)] * 4


def _rand(h_q, h_k, n_q, n_k, d):
    q = RNG.standard_normal((h_q, n_q, d))
    k = RNG.standard_normal((h_k, n_k, d))
    v = RNG.standard_normal((h_k, n_k, d))
    return q, k, v


def _sdpa(q, k, v, scale, mask=None, causal=False):
    tq, tk, tv = (torch.from_numpy(x) for x in (q, k, v))
    g = q.shape[0] // k.shape[0]
    tk = tk.repeat_interleave(g, dim=0)
    tv = tv.repeat_interleave(g, dim=0)
    am = None if mask is None else torch.from_numpy(mask)
    return torch.nn.functional.scaled_dot_product_attention(
        tq, tk, tv, attn_mask=am, is_causal=causal, scale=scale).numpy()


def test_forward_dense_cases_match_sdpa():
    h_q, h_k, n, d = 4, 2, 96, 16
    q, k, v = _rand(h_q, h_k, n, n, d)
    scale = 0.3
    ref = _sdpa(q, k, v, scale, causal=True)
    # (a) sink + near > N_k  => dense causal
    o, lse = orc.forward(q, k, v, orc.default_windows(n, h_k, 40, 60), scale)
    np.testing.assert_allclose(o, ref, atol=1e-12)
    # (b) one window covering everything (the FullAttn tuple)
    o2, _ = orc.forward(q, k, v, [(0, n, 0, 0)] * h_k, scale)
    np.testing.assert_allclose(o2, ref, atol=1e-12)
    # (c) H_k = 1 => the single head's windows cover the prefix
    q1, k1, v1 = _rand(4, 1, n, n, d)
    o3, lse3 = orc.forward(q1, k1, v1, orc.default_windows(n, 1, 3, 5), scale)
    np.testing.assert_allclose(o3, _sdpa(q1, k1, v1, scale, causal=True), atol=1e-12)
    # LSE against torch.logsumexp over the causal scores
    s = scale * torch.from_numpy(q1[2]) @ torch.from_numpy(k1[0]).T
    s = s.masked_fill(~torch.ones(n, n, dtype=torch.bool).tril(), float("-inf"))
    np.testing.assert_allclose(lse3[2], torch.logsumexp(s, dim=1).numpy(), atol=1e-12)


def test_forward_head0_is_sliding_window():
    # sink = 0, head 0: near and its adjacent long band form one band of width
    # near + b_1; compare with a banded mask built by numpy's tril/triu.
    h_q, h_k, n, d = 2, 2, 80, 8
    q, k, v = _rand(h_q, h_k, n, n, d)
    near = 7
    ws = orc.default_windows(n, h_k, 0, near)
    width = near + ws[0][3]
    band = np.tril(np.ones((n, n), dtype=bool)) & np.triu(np.ones((n, n), dtype=bool), -(width - 1))
    o, _ = orc.forward(q, k, v, ws, 0.5)
    ref = _sdpa(q[:1], k[:1], v[:1], 0.5, mask=band)
    np.testing.assert_allclose(o[0], ref[0], atol=1e-12)


def test_forward_general_vs_masked_sdpa_and_loops():
    h_q, h_k, n_q, n_k, d = 4, 2, 37, 53, 8
    q, k, v = _rand(h_q, h_k, n_q, n_k, d)
    ws = [(3, 5, 4, 9), (2, 6, 13, 20)]
    scale = 0.25
    o, lse = orc.forward(q, k, v, ws, scale)
    # pure-python definition for one head
    h, hk = 3, 1
    for iq in (0, 11, 36):
        vis = [ik for ik in range(n_k) if orc.visible_mask(n_q, n_k, ws[hk])[iq, ik]]
        sc = np.array([scale * float(q[h, iq] @ k[hk, ik]) for ik in vis])
        z = np.log(np.exp(sc).sum())
        assert abs(z - lse[h, iq]) < 1e-12
        ref = sum(np.exp(s_ - z) * v[hk, ik] for s_, ik in zip(sc, vis))
        np.testing.assert_allclose(o[h, iq], ref, atol=1e-12)
    # rows= gives the same rows; forward_rows agrees
    o_r, lse_r = orc.forward(q, k, v, ws, scale, rows=[5, 36])
    np.testing.assert_allclose(o_r, o[:, [5, 36]], atol=0)
    o_b, lse_b = orc.forward_rows(q, k, v, ws, scale, 2, np.arange(10, 30))
    np.testing.assert_allclose(o_b, o[2, 10:30], atol=1e-13)
    np.testing.assert_allclose(lse_b, lse[2, 10:30], atol=1e-13)


# ---------------------------------------------------------------- backward

def _loss(q, k, v, ws, scale, d_o):
    o, _ = orc.forward(q, k, v, ws, scale)
    return float((o * d_o).sum())


def test_backward_finite_differences():
    h_q, h_k, n, d = 4, 2, 19, 5
    q, k, v = _rand(h_q, h_k, n, n, d)
    d_o = RNG.standard_normal(q.shape)
    ws = [(2, 3, 2, 5), (1, 4, 6, 7)]
    scale = 0.4
    dq, dk, dv = orc.backward(q, k, v, d_o, ws, scale)
    eps = 1e-6
    for arr, grad in ((q, dq), (k, dk), (v, dv)):
        idx = [tuple(RNG.integers(0, s) for s in arr.shape) for _ in range(25)]
        for ix in idx:
            old = arr[ix]
            arr[ix] = old + eps
            fp = _loss(q, k, v, ws, scale, d_o)
            arr[ix] = old - eps
            fm = _loss(q, k, v, ws, scale, d_o)
            arr[ix] = old
            assert abs((fp - fm) / (2 * eps) - grad[ix]) < 1e-7


def test_backward_vs_autograd_and_row_col_variants():
    h_q, h_k, n_q, n_k, d = 4, 2, 48, 48, 8
    q, k, v = _rand(h_q, h_k, n_q, n_k, d)
    d_o = RNG.standard_normal(q.shape)
    ws = orc.default_windows(n_k, h_k, 4, 9)
    scale = 0.35
    dq, dk, dv = orc.backward(q, k, v, d_o, ws, scale)
    tq, tk, tv = (torch.from_numpy(x.copy()).requires_grad_(True) for x in (q, k, v))
    loss = 0.0
    for h in range(h_q):
        hk = h // (h_q // h_k)
        m = torch.from_numpy(orc.visible_mask(n_q, n_k, ws[hk]))
        s = (scale * tq[h] @ tk[hk].T).masked_fill(~m, float("-inf"))
        loss = loss + (torch.softmax(s, dim=1) @ tv[hk] * torch.from_numpy(d_o[h])).sum()
    loss.backward()
    np.testing.assert_allclose(dq, tq.grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(dk, tk.grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(dv, tv.grad.numpy(), atol=1e-12)
    # Delta identity: rowsum(O * dO) == rowsum(P * dP)
    o, _ = orc.forward(q, k, v, ws, scale)
    p, _ = orc._masked_softmax_rows(scale * q[1] @ k[0].T, orc.visible_mask(n_q, n_k, ws[0]))
    np.testing.assert_allclose((o[1] * d_o[1]).sum(1), (p * (d_o[1] @ v[0].T)).sum(1), atol=1e-12)
    # the large-sequence variants compute the same numbers
    rows = np.arange(7, 31)
    np.testing.assert_allclose(orc.backward_dq_rows(q, k, v, d_o, ws, scale, 3, rows),
                               dq[3, rows], atol=1e-12)
    cols = np.arange(0, 16)
    dk_c, dv_c = orc.backward_dkdv_cols(q, k, v, d_o, ws, scale, 1, cols, row_block=10)
    np.testing.assert_allclose(dk_c, dk[1, cols], atol=1e-12)
    np.testing.assert_allclose(dv_c, dv[1, cols], atol=1e-12)
    cols = np.arange(20, 33)
    dk_c, dv_c = orc.backward_dkdv_cols(q, k, v, d_o, ws, scale, 0, cols, row_block=7)
    np.testing.assert_allclose(dk_c, dk[0, cols], atol=1e-12)
    np.testing.assert_allclose(dv_c, dv[0, cols], atol=1e-12)
    # disjoint query-row ranges add up to the whole
    parts = [orc.backward_dkdv_cols(q, k, v, d_o, ws, scale, 0, cols, row_block=7, row_range=r)
             for r in ((0, 11), (11, 12), (12, n_q))]
    np.testing.assert_allclose(sum(x[0] for x in parts), dk[0, cols], atol=1e-12)
    np.testing.assert_allclose(sum(x[1] for x in parts), dv[0, cols], atol=1e-12)


# ---------------------------------------------------------------- decode

def test_decode_is_last_forward_row():
    b_sz, h_q, h_k, t_max, d = 3, 4, 2, 70, 8
    q = RNG.standard_normal((b_sz, h_q, d))
    kc = RNG.standard_normal((b_sz, h_k, t_max, d))
    vc = RNG.standard_normal((b_sz, h_k, t_max, d))
    lens = np.array([70, 1, 37])
    sink, near, scale = 3, 6, 0.3
    o, lse = orc.decode(q, kc, vc, lens, sink, near, scale)
    for b in range(b_sz):
        n = int(lens[b])
        ws = orc.default_windows(n, h_k, sink, near)
        # a full forward whose last query is the decode query
        qq = RNG.standard_normal((h_q, n, d))
        qq[:, n - 1] = q[b]
        of, lf = orc.forward(qq, kc[b][:, :n], vc[b][:, :n], ws, scale)
        np.testing.assert_allclose(o[b], of[:, n - 1], atol=1e-12)
        np.testing.assert_allclose(lse[b], lf[:, n - 1], atol=1e-12)


def test_decode_ranges_count_and_structure():
    # final-query count: sink + near + long width when they do not overlap
    for n_k, h_k, sink, near in [(1000, 8, 16, 100), (98304, 8, 128, 4096), (50, 4, 30, 30), (5, 2, 0, 1)]:
        ws = orc.default_windows(n_k, h_k, sink, near)
        tot = 0
        for w in ws:
            rg = orc.decode_visible_ranges(n_k, w)
            cnt = sum(b - a for a, b in rg)
            tot += cnt
            assert len(rg) <= 3
            if sink + near <= n_k:
                assert cnt == sink + near + w[3]
            else:
                assert rg == [(0, n_k)]
            rg2, blocks = orc.decode_schedule(n_k, w, 128)
            assert rg2 == rg
            want = sorted({x // 128 for a, b in rg for x in (range(a, b))})
            assert blocks == want
        if sink + near <= n_k:
            assert tot == h_k * (sink + near) + (n_k - sink - near)


# ---------------------------------------------------------------- schedule

@pytest.mark.parametrize("n_q,n_k,b_q,b_k", [(200, 200, 32, 32), (96, 160, 32, 16), (130, 130, 64, 64)])
def test_schedule_from_mask(n_q, n_k, b_q, b_k):
    ws = orc.default_windows(n_k, 3, 5, 20) + [(0, n_k, 0, 0), (7, 3, 11, 40)]
    fwd = orc.tile_schedule_fwd(n_q, n_k, ws, b_q, b_k)
    bwd = orc.tile_schedule_bwd(n_q, n_k, ws, b_q, b_k)
    t_q, t_k = -(-n_q // b_q), -(-n_k // b_k)
    for hk, w in enumerate(ws):
        m = orc.visible_mask(n_q, n_k, w)
        for i in range(t_q):
            lst = fwd[(hk, i)]
            assert [j for j, _ in lst] == sorted((j for j, _ in lst), reverse=True)
            listed = dict(lst)
            for j in range(t_k):
                blk = m[i * b_q:(i + 1) * b_q, j * b_k:(j + 1) * b_k]
                assert (j in listed) == bool(blk.any())
                if j in listed:
                    is_full = blk.shape == (b_q, b_k) and bool(blk.all())
                    assert listed[j] == is_full
        # backward lists are the transpose relation, ascending
        for j in range(t_k):
            lst = bwd[(hk, j)]
            assert [i for i, _ in lst] == sorted(i for i, _ in lst)
            for i in range(t_q):
                in_f = dict(fwd[(hk, i)]).get(j)
                in_b = dict(lst).get(i)
                assert in_f == in_b
