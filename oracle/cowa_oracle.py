"""CPU oracle for CoWindow Attention (CoWA).  TEST INFRASTRUCTURE ONLY.

This file is the parity reference for the CUDA library: a plain, slow, float64
restatement of what the paper defines.  Only tests, the smoke check and the
benchmark's CPU-baseline leg may import it; the product never does, and this
file imports nothing from the product.

Everything is computed from the explicit boolean visibility mask: no tiling, no
online softmax, no schedule.  Functions and the passage each follows:

  default_windows     Eq. (fwa_long_range_span) + the 4-tuple of Sec. 2.1
                      (sink width, near width, gap after near, long width),
                      global KV-head index per Eq. (fwa_global_head)
  duplicated_windows  App. A.1 "Collective-coverage layouts" (W_1..W_m repeated)
  causal_distance     Eq. (fwa_distance)
  visible_mask        the three window sets and their union, Eq. (fwa_support)
  kv_head_of          GQA map of Sec. 2.1 (h_k = floor(h H_k / H_q))
  forward             result of Algorithm 1 (masked softmax; LSE = m + log l)
  backward            result of Algorithm 2 (exact gradient of the forward)
  decode              Sec. 2.3 "Decoding": forward with N_q = 1, N_k = cached+1,
                      breakpoints from the current key length
  tile_schedule_*     block sets J_h(i), I_h(j) of Sec. 2.3 (>= 1 legal pair),
                      with the full / boundary split of the same paragraph
  support_sizes       |A_h(i_q)| per query (used for the s-bar pins, App. A.3)

Pins (tests/test_oracle_pins.py): the paper's printed final-query budgets and
mean support sizes, the closed form of Eq. (fwa_support_counts), collective
coverage Eq. (fwa_collective_coverage), dense-causal special cases checked
against torch's float64 scaled_dot_product_attention, a banded-matrix sliding
window, finite differences and autograd for the gradients, decode == last
forward row.  No function here is unpinned.

Shapes follow the algorithms' REQUIRE lines: q [Hq, Nq, D]; k, v [Hk, Nk, D];
lse [Hq, Nq].  A batch is handled by the caller looping over it.
"""
from __future__ import annotations

import numpy as np

# --------------------------------------------------------------------------
# Windows
# --------------------------------------------------------------------------


def default_windows(n_k, h_k_global, w_sink, w_near, hk_offset=0, hk_local=None):
    """Per-KV-head 4-tuples (sink, near, gap, long) of the default pattern.

    L = max(N_k - w_sink - w_near, 0); b_h = floor(h L / H_k), h = 0..H_k
    (Eq. fwa_long_range_span); tuple_h = (w_sink, w_near, b_h, b_{h+1} - b_h).
    Heads are indexed globally (Eq. fwa_global_head): a rank holding
    hk_local heads starting at hk_offset gets tuples hk_offset..hk_offset+hk_local-1.
    """
    if hk_local is None:
        hk_local = h_k_global - hk_offset
    span = max(int(n_k) - int(w_sink) - int(w_near), 0)
    b = [(h * span) // h_k_global for h in range(h_k_global + 1)]
    return [
        (int(w_sink), int(w_near), b[g], b[g + 1] - b[g])
        for g in range(hk_offset, hk_offset + hk_local)
    ]


def equal_area_windows(n_q, n_k, h_k_global, w_sink, w_near, hk_offset=0, hk_local=None):
    """Equal-area breakpoints: another breakpoint schedule under the same support rule
    (Eq. fwa_support; Sec. 2.1 notes that other schedules redistribute long-range work and
    leaves equal-area allocation for training out of its scope, so the rule is this build's).

    The band offset x (distance delta = w_near + x, 0 <= x < L) is weighted by the number of
    queries for which that distance is causal and points at a key outside the sink:
        c(x) = #{ i_q in [0, N_q) : i_q + (N_k - N_q) - (w_near + x) >= w_sink },
    W(b) = sum_{x < b} c(x), and b_h is the smallest b with H_k * W(b) >= h * W(L), h = 0..H_k.
    The tuples have the default pattern's form (w_sink, w_near, b_h, b_{h+1} - b_h)."""
    if hk_local is None:
        hk_local = h_k_global - hk_offset
    n_q, n_k, w_sink, w_near = int(n_q), int(n_k), int(w_sink), int(w_near)
    span = max(n_k - w_sink - w_near, 0)
    off = n_k - n_q
    x = np.arange(span, dtype=np.int64)
    first_query = np.maximum(w_near + x + w_sink - off, 0)  # first query that reaches a non-sink key
    c = np.clip(n_q - first_query, 0, n_q)
    cum = np.concatenate([[0], np.cumsum(c)]).astype(object)  # exact integers
    total = cum[-1]
    b = []
    for h in range(h_k_global + 1):
        lo = 0
        while h_k_global * cum[lo] < h * total:  # plain scan: obviously the smallest such b
            lo += 1
        b.append(lo)
    return [
        (w_sink, w_near, b[g], b[g + 1] - b[g])
        for g in range(hk_offset, hk_offset + hk_local)
    ]


def duplicated_windows(n_k, h_k, w_sink, w_near, m):
    """m-unique-window control layout (App. A.1): the m long-range regions
    nearest the near window, W_1..W_m of the H_k-way split, are repeated over
    the H_k heads; head h gets W_{(h mod m)+1}.  m = H_k is the default pattern."""
    base = default_windows(n_k, h_k, w_sink, w_near)
    return [base[h % m] for h in range(h_k)]


def kv_head_of(h, h_q, h_k):
    """GQA map: QO head h uses KV head floor(h * H_k / H_q)."""
    return (h * h_k) // h_q


# --------------------------------------------------------------------------
# Mask
# --------------------------------------------------------------------------


def causal_distance(n_q, n_k, rows=None, cols=None):
    """delta[i_q, i_k] = i_q + (N_k - N_q) - i_k  (bottom-right aligned), for the given query rows and key
    columns (all of them by default)."""
    # int32 holds every distance for sequences below 2^30 tokens
    it = np.int32 if max(int(n_q), int(n_k)) < (1 << 30) else np.int64
    rows = np.arange(n_q, dtype=it) if rows is None else np.asarray(rows, dtype=it)
    i_k = np.arange(n_k, dtype=it) if cols is None else np.asarray(cols, dtype=it)
    return rows[:, None] + it(int(n_k) - int(n_q)) - i_k[None, :]


def visible_mask(n_q, n_k, window, rows=None, cols=None):
    """Boolean [len(rows), len(cols)] (all N_k keys by default): key visible to the query under one head's
    tuple.

    near: 0 <= delta < near;  sink: i_k < sink and delta >= 0;
    long: near + gap <= delta < near + gap + long.  Union of the three.
    """
    w_sink, w_near, gap, w_long = (int(x) for x in window)
    delta = causal_distance(n_q, n_k, rows, cols)
    i_k = (np.arange(n_k, dtype=delta.dtype) if cols is None else np.asarray(cols, dtype=delta.dtype))[None, :]
    near = (delta >= 0) & (delta < w_near)
    sink = (i_k < w_sink) & (delta >= 0)
    far = (delta >= w_near + gap) & (delta < w_near + gap + w_long)
    return near | sink | far


def support_sizes(n_q, n_k, window, row_block=64):
    """|A_h(i_q)| for every query, by counting the explicit mask row by row."""
    out = np.empty(n_q, dtype=np.int64)
    for r0 in range(0, n_q, row_block):
        rows = np.arange(r0, min(r0 + row_block, n_q))
        out[r0:r0 + len(rows)] = visible_mask(n_q, n_k, window, rows).sum(axis=1)
    return out


# --------------------------------------------------------------------------
# Forward / backward (whole sequences, dense mask)
# --------------------------------------------------------------------------


def _masked_softmax_rows(s, mask):
    """Row-wise LSE and probabilities of scores s restricted to mask."""
    s = np.where(mask, s, -np.inf)
    m = s.max(axis=1, keepdims=True)
    e = np.exp(s - m)
    l = e.sum(axis=1, keepdims=True)
    lse = (m + np.log(l))[:, 0]
    p = e / l
    return p, lse


def forward(q, k, v, windows, scale, rows=None):
    """O and LSE of the CoWA operator.

    q [Hq,Nq,D], k/v [Hk,Nk,D] float64; windows: one 4-tuple per KV head.
    S = scale * Q K^T on visible pairs, LSE = log sum exp S (natural log),
    O = softmax(S) V.  `rows` restricts the computed queries (the definition is
    per query row, so a subset of rows is the same computation).
    Returns o [Hq, R, D], lse [Hq, R].
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    h_q, n_q, d = q.shape
    h_k, n_k, _ = k.shape
    rows = np.arange(n_q) if rows is None else np.asarray(rows)
    o = np.zeros((h_q, len(rows), v.shape[2]))
    lse = np.zeros((h_q, len(rows)))
    for h in range(h_q):
        hk = kv_head_of(h, h_q, h_k)
        mask = visible_mask(n_q, n_k, windows[hk], rows)
        s = scale * (q[h][rows] @ k[hk].T)
        p, lse[h] = _masked_softmax_rows(s, mask)
        o[h] = p @ v[hk]
    return o, lse


def backward(q, k, v, d_o, windows, scale):
    """dQ, dK, dV: the exact gradient of `forward` w.r.t. its inputs for the
    upstream gradient d_o (textbook softmax-attention gradient; equal to what
    Algorithm 2 accumulates).  dK, dV sum over the QO heads of each group."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    d_o = np.asarray(d_o, dtype=np.float64)
    h_q, n_q, d = q.shape
    h_k, n_k, _ = k.shape
    dq = np.zeros_like(q)
    dk = np.zeros_like(k)
    dv = np.zeros_like(v)
    for h in range(h_q):
        hk = kv_head_of(h, h_q, h_k)
        mask = visible_mask(n_q, n_k, windows[hk])
        s = scale * (q[h] @ k[hk].T)
        p, _ = _masked_softmax_rows(s, mask)
        dv[hk] += p.T @ d_o[h]
        dp = d_o[h] @ v[hk].T
        delta = (p * dp).sum(axis=1, keepdims=True)
        ds = p * (dp - delta)
        dq[h] = scale * (ds @ k[hk])
        dk[hk] += scale * (ds.T @ q[h])
    return dq, dk, dv


# --------------------------------------------------------------------------
# Large sequences: the same definitions, one block of query rows at a time.
# Columns whose mask is False for every row of the block are left out of the
# matrix products (their probability is exactly zero).
# --------------------------------------------------------------------------


def forward_rows(q, k, v, windows, scale, h, rows):
    """O [R,D] and LSE [R] of QO head h for the given query rows."""
    h_q, n_q, _ = q.shape
    h_k, n_k, _ = k.shape
    hk = kv_head_of(h, h_q, h_k)
    rows = np.asarray(rows)
    mask = visible_mask(n_q, n_k, windows[hk], rows)
    cols = np.flatnonzero(mask.any(axis=0))
    qr = np.asarray(q[h][rows], dtype=np.float64)
    kc = np.asarray(k[hk][cols], dtype=np.float64)
    vc = np.asarray(v[hk][cols], dtype=np.float64)
    s = scale * (qr @ kc.T)
    p, lse = _masked_softmax_rows(s, mask[:, cols])
    return p @ vc, lse


def backward_dq_rows(q, k, v, d_o, windows, scale, h, rows):
    """dQ [R,D] of QO head h for the given query rows."""
    h_q, n_q, _ = q.shape
    h_k, n_k, _ = k.shape
    hk = kv_head_of(h, h_q, h_k)
    rows = np.asarray(rows)
    mask = visible_mask(n_q, n_k, windows[hk], rows)
    cols = np.flatnonzero(mask.any(axis=0))
    qr = np.asarray(q[h][rows], dtype=np.float64)
    kc = np.asarray(k[hk][cols], dtype=np.float64)
    vc = np.asarray(v[hk][cols], dtype=np.float64)
    dor = np.asarray(d_o[h][rows], dtype=np.float64)
    s = scale * (qr @ kc.T)
    p, _ = _masked_softmax_rows(s, mask[:, cols])
    dp = dor @ vc.T
    delta = (p * dp).sum(axis=1, keepdims=True)
    ds = p * (dp - delta)
    return scale * (ds @ kc)


def backward_dkdv_cols(q, k, v, d_o, windows, scale, hk, cols, row_block=1024, row_range=None):
    """dK [C,D], dV [C,D] of KV head hk for the given key columns, summed over
    the QO heads of the group and over every query row that sees any of them.
    With row_range = (r0, r1) only the query rows r0 <= i_q < r1 are summed: the
    gradients are sums over query rows, so the results of disjoint ranges add up
    to the whole (a caller may walk the ranges in parallel)."""
    h_q, n_q, d = q.shape
    h_k, n_k, _ = k.shape
    cols = np.asarray(cols)
    group = [h for h in range(h_q) if kv_head_of(h, h_q, h_k) == hk]
    dk = np.zeros((len(cols), d))
    dv = np.zeros((len(cols), v.shape[2]))
    kc_sel = np.asarray(k[hk][cols], dtype=np.float64)
    vc_sel = np.asarray(v[hk][cols], dtype=np.float64)
    first, last = (0, n_q) if row_range is None else (max(int(row_range[0]), 0), min(int(row_range[1]), n_q))
    for r0 in range(first, last, row_block):
        rows = np.arange(r0, min(r0 + row_block, last))
        # rows that see none of the selected columns contribute nothing: find them from the mask on those
        # columns alone before the mask over all keys is built for the rest
        sel = visible_mask(n_q, n_k, windows[hk], rows, cols)
        live = np.flatnonzero(sel.any(axis=1))
        if len(live) == 0:
            continue
        rows = rows[live]
        mask = visible_mask(n_q, n_k, windows[hk], rows)
        keep = mask.any(axis=0)
        keep[cols] = True  # selected columns stay addressable even if unseen here
        allc = np.flatnonzero(keep)
        kc = np.asarray(k[hk][allc], dtype=np.float64)
        vc = np.asarray(v[hk][allc], dtype=np.float64)
        pos = np.searchsorted(allc, cols)  # the selected columns inside allc
        for h in group:
            qr = np.asarray(q[h][rows], dtype=np.float64)
            dor = np.asarray(d_o[h][rows], dtype=np.float64)
            s = scale * (qr @ kc.T)
            p, _ = _masked_softmax_rows(s, mask[:, allc])
            dp = dor @ vc.T
            delta = (p * dp).sum(axis=1, keepdims=True)
            p_sel = p[:, pos] * sel[live]
            ds_sel = p_sel * (dor @ vc_sel.T - delta)
            dv += p_sel.T @ dor
            dk += scale * (ds_sel.T @ qr)
    return dk, dv


# --------------------------------------------------------------------------
# Decode
# --------------------------------------------------------------------------


def decode(q, kcache, vcache, lens, w_sink, w_near, scale, h_k_global=None, hk_offset=0):
    """Single-token decode.  q [B,Hq,D]; caches [B,Hk,Tmax,D]; lens[b] = N_k
    including the current token (already stored at index lens[b]-1).
    For each sequence: windows from the current N_k, then forward with N_q = 1.
    Returns o [B,Hq,D], lse [B,Hq]."""
    b_sz, h_q, d = q.shape
    h_k = kcache.shape[1]
    if h_k_global is None:
        h_k_global = h_k
    o = np.zeros((b_sz, h_q, vcache.shape[3]))
    lse = np.zeros((b_sz, h_q))
    for b in range(b_sz):
        n_k = int(lens[b])
        windows = default_windows(n_k, h_k_global, w_sink, w_near, hk_offset, h_k)
        for h in range(h_q):
            hk = kv_head_of(h, h_q, h_k)
            mask = visible_mask(1, n_k, windows[hk])
            cols = np.flatnonzero(mask[0])
            kc = np.asarray(kcache[b, hk][cols], dtype=np.float64)
            vc = np.asarray(vcache[b, hk][cols], dtype=np.float64)
            s = scale * (np.asarray(q[b, h], dtype=np.float64)[None, :] @ kc.T)
            p, l = _masked_softmax_rows(s, np.ones_like(s, dtype=bool))
            o[b, h] = (p @ vc)[0]
            lse[b, h] = l[0]
    return o, lse


def decode_visible_ranges(n_k, window):
    """Maximal runs [start, end) of visible keys for the single decode query,
    read off the explicit mask row."""
    row = visible_mask(1, n_k, window)[0].astype(np.int8)
    edges = np.diff(np.concatenate(([0], row, [0])))
    starts = np.flatnonzero(edges == 1)
    ends = np.flatnonzero(edges == -1)
    return [(int(a), int(b)) for a, b in zip(starts, ends)]


# --------------------------------------------------------------------------
# Tile schedule, derived from the mask by any() / all()
# --------------------------------------------------------------------------


def _tile_any_all(n_q, n_k, window, b_q, b_k, row_tiles=None):
    """For each requested QO tile: arrays any[j], all[j] over the nominal
    b_q x b_k tiles of the mask padded with False to tile multiples."""
    t_q = -(-n_q // b_q)
    t_k = -(-n_k // b_k)
    row_tiles = range(t_q) if row_tiles is None else row_tiles
    res = {}
    for i in row_tiles:
        rows = np.arange(i * b_q, min((i + 1) * b_q, n_q))
        m = np.zeros((b_q, t_k * b_k), dtype=bool)
        m[:len(rows), :n_k] = visible_mask(n_q, n_k, window, rows)
        m = m.reshape(b_q, t_k, b_k)
        res[i] = (m.any(axis=(0, 2)), m.all(axis=(0, 2)))
    return res


def tile_schedule_fwd(n_q, n_k, windows, b_q, b_k):
    """{(h_k, i): [(j, full), ...]} with j descending (Algorithm 1's order).
    A tile is listed when it holds >= 1 legal pair; full when all b_q*b_k
    pairs of the nominal tile are legal (so sequence-tail tiles are not)."""
    out = {}
    for hk, w in enumerate(windows):
        aa = _tile_any_all(n_q, n_k, w, b_q, b_k)
        for i, (any_j, all_j) in aa.items():
            js = np.flatnonzero(any_j)[::-1]
            out[(hk, i)] = [(int(j), bool(all_j[j])) for j in js]
    return out


def tile_schedule_bwd(n_q, n_k, windows, b_q, b_k):
    """{(h_k, j): [(i, full), ...]} with i ascending (Algorithm 2's order)."""
    t_k = -(-n_k // b_k)
    out = {}
    for hk, w in enumerate(windows):
        lists = {j: [] for j in range(t_k)}
        aa = _tile_any_all(n_q, n_k, w, b_q, b_k)
        for i in sorted(aa):
            any_j, all_j = aa[i]
            for j in np.flatnonzero(any_j):
                lists[int(j)].append((int(i), bool(all_j[j])))
        for j in range(t_k):
            out[(hk, j)] = lists[j]
    return out


def decode_schedule(n_k, window, b_k):
    """(ranges, blocks): visible key ranges of the decode query and the
    b_k-blocks holding at least one visible key, ascending."""
    ranges = decode_visible_ranges(n_k, window)
    row = visible_mask(1, n_k, window)[0]
    t_k = -(-n_k // b_k)
    pad = np.zeros(t_k * b_k, dtype=bool)
    pad[:n_k] = row
    blocks = np.flatnonzero(pad.reshape(t_k, b_k).any(axis=1))
    return ranges, [int(x) for x in blocks]
