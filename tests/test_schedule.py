"""The library's analytic scheduler (cowa_schedule_dump, host-only) against the oracle's
schedule derived from the explicit mask: bit-exact.  Also checks that the C-ABI library loads
and exports every function declared in include/cowa.h.  CPU only."""
import os
import re

import numpy as np
import pytest

import cowa_inputs
import paper_2609_32704_b200 as cowa
from oracle import cowa_oracle as orc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    text = open(os.path.join(ROOT, "include", "cowa.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(cowa_[a-z_0-9]+)\s*\(", text)
    assert {"cowa_fwd", "cowa_bwd", "cowa_decode"} <= set(names)
    L = cowa.lib()
    for n in set(names):
        assert hasattr(L, n), n


def parse_tiles(stream):
    out, p = {}, 0
    while p < len(stream):
        h, i, n = stream[p:p + 3]
        p += 3
        out[(h, i)] = [(stream[p + 2 * t], bool(stream[p + 2 * t + 1])) for t in range(n)]
        p += 2 * n
    return out


def parse_decode(stream):
    out, p = {}, 0
    while p < len(stream):
        h, r = stream[p:p + 2]
        p += 2
        ranges = [(stream[p + 2 * t], stream[p + 2 * t + 1]) for t in range(r)]
        p += 2 * r
        m = stream[p]
        p += 1
        out[h] = (ranges, list(stream[p:p + m]))
        p += m
    return out


SHAPES = [
    # Nq, Nk, Hkv, sink, near, Bq, Bk
    (1024, 1024, 2, 64, 128, 64, 64),      # the tiny configuration
    (1024, 1024, 2, 64, 128, 128, 128),    # ... at the kernels' tile size
    (1000, 1000, 4, 16, 100, 128, 128),    # ragged tail
    (300, 300, 3, 0, 7, 32, 64),           # Bq != Bk, no sink
    (257, 700, 5, 9, 33, 64, 32),          # Nq < Nk (bottom-right aligned)
    (512, 512, 8, 200, 400, 64, 64),       # sink + near > N: dense
    (640, 640, 8, 3, 5, 128, 128),         # L/Hk not a tile multiple
    (384, 384, 16, 300, 8, 64, 64),        # sink wider than everything else
    (130, 130, 64, 1, 1, 16, 16),          # L < Hk for some heads? (L=128, Hk=64)
    (50, 50, 64, 1, 1, 8, 8),              # L < Hk: zero-width bands
    (1536, 1536, 2, 200, 64, 128, 128),    # sink reaches above a far band's keys
]


@pytest.mark.parametrize("Nq,Nk,Hkv,sink,near,Bq,Bk", SHAPES)
def test_schedule_default_rule(Nq, Nk, Hkv, sink, near, Bq, Bk):
    p = cowa.make_params(sink=sink, local=near, block_q=Bq, block_k=Bk)
    ws = orc.default_windows(Nk, Hkv, sink, near)
    assert cowa.cowa_default_windows(Nk, Hkv, 0, Hkv, sink, near) == ws
    fwd = parse_tiles(cowa.cowa_schedule_dump(cowa.SCHED_FWD, Nq, Nk, Hkv, p))
    assert fwd == orc.tile_schedule_fwd(Nq, Nk, ws, Bq, Bk)
    bwd = parse_tiles(cowa.cowa_schedule_dump(cowa.SCHED_BWD, Nq, Nk, Hkv, p))
    assert bwd == orc.tile_schedule_bwd(Nq, Nk, ws, Bq, Bk)


def test_schedule_random_explicit_tuples():
    rng = np.random.default_rng(7)
    for it in range(400):
        Nk = int(rng.integers(1, 400))
        Nq = int(rng.integers(1, Nk + 1))
        Hkv = int(rng.integers(1, 5))
        Bq, Bk = (int(rng.choice([8, 16, 32, 64])) for _ in range(2))
        smax = 80 if it % 2 else Nk + 1  # every other case lets the sink reach anywhere
        ws = [(int(rng.integers(0, smax)), int(rng.integers(1, 90)), int(rng.integers(0, 150)),
               int(rng.integers(0, 200))) for _ in range(Hkv)]
        p = cowa.make_params(windows=ws, block_q=Bq, block_k=Bk)
        fwd = parse_tiles(cowa.cowa_schedule_dump(cowa.SCHED_FWD, Nq, Nk, Hkv, p))
        assert fwd == orc.tile_schedule_fwd(Nq, Nk, ws, Bq, Bk), (Nq, Nk, ws, Bq, Bk)
        bwd = parse_tiles(cowa.cowa_schedule_dump(cowa.SCHED_BWD, Nq, Nk, Hkv, p))
        assert bwd == orc.tile_schedule_bwd(Nq, Nk, ws, Bq, Bk), (Nq, Nk, ws, Bq, Bk)


def test_schedule_full_attn_and_tp_offset():
    Nq = Nk = 500
    p = cowa.make_params(full_attn=True, block=64)
    fwd = parse_tiles(cowa.cowa_schedule_dump(cowa.SCHED_FWD, Nq, Nk, 2, p))
    assert fwd == orc.tile_schedule_fwd(Nq, Nk, [(0, Nk, 0, 0)] * 2, 64, 64)
    # a tensor-parallel rank holding global heads 4..5 of 8
    p = cowa.make_params(sink=8, local=40, block=32, hkv_global=8, hkv_offset=4)
    ws = orc.default_windows(Nk, 8, 8, 40, hk_offset=4, hk_local=2)
    fwd = parse_tiles(cowa.cowa_schedule_dump(cowa.SCHED_FWD, Nq, Nk, 2, p))
    assert fwd == orc.tile_schedule_fwd(Nq, Nk, ws, 32, 32)


@pytest.mark.parametrize("name", ["8k", "32k", "128k"])
def test_schedule_benchmark_configs_sampled(name):
    # Whole lists at these sizes would walk the full T x T mask; compare a sample of
    # QO tiles per head (first, last, and tiles around every band edge) in full.
    c = cowa_inputs.CONFIGS[name]
    T, Hkv, B = c["T"], c["Hkv"], c["block"]
    p = cowa.make_params(sink=c["sink"], local=c["local"], block=B)
    ws = orc.default_windows(T, Hkv, c["sink"], c["local"])
    fwd = parse_tiles(cowa.cowa_schedule_dump(cowa.SCHED_FWD, T, T, Hkv, p))
    nt = T // B
    for hk, w in enumerate(ws):
        edges = {0, 1, nt - 1, nt // 2}
        for e in (w[0], w[1], w[1] + w[2], w[1] + w[2] + w[3]):
            for d in (-1, 0, 1):
                edges.add(min(max(e // B + d, 0), nt - 1))
        aa = orc._tile_any_all(T, T, w, B, B, row_tiles=sorted(edges))
        for i, (any_j, all_j) in aa.items():
            want = [(int(j), bool(all_j[j])) for j in np.flatnonzero(any_j)[::-1]]
            assert fwd[(hk, i)] == want, (hk, i)
    # counts agree with the dump
    cnt = cowa.cowa_tile_counts(T, T, Hkv, p)
    assert cnt["visited"] == sum(len(v) for v in fwd.values())
    assert cnt["full"] == sum(f for v in fwd.values() for _, f in v)
    assert cnt["causal"] == Hkv * nt * (nt + 1) // 2


def test_equal_area_windows_match_oracle():
    rng = np.random.default_rng(99)
    cases = [(131072, 131072, 8, 128, 896), (32768, 32768, 8, 128, 2048), (1, 5000, 7, 3, 50),
             (50, 50, 4, 30, 30), (64, 150, 3, 5, 7)]
    for _ in range(60):
        nk = int(rng.integers(1, 5000))
        nq = int(rng.integers(1, nk + 1))
        cases.append((nq, nk, int(rng.integers(1, 17)), int(rng.integers(0, 300)), int(rng.integers(1, 600))))
    for nq, nk, hk, sink, near in cases:
        want = orc.equal_area_windows(nq, nk, hk, sink, near)
        assert cowa.cowa_equal_area_windows(nq, nk, hk, 0, hk, sink, near) == want, (nq, nk, hk, sink, near)
        lo = hk // 3
        assert cowa.cowa_equal_area_windows(nq, nk, hk, lo, hk - lo, sink, near) == want[lo:]
    with pytest.raises(cowa.CowaError):
        cowa.cowa_equal_area_windows(10, 5, 2, 0, 2, 0, 1)      # N_q > N_k
    with pytest.raises(cowa.CowaError):
        cowa.cowa_equal_area_windows(10, 10, 2, 1, 2, 0, 1)     # heads beyond the global count


def test_equal_area_schedule_balances_visited_tiles():
    """With the equal-area tuples passed as explicit windows, the visited-tile counts of the heads
    (128K benchmark shape of one TP group) are within a few percent of each other, while the default
    equal-width bands differ by a factor of several."""
    T, hk, sink, near = 131072, 8, 128, 896
    def per_head(ws):
        out = []
        for w in ws:
            p = cowa.make_params(windows=[w], softmax_scale=1.0)
            out.append(cowa.cowa_tile_counts(T, T, 1, p)["visited"])
        return out
    eq = per_head(cowa.cowa_equal_area_windows(T, T, hk, 0, hk, sink, near))
    df = per_head(cowa.cowa_default_windows(T, hk, 0, hk, sink, near))
    assert max(eq) / min(eq) < 1.05
    assert max(df) / min(df) > 3.0
    assert abs(sum(eq) - sum(df)) / sum(df) < 0.02   # same total work, redistributed


def test_bench_legal_pair_count_matches_masks():
    import bench
    rng = np.random.default_rng(7)
    cases = [(300, 4, 7, 20), (1000, 8, 128, 100), (257, 3, 0, 1), (64, 2, 40, 40)]
    cases += [(int(rng.integers(1, 700)), int(rng.integers(1, 9)), int(rng.integers(0, 200)), int(rng.integers(1, 300)))
              for _ in range(20)]
    for T, H, s_, n_ in cases:
        ws = cowa.cowa_default_windows(T, H, 0, H, s_, n_)
        want = sum(int(orc.visible_mask(T, T, w).sum()) for w in ws)
        assert bench.count_legal_pairs(T, ws) == want, (T, H, s_, n_)


def test_decode_schedule():
    for Nk, Hkv, sink, near, Bk in [(131072, 8, 128, 4096, 128), (98304, 8, 128, 4096, 128),
                                    (100001, 8, 128, 4096, 128), (777, 4, 5, 60, 64), (50, 8, 30, 30, 16),
                                    (1, 2, 4, 4, 128), (4225, 8, 128, 4096, 128), (4230, 8, 128, 4096, 128)]:
        p = cowa.make_params(sink=sink, local=near, block=Bk)
        got = parse_decode(cowa.cowa_schedule_dump(cowa.SCHED_DECODE, 1, Nk, Hkv, p))
        ws = orc.default_windows(Nk, Hkv, sink, near)
        for hk, w in enumerate(ws):
            ranges, blocks = orc.decode_schedule(Nk, w, Bk)
            assert got[hk] == (ranges, blocks), (Nk, hk)


def test_decode_schedule_of_several_newest_tokens():
    """Union of the keys the Nq newest tokens see (what the multi-token decode kernel streams), from the
    oracle's explicit mask of those Nq query rows."""
    for Nk, Nq, Hkv, sink, near, Bk in [(5000, 2, 4, 16, 100, 64), (777, 5, 4, 5, 60, 64), (4230, 8, 8, 128, 4096, 128),
                                        (300, 3, 2, 0, 7, 16), (64, 64, 2, 3, 9, 16), (1000, 4, 8, 40, 40, 32)]:
        p = cowa.make_params(sink=sink, local=near, block=Bk)
        got = parse_decode(cowa.cowa_schedule_dump(cowa.SCHED_DECODE, Nq, Nk, Hkv, p))
        for hk, w in enumerate(orc.default_windows(Nk, Hkv, sink, near)):
            seen = orc.visible_mask(Nq, Nk, w).any(axis=0)
            idx = np.flatnonzero(seen)
            cuts = np.flatnonzero(np.diff(idx) > 1)
            starts = np.concatenate([[idx[0]], idx[cuts + 1]])
            ends = np.concatenate([idx[cuts], [idx[-1]]]) + 1
            ranges = [(int(a_), int(b_)) for a_, b_ in zip(starts, ends)]
            blocks = sorted(set(int(i) // Bk for i in idx))
            assert got[hk] == (ranges, blocks), (Nk, Nq, hk)


def test_argument_validation_without_gpu():
    L = cowa.lib()
    p = cowa.make_params(sink=1, local=0)
    assert cowa.cowa_status_string(-2) == "unsupported configuration"
    with pytest.raises(cowa.CowaError):
        cowa.cowa_schedule_dump(cowa.SCHED_FWD, 10, 10, 2, p)      # local < 1
    with pytest.raises(cowa.CowaError):
        cowa.cowa_schedule_dump(cowa.SCHED_FWD, 20, 10, 2, cowa.make_params(sink=1, local=2))  # Nq > Nk
    # null pointers are rejected before any CUDA call
    pp = cowa.make_params(sink=1, local=2, softmax_scale=1.0)
    import ctypes as C
    assert L.cowa_fwd(None, None, None, None, None, 1, 128, 2, 1, 128, C.byref(pp), None) == -1
    assert L.cowa_decode(None, None, None, None, None, None, 1, 128, 2, 1, 128, C.byref(pp), None, 0, None) == -1
