"""GPU parity: the CUDA path (through the C ABI) against the float64 CPU oracle on the same
seeded bf16 inputs.  Tolerances (bf16 inputs/outputs, fp32 accumulation, P and dS rounded to bf16
before their second product): O and gradients max-abs 2e-2 and mean-abs 2e-3, LSE max-abs 1e-3.
Gradients are stored as bf16 and reach magnitudes above 4, where rounding the exact value to bf16
alone costs up to |x| * 2^-8 (half an ulp) and |x| * 2^-10 on average (a quarter of an ulp of at
least |x| * 2^-8); the gradient check therefore allows 2e-2 + 2^-8 * |reference| per element and
2e-3 + 2^-10 * mean|reference| on average.  The second term only matters where most entries are
large, e.g. a packed sequence of five tokens whose every key is attended with weight near one."""
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

import cowa_inputs
import paper_2609_32704_b200 as cowa
from oracle import cowa_oracle as orc

pytestmark = pytest.mark.gpu

TOL_MAX, TOL_MEAN, TOL_LSE = 2e-2, 2e-3, 1e-3
DEV = "cuda"


MEASURED = {}  # (configuration, tensor) -> [max-abs error, sum of mean-abs errors, checks]; written out by conftest.py
_CONFIG = [None]


def check(name, got, want, tol_max=TOL_MAX, tol_mean=TOL_MEAN, rtol=0.0, rtol_mean=0.0):
    got = np.asarray(got, dtype=np.float64)
    err = np.abs(got - want)
    if _CONFIG[0] is not None and np.isfinite(err).all():
        tensor = name.replace(_CONFIG[0], "").split("[")[0].split()[-1]
        rec = MEASURED.setdefault((_CONFIG[0], tensor), [0.0, 0.0, 0, 0.0])
        rec[0] = max(rec[0], float(err.max())); rec[1] += float(err.mean()); rec[2] += 1
        rec[3] = max(rec[3], float(np.abs(want).max()))
    assert np.isfinite(got).all(), f"{name}: non-finite output"
    excess = err - rtol * np.abs(want)
    assert excess.max() <= tol_max, f"{name}: max-abs {err.max():.3e} (excess {excess.max():.3e}) > {tol_max}"
    bound = tol_mean + rtol_mean * np.abs(want).mean()
    assert err.mean() <= bound, f"{name}: mean-abs {err.mean():.3e} > {bound:.3e}"


BF16_HALF_ULP = 2.0 ** -8


def check_grad(name, got, want):
    check(name, got, want, rtol=BF16_HALF_ULP, rtol_mean=BF16_HALF_ULP / 4)


def run_fwd(q, k, v, params):
    B, Hq, T, D = q.shape
    o = torch.full_like(q, float("nan"))
    lse = torch.full((B, Hq, T), float("nan"), dtype=torch.float32, device=q.device)
    cowa.cowa_fwd(q, k, v, o, lse, params)
    torch.cuda.synchronize()
    cowa.cowa_check_device_status()
    return o, lse


def fwd_case(B, T, Hq, Hkv, D, sink, local, seed=50, windows=None, full_attn=False):
    q, k, v, _ = cowa_inputs.make_train_inputs(seed, B, T, Hq, Hkv, D)
    scale = cowa_inputs.softmax_scale(D)
    params = cowa.make_params(sink=sink, local=local, softmax_scale=scale, windows=windows, full_attn=full_attn)
    o, lse = run_fwd(q.to(DEV), k.to(DEV), v.to(DEV), params)
    if full_attn:
        ws = [(0, T, 0, 0)] * Hkv
    else:
        ws = windows if windows is not None else orc.default_windows(T, Hkv, sink, local)
    for b in range(B):
        o_ref, lse_ref = orc.forward(cowa_inputs.to_f64(q[b]), cowa_inputs.to_f64(k[b]), cowa_inputs.to_f64(v[b]),
                                     ws, scale)
        check(f"lse[b={b}]", lse[b].cpu().numpy(), lse_ref, TOL_LSE, TOL_LSE)
        check(f"o[b={b}]", o[b].float().cpu().numpy(), o_ref)


# ------------------------------------------------------------------ forward

def test_fwd_tiny_config():
    c = cowa_inputs.CONFIGS["tiny"]
    _CONFIG[0] = "tiny"
    try:
        fwd_case(c["B"], c["T"], c["Hq"], c["Hkv"], c["D"], c["sink"], c["local"], seed=c["index"])
    finally:
        _CONFIG[0] = None


@pytest.mark.parametrize("B,T,Hq,Hkv,D,sink,local", [
    (1, 128, 1, 1, 128, 0, 128),      # one tile, dense
    (1, 256, 2, 1, 128, 0, 1),        # near = 1: every row sees only itself (+ bands)
    (2, 640, 8, 2, 128, 16, 100),     # bands not tile aligned
    (1, 1000, 4, 4, 64, 7, 33),       # ragged tail, G = 1, D = 64
    (1, 1100, 8, 1, 128, 5, 9),       # H_k = 1: dense causal through the bands
    (1, 512, 4, 2, 128, 300, 300),    # sink + near > T: dense causal
    (1, 1536, 16, 2, 64, 200, 64),    # G = 8, wide sink
    (1, 77, 2, 2, 128, 3, 4),         # shorter than one tile
])
def test_fwd_shapes(B, T, Hq, Hkv, D, sink, local):
    fwd_case(B, T, Hq, Hkv, D, sink, local)


def test_fwd_full_attn_and_explicit_windows():
    fwd_case(1, 900, 4, 2, 128, 0, 1, full_attn=True)
    # duplicated-window control (both heads get the band nearest the near window) and a
    # head-specific layout with a gap and no sink
    ws = orc.duplicated_windows(1024, 2, 64, 128, 1)
    fwd_case(1, 1024, 4, 2, 64, 64, 128, windows=ws)
    fwd_case(1, 700, 2, 2, 128, 0, 1, windows=[(0, 50, 100, 200), (20, 10, 0, 0)])


def test_fwd_8k_config_sampled_heads():
    c = cowa_inputs.CONFIGS["8k"]
    B, T, Hq, Hkv, D = c["B"], c["T"], c["Hq"], c["Hkv"], c["D"]
    q, k, v, _ = cowa_inputs.make_train_inputs(c["index"], B, T, Hq, Hkv, D)
    scale = cowa_inputs.softmax_scale(D)
    params = cowa.make_params(sink=c["sink"], local=c["local"], softmax_scale=scale)
    o, lse = run_fwd(q.to(DEV), k.to(DEV), v.to(DEV), params)
    ws = orc.default_windows(T, Hkv, c["sink"], c["local"])
    rows = np.arange(T)
    _CONFIG[0] = "8k"
    for b, h in [(0, 0), (0, 7), (1, 9), (1, 15)]:
        o_ref, lse_ref = orc.forward_rows(cowa_inputs.to_f64(q[b]), cowa_inputs.to_f64(k[b]),
                                          cowa_inputs.to_f64(v[b]), ws, scale, h, rows)
        check(f"lse[{b},{h}]", lse[b, h].cpu().numpy(), lse_ref, TOL_LSE, TOL_LSE)
        check(f"o[{b},{h}]", o[b, h].float().cpu().numpy(), o_ref)
    _CONFIG[0] = None
    # duplicated-window control at the same shape: one head pair
    wd = orc.duplicated_windows(T, Hkv, c["sink"], c["local"], 1)
    pd = cowa.make_params(softmax_scale=scale, windows=wd)
    o, lse = run_fwd(q.to(DEV), k.to(DEV), v.to(DEV), pd)
    o_ref, lse_ref = orc.forward_rows(cowa_inputs.to_f64(q[0]), cowa_inputs.to_f64(k[0]), cowa_inputs.to_f64(v[0]),
                                      wd, scale, 13, rows)
    check("dup lse", lse[0, 13].cpu().numpy(), lse_ref, TOL_LSE, TOL_LSE)
    check("dup o", o[0, 13].float().cpu().numpy(), o_ref)


# ------------------------------------------------------------------ prefill (N_q <= N_k)

@pytest.mark.parametrize("B,Nq,Nk,Hq,Hkv,D,sink,local", [
    (1, 256, 1024, 4, 2, 128, 16, 100),    # a chunk appended to an existing cache
    (2, 100, 777, 8, 2, 64, 5, 60),        # ragged sizes
    (1, 1, 2000, 4, 2, 128, 32, 200),      # one query: the decode case through the forward kernel
    (1, 513, 514, 2, 1, 128, 0, 7),        # off = 1, H_k = 1
    (1, 300, 5000, 8, 4, 128, 64, 256),    # far bands clipped at the first keys
])
def test_prefill_shapes(B, Nq, Nk, Hq, Hkv, D, sink, local):
    q, _, _, _ = cowa_inputs.make_train_inputs(53, B, Nq, Hq, Hkv, D)
    _, k, v, _ = cowa_inputs.make_train_inputs(54, B, Nk, Hq, Hkv, D)
    scale = cowa_inputs.softmax_scale(D)
    params = cowa.make_params(sink=sink, local=local, softmax_scale=scale)
    o = torch.full_like(q, float("nan")).to(DEV)
    lse = torch.full((B, Hq, Nq), float("nan"), dtype=torch.float32, device=DEV)
    cowa.cowa_prefill(q.to(DEV), k.to(DEV), v.to(DEV), o, lse, params)
    torch.cuda.synchronize()
    cowa.cowa_check_device_status()
    ws = orc.default_windows(Nk, Hkv, sink, local)
    f = cowa_inputs.to_f64
    for b in range(B):
        o_ref, lse_ref = orc.forward(f(q[b]), f(k[b]), f(v[b]), ws, scale)
        check(f"prefill lse[b={b}]", lse[b].cpu().numpy(), lse_ref, TOL_LSE, TOL_LSE)
        check(f"prefill o[b={b}]", o[b].float().cpu().numpy(), o_ref)


# ------------------------------------------------------------------ prefill over a packed batch

def _packed_inputs(seed, seqs, Hq, Hkv, D):
    """Per-sequence inputs concatenated along the token axis: q [Hq,total_q,D], k, v [Hkv,total_k,D]."""
    qs, ks, vs = [], [], []
    for b, (nq, nk) in enumerate(seqs):
        if nq > 0:
            qs.append(cowa_inputs.make_train_inputs(seed + 2 * b, 1, nq, Hq, Hkv, D)[0][0])
        _, kb, vb, _ = cowa_inputs.make_train_inputs(seed + 2 * b + 1, 1, nk, Hq, Hkv, D)
        ks.append(kb[0]); vs.append(vb[0])
    cu_q = np.concatenate([[0], np.cumsum([s[0] for s in seqs])]).astype(np.int32)
    cu_k = np.concatenate([[0], np.cumsum([s[1] for s in seqs])]).astype(np.int32)
    return torch.cat(qs, 1).contiguous(), torch.cat(ks, 1).contiguous(), torch.cat(vs, 1).contiguous(), cu_q, cu_k


def _run_varlen(q, k, v, cu_q, cu_k, params):
    Hq, total_q, _ = q.shape
    o = torch.full_like(q, float("nan")).to(DEV)
    lse = torch.full((Hq, total_q), float("nan"), dtype=torch.float32, device=DEV)
    cowa.cowa_prefill_varlen(q.to(DEV), k.to(DEV), v.to(DEV), o, lse, torch.from_numpy(cu_q).to(DEV),
                             torch.from_numpy(cu_k).to(DEV), params)
    torch.cuda.synchronize()
    return o, lse


@pytest.mark.parametrize("seqs,Hq,Hkv,D,sink,local,mode", [
    ([(100, 100), (1, 700), (300, 1000), (0, 50), (257, 300), (128, 128), (129, 4000)], 4, 2, 128, 16, 100, "default"),
    ([(64, 64), (65, 129), (1000, 1000), (5, 5)], 8, 2, 64, 5, 60, "default"),
    ([(200, 900), (333, 333), (1, 1)], 4, 4, 128, 8, 50, "full"),
    ([(384, 2000), (500, 2000), (77, 1500)], 4, 2, 128, 0, 0, "explicit"),
])
def test_prefill_varlen(seqs, Hq, Hkv, D, sink, local, mode):
    q, k, v, cu_q, cu_k = _packed_inputs(71, seqs, Hq, Hkv, D)
    scale = cowa_inputs.softmax_scale(D)
    tuples = None
    if mode == "explicit":  # the same tuples for every sequence, whatever its length
        tuples = [(24, 90, 100, 400), (3, 130, 700, 900)][:Hkv]
        params = cowa.make_params(windows=tuples, softmax_scale=scale)
    else:
        params = cowa.make_params(sink=sink, local=local, softmax_scale=scale, full_attn=(mode == "full"))
    o, lse = _run_varlen(q, k, v, cu_q, cu_k, params)
    cowa.cowa_check_device_status()
    f = cowa_inputs.to_f64
    for b, (nq, nk) in enumerate(seqs):
        if nq == 0:
            continue
        if mode == "explicit":
            ws = np.array(tuples, dtype=np.int64)
        elif mode == "full":
            ws = np.array([(0, nk, 0, 0)] * Hkv, dtype=np.int64)
        else:
            ws = orc.default_windows(nk, Hkv, sink, local)
        qs, ks = slice(cu_q[b], cu_q[b + 1]), slice(cu_k[b], cu_k[b + 1])
        o_ref, lse_ref = orc.forward(f(q[:, qs]), f(k[:, ks]), f(v[:, ks]), ws, scale)
        check(f"varlen lse[seq {b}]", lse[:, qs].cpu().numpy(), lse_ref, TOL_LSE, TOL_LSE)
        check(f"varlen o[seq {b}]", o[:, qs].float().cpu().numpy(), o_ref)


def test_prefill_varlen_equals_batched():
    """Equal-length sequences: the packed call must reproduce the batched call bit for bit."""
    B, Nq, Nk, Hq, Hkv, D = 3, 384, 1024, 4, 2, 128
    q, _, _, _ = cowa_inputs.make_train_inputs(81, B, Nq, Hq, Hkv, D)
    _, k, v, _ = cowa_inputs.make_train_inputs(82, B, Nk, Hq, Hkv, D)
    params = cowa.make_params(sink=16, local=128, softmax_scale=cowa_inputs.softmax_scale(D))
    o = torch.empty_like(q).to(DEV)
    lse = torch.empty((B, Hq, Nq), dtype=torch.float32, device=DEV)
    cowa.cowa_prefill(q.to(DEV), k.to(DEV), v.to(DEV), o, lse, params)
    pack = lambda x: x.permute(1, 0, 2, 3).reshape(x.shape[1], -1, x.shape[3]).contiguous()
    cu_q = (np.arange(B + 1) * Nq).astype(np.int32)
    cu_k = (np.arange(B + 1) * Nk).astype(np.int32)
    o2, lse2 = _run_varlen(pack(q), pack(k), pack(v), cu_q, cu_k, params)
    cowa.cowa_check_device_status()
    assert torch.equal(pack(o), o2)
    assert torch.equal(lse.permute(1, 0, 2).reshape(Hq, -1), lse2)


def test_prefill_varlen_bad_offsets_reported():
    """A sequence with N_q > N_k is skipped on the device and reported by the status call; the library
    stays usable."""
    seqs = [(64, 64), (100, 200)]
    q, k, v, cu_q, cu_k = _packed_inputs(91, seqs, 2, 1, 64)
    params = cowa.make_params(sink=4, local=16, softmax_scale=0.125)
    bad_q = np.array([0, 24, 164], dtype=np.int32)   # second sequence: 140 queries for ...
    bad_k = np.array([0, 164, 264], dtype=np.int32)  # ... 100 keys
    o, _ = _run_varlen(q, k, v, bad_q, bad_k, params)
    with pytest.raises(cowa.CowaError) as e:
        cowa.cowa_check_device_status()
    assert e.value.status == -8
    assert torch.isnan(o[:, 24:].float()).all()      # nothing of the malformed sequence was written
    cowa.cowa_check_device_status()                   # flag cleared
    o, lse = _run_varlen(q, k, v, cu_q, cu_k, params)
    cowa.cowa_check_device_status()
    assert torch.isfinite(o.float()).all() and torch.isfinite(lse).all()


# ------------------------------------------------------------------ backward

def run_fwd_bwd(q, k, v, d_o, params):
    B, Hq, T, D = q.shape
    Hkv = k.shape[1]
    o, lse = run_fwd(q, k, v, params)
    dq, dk, dv = (torch.full_like(x, float("nan")) for x in (q, k, v))
    nbytes = cowa.cowa_bwd_workspace_bytes(B, T, Hq, Hkv, D, params)
    ws = torch.empty(nbytes + 64, dtype=torch.uint8, device=q.device)
    ws.fill_(0xFF)  # the workspace needs no initialisation by the caller
    cowa.cowa_bwd(q, k, v, o, lse, d_o, dq, dk, dv, params, ws[:nbytes])
    torch.cuda.synchronize()
    cowa.cowa_check_device_status()
    assert (ws[nbytes:] == 0xFF).all(), "backward wrote past its workspace"
    return dq, dk, dv


def bwd_case(B, T, Hq, Hkv, D, sink, local, seed=51, windows=None, full_attn=False):
    q, k, v, d_o = cowa_inputs.make_train_inputs(seed, B, T, Hq, Hkv, D)
    scale = cowa_inputs.softmax_scale(D)
    params = cowa.make_params(sink=sink, local=local, softmax_scale=scale, windows=windows, full_attn=full_attn)
    dq, dk, dv = run_fwd_bwd(q.to(DEV), k.to(DEV), v.to(DEV), d_o.to(DEV), params)
    if full_attn:
        ws = [(0, T, 0, 0)] * Hkv
    else:
        ws = windows if windows is not None else orc.default_windows(T, Hkv, sink, local)
    f = cowa_inputs.to_f64
    for b in range(B):
        dq_r, dk_r, dv_r = orc.backward(f(q[b]), f(k[b]), f(v[b]), f(d_o[b]), ws, scale)
        check_grad(f"dq[b={b}]", dq[b].float().cpu().numpy(), dq_r)
        check_grad(f"dk[b={b}]", dk[b].float().cpu().numpy(), dk_r)
        check_grad(f"dv[b={b}]", dv[b].float().cpu().numpy(), dv_r)


def test_bwd_tiny_config():
    c = cowa_inputs.CONFIGS["tiny"]
    _CONFIG[0] = "tiny"
    try:
        bwd_case(c["B"], c["T"], c["Hq"], c["Hkv"], c["D"], c["sink"], c["local"], seed=c["index"])
    finally:
        _CONFIG[0] = None


@pytest.mark.parametrize("B,T,Hq,Hkv,D,sink,local", [
    (1, 64, 1, 1, 128, 0, 64),        # a single step
    (1, 256, 2, 1, 128, 0, 1),        # near = 1
    (2, 640, 8, 2, 128, 16, 100),     # bands not tile aligned, G = 4
    (1, 1000, 4, 4, 64, 7, 33),       # ragged tail, G = 1, D = 64
    (1, 1100, 8, 1, 128, 5, 9),       # H_k = 1, G = 8
    (1, 512, 4, 2, 128, 300, 300),    # dense causal
    (1, 1536, 16, 2, 64, 200, 64),    # wide sink
    (1, 77, 2, 2, 128, 3, 4),         # shorter than one tile
])
def test_bwd_shapes(B, T, Hq, Hkv, D, sink, local):
    bwd_case(B, T, Hq, Hkv, D, sink, local)


def test_bwd_full_attn_and_explicit_windows():
    bwd_case(1, 900, 4, 2, 128, 0, 1, full_attn=True)
    bwd_case(1, 1024, 4, 2, 64, 64, 128, windows=orc.duplicated_windows(1024, 2, 64, 128, 1))
    bwd_case(1, 700, 2, 2, 128, 0, 1, windows=[(0, 50, 100, 200), (20, 10, 0, 0)])


def _bwd_blocks_per_tile(B, T, Hq, Hkv, D, params):
    """How many blocks share a KV tile's GQA group, read off the workspace size."""
    tpad = (T + 63) // 64 * 64
    extra = cowa.cowa_bwd_workspace_bytes(B, T, Hq, Hkv, D, params) - B * Hq * tpad * (D + 2) * 4
    per = B * Hkv * ((T + 127) // 128) * 2 * 128 * D * 4
    assert extra % per == 0
    return max(extra // per, 1)


def test_bwd_tensor_parallel_shard():
    # One KV head of eight and its 8 QO heads, as a TP=8 rank holds them: windows of the global head, and
    # (few blocks, long sink tiles) the group's heads spread over several blocks per KV tile.
    T, Hq, D, sink, local = 3000, 8, 128, 40, 200
    scale = cowa_inputs.softmax_scale(D)
    for r in (0, 5):
        q, k, v, d_o = cowa_inputs.make_train_inputs(56 + r, 1, T, Hq, 1, D)
        params = cowa.make_params(sink=sink, local=local, softmax_scale=scale, hkv_global=8, hkv_offset=r)
        assert _bwd_blocks_per_tile(1, T, Hq, 1, D, params) == 8
        dq, dk, dv = run_fwd_bwd(q.to(DEV), k.to(DEV), v.to(DEV), d_o.to(DEV), params)
        ws = orc.default_windows(T, 8, sink, local)[r:r + 1]
        f = cowa_inputs.to_f64
        dq_r, dk_r, dv_r = orc.backward(f(q[0]), f(k[0]), f(v[0]), f(d_o[0]), ws, scale)
        check_grad(f"shard {r} dq", dq[0].float().cpu().numpy(), dq_r)
        check_grad(f"shard {r} dk", dk[0].float().cpu().numpy(), dk_r)
        check_grad(f"shard {r} dv", dv[0].float().cpu().numpy(), dv_r)


def test_bwd_group_split_over_some_blocks():
    # A shape where the group of 8 heads is split over 4 blocks of 2 heads each; dK, dV stay bitwise
    # repeatable because the partial sums are added in slot order.
    B, T, Hq, Hkv, D, sink, local = 4, 2048, 16, 2, 64, 16, 256
    params = cowa.make_params(sink=sink, local=local, softmax_scale=cowa_inputs.softmax_scale(D))
    assert _bwd_blocks_per_tile(B, T, Hq, Hkv, D, params) == 4
    bwd_case(B, T, Hq, Hkv, D, sink, local, seed=58)
    q, k, v, d_o = cowa_inputs.make_train_inputs(58, B, T, Hq, Hkv, D, device=DEV)
    _, dk1, dv1 = run_fwd_bwd(q, k, v, d_o, params)
    _, dk2, dv2 = run_fwd_bwd(q, k, v, d_o, params)
    assert torch.equal(dk1, dk2) and torch.equal(dv1, dv2)


def test_fwd_bwd_equal_area_windows():
    # the library's equal-area breakpoints passed back as explicit tuples (training shape, ragged tail)
    T, Hq, Hkv, D, sink, local = 1900, 8, 4, 128, 24, 100
    ws = cowa.cowa_equal_area_windows(T, T, Hkv, 0, Hkv, sink, local)
    assert ws == orc.equal_area_windows(T, T, Hkv, sink, local)
    fwd_case(1, T, Hq, Hkv, D, sink, local, seed=59, windows=ws)
    bwd_case(1, T, Hq, Hkv, D, sink, local, seed=59, windows=ws)


def test_bwd_dkdv_bitwise_repeatable():
    # dK and dV are accumulated in a fixed order inside one block: two runs must agree bit for bit.
    q, k, v, d_o = cowa_inputs.make_train_inputs(52, 1, 2048, 8, 2, 128, device=DEV)
    params = cowa.make_params(sink=32, local=256, softmax_scale=cowa_inputs.softmax_scale(128))
    _, dk1, dv1 = run_fwd_bwd(q, k, v, d_o, params)
    _, dk2, dv2 = run_fwd_bwd(q, k, v, d_o, params)
    assert torch.equal(dk1, dk2) and torch.equal(dv1, dv2)


def test_bwd_deterministic_dq():
    # Fixed-point accumulation of the dQ partial sums: bitwise equal from run to run, and still within
    # the parity tolerance.
    B, T, Hq, Hkv, D, sink, local = 1, 4096, 8, 2, 128, 64, 512
    q, k, v, d_o = cowa_inputs.make_train_inputs(55, B, T, Hq, Hkv, D)
    scale = cowa_inputs.softmax_scale(D)
    params = cowa.make_params(sink=sink, local=local, softmax_scale=scale, deterministic=True)
    args = [x.to(DEV) for x in (q, k, v, d_o)]
    dq1, dk1, dv1 = run_fwd_bwd(*args, params)
    dq2, dk2, dv2 = run_fwd_bwd(*args, params)
    assert torch.equal(dq1, dq2) and torch.equal(dk1, dk2) and torch.equal(dv1, dv2)
    ws = orc.default_windows(T, Hkv, sink, local)
    f = cowa_inputs.to_f64
    for h in (0, 5):
        ref = orc.backward_dq_rows(f(q[0]), f(k[0]), f(v[0]), f(d_o[0]), ws, scale, h, np.arange(T))
        check_grad(f"deterministic dq[{h}]", dq1[0, h].float().cpu().numpy(), ref)


def test_bwd_8k_config_sampled():
    c = cowa_inputs.CONFIGS["8k"]
    B, T, Hq, Hkv, D = c["B"], c["T"], c["Hq"], c["Hkv"], c["D"]
    q, k, v, d_o = cowa_inputs.make_train_inputs(c["index"], B, T, Hq, Hkv, D)
    scale = cowa_inputs.softmax_scale(D)
    params = cowa.make_params(sink=c["sink"], local=c["local"], softmax_scale=scale)
    dq, dk, dv = run_fwd_bwd(q.to(DEV), k.to(DEV), v.to(DEV), d_o.to(DEV), params)
    ws = orc.default_windows(T, Hkv, c["sink"], c["local"])
    f = cowa_inputs.to_f64
    # dQ: whole heads; dK/dV: KV tiles incl. the sink tile, a band edge and the last tile
    _CONFIG[0] = "8k"
    for b, h in [(0, 1), (1, 14)]:
        ref = orc.backward_dq_rows(f(q[b]), f(k[b]), f(v[b]), f(d_o[b]), ws, scale, h, np.arange(T))
        check_grad(f"dq[{b},{h}]", dq[b, h].float().cpu().numpy(), ref)
    for b, hk, tile in [(0, 0, 0), (0, 2, 17), (1, 3, 63), (1, 1, 30)]:
        cols = np.arange(tile * 128, tile * 128 + 128)
        dk_r, dv_r = orc.backward_dkdv_cols(f(q[b]), f(k[b]), f(v[b]), f(d_o[b]), ws, scale, hk, cols)
        check_grad(f"dk[{b},{hk},{tile}]", dk[b, hk, cols].float().cpu().numpy(), dk_r)
        check_grad(f"dv[{b},{hk},{tile}]", dv[b, hk, cols].float().cpu().numpy(), dv_r)
    _CONFIG[0] = None


def test_bwd_8k_duplicated_window_control():
    """The 8K configuration's control layout (Sec. 3, "Collective Coverage with Matched Per-Head Window
    Widths"): every KV head gets the band next to the near window (m = 1), passed as explicit tuples."""
    c = cowa_inputs.CONFIGS["8k"]
    B, T, Hq, Hkv, D = c["B"], c["T"], c["Hq"], c["Hkv"], c["D"]
    q, k, v, d_o = cowa_inputs.make_train_inputs(c["index"], B, T, Hq, Hkv, D)
    scale = cowa_inputs.softmax_scale(D)
    wd = orc.duplicated_windows(T, Hkv, c["sink"], c["local"], 1)
    params = cowa.make_params(softmax_scale=scale, windows=wd)
    dq, dk, dv = run_fwd_bwd(q.to(DEV), k.to(DEV), v.to(DEV), d_o.to(DEV), params)
    f = cowa_inputs.to_f64
    _CONFIG[0] = "8k control"
    b, h = 1, 6
    ref = orc.backward_dq_rows(f(q[b]), f(k[b]), f(v[b]), f(d_o[b]), wd, scale, h, np.arange(T))
    check_grad(f"dq[{b},{h}]", dq[b, h].float().cpu().numpy(), ref)
    for b, hk, tile in [(0, 3, 0), (1, 2, 41)]:  # the sink tile and a tile whose queries straddle the band's far edge
        cols = np.arange(tile * 128, tile * 128 + 128)
        dk_r, dv_r = orc.backward_dkdv_cols(f(q[b]), f(k[b]), f(v[b]), f(d_o[b]), wd, scale, hk, cols)
        check_grad(f"dk[{b},{hk},{tile}]", dk[b, hk, cols].float().cpu().numpy(), dk_r)
        check_grad(f"dv[{b},{hk},{tile}]", dv[b, hk, cols].float().cpu().numpy(), dv_r)
    _CONFIG[0] = None


# ------------------------------------------------------------------ full-size configurations, sampled

def _full_size_sampled(name, q_tiles, kv_samples):
    """Runs forward + backward at a benchmark configuration in the launch configuration bench.py
    times, and compares sampled outputs with the oracle: O/LSE/dQ on whole 128-row query tiles,
    dK/dV on whole 128-row KV tiles (each needs every query row that sees the tile)."""
    c = cowa_inputs.CONFIGS[name]
    B, T, Hq, Hkv, D = c["B"], c["T"], c["Hq"], c["Hkv"], c["D"]
    q, k, v, d_o = cowa_inputs.make_train_inputs(c["index"], B, T, Hq, Hkv, D, device=DEV)
    scale = cowa_inputs.softmax_scale(D)
    params = cowa.make_params(sink=c["sink"], local=c["local"], softmax_scale=scale)
    o, lse = run_fwd(q, k, v, params)
    dq, dk, dv = (torch.empty_like(x) for x in (q, k, v))
    ws_b = torch.empty(cowa.cowa_bwd_workspace_bytes(B, T, Hq, Hkv, D, params), dtype=torch.uint8, device=DEV)
    cowa.cowa_bwd(q, k, v, o, lse, d_o, dq, dk, dv, params, ws_b)
    torch.cuda.synchronize()
    cowa.cowa_check_device_status()
    del ws_b
    ws = orc.default_windows(T, Hkv, c["sink"], c["local"])
    f = cowa_inputs.to_f64
    G = Hq // Hkv
    cache = {}

    def head_inputs(h):  # float64 copies of one QO head and its KV head, shaped like a 1-head problem
        hk = h // G
        if hk not in cache:
            cache.clear()
            cache[hk] = (f(k[0, hk:hk + 1]), f(v[0, hk:hk + 1]))
        return f(q[0, h:h + 1]), cache[hk][0], cache[hk][1], f(d_o[0, h:h + 1]), [ws[hk]]

    _CONFIG[0] = name
    for h, tile in q_tiles:
        rows = np.arange(tile * 128, tile * 128 + 128)
        qh, kh, vh, doh, w1 = head_inputs(h)
        o_ref, lse_ref = orc.forward_rows(qh, kh, vh, w1, scale, 0, rows)
        check(f"{name} lse[h{h},tile{tile}]", lse[0, h, rows].cpu().numpy(), lse_ref, TOL_LSE, TOL_LSE)
        check(f"{name} o[h{h},tile{tile}]", o[0, h, rows].float().cpu().numpy(), o_ref)
        dq_ref = orc.backward_dq_rows(qh, kh, vh, doh, w1, scale, 0, rows)
        check_grad(f"{name} dq[h{h},tile{tile}]", dq[0, h, rows].float().cpu().numpy(), dq_ref)
    for hk, tile in kv_samples:
        cols = np.arange(tile * 128, tile * 128 + 128)
        qg, dog = f(q[0, hk * G:(hk + 1) * G]), f(d_o[0, hk * G:(hk + 1) * G])
        kg, vg = f(k[0, hk:hk + 1]), f(v[0, hk:hk + 1])
        # dK, dV are sums over query rows: the oracle walks disjoint row ranges on the host's cores at once
        # (numpy releases the interpreter lock) and the partial sums are added
        edges = np.linspace(0, T, 17).astype(int)
        with ThreadPoolExecutor(max_workers=8) as pool:
            parts = list(pool.map(lambda r: orc.backward_dkdv_cols(qg, kg, vg, dog, [ws[hk]], scale, 0, cols,
                                                                   row_range=(edges[r], edges[r + 1])), range(16)))
        dk_r, dv_r = sum(x[0] for x in parts), sum(x[1] for x in parts)
        check_grad(f"{name} dk[hk{hk},tile{tile}]", dk[0, hk, cols].float().cpu().numpy(), dk_r)
        check_grad(f"{name} dv[hk{hk},tile{tile}]", dv[0, hk, cols].float().cpu().numpy(), dv_r)
    _CONFIG[0] = None


# ------------------------------------------------------------------ backward with N_q < N_k

@pytest.mark.parametrize("B,Nq,Nk,Hq,Hkv,D,sink,local", [
    (1, 256, 1024, 4, 2, 128, 16, 100),    # a chunk appended to an existing cache
    (2, 100, 777, 8, 2, 64, 5, 60),        # ragged sizes
    (1, 1, 900, 4, 2, 128, 32, 200),       # one query
    (1, 513, 514, 2, 1, 128, 0, 7),        # off = 1, H_k = 1
    (1, 300, 3000, 8, 4, 128, 64, 256),    # far bands clipped; most keys seen by no query of their head
])
def test_bwd_prefill_shapes(B, Nq, Nk, Hq, Hkv, D, sink, local):
    q, _, _, d_o = cowa_inputs.make_train_inputs(55, B, Nq, Hq, Hkv, D)
    _, k, v, _ = cowa_inputs.make_train_inputs(56, B, Nk, Hq, Hkv, D)
    scale = cowa_inputs.softmax_scale(D)
    params = cowa.make_params(sink=sink, local=local, softmax_scale=scale)
    qd, kd, vd, dod = q.to(DEV), k.to(DEV), v.to(DEV), d_o.to(DEV)
    o = torch.empty_like(qd)
    lse = torch.empty((B, Hq, Nq), dtype=torch.float32, device=DEV)
    cowa.cowa_prefill(qd, kd, vd, o, lse, params)
    dq, dk, dv = (torch.full_like(x, float("nan")) for x in (qd, kd, vd))
    nbytes = cowa.cowa_bwd_prefill_workspace_bytes(B, Nq, Nk, Hq, Hkv, D, params)
    ws = torch.empty(nbytes + 64, dtype=torch.uint8, device=DEV)
    ws.fill_(0xFF)
    cowa.cowa_bwd_prefill(qd, kd, vd, o, lse, dod, dq, dk, dv, params, ws[:nbytes])
    torch.cuda.synchronize()
    cowa.cowa_check_device_status()
    assert (ws[nbytes:] == 0xFF).all()
    wins = orc.default_windows(Nk, Hkv, sink, local)
    f = cowa_inputs.to_f64
    for b in range(B):
        dq_r, dk_r, dv_r = orc.backward(f(q[b]), f(k[b]), f(v[b]), f(d_o[b]), wins, scale)
        check_grad(f"prefill dq[b={b}]", dq[b].float().cpu().numpy(), dq_r)
        check_grad(f"prefill dk[b={b}]", dk[b].float().cpu().numpy(), dk_r)
        check_grad(f"prefill dv[b={b}]", dv[b].float().cpu().numpy(), dv_r)


# ------------------------------------------------------------------ backward over a packed batch

@pytest.mark.parametrize("lens,Hq,Hkv,D,sink,local,mode", [
    ([100, 700, 1, 300, 128, 129, 1000], 4, 2, 128, 16, 100, "default"),
    ([64, 65, 2048, 5], 8, 2, 64, 5, 60, "default"),
    ([900, 333], 4, 4, 128, 8, 50, "full"),
    ([1500, 2000, 77], 4, 2, 128, 0, 0, "explicit"),
])
def test_bwd_varlen(lens, Hq, Hkv, D, sink, local, mode):
    seqs = [(n, n) for n in lens]
    q, k, v, cu, _ = _packed_inputs(73, seqs, Hq, Hkv, D)
    d_o = torch.cat([cowa_inputs.make_train_inputs(74 + b, 1, n, Hq, Hkv, D)[3][0] for b, n in enumerate(lens)], 1).contiguous()
    scale = cowa_inputs.softmax_scale(D)
    tuples = None
    if mode == "explicit":
        tuples = [(24, 90, 100, 400), (3, 130, 700, 900)][:Hkv]
        params = cowa.make_params(windows=tuples, softmax_scale=scale)
    else:
        params = cowa.make_params(sink=sink, local=local, softmax_scale=scale, full_attn=(mode == "full"))
    o, lse = _run_varlen(q, k, v, cu, cu, params)
    qd, kd, vd, dod = q.to(DEV), k.to(DEV), v.to(DEV), d_o.to(DEV)
    dq, dk, dv = (torch.full_like(x, float("nan")) for x in (qd, kd, vd))
    total = int(cu[-1])
    nbytes = cowa.cowa_bwd_varlen_workspace_bytes(len(lens), total, Hq, Hkv, D, params)
    ws = torch.empty(nbytes + 64, dtype=torch.uint8, device=DEV)
    ws.fill_(0xFF)
    cowa.cowa_bwd_varlen(qd, kd, vd, o, lse, dod, dq, dk, dv, torch.from_numpy(cu).to(DEV), params, ws[:nbytes])
    torch.cuda.synchronize()
    cowa.cowa_check_device_status()
    assert (ws[nbytes:] == 0xFF).all()
    f = cowa_inputs.to_f64
    for b, n in enumerate(lens):
        if mode == "explicit":
            wsb = tuples
        elif mode == "full":
            wsb = [(0, n, 0, 0)] * Hkv
        else:
            wsb = orc.default_windows(n, Hkv, sink, local)
        sl = slice(cu[b], cu[b + 1])
        dq_r, dk_r, dv_r = orc.backward(f(q[:, sl]), f(k[:, sl]), f(v[:, sl]), f(d_o[:, sl]), wsb, scale)
        check_grad(f"varlen dq[seq {b}]", dq[:, sl].float().cpu().numpy(), dq_r)
        check_grad(f"varlen dk[seq {b}]", dk[:, sl].float().cpu().numpy(), dk_r)
        check_grad(f"varlen dv[seq {b}]", dv[:, sl].float().cpu().numpy(), dv_r)


@pytest.mark.parametrize("bad", [float("nan"), float("inf")])
def test_packed_batch_nonfinite_neighbour_does_not_leak(bad):
    """Rows past the end of a sequence share its last tiles in shared memory.  They are multiplied by exact
    zeros, which is not enough when they hold Inf or NaN: a sequence's outputs must not depend on its
    neighbour's values at all.  Sequence 1 is filled with non-finite values; sequences 0 and 2 must still match
    the oracle (forward and backward), and sequence 1's own outputs are allowed to be anything."""
    lens, Hq, Hkv, D, sink, local = [100, 300, 777], 4, 2, 128, 8, 40
    seqs = [(n, n) for n in lens]
    q, k, v, cu, _ = _packed_inputs(120, seqs, Hq, Hkv, D)
    d_o = torch.cat([cowa_inputs.make_train_inputs(130 + b, 1, n, Hq, Hkv, D)[3][0] for b, n in enumerate(lens)], 1).contiguous()
    sl1 = slice(int(cu[1]), int(cu[2]))
    for t in (q, k, v, d_o):
        t[:, sl1] = bad
    scale = cowa_inputs.softmax_scale(D)
    params = cowa.make_params(sink=sink, local=local, softmax_scale=scale)
    o, lse = _run_varlen(q, k, v, cu, cu, params)
    qd, kd, vd, dod = q.to(DEV), k.to(DEV), v.to(DEV), d_o.to(DEV)
    dq, dk, dv = (torch.full_like(x, float("nan")) for x in (qd, kd, vd))
    total = int(cu[-1])
    ws = torch.empty(cowa.cowa_bwd_varlen_workspace_bytes(len(lens), total, Hq, Hkv, D, params), dtype=torch.uint8, device=DEV)
    cowa.cowa_bwd_varlen(qd, kd, vd, o, lse, dod, dq, dk, dv, torch.from_numpy(cu).to(DEV), params, ws)
    torch.cuda.synchronize()
    cowa.cowa_check_device_status()
    f = cowa_inputs.to_f64
    for b in (0, 2):
        sl = slice(int(cu[b]), int(cu[b + 1]))
        wins = orc.default_windows(lens[b], Hkv, sink, local)
        o_ref, lse_ref = orc.forward(f(q[:, sl]), f(k[:, sl]), f(v[:, sl]), wins, scale)
        check(f"neighbour lse[{b}]", lse[:, sl].cpu().numpy(), lse_ref, TOL_LSE, TOL_LSE)
        check(f"neighbour o[{b}]", o[:, sl].float().cpu().numpy(), o_ref)
        dq_r, dk_r, dv_r = orc.backward(f(q[:, sl]), f(k[:, sl]), f(v[:, sl]), f(d_o[:, sl]), wins, scale)
        check_grad(f"neighbour dq[{b}]", dq[:, sl].float().cpu().numpy(), dq_r)
        check_grad(f"neighbour dk[{b}]", dk[:, sl].float().cpu().numpy(), dk_r)
        check_grad(f"neighbour dv[{b}]", dv[:, sl].float().cpu().numpy(), dv_r)


def test_bwd_varlen_equals_batched_dkdv():
    """Equal-length sequences: dK and dV of the packed call equal the batched call's bit for bit (same block
    arithmetic); dQ agrees within the tolerance (reduction order differs)."""
    B, T, Hq, Hkv, D = 3, 1024, 4, 2, 128
    q, k, v, d_o = cowa_inputs.make_train_inputs(83, B, T, Hq, Hkv, D, device=DEV)
    params = cowa.make_params(sink=16, local=128, softmax_scale=cowa_inputs.softmax_scale(D))
    o, lse = run_fwd(q, k, v, params)
    dq, dk, dv = (torch.empty_like(x) for x in (q, k, v))
    ws = torch.empty(cowa.cowa_bwd_workspace_bytes(B, T, Hq, Hkv, D, params), dtype=torch.uint8, device=DEV)
    cowa.cowa_bwd(q, k, v, o, lse, d_o, dq, dk, dv, params, ws)
    pack = lambda x: x.permute(1, 0, 2, 3).reshape(x.shape[1], -1, x.shape[3]).contiguous()
    cu = torch.arange(B + 1, dtype=torch.int32, device=DEV) * T
    dq2, dk2, dv2 = (torch.empty_like(pack(x)) for x in (q, k, v))
    ws2 = torch.empty(cowa.cowa_bwd_varlen_workspace_bytes(B, B * T, Hq, Hkv, D, params), dtype=torch.uint8, device=DEV)
    cowa.cowa_bwd_varlen(pack(q), pack(k), pack(v), pack(o), lse.permute(1, 0, 2).reshape(Hq, -1).contiguous(), pack(d_o),
                         dq2, dk2, dv2, cu, params, ws2)
    torch.cuda.synchronize()
    cowa.cowa_check_device_status()
    if cowa.cowa_bwd_workspace_bytes(B, T, Hq, Hkv, D, params) == B * Hq * T * (D + 2) * 4:  # whole group per block
        assert torch.equal(pack(dk), dk2) and torch.equal(pack(dv), dv2)
    assert (pack(dk).float() - dk2.float()).abs().max().item() <= 2e-2
    assert (pack(dq).float() - dq2.float()).abs().max().item() <= 2e-2


def test_32k_config_sampled():
    # query tiles: first, last, and tiles whose rows straddle a band edge of their head
    _full_size_sampled("32k", q_tiles=[(0, 0), (3, 255), (9, 17), (14, 100), (31, 255), (20, 46)],
                       kv_samples=[(0, 0), (2, 77), (7, 255)])


def test_128k_config_sampled():
    # KV tiles: one in the middle of a far head's range, the sink tile (the longest block of the launch: every
    # query tile of the group's four heads visits it) and the tile of head 0 whose queries straddle the far
    # edge of that head's band (near + band = 4096 + 15856 keys back)
    _full_size_sampled("128k", q_tiles=[(0, 1023), (5, 33), (13, 500), (31, 1023), (18, 157)],
                       kv_samples=[(6, 901), (0, 0), (0, 867)])


def test_one_million_tokens_sampled():
    """Largest size exercised: T = 2^20 (indices and byte offsets beyond 2^31 in the tensors).  Forward
    and backward run in full; O, LSE and dQ are compared on sampled query tiles, decode on the full row."""
    T, Hq, Hkv, D, sink, local = 1 << 20, 2, 2, 64, 128, 4096
    q, k, v, d_o = cowa_inputs.make_train_inputs(77, 1, T, Hq, Hkv, D, device=DEV)
    scale = cowa_inputs.softmax_scale(D)
    params = cowa.make_params(sink=sink, local=local, softmax_scale=scale)
    o, lse = run_fwd(q, k, v, params)
    dq, dk, dv = (torch.empty_like(x) for x in (q, k, v))
    ws_b = torch.empty(cowa.cowa_bwd_workspace_bytes(1, T, Hq, Hkv, D, params), dtype=torch.uint8, device=DEV)
    cowa.cowa_bwd(q, k, v, o, lse, d_o, dq, dk, dv, params, ws_b)
    torch.cuda.synchronize()
    cowa.cowa_check_device_status()
    del ws_b
    assert torch.isfinite(dk.float()).all() and torch.isfinite(dv.float()).all()
    ws = orc.default_windows(T, Hkv, sink, local)
    f = cowa_inputs.to_f64
    for h, tile in [(0, 0), (1, T // 128 - 1), (0, 5000)]:
        rows = np.arange(tile * 128, tile * 128 + 128)
        qh, kh, vh, doh = f(q[0, h:h + 1]), f(k[0, h:h + 1]), f(v[0, h:h + 1]), f(d_o[0, h:h + 1])
        o_ref, lse_ref = orc.forward_rows(qh, kh, vh, [ws[h]], scale, 0, rows)
        check(f"1M lse[h{h},tile{tile}]", lse[0, h, rows].cpu().numpy(), lse_ref, TOL_LSE, TOL_LSE)
        check(f"1M o[h{h},tile{tile}]", o[0, h, rows].float().cpu().numpy(), o_ref)
        dq_ref = orc.backward_dq_rows(qh, kh, vh, doh, [ws[h]], scale, 0, rows)
        check_grad(f"1M dq[h{h},tile{tile}]", dq[0, h, rows].float().cpu().numpy(), dq_ref)
        del qh, kh, vh, doh
    # decode of the last position on the same tensors used as a cache of length T
    lens = torch.tensor([T], dtype=torch.int32, device=DEV)
    o_d, lse_d = run_decode(q[:, :, T - 1].contiguous(), k, v, lens, params)
    assert (o_d.float() - o[:, :, T - 1].float()).abs().max().item() <= 2e-2
    assert (lse_d - lse[:, :, T - 1]).abs().max().item() <= 1e-3


# ------------------------------------------------------------------ decode

def run_decode(q, kc, vc, lens, params):
    B, Hq, D = q.shape
    Hkv, Tmax = kc.shape[1], kc.shape[2]
    o = torch.full_like(q, float("nan"))
    lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=q.device)
    nbytes = cowa.cowa_decode_workspace_bytes(B, Tmax, Hq, Hkv, D, params)
    ws = torch.empty(nbytes + 64, dtype=torch.uint8, device=q.device)
    ws.fill_(0xFF)  # NaN pattern: the workspace needs no initialisation
    cowa.cowa_decode(q, kc, vc, lens, o, lse, params, ws[:nbytes])
    torch.cuda.synchronize()
    assert (ws[nbytes:] == 0xFF).all(), "decode wrote past its workspace"
    return o, lse


def decode_case(B, Tmax, Hq, Hkv, D, sink, local, lens, seed=60, full_attn=False):
    q, kc, vc, _ = cowa_inputs.make_decode_inputs(seed, B, Tmax, Hq, Hkv, D, Tmax, Tmax)
    lens = torch.tensor(lens, dtype=torch.int32)
    for b in range(B):  # NaN beyond the chosen lengths: an over-read shows up
        kc[b, :, int(lens[b]):] = float("nan")
        vc[b, :, int(lens[b]):] = float("nan")
    scale = cowa_inputs.softmax_scale(D)
    params = cowa.make_params(sink=sink, local=local, softmax_scale=scale, full_attn=full_attn)
    o, lse = run_decode(q.to(DEV), kc.to(DEV), vc.to(DEV), lens.to(DEV), params)
    if full_attn:
        sink, local = 0, Tmax
    kf, vf = kc.float().numpy(), vc.float().numpy()
    o_ref, lse_ref = orc.decode(cowa_inputs.to_f64(q), kf, vf, lens.numpy(), sink, local, scale)
    check("decode lse", lse.cpu().numpy(), lse_ref, TOL_LSE, TOL_LSE)
    check("decode o", o.float().cpu().numpy(), o_ref)


@pytest.mark.parametrize("B,Tmax,Hq,Hkv,D,sink,local,lens", [
    (3, 5000, 8, 2, 128, 16, 100, [5000, 1, 2777]),
    (2, 3001, 8, 8, 64, 4, 31, [3001, 17]),            # G = 1, D = 64
    (2, 4096, 16, 2, 128, 128, 512, [4096, 640]),      # G = 8; second sequence is dense
    (1, 40000, 4, 2, 128, 128, 4096, [39999]),         # several splits per head
    (4, 300, 4, 2, 64, 0, 5, [300, 299, 6, 5]),        # no sink
])
def test_decode_shapes(B, Tmax, Hq, Hkv, D, sink, local, lens):
    decode_case(B, Tmax, Hq, Hkv, D, sink, local, lens)


def test_decode_full_attn():
    decode_case(2, 9000, 8, 2, 128, 0, 1, [9000, 4321], full_attn=True)


def test_decode_128k_config():
    c = cowa_inputs.CONFIGS["decode128k"]
    q, kc, vc, lens = cowa_inputs.make_decode_inputs(c["index"], c["B"], c["Tmax"], c["Hq"], c["Hkv"], c["D"],
                                                     c["len_lo"], c["len_hi"], device=DEV)
    scale = cowa_inputs.softmax_scale(c["D"])
    params = cowa.make_params(sink=c["sink"], local=c["local"], softmax_scale=scale)
    o, lse = run_decode(q, kc, vc, lens, params)
    lens_h = lens.cpu().numpy()
    o_h, lse_h = o.float().cpu().numpy(), lse.cpu().numpy()
    # the oracle walks each head's visible rows only; move one (sequence, KV head) at a time
    G = c["Hq"] // c["Hkv"]
    for b in range(c["B"]):
        for hk in range(c["Hkv"]):
            kf = kc[b:b + 1, hk:hk + 1].cpu().to(torch.float64).numpy()
            vf = vc[b:b + 1, hk:hk + 1].cpu().to(torch.float64).numpy()
            qf = q[b:b + 1, hk * G:(hk + 1) * G].cpu().to(torch.float64).numpy()
            o_ref, lse_ref = orc.decode(qf, kf, vf, lens_h[b:b + 1], c["sink"], c["local"], scale,
                                        h_k_global=c["Hkv"], hk_offset=hk)
            _CONFIG[0] = "decode128k"
            check(f"decode128k lse[{b},{hk}]", lse_h[b, hk * G:(hk + 1) * G], lse_ref[0], TOL_LSE, TOL_LSE)
            check(f"decode128k o[{b},{hk}]", o_h[b, hk * G:(hk + 1) * G], o_ref[0])
            _CONFIG[0] = None


@pytest.mark.parametrize("offset,local_heads", [(0, 2), (3, 1), (7, 1), (5, 2)])
def test_fwd_and_decode_with_global_head_offsets(offset, local_heads):
    """A tensor-parallel rank holds KV heads offset .. offset+local_heads-1 of 8 and must use the windows of
    the global head index (Eq. fwa_global_head; Sec. 2.3 "Global KV-head assignment"): forward O / LSE and
    decode against the oracle evaluated with the same offset."""
    T, G, D, sink, local = 2500, 4, 128, 24, 160
    Hkv, Hq = local_heads, local_heads * G
    scale = cowa_inputs.softmax_scale(D)
    q, k, v, _ = cowa_inputs.make_train_inputs(90 + offset, 1, T, Hq, Hkv, D)
    params = cowa.make_params(sink=sink, local=local, softmax_scale=scale, hkv_global=8, hkv_offset=offset)
    o, lse = run_fwd(q.to(DEV), k.to(DEV), v.to(DEV), params)
    ws = orc.default_windows(T, 8, sink, local, offset, local_heads)
    assert ws == orc.default_windows(T, 8, sink, local)[offset:offset + local_heads]
    f = cowa_inputs.to_f64
    o_ref, lse_ref = orc.forward(f(q[0]), f(k[0]), f(v[0]), ws, scale)
    check(f"shard {offset} lse", lse[0].cpu().numpy(), lse_ref, TOL_LSE, TOL_LSE)
    check(f"shard {offset} o", o[0].float().cpu().numpy(), o_ref)
    # decode over the same tensors used as a cache, two sequences of different lengths
    lens = [T, 1777]
    qd = torch.stack([q[0, :, n - 1] for n in lens]).contiguous()
    kc, vc = k.expand(2, -1, -1, -1).contiguous(), v.expand(2, -1, -1, -1).contiguous()
    o_d, lse_d = run_decode(qd.to(DEV), kc.to(DEV), vc.to(DEV), torch.tensor(lens, dtype=torch.int32, device=DEV), params)
    od_ref, lsed_ref = orc.decode(f(qd), f(kc), f(vc), np.asarray(lens), sink, local, scale, h_k_global=8, hk_offset=offset)
    check(f"shard {offset} decode lse", lse_d.cpu().numpy(), lsed_ref, TOL_LSE, TOL_LSE)
    check(f"shard {offset} decode o", o_d.float().cpu().numpy(), od_ref)


def test_decode_equals_last_forward_row():
    # cross-path: decode output == last row of the training forward at T = len
    T, Hq, Hkv, D, sink, local = 1500, 4, 2, 128, 32, 200
    q, k, v, _ = cowa_inputs.make_train_inputs(61, 1, T, Hq, Hkv, D, device=DEV)
    scale = cowa_inputs.softmax_scale(D)
    params = cowa.make_params(sink=sink, local=local, softmax_scale=scale)
    o_f, lse_f = run_fwd(q, k, v, params)
    lens = torch.tensor([T], dtype=torch.int32, device=DEV)
    o_d, lse_d = run_decode(q[:, :, T - 1].contiguous(), k, v, lens, params)
    assert (o_d.float() - o_f[:, :, T - 1].float()).abs().max().item() <= 2e-2
    assert (lse_d - lse_f[:, :, T - 1]).abs().max().item() <= 1e-3


# ------------------------------------------------------------------ multi-token and paged decode

def multi_case(B, Nq, Tmax, Hq, Hkv, D, sink, local, lens, page_size=None, full_attn=False, seed=62):
    """The Nq newest tokens of every sequence against the oracle's forward with N_q = Nq, N_k = lens[b]."""
    q = cowa_inputs.make_train_inputs(seed, B, Nq, Hq, Hkv, D)[0].permute(0, 2, 1, 3).contiguous()  # [B,Nq,Hq,D]
    _, kc, vc, _ = cowa_inputs.make_decode_inputs(seed + 1, B, Tmax, Hq, Hkv, D, Tmax, Tmax)
    lens_t = torch.tensor(lens, dtype=torch.int32)
    for b in range(B):
        kc[b, :, lens[b]:] = float("nan")
        vc[b, :, lens[b]:] = float("nan")
    scale = cowa_inputs.softmax_scale(D)
    params = cowa.make_params(sink=sink, local=local, softmax_scale=scale, full_attn=full_attn)
    o = torch.full_like(q, float("nan")).to(DEV)
    lse = torch.full((B, Nq, Hq), float("nan"), dtype=torch.float32, device=DEV)
    if page_size is None:
        nbytes = cowa.cowa_decode_multi_workspace_bytes(B, Nq, Tmax, Hq, Hkv, D, params)
        ws = torch.empty(nbytes + 64, dtype=torch.uint8, device=DEV)
        ws.fill_(0xFF)
        cowa.cowa_decode_multi(q.to(DEV), kc.to(DEV), vc.to(DEV), lens_t.to(DEV), o, lse, params, ws[:nbytes])
    else:
        max_pages = (Tmax + page_size - 1) // page_size
        num_pages = B * max_pages + 5
        g = torch.Generator().manual_seed(seed)
        perm = torch.randperm(num_pages, generator=g)
        table = torch.full((B, max_pages), -1, dtype=torch.int32)
        kp = torch.full((num_pages, Hkv, page_size, D), float("nan"), dtype=torch.bfloat16)
        vp = torch.full_like(kp, float("nan"))
        n = 0
        for b in range(B):
            for i in range((lens[b] + page_size - 1) // page_size):  # pages past the sequence stay unmapped
                pg = int(perm[n]); n += 1
                table[b, i] = pg
                rows = min(page_size, Tmax - i * page_size)
                kp[pg, :, :rows] = kc[b, :, i * page_size:i * page_size + rows]
                vp[pg, :, :rows] = vc[b, :, i * page_size:i * page_size + rows]
        nbytes = cowa.cowa_decode_multi_workspace_bytes(B, Nq, max_pages * page_size, Hq, Hkv, D, params)
        ws = torch.empty(nbytes + 64, dtype=torch.uint8, device=DEV)
        ws.fill_(0xFF)
        cowa.cowa_decode_paged(q.to(DEV), kp.to(DEV), vp.to(DEV), table.to(DEV), lens_t.to(DEV), o, lse, params,
                               ws[:nbytes])
    torch.cuda.synchronize()
    cowa.cowa_check_device_status()
    assert (ws[nbytes:] == 0xFF).all(), "decode wrote past its workspace"
    f = cowa_inputs.to_f64
    for b in range(B):
        n = lens[b]
        ws_ = [(0, n, 0, 0)] * Hkv if full_attn else orc.default_windows(n, Hkv, sink, local)
        o_ref, lse_ref = orc.forward(f(q[b].permute(1, 0, 2)), f(kc[b, :, :n]), f(vc[b, :, :n]), ws_, scale)
        check(f"multi lse[b={b}]", lse[b].permute(1, 0).cpu().numpy(), lse_ref, TOL_LSE, TOL_LSE)
        check(f"multi o[b={b}]", o[b].permute(1, 0, 2).float().cpu().numpy(), o_ref)


@pytest.mark.parametrize("B,Nq,Tmax,Hq,Hkv,D,sink,local,lens", [
    (2, 2, 5000, 8, 2, 128, 16, 100, [5000, 2777]),        # G = 4: both tokens share one pass
    (2, 5, 3000, 8, 2, 128, 16, 100, [3000, 5]),           # three token groups, the last half empty; len = Nq
    (2, 8, 3001, 4, 4, 64, 4, 31, [3001, 17]),             # G = 1: eight tokens in one pass, D = 64
    (1, 3, 4096, 16, 2, 128, 128, 512, [4096]),            # G = 8: one token per block
    (3, 3, 2000, 4, 2, 128, 7, 50, [2000, 640, 57]),       # G = 2, odd token count; a dense short sequence
    (1, 4, 40000, 4, 2, 128, 128, 4096, [39999]),          # several splits per head
    (1, 1, 2500, 8, 2, 128, 16, 100, [2400]),              # Nq = 1 through the extended kernel
])
def test_decode_multi_shapes(B, Nq, Tmax, Hq, Hkv, D, sink, local, lens):
    multi_case(B, Nq, Tmax, Hq, Hkv, D, sink, local, lens)


def test_decode_multi_full_attn():
    multi_case(2, 4, 6000, 8, 2, 128, 0, 1, [6000, 4321], full_attn=True)


@pytest.mark.parametrize("B,Nq,Tmax,Hq,Hkv,D,sink,local,lens,page", [
    (3, 1, 5000, 8, 2, 128, 16, 100, [5000, 1, 2777], 16),
    (2, 4, 4100, 8, 4, 128, 32, 200, [4100, 999], 64),
    (2, 2, 8192, 16, 2, 64, 128, 512, [8192, 640], 256),
    (1, 1, 40000, 4, 2, 128, 128, 4096, [39999], 128),
    (2, 3, 3000, 4, 2, 128, 16, 100, [3000, 1111], 48),    # page size not a power of two
])
def test_decode_paged_shapes(B, Nq, Tmax, Hq, Hkv, D, sink, local, lens, page):
    multi_case(B, Nq, Tmax, Hq, Hkv, D, sink, local, lens, page_size=page)


def test_decode_multi_last_token_equals_single_token_decode():
    # the newest of the Nq tokens is the token cowa_decode computes for the same cache
    B, Nq, Tmax, Hq, Hkv, D = 2, 4, 3000, 8, 2, 128
    q = cowa_inputs.make_train_inputs(64, B, Nq, Hq, Hkv, D, device=DEV)[0].permute(0, 2, 1, 3).contiguous()
    _, kc, vc, _ = cowa_inputs.make_decode_inputs(65, B, Tmax, Hq, Hkv, D, Tmax, Tmax, device=DEV)
    lens = torch.tensor([3000, 1234], dtype=torch.int32, device=DEV)
    params = cowa.make_params(sink=16, local=128, softmax_scale=cowa_inputs.softmax_scale(D))
    o = torch.empty_like(q)
    lse = torch.empty((B, Nq, Hq), dtype=torch.float32, device=DEV)
    ws = torch.empty(cowa.cowa_decode_multi_workspace_bytes(B, Nq, Tmax, Hq, Hkv, D, params), dtype=torch.uint8,
                     device=DEV)
    cowa.cowa_decode_multi(q, kc, vc, lens, o, lse, params, ws)
    o1, lse1 = run_decode(q[:, Nq - 1].contiguous(), kc, vc, lens, params)
    assert (o[:, Nq - 1].float() - o1.float()).abs().max().item() <= 1e-2
    assert (lse[:, Nq - 1] - lse1).abs().max().item() <= 1e-4


# ------------------------------------------------------------------ seeded random shapes

def _random_tuples(rng, T, Hkv):
    """Explicit per-head tuples with arbitrary sinks, gaps and widths (possibly overlapping, possibly beyond T)."""
    return [(int(rng.integers(0, 200)), int(rng.integers(1, 300)), int(rng.integers(0, T)), int(rng.integers(0, T)))
            for _ in range(Hkv)]


@pytest.mark.parametrize("case", range(24))
def test_random_shapes(case):
    """Forward, backward and decode on shapes drawn from a fixed seed: odd lengths, every supported group size,
    default rule and arbitrary explicit tuples."""
    rng = np.random.default_rng(1000 + case)
    D = int(rng.choice([64, 128]))
    Hkv = int(rng.choice([1, 2, 3, 4]))
    G = int(rng.choice([1, 2, 4, 8]))
    Hq = Hkv * G
    B = int(rng.integers(1, 3))
    T = int(rng.integers(1, 1400))
    sink, local = int(rng.integers(0, 150)), int(rng.integers(1, 400))
    windows = _random_tuples(rng, T, Hkv) if case % 3 == 2 else None
    fwd_case(B, T, Hq, Hkv, D, sink, local, seed=300 + case, windows=windows)
    bwd_case(B, T, Hq, Hkv, D, sink, local, seed=300 + case, windows=windows)
    lens = [int(rng.integers(1, T + 1)) for _ in range(B)]
    decode_case(B, T, Hq, Hkv, D, sink, local, lens, seed=400 + case)
    nq = int(rng.integers(1, 6))
    multi_case(B, nq, T + nq, Hq, Hkv, D, sink, local, [n + nq - 1 for n in lens], seed=500 + case,
               page_size=(16 * int(rng.integers(1, 9)) if case % 2 else None))


@pytest.mark.parametrize("case", range(6))
def test_random_packed_batches(case):
    """Packed forward (N_q <= N_k per sequence) and packed backward (N_q = N_k) on random length mixes."""
    rng = np.random.default_rng(2000 + case)
    D = int(rng.choice([64, 128]))
    Hkv = int(rng.choice([1, 2, 4]))
    Hq = Hkv * int(rng.choice([1, 2, 4]))
    sink, local = int(rng.integers(0, 100)), int(rng.integers(1, 300))
    nseq = int(rng.integers(1, 7))
    seqs = []
    for _ in range(nseq):
        nk = int(rng.integers(1, 900))
        seqs.append((int(rng.integers(0, nk + 1)), nk))
    if all(nq == 0 for nq, _ in seqs):
        seqs[0] = (seqs[0][1], seqs[0][1])
    scale = cowa_inputs.softmax_scale(D)
    params = cowa.make_params(sink=sink, local=local, softmax_scale=scale)
    q, k, v, cu_q, cu_k = _packed_inputs(600 + 20 * case, seqs, Hq, Hkv, D)
    o, lse = _run_varlen(q, k, v, cu_q, cu_k, params)
    cowa.cowa_check_device_status()
    f = cowa_inputs.to_f64
    for b, (nq, nk) in enumerate(seqs):
        if nq == 0:
            continue
        qs, ks = slice(cu_q[b], cu_q[b + 1]), slice(cu_k[b], cu_k[b + 1])
        o_ref, lse_ref = orc.forward(f(q[:, qs]), f(k[:, ks]), f(v[:, ks]), orc.default_windows(nk, Hkv, sink, local), scale)
        check(f"packed lse[seq {b}]", lse[:, qs].cpu().numpy(), lse_ref, TOL_LSE, TOL_LSE)
        check(f"packed o[seq {b}]", o[:, qs].float().cpu().numpy(), o_ref)
    # backward on the same key lengths with N_q = N_k
    lens = [nk for _, nk in seqs]
    q, k, v, cu, _ = _packed_inputs(700 + 20 * case, [(n, n) for n in lens], Hq, Hkv, D)
    d_o = torch.cat([cowa_inputs.make_train_inputs(800 + b, 1, n, Hq, Hkv, D)[3][0] for b, n in enumerate(lens)], 1).contiguous()
    o, lse = _run_varlen(q, k, v, cu, cu, params)
    qd, kd, vd, dod = q.to(DEV), k.to(DEV), v.to(DEV), d_o.to(DEV)
    dq, dk, dv = (torch.full_like(x, float("nan")) for x in (qd, kd, vd))
    ws = torch.empty(cowa.cowa_bwd_varlen_workspace_bytes(len(lens), int(cu[-1]), Hq, Hkv, D, params), dtype=torch.uint8,
                     device=DEV)
    cowa.cowa_bwd_varlen(qd, kd, vd, o, lse, dod, dq, dk, dv, torch.from_numpy(cu).to(DEV), params, ws)
    torch.cuda.synchronize()
    cowa.cowa_check_device_status()
    for b, n in enumerate(lens):
        sl = slice(cu[b], cu[b + 1])
        dq_r, dk_r, dv_r = orc.backward(f(q[:, sl]), f(k[:, sl]), f(v[:, sl]), f(d_o[:, sl]),
                                        orc.default_windows(n, Hkv, sink, local), scale)
        check_grad(f"packed dq[seq {b}]", dq[:, sl].float().cpu().numpy(), dq_r)
        check_grad(f"packed dk[seq {b}]", dk[:, sl].float().cpu().numpy(), dk_r)
        check_grad(f"packed dv[seq {b}]", dv[:, sl].float().cpu().numpy(), dv_r)


# ------------------------------------------------------------------ CUDA graphs

def test_calls_replay_from_a_cuda_graph():
    """The library's launches (kernels, the accumulator memset, the programmatic dependent launch of the decode
    merge) can be captured into a CUDA graph after one warm-up call, and the replay reproduces the direct
    call bit for bit on new inputs written into the same buffers."""
    B, T, Hq, Hkv, D = 2, 1536, 8, 2, 128
    params = cowa.make_params(sink=16, local=128, softmax_scale=cowa_inputs.softmax_scale(D), deterministic=True)
    q, k, v, d_o = cowa_inputs.make_train_inputs(91, B, T, Hq, Hkv, D, device=DEV)
    o = torch.empty_like(q)
    lse = torch.empty((B, Hq, T), dtype=torch.float32, device=DEV)
    dq, dk, dv = (torch.empty_like(x) for x in (q, k, v))
    ws = torch.empty(cowa.cowa_bwd_workspace_bytes(B, T, Hq, Hkv, D, params), dtype=torch.uint8, device=DEV)
    qd = q[:, :, -1].contiguous()
    od = torch.empty_like(qd)
    lsed = torch.empty((B, Hq), dtype=torch.float32, device=DEV)
    lens = torch.tensor([T, T - 300], dtype=torch.int32, device=DEV)
    wsd = torch.empty(cowa.cowa_decode_workspace_bytes(B, T, Hq, Hkv, D, params), dtype=torch.uint8, device=DEV)

    def step():
        cowa.cowa_fwd(q, k, v, o, lse, params)
        cowa.cowa_bwd(q, k, v, o, lse, d_o, dq, dk, dv, params, ws)
        cowa.cowa_decode(qd, k, v, lens, od, lsed, params, wsd)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        step()                                   # warm-up outside the capture
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, stream=side):
            step()
    torch.cuda.synchronize()
    # new inputs in place, then direct call vs replay
    q2, k2, v2, d_o2 = cowa_inputs.make_train_inputs(92, B, T, Hq, Hkv, D, device=DEV)
    q.copy_(q2); k.copy_(k2); v.copy_(v2); d_o.copy_(d_o2); qd.copy_(q2[:, :, -1])
    step()
    torch.cuda.synchronize()
    want = [x.clone() for x in (o, lse, dq, dk, dv, od, lsed)]
    for x in (o, lse, dq, dk, dv, od, lsed):
        x.zero_()
    graph.replay()
    torch.cuda.synchronize()
    cowa.cowa_check_device_status()
    for name, a_, b_ in zip(("o", "lse", "dq", "dk", "dv", "o_decode", "lse_decode"), (o, lse, dq, dk, dv, od, lsed), want):
        assert torch.equal(a_, b_), name
