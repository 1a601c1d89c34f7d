"""GPU tests of the boundary's layout and status handling: q/k/v/o passed with explicit (batch, head, token)
strides (no copies), the device status word's three flags, and the calls that refuse strides.  Results are
compared with the float64 oracle on the same seeded inputs, through the C ABI."""
import ctypes as C

import numpy as np
import pytest
import torch

import cowa_inputs
import paper_2609_32704_b200 as cowa
from oracle import cowa_oracle as orc

pytestmark = pytest.mark.gpu
DEV = "cuda"
TOL_MAX, TOL_MEAN, TOL_LSE = 2e-2, 2e-3, 1e-3
BF16_HALF_ULP = 2.0 ** -8


def _check(name, got, want, tol_max=TOL_MAX, tol_mean=TOL_MEAN, grad=False):
    got = np.asarray(got, dtype=np.float64)
    assert np.isfinite(got).all(), f"{name}: non-finite output"
    err = np.abs(got - want)
    rtol, rtol_mean = (BF16_HALF_ULP, BF16_HALF_ULP / 4) if grad else (0.0, 0.0)
    assert (err - rtol * np.abs(want)).max() <= tol_max, f"{name}: max-abs {err.max():.3e}"
    assert err.mean() <= tol_mean + rtol_mean * np.abs(want).mean(), f"{name}: mean-abs {err.mean():.3e}"


def _bthd(x):
    """The same values stored token-major: a [B,T,H,D] buffer viewed as [B,H,T,D] (what a fused QKV projection
    hands over); the view shares no layout with the contiguous head-major tensor."""
    return x.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)


@pytest.mark.parametrize("B,T,Hq,Hkv,D,sink,local", [
    (2, 700, 8, 2, 128, 16, 100),   # ragged tail, G = 4
    (1, 1030, 4, 4, 64, 5, 60),     # D = 64, G = 1
])
def test_fwd_bwd_token_major_layout(B, T, Hq, Hkv, D, sink, local):
    q, k, v, d_o = cowa_inputs.make_train_inputs(95, B, T, Hq, Hkv, D)
    scale = cowa_inputs.softmax_scale(D)
    params = cowa.make_params(sink=sink, local=local, softmax_scale=scale)
    qs, ks, vs, dos = (_bthd(x.to(DEV)) for x in (q, k, v, d_o))
    assert not qs.is_contiguous() and qs.stride(1) == D and qs.stride(2) == Hq * D
    guard = float("nan")
    o = _bthd(torch.full((B, Hq, T, D), guard, dtype=torch.bfloat16, device=DEV))
    lse = torch.full((B, Hq, T), guard, dtype=torch.float32, device=DEV)
    cowa.cowa_fwd(qs, ks, vs, o, lse, params)
    dq, dk, dv = (_bthd(torch.full_like(x, guard).to(DEV)) for x in (q, k, v))
    ws = torch.empty(cowa.cowa_bwd_workspace_bytes(B, T, Hq, Hkv, D, params), dtype=torch.uint8, device=DEV)
    cowa.cowa_bwd(qs, ks, vs, o, lse, dos, dq, dk, dv, params, ws)
    torch.cuda.synchronize()
    cowa.cowa_check_device_status()
    wins = orc.default_windows(T, Hkv, sink, local)
    f = cowa_inputs.to_f64
    for b in range(B):
        o_ref, lse_ref = orc.forward(f(q[b]), f(k[b]), f(v[b]), wins, scale)
        _check(f"strided lse[{b}]", lse[b].cpu().numpy(), lse_ref, TOL_LSE, TOL_LSE)
        _check(f"strided o[{b}]", o[b].float().cpu().numpy(), o_ref)
        dq_r, dk_r, dv_r = orc.backward(f(q[b]), f(k[b]), f(v[b]), f(d_o[b]), wins, scale)
        _check(f"strided dq[{b}]", dq[b].float().cpu().numpy(), dq_r, grad=True)
        _check(f"strided dk[{b}]", dk[b].float().cpu().numpy(), dk_r, grad=True)
        _check(f"strided dv[{b}]", dv[b].float().cpu().numpy(), dv_r, grad=True)
    # the strided call and the contiguous call run the same arithmetic: O and LSE agree bit for bit
    o2 = torch.empty((B, Hq, T, D), dtype=torch.bfloat16, device=DEV)
    lse2 = torch.empty_like(lse)
    cowa.cowa_fwd(q.to(DEV), k.to(DEV), v.to(DEV), o2, lse2, params)
    torch.cuda.synchronize()
    assert torch.equal(o2, o) and torch.equal(lse2, lse)


def test_bwd_token_major_layout_with_split_groups():
    """Few KV tiles: the group's heads are spread over several blocks and a last kernel adds their partial
    dK, dV; that kernel writes through the strides too."""
    B, T, Hq, Hkv, D, sink, local = 1, 1500, 8, 1, 128, 40, 200
    q, k, v, d_o = cowa_inputs.make_train_inputs(96, B, T, Hq, Hkv, D)
    scale = cowa_inputs.softmax_scale(D)
    params = cowa.make_params(sink=sink, local=local, softmax_scale=scale)
    assert cowa.cowa_bwd_workspace_bytes(B, T, Hq, Hkv, D, params) > B * Hq * ((T + 63) // 64 * 64) * (D + 2) * 4
    qs, ks, vs, dos = (_bthd(x.to(DEV)) for x in (q, k, v, d_o))
    o = _bthd(torch.empty((B, Hq, T, D), dtype=torch.bfloat16, device=DEV))
    lse = torch.empty((B, Hq, T), dtype=torch.float32, device=DEV)
    cowa.cowa_fwd(qs, ks, vs, o, lse, params)
    dq, dk, dv = (_bthd(torch.full_like(x, float("nan")).to(DEV)) for x in (q, k, v))
    ws = torch.empty(cowa.cowa_bwd_workspace_bytes(B, T, Hq, Hkv, D, params), dtype=torch.uint8, device=DEV)
    cowa.cowa_bwd(qs, ks, vs, o, lse, dos, dq, dk, dv, params, ws)
    torch.cuda.synchronize()
    cowa.cowa_check_device_status()
    f = cowa_inputs.to_f64
    dq_r, dk_r, dv_r = orc.backward(f(q[0]), f(k[0]), f(v[0]), f(d_o[0]), orc.default_windows(T, Hkv, sink, local), scale)
    _check("split dq", dq[0].float().cpu().numpy(), dq_r, grad=True)
    _check("split dk", dk[0].float().cpu().numpy(), dk_r, grad=True)
    _check("split dv", dv[0].float().cpu().numpy(), dv_r, grad=True)


def test_decode_token_major_cache_and_sliced_cache():
    """A [B,Tmax,Hkv,D] cache, and a cache that is a slice (every other head) of a larger buffer."""
    B, Tmax, Hq, Hkv, D, sink, local = 3, 3000, 8, 2, 128, 16, 100
    lens = [3000, 1, 1777]
    q, kc, vc, _ = cowa_inputs.make_decode_inputs(97, B, Tmax, Hq, Hkv, D, Tmax, Tmax)
    lens_t = torch.tensor(lens, dtype=torch.int32)
    for b in range(B):
        kc[b, :, lens[b]:] = float("nan")
        vc[b, :, lens[b]:] = float("nan")
    scale = cowa_inputs.softmax_scale(D)
    params = cowa.make_params(sink=sink, local=local, softmax_scale=scale)
    o_ref, lse_ref = orc.decode(cowa_inputs.to_f64(q), kc.float().numpy(), vc.float().numpy(), np.asarray(lens),
                                sink, local, scale)
    wide_k = torch.full((B, 2 * Hkv, Tmax, D), float("nan"), dtype=torch.bfloat16, device=DEV)
    wide_v = torch.full_like(wide_k, float("nan"))
    wide_k[:, ::2] = kc.to(DEV)
    wide_v[:, ::2] = vc.to(DEV)
    for name, kk, vv in (("token-major", _bthd(kc.to(DEV)), _bthd(vc.to(DEV))),
                         ("sliced", wide_k[:, ::2], wide_v[:, ::2])):
        assert not kk.is_contiguous()
        o = torch.full((B, Hq, D), float("nan"), dtype=torch.bfloat16, device=DEV)
        lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=DEV)
        ws = torch.empty(cowa.cowa_decode_workspace_bytes(B, Tmax, Hq, Hkv, D, params), dtype=torch.uint8, device=DEV)
        cowa.cowa_decode(q.to(DEV), kk, vv, lens_t.to(DEV), o, lse, params, ws)
        torch.cuda.synchronize()
        _check(f"{name} decode lse", lse.cpu().numpy(), lse_ref, TOL_LSE, TOL_LSE)
        _check(f"{name} decode o", o.float().cpu().numpy(), o_ref)


def test_strides_are_validated():
    B, T, Hq, Hkv, D = 1, 256, 2, 1, 128
    q, k, v, _ = cowa_inputs.make_train_inputs(98, B, T, Hq, Hkv, D, device=DEV)
    o = torch.empty_like(q)
    lse = torch.empty((B, Hq, T), dtype=torch.float32, device=DEV)
    vp = lambda t: C.c_void_p(t.data_ptr())
    call = lambda p: cowa.lib().cowa_fwd(vp(q), vp(k), vp(v), vp(o), vp(lse), B, T, Hq, Hkv, D, C.byref(p), None)
    p = cowa.make_params(sink=4, local=32, softmax_scale=0.1)
    p.q_strides[:] = [Hq * T * D, T * D, D + 4]      # token stride not a multiple of 8 elements
    assert call(p) == -3
    p.q_strides[:] = [Hq * T * D, T * D, D - 8]      # rows would overlap
    assert call(p) == -1
    p.q_strides[:] = [Hq * T * D, T * D, D]          # the contiguous strides spelled out: accepted
    assert call(p) == 0
    torch.cuda.synchronize()
    # the packed, multi-token and paged calls take contiguous tensors only
    cu = torch.tensor([0, T], dtype=torch.int32, device=DEV)
    rc = cowa.lib().cowa_prefill_varlen(vp(q), vp(k), vp(v), vp(o), vp(lse), vp(cu), vp(cu), 1, T, T, Hq, Hkv, D,
                                        C.byref(p), None)
    assert rc == -2
    lens = torch.tensor([T], dtype=torch.int32, device=DEV)
    pm = cowa.make_params(sink=4, local=32, softmax_scale=0.1)
    ws = torch.empty(cowa.cowa_decode_multi_workspace_bytes(1, 2, T, Hq, Hkv, D, pm), dtype=torch.uint8, device=DEV)
    pm.k_strides[:] = [Hkv * T * D, T * D, D]
    rc = cowa.lib().cowa_decode_multi(vp(q), vp(k), vp(v), vp(lens), vp(o), None, 1, 2, T, Hq, Hkv, D, C.byref(pm),
                                      vp(ws), ws.numel(), None)
    assert rc == -2


def test_bounded_wait_gives_up_and_is_reported_once():
    """A device-side wait that nothing satisfies must run out, set the status flag and let the kernel end; the
    context stays usable and the flag is cleared by the call that reports it."""
    cowa.cowa_check_device_status()            # start clean
    cowa.cowa_selftest_bounded_wait(1 << 20)   # about a millisecond of waiting
    with pytest.raises(cowa.CowaError) as e:
        cowa.cowa_check_device_status()
    assert e.value.status == -6 and "wait" in str(e.value)
    cowa.cowa_check_device_status()            # reported once
    # the library still works afterwards
    q, k, v, _ = cowa_inputs.make_train_inputs(99, 1, 128, 1, 1, 64, device=DEV)
    o = torch.empty_like(q)
    lse = torch.empty((1, 1, 128), dtype=torch.float32, device=DEV)
    cowa.cowa_fwd(q, k, v, o, lse, cowa.make_params(sink=0, local=128, softmax_scale=0.125))
    torch.cuda.synchronize()
    cowa.cowa_check_device_status()
    assert torch.isfinite(o.float()).all()


def test_deterministic_dq_out_of_range_is_reported():
    """deterministic = 1 adds dQ partial sums as 2^-18 fixed point, good for |dQ| < 8192; values beyond that are
    flagged instead of wrapping silently."""
    B, T, Hq, Hkv, D = 1, 256, 2, 1, 64
    q, k, v, d_o = cowa_inputs.make_train_inputs(100, B, T, Hq, Hkv, D, device=DEV)
    scale = cowa_inputs.softmax_scale(D)
    params = cowa.make_params(sink=8, local=64, softmax_scale=scale, deterministic=True)
    o = torch.empty_like(q)
    lse = torch.empty((B, Hq, T), dtype=torch.float32, device=DEV)
    cowa.cowa_fwd(q, k, v, o, lse, params)
    dq, dk, dv = (torch.empty_like(x) for x in (q, k, v))
    ws = torch.empty(cowa.cowa_bwd_workspace_bytes(B, T, Hq, Hkv, D, params), dtype=torch.uint8, device=DEV)
    cowa.cowa_bwd(q, k, v, o, lse, d_o, dq, dk, dv, params, ws)
    torch.cuda.synchronize()
    cowa.cowa_check_device_status()            # ordinary magnitudes: no flag
    cowa.cowa_bwd(q, k, v, o, lse, d_o * 3.0e4, dq, dk, dv, params, ws)   # gradients ~1e5
    torch.cuda.synchronize()
    with pytest.raises(cowa.CowaError) as e:
        cowa.cowa_check_device_status()
    assert e.value.status == -9
    cowa.cowa_check_device_status()


def test_prefill_and_its_backward_on_strided_views():
    """N_q < N_k (a chunk appended to a cache) with q/o token-major and k/v slices of a wider cache buffer."""
    B, Nq, Nk, Hq, Hkv, D, sink, local = 2, 200, 900, 8, 2, 128, 8, 90
    q, _, _, d_o = cowa_inputs.make_train_inputs(101, B, Nq, Hq, Hkv, D)
    _, k, v, _ = cowa_inputs.make_train_inputs(102, B, Nk, Hq, Hkv, D)
    scale = cowa_inputs.softmax_scale(D)
    params = cowa.make_params(sink=sink, local=local, softmax_scale=scale)
    qs, dos = _bthd(q.to(DEV)), _bthd(d_o.to(DEV))
    wide_k = torch.full((B, Hkv, Nk + 56, D), float("nan"), dtype=torch.bfloat16, device=DEV)
    wide_v = torch.full_like(wide_k, float("nan"))
    ks, vs = wide_k[:, :, 24:24 + Nk], wide_v[:, :, 24:24 + Nk]   # 16-byte aligned start, batch / head strides of the wide buffer
    ks.copy_(k.to(DEV)); vs.copy_(v.to(DEV))
    assert not ks.is_contiguous()
    o = _bthd(torch.full((B, Hq, Nq, D), float("nan"), dtype=torch.bfloat16, device=DEV))
    lse = torch.full((B, Hq, Nq), float("nan"), dtype=torch.float32, device=DEV)
    cowa.cowa_prefill(qs, ks, vs, o, lse, params)
    dq = _bthd(torch.full((B, Hq, Nq, D), float("nan"), dtype=torch.bfloat16, device=DEV))
    wide_dk, wide_dv = torch.zeros_like(wide_k), torch.zeros_like(wide_v)
    dk, dv = wide_dk[:, :, 24:24 + Nk], wide_dv[:, :, 24:24 + Nk]
    ws = torch.empty(cowa.cowa_bwd_prefill_workspace_bytes(B, Nq, Nk, Hq, Hkv, D, params), dtype=torch.uint8, device=DEV)
    cowa.cowa_bwd_prefill(qs, ks, vs, o, lse, dos, dq, dk, dv, params, ws)
    torch.cuda.synchronize()
    cowa.cowa_check_device_status()
    # nothing outside the slices was written
    assert (wide_dk[:, :, :24] == 0).all() and (wide_dk[:, :, 24 + Nk:] == 0).all()
    assert (wide_dv[:, :, :24] == 0).all() and (wide_dv[:, :, 24 + Nk:] == 0).all()
    wins = orc.default_windows(Nk, Hkv, sink, local)
    f = cowa_inputs.to_f64
    for b in range(B):
        o_ref, lse_ref = orc.forward(f(q[b]), f(k[b]), f(v[b]), wins, scale)
        _check(f"prefill lse[{b}]", lse[b].cpu().numpy(), lse_ref, TOL_LSE, TOL_LSE)
        _check(f"prefill o[{b}]", o[b].float().cpu().numpy(), o_ref)
        dq_r, dk_r, dv_r = orc.backward(f(q[b]), f(k[b]), f(v[b]), f(d_o[b]), wins, scale)
        _check(f"prefill dq[{b}]", dq[b].float().cpu().numpy(), dq_r, grad=True)
        _check(f"prefill dk[{b}]", dk[b].float().cpu().numpy(), dk_r, grad=True)
        _check(f"prefill dv[{b}]", dv[b].float().cpu().numpy(), dv_r, grad=True)
