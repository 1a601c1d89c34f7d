"""cowa_decode_static: the decode entry point for callers that cannot allocate device memory
(allocation-free serving loops, plugins whose host owns device memory).  It must give what
cowa_decode gives, on back-to-back calls that share the library's built-in scratch array, and
must refuse calls that would not fit that array.  Collected last on purpose: a run that stops
at the first failure has then already run every other test."""
import ctypes as C

import pytest
import torch

import cowa_inputs
import paper_2609_32704_b200 as cowa
from oracle import cowa_oracle as orc

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _inputs(seed, B, Tmax, Hq, Hkv, D, lens):
    q, kc, vc, _ = cowa_inputs.make_decode_inputs(seed, B, Tmax, Hq, Hkv, D, Tmax, Tmax)
    lens = torch.tensor(lens, dtype=torch.int32)
    for b in range(B):
        kc[b, :, int(lens[b]):] = float("nan")
        vc[b, :, int(lens[b]):] = float("nan")
    return q.to(DEV), kc.to(DEV), vc.to(DEV), lens.to(DEV)


def _reference(q, kc, vc, lens, params):
    B, Hq, D = q.shape
    o = torch.empty_like(q)
    lse = torch.empty((B, Hq), dtype=torch.float32, device=DEV)
    ws = torch.empty(cowa.cowa_decode_workspace_bytes(B, kc.shape[2], Hq, kc.shape[1], D, params),
                     dtype=torch.uint8, device=DEV)
    cowa.cowa_decode(q, kc, vc, lens, o, lse, params, ws)
    torch.cuda.synchronize()
    return o, lse


def test_decode_static_matches_decode_on_two_calls_in_a_row():
    # two different problems, so the second call meets the first call's leftovers in the array
    cases = [
        (71, 3, 6000, 8, 2, 128, 16, 200, [6000, 1, 3333]),
        (72, 2, 2500, 8, 8, 64, 4, 50, [2500, 999]),
    ]
    prepared, oracle_out = [], []
    for seed, B, Tmax, Hq, Hkv, D, sink, local, lens in cases:
        params = cowa.make_params(sink=sink, local=local, softmax_scale=cowa_inputs.softmax_scale(D))
        t = _inputs(seed, B, Tmax, Hq, Hkv, D, lens)
        prepared.append((t, params, _reference(*t, params)))
        q, kc, vc, ln = (x.cpu() for x in t)
        oracle_out.append(orc.decode(cowa_inputs.to_f64(q), kc.float().numpy(), vc.float().numpy(), ln.numpy(),
                                     sink, local, cowa_inputs.softmax_scale(D)))
    outs = []
    for (q, kc, vc, lens), params, _ in prepared:  # back to back on one stream, no sync between
        o = torch.full_like(q, float("nan"))
        lse = torch.full((q.shape[0], q.shape[1]), float("nan"), dtype=torch.float32, device=DEV)
        cowa.cowa_decode_static(q, kc, vc, lens, o, lse, params)
        outs.append((o, lse))
    torch.cuda.synchronize()
    for (o, lse), (_, _, (o_ref, lse_ref)), (o_orc, lse_orc) in zip(outs, prepared, oracle_out):
        assert torch.isfinite(o.float()).all() and torch.isfinite(lse).all()
        assert (o.float() - o_ref.float()).abs().max().item() <= 2e-2
        assert (lse - lse_ref).abs().max().item() <= 1e-3
        # and against the float64 oracle, like every other decode test
        assert abs(o.float().cpu().numpy() - o_orc).max() <= 2e-2
        assert abs(lse.cpu().numpy() - lse_orc).max() <= 1e-3


def test_decode_static_rejects_oversized_calls():
    cap = cowa.cowa_decode_static_capacity()
    assert cap == 8 << 20
    B, Tmax, Hq, Hkv, D = 64, 131072, 64, 8, 128
    params = cowa.make_params(sink=128, local=4096, softmax_scale=1.0)
    assert cowa.cowa_decode_workspace_bytes(B, Tmax, Hq, Hkv, D, params) > cap
    # validation happens before any launch, so small stand-in buffers are never dereferenced
    dummy = torch.zeros(64, dtype=torch.bfloat16, device=DEV)
    lens = torch.ones(B, dtype=torch.int32, device=DEV)
    rc = cowa.lib().cowa_decode_static(C.c_void_p(dummy.data_ptr()), C.c_void_p(dummy.data_ptr()),
                                       C.c_void_p(dummy.data_ptr()), C.c_void_p(lens.data_ptr()),
                                       C.c_void_p(dummy.data_ptr()), None, B, Tmax, Hq, Hkv, D,
                                       C.byref(params), None)
    assert rc == -7
    assert "scratch" in cowa.cowa_status_string(rc)
