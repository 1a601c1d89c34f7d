"""ctypes binding of include/cowa.h.  Function names equal the C entry points.

The shared library must have been built (python -m paper_2609_32704_b200.build or
__graft_entry__.build()); there is no fallback when it is missing.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
lib_path = os.path.join(_HERE, "libcowa.so")

SCHED_FWD, SCHED_BWD, SCHED_DECODE = 0, 1, 2


class CowaError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        msg = lib().cowa_status_string(status).decode()
        extra = f" (cudaError {lib().cowa_last_cuda_error()})" if status == -5 else ""
        super().__init__(f"{where}: {msg}{extra} [{status}]")


class Window(C.Structure):
    _fields_ = [("sink", C.c_int32), ("near", C.c_int32), ("gap", C.c_int32), ("len", C.c_int32)]


class Params(C.Structure):
    _fields_ = [
        ("sink", C.c_int32), ("local", C.c_int32), ("block_q", C.c_int32), ("block_k", C.c_int32),
        ("hkv_global", C.c_int32), ("hkv_offset", C.c_int32), ("windows", C.POINTER(Window)),
        ("full_attn", C.c_int32), ("softmax_scale", C.c_float), ("deterministic", C.c_int32),
        ("q_strides", C.c_int64 * 3), ("k_strides", C.c_int64 * 3), ("v_strides", C.c_int64 * 3),
        ("o_strides", C.c_int64 * 3),
        ("bwd_main_start_event", C.c_void_p), ("bwd_main_stop_event", C.c_void_p),
    ]


_lib = None


def lib():
    """The loaded C library (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(lib_path):
            raise ImportError(f"{lib_path} not found: build it with `python -m paper_2609_32704_b200.build`")
        L = C.CDLL(lib_path)
        vp, i32, sz = C.c_void_p, C.c_int, C.c_size_t
        pp = C.POINTER(Params)
        L.cowa_fwd.argtypes = [vp] * 5 + [i32] * 5 + [pp, vp]
        L.cowa_fwd.restype = i32
        L.cowa_prefill.argtypes = [vp] * 5 + [i32] * 6 + [pp, vp]
        L.cowa_prefill.restype = i32
        L.cowa_prefill_varlen.argtypes = [vp] * 7 + [i32] * 6 + [pp, vp]
        L.cowa_prefill_varlen.restype = i32
        L.cowa_bwd.argtypes = [vp] * 9 + [i32] * 5 + [pp, vp, sz, vp]
        L.cowa_bwd.restype = i32
        L.cowa_bwd_prefill.argtypes = [vp] * 9 + [i32] * 6 + [pp, vp, sz, vp]
        L.cowa_bwd_prefill.restype = i32
        L.cowa_bwd_prefill_workspace_bytes.argtypes = [i32] * 6 + [pp]
        L.cowa_bwd_prefill_workspace_bytes.restype = sz
        L.cowa_bwd_varlen.argtypes = [vp] * 10 + [i32] * 5 + [pp, vp, sz, vp]
        L.cowa_bwd_varlen.restype = i32
        L.cowa_bwd_varlen_workspace_bytes.argtypes = [i32] * 5 + [pp]
        L.cowa_bwd_varlen_workspace_bytes.restype = sz
        L.cowa_decode.argtypes = [vp] * 6 + [i32] * 5 + [pp, vp, sz, vp]
        L.cowa_decode.restype = i32
        L.cowa_decode_static.argtypes = [vp] * 6 + [i32] * 5 + [pp, vp]
        L.cowa_decode_static.restype = i32
        L.cowa_decode_multi.argtypes = [vp] * 6 + [i32] * 6 + [pp, vp, sz, vp]
        L.cowa_decode_multi.restype = i32
        L.cowa_decode_paged.argtypes = [vp] * 7 + [i32] * 7 + [pp, vp, sz, vp]
        L.cowa_decode_paged.restype = i32
        L.cowa_decode_multi_workspace_bytes.argtypes = [i32] * 6 + [pp]
        L.cowa_decode_multi_workspace_bytes.restype = sz
        L.cowa_decode_static_capacity.argtypes = []
        L.cowa_decode_static_capacity.restype = sz
        L.cowa_bwd_workspace_bytes.argtypes = [i32] * 5 + [pp]
        L.cowa_bwd_workspace_bytes.restype = sz
        L.cowa_decode_workspace_bytes.argtypes = [i32] * 5 + [pp]
        L.cowa_decode_workspace_bytes.restype = sz
        L.cowa_default_windows.argtypes = [i32] * 6 + [C.POINTER(Window)]
        L.cowa_default_windows.restype = i32
        L.cowa_equal_area_windows.argtypes = [i32] * 7 + [C.POINTER(Window)]
        L.cowa_equal_area_windows.restype = i32
        L.cowa_schedule_dump.argtypes = [i32, i32, i32, i32, pp, C.POINTER(C.c_int32), sz, C.POINTER(sz)]
        L.cowa_schedule_dump.restype = i32
        L.cowa_tile_counts.argtypes = [i32, i32, i32, pp, C.POINTER(C.c_int64)]
        L.cowa_tile_counts.restype = i32
        L.cowa_check_device_status.argtypes = [vp]
        L.cowa_check_device_status.restype = i32
        L.cowa_selftest_bounded_wait.argtypes = [C.c_longlong, vp]
        L.cowa_selftest_bounded_wait.restype = i32
        L.cowa_status_string.argtypes = [i32]
        L.cowa_status_string.restype = C.c_char_p
        L.cowa_last_cuda_error.argtypes = []
        L.cowa_last_cuda_error.restype = i32
        _lib = L
    return _lib


def make_params(sink=0, local=1, block=128, softmax_scale=1.0, windows=None, full_attn=False,
                hkv_global=0, hkv_offset=0, block_q=None, block_k=None, deterministic=False):
    """Fills a cowa_params_t.  `windows`: optional list of (sink, near, gap, len) per KV head."""
    p = Params()
    p.sink, p.local = int(sink), int(local)
    p.block_q = int(block_q if block_q is not None else block)
    p.block_k = int(block_k if block_k is not None else block)
    p.hkv_global, p.hkv_offset = int(hkv_global), int(hkv_offset)
    p.full_attn = 1 if full_attn else 0
    p.softmax_scale = float(softmax_scale)
    p.deterministic = 1 if deterministic else 0
    if windows is not None:
        arr = (Window * len(windows))(*[Window(*map(int, w)) for w in windows])
        p.windows = C.cast(arr, C.POINTER(Window))
        p._keepalive = arr
    return p


def _check(status, where):
    if status != 0:
        raise CowaError(status, where)


def _stream():
    import torch
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr(t):
    return C.c_void_p(0 if t is None else t.data_ptr())


def _need(t, dtype, name, strided=False):
    """Contiguous CUDA tensor of `dtype`; with strided=True any batch / head / token strides are accepted as
    long as the last axis is contiguous (the strides then travel in cowa_params_t)."""
    import torch
    ok = isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == dtype
    if ok and strided:
        ok = t.stride(-1) == 1 or t.shape[-1] == 1
    elif ok:
        ok = t.is_contiguous()
    if not ok:
        kind = "CUDA tensor with a contiguous last axis" if strided else "contiguous CUDA tensor"
        raise TypeError(f"{name}: expected a {kind} of {dtype}")


def _copy_params(params):
    p = Params.from_buffer_copy(params)
    p._keepalive = params  # the windows array (if any) lives as long as the original
    return p


def _with_strides(params, **tensors):
    """`params` itself when every tensor is contiguous, else a copy whose <name>_strides hold the tensors'
    (batch, head, token) element strides."""
    if all(t.is_contiguous() for t in tensors.values()):
        return params
    p = _copy_params(params)
    for name, t in tensors.items():
        getattr(p, name + "_strides")[:] = [t.stride(0), t.stride(1), t.stride(2)]
    return p


def with_bwd_events(params, start_event, stop_event):
    """Copy of `params` that makes cowa_bwd record the two torch.cuda.Event objects (already created, e.g.
    recorded once) just before and after its main kernel."""
    p = _copy_params(params)
    p.bwd_main_start_event = start_event.cuda_event
    p.bwd_main_stop_event = stop_event.cuda_event
    return p


def _same_layout(a, b, na, nb):
    if a.shape != b.shape or a.stride() != b.stride():
        raise TypeError(f"{na} must have the shape and strides of {nb}")


def cowa_fwd(q, k, v, o, lse, params):
    """q [B,Hq,T,D], k/v [B,Hkv,T,D] bf16 -> o (bf16), lse (fp32 [B,Hq,T]); all preallocated.  q, k, v, o may
    be strided views with that shape (e.g. x.transpose(1, 2) of a [B,T,H,D] tensor)."""
    import torch
    for t, n in ((q, "q"), (k, "k"), (v, "v"), (o, "o")):
        _need(t, torch.bfloat16, n, strided=True)
    _need(lse, torch.float32, "lse")
    B, Hq, T, D = q.shape
    Hkv = k.shape[1]
    params = _with_strides(params, q=q, k=k, v=v, o=o)
    _check(lib().cowa_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), B, T, Hq, Hkv, D,
                          C.byref(params), _stream()), "cowa_fwd")


def cowa_prefill(q, k, v, o, lse, params):
    """Forward with N_q <= N_k (bottom-right aligned): q [B,Hq,Nq,D], k/v [B,Hkv,Nk,D] -> o, lse [B,Hq,Nq]."""
    import torch
    for t, n in ((q, "q"), (k, "k"), (v, "v"), (o, "o")):
        _need(t, torch.bfloat16, n, strided=True)
    _need(lse, torch.float32, "lse")
    B, Hq, Nq, D = q.shape
    Hkv, Nk = k.shape[1], k.shape[2]
    params = _with_strides(params, q=q, k=k, v=v, o=o)
    _check(lib().cowa_prefill(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), B, Nq, Nk, Hq, Hkv, D,
                              C.byref(params), _stream()), "cowa_prefill")


def cowa_prefill_varlen(q, k, v, o, lse, cu_seqlens_q, cu_seqlens_k, params):
    """Packed batch: q [Hq,total_q,D], k/v [Hkv,total_k,D] -> o, lse [Hq,total_q]; cu_seqlens_* are CUDA int32
    tensors of B+1 row offsets."""
    import torch
    for t, n in ((q, "q"), (k, "k"), (v, "v"), (o, "o")):
        _need(t, torch.bfloat16, n)
    _need(lse, torch.float32, "lse")
    _need(cu_seqlens_q, torch.int32, "cu_seqlens_q")
    _need(cu_seqlens_k, torch.int32, "cu_seqlens_k")
    if cu_seqlens_q.numel() != cu_seqlens_k.numel() or cu_seqlens_q.numel() < 2:
        raise ValueError("cu_seqlens_q and cu_seqlens_k must both hold B+1 offsets")
    Hq, total_q, D = q.shape
    Hkv, total_k = k.shape[0], k.shape[1]
    B = cu_seqlens_q.numel() - 1
    _check(lib().cowa_prefill_varlen(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(cu_seqlens_q),
                                     _ptr(cu_seqlens_k), B, total_q, total_k, Hq, Hkv, D,
                                     C.byref(params), _stream()), "cowa_prefill_varlen")


def cowa_bwd_workspace_bytes(B, T, Hq, Hkv, D, params):
    return int(lib().cowa_bwd_workspace_bytes(B, T, Hq, Hkv, D, C.byref(params)))


def cowa_bwd(q, k, v, o, lse, d_o, dq, dk, dv, params, workspace):
    """Gradients dq, dk, dv (bf16, preallocated) of cowa_fwd; workspace: uint8 CUDA tensor.  Strided views are
    accepted when d_o is laid out like o, dq like q, dk like k and dv like v."""
    import torch
    for t, n in ((q, "q"), (k, "k"), (v, "v"), (o, "o"), (d_o, "d_o"), (dq, "dq"), (dk, "dk"), (dv, "dv")):
        _need(t, torch.bfloat16, n, strided=True)
    _need(lse, torch.float32, "lse")
    for a_, b_, na, nb in ((d_o, o, "d_o", "o"), (dq, q, "dq", "q"), (dk, k, "dk", "k"), (dv, v, "dv", "v")):
        _same_layout(a_, b_, na, nb)
    B, Hq, T, D = q.shape
    Hkv = k.shape[1]
    params = _with_strides(params, q=q, k=k, v=v, o=o)
    _check(lib().cowa_bwd(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(d_o), _ptr(dq), _ptr(dk),
                          _ptr(dv), B, T, Hq, Hkv, D, C.byref(params), _ptr(workspace),
                          workspace.numel() * workspace.element_size(), _stream()), "cowa_bwd")


def cowa_bwd_prefill_workspace_bytes(B, Nq, Nk, Hq, Hkv, D, params):
    return int(lib().cowa_bwd_prefill_workspace_bytes(B, Nq, Nk, Hq, Hkv, D, C.byref(params)))


def cowa_bwd_prefill(q, k, v, o, lse, d_o, dq, dk, dv, params, workspace):
    """Backward with N_q <= N_k: q/o/d_o/dq [B,Hq,Nq,D], k/v/dk/dv [B,Hkv,Nk,D], lse [B,Hq,Nq]."""
    import torch
    for t, n in ((q, "q"), (k, "k"), (v, "v"), (o, "o"), (d_o, "d_o"), (dq, "dq"), (dk, "dk"), (dv, "dv")):
        _need(t, torch.bfloat16, n, strided=True)
    _need(lse, torch.float32, "lse")
    for a_, b_, na, nb in ((d_o, o, "d_o", "o"), (dq, q, "dq", "q"), (dk, k, "dk", "k"), (dv, v, "dv", "v")):
        _same_layout(a_, b_, na, nb)
    B, Hq, Nq, D = q.shape
    Hkv, Nk = k.shape[1], k.shape[2]
    params = _with_strides(params, q=q, k=k, v=v, o=o)
    _check(lib().cowa_bwd_prefill(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(d_o), _ptr(dq), _ptr(dk),
                                  _ptr(dv), B, Nq, Nk, Hq, Hkv, D, C.byref(params), _ptr(workspace),
                                  workspace.numel() * workspace.element_size(), _stream()), "cowa_bwd_prefill")


def cowa_bwd_varlen_workspace_bytes(B, total, Hq, Hkv, D, params):
    return int(lib().cowa_bwd_varlen_workspace_bytes(B, total, Hq, Hkv, D, C.byref(params)))


def cowa_bwd_varlen(q, k, v, o, lse, d_o, dq, dk, dv, cu_seqlens, params, workspace):
    """Packed batch (N_q = N_k per sequence): q/o/d_o/dq [Hq,total,D], k/v/dk/dv [Hkv,total,D], lse [Hq,total];
    cu_seqlens CUDA int32 [B+1]."""
    import torch
    for t, n in ((q, "q"), (k, "k"), (v, "v"), (o, "o"), (d_o, "d_o"), (dq, "dq"), (dk, "dk"), (dv, "dv")):
        _need(t, torch.bfloat16, n)
    _need(lse, torch.float32, "lse")
    _need(cu_seqlens, torch.int32, "cu_seqlens")
    Hq, total, D = q.shape
    Hkv = k.shape[0]
    B = cu_seqlens.numel() - 1
    _check(lib().cowa_bwd_varlen(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(d_o), _ptr(dq), _ptr(dk),
                                 _ptr(dv), _ptr(cu_seqlens), B, total, Hq, Hkv, D, C.byref(params), _ptr(workspace),
                                 workspace.numel() * workspace.element_size(), _stream()), "cowa_bwd_varlen")


def cowa_decode_workspace_bytes(B, Tmax, Hq, Hkv, D, params):
    return int(lib().cowa_decode_workspace_bytes(B, Tmax, Hq, Hkv, D, C.byref(params)))


def cowa_decode(q, kcache, vcache, lens, o, lse, params, workspace):
    """q [B,Hq,D], caches [B,Hkv,Tmax,D] bf16 (strided views with that shape are accepted, e.g. a
    [B,Tmax,Hkv,D] cache transposed), lens int32 [B] (device) -> o [B,Hq,D], lse [B,Hq] or None."""
    import torch
    for t, n in ((q, "q"), (o, "o")):
        _need(t, torch.bfloat16, n)
    for t, n in ((kcache, "kcache"), (vcache, "vcache")):
        _need(t, torch.bfloat16, n, strided=True)
    _need(lens, torch.int32, "lens")
    if lse is not None:
        _need(lse, torch.float32, "lse")
    B, Hq, D = q.shape
    Hkv, Tmax = kcache.shape[1], kcache.shape[2]
    params = _with_strides(params, k=kcache, v=vcache)
    _check(lib().cowa_decode(_ptr(q), _ptr(kcache), _ptr(vcache), _ptr(lens), _ptr(o), _ptr(lse), B, Tmax,
                             Hq, Hkv, D, C.byref(params), _ptr(workspace),
                             workspace.numel() * workspace.element_size(), _stream()), "cowa_decode")


def cowa_decode_static_capacity():
    return int(lib().cowa_decode_static_capacity())


def cowa_decode_multi_workspace_bytes(B, Nq, Tmax, Hq, Hkv, D, params):
    return int(lib().cowa_decode_multi_workspace_bytes(B, Nq, Tmax, Hq, Hkv, D, C.byref(params)))


def cowa_decode_multi(q, kcache, vcache, lens, o, lse, params, workspace):
    """q, o [B,Nq,Hq,D]; kcache/vcache [B,Hkv,Tmax,D]; lens int32 [B] (device); lse [B,Nq,Hq] or None."""
    import torch
    for t, n in ((q, "q"), (kcache, "kcache"), (vcache, "vcache"), (o, "o")):
        _need(t, torch.bfloat16, n)
    _need(lens, torch.int32, "lens")
    if lse is not None:
        _need(lse, torch.float32, "lse")
    B, Nq, Hq, D = q.shape
    Hkv, Tmax = kcache.shape[1], kcache.shape[2]
    _check(lib().cowa_decode_multi(_ptr(q), _ptr(kcache), _ptr(vcache), _ptr(lens), _ptr(o),
                                   _ptr(lse) if lse is not None else None, B, Nq, Tmax, Hq, Hkv, D, C.byref(params),
                                   _ptr(workspace), workspace.numel() * workspace.element_size(), _stream()),
           "cowa_decode_multi")


def cowa_decode_paged(q, kpages, vpages, block_table, lens, o, lse, params, workspace):
    """q, o [B,Nq,Hq,D]; kpages/vpages [num_pages,Hkv,page_size,D]; block_table int32 [B,max_pages] (device)."""
    import torch
    for t, n in ((q, "q"), (kpages, "kpages"), (vpages, "vpages"), (o, "o")):
        _need(t, torch.bfloat16, n)
    _need(lens, torch.int32, "lens")
    _need(block_table, torch.int32, "block_table")
    if lse is not None:
        _need(lse, torch.float32, "lse")
    B, Nq, Hq, D = q.shape
    Hkv, page_size = kpages.shape[1], kpages.shape[2]
    max_pages = block_table.shape[1]
    _check(lib().cowa_decode_paged(_ptr(q), _ptr(kpages), _ptr(vpages), _ptr(block_table), _ptr(lens), _ptr(o),
                                   _ptr(lse) if lse is not None else None, B, Nq, max_pages, page_size, Hq, Hkv, D,
                                   C.byref(params), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                   _stream()), "cowa_decode_paged")


def cowa_decode_static(q, kcache, vcache, lens, o, lse, params):
    """cowa_decode without a workspace argument: for callers that may not allocate device
    memory.  The split states go to a fixed 8 MiB array inside the library; calls that need more
    raise CowaError (status -7).  Calls that overlap on the GPU must be serialised."""
    import torch
    for t, n in ((q, "q"), (kcache, "kcache"), (vcache, "vcache"), (o, "o")):
        _need(t, torch.bfloat16, n)
    _need(lens, torch.int32, "lens")
    if lse is not None:
        _need(lse, torch.float32, "lse")
    B, Hq, D = q.shape
    Hkv, Tmax = kcache.shape[1], kcache.shape[2]
    _check(lib().cowa_decode_static(_ptr(q), _ptr(kcache), _ptr(vcache), _ptr(lens), _ptr(o), _ptr(lse), B,
                                    Tmax, Hq, Hkv, D, C.byref(params), _stream()), "cowa_decode_static")


def cowa_default_windows(Nk, Hkv_global, hkv_offset, Hkv_local, sink, local):
    out = (Window * Hkv_local)()
    _check(lib().cowa_default_windows(Nk, Hkv_global, hkv_offset, Hkv_local, sink, local, out),
           "cowa_default_windows")
    return [(w.sink, w.near, w.gap, w.len) for w in out]


def cowa_equal_area_windows(Nq, Nk, Hkv_global, hkv_offset, Hkv_local, sink, local):
    out = (Window * Hkv_local)()
    _check(lib().cowa_equal_area_windows(Nq, Nk, Hkv_global, hkv_offset, Hkv_local, sink, local, out),
           "cowa_equal_area_windows")
    return [(w.sink, w.near, w.gap, w.len) for w in out]


def cowa_schedule_dump(which, Nq, Nk, Hkv, params):
    """Returns the int32 stream described in cowa.h as a list."""
    n = C.c_size_t(0)
    st = lib().cowa_schedule_dump(which, Nq, Nk, Hkv, C.byref(params), None, 0, C.byref(n))
    if st not in (0, -4):
        _check(st, "cowa_schedule_dump")
    buf = (C.c_int32 * max(n.value, 1))()
    _check(lib().cowa_schedule_dump(which, Nq, Nk, Hkv, C.byref(params), buf, n.value, C.byref(n)),
           "cowa_schedule_dump")
    return list(buf[:n.value])


def cowa_tile_counts(Nq, Nk, Hkv, params):
    out = (C.c_int64 * 3)()
    _check(lib().cowa_tile_counts(Nq, Nk, Hkv, C.byref(params), out), "cowa_tile_counts")
    return dict(visited=out[0], full=out[1], causal=out[2])


def cowa_check_device_status():
    _check(lib().cowa_check_device_status(_stream()), "cowa_check_device_status")


def cowa_selftest_bounded_wait(limit_clocks=1 << 20):
    """Enqueues the library's self-test kernel whose bounded wait must run out (see cowa.h)."""
    _check(lib().cowa_selftest_bounded_wait(int(limit_clocks), _stream()), "cowa_selftest_bounded_wait")


def cowa_status_string(status):
    return lib().cowa_status_string(status).decode()
