"""Argument validation of every entry point, on the host: a misaligned pointer or a workspace that is too
small must be refused before anything is launched, so these calls are made with made-up addresses that are
never dereferenced and need no GPU."""
import ctypes as C

import pytest

import paper_2609_32704_b200 as cowa

OK_PTR = 0x7F0000001000        # 16-byte aligned, never dereferenced
BAD_PTR = OK_PTR + 8           # not 16-byte aligned
MISALIGNED, TOO_SMALL, INVALID = -3, -4, -1
B, T, HQ, HKV, D = 2, 4096, 8, 2, 128


def _p(**kw):
    return cowa.make_params(sink=16, local=128, softmax_scale=0.1, **kw)


def _ptrs(n, bad=None):
    return [C.c_void_p(BAD_PTR if i == bad else OK_PTR) for i in range(n)]


@pytest.mark.parametrize("bad", [0, 1, 2, 3])
def test_fwd_and_prefill_refuse_misaligned_tensors(bad):
    L, p = cowa.lib(), _p()
    a = _ptrs(5, bad)
    assert L.cowa_fwd(*a, B, T, HQ, HKV, D, C.byref(p), None) == MISALIGNED
    assert L.cowa_prefill(*a, B, 64, T, HQ, HKV, D, C.byref(p), None) == MISALIGNED
    a = _ptrs(7, bad)
    assert L.cowa_prefill_varlen(*a, B, T, T, HQ, HKV, D, C.byref(p), None) == MISALIGNED


@pytest.mark.parametrize("bad", [0, 1, 2, 3, 5, 6, 7, 8])
def test_bwd_refuses_misaligned_tensors(bad):
    L, p = cowa.lib(), _p()
    big = 1 << 40
    a = _ptrs(9, bad)
    ws = C.c_void_p(OK_PTR)
    assert L.cowa_bwd(*a, B, T, HQ, HKV, D, C.byref(p), ws, big, None) == MISALIGNED
    assert L.cowa_bwd_prefill(*a, B, 64, T, HQ, HKV, D, C.byref(p), ws, big, None) == MISALIGNED
    a = _ptrs(10, bad)
    assert L.cowa_bwd_varlen(*a, B, T, HQ, HKV, D, C.byref(p), ws, big, None) == MISALIGNED


def test_bwd_refuses_misaligned_or_small_workspace():
    L, p = cowa.lib(), _p()
    a = _ptrs(9)
    need = cowa.cowa_bwd_workspace_bytes(B, T, HQ, HKV, D, p)
    assert need >= B * HQ * T * (D + 2) * 4
    assert L.cowa_bwd(*a, B, T, HQ, HKV, D, C.byref(p), C.c_void_p(BAD_PTR), need, None) == MISALIGNED
    assert L.cowa_bwd(*a, B, T, HQ, HKV, D, C.byref(p), C.c_void_p(OK_PTR), need - 1, None) == TOO_SMALL
    need = cowa.cowa_bwd_prefill_workspace_bytes(B, 64, T, HQ, HKV, D, p)
    assert L.cowa_bwd_prefill(*a, B, 64, T, HQ, HKV, D, C.byref(p), C.c_void_p(OK_PTR), need - 1, None) == TOO_SMALL
    a = _ptrs(10)
    need = cowa.cowa_bwd_varlen_workspace_bytes(B, T, HQ, HKV, D, p)
    assert L.cowa_bwd_varlen(*a, B, T, HQ, HKV, D, C.byref(p), C.c_void_p(BAD_PTR), need, None) == MISALIGNED
    assert L.cowa_bwd_varlen(*a, B, T, HQ, HKV, D, C.byref(p), C.c_void_p(OK_PTR), need - 1, None) == TOO_SMALL


@pytest.mark.parametrize("bad", [0, 1, 2, 4])
def test_decode_calls_refuse_misaligned_tensors(bad):
    L, p = cowa.lib(), _p()
    a = _ptrs(6, bad)
    ws, big = C.c_void_p(OK_PTR), 1 << 40
    assert L.cowa_decode(*a, B, T, HQ, HKV, D, C.byref(p), ws, big, None) == MISALIGNED
    assert L.cowa_decode_static(*a, B, T, HQ, HKV, D, C.byref(p), None) == MISALIGNED
    assert L.cowa_decode_multi(*a, B, 2, T, HQ, HKV, D, C.byref(p), ws, big, None) == MISALIGNED
    a7 = a[:3] + [C.c_void_p(OK_PTR)] + a[3:]   # block table inserted after the pages
    assert L.cowa_decode_paged(*a7, B, 2, T // 64, 64, HQ, HKV, D, C.byref(p), ws, big, None) == MISALIGNED


def test_decode_calls_refuse_misaligned_or_small_workspace():
    L, p = cowa.lib(), _p()
    a = _ptrs(6)
    need = cowa.cowa_decode_workspace_bytes(B, T, HQ, HKV, D, p)
    assert need > 0
    assert L.cowa_decode(*a, B, T, HQ, HKV, D, C.byref(p), C.c_void_p(BAD_PTR), need, None) == MISALIGNED
    assert L.cowa_decode(*a, B, T, HQ, HKV, D, C.byref(p), C.c_void_p(OK_PTR), need - 1, None) == TOO_SMALL
    need = cowa.cowa_decode_multi_workspace_bytes(B, 2, T, HQ, HKV, D, p)
    assert L.cowa_decode_multi(*a, B, 2, T, HQ, HKV, D, C.byref(p), C.c_void_p(BAD_PTR), need, None) == MISALIGNED
    assert L.cowa_decode_multi(*a, B, 2, T, HQ, HKV, D, C.byref(p), C.c_void_p(OK_PTR), need - 1, None) == TOO_SMALL
    a7 = a[:3] + [C.c_void_p(OK_PTR)] + a[3:]
    assert L.cowa_decode_paged(*a7, B, 2, T // 64, 64, HQ, HKV, D, C.byref(p), C.c_void_p(OK_PTR), need - 1,
                               None) == TOO_SMALL


def test_scale_and_window_arguments():
    L = cowa.lib()
    a = _ptrs(6)
    p = cowa.make_params(sink=16, local=128, softmax_scale=0.0)
    assert L.cowa_decode(*a, B, T, HQ, HKV, D, C.byref(p), C.c_void_p(OK_PTR), 1 << 40, None) == INVALID
    assert L.cowa_fwd(*a[:5], B, T, HQ, HKV, D, C.byref(p), None) == INVALID
    # explicit tuples far beyond the sequence mean what Nk means: clamped, accepted by the host-only calls
    huge = 2 ** 31 - 1
    p = cowa.make_params(windows=[(huge, huge, huge, huge)] * HKV, softmax_scale=0.1, block=128)
    ref = cowa.make_params(windows=[(T, T, T, T)] * HKV, softmax_scale=0.1, block=128)
    assert cowa.cowa_schedule_dump(cowa.SCHED_FWD, 512, 512, HKV, p) == \
        cowa.cowa_schedule_dump(cowa.SCHED_FWD, 512, 512, HKV, ref)
    assert cowa.cowa_tile_counts(512, 512, HKV, p) == cowa.cowa_tile_counts(512, 512, HKV, ref)


def test_params_struct_layout_matches_the_header(tmp_path):
    """The ctypes mirror of cowa_params_t must have the C compiler's layout of the struct in include/cowa.h."""
    import os
    import shutil
    import subprocess
    if shutil.which("gcc") is None:
        pytest.skip("no C compiler")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    fields = [n for n, _ in cowa.Params._fields_]
    prog = ['#include <stdio.h>', '#include <stddef.h>', '#include "cowa.h"', 'int main(void) {',
            '  printf("%zu\\n", sizeof(cowa_params_t));']
    prog += [f'  printf("%zu\\n", offsetof(cowa_params_t, {n}));' for n in fields]
    prog += ['  printf("%zu\\n", sizeof(cowa_window_t));', '  return 0;', '}']
    src = tmp_path / "layout.c"
    src.write_text("\n".join(prog))
    exe = tmp_path / "layout"
    subprocess.check_call(["gcc", "-std=c99", "-I", os.path.join(root, "include"), "-o", str(exe), str(src)])
    out = [int(x) for x in subprocess.check_output([str(exe)]).split()]
    assert out[0] == C.sizeof(cowa.Params)
    assert out[1:-1] == [getattr(cowa.Params, n).offset for n in fields]
    assert out[-1] == C.sizeof(cowa.Window)
