"""Failure detection on the device without faulting anything: every wait of the kernels is
bounded, and when one runs out the kernel stops by itself and leaves RATTN_ERR_TIMEOUT in the
workspace's status word.  The debug build of the library (librattn_dbg.so, include/rattn_debug.h)
can be told to withhold one mbarrier arrival -- a flag that nothing sets -- so that a wait does
run out; the test checks that the call returns, that the host reads the status, and that the
very next ordinary call on the same context is correct."""
import ctypes
import os

import numpy as np
import pytest
import torch

from oracle import rattn_oracle as O
from paper_2506_15545_b200 import binding as R
from paper_2506_15545_b200 import build as B
from paper_2506_15545_b200 import workloads as W
from test_gpu_parity import check, np64, small

pytestmark = pytest.mark.gpu

RATTN_ERR_TIMEOUT = -7


@pytest.fixture(scope="module")
def dbg():
    path = B.build(debug=True)
    L = ctypes.CDLL(path)
    vp, ci = ctypes.c_void_p, ctypes.c_int
    L.rattn_forward_ex.argtypes = [ctypes.POINTER(R.RattnParams), vp]
    L.rattn_forward_ex.restype = ci
    L.rattn_read_status.argtypes = [vp, vp]
    L.rattn_read_status.restype = ci
    L.rattn_debug_withhold_arrival.argtypes = [ci]
    L.rattn_debug_withhold_arrival.restype = ci
    yield L
    L.rattn_debug_withhold_arrival(0)


def _forward(L, q, k, v, out, ws, wl):
    p = R._params(q, k, v, out, wl.w, wl.scale, 1e-6, None, None, R.MODE_RATTN, ws, 0)
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    return L.rattn_forward_ex(ctypes.byref(p), stream), stream


def test_expired_wait_is_reported_and_the_context_stays_usable(dbg):
    wl = small("fd", 1, 1, 1, 256, 128, 128, "bf16", 8100, unit=True)    # one work unit, one CTA
    assert R.rattn_uses_tensor_path(wl.d, wl.w)
    q, k, v = W.make_qkv(wl)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    ws = R.alloc_workspace(qd, kd, wl.w)
    out = torch.zeros_like(qd)

    dbg.rattn_debug_withhold_arrival(1)
    rc, stream = _forward(dbg, qd, kd, vd, out, ws, wl)
    assert rc == 0                                   # the launch itself is fine
    status = dbg.rattn_read_status(ctypes.c_void_p(ws.data_ptr()), stream)   # synchronises: the kernel has returned
    assert status == RATTN_ERR_TIMEOUT
    assert torch.cuda.current_stream().query()       # nothing left running

    # the switch off again: the same context, the same buffers, a correct result
    dbg.rattn_debug_withhold_arrival(0)
    rc, stream = _forward(dbg, qd, kd, vd, out, ws, wl)
    assert rc == 0
    assert dbg.rattn_read_status(ctypes.c_void_p(ws.data_ptr()), stream) == 0
    check(out, O.forward(np64(q), np64(k), np64(v), wl.w, wl.scale), "bf16", "after the time-out")
    # and the product library, loaded in the same process, is unaffected by the switch
    y = R.rattn_forward_ex(qd, kd, vd, wl.w, scale=wl.scale, workspace=ws)
    assert R.rattn_read_status(ws) == 0
    assert torch.equal(y, out)


def test_plain_forward_latches_its_status_before_freeing_its_scratch(dbg):
    """rattn_forward takes its scratch from the stream-ordered pool and frees it before it returns, so
    the status word in it is copied into the library first: rattn_forward_status reports the expired
    wait, is clear again afterwards, and the next call is correct."""
    vp, ci = ctypes.c_void_p, ctypes.c_int
    dbg.rattn_forward.argtypes = [vp, vp, vp, ci, ci, ci, ci, ci, ci, vp, vp]
    dbg.rattn_forward.restype = ci
    dbg.rattn_forward_status.argtypes = [vp]
    dbg.rattn_forward_status.restype = ci
    wl = small("fdp", 1, 1, 1, 256, 128, 128, "bf16", 8200, unit=True, scale=1.0)
    q, k, v = W.make_qkv(wl)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    out = torch.zeros_like(qd)
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    call = lambda: dbg.rattn_forward(qd.data_ptr(), kd.data_ptr(), vd.data_ptr(), 1, 1, 1, wl.T, 128, wl.w,
                                     out.data_ptr(), stream)
    assert dbg.rattn_forward_status(stream) == 0
    dbg.rattn_debug_withhold_arrival(1)
    assert call() == 0
    assert dbg.rattn_forward_status(stream) == RATTN_ERR_TIMEOUT
    assert dbg.rattn_forward_status(stream) == 0          # reading clears it
    dbg.rattn_debug_withhold_arrival(0)
    assert call() == 0
    assert dbg.rattn_forward_status(stream) == 0
    check(out, O.forward(np64(q), np64(k), np64(v), wl.w, 1.0), "bf16", "after the time-out")
    # the product library's own word was never touched
    y = R.rattn_forward(qd, kd, vd, wl.w)
    assert R.rattn_forward_status() == 0 and torch.equal(y, out)
