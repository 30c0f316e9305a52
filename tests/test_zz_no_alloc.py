"""rattn_forward_static, the entry point for callers that cannot allocate device memory
(its scratch is a fixed array inside the library).  Collected last on purpose: if it
fails, a run that stops at the first failure has already run every other test.

It is checked against the existing entry point (rattn_forward_ex with a caller-owned
workspace) on two calls in a row; the second call uses other data and a shorter sequence,
so anything the first call left in the shared array would show."""
import ctypes
import math

import pytest
import torch

from paper_2506_15545_b200 import binding as R
from paper_2506_15545_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _wl(T, seed, Hq=4, Hkv=2, d=128, w=128):
    return W.Workload("na", 1, Hq, Hkv, T, d, w, "bf16", seed, True, 1.0, 1.0 / math.sqrt(d))


def _both(wl):
    q, k, v = (t.cuda() for t in W.make_qkv(wl))
    ws = R.alloc_workspace(q, k, wl.w)
    want = R.rattn_forward_ex(q, k, v, wl.w, scale=wl.scale, workspace=ws)
    out = torch.empty_like(q)
    # A first call may still load the kernels' code and look up the array's address; the
    # property is checked on the call after it.  Free device memory as the driver reports it
    # covers every kind of allocation (cudaMalloc, a growing stream-ordered pool), not only
    # those made through torch's caching allocator.
    R.rattn_forward_static(q, k, v, wl.w, wl.scale, out=out)
    torch.cuda.synchronize()
    before, free_before = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
    got = R.rattn_forward_static(q, k, v, wl.w, wl.scale, out=out)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before
    assert torch.cuda.mem_get_info()[0] >= free_before
    assert R.rattn_static_status() == 0          # no bounded device-side wait expired
    return got, want


def test_static_forward_matches_workspace_forward_twice_in_a_row():
    # first call: 2 K/V heads x 8 chunks = 16 chunk states in the shared array
    assert R.rattn_uses_tensor_path(128, 128)
    got, want = _both(_wl(1024, 901))
    err = (got.float() - want.float()).abs()
    assert err.max().item() <= 2e-2 and err.mean().item() <= 2e-3
    # second call straight after it: other data, shorter sequence (stale states must not leak)
    got, want = _both(_wl(640, 902))
    err = (got.float() - want.float()).abs()
    assert err.max().item() <= 2e-2 and err.mean().item() <= 2e-3
    assert torch.equal(got, want)        # same kernels, same inputs: the very same bits


def test_static_forward_portable_shapes_need_no_scratch():
    wl = _wl(200, 903, d=64, w=24)
    got, want = _both(wl)
    assert torch.equal(got, want)


def test_static_forward_refuses_sizes_beyond_its_scratch():
    # 2 K/V heads x 33 chunks = 66 > RATTN_STATIC_MAX_CHUNK_STATES (64)
    wl = _wl(33 * 128, 904)
    q, k, v = (torch.zeros(s, dtype=torch.bfloat16, device="cuda")
               for s in ((1, 4, wl.T, 128), (1, 2, wl.T, 128), (1, 2, wl.T, 128)))
    before = R.rattn_launch_count()
    with pytest.raises(R.RattnError) as ei:
        R.rattn_forward_static(q, k, v, wl.w, wl.scale)
    assert ei.value.code == -8 and "fixed scratch" in str(ei.value)
    assert R.rattn_launch_count() == before
    # exactly at the limit it runs: 2 x 32 = 64
    wl = _wl(32 * 128, 905)
    got, want = _both(wl)
    assert torch.equal(got, want)
