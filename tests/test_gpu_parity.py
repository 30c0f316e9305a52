"""Parity of the CUDA path (through the C ABI) against the fp64 oracle, element by element
on the same seeded inputs.  Tolerances: fp32 I/O max-abs <= 1e-4; bf16 I/O max-abs <= 2e-2
and mean-abs <= 2e-3; gradients <= 5e-2 relative Frobenius norm per tensor."""
import math

import numpy as np
import pytest
import torch

from oracle import rattn_oracle as O
from paper_2506_15545_b200 import binding as R
from paper_2506_15545_b200 import workloads as W

pytestmark = pytest.mark.gpu

TOL = {"f32": dict(max_abs=1e-4, mean_abs=1e-5), "bf16": dict(max_abs=2e-2, mean_abs=2e-3)}
GRAD_TOL = 5e-2


def np64(t):
    return t.detach().to("cpu", torch.float64).numpy()


def check(y_gpu, y_ref, dtype, what=""):
    err = np.abs(np64(y_gpu) - y_ref)
    assert np.isfinite(np64(y_gpu)).all(), what
    assert err.max() <= TOL[dtype]["max_abs"], (what, err.max())
    assert err.mean() <= TOL[dtype]["mean_abs"], (what, err.mean())


def small(name, B, Hq, Hkv, T, d, w, dtype, seed, unit=False, scale=None, prescale=1.0):
    return W.Workload(name, B, Hq, Hkv, T, d, w, dtype, seed, unit, prescale,
                      1.0 / math.sqrt(d) if scale is None else scale)


def run_fwd(wl, mode=R.MODE_RATTN, gains=False, flags=0, workspace=True, save=False):
    q, k, v = W.make_qkv(wl, "cpu")
    gs = gr = None
    if gains:
        gs, gr = W.make_gains(wl, "cpu")
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    ws = R.alloc_workspace(qd, kd, wl.w) if workspace else None
    y = R.rattn_forward_ex(qd, kd, vd, wl.w, scale=wl.scale, mode=mode, workspace=ws,
                           gamma_swa=None if gs is None else gs.cuda(),
                           gamma_rla=None if gr is None else gr.cuda(), flags=flags,
                           save_residuals=save)
    torch.cuda.synchronize()
    if ws is not None:
        assert R.rattn_read_status(ws) == 0
    ref = O.forward(np64(q), np64(k), np64(v), wl.w, wl.scale, 1e-6,
                    None if gs is None else np64(gs), None if gr is None else np64(gr), mode)
    return y, ref, (qd, kd, vd, ws, gs, gr)


# ------------------------------------------------------------------ forward, portable path

def test_config1_fp32_full():
    """B=1, H=2/2, T=1024, d=64, w=128, fp32, q pre-scaled by 1/sqrt(d), scale = 1."""
    y, ref, _ = run_fwd(W.C1)
    check(y, ref, "f32", "c1")


@pytest.mark.parametrize("T,d,w,Hq,Hkv,dtype", [
    (1, 64, 4, 1, 1, "f32"),            # a single token
    (5, 64, 1, 2, 1, "f32"),            # w = 1: window is the token and its predecessor
    (130, 64, 7, 4, 2, "f32"),          # ragged T, odd window, GQA
    (257, 128, 64, 2, 2, "f32"),        # d = 128, T = tile + 1
    (200, 128, 300, 2, 1, "f32"),       # w > T: no residual token at all
    (192, 64, 63, 6, 2, "bf16"),        # group of three
    (384, 128, 100, 4, 4, "bf16"),      # bf16 with a window that is no tile multiple
    (320, 128, 128, 8, 2, "bf16"),      # shapes the tensor path takes, forced portable
])
def test_forward_portable_shapes(T, d, w, Hq, Hkv, dtype):
    wl = small("s", 2, Hq, Hkv, T, d, w, dtype, 31 + T)
    y, ref, _ = run_fwd(wl, gains=True, flags=R.FLAG_FORCE_GENERIC)
    check(y, ref, dtype, f"T={T} d={d} w={w}")


@pytest.mark.parametrize("mode", [R.MODE_SWA_ONLY, R.MODE_FULL_CAUSAL])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_forward_portable_control_modes(mode, dtype):
    wl = small("m", 1, 4, 2, 300, 64, 32, dtype, 77)
    y, ref, _ = run_fwd(wl, mode=mode, gains=True, flags=R.FLAG_FORCE_GENERIC)
    check(y, ref, dtype, f"mode={mode}")


def test_rows_beyond_T_are_not_written_and_no_workspace_is_needed():
    wl = small("pad", 1, 2, 2, 100, 64, 16, "f32", 5)
    q, k, v = (t.cuda() for t in W.make_qkv(wl))
    n = 2 * 100 * 64
    big = torch.full((n + 4096,), 7.0, device="cuda")
    out, guard = big[:n].view(1, 2, 100, 64), big[n:]
    R.rattn_forward_ex(q, k, v, wl.w, scale=wl.scale, out=out, flags=R.FLAG_FORCE_GENERIC)
    torch.cuda.synchronize()
    assert torch.all(guard == 7.0)
    ref = O.forward(np64(q), np64(k), np64(v), wl.w, wl.scale)
    check(out, ref, "f32")


def test_run_to_run_determinism():
    wl = small("det", 2, 4, 2, 333, 64, 40, "bf16", 9)
    q, k, v = (t.cuda() for t in W.make_qkv(wl))
    a = R.rattn_forward_ex(q, k, v, wl.w, scale=wl.scale, flags=R.FLAG_FORCE_GENERIC)
    b = R.rattn_forward_ex(q, k, v, wl.w, scale=wl.scale, flags=R.FLAG_FORCE_GENERIC)
    assert torch.equal(a, b)


def test_plain_entry_point_matches_oracle():
    """rattn_forward: bf16, scale = 1 (logits q.k as the paper prints them), unit gains."""
    wl = small("plain", 1, 2, 1, 160, 64, 24, "bf16", 11, prescale=0.2, scale=1.0)
    q, k, v = W.make_qkv(wl)
    y = R.rattn_forward(q.cuda(), k.cuda(), v.cuda(), wl.w)
    ref = O.forward(np64(q), np64(k), np64(v), wl.w, 1.0)
    check(y, ref, "bf16")


# ------------------------------------------------------------------ decode

@pytest.mark.parametrize("d,w,Hq,Hkv,dtype,T0,steps", [
    (64, 8, 4, 2, "f32", 0, 30),        # from an empty cache through pos = w-1, w, w+1, 2w
    (128, 16, 8, 2, "bf16", 40, 20),    # after a prefill, GQA group of 4
    (128, 32, 12, 2, "bf16", 5, 70),    # group of 6 (> heads per pass), prefill shorter than w
    (64, 4, 2, 2, "bf16", 9, 12),
])
def test_decode_after_prefill_equals_full_forward(d, w, Hq, Hkv, dtype, T0, steps):
    """Prefill hand-off (ring + state) followed by n decode steps must reproduce rows
    T0..T0+n-1 of the operator on the whole sequence (the oracle has no ring, no state)."""
    B = 2
    wl = small("dec", B, Hq, Hkv, T0 + steps, d, w, dtype, 101 + d + w)
    q, k, v = W.make_qkv(wl)
    gs, gr = W.make_gains(wl)
    dt = wl.torch_dtype
    state = torch.zeros(B, Hkv, d, d, device="cuda")
    k_ring = torch.zeros(B, Hkv, w, d, device="cuda", dtype=dt)
    v_ring = torch.zeros_like(k_ring)
    if T0 > 0:
        R.rattn_forward_ex(q[:, :, :T0].contiguous().cuda(), k[:, :, :T0].contiguous().cuda(),
                           v[:, :, :T0].contiguous().cuda(), w, scale=wl.scale,
                           state_out=state, k_ring_out=k_ring, v_ring_out=v_ring,
                           flags=R.FLAG_FORCE_GENERIC)
        ref_state = np.stack([[O.rla_state(np64(k[b, h, :T0]), np64(v[b, h, :T0]), T0 - w)
                               for h in range(Hkv)] for b in range(B)])
        assert np.abs(np64(state) - ref_state).max() <= 1e-3 * max(1.0, np.abs(ref_state).max())
    outs = []
    for s in range(steps):
        pos = T0 + s
        outs.append(R.rattn_decode_step_ex(
            q[:, :, pos].contiguous().cuda(), k[:, :, pos].contiguous().cuda(),
            v[:, :, pos].contiguous().cuda(), k_ring, v_ring, state, pos, scale=wl.scale,
            gamma_swa=gs.cuda(), gamma_rla=gr.cuda()))
    torch.cuda.synchronize()
    y = torch.stack(outs, dim=2)
    ref = O.forward(np64(q), np64(k), np64(v), w, wl.scale, 1e-6, np64(gs), np64(gr))[:, :, T0:]
    check(y, ref, dtype, "decode")
    # the ring ends up holding the last w tokens at slot j % w
    T = T0 + steps
    for j in range(max(0, T - w), T):
        assert torch.equal(k_ring[:, :, j % w].cpu(), k[:, :, j])
        assert torch.equal(v_ring[:, :, j % w].cpu(), v[:, :, j])
    ref_state = np.stack([[O.rla_state(np64(k[b, h]), np64(v[b, h]), T - w) for h in range(Hkv)]
                          for b in range(B)])
    assert np.abs(np64(state) - ref_state).max() <= 2e-3 * max(1.0, np.abs(ref_state).max())


def test_plain_decode_entry_point():
    B, Hq, Hkv, d, w, steps = 1, 2, 1, 64, 6, 15
    wl = small("pd", B, Hq, Hkv, steps, d, w, "bf16", 55, prescale=0.3, scale=1.0)
    q, k, v = W.make_qkv(wl)
    state = torch.zeros(B, Hkv, d, d, device="cuda")
    k_ring = torch.zeros(B, Hkv, w, d, device="cuda", dtype=torch.bfloat16)
    v_ring = torch.zeros_like(k_ring)
    outs = [R.rattn_decode_step(q[:, :, p].contiguous().cuda(), k[:, :, p].contiguous().cuda(),
                                v[:, :, p].contiguous().cuda(), k_ring, v_ring, state, p)
            for p in range(steps)]
    ref = O.forward(np64(q), np64(k), np64(v), w, 1.0)
    check(torch.stack(outs, dim=2), ref, "bf16")


# ------------------------------------------------------------------ backward

def rel_fro(a, b):
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-30))


@pytest.mark.parametrize("T,d,w,Hq,Hkv,dtype,mode", [
    (256, 64, 64, 2, 2, "f32", R.MODE_RATTN),      # the T=256 slice, w = 64 (RLA alive)
    (256, 128, 32, 4, 2, "bf16", R.MODE_RATTN),    # GQA: dk, dv summed over the group
    (256, 128, 512, 2, 2, "bf16", R.MODE_RATTN),   # w >= T: the SWA-only limit
    (203, 64, 17, 3, 1, "f32", R.MODE_RATTN),      # ragged T, odd window, group of 3
    (160, 64, 16, 2, 2, "bf16", R.MODE_SWA_ONLY),
    (160, 128, 16, 2, 1, "f32", R.MODE_FULL_CAUSAL),
])
def test_backward_against_oracle(T, d, w, Hq, Hkv, dtype, mode):
    wl = small("bwd", 2, Hq, Hkv, T, d, w, dtype, 900 + T + w, unit=True)
    q, k, v = W.make_qkv(wl)
    dy = W.make_dout(wl)
    gs, gr = W.make_gains(wl)
    qd, kd, vd, dyd = q.cuda(), k.cuda(), v.cuda(), dy.cuda()
    ws = R.alloc_workspace(qd, kd, w)
    R.rattn_forward_ex(qd, kd, vd, w, scale=wl.scale, mode=mode, workspace=ws, save_residuals=True,
                       gamma_swa=gs.cuda(), gamma_rla=gr.cuda(), flags=R.FLAG_FORCE_GENERIC)
    dgs = torch.empty(Hq, d, device="cuda")
    dgr = torch.empty(Hq, d, device="cuda")
    dq, dk, dv = R.rattn_backward_ex(qd, kd, vd, dyd, w, ws, scale=wl.scale, mode=mode,
                                     gamma_swa=gs.cuda(), gamma_rla=gr.cuda(),
                                     dgamma_swa=dgs, dgamma_rla=dgr, flags=R.FLAG_FORCE_GENERIC)
    torch.cuda.synchronize()
    ref = O.backward(np64(q), np64(k), np64(v), np64(dy), w, wl.scale, 1e-6, np64(gs), np64(gr), mode)
    for name, got, want in zip(("dq", "dk", "dv", "dgamma_swa"), (dq, dk, dv, dgs), ref):
        assert np.isfinite(np64(got)).all(), name
        assert rel_fro(np64(got), want) <= GRAD_TOL, (name, rel_fro(np64(got), want))
    if mode == R.MODE_RATTN and w < T:
        assert rel_fro(np64(dgr), ref[4]) <= GRAD_TOL
    if dtype == "f32":          # the fp32 path is far inside the bound
        for got, want in zip((dq, dk, dv), ref):
            assert rel_fro(np64(got), want) <= 1e-4


def test_plain_backward_entry_point():
    wl = small("pb", 1, 2, 1, 128, 64, 16, "bf16", 321, prescale=0.25, scale=1.0)
    q, k, v = W.make_qkv(wl)
    dy = W.make_dout(wl)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    ws = R.alloc_workspace(qd, kd, wl.w)
    R.rattn_forward_ex(qd, kd, vd, wl.w, workspace=ws, save_residuals=True)
    dq, dk, dv = R.rattn_backward(qd, kd, vd, dy.cuda(), ws, wl.w)
    ref = O.backward(np64(q), np64(k), np64(v), np64(dy), wl.w, 1.0)
    for got, want in zip((dq, dk, dv), ref):
        assert rel_fro(np64(got), want) <= GRAD_TOL
