"""Parity of the tensor-core (tcgen05) forward against the fp64 oracle: bf16, d = 128,
window a multiple of 128.  Same tolerances as the portable path: max-abs <= 2e-2,
mean-abs <= 2e-3 on outputs that are the sum of two unit-RMS vectors."""
import math

import numpy as np
import pytest
import torch

from oracle import rattn_oracle as O
from paper_2506_15545_b200 import binding as R
from paper_2506_15545_b200 import workloads as W
from test_gpu_parity import GRAD_TOL, check, np64, rel_fro, small

pytestmark = pytest.mark.gpu


def run(wl, mode=R.MODE_RATTN, gains=True, save=False):
    assert R.rattn_uses_tensor_path(wl.d, wl.w, R.RATTN_BF16, mode)
    q, k, v = W.make_qkv(wl)
    gs, gr = W.make_gains(wl) if gains else (None, None)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    ws = R.alloc_workspace(qd, kd, wl.w)
    ws.zero_()
    y = R.rattn_forward_ex(qd, kd, vd, wl.w, scale=wl.scale, mode=mode, workspace=ws,
                           gamma_swa=None if gs is None else gs.cuda(),
                           gamma_rla=None if gr is None else gr.cuda(), save_residuals=save)
    torch.cuda.synchronize()
    assert R.rattn_read_status(ws) == 0, "a device-side wait expired"
    ref = O.forward(np64(q), np64(k), np64(v), wl.w, wl.scale, 1e-6,
                    None if gs is None else np64(gs), None if gr is None else np64(gr), mode)
    return y, ref, (qd, kd, vd, ws)


@pytest.mark.parametrize("T,w,Hq,Hkv,unit", [
    (128, 128, 1, 1, False),     # one tile, nothing outside the window
    (256, 128, 1, 1, False),     # second tile reads chunk 0 in intra form, no stored state
    (384, 128, 2, 1, True),      # third tile: stored state of chunk 0 + intra form of chunk 1
    (1024, 256, 4, 2, True),     # window of two tiles, GQA
    (1280, 512, 2, 2, False),    # the w = 512 band: five key tiles
    (300, 128, 2, 1, False),     # ragged T: last tile partly beyond the sequence
    (77, 128, 2, 2, False),      # T below one tile
    (640, 1024, 2, 1, True),     # w > T: SWA covers everything
])
def test_tensor_forward_shapes(T, w, Hq, Hkv, unit):
    wl = small("tc", 2, Hq, Hkv, T, 128, w, "bf16", 4000 + T + w, unit=unit)
    y, ref, _ = run(wl)
    check(y, ref, "bf16", f"T={T} w={w}")


@pytest.mark.parametrize("mode", [R.MODE_SWA_ONLY, R.MODE_FULL_CAUSAL])
def test_tensor_forward_control_modes(mode):
    wl = small("tcm", 1, 4, 2, 896, 128, 256, "bf16", 4100, unit=True)
    y, ref, _ = run(wl, mode=mode)
    check(y, ref, "bf16", f"mode={mode}")


def test_tensor_forward_large_logits_trigger_rescale():
    """Un-normalised q, k with scale 1/4: logits of std ~ 30, so the running maximum moves by
    far more than the lazy-rescale threshold between key tiles."""
    wl = small("tcr", 1, 2, 2, 768, 128, 256, "bf16", 4200, unit=False, scale=0.25)
    y, ref, _ = run(wl)
    check(y, ref, "bf16", "large logits")


@pytest.mark.parametrize("T,w,Hq,Hkv", [(1280, 256, 4, 2), (1100, 128, 4, 1), (2048, 512, 2, 2), (4096, 128, 2, 1)])
def test_tensor_forward_states_taken_as_published(T, w, Hq, Hkv):
    """The main kernel reading each chunk state as soon as the chunk-state kernel has published it
    (knob forced on; by default only long chains on few heads do this) computes the same operator,
    with the same bits as the default schedule: only the order of the work units differs."""
    wl = small("tcprog", 2, Hq, Hkv, T, 128, w, "bf16", 4500 + T + w, unit=True)
    y0, ref, _ = run(wl)
    prev = R.rattn_tune(R.TUNE_STATE_PROGRESS, 1)
    try:
        y1, _, _ = run(wl)
        y2, _, _ = run(wl, save=True)
    finally:
        R.rattn_tune(R.TUNE_STATE_PROGRESS, prev)
    # (with gains an output beyond |y| = 8 occurs in these inputs, where half a bf16 step alone is 3e-2:
    # the bound that takes the output format into account, as for the element-wise maps)
    from test_gpu_feature_maps import check_bf16_heavy_tails
    check_bf16_heavy_tails(y1, ref, f"progress words, T={T} w={w}")
    check_bf16_heavy_tails(y2, ref, f"progress words, training mode, T={T} w={w}")
    assert torch.equal(y0, y1)


def test_states_taken_as_published_never_read_stale_memory():
    """With the main kernel reading chunk states while the chunk-state kernel is still writing them, a
    state read before it was complete would show as whatever the workspace held before: poison it
    between calls and demand the bits of the schedule that waits for the whole chain, every time."""
    wl = small("tcstale", 1, 4, 1, 4096, 128, 128, "bf16", 4600, unit=True)
    q, k, v = (t.cuda() for t in W.make_qkv(wl))
    ws = R.alloc_workspace(q, k, wl.w)
    prev = R.rattn_tune(R.TUNE_STATE_PROGRESS, 2)
    try:
        want = R.rattn_forward_ex(q, k, v, wl.w, scale=wl.scale, workspace=ws).clone()
        R.rattn_tune(R.TUNE_STATE_PROGRESS, 1)
        out = torch.empty_like(q)
        for it in range(12):
            ws.fill_(0x5A if it % 2 else 0xFF)
            R.rattn_forward_ex(q, k, v, wl.w, scale=wl.scale, workspace=ws, out=out)
            torch.cuda.synchronize()
            assert R.rattn_read_status(ws) == 0
            assert torch.equal(out, want), it
    finally:
        R.rattn_tune(R.TUNE_STATE_PROGRESS, prev)


def test_tensor_forward_c2_like_heads():
    """Config 2's sequence (T=4096, w=512, unit-RMS q/k, scale 1/sqrt(128)) on two heads."""
    wl = W.C2.replace(B=1, H_q=2, H_kv=2)
    y, ref, _ = run(wl, gains=False)
    check(y, ref, "bf16", "c2 heads")


def test_tensor_residuals_match_portable_path():
    """The residuals the training-mode forward leaves for the backward: log-sum-exp (fp32, first
    region after the status block: 256 bytes, plus 256 bytes of per-head progress words on the
    tensor-core path) and the un-normalised window output (second region; fp32 on the portable
    path, bf16 on the tensor-core path) agree between the two paths."""
    wl = small("tcs", 1, 2, 1, 512, 128, 128, "bf16", 4300, unit=True)
    y, ref, (q, k, v, ws) = run(wl, save=True)
    ws2 = torch.zeros_like(ws)
    y2 = R.rattn_forward_ex(q, k, v, wl.w, scale=wl.scale, workspace=ws2, save_residuals=True,
                            gamma_swa=W.make_gains(wl)[0].cuda(), gamma_rla=W.make_gains(wl)[1].cuda(),
                            flags=R.FLAG_FORCE_GENERIC)
    torch.cuda.synchronize()
    n = 2 * 512
    head1 = 512                                   # status block + progress words (one K/V head: 256 bytes)
    f1 = ws[head1:].view(torch.float32)
    f2 = ws2[256:].view(torch.float32)
    lse1, lse2 = f1[:n], f2[:n]
    assert (lse1 - lse2).abs().max() < 2e-2
    off = (n * 4 + 255) // 256 * 256
    o1 = ws[head1 + off:head1 + off + n * 128 * 2].view(torch.bfloat16).float()
    o2 = f2[off // 4:off // 4 + n * 128]
    assert (o1 - o2).abs().max() < 3e-2
    check(y, ref, "bf16")


def test_tensor_run_to_run_determinism():
    wl = small("tcd", 2, 2, 1, 1024, 128, 256, "bf16", 4400, unit=True)
    q, k, v = (t.cuda() for t in W.make_qkv(wl))
    ws = R.alloc_workspace(q, k, wl.w)
    a = R.rattn_forward_ex(q, k, v, wl.w, scale=wl.scale, workspace=ws).clone()
    b = R.rattn_forward_ex(q, k, v, wl.w, scale=wl.scale, workspace=ws)
    assert torch.equal(a, b)


# ------------------------------------------------------------------ backward (tcgen05)

def run_bwd(wl, mode=R.MODE_RATTN, gains=True):
    """Tensor-core forward (saving residuals) + tensor-core backward against the oracle's
    analytic fp64 gradients; returns the relative Frobenius errors per tensor."""
    assert R.rattn_uses_tensor_path(wl.d, wl.w, R.RATTN_BF16, mode)
    q, k, v = W.make_qkv(wl)
    dy = W.make_dout(wl)
    gs, gr = W.make_gains(wl) if gains else (None, None)
    gsd = None if gs is None else gs.cuda()
    grd = None if gr is None else gr.cuda()
    qd, kd, vd, dyd = q.cuda(), k.cuda(), v.cuda(), dy.cuda()
    ws = R.alloc_workspace(qd, kd, wl.w)
    ws.zero_()
    R.rattn_forward_ex(qd, kd, vd, wl.w, scale=wl.scale, mode=mode, workspace=ws, gamma_swa=gsd,
                       gamma_rla=grd, save_residuals=True)
    dgs = torch.empty(wl.H_q, wl.d, device="cuda")
    dgr = torch.empty(wl.H_q, wl.d, device="cuda")
    dq = torch.full_like(qd, float("nan"))
    dk = torch.full_like(kd, float("nan"))
    dv = torch.full_like(vd, float("nan"))
    R.rattn_backward_ex(qd, kd, vd, dyd, wl.w, ws, scale=wl.scale, mode=mode, gamma_swa=gsd,
                        gamma_rla=grd, dq=dq, dk=dk, dv=dv, dgamma_swa=dgs, dgamma_rla=dgr)
    torch.cuda.synchronize()
    assert R.rattn_read_status(ws) == 0, "a device-side wait expired"
    ref = O.backward(np64(q), np64(k), np64(v), np64(dy), wl.w, wl.scale, 1e-6,
                     None if gs is None else np64(gs), None if gr is None else np64(gr), mode)
    errs = {}
    for name, got, want in zip(("dq", "dk", "dv", "dgamma_swa"), (dq, dk, dv, dgs), ref):
        assert np.isfinite(np64(got)).all(), name
        errs[name] = rel_fro(np64(got), want)
    if mode == R.MODE_RATTN and wl.w < wl.T - 1:
        errs["dgamma_rla"] = rel_fro(np64(dgr), ref[4])
    return errs


@pytest.mark.parametrize("T,w,Hq,Hkv,unit", [
    (128, 128, 1, 1, False),     # one tile: window branch only, diagonal mask only
    (256, 128, 1, 1, True),      # residual branch in intra form only (no stored state either way)
    (384, 128, 2, 1, True),      # forward state S_1 and reverse state R_0 both in play, group of 2
    (640, 256, 4, 2, True),      # window of two tiles, GQA
    (1280, 512, 2, 2, True),     # the w = 512 band
    (300, 128, 2, 1, False),     # ragged T
    (77, 128, 2, 2, False),      # T below one tile
    (640, 1024, 2, 1, True),     # w > T: window branch covers everything
])
def test_tensor_backward_shapes(T, w, Hq, Hkv, unit):
    wl = small("tcb", 2, Hq, Hkv, T, 128, w, "bf16", 5000 + T + w, unit=unit)
    errs = run_bwd(wl)
    for name, e in errs.items():
        assert e <= GRAD_TOL, (name, e, errs)


@pytest.mark.parametrize("mode", [R.MODE_SWA_ONLY, R.MODE_FULL_CAUSAL])
def test_tensor_backward_control_modes(mode):
    wl = small("tcbm", 1, 4, 2, 600, 128, 256, "bf16", 5100, unit=True)
    errs = run_bwd(wl, mode=mode)
    for name, e in errs.items():
        assert e <= GRAD_TOL, (name, e, errs)


def test_tensor_backward_matches_portable_backward():
    """Forward + backward on the tensor-core path against forward + backward on the portable
    path (each backward reads the residuals its own forward left): the two CUDA
    implementations agree far inside the bound either has against the oracle."""
    wl = small("tcbp", 1, 2, 1, 512, 128, 128, "bf16", 5200, unit=True)
    q, k, v = (t.cuda() for t in W.make_qkv(wl))
    dy = W.make_dout(wl).cuda()
    ws = R.alloc_workspace(q, k, wl.w)
    R.rattn_forward_ex(q, k, v, wl.w, scale=wl.scale, workspace=ws, save_residuals=True)
    a = [t.clone() for t in R.rattn_backward_ex(q, k, v, dy, wl.w, ws, scale=wl.scale)]
    R.rattn_forward_ex(q, k, v, wl.w, scale=wl.scale, workspace=ws, save_residuals=True,
                       flags=R.FLAG_FORCE_GENERIC)
    b = R.rattn_backward_ex(q, k, v, dy, wl.w, ws, scale=wl.scale, flags=R.FLAG_FORCE_GENERIC)
    torch.cuda.synchronize()
    for x, y in zip(a, b):
        assert rel_fro(np64(x), np64(y)) <= 2e-2


def test_tensor_backward_determinism():
    wl = small("tcbd", 1, 4, 2, 768, 128, 256, "bf16", 5300, unit=True)
    q, k, v = (t.cuda() for t in W.make_qkv(wl))
    dy = W.make_dout(wl).cuda()
    ws = R.alloc_workspace(q, k, wl.w)
    R.rattn_forward_ex(q, k, v, wl.w, scale=wl.scale, workspace=ws, save_residuals=True)
    a = [t.clone() for t in R.rattn_backward_ex(q, k, v, dy, wl.w, ws, scale=wl.scale)]
    b = R.rattn_backward_ex(q, k, v, dy, wl.w, ws, scale=wl.scale)
    for x, y in zip(a, b):
        assert torch.equal(x, y)


def test_tensor_paths_with_several_items_per_cta():
    """More (head, tile) items than the GPU has SMs, ragged T, a group of four query heads per
    K/V head: the persistent kernels walk several items per CTA with their barriers running on
    (the small shapes above give every CTA at most one item)."""
    wl = small("tcp", 6, 8, 2, 700, 128, 256, "bf16", 5400, unit=True)      # 6 tiles x 48 heads = 288 items
    y, ref, _ = run(wl)
    check(y, ref, "bf16", "persistent forward")
    errs = run_bwd(wl)
    for name, e in errs.items():
        assert e <= GRAD_TOL, (name, e, errs)


@pytest.mark.parametrize("Hq,Hkv", [(16, 4), (40, 8)])
def test_paper_head_shapes(Hq, Hkv):
    """Head counts of the paper's 3B (16 query / 4 K/V heads) and 12B (40 / 8: a group of five,
    not a power of two) models (Table 1), head size 128, forward and backward."""
    wl = small("tab1", 1, Hq, Hkv, 768, 128, 256, "bf16", 5500 + Hq, unit=True)
    y, ref, _ = run(wl)
    check(y, ref, "bf16", f"H={Hq}/{Hkv}")
    errs = run_bwd(wl)
    for name, e in errs.items():
        assert e <= GRAD_TOL, (name, e, errs)


@pytest.mark.parametrize("v_scale,clip", [(1.5e4, 6.0e4), (2.0 ** -9, None)])
def test_tensor_forward_value_range(v_scale, clip):
    """The tensor-core kernels read v through fp16 (range 6.1e-5 .. 65504 at full precision).
    Values up to 6e4 in magnitude, and values around 2^-9 (whose tails reach fp16's subnormals),
    still give the oracle's output: both norms divide the common scale of v out again."""
    wl = small("tcv", 1, 4, 2, 896, 128, 256, "bf16", 4700, unit=True)
    q, k, v = W.make_qkv(wl)
    v = v.float() * v_scale
    if clip is not None:
        v = v.clamp(-clip, clip)
        assert v.abs().max() >= 0.99 * clip
    v = v.to(torch.bfloat16)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    ws = R.alloc_workspace(qd, kd, wl.w)
    y = R.rattn_forward_ex(qd, kd, vd, wl.w, scale=wl.scale, workspace=ws)
    torch.cuda.synchronize()
    assert R.rattn_read_status(ws) == 0
    eps = 1e-6 * v_scale * v_scale      # keeps eps in the same proportion to mean(o^2)
    y2 = R.rattn_forward_ex(qd, kd, vd, wl.w, scale=wl.scale, workspace=ws, eps=eps)
    ref = O.forward(np64(q), np64(k), np64(v), wl.w, wl.scale, eps, None, None, R.MODE_RATTN)
    check(y2, ref, "bf16", f"v scale {v_scale}")
    assert torch.isfinite(y.float()).all()
