"""Parity at the full benchmark sizes, in the launch configuration bench.py times, on sampled
outputs: every output row of the operator depends on its own query row and on the K/V history
of its head only, so the fp64 oracle can evaluate any row of any head on its own
(`forward_rows`).  Rows are sampled at the places where the kernels switch behaviour: the start
of the sequence, t = w and w + 1, tile edges, the last rows, plus random ones.  Gradients are
compared for whole heads (the oracle's dense backward of one head at T = 4096 takes seconds).
Tolerances as everywhere: bf16 outputs max-abs <= 2e-2 and mean-abs <= 2e-3, gradients
<= 5e-2 relative Frobenius norm."""
import numpy as np
import pytest
import torch

from oracle import rattn_oracle as O
from paper_2506_15545_b200 import binding as R
from paper_2506_15545_b200 import workloads as W
from test_gpu_parity import GRAD_TOL, TOL, np64, rel_fro

pytestmark = pytest.mark.gpu


def sample_rows(T, w, n_random, seed):
    fixed = [0, 1, 63, 64, 127, 128, 129, w - 1, w, w + 1, w + 127, w + 128, w + 129, 2 * w, 2 * w + 1,
             T // 2 - 1, T // 2, T - 130, T - 129, T - 128, T - 2, T - 1]
    rng = np.random.default_rng(seed)
    rows = set(t for t in fixed if 0 <= t < T)
    rows.update(int(t) for t in rng.integers(0, T, n_random))
    return np.array(sorted(rows))


def check_sampled_forward(wl, y, q, k, v, pairs, mode=R.MODE_RATTN, n_random=48):
    g = wl.H_q // wl.H_kv
    errs = []
    for b, h in pairs:
        rows = sample_rows(wl.T, min(wl.w, wl.T - 1), n_random, 17 * b + h)
        ref = O.forward_rows(np64(q[b, h]), np64(k[b, h // g]), np64(v[b, h // g]), rows, wl.w, wl.scale,
                             mode=mode)
        got = np64(y[b, h][torch.as_tensor(rows, device=y.device)])
        assert np.isfinite(got).all()
        errs.append(np.abs(got - ref))
    err = np.concatenate(errs)
    assert err.max() <= TOL["bf16"]["max_abs"], err.max()
    assert err.mean() <= TOL["bf16"]["mean_abs"], err.mean()


def forward_full(wl, mode=R.MODE_RATTN, save=False):
    assert R.rattn_uses_tensor_path(wl.d, wl.w, R.RATTN_BF16, mode)
    q, k, v = W.make_qkv(wl, "cuda")
    # exactly what this call needs: an inference forward keeps only the chunk states
    ws = R.alloc_workspace(q, k, wl.w, mode, R.FLAG_SAVE_RESIDUALS if save else 0)
    y = R.rattn_forward_ex(q, k, v, wl.w, scale=wl.scale, mode=mode, workspace=ws, save_residuals=save)
    torch.cuda.synchronize()
    assert R.rattn_read_status(ws) == 0, "a device-side wait expired"
    return q, k, v, y, ws


def test_config2_forward_full_size():
    """B=4, H=16/16, T=4096, d=128, w=512, unit-RMS q/k."""
    wl = W.C2
    q, k, v, y, _ = forward_full(wl)
    check_sampled_forward(wl, y, q, k, v, [(0, 0), (1, 7), (3, 15)])


@pytest.mark.parametrize("w,mode", [(128, R.MODE_RATTN), (256, R.MODE_RATTN), (512, R.MODE_RATTN),
                                    (1024, R.MODE_RATTN), (2048, R.MODE_RATTN), (4096, R.MODE_RATTN),
                                    (512, R.MODE_SWA_ONLY), (2048, R.MODE_SWA_ONLY), (512, R.MODE_FULL_CAUSAL)])
def test_config3_gqa_windows_and_controls(w, mode):
    """B=2, H=32/8, T=8192: every window of the sweep, SWA-only and full-causal controls."""
    wl = W.C3.replace(w=w)
    q, k, v, y, _ = forward_full(wl, mode)
    check_sampled_forward(wl, y, q, k, v, [(0, 0), (1, 29)], mode=mode, n_random=32)


def test_config4_training_step_full_size():
    """B=8, H=16/16, T=4096, w=512: forward rows sampled, gradients of two whole heads."""
    wl = W.C4
    q, k, v, y, ws = forward_full(wl, save=True)
    check_sampled_forward(wl, y, q, k, v, [(0, 3), (7, 12)], n_random=32)
    dy = W.make_dout(wl, "cuda")
    dq, dk, dv = R.rattn_backward_ex(q, k, v, dy, wl.w, ws, scale=wl.scale)
    torch.cuda.synchronize()
    assert R.rattn_read_status(ws) == 0
    for b, h in [(0, 3), (7, 12)]:            # H_q == H_kv: dk, dv of a K/V head come from one query head
        ref = O.backward_head(np64(q[b, h]), np64(k[b, h]), np64(v[b, h]), np64(dy[b, h]), wl.w, wl.scale)
        for name, got, want in zip(("dq", "dk", "dv"), (dq[b, h], dk[b, h], dv[b, h]), ref):
            assert np.isfinite(np64(got)).all(), name
            assert rel_fro(np64(got), want) <= GRAD_TOL, (name, b, h, rel_fro(np64(got), want))


def _prefill_then_decode(wl, pairs, n_random=32):
    q, k, v, y, ws = forward_full(wl)
    check_sampled_forward(wl, y, q, k, v, pairs, n_random=n_random)
    del y
    # hand-off, then decode with fresh tokens
    state = torch.zeros(wl.B, wl.H_kv, wl.d, wl.d, device="cuda")
    k_ring = torch.zeros(wl.B, wl.H_kv, wl.w, wl.d, device="cuda", dtype=torch.bfloat16)
    v_ring = torch.zeros_like(k_ring)
    out = torch.empty_like(q)
    R.rattn_forward_ex(q, k, v, wl.w, scale=wl.scale, workspace=ws, state_out=state, k_ring_out=k_ring,
                       v_ring_out=v_ring, out=out)
    del out
    steps = wl.decode_steps
    toks = [W.make_decode_token(wl, s, "cuda") for s in range(steps)]
    outs = [R.rattn_decode_step_ex(tq, tk, tv, k_ring, v_ring, state, wl.T + s, scale=wl.scale)
            for s, (tq, tk, tv) in enumerate(toks)]
    torch.cuda.synchronize()
    assert R.rattn_read_status(ws) == 0
    yd = torch.stack(outs, dim=2)                              # [B, H_q, steps, d]
    g = wl.H_q // wl.H_kv
    errs = []
    for b, h in pairs:
        qh = np.concatenate([np64(q[b, h]), np64(torch.stack([t[0][b, h] for t in toks]))])
        kh = np.concatenate([np64(k[b, h // g]), np64(torch.stack([t[1][b, h // g] for t in toks]))])
        vh = np.concatenate([np64(v[b, h // g]), np64(torch.stack([t[2][b, h // g] for t in toks]))])
        rows = np.arange(wl.T, wl.T + steps)
        ref = O.forward_rows(qh, kh, vh, rows, wl.w, wl.scale)
        errs.append(np.abs(np64(yd[b, h]) - ref))
    err = np.concatenate(errs)
    assert err.max() <= TOL["bf16"]["max_abs"], err.max()
    assert err.mean() <= TOL["bf16"]["mean_abs"], err.mean()


def test_config5_long_prefill_then_decode_full_batch():
    """The configuration as stated: B=32, H=32/8, d=128, w=512, prefill T=32768 (q, k, v, out
    21.5 GB, chunk states 2.1 GB), then 256 decode steps with the ring and state the prefill
    hands over.  256 K/V heads, each a chain of 256 chunk steps in the state kernel (two waves of CTAs),
    which also leaves the fp32 decode state.  Oracle on sampled rows of three heads and on all 256 decode rows."""
    _prefill_then_decode(W.C5, [(0, 0), (13, 6), (31, 31)], n_random=24)


def test_config5_few_heads():
    """Four batch entries of the same configuration (32 K/V heads in all): the chunk-state chains
    occupy only 32 SMs while the main kernel already runs on the others."""
    _prefill_then_decode(W.C5.replace(B=4), [(0, 0), (3, 31)])


def test_config3_prefill_in_four_chunks():
    """B=2, H=32/8, T=8192, w=512 cut into four chunks of 2048 tokens, each resuming from the ring and
    state the previous one handed out (tensor-core kernels throughout): sampled rows against the oracle
    on the whole sequence, and the final state against the one-pass hand-off."""
    wl = W.C3
    q, k, v = W.make_qkv(wl, "cuda")
    C = 2048
    state = torch.zeros(wl.B, wl.H_kv, wl.d, wl.d, device="cuda")
    k_ring = torch.zeros(wl.B, wl.H_kv, wl.w, wl.d, device="cuda", dtype=torch.bfloat16)
    v_ring = torch.zeros_like(k_ring)
    y = torch.empty_like(q)
    for c in range(wl.T // C):
        sl = slice(c * C, (c + 1) * C)
        qc, kc, vc = (t[:, :, sl].contiguous() for t in (q, k, v))
        kw = dict(scale=wl.scale, state_out=state, k_ring_out=k_ring, v_ring_out=v_ring)
        if c == 0:
            ws = R.alloc_workspace(qc, kc, wl.w, R.MODE_RATTN, 0)
        else:
            ws = R.alloc_workspace_chunked(qc, kc, wl.w)
            kw.update(state_in=state, k_ring_in=k_ring, v_ring_in=v_ring, pos0=c * C)
        y[:, :, sl] = R.rattn_forward_ex(qc, kc, vc, wl.w, workspace=ws, **kw)
        torch.cuda.synchronize()
        assert R.rattn_read_status(ws) == 0
    check_sampled_forward(wl, y, q, k, v, [(0, 5), (1, 30)], n_random=48)
    one_pass = torch.zeros_like(state)
    ws = R.alloc_workspace(q, k, wl.w, R.MODE_RATTN, 0)
    R.rattn_forward_ex(q, k, v, wl.w, scale=wl.scale, workspace=ws, state_out=one_pass)
    torch.cuda.synchronize()
    assert (state - one_pass).abs().max().item() <= 2.0 ** -8 * max(1.0, one_pass.abs().max().item())
