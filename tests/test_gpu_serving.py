"""Serving-side use of the operator: a prefill cut into chunks that resume from the (ring, state)
pair the previous chunk handed out, batches whose entries have different lengths, and decode steps
whose batch entries stand at different positions.  Every result is compared with the fp64 oracle
evaluated on each entry's whole sequence (it has no ring, no state, no chunks)."""
import numpy as np
import pytest
import torch

from oracle import rattn_oracle as O
from paper_2506_15545_b200 import binding as R
from paper_2506_15545_b200 import workloads as W
from test_gpu_parity import TOL, check, np64, small

pytestmark = pytest.mark.gpu


def _buffers(B, Hkv, w, d, dt):
    state = torch.zeros(B, Hkv, d, d, device="cuda")
    k_ring = torch.zeros(B, Hkv, w, d, device="cuda", dtype=dt)
    return state, k_ring, torch.zeros_like(k_ring)


@pytest.mark.parametrize("d,w,chunks,dtype,Hq,Hkv", [
    (64, 16, (40, 33, 27, 16), "f32", 2, 1),
    (64, 8, (8, 8, 9), "bf16", 4, 2),                 # first chunk exactly w tokens
    (128, 128, (256, 200, 131), "bf16", 4, 2),        # shapes of the tensor-core path
])
def test_chunked_prefill_equals_one_pass(d, w, chunks, dtype, Hq, Hkv):
    B, T = 2, sum(chunks)
    wl = small("cp", B, Hq, Hkv, T, d, w, dtype, 8200 + d + w, unit=True)
    q, k, v = W.make_qkv(wl)
    gs, gr = W.make_gains(wl)
    state, k_ring, v_ring = _buffers(B, Hkv, w, d, wl.torch_dtype)
    outs, pos0 = [], 0
    for n in chunks:
        sl = slice(pos0, pos0 + n)
        qc, kc, vc = (t[:, :, sl].contiguous().cuda() for t in (q, k, v))
        if pos0 == 0:
            ws = R.alloc_workspace(qc, kc, w, R.MODE_RATTN, 0)
            y = R.rattn_forward_ex(qc, kc, vc, w, scale=wl.scale, workspace=ws, gamma_swa=gs.cuda(),
                                   gamma_rla=gr.cuda(), state_out=state, k_ring_out=k_ring, v_ring_out=v_ring)
        else:
            ws = R.alloc_workspace_chunked(qc, kc, w)
            # the same buffers in and out: the hand-off is written after the chunk has read them
            y = R.rattn_forward_ex(qc, kc, vc, w, scale=wl.scale, workspace=ws, gamma_swa=gs.cuda(),
                                   gamma_rla=gr.cuda(), state_in=state, k_ring_in=k_ring, v_ring_in=v_ring,
                                   pos0=pos0, state_out=state, k_ring_out=k_ring, v_ring_out=v_ring)
        torch.cuda.synchronize()
        assert R.rattn_read_status(ws) == 0
        outs.append(y)
        pos0 += n
    ref = O.forward(np64(q), np64(k), np64(v), w, wl.scale, 1e-6, np64(gs), np64(gr))
    check(torch.cat(outs, dim=2), ref, dtype, "chunked prefill")
    ref_state = np.stack([[O.rla_state(np64(k[b, h]), np64(v[b, h]), T - w) for h in range(Hkv)] for b in range(B)])
    # the tensor-core state kernel multiplies phi(k) rounded to bf16 (relative 2^-9 per term, fp32 sums)
    assert np.abs(np64(state) - ref_state).max() <= 2.0 ** -8 * max(1.0, np.abs(ref_state).max())
    for j in range(T - w, T):
        assert torch.equal(k_ring[:, :, j % w].cpu(), k[:, :, j]) and torch.equal(v_ring[:, :, j % w].cpu(), v[:, :, j])


def test_serving_paths_with_states_taken_as_published():
    """The same chunked prefill (a resumed chunk's chain starts from the incoming state, which is its
    first published matrix) and variable-length batch (every entry's chain has its own length) with
    the main kernel reading each chunk state as soon as it is published, which by default only long
    sequences on few heads do."""
    prev = R.rattn_tune(R.TUNE_STATE_PROGRESS, 1)
    try:
        test_chunked_prefill_equals_one_pass(128, 128, (256, 200, 131), "bf16", 4, 2)
        test_chunked_prefill_equals_one_pass(128, 256, (768, 640, 300), "bf16", 2, 1)
        test_variable_length_batch(128, 128, "bf16")
    finally:
        R.rattn_tune(R.TUNE_STATE_PROGRESS, prev)


def test_chunked_prefill_argument_checks():
    wl = small("cpa", 1, 2, 1, 32, 64, 16, "bf16", 1)
    q, k, v = (t.cuda() for t in W.make_qkv(wl))
    state, k_ring, v_ring = _buffers(1, 1, 16, 64, torch.bfloat16)
    ws = R.alloc_workspace_chunked(q, k, 16)
    kw = dict(workspace=ws, state_in=state, k_ring_in=k_ring, v_ring_in=v_ring)
    for bad, code in ((dict(kw, pos0=5), -1),                           # fewer than w tokens before the chunk
                      (dict(kw, pos0=32, state_in=None), -2),
                      (dict(kw, pos0=32, workspace=None), -5),
                      (dict(kw, pos0=32, save_residuals=True), -4)):      # forward only
        with pytest.raises(R.RattnError) as ei:
            R.rattn_forward_ex(q, k, v, 16, **bad)
        assert ei.value.code == code, bad.keys()


@pytest.mark.parametrize("d,w,dtype", [(64, 12, "f32"), (128, 128, "bf16")])
def test_variable_length_batch(d, w, dtype):
    """Entries of different lengths in one call: valid rows match the oracle on that entry alone,
    tiles wholly beyond an entry's length are not touched, and ring and state are taken at its own length."""
    B, Hq, Hkv, T = 3, 4, 2, 3 * w + 41
    lens = [T, T - 37, 5]
    wl = small("vl", B, Hq, Hkv, T, d, w, dtype, 8300 + d, unit=True)
    q, k, v = W.make_qkv(wl)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    out = torch.full_like(qd, 7.0)
    state, k_ring, v_ring = _buffers(B, Hkv, w, d, wl.torch_dtype)
    R.rattn_forward_ex(qd, kd, vd, w, scale=wl.scale, out=out, state_out=state, k_ring_out=k_ring,
                       v_ring_out=v_ring, seq_lens=torch.tensor(lens, dtype=torch.int32, device="cuda"),
                       workspace=R.alloc_workspace(qd, kd, w))
    torch.cuda.synchronize()
    for b, n in enumerate(lens):
        ref = O.forward(np64(q[b:b + 1, :, :n]), np64(k[b:b + 1, :, :n]), np64(v[b:b + 1, :, :n]), w, wl.scale)
        check(out[b:b + 1, :, :n], ref, dtype, f"entry {b}")
        assert torch.all(out[b, :, (n + 127) // 128 * 128:] == 7.0)
        for h in range(Hkv):
            want = O.rla_state(np64(k[b, h, :n]), np64(v[b, h, :n]), n - w)
            assert np.abs(np64(state[b, h]) - want).max() <= 2.0 ** -8 * max(1.0, np.abs(want).max())
        for j in range(max(0, n - w), n):
            assert torch.equal(k_ring[b, :, j % w].cpu(), k[b, :, j])


def test_decode_with_one_position_per_batch_entry():
    """After a variable-length prefill every entry decodes from its own position."""
    B, Hq, Hkv, d, w, T, steps = 3, 4, 2, 64, 8, 50, 12
    lens = [30, 9, 21]
    wl = small("pp", B, Hq, Hkv, T, d, w, "bf16", 8400, unit=True)
    q, k, v = W.make_qkv(wl)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    state, k_ring, v_ring = _buffers(B, Hkv, w, d, torch.bfloat16)
    T0 = max(lens)
    R.rattn_forward_ex(qd[:, :, :T0].contiguous(), kd[:, :, :T0].contiguous(), vd[:, :, :T0].contiguous(), w,
                       scale=wl.scale, state_out=state, k_ring_out=k_ring, v_ring_out=v_ring,
                       seq_lens=torch.tensor(lens, dtype=torch.int32, device="cuda"))
    got = []
    for s in range(steps):
        pos = torch.tensor([n + s for n in lens], dtype=torch.int32, device="cuda")
        tok = [torch.stack([t[b, :, lens[b] + s] for b in range(B)]).contiguous().cuda() for t in (q, k, v)]
        got.append(R.rattn_decode_step_ex(*tok, k_ring, v_ring, state, 0, scale=wl.scale, pos_dev=pos))
    torch.cuda.synchronize()
    y = torch.stack(got, dim=2)                      # [B, H_q, steps, d]
    for b, n in enumerate(lens):
        ref = O.forward(np64(q[b:b + 1, :, :n + steps]), np64(k[b:b + 1, :, :n + steps]),
                        np64(v[b:b + 1, :, :n + steps]), w, wl.scale)[:, :, n:]
        check(y[b:b + 1], ref, "bf16", f"entry {b}")
