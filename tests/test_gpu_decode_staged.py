"""The decode step that streams the ring and the state through shared memory (bf16, d = 128, window a
multiple of 64, groups of up to 8 query heads) against the oracle: a prefill hand-off followed by n
steps must reproduce rows T0 .. T0+n-1 of the operator on the whole sequence.  Same tolerances as
every bf16 output (max-abs 2e-2, mean-abs 2e-3 on sums of two unit-RMS vectors)."""
import numpy as np
import pytest
import torch

from oracle import rattn_oracle as O
from paper_2506_15545_b200 import binding as R
from paper_2506_15545_b200 import workloads as W
from test_gpu_parity import check, np64, small

pytestmark = pytest.mark.gpu


def run_steps(wl, T0, steps, poison=False, phi=R.PHI_SOFTMAX, flags=0):
    B, Hq, Hkv, d, w = wl.B, wl.H_q, wl.H_kv, wl.d, wl.w
    q, k, v = W.make_qkv(wl)
    gs, gr = W.make_gains(wl)
    state = torch.zeros(B, Hkv, d, d, device="cuda")
    fill = float("nan") if poison else 0.0
    k_ring = torch.full((B, Hkv, w, d), fill, device="cuda", dtype=torch.bfloat16)
    v_ring = torch.full_like(k_ring, fill)
    if T0 > 0:
        R.rattn_forward_ex(q[:, :, :T0].contiguous().cuda(), k[:, :, :T0].contiguous().cuda(),
                           v[:, :, :T0].contiguous().cuda(), w, scale=wl.scale, phi=phi,
                           state_out=state, k_ring_out=k_ring, v_ring_out=v_ring, flags=R.FLAG_FORCE_GENERIC)
        if poison and T0 < w:                       # the hand-off zeroes the unused slots: poison them again
            k_ring[:, :, T0:] = float("nan")
            v_ring[:, :, T0:] = float("nan")
    outs = []
    for s in range(steps):
        pos = T0 + s
        outs.append(R.rattn_decode_step_ex(
            q[:, :, pos].contiguous().cuda(), k[:, :, pos].contiguous().cuda(), v[:, :, pos].contiguous().cuda(),
            k_ring, v_ring, state, pos, scale=wl.scale, gamma_swa=gs.cuda(), gamma_rla=gr.cuda(), phi=phi,
            flags=flags))
    assert R.rattn_decode_status() == 0, "a device-side wait expired"
    y = torch.stack(outs, dim=2)
    ref = O.forward(np64(q), np64(k), np64(v), w, wl.scale, 1e-6, np64(gs), np64(gr), O.MODE_RATTN, phi)[:, :, T0:]
    T = T0 + steps
    for j in range(max(0, T - w), T):
        assert torch.equal(k_ring[:, :, j % w].cpu(), k[:, :, j])
        assert torch.equal(v_ring[:, :, j % w].cpu(), v[:, :, j])
    ref_state = np.stack([[O.rla_state(np64(k[b, h]), np64(v[b, h]), T - w, phi) for h in range(Hkv)]
                          for b in range(B)])
    assert np.abs(np64(state) - ref_state).max() <= 2e-3 * max(1.0, np.abs(ref_state).max())
    return y, ref


@pytest.mark.parametrize("w,Hq,Hkv,T0,steps,poison", [
    (64, 4, 1, 0, 150, True),        # from an empty, NaN-filled cache through pos = w-1, w, w+1, 2w
    (128, 2, 2, 200, 40, False),     # group of 1
    (128, 4, 2, 200, 40, False),     # group of 2
    (128, 10, 2, 200, 24, False),    # group of 5 (the 12B shape's group)
    (128, 8, 1, 130, 24, False),     # group of 8
    (192, 8, 2, 100, 120, True),     # three pieces, prefill shorter than the window, slots poisoned
    (512, 8, 2, 700, 6, False),      # config 5's window and group
])
def test_staged_decode_after_prefill(w, Hq, Hkv, T0, steps, poison):
    wl = small("dst", 2, Hq, Hkv, T0 + steps, 128, w, "bf16", 7000 + w + Hq, unit=True)
    y, ref = run_steps(wl, T0, steps, poison)
    check(y, ref, "bf16", f"w={w} g={Hq // Hkv}")


@pytest.mark.parametrize("phi", [R.PHI_RELU, R.PHI_IDENTITY])
def test_staged_decode_other_feature_maps(phi):
    wl = small("dsp", 1, 4, 2, 230, 128, 64, "bf16", 7100 + phi, unit=True)
    y, ref = run_steps(wl, 200, 30, phi=phi)
    err = np.abs(np64(y) - ref)
    assert err.mean() <= 2e-3 and err.max() <= 2e-2 + 2.0 ** -8 * np.abs(ref).max()


def test_staged_and_portable_decode_agree():
    """The two decode kernels on the same caches: outputs within the bf16 tolerance of each other's oracle,
    rings identical, states equal to fp32 rounding."""
    wl = small("dsg", 2, 8, 2, 300, 128, 128, "bf16", 7200, unit=True)
    y1, ref = run_steps(wl, 256, 44)
    y2, _ = run_steps(wl, 256, 44, flags=R.FLAG_FORCE_GENERIC)
    check(y1, ref, "bf16", "staged")
    check(y2, ref, "bf16", "portable")
    assert (y1.float() - y2.float()).abs().max() <= 2e-2


def test_staged_decode_one_position_per_entry():
    """Batch entries at different fill levels (empty, below the window, beyond it) in one call."""
    B, Hq, Hkv, d, w = 3, 4, 2, 128, 64
    lens = [0, 40, 200]
    wl = small("dsv", B, Hq, Hkv, max(lens) + 8, d, w, "bf16", 7300, unit=True)
    q, k, v = W.make_qkv(wl)
    state = torch.zeros(B, Hkv, d, d, device="cuda")
    k_ring = torch.zeros(B, Hkv, w, d, device="cuda", dtype=torch.bfloat16)
    v_ring = torch.zeros_like(k_ring)
    for b, n in enumerate(lens):
        if n:
            R.rattn_forward_ex(q[b:b + 1, :, :n].contiguous().cuda(), k[b:b + 1, :, :n].contiguous().cuda(),
                               v[b:b + 1, :, :n].contiguous().cuda(), w, scale=wl.scale, state_out=state[b:b + 1],
                               k_ring_out=k_ring[b:b + 1], v_ring_out=v_ring[b:b + 1], flags=R.FLAG_FORCE_GENERIC)
    outs = []
    for s in range(8):
        pos = torch.tensor([n + s for n in lens], dtype=torch.int32, device="cuda")
        tok = lambda x: torch.stack([x[b, :, lens[b] + s] for b in range(B)]).contiguous().cuda()
        outs.append(R.rattn_decode_step_ex(tok(q), tok(k), tok(v), k_ring, v_ring, state, 0, scale=wl.scale,
                                           pos_dev=pos))
    assert R.rattn_decode_status() == 0
    y = torch.stack(outs, dim=2)
    for b, n in enumerate(lens):
        ref = O.forward(np64(q[b:b + 1, :, :n + 8]), np64(k[b:b + 1, :, :n + 8]), np64(v[b:b + 1, :, :n + 8]), w,
                        wl.scale)[:, :, n:]
        check(y[b:b + 1], ref, "bf16", f"entry {b}")
