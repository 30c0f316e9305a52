"""rattn_params.layout = RATTN_LAYOUT_BTHD: q, k, v, out and the gradients as [B, T, H, d] (what a layer's
projections produce) instead of [B, H, T, d].  The arithmetic is the same, only addresses change, so every
result must equal, bit for bit, the transposed result of the default layout -- which the other tests check
against the oracle; one case here is also checked against the oracle directly."""
import numpy as np
import pytest
import torch

from oracle import rattn_oracle as O
from paper_2506_15545_b200 import binding as R
from paper_2506_15545_b200 import workloads as W
from test_gpu_parity import check, np64, small

pytestmark = pytest.mark.gpu

T_ = lambda x: x.transpose(1, 2).contiguous()          # [B,H,T,d] <-> [B,T,H,d]

CASES = [
    ("tc", 2, 4, 2, 384, 128, 128, "bf16", 0),           # tensor-core kernels, GQA
    ("tc-ragged", 1, 2, 2, 300, 128, 128, "bf16", 0),    # last tile partly beyond the sequence
    ("portable-f32", 2, 4, 2, 200, 64, 40, "f32", 0),    # portable kernels, fp32
    ("portable-bf16", 1, 3, 1, 150, 128, 24, "bf16", R.FLAG_FORCE_GENERIC),
]


@pytest.mark.parametrize("name,B,Hq,Hkv,T,d,w,dtype,flags", CASES)
def test_forward_backward_and_handoff_in_bthd_layout(name, B, Hq, Hkv, T, d, w, dtype, flags):
    wl = small(name, B, Hq, Hkv, T, d, w, dtype, 6100 + T, unit=True)
    q, k, v = (t.cuda() for t in W.make_qkv(wl))
    dy = W.make_dout(wl, "cuda")
    gs, gr = (t.cuda() for t in W.make_gains(wl))

    def run(layout):
        f = (lambda x: x) if layout == R.LAYOUT_BHTD else T_
        qq, kk, vv, dd = f(q), f(k), f(v), f(dy)
        ws = R.alloc_workspace(qq, kk, w, R.MODE_RATTN, flags | R.FLAG_SAVE_RESIDUALS, layout=layout)
        ws.zero_()
        st = torch.zeros(B, Hkv, d, d, device="cuda")
        kr = torch.zeros(B, Hkv, w, d, device="cuda", dtype=q.dtype)
        vr = torch.zeros_like(kr)
        y = R.rattn_forward_ex(qq, kk, vv, w, scale=wl.scale, workspace=ws, save_residuals=True, flags=flags,
                               gamma_swa=gs, gamma_rla=gr, state_out=st, k_ring_out=kr, v_ring_out=vr, layout=layout)
        dq, dk, dv = R.rattn_backward_ex(qq, kk, vv, dd, w, ws, scale=wl.scale, flags=flags, gamma_swa=gs,
                                         gamma_rla=gr, layout=layout)
        assert R.rattn_read_status(ws) == 0
        return [f(t) for t in (y, dq, dk, dv)] + [st, kr, vr]

    a, b = run(R.LAYOUT_BHTD), run(R.LAYOUT_BTHD)
    for what, x, z in zip(["y", "dq", "dk", "dv", "state", "k ring", "v ring"], a, b):
        assert torch.equal(x, z), what
    ref = O.forward(np64(q), np64(k), np64(v), w, wl.scale, 1e-6, np64(gs), np64(gr))
    check(b[0], ref, dtype, name)


def test_chunked_prefill_with_bthd_chunks():
    """A resumed sequence whose chunks arrive as [B, T, H, d]: the history gather reads them with their own
    strides.  Same bits as the same chunking in the default layout, and the oracle's rows within the bf16
    tolerance (as is one call on the whole sequence)."""
    wl = small("lc", 1, 4, 2, 768, 128, 128, "bf16", 6200, unit=True)
    q, k, v = (t.cuda() for t in W.make_qkv(wl))
    w, B, Hkv, d = wl.w, wl.B, wl.H_kv, wl.d
    whole = R.rattn_forward_ex(q, k, v, w, scale=wl.scale, workspace=R.alloc_workspace(q, k, w))

    def chunked(layout):
        f = (lambda x: x.contiguous()) if layout == R.LAYOUT_BHTD else T_
        st = torch.zeros(B, Hkv, d, d, device="cuda")
        kr = torch.zeros(B, Hkv, w, d, device="cuda", dtype=q.dtype)
        vr = torch.zeros_like(kr)
        outs, pos0 = [], 0
        for n in (256, 384, 128):
            sl = slice(pos0, pos0 + n)
            qq, kk, vv = f(q[:, :, sl]), f(k[:, :, sl]), f(v[:, :, sl])
            kw = dict(scale=wl.scale, state_out=st, k_ring_out=kr, v_ring_out=vr, layout=layout)
            if pos0 == 0:
                ws = R.alloc_workspace(qq, kk, w, R.MODE_RATTN, 0, layout=layout)
            else:
                ws = torch.empty(R.rattn_workspace_bytes_chunked(B, wl.H_q, Hkv, n, d, w), dtype=torch.uint8,
                                 device="cuda")
                kw.update(state_in=st, k_ring_in=kr, v_ring_in=vr, pos0=pos0)
            outs.append(f(R.rattn_forward_ex(qq, kk, vv, w, workspace=ws, **kw)))
            assert R.rattn_read_status(ws) == 0
            pos0 += n
        return torch.cat(outs, dim=2), st, kr, vr

    a, b = chunked(R.LAYOUT_BHTD), chunked(R.LAYOUT_BTHD)
    for x, z in zip(a, b):
        assert torch.equal(x, z)
    ref = O.forward(np64(q), np64(k), np64(v), w, wl.scale)
    check(b[0], ref, "bf16", "chunked, [B,T,H,d]")
    check(whole, ref, "bf16", "one call")


def test_config2_forward_in_bthd_layout():
    """Config 2 at full size (the launch configuration bench.py times): same bits in both layouts."""
    wl = W.C2
    q, k, v = W.make_qkv(wl, "cuda")
    ws = R.alloc_workspace(q, k, wl.w, R.MODE_RATTN, 0)
    a = R.rattn_forward_ex(q, k, v, wl.w, scale=wl.scale, workspace=ws)
    b = R.rattn_forward_ex(T_(q), T_(k), T_(v), wl.w, scale=wl.scale, workspace=ws, layout=R.LAYOUT_BTHD)
    assert R.rattn_read_status(ws) == 0
    assert torch.equal(T_(b), a)


def test_unknown_layout_is_refused():
    wl = small("lx", 1, 2, 1, 64, 64, 8, "bf16", 6300)
    q, k, v = (t.cuda() for t in W.make_qkv(wl))
    with pytest.raises(R.RattnError) as e:
        R.rattn_forward_ex(q, k, v, wl.w, layout=7)
    assert e.value.code == -4
