"""Parity of the qk-norm + rotary prologue kernels, their gradient, and a local/global layer stack
built on them, against the fp64 oracle.

Tolerances.  fp32 I/O: the kernel's arithmetic is fp32 with the angle reduced in fp64, so errors are
a few ulp of values of size <= |gain| * sqrt(d): 2e-5 absolute.  bf16 I/O: the result is rounded
once to bf16, half an ulp = 2^-9 relative, plus the same fp32 noise: |err| <= 2^-8 |ref| + 1e-5.
Gain gradients are sums over B*H*T rows of O(1) terms in fp32: relative 1e-4 of the largest entry
(bf16 inputs are exact in fp32, so the same bound holds for both types)."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import prologue_oracle as P
from oracle import rattn_oracle as O
from paper_2506_15545_b200 import binding as R
from test_gpu_parity import np64, rel_fro

pytestmark = pytest.mark.gpu


def make(B, Hq, Hkv, T, d, dtype, seed, gains=True):
    g = torch.Generator().manual_seed(seed)
    dt = torch.bfloat16 if dtype == "bf16" else torch.float32
    q = (torch.randn(B, Hq, T, d, generator=g) * 1.7).to(dt)
    k = (torch.randn(B, Hkv, T, d, generator=g) * 0.6).to(dt)
    gq = (1.0 + 0.2 * torch.randn(d, generator=g)) if gains else None
    gk = (1.0 + 0.2 * torch.randn(d, generator=g)) if gains else None
    return q, k, gq, gk


def close(got, ref, dtype, what):
    got = np64(got)
    assert np.isfinite(got).all(), what
    err = np.abs(got - ref)
    bound = (2.0 ** -8) * np.abs(ref) + 1e-5 if dtype == "bf16" else np.full_like(ref, 2e-5)
    assert (err <= bound).all(), (what, float(err.max()), float((err - bound).max()))


def cu(t):
    return None if t is None else t.cuda()


@pytest.mark.parametrize("B,Hq,Hkv,T,d,dtype,pos0,theta", [
    (2, 4, 2, 300, 128, "bf16", 0, 5.0e5),        # several row blocks and a ragged tail
    (2, 4, 2, 300, 128, "f32", 0, 5.0e5),
    (1, 3, 1, 77, 64, "f32", 1000, 5.0e5),        # d = 64, odd head counts
    (1, 40, 8, 129, 128, "bf16", 0, 5.0e5),       # 48 heads: six head slices per batch entry
    (1, 2, 2, 64, 128, "f32", 131072 - 64, 5.0e5),  # positions near 2^17: angles up to 1.3e5 rad
    (1, 2, 2, 64, 128, "f32", 2 ** 30, 5.0e5),    # a position fp32 could not even hold exactly + 1
    (2, 2, 1, 200, 128, "bf16", 0, None),         # global layer: norm only
    (2, 2, 1, 50, 64, "f32", 7, 1.0e4),           # another base
    (3, 16, 4, 1100, 128, "bf16", 0, 5.0e5),      # more chunks than stages in every CTA
    (2, 8, 8, 700, 64, "bf16", 3, 5.0e5),         # d = 64, bf16: 64 rows per chunk
])
def test_prologue_forward(B, Hq, Hkv, T, d, dtype, pos0, theta):
    q, k, gq, gk = make(B, Hq, Hkv, T, d, dtype, 9000 + T + d)
    qo, ko = R.rattn_qk_prologue(q.cuda(), k.cuda(), q_gain=cu(gq), k_gain=cu(gk), theta=theta, pos0=pos0)
    assert R.rattn_qk_prologue_status() == 0, "a device-side wait expired"
    pos = pos0 + np.arange(T)
    close(qo, P.qk_prologue(np64(q), np64(gq), pos, theta), dtype, "q")
    close(ko, P.qk_prologue(np64(k), np64(gk), pos, theta), dtype, "k")


def test_prologue_in_place_one_tensor_and_per_entry_positions():
    q, k, gq, gk = make(3, 4, 2, 40, 128, "bf16", 9100)
    qd, kd = q.cuda(), k.cuda()
    pos = torch.tensor([5, 70000, 0], dtype=torch.int32)
    qo, ko = R.rattn_qk_prologue(qd, kd, q_gain=cu(gq), k_gain=cu(gk), pos=pos.cuda())
    for b in range(3):
        p = int(pos[b]) + np.arange(40)
        close(qo[b], P.qk_prologue(np64(q[b]), np64(gq), p, P.THETA_LOCAL), "bf16", f"q entry {b}")
        close(ko[b], P.qk_prologue(np64(k[b]), np64(gk), p, P.THETA_LOCAL), "bf16", f"k entry {b}")
    # one tensor only
    q1, none = R.rattn_qk_prologue(qd, None, q_gain=cu(gq), pos=pos.cuda())
    assert none is None and torch.equal(q1, qo)
    # in place gives the same bits and touches nothing else
    q2, k2 = qd.clone(), kd.clone()
    r = R.rattn_qk_prologue(q2, k2, q_gain=cu(gq), k_gain=cu(gk), pos=pos.cuda(), inplace=True)
    assert r[0] is q2 and torch.equal(q2, qo) and torch.equal(k2, ko)


def test_prologue_decode_shape():
    """T = 1 with a position per batch entry: what a decode step applies to its new token."""
    q, k, gq, gk = make(5, 8, 2, 1, 128, "bf16", 9200)
    pos = torch.tensor([0, 1, 511, 4096, 131071], dtype=torch.int32)
    qo, ko = R.rattn_qk_prologue(q.cuda(), k.cuda(), q_gain=cu(gq), k_gain=cu(gk), pos=pos.cuda())
    for b in range(5):
        close(qo[b], P.qk_prologue(np64(q[b]), np64(gq), pos[b:b + 1].numpy(), P.THETA_LOCAL), "bf16", f"q {b}")
        close(ko[b], P.qk_prologue(np64(k[b]), np64(gk), pos[b:b + 1].numpy(), P.THETA_LOCAL), "bf16", f"k {b}")


@pytest.mark.parametrize("B,Hq,Hkv,T,d,dtype,theta", [
    (2, 4, 2, 300, 128, "f32", 5.0e5),
    (2, 4, 2, 300, 128, "bf16", 5.0e5),
    (1, 3, 1, 77, 64, "f32", 5.0e5),
    (2, 16, 16, 130, 128, "bf16", None),
    (3, 16, 4, 1100, 128, "bf16", 5.0e5),         # long enough for the ring to wrap in every CTA
    (2, 8, 8, 700, 64, "f32", 5.0e5),
])
def test_prologue_backward(B, Hq, Hkv, T, d, dtype, theta):
    q, k, gq, gk = make(B, Hq, Hkv, T, d, dtype, 9300 + T)
    g = torch.Generator().manual_seed(77)
    dqo = torch.randn(q.shape, generator=g).to(q.dtype)
    dko = torch.randn(k.shape, generator=g).to(k.dtype)
    pos0 = 12345
    out = R.rattn_qk_prologue_backward(q.cuda(), k.cuda(), dqo.cuda(), dko.cuda(), q_gain=cu(gq), k_gain=cu(gk),
                                       theta=theta, pos0=pos0)
    out2 = R.rattn_qk_prologue_backward(q.cuda(), k.cuda(), dqo.cuda(), dko.cuda(), q_gain=cu(gq), k_gain=cu(gk),
                                        theta=theta, pos0=pos0)
    torch.cuda.synchronize()
    pos = pos0 + np.arange(T)
    for name, x, gain, dy, dx, dg, dx2, dg2 in [("q", q, gq, dqo, out[0], out[2], out2[0], out2[2]),
                                                ("k", k, gk, dko, out[1], out[3], out2[1], out2[3])]:
        rx, rg = P.qk_prologue_bwd(np64(x), np64(gain), pos, theta, np64(dy))
        err = np.abs(np64(dx) - rx)
        bound = (2.0 ** -8) * np.abs(rx) + 2e-5 if dtype == "bf16" else 5e-5 * (1 + np.abs(rx))
        assert (err <= bound).all(), (name, float(err.max()))
        assert np.abs(np64(dg) - rg).max() <= 1e-4 * np.abs(rg).max(), name
        assert torch.equal(dx, dx2) and torch.equal(dg, dg2), "run-to-run bits"
    assert R.rattn_qk_prologue_status() == 0
    # without gain gradients no workspace is needed and the input gradients are the same bits
    out3 = R.rattn_qk_prologue_backward(q.cuda(), k.cuda(), dqo.cuda(), dko.cuda(), q_gain=cu(gq), k_gain=cu(gk),
                                        theta=theta, pos0=pos0, gain_grads=False)
    assert out3[2] is None and torch.equal(out3[0], out[0]) and torch.equal(out3[1], out[1])


def test_prologue_full_size_sampled_rows():
    """Config 2's q and k tensors (B=4, 16/16 heads, T=4096, d=128, bf16): rows sampled across
    batch entries, heads and positions against the oracle, one by one."""
    B, H, T, d = 4, 16, 4096, 128
    q, k, gq, gk = make(B, H, H, T, d, "bf16", 9400)
    qo, ko = R.rattn_qk_prologue(q.cuda(), k.cuda(), q_gain=cu(gq), k_gain=cu(gk))
    torch.cuda.synchronize()
    r = np.random.default_rng(5)
    for _ in range(200):
        b, h, t = int(r.integers(B)), int(r.integers(H)), int(r.integers(T))
        if _ < 8:
            t = [0, 1, 31, 32, T - 33, T - 32, T - 2, T - 1][_]
        close(qo[b, h, t], P.qk_prologue(np64(q[b, h, t:t + 1]), np64(gq), np.array([t]), P.THETA_LOCAL)[0],
              "bf16", f"q {b},{h},{t}")
        close(ko[b, h, t], P.qk_prologue(np64(k[b, h, t:t + 1]), np64(gk), np.array([t]), P.THETA_LOCAL)[0],
              "bf16", f"k {b},{h},{t}")


def test_prologue_argument_checks():
    q, k, gq, gk = make(1, 2, 1, 16, 128, "bf16", 9500)
    qd, kd = q.cuda(), k.cuda()
    with pytest.raises(R.RattnError) as e:
        R.rattn_qk_prologue(qd[..., :32].contiguous(), None)           # d = 32
    assert e.value.code == -4
    with pytest.raises(R.RattnError) as e:
        R.rattn_qk_prologue(qd, kd, pos0=-1)
    assert e.value.code == -1
    with pytest.raises(R.RattnError) as e:
        R.rattn_qk_prologue(qd, kd, eps=float("nan"))
    assert e.value.code == -1
    with pytest.raises(R.RattnError) as e:                             # gain gradients without room for them
        R.rattn_qk_prologue_backward(qd, kd, qd, kd, workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
    assert e.value.code == -5


# ---------------------------------------------------------------- a stack of attention layers
def gpu_layer(x, lay, *, H_q, H_kv, d, w, local, scale, dt, layout, flags=0):
    """The oracle's layer with the library's kernels for the prologue and the operator, and torch
    for what surrounds them (RMS norm of the layer input, the four projections, the residual add).
    With the [B, T, H, d] layout the projections' outputs are used as they are: no transposing copy."""
    Wq, Wk, Wv, Wo, gq, gk = lay
    B, T, D = x.shape
    h = F.rms_norm(x, (D,), eps=1e-6).to(dt)
    if layout == R.LAYOUT_BTHD:
        heads = lambda z, H: z.reshape(B, T, H, d)
        merge = lambda y: y.reshape(B, T, H_q * d)
    else:
        heads = lambda z, H: z.reshape(B, T, H, d).transpose(1, 2).contiguous()
        merge = lambda y: y.transpose(1, 2).reshape(B, T, H_q * d)
    q, k, v = heads(h @ Wq.to(dt), H_q), heads(h @ Wk.to(dt), H_kv), heads(h @ Wv.to(dt), H_kv)
    R.rattn_qk_prologue(q, k, q_gain=gq, k_gain=gk, theta=P.THETA_LOCAL if local else None, inplace=True,
                        layout=layout)
    mode = R.MODE_RATTN if local else R.MODE_FULL_CAUSAL
    ws = R.alloc_workspace(q, k, w, mode, flags, layout=layout)
    y = R.rattn_forward_ex(q, k, v, w, scale=scale, mode=mode, workspace=ws, flags=flags, layout=layout)
    assert R.rattn_read_status(ws) == 0
    return x + (merge(y) @ Wo.to(dt)).float()


@pytest.mark.parametrize("layout", [R.LAYOUT_BHTD, R.LAYOUT_BTHD])
@pytest.mark.parametrize("dtype,D,H_q,H_kv,d,T,w,tol", [
    ("f32", 128, 4, 2, 64, 160, 32, 2e-4),       # portable fp32 kernels
    ("bf16", 256, 4, 2, 128, 640, 128, 3e-2),    # tensor-core kernels
])
def test_local_local_local_global_stack(dtype, D, H_q, H_kv, d, T, w, tol, layout):
    """Three local layers (RAttention with rotary q, k) and one global layer (full causal attention,
    no rotary), Section 4 "Model Setup", on synthetic weights: relative Frobenius error of the
    final residual stream.  bf16: every layer rounds q, k, v, y to bf16 and the operator's own error
    (2e-3 mean on unit-RMS outputs) enters the stream four times."""
    g = torch.Generator().manual_seed(9600)
    dt = torch.bfloat16 if dtype == "bf16" else torch.float32
    rnd = lambda *s: torch.randn(*s, generator=g)
    x = rnd(2, T, D)
    layers = []
    for _ in range(4):
        lay = (rnd(D, H_q * d) / math.sqrt(D), rnd(D, H_kv * d) / math.sqrt(D), rnd(D, H_kv * d) / math.sqrt(D),
               rnd(H_q * d, D) / math.sqrt(H_q * d), 1.0 + 0.1 * rnd(d), 1.0 + 0.1 * rnd(d))
        layers.append(tuple(t.to(dt).float() if i < 4 else t for i, t in enumerate(lay)))
    scale = 1.0 / math.sqrt(d)
    ref = P.attention_stack(np64(x), [tuple(np64(t) for t in lay) for lay in layers],
                            H_q=H_q, H_kv=H_kv, d=d, w=w, scale=scale)
    y = x.cuda()
    for l, lay in enumerate(layers):
        if dtype == "bf16":
            assert R.rattn_uses_tensor_path(d, w, R.RATTN_BF16, R.MODE_RATTN)
        y = gpu_layer(y, tuple(t.cuda() for t in lay), H_q=H_q, H_kv=H_kv, d=d, w=w, local=(l + 1) % 4 != 0,
                      scale=scale, dt=dt, layout=layout)
    torch.cuda.synchronize()
    assert rel_fro(np64(y), ref) <= tol, rel_fro(np64(y), ref)


@pytest.mark.parametrize("B,Hq,Hkv,T,d,dtype,theta", [
    (2, 16, 4, 300, 128, "bf16", 5.0e5),      # 16 and 4 heads: two and eight positions per chunk
    (1, 40, 8, 130, 128, "f32", 5.0e5),       # 40 heads: a chunk is part of one position's heads
    (2, 3, 1, 77, 64, "bf16", 5.0e5),         # head counts that do not divide the chunk
    (2, 4, 2, 200, 128, "bf16", None),
])
def test_prologue_in_bthd_layout(B, Hq, Hkv, T, d, dtype, theta):
    """[B, T, H, d] tensors: forward outputs and input gradients carry the same bits as the default layout
    (the same arithmetic per head vector); gain gradients are summed in another order."""
    q, k, gq, gk = make(B, Hq, Hkv, T, d, dtype, 9700 + T)
    g = torch.Generator().manual_seed(78)
    dqo = torch.randn(q.shape, generator=g).to(q.dtype)
    dko = torch.randn(k.shape, generator=g).to(k.dtype)
    tr = lambda x: x.transpose(1, 2).contiguous()
    pos = torch.arange(B, dtype=torch.int32) * 1000 + 17
    kw = dict(q_gain=cu(gq), k_gain=cu(gk), theta=theta, pos=pos.cuda())
    qa, ka = R.rattn_qk_prologue(q.cuda(), k.cuda(), **kw)
    qb, kb = R.rattn_qk_prologue(tr(q).cuda(), tr(k).cuda(), layout=R.LAYOUT_BTHD, **kw)
    assert torch.equal(tr(qb), qa) and torch.equal(tr(kb), ka)
    ga = R.rattn_qk_prologue_backward(q.cuda(), k.cuda(), dqo.cuda(), dko.cuda(), **kw)
    gb = R.rattn_qk_prologue_backward(tr(q).cuda(), tr(k).cuda(), tr(dqo).cuda(), tr(dko).cuda(),
                                      layout=R.LAYOUT_BTHD, **kw)
    assert torch.equal(tr(gb[0]), ga[0]) and torch.equal(tr(gb[1]), ga[1])
    for x, y in ((ga[2], gb[2]), (ga[3], gb[3])):
        assert (x - y).abs().max() <= 1e-4 * x.abs().max()
    assert R.rattn_qk_prologue_status() == 0
    for b in range(B):
        p = int(pos[b]) + np.arange(T)
        close(tr(qb)[b], P.qk_prologue(np64(q[b]), np64(gq), p, theta), dtype, f"q entry {b}")
