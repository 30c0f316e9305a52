"""Pins of the prologue oracle (qk-norm, rotary embedding, their gradient, the layer built from
them) against things it does not compute itself: closed forms, the complex-number form of the
rotation in torch, torch's rms_norm and scaled_dot_product_attention, autograd and central
differences."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import prologue_oracle as P
from oracle import rattn_oracle as O


def rng(seed):
    return np.random.default_rng(seed)


def torch_rope_complex(x, pos, theta):
    """Independent coding: pairs (i, i + d/2) as complex numbers times exp(i * angle)."""
    x = torch.as_tensor(x, dtype=torch.float64)
    d = x.shape[-1]
    z = torch.complex(x[..., : d // 2], x[..., d // 2:])
    inv = torch.exp(-torch.arange(d // 2, dtype=torch.float64) * (2.0 / d) * math.log(theta))
    ang = torch.as_tensor(pos, dtype=torch.float64)[:, None] * inv[None, :]
    z = z * torch.polar(torch.ones_like(ang), ang)
    return torch.cat([z.real, z.imag], dim=-1)


def test_rope_hand_computed_vector():
    """d = 4, theta = 5e5, position 3: pair (x0, x2) turns by 3 rad, pair (x1, x3) by
    3 / sqrt(5e5) = 3 / 707.1067811865476 rad."""
    y = P.rope(np.array([[1.0, 2.0, 3.0, 4.0]]), np.array([3]), 5.0e5)[0]
    a0, a1 = 3.0, 3.0 / 707.1067811865476
    want = [1 * math.cos(a0) - 3 * math.sin(a0), 2 * math.cos(a1) - 4 * math.sin(a1),
            3 * math.cos(a0) + 1 * math.sin(a0), 4 * math.cos(a1) + 2 * math.sin(a1)]
    np.testing.assert_allclose(y, want, rtol=0, atol=1e-14)
    # the neighbouring-feature pairing would give something else for the same input
    assert abs(y[1] - (2 * math.cos(a0) + 1 * math.sin(a0))) > 0.1


def test_rope_angles_first_and_last_pair():
    a = P.rope_angles(np.array([0, 1, 1000]), 128, 5.0e5)
    assert a.shape == (3, 64)
    np.testing.assert_allclose(a[:, 0], [0, 1, 1000])
    np.testing.assert_allclose(a[2, 63], 1000 * 5.0e5 ** (-126 / 128), rtol=1e-14)
    assert (np.diff(a[1]) < 0).all()                      # frequencies fall with the pair index


def test_rope_position_zero_is_identity_and_norms_are_kept():
    x = rng(1).standard_normal((3, 5, 64))
    np.testing.assert_array_equal(P.rope(x, np.zeros(5), 5.0e5), x)
    y = P.rope(x, np.arange(100, 105), 5.0e5)
    np.testing.assert_allclose((y ** 2).sum(-1), (x ** 2).sum(-1), rtol=1e-13)
    np.testing.assert_allclose(y[..., :32] ** 2 + y[..., 32:] ** 2, x[..., :32] ** 2 + x[..., 32:] ** 2,
                               rtol=1e-12)


def test_rope_dot_product_depends_on_distance_only():
    r = rng(2)
    q, k = r.standard_normal((1, 128)), r.standard_normal((1, 128))
    for m, n in [(7, 3), (1000, 996), (131071, 131067)]:
        a = (P.rope(q, np.array([m]), 5.0e5) * P.rope(k, np.array([n]), 5.0e5)).sum()
        b = (P.rope(q, np.array([m - n]), 5.0e5) * k).sum()
        np.testing.assert_allclose(a, b, rtol=0, atol=1e-9)


@pytest.mark.parametrize("d,theta", [(128, 5.0e5), (64, 1.0e4), (8, 5.0e5)])
def test_rope_matches_complex_multiplication(d, theta):
    x = rng(3).standard_normal((2, 3, 17, d))
    pos = np.arange(40, 57)
    np.testing.assert_allclose(P.rope(x, pos, theta), torch_rope_complex(x, pos, theta).numpy(),
                               rtol=0, atol=1e-12)


def test_rope_inverse_is_the_opposite_angle():
    x = rng(4).standard_normal((4, 9, 32))
    pos = np.arange(9) * 1000
    np.testing.assert_allclose(P.rope(P.rope(x, pos, 5.0e5), -pos, 5.0e5), x, rtol=0, atol=1e-12)


def test_prologue_without_rotation_is_torch_rms_norm():
    r = rng(5)
    x, g = r.standard_normal((2, 3, 11, 64)), r.standard_normal(64)
    want = F.rms_norm(torch.as_tensor(x), (64,), torch.as_tensor(g), eps=1e-6).numpy()
    np.testing.assert_allclose(P.qk_prologue(x, g, np.arange(11), None, 1e-6), want, rtol=0, atol=1e-13)
    # order: norm first, rotation second (the rotation keeps the norm, the gain does not commute)
    y = P.qk_prologue(x, g, np.arange(11), 5.0e5, 1e-6)
    np.testing.assert_allclose(y, torch_rope_complex(want, np.arange(11), 5.0e5).numpy(), atol=1e-12)


@pytest.mark.parametrize("theta", [5.0e5, None])
def test_prologue_gradient_against_autograd_and_differences(theta):
    r = rng(6)
    x, g, dy = r.standard_normal((2, 2, 7, 16)), r.standard_normal(16), r.standard_normal((2, 2, 7, 16))
    pos = np.arange(20, 27)
    dx, dg = P.qk_prologue_bwd(x, g, pos, theta, dy, 1e-6)

    xt = torch.tensor(x, requires_grad=True)
    gt = torch.tensor(g, requires_grad=True)
    y = F.rms_norm(xt, (16,), gt, eps=1e-6)
    if theta is not None:
        y = torch_rope_complex(y, pos, theta)
    (y * torch.as_tensor(dy)).sum().backward()
    np.testing.assert_allclose(dx, xt.grad.numpy(), rtol=0, atol=1e-12)
    np.testing.assert_allclose(dg, gt.grad.numpy(), rtol=0, atol=1e-12)

    f = lambda xx, gg: (P.qk_prologue(xx, gg, pos, theta, 1e-6) * dy).sum()
    h = 1e-6
    for idx in [(0, 0, 0, 0), (1, 1, 6, 15), (0, 1, 3, 8)]:
        e = np.zeros_like(x)
        e[idx] = h
        np.testing.assert_allclose((f(x + e, g) - f(x - e, g)) / (2 * h), dx[idx], rtol=1e-6, atol=1e-8)
    e = np.zeros_like(g)
    e[9] = h
    np.testing.assert_allclose((f(x, g + e) - f(x, g - e)) / (2 * h), dg[9], rtol=1e-6, atol=1e-8)


def torch_layer(x, Wq, Wk, Wv, Wo, gq, gk, H_q, H_kv, d, scale, theta, pos0, eps):
    """Independent coding of a layer whose window covers the whole sequence: rms_norm, complex
    rotation, scaled_dot_product_attention with a causal mask, rms_norm of the head outputs."""
    x = torch.as_tensor(x)
    B, T, _ = x.shape
    h = F.rms_norm(x, (x.shape[-1],), eps=eps)
    heads = lambda z, H: z.reshape(B, T, H, d).transpose(1, 2)
    q = F.rms_norm(heads(h @ torch.as_tensor(Wq), H_q), (d,), torch.as_tensor(gq), eps=eps)
    k = F.rms_norm(heads(h @ torch.as_tensor(Wk), H_kv), (d,), torch.as_tensor(gk), eps=eps)
    v = heads(h @ torch.as_tensor(Wv), H_kv)
    if theta is not None:
        pos = pos0 + np.arange(T)
        q, k = torch_rope_complex(q, pos, theta), torch_rope_complex(k, pos, theta)
    g = H_q // H_kv
    o = F.scaled_dot_product_attention(q, k.repeat_interleave(g, 1), v.repeat_interleave(g, 1),
                                       is_causal=True, scale=scale)
    y = F.rms_norm(o, (d,), eps=eps)
    return (x + y.transpose(1, 2).reshape(B, T, H_q * d) @ torch.as_tensor(Wo)).numpy()


def make_layer(r, D, H_q, H_kv, d):
    s = 1.0 / math.sqrt(D)
    return (r.standard_normal((D, H_q * d)) * s, r.standard_normal((D, H_kv * d)) * s,
            r.standard_normal((D, H_kv * d)) * s, r.standard_normal((H_q * d, D)) / math.sqrt(H_q * d),
            1.0 + 0.1 * r.standard_normal(d), 1.0 + 0.1 * r.standard_normal(d))


@pytest.mark.parametrize("local", [True, False])
def test_layer_with_window_over_everything_is_causal_attention(local):
    """With w >= T the linear branch has no token to read (its output and the norm of it are
    zero), so a local layer is rotary causal attention and a global layer plain causal attention."""
    r = rng(7)
    D, H_q, H_kv, d, T = 48, 4, 2, 16, 23
    x = r.standard_normal((2, T, D))
    lay = make_layer(r, D, H_q, H_kv, d)
    got = P.attention_layer(x, *lay, H_q=H_q, H_kv=H_kv, d=d, w=64, local=local, scale=0.25, pos0=5)
    want = torch_layer(x, *lay, H_q, H_kv, d, 0.25, P.THETA_LOCAL if local else None, 5, 1e-6)
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-11)


def test_stack_pattern_is_three_local_layers_then_a_global_one():
    """Layer 4 of 4 must ignore the window (global); changing w must change the output of the
    three local layers only through them.  Checked by composing the layers by hand."""
    r = rng(8)
    D, H_q, H_kv, d, T, w = 32, 2, 1, 16, 40, 8
    x = r.standard_normal((1, T, D))
    layers = [make_layer(r, D, H_q, H_kv, d) for _ in range(4)]
    kw = dict(H_q=H_q, H_kv=H_kv, d=d, w=w, scale=0.25)
    got = P.attention_stack(x, layers, **kw)
    y = x
    for l in range(3):
        y = P.attention_layer(y, *layers[l], local=True, **kw)
    want = torch_layer(y, *layers[3], H_q, H_kv, d, 0.25, None, 0, 1e-6)
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-11)
    # a local layer with a short window really uses the linear branch
    a = P.attention_layer(x, *layers[0], local=True, **kw)
    b = P.attention_layer(x, *layers[0], local=True, **{**kw, "w": 64})
    assert np.abs(a - b).max() > 1e-3
