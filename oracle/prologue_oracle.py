"""fp64 CPU oracle for what the paper's models do to q and k before the attention operator,
and for a small stack of attention layers built from it.  TEST INFRASTRUCTURE ONLY: imported
by the tests and by nothing in the product.

What it computes:

* qk-norm (Table 1, row "qk-norm: yes"): an RMS norm over the d features of every query and
  key head vector, with one learnable gain vector of length d for the queries and one for the
  keys (shared by all heads of the layer);
* rotary position embedding (Section 4, "Model Setup": local layers use it with theta = 5e5,
  global layers use none): the vector is cut into d/2 pairs, pair i is rotated by the angle
  ``pos * theta**(-2i/d)``;
* the gradient of both, derived from these two definitions;
* an attention layer ``x + concat_heads(operator(q, k, v)) W_o`` with ``q, k, v`` projected from
  the RMS-normed layer input, and a stack of such layers in the paper's pattern of three local
  layers (RAttention, rotary) followed by one global layer (full causal attention, no rotary).

Readings fixed here, not printed in the paper ("parity unpinned" for the choice itself; the
arithmetic under each choice is pinned by the tests):
the pair of feature i is feature i + d/2 (the "rotate-half" layout of the public RoPE
implementations the paper's framework family uses), not feature i + 1; the norm comes first and
the rotation second; both branches of the operator (window and linear) read the same rotated
q and k, because the paper states that the linear branch re-uses the window branch's
projections and names no second set of inputs; the global layer is the same operator in its
full-causal mode, so its output also passes the operator's RMS norm.
"""
from __future__ import annotations

import numpy as np

from . import rattn_oracle as O

THETA_LOCAL = 5.0e5      # Section 4, "Model Setup"


def rope_angles(pos: np.ndarray, d: int, theta: float) -> np.ndarray:
    """angle[p, i] = pos[p] * theta**(-2 i / d) for the d/2 feature pairs."""
    i = np.arange(d // 2, dtype=np.float64)
    return np.asarray(pos, dtype=np.float64)[:, None] * theta ** (-2.0 * i / d)[None, :]


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotate feature pair (i, i + d/2) of x[..., p, :] by angle[p, i].  x is [..., T, d],
    pos holds the T absolute positions."""
    x = np.asarray(x, dtype=np.float64)
    d = x.shape[-1]
    a = rope_angles(pos, d, theta)
    c, s = np.cos(a), np.sin(a)
    lo, hi = x[..., : d // 2], x[..., d // 2:]
    return np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=-1)


def qk_prologue(x: np.ndarray, gain: np.ndarray | None, pos: np.ndarray, theta: float | None,
                eps: float = O.DEFAULT_EPS) -> np.ndarray:
    """rope(rmsnorm(x; gain)); no rotation when theta is None (global layers)."""
    y = O.rmsnorm(x, gain, eps)
    return y if theta is None else rope(y, pos, theta)


def qk_prologue_bwd(x: np.ndarray, gain: np.ndarray | None, pos: np.ndarray, theta: float | None,
                    dy: np.ndarray, eps: float = O.DEFAULT_EPS):
    """Gradient of sum(qk_prologue(x) * dy) with respect to x and the gain."""
    x = np.asarray(x, dtype=np.float64)
    dy = np.asarray(dy, dtype=np.float64)
    d = x.shape[-1]
    g = np.ones(d) if gain is None else np.asarray(gain, dtype=np.float64)
    # the rotation is orthogonal: its transpose rotates by the opposite angle
    du = dy if theta is None else rope(dy, -np.asarray(pos, dtype=np.float64), theta)
    r = 1.0 / np.sqrt((x * x).mean(axis=-1, keepdims=True) + eps)
    n = x * r
    dgain = (du * n).reshape(-1, d).sum(axis=0)
    dn = du * g
    dx = r * (dn - n * (dn * n).mean(axis=-1, keepdims=True))
    return dx, dgain


def attention_layer(x, Wq, Wk, Wv, Wo, gq, gk, *, H_q, H_kv, d, w, local, scale, pos0=0,
                    eps=O.DEFAULT_EPS):
    """One layer on x [B, T, D]:  h = rmsnorm(x);  q, k, v = h Wq, h Wk, h Wv split into heads;
    q, k through the prologue (rotary only when `local`);  the operator (RAttention with window
    w when `local`, full causal attention otherwise);  x + concat_heads(y) Wo."""
    x = np.asarray(x, dtype=np.float64)
    B, T, _ = x.shape
    h = O.rmsnorm(x, None, eps)

    def heads(z, H):
        return z.reshape(B, T, H, d).transpose(0, 2, 1, 3)

    pos = pos0 + np.arange(T)
    theta = THETA_LOCAL if local else None
    q = qk_prologue(heads(h @ Wq, H_q), gq, pos, theta, eps)
    k = qk_prologue(heads(h @ Wk, H_kv), gk, pos, theta, eps)
    v = heads(h @ Wv, H_kv)
    mode = O.MODE_RATTN if local else O.MODE_FULL_CAUSAL
    y = O.forward(q, k, v, w, scale, eps, None, None, mode)
    return x + y.transpose(0, 2, 1, 3).reshape(B, T, H_q * d) @ Wo


def attention_stack(x, layers, **kw):
    """Layers in order; layer l is local unless (l + 1) % 4 == 0 (three local layers, then one
    global layer: Section 4, "Model Setup")."""
    for l, (Wq, Wk, Wv, Wo, gq, gk) in enumerate(layers):
        x = attention_layer(x, Wq, Wk, Wv, Wo, gq, gk, local=(l + 1) % 4 != 0, **kw)
    return x
