"""fp64 CPU oracle for the RAttention operator.  TEST INFRASTRUCTURE ONLY.

This module is the slow, plain definition the CUDA path is checked against.  It is
imported by the tests, by the smoke check and by the benchmark's CPU-baseline leg, and
by nothing else; the product never routes through it.  It shares no code with the CUDA
path and imports nothing from the package.

What it computes, for one query head (row vectors, 0-indexed positions t, j):

* sliding-window attention (Section 2.1, the SWA equation): softmax over the keys
  ``max(0, t-w) <= j <= t`` -- at most ``w+1`` keys including the current one -- of the
  logits ``scale * q_t . k_j``, applied to the values;
* residual linear attention (Section 3.1, Eq. 4, with the recurrence unrolled):
  ``o_rla_t = sum_{j < t-w} (phi(q_t) . phi(k_j)) v_j`` -- the read-out of the state
  that ends at token ``t-w-1``.  It is evaluated as the explicit quadratic sum; no
  recurrence, no chunking;
* the feature map ``phi`` (Section 3.1, "Parameterization"): a softmax over the head
  features, same map for q and k, ``d' = d``; the two alternatives of the paper's ablation
  (Table 6: ReLU, identity) are selectable and change nothing else;
* the combination (Section 3.2): ``y_t = rmsnorm(o_swa_t; g_swa) + rmsnorm(o_rla_t; g_rla)``
  with two separate per-head RMS norms, ``eps`` inside the square root;
* grouped-query sharing (Section 3.1, "Group-Query Variant"): query head ``h`` reads
  K/V head ``h // (H_q // H_kv)``;
* the analytic gradient of ``sum(y * dy)`` with respect to q, k, v and the two gains,
  derived from the four definitions above (the paper prints no backward formulas);
* decoding: row ``t = pos`` of the same definition over the whole history.

Readings of the paper that are fixed here rather than printed there (each is "parity
unpinned" -- no value in the paper can confirm them): the window is the equation's
``w+1`` keys; the feature map is a plain softmax over d features; ``scale`` multiplies
the SWA logits only; ``eps = 1e-6`` inside the root and unit gains by default; GQA
groups are contiguous.

Everything is float64 numpy.  A matrix product is used as a step; nothing is blocked,
fused or reordered beyond evaluating groups of output rows independently.
"""
from __future__ import annotations

import numpy as np

MODE_RATTN = 0
MODE_SWA_ONLY = 1
MODE_FULL_CAUSAL = 2

DEFAULT_EPS = 1e-6

PHI_SOFTMAX = 0      # the paper's choice (Section 3.1)
PHI_RELU = 1         # ablation, Table 6
PHI_IDENTITY = 2     # ablation, Table 6


def feature_map(x: np.ndarray, phi: int = PHI_SOFTMAX) -> np.ndarray:
    """phi(x) over the last axis: softmax (Section 3.1, softmax-based feature map), or one
    of the ablation's element-wise maps: max(x, 0), x (Table 6)."""
    x = np.asarray(x, dtype=np.float64)
    if phi == PHI_RELU:
        return np.maximum(x, 0.0)
    if phi == PHI_IDENTITY:
        return x.copy()
    assert phi == PHI_SOFTMAX
    e = np.exp(x - x.max(axis=-1, keepdims=True))
    return e / e.sum(axis=-1, keepdims=True)


def rmsnorm(x: np.ndarray, gamma: np.ndarray | None, eps: float) -> np.ndarray:
    """gamma * x / sqrt(mean(x^2) + eps) over the last axis (Section 3.2)."""
    x = np.asarray(x, dtype=np.float64)
    r = np.sqrt((x * x).mean(axis=-1, keepdims=True) + eps)
    y = x / r
    if gamma is not None:
        y = y * np.asarray(gamma, dtype=np.float64)
    return y


def swa_mask(rows: np.ndarray, T: int, w: int) -> np.ndarray:
    """Boolean [len(rows), T]: key j is in query t's window, t-w <= j <= t (Section 2.1)."""
    j = np.arange(T)[None, :]
    t = np.asarray(rows)[:, None]
    return (j >= t - w) & (j <= t)


def rla_mask(rows: np.ndarray, T: int, w: int) -> np.ndarray:
    """Boolean [len(rows), T]: key j is a residual token of query t, j < t-w (Eq. 4)."""
    j = np.arange(T)[None, :]
    t = np.asarray(rows)[:, None]
    return j < t - w


def swa_rows(q_rows, rows, k, v, w, scale):
    """SWA outputs for the listed query rows of one head (Section 2.1).

    q_rows [n, d] are the query vectors of positions ``rows``; k, v are [T, d].
    Returns (o_swa [n, d], p [n, T]) with p the attention weights (zero off-window).
    """
    T = k.shape[0]
    s = scale * (q_rows @ k.T)
    m = swa_mask(rows, T, w)
    s = np.where(m, s, -np.inf)
    p = np.exp(s - s.max(axis=1, keepdims=True))
    p = p / p.sum(axis=1, keepdims=True)
    return p @ v, p


def rla_rows(q_rows, rows, k, v, w, phi=PHI_SOFTMAX):
    """RLA outputs for the listed query rows of one head: Eq. 4 unrolled into the
    explicit sum over residual tokens.  Returns (o_rla [n, d], a [n, T])."""
    T = k.shape[0]
    a = feature_map(q_rows, phi) @ feature_map(k, phi).T
    a = np.where(rla_mask(rows, T, w), a, 0.0)
    return a @ v, a


def forward_head(q, k, v, w, scale=1.0, eps=DEFAULT_EPS, gamma_swa=None, gamma_rla=None,
                 mode=MODE_RATTN, rows=None, row_block=512, parts=False, phi=PHI_SOFTMAX):
    """The operator for one query head.  q, k, v: [T, d].  ``rows`` selects output rows
    (default all).  Returns y [n, d], or (y, o_swa, o_rla) when ``parts`` is set."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    T, d = q.shape
    if mode == MODE_FULL_CAUSAL:
        w = T
    rows = np.arange(T) if rows is None else np.asarray(rows, dtype=np.int64)
    o_s = np.empty((len(rows), d))
    o_r = np.zeros((len(rows), d))
    for lo in range(0, len(rows), row_block):
        r = rows[lo:lo + row_block]
        o_s[lo:lo + len(r)], _ = swa_rows(q[r], r, k, v, w, scale)
        if mode == MODE_RATTN:
            o_r[lo:lo + len(r)], _ = rla_rows(q[r], r, k, v, w, phi)
    y = rmsnorm(o_s, gamma_swa, eps)
    if mode == MODE_RATTN:
        y = y + rmsnorm(o_r, gamma_rla, eps)
    return (y, o_s, o_r) if parts else y


def _gain(gamma, h):
    return None if gamma is None else np.asarray(gamma, dtype=np.float64)[h]


def forward(q, k, v, w, scale=1.0, eps=DEFAULT_EPS, gamma_swa=None, gamma_rla=None,
            mode=MODE_RATTN, phi=PHI_SOFTMAX):
    """The operator for a batch.  q [B, H_q, T, d]; k, v [B, H_kv, T, d]; gains [H_q, d]
    or None.  Query head h uses K/V head h // (H_q // H_kv)."""
    q = np.asarray(q, dtype=np.float64)
    B, Hq, T, d = q.shape
    Hkv = k.shape[1]
    assert Hq % Hkv == 0
    g = Hq // Hkv
    y = np.empty((B, Hq, T, d))
    for b in range(B):
        for h in range(Hq):
            y[b, h] = forward_head(q[b, h], k[b, h // g], v[b, h // g], w, scale, eps,
                                   _gain(gamma_swa, h), _gain(gamma_rla, h), mode, phi=phi)
    return y


def forward_rows(q_head, k_head, v_head, rows, w, scale=1.0, eps=DEFAULT_EPS,
                 gamma_swa=None, gamma_rla=None, mode=MODE_RATTN, phi=PHI_SOFTMAX):
    """Selected output rows of one head, each from the full definition (rows are
    independent of one another, so sampling rows is exact)."""
    return forward_head(q_head, k_head, v_head, w, scale, eps, gamma_swa, gamma_rla,
                        mode, rows=rows, phi=phi)


def decode_row(q_hist, k_hist, v_hist, pos, w, scale=1.0, eps=DEFAULT_EPS,
               gamma_swa=None, gamma_rla=None, phi=PHI_SOFTMAX):
    """Output of the decode step at position ``pos``: the same definition evaluated on
    the full history [0..pos] -- no ring buffer, no running state."""
    n = pos + 1
    return forward_head(q_hist[:n], k_hist[:n], v_hist[:n], w, scale, eps, gamma_swa,
                        gamma_rla, rows=np.array([pos]), phi=phi)[0]


def _rmsnorm_bwd(x, gamma, eps, dy):
    """Gradient of rmsnorm: with r = sqrt(mean(x^2)+eps), n = x/r, gh = dy*gamma:
    dx = (gh - n * mean(gh*n)) / r ; dgamma = sum_t dy_t * n_t."""
    r = np.sqrt((x * x).mean(axis=-1, keepdims=True) + eps)
    n = x / r
    gh = dy if gamma is None else dy * gamma
    dx = (gh - n * (gh * n).mean(axis=-1, keepdims=True)) / r
    dgamma = (dy * n).sum(axis=0)
    return dx, dgamma


def _feature_map_bwd(f, df, x=None, phi=PHI_SOFTMAX):
    """Gradient through the feature map, f = phi(x), df = dL/df.
    softmax: dx = f * (df - <df, f>);  ReLU: dx = df where x > 0;  identity: dx = df."""
    if phi == PHI_RELU:
        return np.where(np.asarray(x) > 0.0, df, 0.0)
    if phi == PHI_IDENTITY:
        return df
    return f * (df - (df * f).sum(axis=-1, keepdims=True))


def backward_head(q, k, v, dy, w, scale=1.0, eps=DEFAULT_EPS, gamma_swa=None,
                  gamma_rla=None, mode=MODE_RATTN, phi=PHI_SOFTMAX):
    """Gradients of L = sum(y * dy) for one query head, by the chain rule through the
    dense [T, T] weight matrices of both branches.  Returns dq, dk, dv (this head's
    contribution to its K/V head), dgamma_swa, dgamma_rla."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    dy = np.asarray(dy, dtype=np.float64)
    T, d = q.shape
    if mode == MODE_FULL_CAUSAL:
        w = T
    rows = np.arange(T)
    gs = None if gamma_swa is None else np.asarray(gamma_swa, dtype=np.float64)
    gr = None if gamma_rla is None else np.asarray(gamma_rla, dtype=np.float64)

    # SWA branch: y_s = rmsnorm(P V), P = masked softmax(scale q k^T)
    o_s, p = swa_rows(q, rows, k, v, w, scale)
    do_s, dgs = _rmsnorm_bwd(o_s, gs, eps, dy)
    dv = p.T @ do_s
    dp = do_s @ v.T
    ds = p * (dp - (dp * p).sum(axis=1, keepdims=True))
    dq = scale * (ds @ k)
    dk = scale * (ds.T @ q)
    dgr = np.zeros(d)

    if mode == MODE_RATTN:
        # RLA branch: y_r = rmsnorm(A V), A = (phi(q) phi(k)^T) masked to j < t-w
        fq = feature_map(q, phi)
        fk = feature_map(k, phi)
        o_r, a = rla_rows(q, rows, k, v, w, phi)
        do_r, dgr = _rmsnorm_bwd(o_r, gr, eps, dy)
        dv = dv + a.T @ do_r
        da = np.where(rla_mask(rows, T, w), do_r @ v.T, 0.0)
        dq = dq + _feature_map_bwd(fq, da @ fk, q, phi)
        dk = dk + _feature_map_bwd(fk, da.T @ fq, k, phi)
    return dq, dk, dv, dgs, dgr


def backward(q, k, v, dy, w, scale=1.0, eps=DEFAULT_EPS, gamma_swa=None, gamma_rla=None,
             mode=MODE_RATTN, phi=PHI_SOFTMAX):
    """Batch gradients.  dk, dv of a K/V head sum over the query heads of its group.
    Returns dq [B,H_q,T,d], dk, dv [B,H_kv,T,d], dgamma_swa, dgamma_rla [H_q,d]."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    B, Hq, T, d = q.shape
    Hkv = k.shape[1]
    g = Hq // Hkv
    dq = np.zeros_like(q)
    dk = np.zeros_like(k)
    dv = np.zeros_like(v)
    dgs = np.zeros((Hq, d))
    dgr = np.zeros((Hq, d))
    for b in range(B):
        for h in range(Hq):
            r = backward_head(q[b, h], k[b, h // g], v[b, h // g], dy[b, h], w, scale, eps,
                              _gain(gamma_swa, h), _gain(gamma_rla, h), mode, phi)
            dq[b, h] = r[0]
            dk[b, h // g] += r[1]
            dv[b, h // g] += r[2]
            dgs[h] += r[3]
            dgr[h] += r[4]
    return dq, dk, dv, dgs, dgr


def rla_state(k, v, n_tokens, phi=PHI_SOFTMAX):
    """S = sum_{j < n_tokens} phi(k_j)^T v_j, the [d, d] state of Eq. 4 after n_tokens
    tokens (zero for n_tokens <= 0).  Used to check the state a prefill hands to decode."""
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    n = max(0, min(int(n_tokens), k.shape[0]))
    return feature_map(k[:n], phi).T @ v[:n]
