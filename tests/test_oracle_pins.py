"""Pins for the fp64 oracle: every check compares it with something that is not itself --
a library routine, a closed form, a brute-force loop, the recurrence the paper prints,
the mask structure the paper's Figure 1 states, or finite differences."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import rattn_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand(T, d, seed, n=3):
    rng = np.random.default_rng(seed)
    return [rng.standard_normal((T, d)) for _ in range(n)]


# ------------------------------------------------------------------ SWA vs library / loops

@pytest.mark.parametrize("T,d,w", [(48, 16, 7), (64, 32, 1), (33, 8, 16), (40, 16, 39),
                                   (40, 16, 100)])
def test_swa_matches_library_sdpa_with_band_mask(T, d, w):
    """Section 2.1: SWA is softmax attention restricted to keys t-w..t.  torch's CPU fp64
    scaled_dot_product_attention with an explicit boolean band is the library routine."""
    q, k, v = _rand(T, d, 1)
    scale = 0.37
    o, _ = O.swa_rows(q, np.arange(T), k, v, w, scale)
    i = torch.arange(T)[:, None]
    j = torch.arange(T)[None, :]
    band = (j <= i) & (j >= i - w)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q)[None], torch.from_numpy(k)[None], torch.from_numpy(v)[None],
        attn_mask=band[None], scale=scale)[0].numpy()
    np.testing.assert_allclose(o, ref, rtol=0, atol=1e-12)


def test_window_at_least_T_is_causal_attention_and_rla_vanishes():
    """w >= T-1 leaves no residual token: SWA equals textbook causal attention (library
    is_causal routine), the RLA branch is exactly zero and y = rmsnorm(causal)."""
    T, d = 50, 16
    q, k, v = _rand(T, d, 2)
    for w in (T - 1, T, 4 * T):
        y, o_s, o_r = O.forward_head(q, k, v, w, scale=1.0, parts=True)
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(q)[None], torch.from_numpy(k)[None], torch.from_numpy(v)[None],
            is_causal=True, scale=1.0)[0].numpy()
        np.testing.assert_allclose(o_s, ref, atol=1e-12)
        assert np.all(o_r == 0.0)
        ref_y = ref / np.sqrt((ref ** 2).mean(-1, keepdims=True) + 1e-6)
        np.testing.assert_allclose(y, ref_y, atol=1e-12)
    y_fc = O.forward_head(q, k, v, 3, mode=O.MODE_FULL_CAUSAL)
    np.testing.assert_allclose(y_fc, ref_y, atol=1e-12)


def _brute_force_head(q, k, v, w, scale, eps, gs, gr):
    """Scalar loops straight from the equations of Sections 2.1, 3.1 and 3.2."""
    T, d = len(q), len(q[0])

    def phi(x):
        m = max(x)
        e = [math.exp(a - m) for a in x]
        s = sum(e)
        return [a / s for a in e]

    out = []
    for t in range(T):
        lo = max(0, t - w)
        logits = [scale * sum(q[t][a] * k[j][a] for a in range(d)) for j in range(lo, t + 1)]
        m = max(logits)
        ex = [math.exp(x - m) for x in logits]
        z = sum(ex)
        o_s = [sum(ex[j - lo] * v[j][a] for j in range(lo, t + 1)) / z for a in range(d)]
        o_r = [0.0] * d
        fq = phi(q[t])
        for j in range(0, t - w):        # j < t - w, i.e. the state S_{t-w-1}
            fk = phi(k[j])
            a_tj = sum(fq[a] * fk[a] for a in range(d))
            for a in range(d):
                o_r[a] += a_tj * v[j][a]
        rs = math.sqrt(sum(x * x for x in o_s) / d + eps)
        rr = math.sqrt(sum(x * x for x in o_r) / d + eps)
        out.append([gs[a] * o_s[a] / rs + gr[a] * o_r[a] / rr for a in range(d)])
    return np.array(out)


@pytest.mark.parametrize("T,d,w", [(12, 4, 3), (16, 5, 1), (10, 3, 4)])
def test_brute_force_tiny(T, d, w):
    q, k, v = _rand(T, d, 3)
    rng = np.random.default_rng(4)
    gs, gr = 1 + 0.2 * rng.standard_normal(d), 1 + 0.2 * rng.standard_normal(d)
    y = O.forward_head(q, k, v, w, scale=0.8, eps=1e-6, gamma_swa=gs, gamma_rla=gr)
    ref = _brute_force_head(q.tolist(), k.tolist(), v.tolist(), w, 0.8, 1e-6, gs, gr)
    np.testing.assert_allclose(y, ref, atol=1e-12)


# ------------------------------------------------------------------ mask structure

def _supports(T, w, seed=5):
    """One-hot values v_j = e_j expose the weights: o_swa_t[j] = p_tj, o_rla_t[j] = a_tj."""
    d = T
    rng = np.random.default_rng(seed)
    q, k = rng.standard_normal((T, d)), rng.standard_normal((T, d))
    v = np.eye(T)
    _, o_s, o_r = O.forward_head(q, k, v, w, parts=True)
    return o_s > 0, o_r > 0, o_s


def test_figure1_caption_mask_structure():
    """Figure 1 caption, read from the golden text fixture (1-indexed tokens)."""
    rows = []
    w = None
    for line in open(os.path.join(GOLDEN, "fig1_mask.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("w "):
            w = int(line.split()[1])
            continue
        t, swa, rla = [part.split() for part in line.split("|")]
        rows.append((int(t[0]), {int(x) for x in swa}, {int(x) for x in rla}))
    assert w == 3 and len(rows) == 2
    s_sup, r_sup, _ = _supports(8, w)
    for t, swa, rla in rows:
        assert {j + 1 for j in np.nonzero(s_sup[t - 1])[0]} == swa
        assert {j + 1 for j in np.nonzero(r_sup[t - 1])[0]} == rla


@pytest.mark.parametrize("T,w", [(9, 1), (12, 3), (16, 8), (10, 20)])
def test_masks_partition_the_causal_triangle(T, w):
    """SWA keys and RLA keys are disjoint and together are exactly {0..t}; the window
    holds at most w+1 keys (Section 2.1) and the residual set is {j < t-w} (Eq. 4)."""
    s_sup, r_sup, o_s = _supports(T, w)
    for t in range(T):
        s = set(np.nonzero(s_sup[t])[0])
        r = set(np.nonzero(r_sup[t])[0])
        assert s.isdisjoint(r)
        assert s | r == set(range(t + 1))
        assert s == set(range(max(0, t - w), t + 1)) and len(s) <= w + 1
        assert r == set(range(0, max(0, t - w)))
    np.testing.assert_allclose(o_s.sum(1), 1.0, atol=1e-12)   # softmax weights sum to one


# ------------------------------------------------------------------ RLA: three other codings

def _rla_recurrent(q, k, v, w):
    """Eq. 4 literally: S_t = S_{t-1} + phi(k_t)^T v_t; o_t = phi(q_t) S_{t-w-1}."""
    T, d = q.shape
    S = [np.zeros((d, d))]                 # S[n] = state after n tokens (S_0 = 0)
    for t in range(T):
        e = np.exp(k[t] - k[t].max())
        S.append(S[-1] + np.outer(e / e.sum(), v[t]))
    out = np.zeros((T, d))
    for t in range(T):
        n = t - w                          # tokens 0..t-w-1 -> n of them
        if n > 0:
            e = np.exp(q[t] - q[t].max())
            out[t] = (e / e.sum()) @ S[n]
    return out


def _rla_chunked(q, k, v, w, C):
    """Chunkwise form (Eq. 2-3) with the window lag: for query chunk i the inter term
    reads the state of all chunks before chunk i - w/C, and the intra term is the
    strictly-lower-triangular part of chunk i - w/C."""
    T, d = q.shape
    assert T % C == 0 and w % C == 0
    sm = lambda x: np.exp(x - x.max(-1, keepdims=True)) / np.exp(x - x.max(-1, keepdims=True)).sum(-1, keepdims=True)
    fq, fk = sm(q), sm(k)
    lag = w // C
    S = np.zeros((d, d))
    out = np.zeros((T, d))
    M = np.tril(np.ones((C, C)), -1)
    for i in range(T // C):
        c = i - lag
        if c < 0:
            continue
        Q = fq[i * C:(i + 1) * C]
        K, V = fk[c * C:(c + 1) * C], v[c * C:(c + 1) * C]
        out[i * C:(i + 1) * C] = Q @ S + ((Q @ K.T) * M) @ V
        S = S + K.T @ V
    return out


@pytest.mark.parametrize("T,d,w,C", [(64, 8, 16, 8), (96, 16, 32, 16), (64, 8, 8, 8)])
def test_rla_quadratic_equals_recurrent_equals_chunked(T, d, w, C):
    q, k, v = _rand(T, d, 6)
    o_quad, _ = O.rla_rows(q, np.arange(T), k, v, w)
    np.testing.assert_allclose(o_quad, _rla_recurrent(q, k, v, w), atol=1e-12)
    np.testing.assert_allclose(o_quad, _rla_chunked(q, k, v, w, C), atol=1e-12)


def test_rla_state_helper_matches_recurrence():
    T, d = 40, 8
    q, k, v = _rand(T, d, 7)
    S = np.zeros((d, d))
    for t in range(25):
        S += np.outer(O.feature_map(k[t]), v[t])
    np.testing.assert_allclose(O.rla_state(k, v, 25), S, atol=1e-13)
    assert np.all(O.rla_state(k, v, -3) == 0)


def test_closed_form_zero_keys():
    """k = 0 makes phi(k_j) uniform (1/d) and every SWA logit equal: for any q,
    o_rla_t = (1/d) * sum_{j<t-w} v_j and o_swa_t = mean of v over the window."""
    T, d, w = 30, 8, 5
    q, _, v = _rand(T, d, 8)
    k = np.zeros((T, d))
    _, o_s, o_r = O.forward_head(q, k, v, w, scale=1.7, parts=True)
    for t in range(T):
        np.testing.assert_allclose(o_r[t], v[:max(0, t - w)].sum(0) / d, atol=1e-13)
        np.testing.assert_allclose(o_s[t], v[max(0, t - w):t + 1].mean(0), atol=1e-13)


def test_feature_map_rows_are_distributions():
    x = np.random.default_rng(9).standard_normal((17, 11)) * 5
    f = O.feature_map(x)
    assert np.all(f > 0)
    np.testing.assert_allclose(f.sum(-1), 1.0, atol=1e-14)
    np.testing.assert_allclose(f, torch.softmax(torch.from_numpy(x), -1).numpy(), atol=1e-15)
    np.testing.assert_allclose(O.feature_map(x + 3.0), f, atol=1e-14)   # shift invariance


# ------------------------------------------------------------------ norm / combine

def test_rmsnorm_closed_forms_and_invariances():
    d = 16
    c = np.full((1, d), 3.0)
    np.testing.assert_allclose(O.rmsnorm(c, None, 0.0), 1.0)            # constant vector
    np.testing.assert_allclose(O.rmsnorm(-c, None, 0.0), -1.0)
    assert np.all(O.rmsnorm(np.zeros((2, d)), None, 1e-6) == 0)          # rmsnorm(0) = 0
    x = np.random.default_rng(10).standard_normal((5, d))
    g = np.random.default_rng(11).standard_normal(d)
    y = O.rmsnorm(x, g, 1e-6)
    np.testing.assert_allclose(y, g * x / np.sqrt((x ** 2).mean(-1, keepdims=True) + 1e-6))
    np.testing.assert_allclose((O.rmsnorm(x, None, 0.0) ** 2).mean(-1), 1.0)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x), (d,), torch.from_numpy(g), 1e-6)
    np.testing.assert_allclose(y, ref.numpy(), atol=1e-14)


def test_value_scaling_leaves_output_unchanged_and_gains_are_linear():
    T, d, w = 40, 8, 6
    q, k, v = _rand(T, d, 12)
    y1 = O.forward_head(q, k, v, w, eps=1e-30)
    y2 = O.forward_head(q, k, 7.5 * v, w, eps=1e-30)
    # rows t <= w have o_rla = 0 exactly; compare the rows with both branches alive
    np.testing.assert_allclose(y1[w + 1:], y2[w + 1:], atol=1e-12)
    gs, gr = np.full(d, 2.0), np.full(d, -3.0)
    _, o_s, o_r = O.forward_head(q, k, v, w, parts=True)
    y3 = O.forward_head(q, k, v, w, gamma_swa=gs, gamma_rla=gr)
    np.testing.assert_allclose(y3, 2 * O.rmsnorm(o_s, None, 1e-6) - 3 * O.rmsnorm(o_r, None, 1e-6),
                               atol=1e-12)
    y_swa = O.forward_head(q, k, v, w, mode=O.MODE_SWA_ONLY)
    np.testing.assert_allclose(y_swa, O.rmsnorm(o_s, None, 1e-6), atol=1e-14)


def test_scale_touches_swa_logits_only():
    T, d, w = 24, 8, 4
    q, k, v = _rand(T, d, 13)
    _, s1, r1 = O.forward_head(q, k, v, w, scale=1.0, parts=True)
    _, s2, r2 = O.forward_head(q, k, v, w, scale=0.25, parts=True)
    assert np.array_equal(r1, r2)
    _, s3, _ = O.forward_head(0.25 * q, k, v, w, scale=1.0, parts=True)
    np.testing.assert_allclose(s2, s3, atol=1e-13)
    assert np.abs(s1 - s2).max() > 1e-3


# ------------------------------------------------------------------ causality / GQA / rows

def test_causality_is_bit_exact():
    T, d, w, j0 = 48, 8, 5, 29
    q, k, v = _rand(T, d, 14)
    y = O.forward_head(q, k, v, w)
    q2, k2, v2 = q.copy(), k.copy(), v.copy()
    q2[j0:] += 1.0
    k2[j0:] -= 2.0
    v2[j0:] *= 3.0
    y2 = O.forward_head(q2, k2, v2, w)
    assert np.array_equal(y[:j0], y2[:j0])
    assert not np.allclose(y[j0:], y2[j0:])


def test_gqa_equals_mha_on_repeated_kv():
    B, Hq, Hkv, T, d, w = 2, 6, 2, 20, 8, 4
    rng = np.random.default_rng(15)
    q = rng.standard_normal((B, Hq, T, d))
    k = rng.standard_normal((B, Hkv, T, d))
    v = rng.standard_normal((B, Hkv, T, d))
    gs = rng.standard_normal((Hq, d))
    gr = rng.standard_normal((Hq, d))
    y = O.forward(q, k, v, w, 0.5, 1e-6, gs, gr)
    g = Hq // Hkv
    y_mha = O.forward(q, np.repeat(k, g, axis=1), np.repeat(v, g, axis=1), w, 0.5, 1e-6, gs, gr)
    assert np.array_equal(y, y_mha)
    # contiguous groups: head 4 (group 1) must read K/V head 1
    np.testing.assert_array_equal(
        y[1, 4], O.forward_head(q[1, 4], k[1, 1], v[1, 1], w, 0.5, 1e-6, gs[4], gr[4]))


def test_row_sampling_and_decode_row_equal_full_forward():
    T, d, w = 70, 8, 9
    q, k, v = _rand(T, d, 16)
    y = O.forward_head(q, k, v, w, scale=0.6)
    rows = np.array([0, 1, w, w + 1, 33, T - 1])
    np.testing.assert_allclose(O.forward_rows(q, k, v, rows, w, scale=0.6), y[rows], atol=1e-14)
    for pos in (0, w - 1, w, w + 1, 2 * w, T - 1):
        np.testing.assert_allclose(O.decode_row(q, k, v, pos, w, scale=0.6), y[pos], atol=1e-14)


# ------------------------------------------------------------------ backward

def _loss(q, k, v, dy, w, scale, gs, gr, mode=O.MODE_RATTN):
    return float((O.forward(q, k, v, w, scale, 1e-6, gs, gr, mode) * dy).sum())


@pytest.mark.parametrize("T,d,w,Hq,Hkv", [(256, 16, 64, 2, 1), (256, 16, 32, 2, 2),
                                          (64, 8, 5, 4, 2)])
def test_backward_matches_central_differences(T, d, w, Hq, Hkv):
    """Directional central differences in fp64 of L = sum(y*dy) along random directions
    in q, k, v and both gains, plus sampled single elements."""
    rng = np.random.default_rng(17)
    B = 1
    q = rng.standard_normal((B, Hq, T, d))
    k = rng.standard_normal((B, Hkv, T, d))
    v = rng.standard_normal((B, Hkv, T, d))
    dy = rng.standard_normal((B, Hq, T, d))
    gs = 1 + 0.3 * rng.standard_normal((Hq, d))
    gr = 1 + 0.3 * rng.standard_normal((Hq, d))
    scale = 0.5
    dq, dk, dv, dgs, dgr = O.backward(q, k, v, dy, w, scale, 1e-6, gs, gr)
    h = 1e-5
    args = dict(q=q, k=k, v=v, gs=gs, gr=gr)
    grads = dict(q=dq, k=dk, v=dv, gs=dgs, gr=dgr)
    for name in args:
        for trial in range(3):
            u = rng.standard_normal(args[name].shape)
            if trial == 2:                       # a single element
                u[:] = 0
                u.flat[rng.integers(u.size)] = 1.0
            plus = dict(args)
            minus = dict(args)
            plus[name] = args[name] + h * u
            minus[name] = args[name] - h * u
            fd = (_loss(plus["q"], plus["k"], plus["v"], dy, w, scale, plus["gs"], plus["gr"]) -
                  _loss(minus["q"], minus["k"], minus["v"], dy, w, scale, minus["gs"], minus["gr"])) / (2 * h)
            an = float((grads[name] * u).sum())
            assert abs(fd - an) <= 1e-6 * max(1.0, abs(an)) + 1e-7, (name, trial, fd, an)


def test_backward_window_covers_sequence_is_swa_only_limit():
    """w >= T: the RLA branch is identically zero, so its gain gets no gradient and the
    gradients equal those of the SWA-only mode."""
    rng = np.random.default_rng(18)
    T, d = 64, 8
    q, k, v, dy = (rng.standard_normal((1, 1, T, d)) for _ in range(4))
    full = O.backward(q, k, v, dy, 512)
    swa = O.backward(q, k, v, dy, 512, mode=O.MODE_SWA_ONLY)
    for a, b in zip(full[:4], swa[:4]):
        np.testing.assert_allclose(a, b, atol=1e-13)
    assert np.all(full[4] == 0)


def test_backward_matches_autograd_of_an_independent_torch_coding():
    rng = np.random.default_rng(19)
    T, d, w, scale = 48, 8, 6, 0.7
    q, k, v, dy = (rng.standard_normal((T, d)) for _ in range(4))
    gs, gr = rng.standard_normal(d), rng.standard_normal(d)
    tq, tk, tv = (torch.tensor(x, requires_grad=True) for x in (q, k, v))
    tgs, tgr = (torch.tensor(x, requires_grad=True) for x in (gs, gr))
    i = torch.arange(T)[:, None]
    j = torch.arange(T)[None, :]
    o_s = torch.softmax((scale * tq @ tk.T).masked_fill(~((j <= i) & (j >= i - w)), -1e300), -1) @ tv
    o_r = ((torch.softmax(tq, -1) @ torch.softmax(tk, -1).T) * (j < i - w)) @ tv
    rn = lambda x, g: g * x * torch.rsqrt((x * x).mean(-1, keepdim=True) + 1e-6)
    ((rn(o_s, tgs) + rn(o_r, tgr)) * torch.tensor(dy)).sum().backward()
    dq, dk, dv, dgs, dgr = O.backward_head(q, k, v, dy, w, scale, 1e-6, gs, gr)
    for a, b in ((dq, tq), (dk, tk), (dv, tv), (dgs, tgs), (dgr, tgr)):
        np.testing.assert_allclose(a, b.grad.numpy(), atol=1e-11)


def test_gradient_causality():
    """Upstream gradient on rows < t0 only: keys/values at j >= t0 get zero gradient."""
    rng = np.random.default_rng(20)
    T, d, w, t0 = 40, 8, 4, 23
    q, k, v, dy = (rng.standard_normal((1, 1, T, d)) for _ in range(4))
    dy[:, :, t0:] = 0
    dq, dk, dv, _, _ = O.backward(q, k, v, dy, w)
    assert np.all(dk[0, 0, t0:] == 0) and np.all(dv[0, 0, t0:] == 0) and np.all(dq[0, 0, t0:] == 0)
    assert np.abs(dk[0, 0, :t0]).min() > 0


# ------------------------------------------------------------------ planted mistakes are caught

def test_pins_would_catch_an_off_by_one_window(monkeypatch):
    """Sensitivity check on the CPU: shifting the residual boundary by one token (a
    plausible slip) breaks the partition and the recurrence pins."""
    T, d, w = 32, 8, 4
    q, k, v = _rand(T, d, 21)
    good, _ = O.rla_rows(q, np.arange(T), k, v, w)
    monkeypatch.setattr(O, "rla_mask", lambda rows, T_, w_: np.arange(T_)[None, :] <= np.asarray(rows)[:, None] - w_)
    bad, _ = O.rla_rows(q, np.arange(T), k, v, w)
    assert np.abs(bad - _rla_recurrent(q, k, v, w)).max() > 1e-3
    np.testing.assert_allclose(good, _rla_recurrent(q, k, v, w), atol=1e-12)


# ------------------------------------------------------------------ ablation feature maps (Table 6)

def _rla_recurrent_phi(q, k, v, w, f):
    """Eq. 4 as printed, with an arbitrary element-wise map f."""
    T, d = q.shape
    S = [np.zeros((d, d))]
    for t in range(T):
        S.append(S[-1] + np.outer(f(k[t]), v[t]))
    out = np.zeros((T, d))
    for t in range(T):
        if t - w > 0:
            out[t] = f(q[t]) @ S[t - w]
    return out


@pytest.mark.parametrize("phi,f", [(O.PHI_RELU, lambda x: np.array([max(a, 0.0) for a in x])),
                                   (O.PHI_IDENTITY, lambda x: np.array(list(x)))])
def test_other_feature_maps_quadratic_equals_recurrence(phi, f):
    """ReLU and identity maps of the paper's ablation: the explicit quadratic sum equals the
    printed recurrence with the same element-wise map (scalar max / copy written out here),
    and the library routine agrees on the map itself."""
    T, d, w = 48, 8, 7
    q, k, v = _rand(T, d, 31)
    o, _ = O.rla_rows(q, np.arange(T), k, v, w, phi)
    np.testing.assert_allclose(o, _rla_recurrent_phi(q, k, v, w, f), atol=1e-12)
    ref = torch.relu(torch.from_numpy(q)).numpy() if phi == O.PHI_RELU else q
    assert np.array_equal(O.feature_map(q, phi), ref)
    np.testing.assert_allclose(O.rla_state(k, v, 13, phi), sum(np.outer(f(k[t]), v[t]) for t in range(13)), atol=1e-13)


def test_identity_map_closed_form_with_one_hot_keys():
    """Identity map, keys k_j = e_{a_j} (one-hot): phi(q_t).phi(k_j) = q_t[a_j], so
    o_rla_t = sum_{j < t-w} q_t[a_j] v_j.  The same keys under ReLU give the same sum with
    max(q_t[a_j], 0)."""
    T, d, w = 30, 8, 4
    rng = np.random.default_rng(32)
    q, v = rng.standard_normal((T, d)), rng.standard_normal((T, d))
    a = rng.integers(0, d, T)
    k = np.eye(d)[a]
    for phi, g in ((O.PHI_IDENTITY, lambda x: x), (O.PHI_RELU, lambda x: max(x, 0.0))):
        _, _, o_r = O.forward_head(q, k, v, w, parts=True, phi=phi)
        for t in range(T):
            want = sum((g(q[t, a[j]]) * v[j] for j in range(max(0, t - w))), np.zeros(d))
            np.testing.assert_allclose(o_r[t], want, atol=1e-13)


@pytest.mark.parametrize("phi", [O.PHI_RELU, O.PHI_IDENTITY])
def test_other_feature_maps_backward_matches_central_differences(phi):
    rng = np.random.default_rng(33 + phi)
    B, Hq, Hkv, T, d, w = 1, 2, 1, 96, 8, 9
    q = rng.standard_normal((B, Hq, T, d))
    k = rng.standard_normal((B, Hkv, T, d))
    v = rng.standard_normal((B, Hkv, T, d))
    dy = rng.standard_normal((B, Hq, T, d))
    dq, dk, dv, _, _ = O.backward(q, k, v, dy, w, 0.5, phi=phi)
    loss = lambda q_, k_, v_: float((O.forward(q_, k_, v_, w, 0.5, phi=phi) * dy).sum())
    h = 1e-6
    for name, x, g in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        for _ in range(3):
            u = rng.standard_normal(x.shape)
            args_p = {"q": q, "k": k, "v": v}
            args_m = dict(args_p)
            args_p[name] = x + h * u
            args_m[name] = x - h * u
            fd = (loss(args_p["q"], args_p["k"], args_p["v"]) - loss(args_m["q"], args_m["k"], args_m["v"])) / (2 * h)
            an = float((g * u).sum())
            assert abs(fd - an) <= 2e-6 * max(1.0, abs(an)) + 1e-6, (name, fd, an)


def test_other_feature_maps_keep_the_window_branch_and_differ_from_softmax():
    T, d, w = 40, 8, 5
    q, k, v = _rand(T, d, 35)
    base = O.forward_head(q, k, v, w, parts=True)
    for phi in (O.PHI_RELU, O.PHI_IDENTITY):
        y, o_s, o_r = O.forward_head(q, k, v, w, parts=True, phi=phi)
        assert np.array_equal(o_s, base[1])                   # the map touches the linear branch only
        assert np.all(o_r[:w + 1] == 0)
        assert np.abs(o_r[w + 1:] - base[2][w + 1:]).max() > 1e-3
