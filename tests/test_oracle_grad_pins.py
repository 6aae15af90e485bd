"""Pins of the gradient oracle (oracle/rt_oracle_grad.py).

Expected values never come from the differentiated torch graph itself: they are the numpy definition
`layer_seq` (forward), central finite differences of that numpy definition (every gradient), the
closed-form Jacobian of the uniform-attention layer (Sec. 4 theorem, App. B) and causality.
"""
import math

import numpy as np
import pytest
import torch

from oracle import RTConfig, RTWeights, layer_seq
from oracle.rt_oracle import NORM_PRE, NORM_QK, NORM_SKIP_Z
from oracle.rt_oracle_grad import G_NAMES, W_NAMES, layer_grad, layer_seq_torch, params_of


def rand_layer(rng, d, H, dff, flags=NORM_PRE | NORM_QK, alpha=1.0, gains=True, alibi=False, g_kv=True):
    slopes = [2.0 ** (-8.0 * (h + 1) / H) for h in range(H)] if alibi else None
    cfg = RTConfig(d, H, d // H, dff, norm_flags=flags, residual_scale=alpha, alibi_slopes=slopes)
    mk = lambda o, i: rng.standard_normal((o, i)) / np.sqrt(i)
    w = RTWeights(mk(d, d), mk(d, d), mk(d, d), mk(d, d), mk(dff, d), mk(d, dff))
    if gains:
        for g in G_NAMES:
            if g == "g_kv" and not g_kv:
                continue
            setattr(w, g, 1.0 + 0.3 * rng.standard_normal(d))
    return cfg, w


CASES = [
    dict(flags=NORM_PRE | NORM_QK, alpha=1.0),
    dict(flags=NORM_PRE | NORM_QK, alpha=0.5, alibi=True),
    dict(flags=NORM_PRE | NORM_QK, alpha=0.7, g_kv=False),            # g_kv aliases g_attn
    dict(flags=NORM_PRE, alpha=1.0),
    dict(flags=0, alpha=0.6),
    dict(flags=NORM_PRE | NORM_QK | NORM_SKIP_Z, alpha=1.0),
    dict(flags=NORM_PRE | NORM_QK, alpha=1.0, gains=False),
]


@pytest.mark.parametrize("case", CASES)
def test_torch_forward_equals_the_numpy_definition(case):
    rng = np.random.default_rng(5)
    cfg, w = rand_layer(rng, 12, 3, 20, **case)
    x = rng.standard_normal((2, 7, 12))
    z_np, _, _ = layer_seq(cfg, w, x)
    with torch.no_grad():
        z_t = layer_seq_torch(cfg, params_of(cfg, w, requires_grad=False), torch.as_tensor(x)).numpy()
    assert np.allclose(z_t, z_np, rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("case", CASES)
def test_gradients_match_finite_differences_of_the_numpy_definition(case):
    rng = np.random.default_rng(11)
    d, H, dff, B, N = 8, 2, 12, 2, 6
    cfg, w = rand_layer(rng, d, H, dff, **case)
    x = rng.standard_normal((B, N, d))
    dz = rng.standard_normal((B, N, d))
    _, dx, g = layer_grad(cfg, w, x, dz)

    def loss(w_, x_):
        return float(np.sum(layer_seq(cfg, w_, x_)[0] * dz))

    eps = 1e-6

    def check(got, plus, minus, name):
        fd = (plus - minus) / (2 * eps)
        assert abs(got - fd) <= 1e-7 * max(1.0, abs(fd)), (name, got, fd)

    for _ in range(3):                                             # the input
        dirn = rng.standard_normal(x.shape)
        check(float(np.sum(dx * dirn)), loss(w, x + eps * dirn), loss(w, x - eps * dirn), "x")
    names = list(W_NAMES) + [n for n in G_NAMES if getattr(w, n) is not None]
    assert set(g) >= set(names)
    for name in names:                                             # every parameter that exists
        base = np.asarray(getattr(w, name), dtype=np.float64)
        for _ in range(2):
            dirn = rng.standard_normal(base.shape)
            vals = []
            for sgn in (+1, -1):
                w2 = RTWeights(**{k: getattr(w, k) for k in W_NAMES + G_NAMES})
                setattr(w2, name, base + sgn * eps * dirn)
                vals.append(loss(w2, x))
            check(float(np.sum(g[name] * dirn)), vals[0], vals[1], name)
    for name in G_NAMES:                                            # absent gains are constants equal to one
        if getattr(w, name) is None and name in g:
            assert g[name].shape == (d,)


def test_every_entry_of_one_small_gradient_by_finite_differences():
    # entry by entry (not only along directions) for the smallest interesting layer
    rng = np.random.default_rng(3)
    d, H, dff, N = 4, 2, 4, 4
    cfg, w = rand_layer(rng, d, H, dff, alpha=0.8)
    x = rng.standard_normal((1, N, d)); dz = rng.standard_normal((1, N, d))
    _, dx, g = layer_grad(cfg, w, x, dz)
    eps = 1e-6
    f = lambda w_, x_: float(np.sum(layer_seq(cfg, w_, x_)[0] * dz))
    for idx in np.ndindex(*x.shape):
        e = np.zeros_like(x); e[idx] = eps
        assert abs(dx[idx] - (f(w, x + e) - f(w, x - e)) / (2 * eps)) < 1e-7
    for name in ("w_k", "w_v", "g_k", "g_kv"):
        base = np.asarray(getattr(w, name))
        for idx in np.ndindex(*base.shape):
            vals = []
            for sgn in (+1, -1):
                w2 = RTWeights(**{k: getattr(w, k) for k in W_NAMES + G_NAMES})
                b2 = base.copy(); b2[idx] += sgn * eps
                setattr(w2, name, b2)
                vals.append(f(w2, x))
            assert abs(g[name][idx] - (vals[0] - vals[1]) / (2 * eps)) < 1e-7, (name, idx)


@pytest.mark.parametrize("alpha", [1.0, 0.5])
def test_input_gradient_of_the_uniform_attention_layer_matches_the_closed_form(alpha):
    # Norms off, W_q = 0, W_o = I, W_down = 0, one head: z_k is linear in x_1 with the Jacobian
    # J_k = (1/k!) prod_{m<k} (alpha V + m I) for k >= 2 (Sec. 4 theorem), J_1 = I + alpha V;
    # so d/dx_1 sum_k <z_k, dz_k> = sum_k J_k^T dz_k.
    d, N = 5, 8
    rng = np.random.default_rng(2)
    V = rng.standard_normal((d, d)) / np.sqrt(d)
    cfg = RTConfig(d, 1, d, 4, norm_flags=0, residual_scale=alpha, softmax_scale=1.0)
    w = RTWeights(np.zeros((d, d)), rng.standard_normal((d, d)), V, np.eye(d),
                  rng.standard_normal((4, d)), np.zeros((d, 4)))
    x = rng.standard_normal((1, N, d))
    dz = rng.standard_normal((1, N, d))
    _, dx, _ = layer_grad(cfg, w, x, dz)
    want = np.zeros(d)
    for k in range(1, N + 1):
        prod = np.eye(d)
        for m in range(k):
            prod = prod @ (alpha * V + m * np.eye(d))
        J = prod / math.factorial(k) if k > 1 else np.eye(d) + alpha * V
        want += J.T @ dz[0, k - 1]
    assert np.allclose(dx[0, 0], want, rtol=1e-12, atol=1e-13)


def test_gradient_is_causal_and_per_sequence():
    rng = np.random.default_rng(9)
    cfg, w = rand_layer(rng, 8, 2, 12)
    x = rng.standard_normal((2, 6, 8))
    dz = np.zeros((2, 6, 8)); dz[0, 2] = rng.standard_normal(8)     # only output 2 of sequence 0 matters
    _, dx, _ = layer_grad(cfg, w, x, dz)
    assert np.all(dx[1] == 0.0)                                      # other sequence untouched
    assert np.all(dx[0, 3:] == 0.0)                                  # later inputs cannot influence z_2
    assert np.all(np.abs(dx[0, :3]).sum(axis=-1) > 0)                # every earlier input does
