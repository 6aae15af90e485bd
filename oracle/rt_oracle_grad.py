"""Gradient oracle of one Recurrent Transformer layer (fp64, CPU).

TEST INFRASTRUCTURE ONLY -- slow, literal, and independent of the CUDA path.

The layer of Sec. 2.2 is written once more, position after position, with torch fp64 tensors
(`layer_seq_torch`), and the gradients of  sum(z * dz)  with respect to the layer input and every
parameter come from reverse-mode differentiation of exactly that graph (`layer_grad`): no custom
backward schedule (Sec. 6, "The backward pass") is involved, so this is the plain definition the
custom reverse loop has to reproduce.

Pins (tests/test_oracle_grad_pins.py): the torch forward equals the numpy definition
`rt_oracle.layer_seq`; every gradient matches central finite differences of that numpy definition
along random directions; the closed-form input Jacobian of the uniform-attention layer (Sec. 4,
App. B); position i's input never receives gradient from outputs before i (causality).
"""
from __future__ import annotations

from typing import Dict

import numpy as np
import torch

from .rt_oracle import NORM_PRE, NORM_QK, NORM_QK_FULL, NORM_SKIP_Z, RTConfig, RTWeights

W_NAMES = ("w_q", "w_k", "w_v", "w_o", "w_up", "w_down")
G_NAMES = ("g_attn", "g_mlp", "g_kv", "g_q", "g_k")


def _rms(u, g, eps):
    return u * g / torch.sqrt(torch.mean(u * u, dim=-1, keepdim=True) + eps)


def _qk_rms(u, g, cfg: RTConfig):
    if not cfg.norm_flags & NORM_QK:
        return u
    if cfg.norm_flags & NORM_QK_FULL:
        return _rms(u, g, cfg.rms_eps)
    H, dh = cfg.n_heads, cfg.head_dim
    return _rms(u.reshape(u.shape[:-1] + (H, dh)), g.reshape(H, dh), cfg.rms_eps).reshape(u.shape)


def _pre(u, g, cfg: RTConfig):
    return _rms(u, g, cfg.rms_eps) if cfg.norm_flags & NORM_PRE else u


def _gelu(a):
    return 0.5 * a * (1.0 + torch.erf(a / np.sqrt(2.0)))


def layer_seq_torch(cfg: RTConfig, p: Dict[str, torch.Tensor], x: torch.Tensor) -> torch.Tensor:
    """z [B, N, d] from x [B, N, d]; p holds the six matrices ([out, in]) and the five gains ([d]).
    Sec. 2.2: query and temporary pair from the input, attention over the persistent pairs of the
    earlier positions plus the own temporary pair, z_i = h_i + alpha MLP[RMS(h_i)] with
    h_i = x_i + alpha W_o c_i, persistent pair (Eqs. 1-2) from z_i."""
    B, N, d = x.shape
    H, dh, s, al = cfg.n_heads, cfg.head_dim, cfg.softmax_scale, cfg.residual_scale
    slopes = None if cfg.alibi_slopes is None else torch.as_tensor(np.asarray(cfg.alibi_slopes), dtype=torch.float64)
    ks, vs, zs = [], [], []
    for i in range(N):
        xi = x[:, i]
        n = _pre(xi, p["g_attn"], cfg)
        q = _qk_rms(n @ p["w_q"].T, p["g_q"], cfg).reshape(B, H, dh)
        kt = _qk_rms(n @ p["w_k"].T, p["g_k"], cfg).reshape(B, H, dh)
        vt = (n @ p["w_v"].T).reshape(B, H, dh)
        lt = s * torch.sum(q * kt, dim=-1, keepdim=True)                       # [B, H, 1]
        if i:
            K = torch.stack(ks, dim=1).reshape(B, i, H, dh)
            V = torch.stack(vs, dim=1).reshape(B, i, H, dh)
            lp = s * torch.einsum("bjhe,bhe->bhj", K, q)
            if slopes is not None:
                dist = torch.arange(i, 0, -1, dtype=torch.float64)              # i - j for j = 0 .. i-1
                lp = lp - slopes[None, :, None] * dist[None, None, :]
            pr = torch.softmax(torch.cat([lp, lt], dim=-1), dim=-1)
            c = torch.einsum("bhj,bjhe->bhe", pr[..., :i], V) + pr[..., i:] * vt
        else:
            c = vt                                                               # a single pair: weight 1
        h = xi + al * (c.reshape(B, d) @ p["w_o"].T)
        zi = h + al * (_gelu(_pre(h, p["g_mlp"], cfg) @ p["w_up"].T) @ p["w_down"].T)
        r = zi if (cfg.norm_flags & NORM_SKIP_Z) else _pre(zi, p["g_kv"], cfg)
        ks.append(_qk_rms(r @ p["w_k"].T, p["g_k"], cfg))
        vs.append(r @ p["w_v"].T)
        zs.append(zi)
    return torch.stack(zs, dim=1)


def params_of(cfg: RTConfig, w: RTWeights, requires_grad: bool = True) -> Dict[str, torch.Tensor]:
    """The eleven parameter tensors as independent fp64 leaves.  g_kv = None aliases g_attn
    (rt_oracle.RTWeights): then "g_kv" IS the "g_attn" leaf and its gradient lands there."""
    d = cfg.d_model
    p = {}
    for nme in W_NAMES:
        p[nme] = torch.tensor(np.asarray(getattr(w, nme), dtype=np.float64), requires_grad=requires_grad)
    for nme in G_NAMES:
        g = getattr(w, nme)
        if g is None and nme == "g_kv":
            p[nme] = p["g_attn"]
            continue
        p[nme] = torch.tensor(np.ones(d) if g is None else np.asarray(g, dtype=np.float64), requires_grad=requires_grad)
    return p


def layer_grad(cfg: RTConfig, w: RTWeights, x: np.ndarray, dz: np.ndarray):
    """Gradients of  sum(z * dz)  (z = the layer's outputs, dz [B, N, d] given):
    returns z, dx [B, N, d] and a dict with one array per parameter (shapes of the parameters).
    With g_kv aliased to g_attn the dict has no "g_kv" entry and "g_attn" carries both uses."""
    xt = torch.tensor(np.asarray(x, dtype=np.float64), requires_grad=True)
    p = params_of(cfg, w)
    z = layer_seq_torch(cfg, p, xt)
    loss = torch.sum(z * torch.as_tensor(np.asarray(dz, dtype=np.float64)))
    names = [n for n in W_NAMES + G_NAMES if not (n == "g_kv" and p[n] is p["g_attn"])]
    grads = torch.autograd.grad(loss, [xt] + [p[n] for n in names], allow_unused=True)
    out = {}
    for n, g in zip(names, grads[1:]):
        out[n] = np.zeros(tuple(p[n].shape)) if g is None else g.numpy()
    return z.detach().numpy(), grads[0].numpy(), out
