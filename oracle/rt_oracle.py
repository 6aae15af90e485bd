"""Plain fp64 oracle of one Recurrent Transformer (RT) layer, a stack of them, and
the one-token decode step.

TEST INFRASTRUCTURE ONLY -- slow, literal, and independent of the CUDA path.

Parity pins (all in tests/test_oracle_pins.py, none of them re-uses this file's
formulas): the closed-form Jacobian of the uniform-attention layer (the training-
stability theorem of Sec. 4, proof in App. B), the two-block construction under which the layer equals textbook causal
softmax attention (App. A), the worked tiling examples of Sec. 5, exactly-once
coverage and the sum of tile sizes of Algorithm 1, blocked == sequential for every
block size, decode == one more prefill position, the unique fixed point, and
causality.  Parity unpinned: agreement with the authors' trained models (no
weights or code exist to compare with); the conventions the paper leaves open
(softmax scale, eps, GELU form, where gains sit) are fixed in the docstrings here.

Notation follows Sec. 2 of the paper: x_i layer input, q_i query, (k~_i, v~_i) the
temporary pair, (k_i, v_i) the persistent pair, a_i attention output, z_i layer
output, L number of layers, alpha = residual scale (1/sqrt(L)).
All arrays are numpy float64.  Batched arrays are [B, N, d]; the B sequences are
independent (the paper states everything per sequence).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Sequence, List, Optional, Tuple

import numpy as np

try:  # exact erf on arrays
    from scipy.special import erf as _erf
except Exception:  # pragma: no cover - scipy is in the image; keep a fallback
    import torch

    def _erf(a):
        return torch.special.erf(torch.from_numpy(np.asarray(a, dtype=np.float64))).numpy()


NORM_PRE = 1      # bit0: RMS(x), RMS(h) before the MLP and RMS(z) are applied
NORM_QK = 2       # bit1: qkRMS on queries and keys
NORM_QK_FULL = 4  # bit2: qkRMS over the full width instead of per head
NORM_SKIP_Z = 8   # bit3: persistent pair from z itself (the "RMSNorm Ablation" appendix)


@dataclass
class RTConfig:
    d_model: int
    n_heads: int
    head_dim: int
    d_ff: int
    norm_flags: int = NORM_PRE | NORM_QK
    rms_eps: float = 1e-6
    softmax_scale: Optional[float] = None   # None -> 1/sqrt(head_dim); 1.0 = Sec. 2's literal Attn
    residual_scale: float = 1.0             # alpha = 1/sqrt(L)  (Sec. 2, pre-LN parameterisation)
    alibi_slopes: Optional[Sequence[float]] = None   # [H]; logit of query i on the persistent pair j gets
                                                     # -slope_h (i - j) (App. D: ALiBi); None = no bias

    def __post_init__(self):
        assert self.n_heads * self.head_dim == self.d_model
        if self.softmax_scale is None:
            self.softmax_scale = 1.0 / np.sqrt(self.head_dim)
        if self.alibi_slopes is not None:
            self.alibi_slopes = np.asarray(self.alibi_slopes, dtype=np.float64)
            assert self.alibi_slopes.shape == (self.n_heads,)

    def slope(self, h: int) -> float:
        return 0.0 if self.alibi_slopes is None else float(self.alibi_slopes[h])


@dataclass
class RTWeights:
    """y = W u, W stored [out, in].  Gains default to ones; g_kv=None aliases g_attn."""
    w_q: np.ndarray
    w_k: np.ndarray
    w_v: np.ndarray
    w_o: np.ndarray
    w_up: np.ndarray
    w_down: np.ndarray
    g_attn: Optional[np.ndarray] = None
    g_mlp: Optional[np.ndarray] = None
    g_kv: Optional[np.ndarray] = None
    g_q: Optional[np.ndarray] = None
    g_k: Optional[np.ndarray] = None

    def gain(self, name: str, d: int) -> np.ndarray:
        g = getattr(self, name)
        if g is None and name == "g_kv":
            g = self.g_attn
        return np.ones(d) if g is None else np.asarray(g, dtype=np.float64)


# ----------------------------------------------------------------------------- primitives

def rms(u: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    """RMS(u) = sqrt(D) u / ||u||  (Sec. 2, Notation), with a learnable gain g and an
    eps inside the root: u * g / sqrt(mean(u^2) + eps), over the last axis."""
    ms = np.mean(u * u, axis=-1, keepdims=True)
    return u * g / np.sqrt(ms + eps)


def qk_rms(u: np.ndarray, g: np.ndarray, cfg: RTConfig) -> np.ndarray:
    """Query/key normalisation (the magenta RMS of Sec. 2): the same formula applied
    to each head's head_dim entries (multi-head = per-head construction), or to the
    whole vector when NORM_QK_FULL is set; identity when NORM_QK is clear."""
    if not cfg.norm_flags & NORM_QK:
        return u
    if cfg.norm_flags & NORM_QK_FULL:
        return rms(u, g, cfg.rms_eps)
    H, dh = cfg.n_heads, cfg.head_dim
    uh = u.reshape(u.shape[:-1] + (H, dh))
    gh = g.reshape(H, dh)
    return rms(uh, gh, cfg.rms_eps).reshape(u.shape)


def _pre(u: np.ndarray, g: np.ndarray, cfg: RTConfig) -> np.ndarray:
    return rms(u, g, cfg.rms_eps) if cfg.norm_flags & NORM_PRE else u


def gelu(a: np.ndarray) -> np.ndarray:
    """Exact GELU: a * Phi(a), Phi the standard normal CDF."""
    return 0.5 * a * (1.0 + _erf(a / np.sqrt(2.0)))


def attn(keys: np.ndarray, values: np.ndarray, q: np.ndarray, scale: float, bias=None) -> np.ndarray:
    """The Attn operator of Sec. 2 for one head and one query:
    sum_i v_i exp(s<k_i,q>) / sum_j exp(s<k_j,q>);  keys, values [l, dh], q [dh].
    bias [l] (optional) is added to the logits (the ALiBi distances of App. D)."""
    logits = scale * (keys @ q)
    if bias is not None:
        logits = logits + bias
    p = np.exp(logits - logits.max())
    p /= p.sum()
    return p @ values


def _mlp(h: np.ndarray, w: RTWeights, cfg: RTConfig) -> np.ndarray:
    u = _pre(h, w.gain("g_mlp", cfg.d_model), cfg)
    return gelu(u @ w.w_up.T) @ w.w_down.T


def _temp_qkv(xi: np.ndarray, w: RTWeights, cfg: RTConfig):
    """q_i, k~_i, v~_i from the layer input (first display of Sec. 2.2)."""
    d = cfg.d_model
    n = _pre(xi, w.gain("g_attn", d), cfg)
    q = qk_rms(n @ w.w_q.T, w.gain("g_q", d), cfg)
    kt = qk_rms(n @ w.w_k.T, w.gain("g_k", d), cfg)
    vt = n @ w.w_v.T
    return q, kt, vt


def _output_and_persistent(xi, ai, w: RTWeights, cfg: RTConfig):
    """z_i = x_i + alpha (a_i + MLP[RMS(x_i + alpha a_i)]) with a_i the multi-head attention
    output after the usual output projection; then Eqs. (1)-(2):
    k_i = qkRMS[K RMS(z_i)], v_i = V RMS(z_i)."""
    d, al = cfg.d_model, cfg.residual_scale
    h = xi + al * ai
    zi = h + al * _mlp(h, w, cfg)
    r = zi if (cfg.norm_flags & NORM_SKIP_Z) else _pre(zi, w.gain("g_kv", d), cfg)
    ki = qk_rms(r @ w.w_k.T, w.gain("g_k", d), cfg)
    vi = r @ w.w_v.T
    return zi, ki, vi


# ----------------------------------------------------------------------------- O-seq

def layer_seq(cfg: RTConfig, w: RTWeights, x: np.ndarray):
    """The plain definition (Sec. 2.2), one position after the other, two-pass softmax.

    x [B, N, d] -> z, k, v, each [B, N, d]  (k, v the persistent pairs)."""
    x = np.asarray(x, dtype=np.float64)
    B, N, d = x.shape
    H, dh, s = cfg.n_heads, cfg.head_dim, cfg.softmax_scale
    z = np.zeros_like(x)
    k = np.zeros_like(x)
    v = np.zeros_like(x)
    for i in range(N):
        q, kt, vt = _temp_qkv(x[:, i], w, cfg)
        qh = q.reshape(B, H, dh)
        # logits against the i persistent pairs of earlier positions, then the temporary pair
        lp = s * np.einsum("bjhe,bhe->bhj", k[:, :i].reshape(B, i, H, dh), qh)
        if cfg.alibi_slopes is not None:             # distance i - j to the persistent pair j; 0 to the temporary pair
            lp = lp - cfg.alibi_slopes[None, :, None] * (i - np.arange(i))[None, None, :]
        lt = s * np.sum(qh * kt.reshape(B, H, dh), axis=-1, keepdims=True)
        logits = np.concatenate([lp, lt], axis=-1)                     # [B, H, i+1]
        p = np.exp(logits - logits.max(axis=-1, keepdims=True))
        p /= p.sum(axis=-1, keepdims=True)
        c = np.einsum("bhj,bjhe->bhe", p[..., :i], v[:, :i].reshape(B, i, H, dh))
        c += p[..., i:] * vt.reshape(B, H, dh)
        a = c.reshape(B, d) @ w.w_o.T
        z[:, i], k[:, i], v[:, i] = _output_and_persistent(x[:, i], a, w, cfg)
    return z, k, v


# ----------------------------------------------------------------------------- Alg. 2 and Alg. 1

def update_tile(qs, ks, vs, m, l, o, scale, bias=None):
    """Algorithm 2 (UpdateTile) for one head: queries qs [nq, dh], tile ks, vs [nk, dh],
    running stats m [nq], l [nq], o [nq, dh]; returns the updated (m, l, o).
    bias [nq, nk] (optional) is added to the tile logits."""
    al = scale * (qs @ ks.T)                      # tile logits
    if bias is not None:
        al = al + bias
    m_tile = al.max(axis=1)
    m_new = np.maximum(m, m_tile)
    resc = np.exp(m - m_new)                      # exp(-inf - finite) = 0 on first use
    e = np.exp(al - m_new[:, None])
    o = o * resc[:, None] + e @ vs
    l = l * resc + e.sum(axis=1)
    return m_new, l, o


def alg1_tiles(N: int, leaf: int = 1) -> List[Tuple[int, int, int, int, int]]:
    """Cross tiles of Algorithm 1, 1-based and inclusive as printed there:
    (t, u, v, s, e) = after position t, queries u..v attend to the pairs s..e.
    leaf=1 is the algorithm as printed (P = 2^nu2(t)); leaf=b>1 applies the same rule to
    blocks of b positions (P = b * 2^nu2(t/b), only when b divides t)."""
    out = []
    for t in range(1, N + 1):
        if t % leaf:
            continue
        tau = t // leaf
        P = leaf * (tau & -tau)
        u, vv = t + 1, min(t + P, N)
        if u <= vv:
            out.append((t, u, vv, t - P + 1, t))
    return out


def layer_blk(cfg: RTConfig, w: RTWeights, x: np.ndarray, leaf: int = 1,
              self_first: bool = True, eager_leaf: bool = False):
    """Algorithm 1 with Algorithm 2, carrying (m, l, o) for every query.

    leaf=1 is Algorithm 1 as printed.  leaf=b>1 keeps the cross tiles whose size is a
    multiple of b (block-level P) and has position t collect the pairs of its own block,
    start..t-1, right before it finalises (or, with eager_leaf, lets every revealed pair
    update all later queries of its block at once).  self_first=False folds the temporary
    pair in last instead of first.  All variants give the same result in exact arithmetic."""
    x = np.asarray(x, dtype=np.float64)
    B, N, d = x.shape
    H, dh, s = cfg.n_heads, cfg.head_dim, cfg.softmax_scale
    z = np.zeros_like(x)
    k = np.zeros_like(x)
    v = np.zeros_like(x)
    tiles = {t: (u, vv, s0, e0) for (t, u, vv, s0, e0) in alg1_tiles(N, leaf)}
    for b in range(B):
        q = np.zeros((N, d)); kt = np.zeros((N, d)); vt = np.zeros((N, d))
        for i in range(N):                              # line 1: queries are available up front
            q[i], kt[i], vt[i] = _temp_qkv(x[b, i], w, cfg)
        m = np.full((H, N), -np.inf); l = np.zeros((H, N)); o = np.zeros((H, N, dh))

        def upd(qlo, qhi, K, V, klo=None):              # 0-based half-open query range; klo = position of K[0]
            for h in range(H):                          # (None: the temporary pair, at distance 0)
                sl = slice(h * dh, (h + 1) * dh)
                bias = None
                if cfg.alibi_slopes is not None and klo is not None:
                    dist = np.arange(qlo, qhi)[:, None] - (klo + np.arange(K.shape[0]))[None, :]
                    bias = -cfg.slope(h) * dist
                m[h, qlo:qhi], l[h, qlo:qhi], o[h, qlo:qhi] = update_tile(
                    q[qlo:qhi, sl], K[:, sl], V[:, sl], m[h, qlo:qhi], l[h, qlo:qhi], o[h, qlo:qhi], s, bias)

        for t in range(1, N + 1):                       # 1-based as in the algorithm
            i = t - 1
            start = (i // leaf) * leaf                  # first position of t's block (0-based)
            if self_first:
                upd(i, i + 1, kt[i:i + 1], vt[i:i + 1])
            if not eager_leaf and i > start:
                upd(i, i + 1, k[b, start:i], v[b, start:i], start)
            if not self_first:
                upd(i, i + 1, kt[i:i + 1], vt[i:i + 1])
            c = np.concatenate([o[h, i] / l[h, i] for h in range(H)])        # a_t = o_t / l_t per head
            a = c @ w.w_o.T
            z[b, i], k[b, i], v[b, i] = _output_and_persistent(x[b, i], a, w, cfg)
            if eager_leaf:
                hi = min(start + leaf, N)
                if i + 1 < hi:
                    upd(i + 1, hi, k[b, i:i + 1], v[b, i:i + 1], i)
            if t in tiles:
                u, vv, s0, e0 = tiles[t]
                upd(u - 1, vv, k[b, s0 - 1:e0], v[b, s0 - 1:e0], s0 - 1)
    return z, k, v


# ----------------------------------------------------------------------------- O-fix

def layer_fixed_point(cfg: RTConfig, w: RTWeights, x: np.ndarray, z_claim: np.ndarray, rows=None):
    """One parallel sweep (Sec. 6, activation checkpointing): rebuild every persistent pair
    from the claimed outputs z, then recompute every a_i and z_i independently of each other.
    Because z_i depends only on z_j, j < i, the true z is the unique fixed point: the claim
    is right iff the returned z' equals it.  Returns z', k, v with (k, v) rebuilt from z_claim.
    rows: optional iterable of positions to recompute (the other rows of z' stay zero)."""
    x = np.asarray(x, dtype=np.float64)
    zc = np.asarray(z_claim, dtype=np.float64)
    B, N, d = x.shape
    H, dh, s = cfg.n_heads, cfg.head_dim, cfg.softmax_scale
    r = zc if (cfg.norm_flags & NORM_SKIP_Z) else _pre(zc, w.gain("g_kv", d), cfg)
    k = qk_rms(r @ w.w_k.T, w.gain("g_k", d), cfg)
    v = r @ w.w_v.T
    q, kt, vt = _temp_qkv(x, w, cfg)                     # all positions at once
    z2 = np.zeros_like(x)
    for b in range(B):
        for i in (range(N) if rows is None else rows):
            c = np.zeros(d)
            for h in range(H):
                sl = slice(h * dh, (h + 1) * dh)
                keys = np.concatenate([k[b, :i, sl], kt[b, i:i + 1, sl]])
                vals = np.concatenate([v[b, :i, sl], vt[b, i:i + 1, sl]])
                bias = None if cfg.alibi_slopes is None else -cfg.slope(h) * (i - np.arange(i + 1))
                c[sl] = attn(keys, vals, q[b, i, sl], s, bias)
            a = c @ w.w_o.T
            hres = x[b, i] + cfg.residual_scale * a
            z2[b, i] = hres + cfg.residual_scale * _mlp(hres, w, cfg)
    return z2, k, v



# ----------------------------------------------------------------------------- blocked recurrence

def layer_blockrec(cfg: RTConfig, w: RTWeights, x: np.ndarray, S: int):
    """Recurrence executed over blocks of S positions (Sec. 9 names this extension in one sentence and does not
    define it; the reading taken here): positions are grouped in consecutive blocks of S.  Position i attends
    to the PERSISTENT pairs (Eqs. 1-2, from the outputs z_j) of every position j in an earlier block and to the
    TEMPORARY pairs (from the inputs x_j, first display of Sec. 2.2) of the positions j <= i of its own block, so
    all positions of a block can be computed at once; the block's persistent pairs follow from its outputs.
    S = 1 is the layer of Sec. 2.2; S >= N is an ordinary pre-LN Transformer layer.  With ALiBi slopes the
    distance i - j applies to both kinds of pair.  Returns z, k, v like layer_seq."""
    x = np.asarray(x, dtype=np.float64)
    B, N, d = x.shape
    H, dh, s = cfg.n_heads, cfg.head_dim, cfg.softmax_scale
    z = np.zeros_like(x); k = np.zeros_like(x); v = np.zeros_like(x)
    q, kt, vt = _temp_qkv(x, w, cfg)
    for b in range(B):
        for i in range(N):
            blk = (i // S) * S                                   # first position of i's block
            c = np.zeros(d)
            for h in range(H):
                sl = slice(h * dh, (h + 1) * dh)
                keys = np.concatenate([k[b, :blk, sl], kt[b, blk:i + 1, sl]])
                vals = np.concatenate([v[b, :blk, sl], vt[b, blk:i + 1, sl]])
                bias = None if cfg.alibi_slopes is None else -cfg.slope(h) * (i - np.arange(i + 1))
                c[sl] = attn(keys, vals, q[b, i, sl], s, bias)
            z[b, i], k[b, i], v[b, i] = _output_and_persistent(x[b, i], c @ w.w_o.T, w, cfg)
    return z, k, v

# ----------------------------------------------------------------------------- O-dec

def layer_decode(cfg: RTConfig, w: RTWeights, x_new: np.ndarray, k_cache: np.ndarray,
                 v_cache: np.ndarray, pos: int):
    """One decode step = one iteration of the prefill loop (Sec. 5: a forward pass is a
    sequence of decode steps).  x_new [B, d]; caches [B, >=pos+1, d] hold pos persistent pairs;
    row pos is written.  Returns z_new [B, d]."""
    B, d = x_new.shape
    H, dh, s = cfg.n_heads, cfg.head_dim, cfg.softmax_scale
    z = np.zeros((B, d))
    for b in range(B):
        q, kt, vt = _temp_qkv(x_new[b], w, cfg)
        c = np.zeros(d)
        for h in range(H):
            sl = slice(h * dh, (h + 1) * dh)
            keys = np.concatenate([k_cache[b, :pos, sl], kt[None, sl]])
            vals = np.concatenate([v_cache[b, :pos, sl], vt[None, sl]])
            bias = None if cfg.alibi_slopes is None else -cfg.slope(h) * (pos - np.arange(pos + 1))
            c[sl] = attn(keys, vals, q[sl], s, bias)
        z[b], k_cache[b, pos], v_cache[b, pos] = _output_and_persistent(x_new[b], c @ w.w_o.T, w, cfg)
    return z


# ----------------------------------------------------------------------------- stack

def stack_prefill(cfg: RTConfig, layers: List[RTWeights], emb: np.ndarray, g_final,
                  ids: np.ndarray, all_logits: bool = False):
    """x^0 = E[ids]; x^l = layer_l(x^{l-1}); logits = E RMS_{g_final}(x^L) (tied head; the
    paper only says embedding and unembedding are those of an ordinary Transformer).
    Returns hidden [B,N,d], logits ([B,V] for the last position, or [B,N,V]), and the
    per-layer caches [(k, v), ...]."""
    emb = np.asarray(emb, dtype=np.float64)
    x = emb[np.asarray(ids)]
    caches = []
    for w in layers:
        x, k, v = layer_seq(cfg, w, x)
        caches.append((k, v))
    gf = np.ones(cfg.d_model) if g_final is None else np.asarray(g_final, dtype=np.float64)
    src = x if all_logits else x[:, -1]
    logits = _pre(src, gf, cfg) @ emb.T
    return x, logits, caches


def stack_decode(cfg: RTConfig, layers: List[RTWeights], emb: np.ndarray, g_final,
                 ids_new: np.ndarray, caches, pos: int):
    """One token per sequence through every layer; caches as returned by stack_prefill but
    with room for row pos.  Returns logits [B, V]."""
    emb = np.asarray(emb, dtype=np.float64)
    x = emb[np.asarray(ids_new)]
    for w, (k, v) in zip(layers, caches):
        x = layer_decode(cfg, w, x, k, v, pos)
    gf = np.ones(cfg.d_model) if g_final is None else np.asarray(g_final, dtype=np.float64)
    return _pre(x, gf, cfg) @ emb.T
