"""GPU parity of the parallel sweep (rt_layer_recompute; Sec. 6, activation checkpointing) against the
oracle's layer_fixed_point on identical seeded inputs, and its use as a verifier of the prefill."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-4, "bf16": 2e-2}


def rel_err(got, ref):
    return float(np.abs(got - ref).max() / np.abs(ref).max())


def _case(dtype, d, H, dff, B, N, seed, gains=False, alibi=False):
    from paper_2604_21215_b200 import inputs
    wl = inputs.Workload("rec", 1, B, N, d, H, dff, dtype)
    data = inputs.make_inputs(wl, seed=seed)
    lw = data["layers"][0]
    if gains:
        rng = np.random.default_rng(seed + 1)
        for g in ("g_attn", "g_mlp", "g_kv", "g_q", "g_k"):
            lw[g] = inputs.round_to(1.0 + 0.2 * rng.standard_normal(d), dtype)
    slopes = np.array([2.0 ** (-8.0 * (h + 1) / H) for h in range(H)]) if alibi else None
    return data["x"], lw, slopes


@pytest.mark.parametrize("dtype,d,H,dff,B,N,flags,gains,alibi,alpha", [
    ("f32", 128, 2, 512, 2, 150, 3, False, False, 1.0),
    ("f32", 192, 3, 208, 3, 77, 3 | 8, True, True, 0.5),
    ("f32", 128, 2, 256, 1, 64, 0, False, False, 1.0),
    ("bf16", 256, 4, 1024, 3, 333, 3, True, False, 1.0),
    ("bf16", 768, 12, 3072, 2, 300, 3, False, True, 0.6),
    ("bf16", 320, 5, 384, 5, 129, 1, False, False, 1.0),
    ("bf16", 128, 2, 512, 16, 1, 3, False, False, 1.0),
    # 9950 rows (not a multiple of the 256-row pair tiles) and 10240 rows with N a multiple of 128: the products and the
    # projections run on persistent CTA pairs, the second case's attention as one causal launch with ALiBi distances
    ("bf16", 256, 4, 1024, 5, 1990, 3, True, False, 1.0),
    ("bf16", 256, 4, 1024, 5, 2048, 3, False, True, 0.7)])
def test_recompute_matches_fixed_point_sweep(dtype, d, H, dff, B, N, flags, gains, alibi, alpha):
    # z_claim is NOT the true output (random): the sweep must still reproduce the oracle's one-sweep map
    # z_claim -> (z', k, v), which exercises every product and every attention pair without relying on
    # the fixed point.
    from oracle import RTConfig, RTWeights, layer_fixed_point
    from paper_2604_21215_b200 import inputs, rt
    x, lw, slopes = _case(dtype, d, H, dff, B, N, 9100 + N, gains, alibi)
    rng = np.random.default_rng(N)
    zc = inputs.round_to(x + 0.5 * rng.standard_normal(x.shape), dtype)
    cfg = RTConfig(d, H, 64, dff, norm_flags=flags, residual_scale=alpha, alibi_slopes=slopes)
    z_ref, k_ref, v_ref = layer_fixed_point(cfg, RTWeights(**lw), x, zc)
    layer = rt.Layer(d, H, dff, dtype=dtype, norm_flags=flags, residual_scale=alpha)
    layer.set_weights(dict(lw, alibi_slopes=slopes) if alibi else lw)
    z, k, v = layer.recompute(x, zc)
    tol = TOL[dtype]
    assert np.isfinite(z).all()
    assert rel_err(k, k_ref) <= tol and rel_err(v, v_ref) <= tol
    assert rel_err(z, z_ref) <= tol


def test_prefill_output_is_the_fixed_point_of_the_sweep_at_c2_size():
    # The GPU's own prefill output, fed back through the GPU's parallel sweep, must come back unchanged
    # (the true z is the unique fixed point), and the rebuilt caches must equal the prefill's caches.
    import torch
    from paper_2604_21215_b200 import inputs, rt
    wl = inputs.WORKLOADS["c2"]
    data = inputs.make_inputs(wl)
    layer = rt.Layer(wl.d_model, wl.n_heads, wl.d_ff, dtype="bf16")
    layer.set_weights(data["layers"][0])
    z, k, v = layer.prefill(data["x"])
    z2, k2, v2 = layer.recompute(data["x"], z)
    assert rel_err(z2, z) <= TOL["bf16"]
    assert rel_err(k2, k) <= TOL["bf16"] and rel_err(v2, v) <= TOL["bf16"]
    # a perturbed claim is not a fixed point
    zp = z.copy(); zp[:, 100] += 0.5
    z3, _, _ = layer.recompute(data["x"], zp)
    assert np.abs(z3[:, 101:] - zp[:, 101:]).max() / np.abs(z).max() > 1e-2


def test_recompute_argument_errors():
    import torch
    from paper_2604_21215_b200 import inputs, rt
    x, lw, _ = _case("f32", 128, 2, 256, 1, 8, 1)
    layer = rt.Layer(128, 2, 256, dtype="f32")
    layer.set_weights(lw)
    layer.reserve(1, 8)
    xd = torch.zeros((1, 8, 128), device="cuda")
    zo = torch.zeros_like(xd)
    ws = torch.zeros(rt.rt_recompute_workspace_bytes(layer.cfg, 1, 8), dtype=torch.uint8, device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    args = lambda x_, zc_, zo_, nbytes: rt.rt_layer_recompute(layer.cfg, layer.w, x_, zc_, 1, 8, zo_, layer.k_cache.data_ptr(),
                                                                layer.v_cache.data_ptr(), 8, ws.data_ptr(), nbytes, s)
    assert args(xd.data_ptr(), xd.data_ptr(), xd.data_ptr(), ws.numel()) == rt.RT_ERR_INVALID_ARG      # output aliases input
    assert args(xd.data_ptr(), xd.data_ptr(), zo.data_ptr(), 1024) == rt.RT_ERR_WORKSPACE
    assert args(None, xd.data_ptr(), zo.data_ptr(), ws.numel()) == rt.RT_ERR_INVALID_ARG
    assert args(xd.data_ptr(), xd.data_ptr(), zo.data_ptr(), ws.numel()) == rt.RT_OK
    torch.cuda.synchronize()
