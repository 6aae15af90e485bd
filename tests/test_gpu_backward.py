"""GPU parity of the layer's backward pass (rt_layer_backward; Sec. 6, "The backward pass") against the gradient
oracle (reverse-mode differentiation of the plain definition, fp64) on identical seeded inputs."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-4, "bf16": 2e-2}
G_NAMES = ("g_attn", "g_mlp", "g_kv", "g_q", "g_k")


def rel_err(got, ref):
    return float(np.abs(got - ref).max() / max(np.abs(ref).max(), 1e-30))


def _case(dtype, d, H, dff, B, N, seed, gains, alibi):
    from paper_2604_21215_b200 import inputs
    wl = inputs.Workload("bwd", 1, B, N, d, H, dff, dtype)
    data = inputs.make_inputs(wl, seed=seed)
    lw = data["layers"][0]
    rng = np.random.default_rng(seed + 1)
    for g in gains:
        lw[g] = inputs.round_to(1.0 + 0.2 * rng.standard_normal(d), dtype)
    slopes = np.array([2.0 ** (-8.0 * (h + 1) / H) for h in range(H)]) if alibi else None
    dz = rng.standard_normal(data["x"].shape).astype(np.float32).astype(np.float64)
    return data["x"], lw, slopes, dz


@pytest.mark.parametrize("dtype,d,H,dff,B,N,flags,gains,alibi,alpha", [
    ("f32", 128, 2, 256, 2, 150, 3, (), False, 1.0),                         # three leaves, ragged last one
    ("f32", 192, 3, 224, 3, 77, 3 | 8, G_NAMES, True, 0.5),                 # every gain, ALiBi, persistent pair from z itself
    ("f32", 128, 2, 256, 1, 64, 0, (), False, 1.0),                          # no norms, one full leaf
    ("f32", 128, 2, 128, 6, 70, 1, ("g_attn", "g_mlp"), False, 0.7),         # no qkRMS; RMS(z) shares g_attn; ragged row chunk
    ("f32", 64, 1, 96, 5, 1, 3, G_NAMES, False, 1.0),                        # a single position
    ("f32", 128, 2, 256, 2, 300, 3, ("g_k", "g_kv"), True, 1.0),             # cross tiles of 64, 128 and 256 keys
    ("bf16", 256, 4, 512, 3, 200, 3, G_NAMES, False, 1.0),
    ("bf16", 128, 2, 384, 9, 130, 3, (), True, 0.6),
    ("bf16", 192, 3, 224, 2, 96, 3, ("g_mlp", "g_q"), False, 1.0),            # widths off the tensor-core products
    ("bf16", 128, 2, 384, 3, 77, 3, G_NAMES, False, 0.8),                    # row count off the tensor-core dW products
    ("bf16", 128, 2, 256, 40, 70, 3, G_NAMES, True, 0.7),                    # wide batch: steps as dense products (tensor cores)
    ("f32", 128, 2, 160, 36, 66, 3 | 8, ("g_attn", "g_k"), False, 1.0),      # wide batch, fp32 products
    ("bf16", 192, 3, 224, 33, 65, 1, (), False, 1.0)])                       # wide batch, widths off the tensor-core products
def test_backward_matches_gradient_oracle(dtype, d, H, dff, B, N, flags, gains, alibi, alpha):
    from oracle import RTConfig, RTWeights, layer_grad
    from paper_2604_21215_b200 import inputs, rt
    x, lw, slopes, dz = _case(dtype, d, H, dff, B, N, 7700 + N, gains, alibi)
    cfg = RTConfig(d, H, 64, dff, norm_flags=flags, residual_scale=alpha, alibi_slopes=slopes)
    z_ref, dx_ref, g_ref = layer_grad(cfg, RTWeights(**lw), x, dz)
    layer = rt.Layer(d, H, dff, dtype=dtype, norm_flags=flags, residual_scale=alpha)
    layer.set_weights(dict(lw, alibi_slopes=slopes) if alibi else lw)
    dx, g = layer.backward(x, inputs.round_to(z_ref, dtype), dz)
    tol = TOL[dtype]
    assert np.isfinite(dx).all()
    assert rel_err(dx, dx_ref) <= tol, ("dx", rel_err(dx, dx_ref))
    want = {"w_q", "w_k", "w_v", "w_o", "w_up", "w_down"} | set(gains)
    assert set(g) == want
    for name in sorted(want):
        if np.abs(g_ref[name]).max() == 0.0:                                  # e.g. a gain no norm uses; q, k at N = 1
            assert np.abs(g[name]).max() <= tol * np.abs(dx_ref).max(), name   # zero up to the rounding of the other terms
            continue
        assert rel_err(g[name], g_ref[name]) <= tol, (name, rel_err(g[name], g_ref[name]))


def test_backward_from_the_prefill_outputs_and_determinism():
    # z as the GPU's own prefill returned it (what a training step has at hand); two runs agree bit for bit
    from oracle import RTConfig, RTWeights, layer_grad
    from paper_2604_21215_b200 import rt
    d, H, dff, B, N = 128, 2, 256, 4, 200
    x, lw, _, dz = _case("f32", d, H, dff, B, N, 31, ("g_attn", "g_kv"), False)
    layer = rt.Layer(d, H, dff, dtype="f32")
    layer.set_weights(lw)
    z, _, _ = layer.prefill(x)
    dx1, g1 = layer.backward(x, z, dz)
    dx2, g2 = layer.backward(x, z, dz)
    assert np.array_equal(dx1, dx2) and all(np.array_equal(g1[n], g2[n]) for n in g1)
    _, dx_ref, g_ref = layer_grad(RTConfig(d, H, 64, dff), RTWeights(**lw), x, dz)
    assert rel_err(dx1, dx_ref) <= TOL["f32"]
    for n in g1:
        assert rel_err(g1[n], g_ref[n]) <= TOL["f32"], n


def test_backward_one_launch_per_step_form_agrees():
    # the same device code as one launch per step (the form for devices without cooperative launch)
    from paper_2604_21215_b200 import rt
    for dtype, B in (("f32", 3), ("bf16", 6)):
        d, H, dff, N = 128, 2, 256, 140
        x, lw, _, dz = _case(dtype, d, H, dff, B, N, 77, ("g_attn", "g_k"), False)
        layer = rt.Layer(d, H, dff, dtype=dtype)
        layer.set_weights(lw)
        z, _, _ = layer.prefill(x)
        dx1, g1 = layer.backward(x, z, dz)
        layer.cfg.flags = rt.RT_FLAG_BACKWARD_STEP_LAUNCHES
        dx2, g2 = layer.backward(x, z, dz)
        layer.cfg.flags = 0
        # same arithmetic, separately compiled: equal up to the contraction of multiply-adds
        tol = 1e-5 if dtype == "f32" else 1e-3             # bf16: a last-bit change can flip an operand's bf16 rounding
        assert rel_err(dx2, dx1) <= tol and all(rel_err(g2[n], g1[n]) <= tol for n in g1)


def test_backward_directional_derivative_at_c2_shape():
    # Full c2 shape (B = 4, N = 2048, d = 768: 32 leaves, tiles backwards up to 1024 keys), fp32 storage, where the
    # gradient oracle would take far too long: the property that holds at any size is
    #   (L(x + e v) - L(x - e v)) / (2 e) = <dL/dx, v>,  L = sum(z * dz),
    # with L evaluated by the GPU's own forward pass (itself checked against the oracle elsewhere), and likewise along a
    # direction in W_v (which enters both the temporary and the persistent pairs) and in W_down.
    import torch
    from paper_2604_21215_b200 import inputs, rt
    wl = inputs.WORKLOADS["c2"]
    d, H, dff, B, N = wl.d_model, wl.n_heads, wl.d_ff, wl.B, wl.N
    x, lw, _, dz = _case("f32", d, H, dff, B, N, 4242, ("g_attn", "g_kv", "g_k"), False)
    rng = np.random.default_rng(99)
    layer = rt.Layer(d, H, dff, dtype="f32")

    def loss(xx, ww):
        layer.set_weights(ww)
        z, _, _ = layer.prefill(xx)
        return z, float(np.sum(z * dz))

    z0, _ = loss(x, lw)
    dx, g = layer.backward(x, z0, dz)
    assert np.isfinite(dx).all()
    eps = 2e-3

    def f32(a):
        return a.astype(np.float32).astype(np.float64)

    v = rng.standard_normal(x.shape)
    xp, xm = f32(x + eps * v), f32(x - eps * v)
    fd = (loss(xp, lw)[1] - loss(xm, lw)[1])
    an = float(np.sum(dx * (xp - xm)))                      # the step actually taken after rounding to fp32
    assert abs(fd - an) <= 1e-2 * abs(fd), ("x", fd, an)
    for name in ("w_v", "w_down"):
        dirn = rng.standard_normal(lw[name].shape) / np.sqrt(lw[name].shape[1])
        wp, wm = dict(lw), dict(lw)
        wp[name], wm[name] = f32(lw[name] + eps * dirn), f32(lw[name] - eps * dirn)
        fd = loss(x, wp)[1] - loss(x, wm)[1]
        an = float(np.sum(g[name] * (wp[name] - wm[name])))
        assert abs(fd - an) <= 1e-2 * abs(fd), (name, fd, an)


def test_backward_argument_errors():
    import torch
    from paper_2604_21215_b200 import rt
    x, lw, _, dz = _case("f32", 128, 2, 256, 1, 8, 1, (), False)
    layer = rt.Layer(128, 2, 256, dtype="f32")
    layer.set_weights(lw)
    xd = torch.zeros((1, 8, 128), device="cuda"); zd = torch.zeros_like(xd); dzd = torch.zeros_like(xd); dxd = torch.zeros_like(xd)
    need = rt.rt_backward_workspace_bytes(layer.cfg, 1, 8)
    assert need > 0
    ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
    gr = rt.RtLayerGrads()
    call = lambda x_, nbytes, cfg=layer.cfg: rt.rt_layer_backward(cfg, layer.w, x_, zd.data_ptr(), dzd.data_ptr(), 1, 8, dxd.data_ptr(),
                                                                  gr, ws.data_ptr(), nbytes, 0)
    assert call(xd.data_ptr(), need) == rt.RT_OK                               # no parameter gradient requested: dx only
    assert call(None, need) == rt.RT_ERR_INVALID_ARG
    assert call(xd.data_ptr(), need - 1) == rt.RT_ERR_WORKSPACE
    blocked = rt.make_config(128, 2, 256, dtype="f32", recur_block=4)
    assert call(xd.data_ptr(), need, blocked) == rt.RT_ERR_UNSUPPORTED
    torch.cuda.synchronize()
