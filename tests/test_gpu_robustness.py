"""GPU checks beyond element-wise parity: run-to-run determinism, writes confined to the result
buffers, and the two large configurations (the 8-layer stack at full size, a long sequence) via
properties the oracle can evaluate on sampled positions."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-4, "bf16": 2e-2}


def rel_err(got, ref):
    return float(np.abs(got - ref).max() / np.abs(ref).max())


def _layer(d, H, dff, dtype, lw, **kw):
    from paper_2604_21215_b200 import rt
    layer = rt.Layer(d, H, dff, dtype=dtype, **kw)
    layer.set_weights(lw)
    return layer


@pytest.mark.parametrize("dtype,d,H,dff,B,N", [("bf16", 768, 12, 3072, 4, 600), ("f32", 128, 2, 512, 3, 150)])
def test_repeat_runs_are_bit_identical(dtype, d, H, dff, B, N):
    # Every reduction has a fixed order (no floating-point atomics), so two runs must agree to the bit;
    # a race in an exchange or a merge would show up as a difference.
    import torch
    from paper_2604_21215_b200 import inputs
    wl = inputs.Workload("rep", 1, B, N, d, H, dff, dtype)
    data = inputs.make_inputs(wl, seed=910)
    layer = _layer(d, H, dff, dtype, data["layers"][0])
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    xd = torch.from_numpy(data["x"]).to(tdt).cuda()
    outs = []
    for _ in range(3):
        layer.reserve(B, N)
        layer.k_cache.zero_(); layer.v_cache.zero_()
        zd = torch.empty_like(xd)
        layer.prefill_device(xd, zd)
        torch.cuda.synchronize()
        assert layer.status() == 0
        outs.append((zd.clone(), layer.k_cache.clone(), layer.v_cache.clone()))
    for o in outs[1:]:
        for a, b in zip(outs[0], o):
            assert torch.equal(a, b)


@pytest.mark.parametrize("dtype,d,H,dff,B,N", [("bf16", 256, 4, 1024, 3, 333), ("f32", 128, 2, 512, 2, 77)])
def test_nothing_outside_the_result_buffers_is_written(dtype, d, H, dff, B, N):
    # z, the caches and the workspace sit inside larger allocations filled with a pattern; after the
    # call the guard bands on both sides (and the cache rows beyond N) must be unchanged.
    import torch
    from paper_2604_21215_b200 import inputs, rt
    wl = inputs.Workload("guard", 1, B, N, d, H, dff, dtype)
    data = inputs.make_inputs(wl, seed=911)
    layer = _layer(d, H, dff, dtype, data["layers"][0])
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    esz = 2 if dtype == "bf16" else 4
    guard = 4096                                   # bytes on each side
    N_max = N + 5

    def banded(nbytes):
        buf = torch.full((guard + nbytes + guard,), 0xA5, dtype=torch.uint8, device="cuda")
        return buf, buf[guard:guard + nbytes]

    xd = torch.from_numpy(data["x"]).to(tdt).cuda().contiguous()
    zbuf, zin = banded(B * N * d * esz)
    kbuf, kin = banded(N_max * B * d * esz)
    vbuf, vin = banded(N_max * B * d * esz)
    need = rt.rt_workspace_bytes(layer.cfg, B, N, 1)
    wbuf, win = banded(need)
    win.zero_()
    s = torch.cuda.current_stream().cuda_stream
    st = rt.rt_layer_prefill(layer.cfg, layer.w, xd.data_ptr(), B, N, zin.data_ptr(), kin.data_ptr(), vin.data_ptr(), N_max,
                             win.data_ptr(), need, s)
    torch.cuda.synchronize()
    assert st == rt.RT_OK and rt.rt_get_status(win.data_ptr()) == rt.RT_OK
    for buf in (zbuf, kbuf, vbuf, wbuf):
        assert bool((buf[:guard] == 0xA5).all()) and bool((buf[-guard:] == 0xA5).all())
    tail = N * B * d * esz                          # cache rows N .. N_max are not part of the result
    assert bool((kin[tail:] == 0xA5).all()) and bool((vin[tail:] == 0xA5).all())
    # and the result itself is the usual one
    z = zin.view(tdt).view(B, N, d).to(torch.float64).cpu().numpy()
    from oracle import RTConfig, RTWeights, layer_seq
    ref = layer_seq(RTConfig(d, H, 64, dff), RTWeights(**data["layers"][0]), data["x"])
    assert rel_err(z, ref[0]) <= TOL[dtype]


@pytest.mark.parametrize("N", [8192, 16384, 32768])
def test_long_sequence_fixed_point_on_sampled_positions(N):
    # Points of the sequence-length sweep (B=1, d=1024; at N=32768 the cross tiles reach 16384 x 16384).
    # The oracle rebuilds all pairs from the GPU's z and recomputes sampled positions independently:
    # both sides of every boundary of the three largest tile levels, the two ends, and a random draw.
    from oracle import RTConfig, RTWeights, layer_fixed_point
    from parity_metrics import check_tensor
    from paper_2604_21215_b200 import inputs
    wl = inputs.sweep(N)
    data = inputs.make_inputs(wl)
    lw = data["layers"][0]
    layer = _layer(wl.d_model, wl.n_heads, wl.d_ff, "bf16", lw)
    z, k, v = layer.prefill(data["x"])
    assert np.isfinite(z).all()
    edges = [N // 8 * i for i in range(1, 8)]
    rows = np.r_[0:6, N - 6:N]
    for e in edges:
        rows = np.r_[rows, e - 3:e + 3]
    rng = np.random.default_rng(N)
    rows = np.unique(np.r_[rows, rng.choice(N, 12, replace=False)])
    cfg = RTConfig(wl.d_model, wl.n_heads, 64, wl.d_ff)
    z2, k2, v2 = layer_fixed_point(cfg, RTWeights(**lw), data["x"], z, rows=rows)
    err = np.abs(z2[:, rows] - z[:, rows]).max(axis=(0, 2)) / np.abs(z).max()
    assert err.max() <= TOL["bf16"], f"N={N}: worst sampled position {int(rows[err.argmax()])}, error {err.max():.3e}"
    # no growth along the sequence (Sec. 4): the late half of the samples is no worse than the bound allows
    assert err[rows >= N // 2].max() <= max(10.0 * err[rows < N // 2].max(), TOL["bf16"] / 20.0)
    check_tensor(f"c5 N={N}", "k (rebuilt from z)", k, k2, TOL["bf16"])
    check_tensor(f"c5 N={N}", "v (rebuilt from z)", v, v2, TOL["bf16"])


def test_stack_full_size_is_consistent_with_its_layers():
    # Configuration 4 at full size (8 layers, B=16, N=2048, vocabulary 32000).  The oracle cannot replay
    # it, so: (1) the stack call equals chaining the single-layer call over a gathered embedding, bit for
    # bit (same kernels, same order); (2) the last layer passes the fixed-point check on sampled positions
    # of one sequence; (3) the logits equal the tied head applied in fp64 to the returned hidden state.
    import torch
    from oracle import RTConfig, RTWeights, layer_fixed_point, rms
    from paper_2604_21215_b200 import inputs, rt
    wl = inputs.WORKLOADS["c4"]
    data = inputs.make_inputs(wl)
    L, d, H, dff, V, B, N = wl.n_layers, wl.d_model, wl.n_heads, wl.d_ff, wl.vocab, wl.B, wl.N
    st = rt.Stack(L, d, H, dff, V, dtype="bf16", residual_scale=wl.residual_scale)
    st.set_weights(data["layers"], data["emb"])
    ids = torch.as_tensor(np.asarray(data["ids"]), dtype=torch.int32, device="cuda").contiguous()
    st.reserve(B, N)
    hid = torch.empty((B, N, d), dtype=torch.bfloat16, device="cuda")
    logits = torch.empty((B, V), dtype=torch.float32, device="cuda")
    st.prefill_device(ids, hid, logits)
    torch.cuda.synchronize()
    assert st.status() == 0
    # (1) chain of single-layer calls; (2) every layer passes the fixed-point check on sampled positions of one
    # sequence (a different sequence per layer): the oracle rebuilds the layer's pairs from its output and
    # recomputes the sampled positions from the layer's input
    from parity_metrics import check_tensor
    cfg = RTConfig(d, H, 64, dff, residual_scale=wl.residual_scale)
    x = st.emb[ids.long()].contiguous()
    x_last = None
    for li in range(L):
        layer = rt.Layer(d, H, dff, dtype="bf16", residual_scale=wl.residual_scale)
        layer.set_weights(data["layers"][li])
        layer.reserve(B, N)
        z = torch.empty_like(x)
        layer.prefill_device(x, z)
        torch.cuda.synchronize()
        assert layer.status() == 0
        assert torch.equal(layer.k_cache, st.k_caches[li]) and torch.equal(layer.v_cache, st.v_caches[li])
        b = (5 * li + 3) % B
        sel = slice(b, b + 1)
        rows = np.unique(np.r_[0:6, 508:516, 1020:1030, 1532:1540, 2042:2048,
                               np.random.default_rng(li).choice(N, 6, replace=False)])
        xin = x[sel].to(torch.float64).cpu().numpy()
        zc = z[sel].to(torch.float64).cpu().numpy()
        z2, k2, v2 = layer_fixed_point(cfg, RTWeights(**data["layers"][li]), xin, zc, rows=rows)
        assert np.abs(z2[:, rows] - zc[:, rows]).max() / np.abs(zc).max() <= TOL["bf16"], f"layer {li}"
        kg = st.k_caches[li][:, b].to(torch.float64).cpu().numpy()[None]
        vg = st.v_caches[li][:, b].to(torch.float64).cpu().numpy()[None]
        check_tensor(f"c4 layer {li} sequence {b}", "k (rebuilt from z)", kg, k2, TOL["bf16"])
        check_tensor(f"c4 layer {li} sequence {b}", "v (rebuilt from z)", vg, v2, TOL["bf16"])
        x_last, x = x, z
        del layer
    assert torch.equal(x, hid)
    # (3) tied head on the last position
    h_last = hid[:, -1].to(torch.float64).cpu().numpy()
    ref_logits = rms(h_last, np.ones(d), cfg.rms_eps) @ np.asarray(data["emb"], dtype=np.float64).T
    assert rel_err(logits.to(torch.float64).cpu().numpy(), ref_logits) <= TOL["bf16"]


def _random_cases():
    rng = np.random.default_rng(20260421)
    cases = []
    for i in range(14):
        H = int(rng.choice([1, 2, 3, 4, 5, 8]))
        d = 64 * H
        dff = int(rng.choice([128, 208, 384, 1024, 1536]))
        B = int(rng.integers(1, 17))
        N = int(rng.integers(1, 420))
        leaf = int(rng.choice([0, 16, 32, 64]))
        dtype = "bf16" if i % 3 else "f32"
        flags = int(rng.choice([3, 3, 3, 1, 2, 0, 3 | 8]))
        gains = bool(rng.integers(0, 2))
        alpha = float(rng.choice([1.0, 0.5, 1 / np.sqrt(8)]))
        cases.append((dtype, d, H, dff, B, N, leaf, flags, gains, alpha))
    return cases


@pytest.mark.parametrize("dtype,d,H,dff,B,N,leaf,flags,gains,alpha", _random_cases())
def test_random_shapes_match_oracle(dtype, d, H, dff, B, N, leaf, flags, gains, alpha):
    # Shapes off the beaten path: head counts that are not powers of two, MLP widths that are not
    # multiples of 64, every batch size up to 16, lengths with ragged last leaves, every leaf size,
    # norm flags, gains and residual scales; tiled schedule, both storage types.
    from oracle import RTConfig, RTWeights, layer_seq
    from paper_2604_21215_b200 import inputs
    wl = inputs.Workload("rnd", 1, B, N, d, H, dff, dtype)
    data = inputs.make_inputs(wl, seed=7000 + d + dff + B + N)
    lw = data["layers"][0]
    if gains:
        rng = np.random.default_rng(N)
        for g in ("g_attn", "g_mlp", "g_kv", "g_q", "g_k"):
            lw[g] = inputs.round_to(1.0 + 0.2 * rng.standard_normal(d), dtype)
    ref = layer_seq(RTConfig(d, H, 64, dff, norm_flags=flags, residual_scale=alpha), RTWeights(**lw), data["x"])
    layer = _layer(d, H, dff, dtype, lw, leaf=leaf, norm_flags=flags, residual_scale=alpha)
    got = layer.prefill(data["x"])
    for name, g_, r_ in zip(("z", "k", "v"), got, ref):
        assert np.isfinite(g_).all(), name
        assert rel_err(g_, r_) <= TOL[dtype], (name, rel_err(g_, r_))


# ---------------------------------------------------------------- ALiBi distances (optional slopes per head)

def _slopes(H, max_bias=8.0):
    return np.array([2.0 ** (-max_bias * (h + 1) / H) for h in range(H)])


@pytest.mark.parametrize("dtype,d,H,dff,B,N,leaf,sched", [
    ("f32", 128, 2, 512, 2, 150, 16, "tiled"), ("f32", 128, 2, 512, 3, 70, 0, "naive"),
    ("bf16", 256, 4, 1024, 5, 300, 32, "tiled"), ("bf16", 768, 12, 3072, 4, 520, 0, "tiled"),
    ("bf16", 512, 8, 2048, 16, 200, 0, "tiled"), ("bf16", 256, 4, 512, 3, 260, 64, "naive")])
def test_alibi_prefill_matches_oracle(dtype, d, H, dff, B, N, leaf, sched):
    from oracle import RTConfig, RTWeights, layer_seq
    from paper_2604_21215_b200 import inputs
    wl = inputs.Workload("alibi", 1, B, N, d, H, dff, dtype)
    data = inputs.make_inputs(wl, seed=8100 + N)
    lw = data["layers"][0]
    ref = layer_seq(RTConfig(d, H, 64, dff, alibi_slopes=_slopes(H)), RTWeights(**lw), data["x"])
    base = layer_seq(RTConfig(d, H, 64, dff), RTWeights(**lw), data["x"])
    assert rel_err(base[0], ref[0]) > 10 * TOL[dtype]          # the distances do change the result
    lw = dict(lw, alibi_slopes=_slopes(H))
    layer = _layer(d, H, dff, dtype, lw, leaf=leaf, sched=sched)
    got = layer.prefill(data["x"])
    for name, g_, r_ in zip(("z", "k", "v"), got, ref):
        assert rel_err(g_, r_) <= TOL[dtype], (name, rel_err(g_, r_))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_alibi_prefill_then_decode_matches_oracle(dtype):
    from oracle import RTConfig, RTWeights, layer_seq
    from paper_2604_21215_b200 import inputs
    d, H, dff, B, N = 128, 2, 256, 3, 45
    wl = inputs.Workload("alibi_dec", 1, B, N + 2, d, H, dff, dtype)
    data = inputs.make_inputs(wl, seed=8200)
    lw = data["layers"][0]
    ref = layer_seq(RTConfig(d, H, 64, dff, alibi_slopes=_slopes(H)), RTWeights(**lw), data["x"])
    layer = _layer(d, H, dff, dtype, dict(lw, alibi_slopes=_slopes(H)), leaf=16)
    got = layer.prefill(data["x"][:, :N], N_max=N + 2)
    assert rel_err(got[0], ref[0][:, :N]) <= TOL[dtype]
    for step in range(2):
        zn = layer.decode(data["x"][:, N + step], N + step)
        assert rel_err(zn, ref[0][:, N + step]) <= TOL[dtype]


@pytest.mark.parametrize("dtype,nq,nk", [("bf16", 200, 128), ("bf16", 130, 320), ("f32", 40, 50)])
def test_alibi_update_tile_matches_algorithm_2(dtype, nq, nk):
    # Algorithm 2 alone with distances: tensor-core kernel (bf16, key counts that are multiples of 64) and SIMT kernel
    import torch
    from oracle import update_tile
    from paper_2604_21215_b200 import inputs, rt
    B, H, d = 2, 3, 192
    rng = np.random.default_rng(8300 + nq)
    rows = 16 + nk + nq
    k0, k1, q0, q1 = 16, 16 + nk, 16 + nk, 16 + nk + nq
    q = inputs.round_to(rng.standard_normal((rows, B, d)), dtype)
    k = inputs.round_to(rng.standard_normal((rows, B, d)), dtype)
    v = inputs.round_to(rng.standard_normal((rows, B, d)), dtype)
    scale = 0.125
    slopes = _slopes(H)
    m0 = rng.standard_normal((rows, B, H)); l0 = 1.0 + rng.random((rows, B, H)); o0 = rng.standard_normal((rows, B, d))
    m_ref, l_ref, o_ref = m0.copy(), l0.copy(), o0.copy()
    dist = np.arange(q0, q1)[:, None] - np.arange(k0, k1)[None, :]
    for b in range(B):
        for h in range(H):
            sl = slice(64 * h, 64 * h + 64)
            m2, l2, o2 = update_tile(q[q0:q1, b, sl], k[k0:k1, b, sl], v[k0:k1, b, sl], m0[q0:q1, b, h], l0[q0:q1, b, h],
                                     o0[q0:q1, b, sl], scale, -slopes[h] * dist)
            m_ref[q0:q1, b, h], l_ref[q0:q1, b, h], o_ref[q0:q1, b, sl] = m2, l2, o2
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    dev = lambda a, t=tdt: torch.from_numpy(np.ascontiguousarray(a)).to(t).cuda()
    qd, kd, vd = dev(q), dev(k), dev(v)
    LOG2E = 1.4426950408889634
    od, md, ld = dev(o0, torch.float32), dev(m0 * LOG2E, torch.float32), dev(l0, torch.float32)
    sd = dev(slopes, torch.float32)
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    cfg = rt.make_config(d, H, 4 * d, dtype=dtype, softmax_scale=scale)
    st = rt.rt_update_tile(cfg, qd.data_ptr(), kd.data_ptr(), vd.data_ptr(), od.data_ptr(), md.data_ptr(), ld.data_ptr(),
                           B, rows, rows, q0, q1, k0, k1, sd.data_ptr(), ws.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert st == rt.RT_OK and rt.rt_get_status(ws.data_ptr()) == rt.RT_OK
    # compare what is unique: the normalised output o/l and the log-sum m + log2(l)
    og, mg, lg = (t.to(torch.float64).cpu().numpy() for t in (od, md, ld))
    tol = TOL[dtype]
    for h in range(H):
        sl = slice(64 * h, 64 * h + 64)
        a_g = og[..., sl] / lg[..., h:h + 1]
        a_r = o_ref[..., sl] / l_ref[..., h:h + 1]
        assert np.abs(a_g - a_r).max() / np.abs(a_r).max() <= tol
    lse_g = mg / LOG2E + np.log(lg)
    lse_r = m_ref + np.log(l_ref)
    assert np.abs(lse_g - lse_r).max() <= tol * max(1.0, np.abs(lse_r).max())


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_alibi_stack_prefill_and_decode_match_oracle(dtype):
    from oracle import RTConfig, RTWeights, stack_prefill, stack_decode
    from paper_2604_21215_b200 import inputs, rt
    L, d, H, dff, V, B, N = 3, 128, 2, 256, 300, 2, 70
    wl = inputs.Workload("alibi_stack", L, B, N + 1, d, H, dff, dtype, vocab=V, residual_scale=1 / np.sqrt(L))
    data = inputs.make_inputs(wl, seed=8400)
    slopes = _slopes(H)
    ocfg = RTConfig(d, H, 64, dff, residual_scale=wl.residual_scale, alibi_slopes=slopes)
    ow = [RTWeights(**lw) for lw in data["layers"]]
    hid_ref, logits_ref, caches_ref = stack_prefill(ocfg, ow, data["emb"], None, data["ids"])
    st = rt.Stack(L, d, H, dff, V, dtype=dtype, leaf=16, residual_scale=wl.residual_scale)
    st.set_weights([dict(lw, alibi_slopes=slopes) for lw in data["layers"]], data["emb"])
    hid, logits = st.prefill(data["ids"])
    tol = TOL[dtype]
    assert rel_err(hid, hid_ref) <= tol and rel_err(logits, logits_ref) <= tol
    hid2, _ = st.prefill(data["ids"][:, :N], N_max=N + 1)
    assert rel_err(hid2, hid_ref[:, :N]) <= tol
    lg = st.decode(data["ids"][:, N], N)
    assert rel_err(lg, logits_ref) <= tol


# ---------------------------------------------------------------- wide batches: the token step as dense products

@pytest.mark.parametrize("dtype,d,H,dff,B,N,leaf,alibi", [
    ("f32", 128, 2, 256, 70, 40, 16, False), ("bf16", 256, 4, 1024, 130, 75, 32, True),
    ("bf16", 128, 2, 512, 96, 33, 16, False), ("bf16", 256, 4, 768, 40, 50, 0, False),
    ("bf16", 192, 3, 208, 30, 40, 16, True)])
def test_wide_batch_prefill_matches_oracle(dtype, d, H, dff, B, N, leaf, alibi):
    # B > 64 (bf16: B > 48): every token step runs as dense products over the B rows (tensor cores for bf16); the bf16
    # cases with B = 30 and 40 run as slices through the small-batch kernel
    from oracle import RTConfig, RTWeights, layer_seq
    from paper_2604_21215_b200 import inputs
    wl = inputs.Workload("wide", 1, B, N, d, H, dff, dtype)
    data = inputs.make_inputs(wl, seed=8500 + B)
    lw = data["layers"][0]
    slopes = _slopes(H) if alibi else None
    ref = layer_seq(RTConfig(d, H, 64, dff, alibi_slopes=slopes, residual_scale=0.7), RTWeights(**lw), data["x"])
    layer = _layer(d, H, dff, dtype, dict(lw, alibi_slopes=slopes) if alibi else lw, leaf=leaf, residual_scale=0.7)
    got = layer.prefill(data["x"])
    for name, g_, r_ in zip(("z", "k", "v"), got, ref):
        assert np.isfinite(g_).all(), name
        assert rel_err(g_, r_) <= TOL[dtype], (name, rel_err(g_, r_))


@pytest.mark.parametrize("d,H,dff,B,N,leaf", [(256, 4, 1024, 17, 150, 16), (128, 2, 512, 33, 200, 0), (256, 4, 768, 48, 90, 32)])
def test_batches_of_17_to_48_run_as_slices_of_the_small_batch_kernel(d, H, dff, B, N, leaf):
    # bf16, tiled: the sequences are independent (Sec. 2.2), so such a batch runs as 2 or 3 slices of at most 16
    # sequences through the tensor-core leaf kernel and shares the pre-pass and the cross tiles.  Checked against the
    # oracle, and bit for bit against the same slices run as batches of their own.
    from oracle import RTConfig, RTWeights, layer_seq
    from paper_2604_21215_b200 import inputs
    wl = inputs.Workload("split", 1, B, N, d, H, dff, "bf16")
    data = inputs.make_inputs(wl, seed=8550 + B)
    lw = data["layers"][0]
    ref = layer_seq(RTConfig(d, H, 64, dff, residual_scale=0.8), RTWeights(**lw), data["x"])
    layer = _layer(d, H, dff, "bf16", lw, leaf=leaf, residual_scale=0.8)
    got = layer.prefill(data["x"])
    for name, g_, r_ in zip(("z", "k", "v"), got, ref):
        assert np.isfinite(g_).all(), name
        assert rel_err(g_, r_) <= TOL["bf16"], (name, rel_err(g_, r_))
    n_sub = (B + 15) // 16
    sub = (B + n_sub - 1) // n_sub
    for b0 in range(0, B, sub):
        part = _layer(d, H, dff, "bf16", lw, leaf=leaf, residual_scale=0.8).prefill(data["x"][b0:b0 + sub])
        for name, g_, p_ in zip(("z", "k", "v"), got, part):
            assert np.array_equal(g_[b0:b0 + sub], p_), (name, b0)


def test_wide_batch_unsupported_paths_say_so():
    from paper_2604_21215_b200 import inputs, rt
    d, H, dff, B, N = 128, 2, 256, 70, 8
    wl = inputs.Workload("wide", 1, B, N, d, H, dff, "f32")
    data = inputs.make_inputs(wl, seed=1)
    layer = _layer(d, H, dff, "f32", data["layers"][0], sched="naive")
    with pytest.raises(rt.RtError) as ei:
        layer.prefill(data["x"])
    assert ei.value.status == rt.RT_ERR_UNSUPPORTED


@pytest.mark.parametrize("gains", [False, True])
def test_phase_timer_variants_compute_the_same(gains):
    # rt_profile_enable(2) selects the leaf-kernel variants with the per-phase timers compiled in; they must
    # give the same output bit for bit and leave non-zero phase times in the workspace's sync area.
    import torch
    from paper_2604_21215_b200 import inputs, rt
    d, H, dff, B, N = 256, 4, 1024, 3, 150
    wl = inputs.Workload("timers", 1, B, N, d, H, dff, "bf16")
    data = inputs.make_inputs(wl, seed=8600)
    lw = data["layers"][0]
    if gains:
        rng = np.random.default_rng(5)
        for g in ("g_attn", "g_mlp", "g_kv", "g_q", "g_k"):
            lw[g] = inputs.round_to(1.0 + 0.2 * rng.standard_normal(d), "bf16")
    layer = _layer(d, H, dff, "bf16", lw)
    xd = torch.from_numpy(data["x"]).to(torch.bfloat16).cuda()
    layer.reserve(B, N)
    outs = []
    try:
        for mode in (0, 2):
            rt.rt_profile_enable(mode)
            zd = torch.empty_like(xd)
            layer.prefill_device(xd, zd)
            torch.cuda.synchronize()
            assert layer.status() == 0
            phase_ns = layer.ws[:256].cpu().numpy().view(np.uint64)[2:12]
            outs.append((zd.clone(), layer.k_cache.clone(), int(phase_ns.sum())))
    finally:
        rt.rt_profile_enable(0)
        rt.rt_profile_read()
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
    assert outs[0][2] == 0 and outs[1][2] > 0


# ---------------------------------------------------------------- recurrence over blocks of positions (config.recur_block)

@pytest.mark.parametrize("dtype,d,H,dff,B,N,S,alibi", [
    ("f32", 128, 2, 256, 2, 70, 16, False), ("f32", 128, 2, 256, 3, 50, 7, True), ("f32", 128, 2, 512, 2, 40, 64, False),
    ("bf16", 256, 4, 1024, 3, 300, 64, False), ("bf16", 256, 4, 1024, 2, 520, 256, True), ("bf16", 768, 12, 3072, 2, 200, 32, False),
    ("bf16", 128, 2, 512, 70, 48, 16, False)])
def test_blocked_recurrence_matches_oracle(dtype, d, H, dff, B, N, S, alibi):
    from oracle import RTConfig, RTWeights, layer_blockrec, layer_seq
    from paper_2604_21215_b200 import inputs
    wl = inputs.Workload("blockrec", 1, B, N, d, H, dff, dtype)
    data = inputs.make_inputs(wl, seed=8700 + N + S)
    lw = data["layers"][0]
    slopes = _slopes(H) if alibi else None
    cfg = RTConfig(d, H, 64, dff, alibi_slopes=slopes, residual_scale=0.8)
    ref = layer_blockrec(cfg, RTWeights(**lw), data["x"], S)
    if S < N:
        assert rel_err(layer_seq(cfg, RTWeights(**lw), data["x"])[0], ref[0]) > 10 * TOL[dtype]    # a different model
    layer = _layer(d, H, dff, dtype, dict(lw, alibi_slopes=slopes) if alibi else lw, residual_scale=0.8, recur_block=S)
    got = layer.prefill(data["x"])
    for name, g_, r_ in zip(("z", "k", "v"), got, ref):
        assert np.isfinite(g_).all(), name
        assert rel_err(g_, r_) <= TOL[dtype], (name, rel_err(g_, r_))


def test_blocked_recurrence_unsupported_paths_say_so():
    from paper_2604_21215_b200 import inputs, rt
    d, H, dff, B, N = 128, 2, 256, 2, 20
    wl = inputs.Workload("blockrec", 1, B, N, d, H, dff, "f32")
    data = inputs.make_inputs(wl, seed=2)
    layer = _layer(d, H, dff, "f32", data["layers"][0], recur_block=8)
    layer.prefill(data["x"][:, :16], N_max=N)
    with pytest.raises(rt.RtError) as ei:
        layer.decode(data["x"][:, 16], 16)
    assert ei.value.status == rt.RT_ERR_UNSUPPORTED
    with pytest.raises(rt.RtError) as ei:
        layer.recompute(data["x"], data["x"])
    assert ei.value.status == rt.RT_ERR_UNSUPPORTED


def test_blocked_recurrence_stack_matches_oracle():
    # the stack entry point with recur_block: embedding, L blocked layers, final norm and tied head
    from oracle import RTConfig, RTWeights, layer_blockrec, rms
    from paper_2604_21215_b200 import inputs, rt
    L, d, H, dff, V, B, N, S = 2, 128, 2, 256, 200, 2, 60, 16
    wl = inputs.Workload("blockrec_stack", L, B, N, d, H, dff, "f32", vocab=V, residual_scale=1 / np.sqrt(L))
    data = inputs.make_inputs(wl, seed=8800)
    cfg = RTConfig(d, H, 64, dff, residual_scale=wl.residual_scale)
    x = np.asarray(data["emb"], dtype=np.float64)[np.asarray(data["ids"])]
    for lw in data["layers"]:
        x, _, _ = layer_blockrec(cfg, RTWeights(**lw), x, S)
    logits_ref = rms(x[:, -1], np.ones(d), cfg.rms_eps) @ np.asarray(data["emb"], dtype=np.float64).T
    st = rt.Stack(L, d, H, dff, V, dtype="f32", residual_scale=wl.residual_scale, recur_block=S)
    st.set_weights(data["layers"], data["emb"])
    hid, logits = st.prefill(data["ids"])
    assert rel_err(hid, x) <= TOL["f32"] and rel_err(logits, logits_ref) <= TOL["f32"]


@pytest.mark.parametrize("alibi", [False, True])
def test_decode_over_a_long_cache_matches_oracle(alibi):
    # From 2048 cached positions on the decode step streams the cache with one lane per (sequence, head) and merges
    # the chunk partials in a second kernel; two steps after a prefill of 2200 positions against the oracle.
    from oracle import RTConfig, RTWeights, layer_seq
    from parity_metrics import check_tensor
    from paper_2604_21215_b200 import inputs, rt
    d, H, dff, B, N = 128, 2, 256, 3, 2200
    wl = inputs.Workload("longdec", 1, B, N + 2, d, H, dff, "bf16")
    data = inputs.make_inputs(wl, seed=77)
    lw = data["layers"][0]
    slopes = [2.0 ** (-8.0 * (h + 1) / H) for h in range(H)] if alibi else None
    ref = layer_seq(RTConfig(d, H, 64, dff, alibi_slopes=slopes), RTWeights(**lw), data["x"])
    lw_gpu = dict(lw, alibi_slopes=slopes) if alibi else lw
    layer = rt.Layer(d, H, dff, dtype="bf16")
    layer.set_weights(lw_gpu)
    layer.prefill(data["x"][:, :N], N_max=N + 2)
    for step in range(2):
        zn = layer.decode(data["x"][:, N + step], N + step)
        check_tensor(f"long-cache decode step {step}", "z", zn, ref[0][:, N + step], TOL["bf16"], curve=False)
    import torch
    k = layer.k_cache.permute(1, 0, 2).to(torch.float64).cpu().numpy()
    v = layer.v_cache.permute(1, 0, 2).to(torch.float64).cpu().numpy()
    check_tensor("long-cache decode", "k", k, ref[1], TOL["bf16"])
    check_tensor("long-cache decode", "v", v, ref[2], TOL["bf16"])
