"""The decode step for callers that cannot allocate (rt_layer_decode_step_static) must give
what the workspace-taking entry point gives.  Collected last on purpose: it is an add-on, and a
run that stops at the first failure should already have run everything else.

Who needs it: a host that receives only its input and output buffers (a framework plug-in), or
that sits in a section where cudaMalloc is not allowed, or whose memory is all spoken for, has
nowhere to get a workspace from; the library then brings its own fixed scratch array."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,tol", [("f32", 1e-6), ("bf16", 1e-6)])
def test_static_scratch_decode_matches_workspace_decode_twice_in_a_row(dtype, tol):
    import torch
    from paper_2604_21215_b200 import inputs, rt

    d, H, dff, B, N = 128, 2, 256, 3, 20
    wl = inputs.Workload("noalloc", 1, B, N + 2, d, H, dff, dtype)
    data = inputs.make_inputs(wl, seed=901)
    layer = rt.Layer(d, H, dff, dtype=dtype, leaf=16)
    layer.set_weights(data["layers"][0])
    layer.prefill(data["x"][:, :N], N_max=N + 2)              # fills rows [0, N) of the caches
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    k_ws, v_ws = layer.k_cache.clone(), layer.v_cache.clone()   # caches for the workspace variant
    k_st, v_st = layer.k_cache.clone(), layer.v_cache.clone()   # caches for the static-scratch variant
    stream = torch.cuda.current_stream().cuda_stream
    need = rt.rt_workspace_bytes(layer.cfg, B, 1, 1)
    assert 0 < need <= rt.RT_STATIC_SCRATCH_BYTES
    ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
    for step in range(2):                                       # two calls in a row share the built-in scratch
        pos = N + step
        x_new = torch.from_numpy(data["x"][:, pos]).to(tdt).cuda().contiguous()
        z_ws, z_st = torch.empty_like(x_new), torch.empty_like(x_new)
        st = rt.rt_layer_decode_step(layer.cfg, layer.w, x_new.data_ptr(), B, pos, z_ws.data_ptr(), k_ws.data_ptr(),
                                     v_ws.data_ptr(), N + 2, ws.data_ptr(), ws.numel(), stream)
        assert st == rt.RT_OK
        st = rt.rt_layer_decode_step_static(layer.cfg, layer.w, x_new.data_ptr(), B, pos, z_st.data_ptr(),
                                            k_st.data_ptr(), v_st.data_ptr(), N + 2, stream)
        assert st == rt.RT_OK
        torch.cuda.synchronize()
        assert rt.rt_get_status(ws.data_ptr()) == rt.RT_OK
        assert rt.rt_static_get_status() == rt.RT_OK           # the status word inside the built-in scratch
        ref = z_ws.double().cpu().numpy()
        got = z_st.double().cpu().numpy()
        assert np.isfinite(got).all()
        assert np.abs(got - ref).max() <= tol * max(1.0, np.abs(ref).max())
        for a, b in ((k_st, k_ws), (v_st, v_ws)):
            assert np.abs(a[pos].double().cpu().numpy() - b[pos].double().cpu().numpy()).max() <= tol * max(
                1.0, float(b[pos].abs().max()))


def test_static_scratch_calls_of_different_shapes_in_a_row():
    # The built-in scratch keeps the previous call's bytes, and another batch size or width moves every region
    # of its layout: whatever a call needs clean it must clear itself.  Three shapes, one after the other, each
    # against the workspace-taking entry point.
    import torch
    from paper_2604_21215_b200 import inputs, rt
    stream = torch.cuda.current_stream().cuda_stream
    for dtype, d, H, dff, B, N in (("bf16", 256, 4, 512, 5, 12), ("f32", 128, 2, 256, 2, 9), ("bf16", 128, 2, 256, 7, 17),
                                   ("bf16", 256, 4, 512, 5, 12)):
        wl = inputs.Workload("noalloc2", 1, B, N + 1, d, H, dff, dtype)
        data = inputs.make_inputs(wl, seed=903 + B)
        layer = rt.Layer(d, H, dff, dtype=dtype, leaf=16)
        layer.set_weights(data["layers"][0])
        layer.prefill(data["x"][:, :N], N_max=N + 1)
        tdt = torch.float32 if dtype == "f32" else torch.bfloat16
        k_ws, v_ws = layer.k_cache.clone(), layer.v_cache.clone()
        k_st, v_st = layer.k_cache.clone(), layer.v_cache.clone()
        need = rt.rt_workspace_bytes(layer.cfg, B, 1, 1)
        ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
        x_new = torch.from_numpy(data["x"][:, N]).to(tdt).cuda().contiguous()
        z_ws, z_st = torch.empty_like(x_new), torch.empty_like(x_new)
        assert rt.rt_layer_decode_step(layer.cfg, layer.w, x_new.data_ptr(), B, N, z_ws.data_ptr(), k_ws.data_ptr(),
                                       v_ws.data_ptr(), N + 1, ws.data_ptr(), ws.numel(), stream) == rt.RT_OK
        assert rt.rt_layer_decode_step_static(layer.cfg, layer.w, x_new.data_ptr(), B, N, z_st.data_ptr(), k_st.data_ptr(),
                                              v_st.data_ptr(), N + 1, stream) == rt.RT_OK
        torch.cuda.synchronize()
        assert rt.rt_get_status(ws.data_ptr()) == rt.RT_OK and rt.rt_static_get_status() == rt.RT_OK
        assert torch.equal(z_st, z_ws) and torch.equal(k_st[N], k_ws[N]) and torch.equal(v_st[N], v_ws[N])


def test_static_scratch_rejects_shapes_beyond_its_size():
    from paper_2604_21215_b200 import rt
    cfg = rt.make_config(4096, 64, 16384, dtype="f32")          # workspace for B = 64 is far above 8 MiB
    assert rt.rt_workspace_bytes(cfg, 64, 1, 1) > rt.RT_STATIC_SCRATCH_BYTES
    w = rt.RtLayerWeights()
    assert rt.rt_layer_decode_step_static(cfg, w, None, 64, 0, None, None, None, 1, None) == rt.RT_ERR_WORKSPACE
