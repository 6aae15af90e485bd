"""Thin binding over the C-ABI library (include/rt.h): argument marshalling only.

Importing this module loads `librt_b200.so` from the package directory and fails loudly
when it is missing or lacks a symbol -- there is no CPU fallback.  Module-level functions
carry the C names (`rt_layer_prefill`, ...) and take raw device pointers; `Layer` and
`Stack` are small conveniences that keep weights, caches and the workspace as torch tensors
(torch is used for device memory and streams only).
"""
from __future__ import annotations

import ctypes as C
import math
import os
from typing import Dict, List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librt_b200.so")

RT_OK, RT_ERR_INVALID_ARG, RT_ERR_UNSUPPORTED, RT_ERR_WORKSPACE, RT_ERR_CUDA, RT_ERR_TIMEOUT = range(6)
RT_F32, RT_BF16 = 0, 1
RT_SCHED_TILED, RT_SCHED_NAIVE = 0, 1
RT_NORM_PRE, RT_NORM_QK, RT_NORM_SKIP_Z = 1, 2, 8
RT_FLAG_BACKWARD_STEP_LAUNCHES = 1

EXPORTS = ("rt_workspace_bytes", "rt_layer_prefill", "rt_stack_prefill", "rt_decode_step",
           "rt_layer_decode_step", "rt_get_status", "rt_status_string", "rt_plan_counters", "rt_plan_tiles",
           "rt_profile_enable", "rt_profile_read", "rt_layer_decode_step_static", "rt_update_tile", "rt_selftest_wait_expiry",
           "rt_recompute_workspace_bytes", "rt_layer_recompute", "rt_backward_workspace_bytes", "rt_layer_backward",
           "rt_static_get_status")
RT_STATIC_SCRATCH_BYTES = 8 << 20


class RtConfig(C.Structure):
    _fields_ = [("d_model", C.c_int32), ("n_heads", C.c_int32), ("head_dim", C.c_int32), ("d_ff", C.c_int32),
                ("dtype", C.c_int32), ("sched", C.c_int32), ("leaf", C.c_int32), ("norm_flags", C.c_int32),
                ("rms_eps", C.c_float), ("softmax_scale", C.c_float), ("residual_scale", C.c_float),
                ("recur_block", C.c_int32), ("flags", C.c_int32)]


class RtLayerWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("w_q", "w_k", "w_v", "w_o", "w_up", "w_down",
                                           "g_attn", "g_mlp", "g_kv", "g_q", "g_k", "alibi_slopes")]


class RtLayerGrads(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("w_q", "w_k", "w_v", "w_o", "w_up", "w_down",
                                           "g_attn", "g_mlp", "g_kv", "g_q", "g_k")]


class RtCounters(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in ("model_bytes_read", "model_bytes_written", "flops_tile", "flops_leaf",
                                           "flops_gemm", "kv_bytes_read", "leaf_kv_bytes_l2", "n_tiles", "n_leaves")]


class RtProfile(C.Structure):
    _fields_ = [("ms", C.c_double * 4), ("launches", C.c_uint64 * 4)]


PROFILE_CLASSES = ("prepass", "leaf", "tile", "other")


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python __graft_entry__.py` (needs nvcc); "
                          "this package has no CPU fallback")
    lib = C.CDLL(LIB_PATH)
    for name in EXPORTS:
        if not hasattr(lib, name):
            raise ImportError(f"{LIB_PATH} does not export {name}")
    P, I, Z = C.c_void_p, C.c_int32, C.c_size_t
    lib.rt_workspace_bytes.restype = Z
    lib.rt_workspace_bytes.argtypes = [C.POINTER(RtConfig), I, I, I]
    lib.rt_layer_prefill.restype = C.c_int
    lib.rt_layer_prefill.argtypes = [C.POINTER(RtConfig), C.POINTER(RtLayerWeights), P, I, I, P, P, P, I, P, Z, P]
    lib.rt_layer_decode_step.restype = C.c_int
    lib.rt_layer_decode_step.argtypes = [C.POINTER(RtConfig), C.POINTER(RtLayerWeights), P, I, I, P, P, P, I, P, Z, P]
    lib.rt_layer_decode_step_static.restype = C.c_int
    lib.rt_layer_decode_step_static.argtypes = [C.POINTER(RtConfig), C.POINTER(RtLayerWeights), P, I, I, P, P, P, I, P]
    lib.rt_static_get_status.restype = C.c_int
    lib.rt_static_get_status.argtypes = []
    lib.rt_selftest_wait_expiry.restype = C.c_int
    lib.rt_selftest_wait_expiry.argtypes = [P, P]
    lib.rt_recompute_workspace_bytes.restype = Z
    lib.rt_recompute_workspace_bytes.argtypes = [C.POINTER(RtConfig), I, I]
    lib.rt_layer_recompute.restype = C.c_int
    lib.rt_backward_workspace_bytes.restype = Z
    lib.rt_backward_workspace_bytes.argtypes = [C.POINTER(RtConfig), I, I]
    lib.rt_layer_backward.restype = C.c_int
    lib.rt_layer_backward.argtypes = [C.POINTER(RtConfig), C.POINTER(RtLayerWeights), P, P, P, I, I, P, C.POINTER(RtLayerGrads), P, Z, P]
    lib.rt_layer_recompute.argtypes = [C.POINTER(RtConfig), C.POINTER(RtLayerWeights), P, P, I, I, P, P, P, I, P, Z, P]
    lib.rt_update_tile.restype = C.c_int
    lib.rt_update_tile.argtypes = [C.POINTER(RtConfig), P, P, P, P, P, P, I, I, I, I, I, I, I, P, P, P]
    lib.rt_stack_prefill.restype = C.c_int
    lib.rt_stack_prefill.argtypes = [C.POINTER(RtConfig), I, C.POINTER(RtLayerWeights), P, P, I, P, I, I, P, P,
                                     C.POINTER(P), C.POINTER(P), I, P, Z, P]
    lib.rt_decode_step.restype = C.c_int
    lib.rt_decode_step.argtypes = [C.POINTER(RtConfig), I, C.POINTER(RtLayerWeights), P, P, I, P, I, I, P,
                                   C.POINTER(P), C.POINTER(P), I, P, Z, P]
    lib.rt_get_status.restype = C.c_int
    lib.rt_get_status.argtypes = [P]
    lib.rt_status_string.restype = C.c_char_p
    lib.rt_status_string.argtypes = [C.c_int]
    lib.rt_plan_counters.restype = C.c_int
    lib.rt_plan_counters.argtypes = [C.POINTER(RtConfig), I, I, I, I, C.POINTER(RtCounters)]
    lib.rt_plan_tiles.restype = I
    lib.rt_plan_tiles.argtypes = [I, I, C.POINTER(I), I]
    lib.rt_profile_enable.restype = C.c_int
    lib.rt_profile_enable.argtypes = [I]
    lib.rt_profile_read.restype = C.c_int
    lib.rt_profile_read.argtypes = [C.POINTER(RtProfile)]
    return lib


_lib = _load()


class RtError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {rt_status_string(status)} (rt_status {status})")


def _check(status: int, where: str):
    if status != RT_OK:
        raise RtError(status, where)


# ------------------------------------------------------------------ the C names

def rt_status_string(status: int) -> str:
    return _lib.rt_status_string(int(status)).decode()


def rt_workspace_bytes(cfg: RtConfig, B: int, N: int, n_layers: int = 1) -> int:
    return int(_lib.rt_workspace_bytes(C.byref(cfg), B, N, n_layers))


def rt_layer_prefill(cfg, w, x, B, N, z, k_cache, v_cache, N_max, workspace, workspace_bytes, stream) -> int:
    return _lib.rt_layer_prefill(C.byref(cfg), C.byref(w), x, B, N, z, k_cache, v_cache, N_max, workspace,
                                 workspace_bytes, stream)


def rt_layer_decode_step(cfg, w, x, B, pos, z, k_cache, v_cache, N_max, workspace, workspace_bytes, stream) -> int:
    return _lib.rt_layer_decode_step(C.byref(cfg), C.byref(w), x, B, pos, z, k_cache, v_cache, N_max, workspace,
                                     workspace_bytes, stream)


def rt_layer_decode_step_static(cfg, w, x, B, pos, z, k_cache, v_cache, N_max, stream) -> int:
    """Decode step for callers that cannot allocate: no workspace argument, the scratch is a fixed
    array inside the library (see include/rt.h).  Calls on one device must not overlap."""
    return _lib.rt_layer_decode_step_static(C.byref(cfg), C.byref(w), x, B, pos, z, k_cache, v_cache, N_max, stream)


def rt_static_get_status() -> int:
    """Device status word of the last rt_layer_decode_step_static call on the current device (after a synchronise)."""
    return _lib.rt_static_get_status()


def rt_stack_prefill(cfg, n_layers, layers, emb, g_final, vocab, ids, B, N, hidden, logits_last, k_caches, v_caches,
                     N_max, workspace, workspace_bytes, stream) -> int:
    return _lib.rt_stack_prefill(C.byref(cfg), n_layers, layers, emb, g_final, vocab, ids, B, N, hidden, logits_last,
                                 k_caches, v_caches, N_max, workspace, workspace_bytes, stream)


def rt_decode_step(cfg, n_layers, layers, emb, g_final, vocab, ids, B, pos, logits, k_caches, v_caches, N_max,
                   workspace, workspace_bytes, stream) -> int:
    return _lib.rt_decode_step(C.byref(cfg), n_layers, layers, emb, g_final, vocab, ids, B, pos, logits, k_caches,
                               v_caches, N_max, workspace, workspace_bytes, stream)


def rt_update_tile(cfg, q, k_cache, v_cache, st_o, st_m, st_l, B, rows_q, rows_kv, q0, q1, k0, k1, alibi_slopes,
                   workspace, stream) -> int:
    return _lib.rt_update_tile(C.byref(cfg), q, k_cache, v_cache, st_o, st_m, st_l, B, rows_q, rows_kv, q0, q1, k0, k1,
                               alibi_slopes, workspace, stream)


def rt_recompute_workspace_bytes(cfg: RtConfig, B: int, N: int) -> int:
    return int(_lib.rt_recompute_workspace_bytes(C.byref(cfg), B, N))


def rt_backward_workspace_bytes(cfg: RtConfig, B: int, N: int) -> int:
    return int(_lib.rt_backward_workspace_bytes(C.byref(cfg), B, N))


def rt_layer_backward(cfg, w, x, z, dz, B, N, dx, grads, workspace, workspace_bytes, stream) -> int:
    return _lib.rt_layer_backward(C.byref(cfg), C.byref(w), x, z, dz, B, N, dx, C.byref(grads), workspace, workspace_bytes, stream)


def rt_layer_recompute(cfg, w, x, z_claim, B, N, z_out, k_cache, v_cache, N_max, workspace, workspace_bytes, stream) -> int:
    return _lib.rt_layer_recompute(C.byref(cfg), C.byref(w), x, z_claim, B, N, z_out, k_cache, v_cache, N_max, workspace,
                                   workspace_bytes, stream)


def rt_selftest_wait_expiry(workspace, stream) -> int:
    return _lib.rt_selftest_wait_expiry(workspace, stream)


def rt_get_status(workspace) -> int:
    return _lib.rt_get_status(workspace)


def rt_plan_counters(cfg: RtConfig, B: int, N: int, n_layers: int = 1, vocab: int = 0) -> Dict[str, int]:
    out = RtCounters()
    _check(_lib.rt_plan_counters(C.byref(cfg), B, N, n_layers, vocab, C.byref(out)), "rt_plan_counters")
    return {n: int(getattr(out, n)) for n, _ in RtCounters._fields_}


def rt_plan_tiles(N: int, leaf: int) -> List[tuple]:
    n = _lib.rt_plan_tiles(N, leaf, None, 0)
    buf = (C.c_int32 * (4 * max(n, 1)))()
    _lib.rt_plan_tiles(N, leaf, buf, n)
    return [tuple(buf[4 * i:4 * i + 4]) for i in range(n)]


def rt_profile_enable(on) -> None:
    """False/0: off; True/1: event spans per kernel class; 2: also the leaf kernels' in-kernel phase timers."""
    _check(_lib.rt_profile_enable(int(on)), "rt_profile_enable")


def rt_profile_read() -> Dict[str, Dict[str, float]]:
    out = RtProfile()
    _check(_lib.rt_profile_read(C.byref(out)), "rt_profile_read")
    return {n: {"ms": float(out.ms[i]), "launches": int(out.launches[i])} for i, n in enumerate(PROFILE_CLASSES)}


def make_config(d_model: int, n_heads: int, d_ff: int, dtype: str = "bf16", sched: str = "tiled", leaf: int = 0,
                norm_flags: int = RT_NORM_PRE | RT_NORM_QK, rms_eps: float = 1e-6,
                softmax_scale: Optional[float] = None, residual_scale: float = 1.0, head_dim: int = 64,
                recur_block: int = 0, flags: int = 0) -> RtConfig:
    return RtConfig(d_model, n_heads, head_dim, d_ff, {"f32": RT_F32, "bf16": RT_BF16}[dtype],
                    {"tiled": RT_SCHED_TILED, "naive": RT_SCHED_NAIVE}[sched], leaf, norm_flags, rms_eps,
                    (1.0 / math.sqrt(head_dim)) if softmax_scale is None else softmax_scale, residual_scale, recur_block, flags)


# ------------------------------------------------------------------ conveniences on torch tensors

def _torch():
    import torch
    return torch


def _tdtype(dtype: str):
    torch = _torch()
    return {"f32": torch.float32, "bf16": torch.bfloat16}[dtype]


def _to_dev(a, dtype: str, device):
    torch = _torch()
    if isinstance(a, np.ndarray):
        a = torch.from_numpy(np.ascontiguousarray(a))
    return a.to(device=device, dtype=_tdtype(dtype)).contiguous()


_W_NAMES = ("w_q", "w_k", "w_v", "w_o", "w_up", "w_down")
_G_NAMES = ("g_attn", "g_mlp", "g_kv", "g_q", "g_k")


def _pack_weights(wd: dict, dtype: str, device):
    """dict of arrays -> (RtLayerWeights, list of tensors kept alive)"""
    keep, st = [], RtLayerWeights()
    for n in _W_NAMES:
        t = _to_dev(wd[n], dtype, device)
        keep.append(t)
        setattr(st, n, t.data_ptr())
    for n in _G_NAMES:
        if wd.get(n) is not None:
            t = _to_dev(wd[n], dtype, device)
            keep.append(t)
            setattr(st, n, t.data_ptr())
    if wd.get("alibi_slopes") is not None:           # [n_heads], always fp32
        t = _to_dev(np.asarray(wd["alibi_slopes"], dtype=np.float64), "f32", device)
        keep.append(t)
        st.alibi_slopes = t.data_ptr()
    return st, keep


class Layer:
    """One RT layer with its weights, K/V cache and workspace resident on the device."""

    def __init__(self, d_model: int, n_heads: int, d_ff: int, dtype: str = "bf16", device: str = "cuda:0", **cfg_kw):
        torch = _torch()
        self.dtype, self.device = dtype, torch.device(device)
        self.cfg = make_config(d_model, n_heads, d_ff, dtype=dtype, **cfg_kw)
        self.w: Optional[RtLayerWeights] = None
        self._keep: list = []
        self.k_cache = self.v_cache = self.ws = None
        self.N_max = 0

    def set_weights(self, wd: dict):
        self.w, self._keep = _pack_weights(wd, self.dtype, self.device)

    def reserve(self, B: int, N: int, N_max: Optional[int] = None):
        torch = _torch()
        N_max = N if N_max is None else N_max
        d = self.cfg.d_model
        if self.k_cache is None or tuple(self.k_cache.shape) != (N_max, B, d):
            self.k_cache = torch.zeros((N_max, B, d), dtype=_tdtype(self.dtype), device=self.device)
            self.v_cache = torch.zeros_like(self.k_cache)
            self.N_max = N_max
        need = rt_workspace_bytes(self.cfg, B, N, 1)
        if need == 0:
            raise RtError(RT_ERR_INVALID_ARG, "rt_workspace_bytes")
        if self.ws is None or self.ws.numel() < need:
            self.ws = torch.zeros(need, dtype=torch.uint8, device=self.device)

    def prefill_device(self, x_dev, z_dev, stream=None) -> None:
        """x_dev, z_dev: contiguous [B, N, d] device tensors of the storage type (enqueue only)."""
        torch = _torch()
        B, N, _ = x_dev.shape
        s = torch.cuda.current_stream(self.device).cuda_stream if stream is None else stream
        _check(rt_layer_prefill(self.cfg, self.w, x_dev.data_ptr(), B, N, z_dev.data_ptr(), self.k_cache.data_ptr(),
                                self.v_cache.data_ptr(), self.N_max, self.ws.data_ptr(), self.ws.numel(), s),
               "rt_layer_prefill")

    def status(self) -> int:
        return rt_get_status(self.ws.data_ptr())

    def prefill(self, x, N_max: Optional[int] = None):
        """x [B,N,d] (numpy or tensor) -> z, k, v as fp64 numpy arrays, each [B,N,d]."""
        torch = _torch()
        xd = _to_dev(x, self.dtype, self.device)
        B, N, _ = xd.shape
        self.reserve(B, N, N_max)
        zd = torch.empty_like(xd)
        self.prefill_device(xd, zd)
        torch.cuda.synchronize(self.device)
        _check(self.status(), "rt_layer_prefill (device)")
        to_np = lambda t: t.to(torch.float64).cpu().numpy()
        return (to_np(zd), to_np(self.k_cache[:N].permute(1, 0, 2)), to_np(self.v_cache[:N].permute(1, 0, 2)))

    def recompute(self, x, z_claim):
        """One parallel sweep: x, z_claim [B,N,d] -> z', k, v (fp64 numpy, each [B,N,d]); the caches are rebuilt from z_claim."""
        torch = _torch()
        xd = _to_dev(x, self.dtype, self.device)
        zc = _to_dev(z_claim, self.dtype, self.device)
        B, N, _ = xd.shape
        self.reserve(B, N)
        need = rt_recompute_workspace_bytes(self.cfg, B, N)
        if self.ws.numel() < need:
            self.ws = torch.zeros(need, dtype=torch.uint8, device=self.device)
        zo = torch.empty_like(xd)
        s = torch.cuda.current_stream(self.device).cuda_stream
        _check(rt_layer_recompute(self.cfg, self.w, xd.data_ptr(), zc.data_ptr(), B, N, zo.data_ptr(), self.k_cache.data_ptr(),
                                  self.v_cache.data_ptr(), self.N_max, self.ws.data_ptr(), self.ws.numel(), s), "rt_layer_recompute")
        torch.cuda.synchronize(self.device)
        _check(self.status(), "rt_layer_recompute (device)")
        to_np = lambda t: t.to(torch.float64).cpu().numpy()
        return (to_np(zo), to_np(self.k_cache[:N].permute(1, 0, 2)), to_np(self.v_cache[:N].permute(1, 0, 2)))

    def backward_device(self, x_dev, z_dev, dz_dev, dx_dev, grads: "RtLayerGrads", ws, stream=None) -> None:
        """x_dev, z_dev [B,N,d] storage type, dz_dev, dx_dev [B,N,d] fp32, ws a uint8 workspace tensor (enqueue only)."""
        torch = _torch()
        B, N, _ = x_dev.shape
        s = torch.cuda.current_stream(self.device).cuda_stream if stream is None else stream
        _check(rt_layer_backward(self.cfg, self.w, x_dev.data_ptr(), z_dev.data_ptr(), dz_dev.data_ptr(), B, N, dx_dev.data_ptr(),
                                 grads, ws.data_ptr(), ws.numel(), s), "rt_layer_backward")

    def backward(self, x, z, dz):
        """x, z [B,N,d] (z = this layer's outputs), dz = dL/dz [B,N,d] -> dx [B,N,d] and a dict of parameter gradients
        (fp64 numpy; one entry per parameter the layer has)."""
        torch = _torch()
        xd = _to_dev(x, self.dtype, self.device)
        zd = _to_dev(z, self.dtype, self.device)
        dzd = _to_dev(dz, "f32", self.device)
        B, N, d = xd.shape
        need = rt_backward_workspace_bytes(self.cfg, B, N)
        if need == 0:
            raise RtError(RT_ERR_INVALID_ARG, "rt_backward_workspace_bytes")
        ws = torch.zeros(need, dtype=torch.uint8, device=self.device)
        dxd = torch.empty((B, N, d), dtype=torch.float32, device=self.device)
        grads, out = RtLayerGrads(), {}
        shapes = {"w_up": (self.cfg.d_ff, d), "w_down": (d, self.cfg.d_ff)}
        for n in _W_NAMES + _G_NAMES:
            if n in _G_NAMES and not getattr(self.w, n):
                continue
            out[n] = torch.empty(shapes.get(n, (d, d) if n in _W_NAMES else (d,)), dtype=torch.float32, device=self.device)
            setattr(grads, n, out[n].data_ptr())
        self.backward_device(xd, zd, dzd, dxd, grads, ws)
        torch.cuda.synchronize(self.device)
        _check(rt_get_status(ws.data_ptr()), "rt_layer_backward (device)")
        to_np = lambda t: t.to(torch.float64).cpu().numpy()
        return to_np(dxd), {n: to_np(t) for n, t in out.items()}

    def decode(self, x_new, pos: int):
        """x_new [B,d] at position pos (caches must hold pos rows) -> z_new [B,d] fp64 numpy."""
        torch = _torch()
        xd = _to_dev(x_new, self.dtype, self.device)
        B, _ = xd.shape
        zd = torch.empty_like(xd)
        need = rt_workspace_bytes(self.cfg, B, 1, 1)
        if self.ws is None or self.ws.numel() < need:
            self.ws = torch.zeros(need, dtype=torch.uint8, device=self.device)
        s = torch.cuda.current_stream(self.device).cuda_stream
        _check(rt_layer_decode_step(self.cfg, self.w, xd.data_ptr(), B, pos, zd.data_ptr(), self.k_cache.data_ptr(),
                                    self.v_cache.data_ptr(), self.N_max, self.ws.data_ptr(), self.ws.numel(), s),
               "rt_layer_decode_step")
        torch.cuda.synchronize(self.device)
        _check(self.status(), "rt_layer_decode_step (device)")
        return zd.to(torch.float64).cpu().numpy()


class Stack:
    """n_layers RT layers with token embedding and tied head."""

    def __init__(self, n_layers: int, d_model: int, n_heads: int, d_ff: int, vocab: int, dtype: str = "bf16",
                 device: str = "cuda:0", **cfg_kw):
        torch = _torch()
        self.dtype, self.device = dtype, torch.device(device)
        self.n_layers, self.vocab = n_layers, vocab
        self.cfg = make_config(d_model, n_heads, d_ff, dtype=dtype, **cfg_kw)
        self._keep: list = []
        self.layers = (RtLayerWeights * n_layers)()
        self.emb = self.g_final = None
        self.k_caches: List = []
        self.v_caches: List = []
        self.ws = None
        self.N_max = 0

    def set_weights(self, layer_dicts: Sequence[dict], emb, g_final=None):
        assert len(layer_dicts) == self.n_layers
        for i, wd in enumerate(layer_dicts):
            st, keep = _pack_weights(wd, self.dtype, self.device)
            self.layers[i] = st
            self._keep += keep
        self.emb = _to_dev(emb, self.dtype, self.device)
        self.g_final = None if g_final is None else _to_dev(g_final, self.dtype, self.device)

    def reserve(self, B: int, N: int, N_max: Optional[int] = None):
        torch = _torch()
        N_max = N if N_max is None else N_max
        d = self.cfg.d_model
        if not self.k_caches or tuple(self.k_caches[0].shape) != (N_max, B, d):
            self.k_caches = [torch.zeros((N_max, B, d), dtype=_tdtype(self.dtype), device=self.device)
                             for _ in range(self.n_layers)]
            self.v_caches = [torch.zeros_like(t) for t in self.k_caches]
            self.N_max = N_max
            self._kp = (C.c_void_p * self.n_layers)(*[t.data_ptr() for t in self.k_caches])
            self._vp = (C.c_void_p * self.n_layers)(*[t.data_ptr() for t in self.v_caches])
        need = rt_workspace_bytes(self.cfg, B, N, self.n_layers)
        if self.ws is None or self.ws.numel() < need:
            self.ws = torch.zeros(need, dtype=torch.uint8, device=self.device)

    def prefill_device(self, ids_dev, hidden_dev, logits_dev, stream=None) -> None:
        torch = _torch()
        B, N = ids_dev.shape
        s = torch.cuda.current_stream(self.device).cuda_stream if stream is None else stream
        _check(rt_stack_prefill(self.cfg, self.n_layers, self.layers, self.emb.data_ptr(),
                                None if self.g_final is None else self.g_final.data_ptr(), self.vocab,
                                ids_dev.data_ptr(), B, N,
                                None if hidden_dev is None else hidden_dev.data_ptr(),
                                None if logits_dev is None else logits_dev.data_ptr(),
                                self._kp, self._vp, self.N_max, self.ws.data_ptr(), self.ws.numel(), s),
               "rt_stack_prefill")

    def status(self) -> int:
        return rt_get_status(self.ws.data_ptr())

    def prefill(self, ids, N_max: Optional[int] = None):
        """ids [B,N] int -> hidden [B,N,d], logits_last [B,V] (fp64 numpy)."""
        torch = _torch()
        idd = torch.as_tensor(np.asarray(ids), dtype=torch.int32, device=self.device).contiguous()
        B, N = idd.shape
        self.reserve(B, N, N_max)
        hid = torch.empty((B, N, self.cfg.d_model), dtype=_tdtype(self.dtype), device=self.device)
        logits = torch.empty((B, self.vocab), dtype=torch.float32, device=self.device)
        self.prefill_device(idd, hid, logits)
        torch.cuda.synchronize(self.device)
        _check(self.status(), "rt_stack_prefill (device)")
        return hid.to(torch.float64).cpu().numpy(), logits.to(torch.float64).cpu().numpy()

    def decode(self, ids_new, pos: int):
        torch = _torch()
        idd = torch.as_tensor(np.asarray(ids_new), dtype=torch.int32, device=self.device).contiguous()
        B = idd.shape[0]
        logits = torch.empty((B, self.vocab), dtype=torch.float32, device=self.device)
        need = rt_workspace_bytes(self.cfg, B, 1, self.n_layers)
        if self.ws is None or self.ws.numel() < need:
            self.ws = torch.zeros(need, dtype=torch.uint8, device=self.device)
        s = torch.cuda.current_stream(self.device).cuda_stream
        _check(rt_decode_step(self.cfg, self.n_layers, self.layers, self.emb.data_ptr(),
                              None if self.g_final is None else self.g_final.data_ptr(), self.vocab,
                              idd.data_ptr(), B, pos, logits.data_ptr(), self._kp, self._vp, self.N_max,
                              self.ws.data_ptr(), self.ws.numel(), s), "rt_decode_step")
        torch.cuda.synchronize(self.device)
        _check(self.status(), "rt_decode_step (device)")
        return logits.to(torch.float64).cpu().numpy()

    def caches_numpy(self, N: int):
        torch = _torch()
        f = lambda t: t[:N].permute(1, 0, 2).to(torch.float64).cpu().numpy()
        return [(f(k), f(v)) for k, v in zip(self.k_caches, self.v_caches)]
