"""Host-side checks that need no GPU: the library loads, exports what include/rt.h declares,
rejects bad arguments before touching the device, and its schedule enumerator agrees with
Algorithm 1 as written out by the oracle."""
import ctypes as C
import os
import re

import pytest

from oracle import alg1_tiles
from paper_2604_21215_b200 import rt

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "rt.h")).read()
    declared = set(re.findall(r"\b(rt_[a-z_]+)\s*\(", header))
    assert declared, "no declarations found"
    lib = C.CDLL(rt.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(rt.EXPORTS)


def test_status_strings():
    assert rt.rt_status_string(rt.RT_OK) == "ok"
    assert "timed out" in rt.rt_status_string(rt.RT_ERR_TIMEOUT)


@pytest.mark.parametrize("leaf", [1, 2, 16, 64])
def test_plan_tiles_is_algorithm_1_at_block_granularity(leaf):
    for N in (1, 2, 7, 8, 64, 65, 100, 256, 1000):
        want = [(u - 1, v, s - 1, e) for (t, u, v, s, e) in alg1_tiles(N, leaf)]   # 1-based inclusive -> 0-based half-open
        assert rt.rt_plan_tiles(N, leaf) == want, (N, leaf)


def test_worked_examples_from_the_paper_through_the_library():
    tiles = {k1: (q0, q1, k0) for (q0, q1, k0, k1) in rt.rt_plan_tiles(8, 1)}
    assert tiles[4] == (4, 8, 0)      # after position 4: pairs 1..4 -> queries 5..8
    assert tiles[6] == (6, 8, 4)      # after position 6: pairs 5..6 -> queries 7..8


def test_invalid_arguments_are_rejected_on_the_host():
    cfg = rt.make_config(128, 2, 512, dtype="f32")
    w = rt.RtLayerWeights()
    # null pointers everywhere: must return before any CUDA call
    assert rt.rt_layer_prefill(cfg, w, None, 1, 16, None, None, None, 16, None, 0, None) == rt.RT_ERR_INVALID_ARG
    bad = rt.make_config(128, 3, 512, dtype="f32")           # heads * head_dim != d_model
    assert rt.rt_workspace_bytes(bad, 1, 16) == 0
    assert rt.rt_workspace_bytes(cfg, 0, 16) == 0
    cfg32 = rt.make_config(128, 4, 512, dtype="f32", head_dim=32)
    buf = (C.c_char * 4096)()
    addr = (C.addressof(buf) + 255) & ~255
    assert rt.rt_layer_prefill(cfg32, w, addr, 1, 16, addr, addr, addr, 16, addr, 1 << 40, None) == rt.RT_ERR_UNSUPPORTED
    need = rt.rt_workspace_bytes(cfg, 1, 16)
    assert need > 0
    assert rt.rt_layer_prefill(cfg, w, addr, 1, 16, addr, addr, addr, 16, addr, need - 1, None) == rt.RT_ERR_WORKSPACE
    leafbad = rt.make_config(128, 2, 512, dtype="f32", leaf=48)
    assert rt.rt_workspace_bytes(leafbad, 1, 16) == 0


def test_backward_host_checks_need_no_gpu():
    # workspace size and argument checks of the backward pass run on the host, before any CUDA call
    cfg = rt.make_config(128, 2, 512, dtype="f32")
    need = rt.rt_backward_workspace_bytes(cfg, 2, 64)
    assert need > 0 and rt.rt_backward_workspace_bytes(cfg, 4, 64) > need
    assert rt.rt_backward_workspace_bytes(rt.make_config(128, 3, 512, dtype="f32"), 2, 64) == 0
    assert rt.rt_backward_workspace_bytes(cfg, 0, 64) == 0
    w, gr = rt.RtLayerWeights(), rt.RtLayerGrads()
    assert rt.rt_layer_backward(cfg, w, None, None, None, 2, 64, None, gr, None, 0, None) == rt.RT_ERR_INVALID_ARG
    buf = (C.c_char * 4096)()
    addr = (C.addressof(buf) + 255) & ~255
    for n in ("w_q", "w_k", "w_v", "w_o", "w_up", "w_down"):
        setattr(w, n, addr)
    call = lambda c, nbytes, g=gr: rt.rt_layer_backward(c, w, addr, addr, addr, 2, 64, addr, g, addr, nbytes, None)
    assert call(cfg, need - 1) == rt.RT_ERR_WORKSPACE
    assert call(rt.make_config(128, 2, 512, dtype="f32", recur_block=8), need) == rt.RT_ERR_UNSUPPORTED
    assert call(rt.make_config(128, 4, 512, dtype="f32", head_dim=32), need) == rt.RT_ERR_UNSUPPORTED
    odd = rt.RtLayerGrads()
    odd.w_q = addr + 4                                        # gradient arrays must be 16-byte aligned
    assert call(cfg, need, odd) == rt.RT_ERR_INVALID_ARG


def test_plan_counters_follow_the_n_log_n_model():
    # K/V rows streamed by the cross tiles: one half of the rows per level above the leaf.
    cfg = rt.make_config(1024, 16, 4096, dtype="bf16", leaf=64)
    B, d, e = 1, 1024, 2
    for N in (1024, 4096, 32768):
        c = rt.rt_plan_counters(cfg, B, N)
        levels = (N // 64).bit_length() - 1
        assert c["kv_bytes_read"] == levels * (N // 2) * 2 * B * d * e
        assert c["n_leaves"] == N // 64 and c["n_tiles"] == N // 64 - 1
        assert c["flops_tile"] == sum(4 * (q1 - q0) * (k1 - k0) * d * B for (q0, q1, k0, k1) in rt.rt_plan_tiles(N, 64))
    naive = rt.make_config(1024, 16, 4096, dtype="bf16", sched="naive")
    c = rt.rt_plan_counters(naive, B, 4096)
    assert c["kv_bytes_read"] == B * d * e * 4096 * 4095


def test_plan_counters_model_the_schedule_that_runs():
    # The counters follow the chain form a shape takes: wide batches use leaves of 16 positions, the tensor-core
    # leaf kernel keeps 64-position leaves also when an SM owns two (sequence, head) pairs, blocked recurrence tiles by blocks.
    N = 2048
    wide = rt.rt_plan_counters(rt.make_config(1024, 16, 4096, dtype="bf16"), 96, N)
    assert wide["n_leaves"] == N // 16 and wide["n_tiles"] == len(rt.rt_plan_tiles(N, 16))
    # 17 .. 48 sequences run as slices of at most 16 through the tensor-core leaf kernel: its leaves, and the chain
    # weights staged once per slice and leaf
    split = rt.rt_plan_counters(rt.make_config(1024, 16, 4096, dtype="bf16"), 32, N)
    assert split["n_leaves"] == N // 64 and split["n_tiles"] == len(rt.rt_plan_tiles(N, 64))
    one = rt.rt_plan_counters(rt.make_config(1024, 16, 4096, dtype="bf16"), 16, N)
    chain_w = (3 * 1024 * 1024 + 2 * 1024 * 4096) * 2
    assert split["model_bytes_read"] - 2 * one["model_bytes_read"] == -(3 * 1024 * 1024 * 2)    # the pre-pass weights once, not twice
    assert one["model_bytes_read"] > (N // 64) * chain_w
    c3 = rt.rt_plan_counters(rt.make_config(1024, 16, 4096, dtype="bf16"), 8, N)
    assert c3["n_leaves"] == N // 64 and c3["n_tiles"] == len(rt.rt_plan_tiles(N, 64))
    c4 = rt.rt_plan_counters(rt.make_config(1024, 16, 4096, dtype="bf16"), 16, N)
    assert c4["n_leaves"] == N // 64 and c4["n_tiles"] == len(rt.rt_plan_tiles(N, 64))
    blk = rt.rt_plan_counters(rt.make_config(1024, 16, 4096, dtype="bf16", recur_block=128), 8, N)
    assert blk["n_leaves"] == N // 128 and blk["n_tiles"] == N // 128 - 1
    f32 = rt.rt_plan_counters(rt.make_config(128, 2, 512, dtype="f32"), 4, 256)
    assert f32["n_leaves"] == 4 and f32["n_tiles"] == 3


def test_unknown_flags_are_invalid_configurations():
    assert rt.rt_workspace_bytes(rt.make_config(128, 2, 512, dtype="f32", norm_flags=4 | 3), 1, 16) == 0
    assert rt.rt_workspace_bytes(rt.make_config(128, 2, 512, dtype="f32", flags=2), 1, 16) == 0
    assert rt.rt_workspace_bytes(rt.make_config(128, 2, 512, dtype="f32", flags=rt.RT_FLAG_BACKWARD_STEP_LAUNCHES), 1, 16) > 0
