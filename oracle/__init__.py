"""fp64 CPU oracle for the Recurrent Transformer layer.

TEST INFRASTRUCTURE ONLY.  Nothing in the product package imports this; only the
tests, the smoke check and the CPU-baseline / reference legs of the benchmark do.
It shares no code with the CUDA path.
"""
from .rt_oracle import (  # noqa: F401
    RTConfig, RTWeights, rms, qk_rms, gelu, attn,
    layer_seq, layer_blk, layer_fixed_point, layer_decode, layer_blockrec,
    stack_prefill, stack_decode, alg1_tiles, update_tile,
)
from .rt_oracle_grad import layer_grad, layer_seq_torch  # noqa: F401,E402
