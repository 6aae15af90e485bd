"""B200-native exact prefill of the Recurrent Transformer layer.

`inputs` draws the seeded synthetic workloads; `rt` is the thin binding over the C-ABI
library (importing it loads the CUDA library and fails loudly when it is missing).
"""
__all__ = ["inputs", "replicas", "rt"]
