"""B200-native fused exact attention (the FLAT paper's Logit-Softmax-Attend hot path).

`paper_2107_06419_b200.api` is the binding to the CUDA library (it raises if the
library is missing: there is no CPU fallback); `paper_2107_06419_b200.inputs` is
the seeded synthetic-input generator (numpy only).  Nothing is imported eagerly.
"""
__all__ = ["api", "inputs", "build"]
