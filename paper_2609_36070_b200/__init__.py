"""B200-native fused MoE layer forward (router, top-k, dispatch schedule, grouped SwiGLU experts, combine).

`paper_2609_36070_b200.mok` is the thin binding over the C-ABI library (it fails loudly when the CUDA
library is not built); `paper_2609_36070_b200.inputs` holds the seeded synthetic workloads.
"""
__version__ = "0.1.0"
