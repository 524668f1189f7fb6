"""B200-native cross-vocabulary speculative verification (OmniDraft, arXiv 2507.02659).

`paper_2507_02659_b200.binding` is the thin ctypes layer over the C-ABI CUDA
library (libomnidraft.so); `paper_2507_02659_b200.synth` makes seeded synthetic
inputs.  Nothing here computes on the CPU: without the built CUDA library the
binding raises.
"""
__all__ = ["binding", "synth", "shard"]
