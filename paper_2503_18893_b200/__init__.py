"""xKV selective reconstruction for B200 (sm_100a): C-ABI CUDA library plus a thin Python binding.

`paper_2503_18893_b200.xkv` is the binding (it loads the CUDA library and fails loudly if
that library has not been built); `paper_2503_18893_b200.synth` draws seeded synthetic
inputs and needs no GPU.
"""
__all__ = ["synth", "xkv", "build", "workload"]
