"""FAEDKV / IWDFT hot path for one NVIDIA B200: CUDA kernels behind a C ABI, plus this thin binding.

    from paper_2507_20030_b200 import binding
    ctx = binding.Context(n_layers=32, n_kv_heads=8, n_q_heads=32, n_dft=32768, max_batch=1)

Importing the package does not load the CUDA library; the first call does, and
fails loudly if it has not been built.
"""
__all__ = ["binding", "synth", "build"]
