"""B200-native token-level PPO math for RLHF: log-prob gather, KL reward, GAE, fused PPO loss.

`paper_2410_15651_b200.binding` is the thin ctypes layer over the C-ABI CUDA library
(`librlhf_ppo.so`, built in-tree by `paper_2410_15651_b200.build`); `inputs` draws the seeded
synthetic workloads.  Importing the package loads nothing; the library is loaded on first use
and the call fails loudly if it has not been built.
"""
__all__ = ["binding", "inputs", "build", "parallel", "memory"]
