"""B200-native batched bandit step (prune, cluster, score/select) behind a C ABI.

`paper_2511_18868_b200.kb` is the thin ctypes binding of the CUDA library;
`paper_2511_18868_b200.workloads` draws the seeded synthetic inputs.
Importing the package does not load the CUDA library; the first call does and
fails loudly if it has not been built.
"""
__all__ = ["workloads"]
