"""B200-native hot path of speculative expand-verify-select search (arxiv 2609.39334): candidate-path
deduplication, tree attention over a shared-prefix paged KV pool, and top-k pruning, as a C-ABI CUDA library
(`libspecscale.so`, built from `csrc/`) with a thin ctypes binding (`binding`).

Importing the package does not load the CUDA library; `binding.lib()` does, and fails loudly if it is missing.
"""
__all__ = ["binding", "build", "pipeline", "synth"]
