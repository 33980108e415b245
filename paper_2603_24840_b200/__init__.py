"""B200-native prune-and-rebatch path of online rollout pruning (quality-head scoring, per-group
balancing selection, survivor compaction with group advantages, fused lm_head log-prob).

The compute lives in the CUDA C-ABI library under ``csrc/``; ``binding`` marshals arguments to it.
Nothing is loaded at import time; the first call into ``binding`` loads the library and fails
loudly if it has not been built.
"""
__all__ = ["synth", "binding"]
