"""B200-native Lethe hot path: decode-step attention over a pruned KV cache with the RASR relevance
recurrence fused in, and the periodic prune round (sparsity -> budgets -> protected top-k -> compaction).

The CUDA library is loaded on first use (`paper_2511_06029_b200.binding`); importing this package or its
`synth` module needs no GPU and no built extension.
"""
__all__ = ["synth", "binding"]
