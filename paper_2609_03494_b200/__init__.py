"""B200-native GrowPage decode path: paged GQA decode attention fused with the dual EMA
query summaries, boundary scoring, working-set estimation, grow-or-compress and in-place
page compaction, behind a C-ABI library.

Importing the package loads nothing; `paper_2609_03494_b200.binding` loads the CUDA library
and raises if it has not been built.
"""
__all__ = ["binding", "workload", "shard"]
