"""ASL prefill hot path for B200 (sm_100a): observation-window scoring, pooling,
rank statistic, per-head top-k and K/V compaction behind a C-ABI library.

Importing the package loads nothing; ``paper_2601_07667_b200.binding`` loads the
CUDA library and fails loudly when it is missing."""
