"""B200-native HEART sparse-attention hot path (drift, mask prediction, block-sparse attention).

`inputs` (synthetic workloads) imports without a GPU; the CUDA library is loaded
on first use of `paper_2605_14513_b200.heart` and fails loudly if it is missing.
"""
