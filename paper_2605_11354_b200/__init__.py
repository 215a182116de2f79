"""FP8 Sparse Linear Attention forward for B200 (sm_100a): thin binding over the C-ABI library."""
