"""Double quantization (AsyLPG / Sparse-AsyLPG / Acc-AsyLPG) hot path for NVIDIA B200."""
