"""B200-native SlimSpec draft LM-head (low-rank head + fused log-softmax / top-k)."""
