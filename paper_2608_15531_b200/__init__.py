"""B200-native fused outlier-aware W4A16 decode matmul (C-ABI library + thin binding)."""
