"""B200-native paged-attention decode and KV-block swap (C-ABI library + thin binding)."""
