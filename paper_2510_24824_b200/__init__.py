"""B200-native CLP decode-step attention of the Parallel Loop Transformer (C-ABI library + thin binding)."""
