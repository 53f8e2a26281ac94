"""B200-native CSD verification path (C-ABI library + Python binding)."""
