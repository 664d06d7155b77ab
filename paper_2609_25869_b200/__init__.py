"""B200-native forward of dynamic block-sparse attention (C-ABI library + thin Python binding)."""
