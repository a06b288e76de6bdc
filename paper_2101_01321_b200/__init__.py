"""B200-native integer-only Transformer encoder layer (I-BERT): C-ABI library + thin binding."""
