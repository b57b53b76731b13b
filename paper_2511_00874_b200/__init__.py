"""B200-native stochastically-rounded quantized linear layer (C-ABI library + thin binding)."""
