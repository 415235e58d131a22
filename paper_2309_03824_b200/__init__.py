"""B200-native training step of low-rank decomposed layers (C-ABI CUDA library + thin binding)."""
