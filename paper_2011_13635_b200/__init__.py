"""B200-native per-stage MSLT BERT training step behind a C-ABI CUDA library."""
