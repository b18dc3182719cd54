"""B200-native Elastic Cache hot path: importance, anchor selection, bucket merge and
decode attention with fixed-point eviction, as CUDA kernels behind a C ABI."""
