"""B200-native EGTP / PLP length-predictor hot path (sm_100a kernels behind a C ABI)."""
