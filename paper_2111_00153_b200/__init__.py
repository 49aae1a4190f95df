"""B200-native RMSMP layer: row-wise mixed-scheme (PoT-4 / Fixed-4 / Fixed-8) weights times
4-bit fixed-point activations, as hand-written CUDA for sm_100a behind a C ABI."""
