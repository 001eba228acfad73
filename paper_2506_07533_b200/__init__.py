"""B200-native MoQAE inference hot path: chunk router, quantise-and-pack,
mixed-precision decode attention.  The compute lives in a C-ABI CUDA library
(`libmoqae.so`, built in-tree); this package only marshals arguments."""
