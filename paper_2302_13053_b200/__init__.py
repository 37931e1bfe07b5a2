"""B200-native hot path of lazy message passing (Retexo): CSR neighbour
aggregation, per-node MLP training and embedding, cross-partition message
count, and the K-round loop, as a C-ABI CUDA library with a ctypes binding.

`workloads` (numpy only) draws the seeded synthetic inputs; `binding` wraps
libretexo.so and needs torch + a CUDA device; `build` compiles the library.
Nothing is imported eagerly so that the input generators can be used without
torch or the built library.
"""
__all__ = ["workloads", "binding", "build"]
