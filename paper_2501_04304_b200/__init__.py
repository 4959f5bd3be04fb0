"""B200-native hot path of DGQ (distribution-aware group quantization).

The product is the C-ABI library built from `csrc/` and declared in
`include/dgq.h`; `binding` is its thin ctypes wrapper and `synth` the seeded
input generator.  Importing this package does not load the library; the first
call into `binding` does, and fails loudly when the library has not been built.
"""
