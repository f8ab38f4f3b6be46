"""B200-native encrypted nearest-neighbour scoring (RNS-CKKS, ciphertext x plaintext).

`paper_2608_21131_b200.binding` is the thin ctypes layer over the C-ABI CUDA library
(`include/hann.h`); `paper_2608_21131_b200.synth` holds the seeded synthetic inputs.
Importing the package does not load the CUDA library; creating a `binding.Context` does,
and fails loudly when the library has not been built.
"""
