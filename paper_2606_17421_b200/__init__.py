"""B200-native CKKS linear layer (ciphertext x encoded-plaintext weights) behind a C ABI.

`bifrost` is the ctypes binding of the CUDA library; `workloads` holds shapes and seeded inputs.
Importing the package does not load the CUDA library; `bifrost.load()` does, and fails loudly
when it has not been built.
"""
