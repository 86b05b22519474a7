"""B200-native mixed-precision training hot path (FP16 GEMMs with FP32 accumulation,
loss-scaled softmax cross-entropy, FP32 master-weight update) behind a C ABI.

`inputs` holds the seeded synthetic input generators; `binding` is the ctypes
layer over the CUDA shared library (loaded lazily, it fails loudly if missing).
"""
