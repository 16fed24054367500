"""Binary (+-1 x +-1) convolution hot path for NVIDIA B200: C-ABI CUDA library + thin binding.

``binding`` marshals torch device buffers into the C ABI declared in include/bcnn.h,
``workloads`` holds the benchmark layer lists and operation counts, ``synth`` the seeded
synthetic inputs and bit-layout helpers, ``build`` compiles the library in-tree.
"""
