"""MixAttention inference attention for B200: CUDA kernels behind a C ABI.

`binding` loads libmixattn.so (built by `build.build()`) and mirrors
include/mixattn.h; importing it fails if the library has not been built.
"""
