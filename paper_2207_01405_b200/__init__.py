"""B200-native integer-only ViT encoder forward pass (I-ViT): CUDA kernels behind a C ABI.

`binding` holds the ctypes front end of libivit.so; `build` compiles the library in-tree.
"""
