"""B200-native GPTQ int4 matmul (C-ABI CUDA library + thin Python binding).

``workloads`` (seeded synthetic inputs) imports without CUDA; everything in
``binding`` needs the compiled library and raises if it is missing.
"""
