"""B200-native kernels for LightVLM's token reduction and KV-cache compression.

``binding`` wraps the C-ABI library (``include/lvlm.h``); ``inputs`` holds the seeded synthetic
workloads; ``build`` compiles the library in-tree with nvcc for sm_100a.
"""
