"""B200-native hot path of KV-cache reuse (prefix keys, residency index, longest cached prefix,
route score, paged-KV gather/scatter) behind a C ABI; see include/aibx.h.

``binding`` is the Python face of the C library, ``build`` compiles the CUDA sources in-tree.
"""
