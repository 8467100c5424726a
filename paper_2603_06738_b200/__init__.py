"""B200-native RIB window attention: C-ABI CUDA library plus a thin binding.

``binding`` marshals torch tensors into the C calls of ``include/rib_window_attn.h``;
``synthetic`` draws the seeded benchmark inputs; ``build`` compiles the library in-tree.
"""
