"""B200-native dynamic activation sparsity (arXiv 2503.20354): C-ABI CUDA library + binding.

`workloads` (shape tables, seeded inputs) imports without the CUDA library; everything in
`binding` needs the compiled `libsurgeon.so` and fails loudly when it is missing.
"""
