"""B200-native executor for combinator array programs: one CUDA kernel per fused cluster.

`binding.Graph` wraps the C ABI of include/acc.h; `build.build()` compiles libacc.so.
The CUDA library is loaded on first use; there is no CPU fallback, and using the
binding fails loudly if the library has not been built.
"""
