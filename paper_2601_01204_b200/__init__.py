"""B200-native compressed KV cache for streaming frame-causal attention.

`paper_2601_01204_b200.xkv` is the binding of the CUDA library (libxkv.so); it
raises at import when the library has not been built.  `synth` is the seeded
input generator (numpy, no CUDA).
"""
