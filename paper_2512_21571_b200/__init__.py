"""B200-native Qwen3 forward pass (prefill + decode) behind the `nnc_*` C ABI.

`synth` (seeded inputs) imports nothing from the CUDA side; the binding in `binding` loads the shared library
lazily and fails loudly if it has not been built.
"""
