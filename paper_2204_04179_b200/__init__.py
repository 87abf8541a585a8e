"""GRAM deduplicated encode/accumulate training step: CUDA library (sm_100a) and its Python binding.

`synth` (seeded inputs) imports without the compiled library; `binding` loads
`libgram.so` on first use and raises if it is missing: there is no CPU fallback.
"""
