"""B200-native weight-grouped LM-head draft step (CORAL, Section 3.3).

`lmhead` binds the C ABI of the CUDA library; `synth` draws seeded inputs.
"""
