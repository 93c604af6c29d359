"""B200-native BitLinear forward of BitNet a4.8 (arXiv 2411.04965).

The computation lives in the CUDA library behind the C ABI declared in
``include/bitnet_a48.h``; ``binding`` marshals arguments to it.
"""
