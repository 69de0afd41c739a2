"""B200-native Temp-Lora chunk-update library: Python binding over the C-ABI.

`inputs` (seeded synthetic tensors) imports without the compiled library;
`binding` loads `libtemplora.so` and fails loudly if it is missing.
"""
__all__ = ["inputs", "binding", "build"]
