"""B200-native mixed-precision KV-cache quantization hot path (quantize-append,
fused low-bit decode attention, dequantize) behind a C-ABI library.

`workloads` (synthetic input generators) imports without the CUDA library;
`kvq` (the binding) loads `libkvq.so` on first access and raises if it is missing.
"""
from . import workloads  # noqa: F401


def __getattr__(name):
    if name == "kvq":
        import importlib
        return importlib.import_module(__name__ + ".kvq")
    raise AttributeError(name)
