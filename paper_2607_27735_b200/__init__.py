"""B200-native attention hot path of SparseSpec-L self-speculative decoding.

Three CUDA entry points behind a C ABI (``include/spec_attn.h``): full-context verification
attention with the fused importance statistic, per-KV-head recall selection, and
index-gathered sparse draft attention.  ``binding`` holds the ctypes front end (imported
lazily so that the input generators can be used without the compiled library).
"""

__all__ = ["binding", "inputs", "build"]


def __getattr__(name):
    if name in __all__:
        import importlib

        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
