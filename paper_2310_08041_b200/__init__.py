"""B200 (sm_100a) hot path of a QLLM quantized linear layer (arXiv 2310.08041).

``binding`` holds the ctypes bindings of the C ABI declared in ``include/qllm.h``;
``synth`` the seeded synthetic inputs.  The CUDA library is loaded on first use
of ``binding`` and its absence is an error: there is no CPU fallback.
"""
__all__ = ["binding", "synth"]


def __getattr__(name):
    if name in ("binding", "synth"):
        import importlib
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
