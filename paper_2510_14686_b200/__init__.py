"""B200-native decode / speculative-verification GQA attention over an xTensor-style KV cache.

The product is the C-ABI library ``libxllm_attn.so`` (sources under ``csrc/``) and the thin
``ctypes`` binding in :mod:`paper_2510_14686_b200.binding`.  Importing the package itself loads no
native code, so the seeded input generators in :mod:`paper_2510_14686_b200.workloads` can be used on a
machine without a GPU; every attribute of the binding is resolved lazily and raises loudly when the
shared library has not been built.
"""

__all__ = ["binding", "workloads", "build"]


def __getattr__(name):
    if name in ("binding", "workloads", "build"):
        import importlib

        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
