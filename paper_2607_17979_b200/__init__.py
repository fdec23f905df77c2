"""B200-native gated delta rule (Gated DeltaNet) decode and chunked prefill.

The product is the C-ABI library built from ``csrc/`` (see ``include/gdn.h``);
``paper_2607_17979_b200.api`` is the thin argument-marshalling binding.  The
binding is imported lazily so that the input generator can be used on a machine
without the CUDA library.
"""

__all__ = ["api", "inputs"]


def __getattr__(name):
    if name in ("api", "inputs"):
        import importlib
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
