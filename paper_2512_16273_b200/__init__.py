"""libtslt: B200-native sparsify / verify / tree-verify kernels of Truncated Sparse Logits
Transmission.  `tslt` is the binding of the C ABI; `synth` draws the synthetic workloads."""
from . import synth  # noqa: F401

__all__ = ["synth", "tslt"]


def __getattr__(name):
    if name == "tslt":
        import importlib
        return importlib.import_module(".tslt", __name__)
    raise AttributeError(name)
