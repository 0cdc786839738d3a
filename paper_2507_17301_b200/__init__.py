"""Column-wise N:M sparse convolution for B200 (sm_100a): Python face of the C-ABI library.

``nm`` (the binding) is imported lazily so that importing the package for its input
recipes does not require the CUDA library to be built.
"""

__all__ = ["inputs", "nm"]


def __getattr__(name):
    if name == "nm":
        import importlib

        return importlib.import_module(__name__ + ".nm")
    raise AttributeError(name)
