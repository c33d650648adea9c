"""B200-native W1.58A8 BitLinear forward (BitNet b1.58 2B4T, Sections 2 and 5.1).

The compute lives in libbitlinear.so (hand-written CUDA for sm_100a behind a C
ABI, see include/bitlinear.h); `binding` marshals torch tensors into it and
`workloads` draws the seeded synthetic inputs.  Submodules load lazily so that
importing the package does not need a GPU or the built library.
"""
import importlib

__all__ = ["binding", "workloads", "build"]


def __getattr__(name):
    if name in __all__:
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
