"""B200-native signSGD / Signum / majority-vote step (Algorithms 1-3 of the paper).

The hot path lives in hand-written sm_100a CUDA kernels behind a C ABI
(``include/signsgd.h``); ``binding`` marshals torch tensors into that ABI and
``workloads`` draws the seeded synthetic inputs.  Importing the package does not
load the CUDA library; the first use of ``binding`` does, and fails loudly if the
library has not been built.
"""

__all__ = ["binding", "workloads"]


def __getattr__(name):
    if name in __all__:
        import importlib
        return importlib.import_module("." + name, __name__)
    raise AttributeError(name)
