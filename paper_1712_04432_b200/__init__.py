"""B200-native matrix-form minibatch-SGD training step over a logical
P_r x P_c block grid (forward Y = W X, backward dX = W^T dY, dW = dY X^T,
update w <- w - (eta/B) dW), as a C-ABI CUDA library plus this thin binding.

Importing the package does not load the CUDA library; the first call that
needs it does, and raises if it has not been built.
"""
from . import inputs  # noqa: F401  (pure numpy, no CUDA)

__all__ = ["inputs", "mbd"]


def __getattr__(name):
    if name == "mbd":
        import importlib
        return importlib.import_module(".mbd", __name__)
    raise AttributeError(name)
