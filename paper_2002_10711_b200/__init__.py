"""B200 (sm_100a) forward pass of the Winograd-aware quantized 3x3 convolution
(arXiv 2002.10711, Eq. 1 with the quantizers of Fig. 2), as a C-ABI CUDA
library plus this thin binding."""
from .cooktoom import STANDARD_POINTS, cook_toom, cook_toom_exact  # noqa: F401


def __getattr__(name):
    # the binding loads the CUDA library; import it lazily so that helpers that
    # need no GPU code (matrix construction) stay importable on their own
    if name in ("binding", "Plan", "layer"):
        import importlib
        if name == "Plan":
            return importlib.import_module(".binding", __name__).Plan
        return importlib.import_module("." + name, __name__)
    raise AttributeError(name)
