"""B200 (sm_100a) mixture-of-experts FFN layer: CUDA library + thin ctypes binding.

`MoELayer` (binding.py) is the public entry; `synth` holds the seeded input generators; `build` compiles the
library in-tree.  Importing the package loads nothing heavy."""


def __getattr__(name):
    if name in ("MoELayer", "load_library", "MoEError", "listwise_loss"):
        from . import binding
        return getattr(binding, name)
    raise AttributeError(name)
