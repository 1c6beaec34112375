"""B200-native candidate screen, timing adjudication and survivor selection
(the data-parallel hot path of KernelBrain's evaluation loop, arxiv 2608.02611).

The work is done by a C-ABI CUDA library (``include/kb.h``, built in-tree as
``libkb.so``); ``binding`` marshals arguments, ``synth`` makes seeded inputs.
"""
from . import synth  # noqa: F401


def __getattr__(name):
    # binding needs ctypes + the built library; import it on first use so that
    # input generation stays usable on a machine without the library.
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
