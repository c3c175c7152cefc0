"""SnapStream hot path for NVIDIA B200: a thin Python binding over libsnapstream.so.

The CUDA library (csrc/, built by ``python -m paper_2511_03092_b200.build``) does all the
work; this package only marshals arguments.  ``synth`` holds the seeded input generators.
"""
from . import synth  # noqa: F401


def __getattr__(name):
    # binding is imported lazily so that `synth` is usable before the library is built
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
