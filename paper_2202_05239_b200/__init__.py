"""F8Net fixed-point 8-bit inference path for NVIDIA B200 (sm_100a).

``synth``  -- seeded synthetic layer descriptions and tensors (pure numpy);
``api``    -- thin binding over the C-ABI CUDA library (imported on demand:
              it needs the compiled library and raises if it is missing).
"""
from . import synth  # noqa: F401

__all__ = ["synth", "api"]


def __getattr__(name):
    if name == "api":
        import importlib
        return importlib.import_module(".api", __name__)
    raise AttributeError(name)
