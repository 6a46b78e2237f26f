"""B200-native binary-decomposition mixed-precision convolution (C-ABI CUDA library + thin binding).

``from paper_2003_07577_b200 import binding as ebs`` gives the Python names of the C entry points
declared in ``include/ebs.h``.  The CUDA library is built in-tree by ``build.build()``.
"""
from . import binding  # noqa: F401
from .build import build  # noqa: F401

__all__ = ["binding", "build"]
