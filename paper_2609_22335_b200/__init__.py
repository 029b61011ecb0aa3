"""B200-native two-phase Vision-Language-Action inference with tile-level co-scheduling.

The product is the CUDA library built from ``csrc/`` (C ABI in ``include/vla.h``);
``api`` is its thin ctypes binding.
"""
from . import api  # noqa: F401
from .api import Engine, load_library, make_desc, policy_probe  # noqa: F401
