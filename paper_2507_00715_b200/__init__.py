"""B200-native attention hot path of EARN (register-token layer-split inference).

``workloads`` draws the seeded synthetic inputs; ``binding`` is the thin
ctypes layer over the C-ABI library built from ``csrc/``.  Importing the
package never loads the CUDA library; ``binding.lib()`` does, and raises if it
is missing.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads"]
