"""SnapKV prompt KV-cache compression step for NVIDIA B200 (sm_100a).

The compute path is the C-ABI shared library built from ``csrc/``; ``binding``
marshals torch tensors into it.  Importing the package does not load the
library; the first call does, and raises if it has not been built.
"""

__all__ = ["binding", "synth"]
