"""B200-native TriAttention KV-compression round: score -> top-B select -> compaction.

The work is done by hand-written sm_100a kernels behind a C-ABI shared library
(``include/tri_attention.h``); :mod:`.binding` marshals torch tensors into it and fails
loudly when the library is missing.  :mod:`.workloads` only makes seeded synthetic inputs.
"""

__all__ = ["binding", "workloads"]
