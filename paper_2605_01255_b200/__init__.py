"""acx: activation-gradient co-compressed linear layers for B200 (sm_100a).

The package holds the CUDA library sources (``csrc/``), the ctypes binding to its C ABI
(``binding``) and the seeded synthetic-input recipes (``inputs``).  Nothing here computes on the
CPU: every call goes to ``libacx.so`` and fails loudly if that library is not built.
"""
__all__ = ["binding", "inputs"]
