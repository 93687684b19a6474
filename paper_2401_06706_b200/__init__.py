"""B200-native multi-candidate speculative-decoding verification (MCSD verify).

The CUDA library is loaded on first use of the binding, never at import time, so
the input generators in :mod:`.synth` stay importable on a machine without it.
"""
__all__ = ["synth"]
