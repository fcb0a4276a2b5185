"""B200-native CCD compression cycle of InfiniPot (arxiv 2410.01518).

``ipot``   : thin ctypes binding of the C-ABI library (``libipot.so``)
``inputs`` : seeded synthetic input generators (no method arithmetic)

Importing the package loads nothing native; the CUDA library is loaded on first
use of ``ipot`` and a missing library is an error, never a fallback.
"""
__all__ = ["inputs", "ipot"]
