"""CPU checker for the CCD compression cycle (test infrastructure only).

Thin ctypes front end of ``ccd_oracle.c``: plain double-precision loops that
follow the paper's definitions (Eq. 2, Sec. 3.3.3, Appendix B).  Nothing here is
imported by the CUDA library or its Python binding; only the tests, the smoke
check and the benchmark's CPU-baseline leg call it.
"""
from .ccd import (build, cap_scores, cap_scores_incl, cycle, decode_attention, gather, max_threads, nuc_top, rope_rows, select,
                  set_threads, token_novelty, widen_storage)

__all__ = ["build", "cap_scores", "cap_scores_incl", "cycle", "decode_attention", "gather", "max_threads", "nuc_top", "rope_rows", "select",
           "set_threads", "token_novelty", "widen_storage"]
