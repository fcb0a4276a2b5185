"""Thin ctypes binding of the memory-pot C ABI (``include/ipot.h``).

Argument marshalling only: every step of the compression cycle runs in the CUDA
kernels of ``libipot.so``.  The functions carry the names of the C entry points
and turn a negative return code into an exception (``IpotError``).  Tensors are
passed as anything with a ``data_ptr()`` method (torch tensors), numpy arrays
(host variants) or raw integer addresses.

The library is loaded on first use.  If it is missing or older than its sources
it is built when ``nvcc`` is available; there is no fallback implementation.
"""
from __future__ import annotations

import ctypes as C
import os

from . import build as _build

IPOT_OK, IPOT_E_INVALID, IPOT_E_STATE, IPOT_E_NOMEM, IPOT_E_CUDA, IPOT_E_TIMEOUT, IPOT_E_BOUNDS, IPOT_E_LIMIT = 0, -1, -2, -3, -4, -5, -6, -7
IPOT_NOALLOC_MAX_ROWS = 65536
IPOT_BF16, IPOT_F32 = 0, 1
IPOT_SCORER_AUTO, IPOT_SCORER_SIMT, IPOT_SCORER_TENSOR, IPOT_SCORER_WARP_MMA, IPOT_SCORER_TENSOR_SWEEPS = 0, 1, 2, 3, 4
IPOT_TUNE_SWEEPS_CLUSTER, IPOT_TUNE_SWEEPS_FMA_EIGHTHS, IPOT_TUNE_WAIT_LIMIT_NS, IPOT_TUNE_TEST_WITHHOLD_RANK = 1, 2, 3, 4
IPOT_ROPE_HALF, IPOT_ROPE_INTERLEAVED = 1, 2

# every symbol include/ipot.h declares
SYMBOLS = [
    "ipot_create", "ipot_create_ex", "ipot_destroy", "ipot_set_stream", "ipot_set_nuc_slots",
    "ipot_set_scorer", "ipot_set_deferred_append", "ipot_reset", "ipot_append_chunk", "ipot_append_chunk_host",
    "ipot_score_and_compress", "ipot_score_and_compress_host", "ipot_score_only", "ipot_view",
    "ipot_last_indices", "ipot_last_scores", "ipot_sync_status", "ipot_set_profiling",
    "ipot_kernel_ms", "ipot_launch_count", "ipot_strerror", "ipot_cap_scores_noalloc",
    "ipot_score_and_compress_cap", "ipot_score_only_cap", "ipot_score_and_compress_cap_host",
    "ipot_nuc_scores", "ipot_enable_rope", "ipot_view_rope",
    "ipot_decode_attention", "ipot_set_tuning",
]


class ipot_config_t(C.Structure):
    _fields_ = [("pot_size", C.c_int), ("keep", C.c_int), ("layers", C.c_int), ("Hq", C.c_int),
                ("Hkv", C.c_int), ("d", C.c_int), ("batch", C.c_int), ("dtype", C.c_int),
                ("nuc_slots", C.c_int), ("max_cap_rows", C.c_int), ("stream", C.c_void_p)]


class IpotError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {ipot_strerror(code)} ({code})")


_lib = None


def lib() -> C.CDLL:
    """The loaded C library (built first if stale and nvcc is present)."""
    global _lib
    if _lib is None:
        path = _build.LIB
        if _build.stale():
            try:
                _build.build()
            except Exception as e:  # no nvcc on this machine
                if not os.path.exists(path):
                    raise RuntimeError(f"libipot.so is missing and could not be built: {e}") from e
        L = C.CDLL(path)
        vp, ip = C.c_void_p, C.c_int
        L.ipot_create.argtypes = [ip] * 6 + [C.POINTER(vp)]
        L.ipot_create_ex.argtypes = [C.POINTER(ipot_config_t), C.POINTER(vp)]
        L.ipot_destroy.argtypes = [vp]
        L.ipot_set_stream.argtypes = [vp, vp]
        L.ipot_set_nuc_slots.argtypes = [vp, ip]
        L.ipot_set_scorer.argtypes = [vp, ip]
        L.ipot_set_deferred_append.argtypes = [vp, ip]
        L.ipot_set_tuning.argtypes = [vp, ip, C.c_longlong]
        L.ipot_reset.argtypes = [vp]
        L.ipot_append_chunk.argtypes = [vp, vp, vp, ip]
        L.ipot_append_chunk_host.argtypes = [vp, vp, vp, ip]
        L.ipot_score_and_compress.argtypes = [vp, vp, ip, vp]
        L.ipot_score_and_compress_host.argtypes = [vp, vp, ip, vp, vp]
        L.ipot_score_only.argtypes = [vp, vp, ip, vp]
        L.ipot_score_and_compress_cap.argtypes = [vp, vp, vp, ip, vp]
        L.ipot_score_only_cap.argtypes = [vp, vp, vp, ip, vp]
        L.ipot_score_and_compress_cap_host.argtypes = [vp, vp, vp, ip, vp, vp]
        L.ipot_nuc_scores.argtypes = [vp, vp, ip, C.c_longlong, vp, ip, ip, vp, C.c_longlong, ip]
        L.ipot_decode_attention.argtypes = [vp, vp, vp, vp]
        L.ipot_enable_rope.argtypes = [vp, vp, vp, ip]
        L.ipot_view_rope.argtypes = [vp, C.POINTER(vp)]
        L.ipot_view.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), C.POINTER(ip)]
        L.ipot_last_indices.argtypes = [vp, C.POINTER(vp)]
        L.ipot_last_scores.argtypes = [vp, C.POINTER(vp), C.POINTER(ip)]
        L.ipot_sync_status.argtypes = [vp]
        L.ipot_set_profiling.argtypes = [vp, ip]
        L.ipot_kernel_ms.argtypes = [vp, C.POINTER(C.c_float), C.POINTER(ip), C.POINTER(ip)]
        L.ipot_launch_count.argtypes = [vp, C.POINTER(C.c_longlong)]
        L.ipot_strerror.argtypes = [ip]
        L.ipot_cap_scores_noalloc.argtypes = [vp, vp, vp, ip, ip, ip, ip, ip, ip, vp]
        L.ipot_strerror.restype = C.c_char_p
        for s in SYMBOLS:
            if s != "ipot_strerror":
                getattr(L, s).restype = ip
        _lib = L
    return _lib


def _ptr(x):
    if x is None:
        return None
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if hasattr(x, "ctypes"):
        return x.ctypes.data
    return int(x)


def _check(rc: int, what: str) -> int:
    if rc < 0:
        raise IpotError(rc, what)
    return rc


def ipot_strerror(code: int) -> str:
    return lib().ipot_strerror(code).decode()


def ipot_create(pot_size, keep, layers, Hq, Hkv, d) -> int:
    h = C.c_void_p()
    _check(lib().ipot_create(pot_size, keep, layers, Hq, Hkv, d, C.byref(h)), "ipot_create")
    return h.value


def ipot_create_ex(pot_size, keep, layers, Hq, Hkv, d, batch=1, dtype=IPOT_BF16, nuc_slots=-1,
                   max_cap_rows=64, stream=None) -> int:
    cfg = ipot_config_t(pot_size, keep, layers, Hq, Hkv, d, batch, dtype, nuc_slots, max_cap_rows, stream)
    h = C.c_void_p()
    _check(lib().ipot_create_ex(C.byref(cfg), C.byref(h)), "ipot_create_ex")
    return h.value


def ipot_destroy(h) -> None:
    _check(lib().ipot_destroy(h), "ipot_destroy")


def ipot_set_stream(h, stream) -> None:
    _check(lib().ipot_set_stream(h, stream), "ipot_set_stream")


def ipot_set_nuc_slots(h, T) -> None:
    _check(lib().ipot_set_nuc_slots(h, T), "ipot_set_nuc_slots")


def ipot_set_scorer(h, scorer) -> None:
    _check(lib().ipot_set_scorer(h, scorer), "ipot_set_scorer")


def ipot_set_tuning(h, what, value) -> None:
    _check(lib().ipot_set_tuning(h, what, value), "ipot_set_tuning")


def ipot_set_deferred_append(h, on) -> None:
    _check(lib().ipot_set_deferred_append(h, 1 if on else 0), "ipot_set_deferred_append")


def ipot_reset(h) -> None:
    _check(lib().ipot_reset(h), "ipot_reset")


def ipot_append_chunk(h, K, V, n_tokens) -> None:
    _check(lib().ipot_append_chunk(h, _ptr(K), _ptr(V), n_tokens), "ipot_append_chunk")


def ipot_append_chunk_host(h, K, V, n_tokens) -> None:
    _check(lib().ipot_append_chunk_host(h, _ptr(K), _ptr(V), n_tokens), "ipot_append_chunk_host")


def ipot_score_and_compress(h, Q_cap, cap_rows, aux_scores) -> None:
    _check(lib().ipot_score_and_compress(h, _ptr(Q_cap), cap_rows, _ptr(aux_scores)), "ipot_score_and_compress")


def ipot_score_and_compress_host(h, Q_cap, cap_rows, aux_scores, idx_out=None) -> None:
    _check(lib().ipot_score_and_compress_host(h, _ptr(Q_cap), cap_rows, _ptr(aux_scores), _ptr(idx_out)),
           "ipot_score_and_compress_host")


def ipot_score_only(h, Q_cap, cap_rows, aux_scores=None) -> None:
    _check(lib().ipot_score_only(h, _ptr(Q_cap), cap_rows, _ptr(aux_scores)), "ipot_score_only")


def ipot_score_and_compress_cap(h, Q_cap, K_cap, cap_rows, aux_scores) -> None:
    _check(lib().ipot_score_and_compress_cap(h, _ptr(Q_cap), _ptr(K_cap), cap_rows, _ptr(aux_scores)),
           "ipot_score_and_compress_cap")


def ipot_score_and_compress_cap_host(h, Q_cap, K_cap, cap_rows, aux_scores, idx_out=None) -> None:
    _check(lib().ipot_score_and_compress_cap_host(h, _ptr(Q_cap), _ptr(K_cap), cap_rows, _ptr(aux_scores), _ptr(idx_out)),
           "ipot_score_and_compress_cap_host")


def ipot_score_only_cap(h, Q_cap, K_cap, cap_rows, aux_scores=None) -> None:
    _check(lib().ipot_score_only_cap(h, _ptr(Q_cap), _ptr(K_cap), cap_rows, _ptr(aux_scores)), "ipot_score_only_cap")


def ipot_nuc_scores(h, logits, logits_dtype, row_stride, labels, n_tokens, vocab, aux_out, aux_stride, slot0) -> None:
    _check(lib().ipot_nuc_scores(h, _ptr(logits), logits_dtype, row_stride, _ptr(labels), n_tokens, vocab,
                                 _ptr(aux_out), aux_stride, slot0), "ipot_nuc_scores")


def ipot_decode_attention(h, q, out, lse=None) -> None:
    _check(lib().ipot_decode_attention(h, _ptr(q), _ptr(out), _ptr(lse)), "ipot_decode_attention")


def ipot_enable_rope(h, cos_table, sin_table, pairing) -> None:
    _check(lib().ipot_enable_rope(h, _ptr(cos_table), _ptr(sin_table), pairing), "ipot_enable_rope")


def ipot_view_rope(h) -> int:
    """-> device address of the rotated copy of the keys."""
    p = C.c_void_p()
    _check(lib().ipot_view_rope(h, C.byref(p)), "ipot_view_rope")
    return p.value


def ipot_view(h):
    """-> (K device address, V device address, len)."""
    K, V, n = C.c_void_p(), C.c_void_p(), C.c_int()
    _check(lib().ipot_view(h, C.byref(K), C.byref(V), C.byref(n)), "ipot_view")
    return K.value, V.value, n.value


def ipot_last_indices(h) -> int:
    p = C.c_void_p()
    _check(lib().ipot_last_indices(h, C.byref(p)), "ipot_last_indices")
    return p.value


def ipot_last_scores(h):
    """-> (device address, len_before)."""
    p, n = C.c_void_p(), C.c_int()
    _check(lib().ipot_last_scores(h, C.byref(p), C.byref(n)), "ipot_last_scores")
    return p.value, n.value


def ipot_sync_status(h) -> int:
    return lib().ipot_sync_status(h)


def ipot_set_profiling(h, on) -> None:
    _check(lib().ipot_set_profiling(h, int(on)), "ipot_set_profiling")


def ipot_kernel_ms(h):
    """-> ([nuc, score, select, compact] mean milliseconds, cycles averaged, scorer used)."""
    ms = (C.c_float * 4)()
    n, s = C.c_int(), C.c_int()
    _check(lib().ipot_kernel_ms(h, ms, C.byref(n), C.byref(s)), "ipot_kernel_ms")
    return list(ms), n.value, s.value


def ipot_launch_count(h) -> int:
    n = C.c_longlong()
    _check(lib().ipot_launch_count(h, C.byref(n)), "ipot_launch_count")
    return n.value


def ipot_cap_scores_noalloc(Q, K, scores, units, rows, N, d, k_unit_rows, dtype, stream=None) -> None:
    """CaP scores for callers that may not allocate device memory: Q [units][rows][d], K
    [units][k_unit_rows][d] (first N rows scored) -> scores [units][N] f32, all device buffers of
    the caller.  Scratch is a fixed array inside the library (units * rows <= IPOT_NOALLOC_MAX_ROWS)."""
    _check(lib().ipot_cap_scores_noalloc(_ptr(Q), _ptr(K), _ptr(scores), units, rows, N, d, k_unit_rows, dtype,
                                         stream), "ipot_cap_scores_noalloc")


def device_array(addr: int, shape, dtype, device="cuda"):
    """A torch tensor over library-owned device memory (no copy; borrowed)."""
    import numpy as np
    import torch

    tdt = {"bf16": torch.bfloat16, "f32": torch.float32, "i32": torch.int32, "u8": torch.uint8}[dtype]
    n = int(np.prod(shape))
    nbytes = n * torch.empty((), dtype=tdt).element_size()

    class _Holder:
        __cuda_array_interface__ = {"shape": (nbytes,), "typestr": "|u1", "data": (addr, False), "version": 2}

    return torch.as_tensor(_Holder(), device=device).view(tdt).view(*shape)
