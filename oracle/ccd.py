"""ctypes front end of the C checker (see ``ccd_oracle.c`` for what each step follows)."""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ccd_oracle.c")
_LIB = os.path.join(_HERE, "libccd_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the checker with gcc (-O2, OpenMP).  Returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"])
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(build())
        dp, ip, bp = C.POINTER(C.c_double), C.POINTER(C.c_int), C.POINTER(C.c_uint8)
        lib.ora_nuc_top.argtypes = [dp, C.c_int, C.c_int, ip]
        lib.ora_cap_scores.argtypes = [dp, dp, C.c_int, C.c_int, C.c_int, dp, dp]
        lib.ora_select.argtypes = [dp, C.c_int, ip, C.c_int, C.c_int, ip]
        lib.ora_gather.argtypes = [bp, C.c_size_t, ip, C.c_int, bp]
        lib.ora_cycle.argtypes = [dp, dp, bp, bp, dp, ip, C.c_int, C.c_int, C.c_int, C.c_int,
                                  C.c_int, C.c_int, C.c_int, C.c_size_t, dp, ip, bp, bp]
        lib.ora_cap_scores_incl.argtypes = [dp, dp, dp, C.c_int, C.c_int, C.c_int, C.c_int, dp, dp]
        lib.ora_cycle_cap.argtypes = [dp, dp, dp, bp, bp, dp, ip, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                      C.c_int, C.c_int, C.c_int, C.c_size_t, dp, ip, bp, bp]
        lib.ora_token_novelty.argtypes = [dp, ip, C.c_long, C.c_int, dp]
        lib.ora_rope_rows.argtypes = [C.c_void_p, C.c_void_p, ip, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_int, dp, dp]
        lib.ora_decode_attention.argtypes = [dp, dp, dp, C.c_int, C.c_int, C.c_int, dp, dp]
        lib.ora_set_threads.argtypes = [C.c_int]
        lib.ora_max_threads.restype = C.c_int
        for f in (lib.ora_nuc_top, lib.ora_cap_scores, lib.ora_select, lib.ora_gather,
                  lib.ora_cycle, lib.ora_set_threads, lib.ora_cap_scores_incl, lib.ora_cycle_cap, lib.ora_token_novelty, lib.ora_rope_rows, lib.ora_decode_attention):
            f.restype = None
        _lib = lib
    return _lib


def _p(a, t):
    return a.ctypes.data_as(C.POINTER(t))


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def widen_storage(a: np.ndarray) -> np.ndarray:
    """float32, or uint16 holding bfloat16 bit patterns -> float64 (exact)."""
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:
        return (a.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    if a.dtype in (np.float32, np.float64):
        return a.astype(np.float64)
    raise TypeError(f"unsupported storage dtype {a.dtype}")


def set_threads(n: int) -> None:
    _load().ora_set_threads(int(n))


def max_threads() -> int:
    return int(_load().ora_max_threads())


def rope_rows(rows, pos, cos_t, sin_t, interleaved: bool = False, with_exact: bool = False):
    """Sec. 3.4: rotary embedding of rows [..., n, d] (storage dtype: float32 or uint16 bf16 bits) at positions
    pos [n] with cos/sin tables [positions][d/2] of the same storage dtype; every leading index uses the same
    positions.  Computed in float64 and rounded once: returns the rotated rows in the storage dtype, and with
    ``with_exact`` also the unrounded float64 values and the size of the two terms each value is the sum or
    difference of (what bounds the cancellation error of a single-precision evaluation)."""
    rows = np.ascontiguousarray(rows)
    cos_t, sin_t = np.ascontiguousarray(cos_t), np.ascontiguousarray(sin_t)
    assert rows.dtype in (np.float32, np.uint16) and cos_t.dtype == rows.dtype and sin_t.dtype == rows.dtype
    n, d = rows.shape[-2], rows.shape[-1]
    pos = np.ascontiguousarray(pos, dtype=np.int32)
    assert pos.shape == (n,) and d % 2 == 0 and cos_t.shape == sin_t.shape and cos_t.shape[1] == d // 2
    assert pos.min(initial=0) >= 0 and pos.max(initial=0) < cos_t.shape[0]
    out = np.empty_like(rows)
    exact = np.empty(rows.shape, dtype=np.float64) if with_exact else None
    mag = np.empty(rows.shape, dtype=np.float64) if with_exact else None
    flat_in, flat_out = rows.reshape(-1, n, d), out.reshape(-1, n, d)
    for i in range(flat_in.shape[0]):
        ex = _p(exact.reshape(-1, n, d)[i], C.c_double) if with_exact else None
        mg = _p(mag.reshape(-1, n, d)[i], C.c_double) if with_exact else None
        _load().ora_rope_rows(flat_in[i].ctypes.data, flat_out[i].ctypes.data, _p(pos, C.c_int), n, d,
                              int(rows.dtype == np.float32), cos_t.ctypes.data, sin_t.ctypes.data, int(interleaved), ex, mg)
    return (out, exact, mag) if with_exact else out


def decode_attention(q, K, V, n: int | None = None):
    """Generation over the pot: q [L][B][Hq][d], K, V [L][B][Hkv][rows][d] in storage dtype (the first ``n`` rows
    count; K as the queries should see it, i.e. rotated if the pot is in rotary mode).  Query head h reads the
    rows of KV head h // G.  Returns (out [L][B][Hq][d], lse [L][B][Hq]) in float64."""
    L, B, Hq, d = q.shape
    Hkv = K.shape[2]
    n = K.shape[3] if n is None else n
    G = Hq // Hkv
    qd = widen_storage(q).reshape(L * B * Hkv, G, d)
    Kd = widen_storage(np.ascontiguousarray(K[:, :, :, :n])).reshape(L * B * Hkv, n, d)
    Vd = widen_storage(np.ascontiguousarray(V[:, :, :, :n])).reshape(L * B * Hkv, n, d)
    out = np.empty((L * B * Hkv, G, d), dtype=np.float64)
    lse = np.empty((L * B * Hkv, G), dtype=np.float64)
    for u in range(L * B * Hkv):
        _load().ora_decode_attention(_p(np.ascontiguousarray(qd[u]), C.c_double), _p(Kd[u], C.c_double), _p(Vd[u], C.c_double),
                                     G, n, d, _p(out[u], C.c_double), _p(lse[u], C.c_double))
    return out.reshape(L, B, Hq, d), lse.reshape(L, B, Hq)


def token_novelty(logits, labels) -> np.ndarray:
    """Eq. 3: logits [n][V] (float64), labels [n] -> -log softmax(logits)[label] per token [n]."""
    z = _f64(logits)
    lab = np.ascontiguousarray(labels, dtype=np.int32)
    n, V = z.shape
    assert lab.shape == (n,)
    out = np.empty(n, dtype=np.float64)
    _load().ora_token_novelty(_p(z, C.c_double), _p(lab, C.c_int), n, V, _p(out, C.c_double))
    return out


def nuc_top(aux, T: int) -> np.ndarray:
    """Sec. 3.3.3: the T slots with the largest novelty, ascending."""
    aux = _f64(aux)
    out = np.empty(T, dtype=np.int32)
    _load().ora_nuc_top(_p(aux, C.c_double), aux.shape[0], T, _p(out, C.c_int))
    return out


def cap_scores(Q, K, return_row_sums: bool = False):
    """Eq. 2 for one KV head: Q [M][d], K [N][d] (float64) -> u [N]."""
    Q, K = _f64(Q), _f64(K)
    M, d = Q.shape
    N = K.shape[0]
    assert K.shape[1] == d
    u = np.empty(N, dtype=np.float64)
    rs = np.empty(M, dtype=np.float64)
    _load().ora_cap_scores(_p(Q, C.c_double), _p(K, C.c_double), M, N, d, _p(u, C.c_double),
                           _p(rs, C.c_double))
    return (u, rs) if return_row_sums else u


def cap_scores_incl(Q, K, Kc, P: int, return_pot_mass: bool = False):
    """Appendix B listing read literally, one KV head: Q [G*P][d], K [N][d], Kc [P][d] (float64) -> u [N].
    Row r sees the pot keys and the CaP keys 0..r % P; only the pot columns are summed."""
    Q, K, Kc = _f64(Q), _f64(K), _f64(Kc)
    M, d = Q.shape
    N = K.shape[0]
    assert K.shape[1] == d and Kc.shape == (P, d) and M % P == 0
    u = np.empty(N, dtype=np.float64)
    pm = np.empty(M, dtype=np.float64)
    _load().ora_cap_scores_incl(_p(Q, C.c_double), _p(K, C.c_double), _p(Kc, C.c_double), M, N, d, P,
                                _p(u, C.c_double), _p(pm, C.c_double))
    return (u, pm) if return_pot_mass else u


def select(u, nuc, keep: int) -> np.ndarray:
    """Sec. 3.3.3 / Appendix B: NuC slots + best (keep - T) other slots, ascending."""
    u = _f64(u)
    nuc = np.ascontiguousarray(nuc, dtype=np.int32)
    idx = np.empty(keep, dtype=np.int32)
    _load().ora_select(_p(u, C.c_double), u.shape[0], _p(nuc, C.c_int), nuc.shape[0], keep,
                       _p(idx, C.c_int))
    return idx


def gather(rows: np.ndarray, idx) -> np.ndarray:
    """Appendix B "KV-cache compression": rows [N][...] -> rows[idx], byte-wise."""
    rows = np.ascontiguousarray(rows)
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    rb = rows[0].nbytes
    out = np.empty((idx.shape[0],) + rows.shape[1:], dtype=rows.dtype)
    _load().ora_gather(_p(rows.view(np.uint8).reshape(-1), C.c_uint8), rb, _p(idx, C.c_int),
                       idx.shape[0], _p(out.view(np.uint8).reshape(-1), C.c_uint8))
    return out


def cycle(Q, K, V, aux, keep: int, T: int, units=None, with_kv: bool = True, K_cap=None, rope=None):
    """One CCD cycle over all (or the listed) units.

    Q [L][B][Hq][P][d], K, V [L][B][Hkv][N][d] in storage dtype (float32 or
    uint16 bfloat16 bits), aux [B][N].  ``units`` lists flat unit indices
    ``(l*B + b)*Hkv + g``.  Returns a dict with ``units``, ``u`` [n][N],
    ``idx`` [n][keep] and, if ``with_kv``, the compacted ``K``, ``V`` [n][keep][d].
    With ``K_cap`` [L][B][Hkv][P][d] the scores are the CaP-inclusive ones.
    With ``rope = (cos_t, sin_t, interleaved)`` K holds keys without rotary embedding: the scores use the keys
    rotated at their slot number 0..N-1 (Sec. 3.4), the gather moves the unrotated rows, and ``K_rot``
    [n][keep][d] is the compacted pot rotated at the new slot numbers 0..keep-1.
    """
    L, B, Hq, P, d = Q.shape
    Hkv, N = K.shape[2], K.shape[3]
    assert K.shape == (L, B, Hkv, N, d) and V.shape == K.shape and Hq % Hkv == 0
    G = Hq // Hkv
    M = G * P
    all_units = L * B * Hkv
    units = np.arange(all_units, dtype=np.int32) if units is None else np.asarray(units, dtype=np.int32)
    n = units.shape[0]
    Kf = np.ascontiguousarray(K).reshape(all_units, N, d)
    Vf = np.ascontiguousarray(V).reshape(all_units, N, d)
    # the G query heads of KV head g are heads g*G .. g*G+G-1: one contiguous [M][d] block
    Qf = np.ascontiguousarray(Q).reshape(all_units, M, d)
    Ks = np.ascontiguousarray(Kf[units])
    Vs = np.ascontiguousarray(Vf[units])
    Qd = widen_storage(Qf[units])
    Kd = widen_storage(Ks if rope is None else rope_rows(Ks, np.arange(N), rope[0], rope[1], rope[2]))
    Kcd = None
    if K_cap is not None:
        assert K_cap.shape == (L, B, Hkv, P, d)
        Kcd = widen_storage(np.ascontiguousarray(K_cap).reshape(all_units, P, d)[units])
    auxd = _f64(aux)
    assert auxd.shape == (B, N)
    stream_of = np.ascontiguousarray((units // Hkv) % B, dtype=np.int32)
    rb = d * Ks.dtype.itemsize
    u = np.empty((n, N), dtype=np.float64)
    idx = np.empty((n, keep), dtype=np.int32)
    Ko = np.empty((n, keep, d), dtype=Ks.dtype) if with_kv else None
    Vo = np.empty((n, keep, d), dtype=Vs.dtype) if with_kv else None
    bp = C.POINTER(C.c_uint8)
    _load().ora_cycle_cap(
        _p(Qd, C.c_double), _p(Kd, C.c_double), _p(Kcd, C.c_double) if Kcd is not None else None,
        Ks.ctypes.data_as(bp), Vs.ctypes.data_as(bp), _p(auxd, C.c_double), _p(stream_of, C.c_int),
        n, B, M, P, d, N, keep, T, rb, _p(u, C.c_double), _p(idx, C.c_int),
        Ko.ctypes.data_as(bp) if with_kv else None, Vo.ctypes.data_as(bp) if with_kv else None)
    out = {"units": units, "u": u, "idx": idx, "K": Ko, "V": Vo}
    if rope is not None and with_kv:
        out["K_rot"] = rope_rows(Ko, np.arange(keep), rope[0], rope[1], rope[2])
    return out
