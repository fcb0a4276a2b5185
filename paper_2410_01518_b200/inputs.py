"""Seeded synthetic inputs for the CCD compression cycle.

This module only *draws numbers*: it holds none of the method's arithmetic (no
logits, no softmax, no selection, no gather).  Both the CUDA path and the CPU
checker are fed from here so that they see byte-identical tensors.

Storage conventions
-------------------
* ``"f32"`` tensors are ``numpy.float32`` arrays.
* ``"bf16"`` tensors are ``numpy.uint16`` arrays holding the bfloat16 bit
  patterns (float32 rounded to nearest-even, upper 16 bits kept).
* ``widen()`` turns either into ``float64`` exactly (no rounding happens when a
  bf16/f32 value is widened).

Layouts (all C-contiguous)
--------------------------
``K, V``  : ``[L][B][Hkv][n][d]``      pot rows of one chunk / one full pot
``Q``     : ``[L][B][Hq][P][d]``       catalyst-prompt (CaP) query rows
``aux``   : ``[B][N]`` float32         per-slot novelty (NuC) score, higher = more novel
``K_cap`` : ``[L][B][Hkv][P][d]``      the CaP's own key rows (CaP-inclusive scoring only)

Random streams are counter based (Philox): every tensor is keyed by
``(seed, config, tensor id, layer, cycle-or-chunk)`` so a subset of layers or
chunks can be produced without generating the rest.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
import numpy as np

SEED_BASE = 0x1F1F0000

_T_K, _T_V, _T_Q, _T_AUX, _T_MISC, _T_KCAP, _T_LOGIT = 1, 2, 3, 4, 5, 6, 7


@dataclass(frozen=True)
class CcdConfig:
    """Shape of one CCD workload.  Names follow the paper: ``pot_size`` is the
    number of context slots of the memory pot, ``keep`` is |C|, ``nuc_slots`` is
    T, ``cap_rows`` is |P|."""

    cfg_id: int
    name: str
    layers: int
    batch: int
    Hq: int
    Hkv: int
    d: int
    pot_size: int
    cap_rows: int
    keep: int
    nuc_slots: int
    dtype: str  # "f32" | "bf16"
    recipe: str  # "normal" | "rope" | "stream" | "lognorm" | "student_dup"
    chunk: int = 0  # tokens per appended chunk (stream recipe)
    stream_tokens: int = 0

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    @property
    def units(self) -> int:
        return self.layers * self.batch * self.Hkv

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    @property
    def seed(self) -> int:
        return SEED_BASE + self.cfg_id

    def with_layers(self, layers: int) -> "CcdConfig":
        return replace(self, layers=layers)


CONFIGS = {
    1: CcdConfig(1, "tiny-f32", 1, 1, 8, 2, 64, 512, 16, 256, 128, "f32", "normal"),
    2: CcdConfig(2, "mistral7b-layer", 1, 1, 32, 8, 128, 4096, 32, 2048, 1024, "bf16", "rope"),
    3: CcdConfig(3, "mistral7b-stream-32L", 32, 1, 32, 8, 128, 4096, 32, 2048, 1024, "bf16",
                 "stream", chunk=2048, stream_tokens=131072),
    4: CcdConfig(4, "llama3-8b-batch16", 1, 16, 32, 8, 128, 8192, 64, 2048, 1024, "bf16", "lognorm"),
    5: CcdConfig(5, "llama3-70b-batch8", 1, 8, 64, 8, 128, 16384, 64, 4096, 2048, "bf16",
                 "student_dup"),
}


# --------------------------------------------------------------------------
# number formats
# --------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns, round to nearest, ties to even."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    b = x.view(np.uint32)
    r = (b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def store(x32: np.ndarray, dtype: str) -> np.ndarray:
    """float32 values -> storage array of the given dtype."""
    if dtype == "f32":
        return np.ascontiguousarray(x32, dtype=np.float32)
    if dtype == "bf16":
        return f32_to_bf16_bits(x32)
    raise ValueError(dtype)


def widen(a: np.ndarray, dtype: str) -> np.ndarray:
    """storage array -> float64, exactly."""
    if dtype == "f32":
        return np.asarray(a, dtype=np.float32).astype(np.float64)
    if dtype == "bf16":
        return bf16_bits_to_f32(a).astype(np.float64)
    raise ValueError(dtype)


def np_storage_dtype(dtype: str):
    return np.float32 if dtype == "f32" else np.uint16


# --------------------------------------------------------------------------
# counter-based random streams
# --------------------------------------------------------------------------
def _gen(seed: int, tensor: int, layer: int = 0, index: int = 0, sub: int = 0) -> np.random.Generator:
    key = np.array([seed & 0xFFFFFFFFFFFFFFFF, tensor], dtype=np.uint64)
    ctr = np.array([0, sub, index, layer], dtype=np.uint64)
    return np.random.Generator(np.random.Philox(counter=ctr, key=key))


def _normal(g: np.random.Generator, shape) -> np.ndarray:
    return g.standard_normal(shape, dtype=np.float32)


def _rope_rotate_half(x: np.ndarray, pos: np.ndarray, base: float = 10000.0) -> np.ndarray:
    """Rotary embedding with the rotate-half pairing (channel c pairs with
    c + d/2).  ``x``: [..., n, d] float32, ``pos``: [n].  Part of the *input
    recipe* only: the compression path treats K and Q as opaque."""
    d = x.shape[-1]
    half = d // 2
    inv = base ** (-np.arange(half, dtype=np.float64) / half)
    ang = pos.astype(np.float64)[:, None] * inv[None, :]
    c, s = np.cos(ang), np.sin(ang)
    x1 = x[..., :half].astype(np.float64)
    x2 = x[..., half:].astype(np.float64)
    out = np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)
    return out.astype(np.float32)


def make_rope_table(positions: int, d: int, dtype: str, base: float = 10000.0):
    """The caller's side of CR-RoPE: cos and sin of ``pos * base**(-c / (d/2))`` for pos < positions and
    frequency c < d/2, evaluated in float64 and stored in the pot's storage dtype.  Returns (cos, sin),
    each [positions][d/2]."""
    half = d // 2
    inv = base ** (-np.arange(half, dtype=np.float64) / half)
    ang = np.arange(positions, dtype=np.float64)[:, None] * inv[None, :]
    return store(np.cos(ang).astype(np.float32), dtype), store(np.sin(ang).astype(np.float32), dtype)


def make_aux(cfg: CcdConfig, cycle: int = 0, n: int | None = None) -> np.ndarray:
    """aux[B][n] ~ U(0,1), float32."""
    n = cfg.pot_size if n is None else n
    g = _gen(cfg.seed, _T_AUX, 0, cycle)
    return g.random((cfg.batch, n), dtype=np.float32)


def make_q(cfg: CcdConfig, cycle: int = 0, layers=None, cap_rows: int | None = None) -> np.ndarray:
    """Q[L][B][Hq][P][d] in storage dtype."""
    P = cfg.cap_rows if cap_rows is None else cap_rows
    layers = range(cfg.layers) if layers is None else layers
    out = []
    for l in layers:
        q = _normal(_gen(cfg.seed, _T_Q, l, cycle), (cfg.batch, cfg.Hq, P, cfg.d))
        if cfg.recipe == "rope":
            q = _rope_rotate_half(q, np.arange(cfg.pot_size, cfg.pot_size + P))
        out.append(store(q, cfg.dtype))
    return np.stack(out, axis=0)


def make_kcap(cfg: CcdConfig, cycle: int = 0, layers=None, cap_rows: int | None = None) -> np.ndarray:
    """K_cap[L][B][Hkv][P][d] in storage dtype: the key rows of the CaP positions."""
    P = cfg.cap_rows if cap_rows is None else cap_rows
    layers = range(cfg.layers) if layers is None else layers
    out = []
    for l in layers:
        k = _normal(_gen(cfg.seed, _T_KCAP, l, cycle), (cfg.batch, cfg.Hkv, P, cfg.d))
        if cfg.recipe == "rope":
            k = _rope_rotate_half(k, np.arange(cfg.pot_size, cfg.pot_size + P))
        out.append(store(k, cfg.dtype))
    return np.stack(out, axis=0)


def make_logits(seed: int, rows: int, vocab: int, dtype: str, chunk: int = 0, ignored: float = 0.0):
    """Stand-in for a language-model head over one chunk: (logits[rows][vocab] in storage dtype,
    labels[rows] int32).  Logits ~ N(0, 2.5^2); the labels are uniform token ids; for about half of
    the rows the label's logit is raised by U(0.6, 1.6) x (log(vocab) + 3) (tokens the model predicted
    well: the log-sum-exp of the other logits is about log(vocab) + 3), so novelty spans near 0 to
    above log(vocab).  A fraction ``ignored`` of the labels is -100 (padding)."""
    g = _gen(seed, _T_LOGIT, 0, chunk)
    z = g.standard_normal((rows, vocab), dtype=np.float32) * np.float32(2.5)
    labels = g.integers(0, vocab, rows).astype(np.int32)
    boost = np.where(g.random(rows) < 0.5, (0.6 + g.random(rows)) * (np.log(vocab) + 3.0), 0.0).astype(np.float32)
    z[np.arange(rows), labels] += boost
    if ignored > 0:
        labels = np.where(g.random(rows) < ignored, np.int32(-100), labels).astype(np.int32)
    return store(z, dtype), labels


def _outlier_scale(cfg: CcdConfig, layer: int) -> np.ndarray:
    """Per (kv-head, channel) scale: x8 with probability 0.01, fixed for the stream."""
    g = _gen(cfg.seed, _T_MISC, layer, 0, 1)
    return np.where(g.random((cfg.Hkv, cfg.d)) < 0.01, 8.0, 1.0).astype(np.float32)


def _dup_plan(cfg: CcdConfig, n: int):
    """For the duplicated-token recipe: per stream, (dst slots ascending, src slots)."""
    plans = []
    for b in range(cfg.batch):
        g = _gen(cfg.seed, _T_MISC, 0, b, 2)
        cnt = (n * 5) // 100
        dst = np.sort(g.choice(np.arange(1, n), size=cnt, replace=False))
        src = (g.random(cnt) * dst).astype(np.int64)  # uniform in [0, dst)
        plans.append((dst, src))
    return plans


def make_kv(cfg: CcdConfig, n: int | None = None, chunk: int = 0, layers=None):
    """K, V[L][B][Hkv][n][d] in storage dtype for one chunk (or one full pot).

    ``chunk`` selects the chunk of a stream; for the single-shot recipes it is 0
    and ``n`` defaults to ``pot_size``.
    """
    if n is None:
        n = cfg.chunk if cfg.recipe == "stream" else cfg.pot_size
    layers = range(cfg.layers) if layers is None else layers
    shape = (cfg.batch, cfg.Hkv, n, cfg.d)
    Ks, Vs = [], []
    dup = _dup_plan(cfg, n) if cfg.recipe == "student_dup" else None
    for l in layers:
        k = _normal(_gen(cfg.seed, _T_K, l, chunk), shape)
        v = _normal(_gen(cfg.seed, _T_V, l, chunk), shape)
        if cfg.recipe == "rope":
            k = _rope_rotate_half(k, np.arange(n))
        elif cfg.recipe == "stream":
            k = k * _outlier_scale(cfg, l)[None, :, None, :]
        elif cfg.recipe == "lognorm":
            z = _normal(_gen(cfg.seed, _T_MISC, l, 0, 3), (cfg.batch, cfg.Hkv))
            k = k * np.exp(0.5 * z)[:, :, None, None].astype(np.float32)
        elif cfg.recipe == "student_dup":
            g = _gen(cfg.seed, _T_MISC, l, chunk, 4)
            chi = g.chisquare(3.0, size=shape).astype(np.float32)
            k = k / np.sqrt(chi / 3.0)
            for b, (dst, src) in enumerate(dup):
                for t, s in zip(dst, src):  # ascending: a source may itself be a copy
                    k[b, :, t, :] = k[b, :, s, :]
                    v[b, :, t, :] = v[b, :, s, :]
        Ks.append(store(k, cfg.dtype))
        Vs.append(store(v, cfg.dtype))
    return np.stack(Ks, axis=0), np.stack(Vs, axis=0)


def make_cycle(cfg: CcdConfig, cycle: int = 0, layers=None):
    """One full pot plus the CaP queries and novelty scores for a single cycle."""
    K, V = make_kv(cfg, cfg.pot_size, chunk=cycle, layers=layers)
    Q = make_q(cfg, cycle, layers=layers)
    aux = make_aux(cfg, cycle)
    return {"K": K, "V": V, "Q": Q, "aux": aux}


def small_config(**kw) -> CcdConfig:
    """A free-form small configuration for randomised parity cases."""
    base = dict(cfg_id=100, name="small", layers=1, batch=1, Hq=4, Hkv=2, d=64, pot_size=96,
                cap_rows=5, keep=40, nuc_slots=20, dtype="f32", recipe="normal")
    base.update(kw)
    return CcdConfig(**base)
