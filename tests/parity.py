"""Helpers shared by the GPU parity tests: run one cycle through the C ABI and
compare it with the CPU checker under the stated tolerances.

Tolerances (floating point decides an integer here, so index sets get a tie band):
  scores   |u_gpu - u_ref| <= 1e-3 * |u_ref| + floor,  floor = M * 2**-126
           (fp32 cannot hold smaller probabilities than 2**-126 per query row);
  indices  exactly `keep`, strictly ascending, the novelty (NuC) slots all present;
           every slot in the symmetric difference with the checker's set must have a
           checker score within 1e-3 * |beta| + floor of beta, the checker's score of
           the last CaP slot admitted;
  K, V     bit-equal to the input rows at the GPU's own indices, and bit-equal to the
           checker's compacted pot whenever the index lists coincide;
  rotated  (Sec. 3.4) the checker multiplies each channel pair by cos + i sin in float64 and rounds
  keys     once; the kernel evaluates fma(lo, cos, -(hi * sin)) in float32 and rounds to the storage
           type, so per element |gpu - exact| <= ulp_storage / 2 + 2**-23 * (|lo cos| + |hi sin|)
           (one rounded product, one float32 rounding, one storage rounding), and the two agree bit
           for bit except where the exact value lies that close to a rounding boundary: at least
           99.9 % of the elements for bf16 (a boundary every 2**-8, an error of 2**-24), at least
           70 % for float32 storage (the rounded product moves the last bit in about a quarter of
           the cases).
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2410_01518_b200 import inputs, ipot

REL = 1e-3


def to_dev(a: np.ndarray, dtype: str) -> torch.Tensor:
    if dtype == "bf16":
        return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def from_dev_bits(t: torch.Tensor, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    return t.contiguous().cpu().numpy()


def make_pot(cfg: inputs.CcdConfig, max_cap_rows=None, nuc_slots=None) -> int:
    return ipot.ipot_create_ex(cfg.pot_size, cfg.keep, cfg.layers, cfg.Hq, cfg.Hkv, cfg.d, batch=cfg.batch,
                               dtype=ipot.IPOT_F32 if cfg.dtype == "f32" else ipot.IPOT_BF16,
                               nuc_slots=cfg.nuc_slots if nuc_slots is None else nuc_slots,
                               max_cap_rows=max_cap_rows or cfg.cap_rows)


def read_results(h, cfg: inputs.CcdConfig, n_before: int):
    """Scores, indices and the compacted pot of the last cycle as numpy arrays."""
    assert ipot.ipot_sync_status(h) == 0
    units = cfg.units
    sp, nb = ipot.ipot_last_scores(h)
    assert nb == n_before
    u = ipot.device_array(sp, (units, nb), "f32").cpu().numpy()
    idx = ipot.device_array(ipot.ipot_last_indices(h), (units, cfg.keep), "i32").cpu().numpy()
    Kp, Vp, ln = ipot.ipot_view(h)
    assert ln == cfg.keep
    shape = (units, cfg.pot_size, cfg.d)
    K = from_dev_bits(ipot.device_array(Kp, shape, cfg.dtype)[:, :cfg.keep], cfg.dtype)
    V = from_dev_bits(ipot.device_array(Vp, shape, cfg.dtype)[:, :cfg.keep], cfg.dtype)
    return u, idx, K, V


def read_rotated(h, cfg: inputs.CcdConfig, rows: int) -> np.ndarray:
    """The first `rows` rows of the rotated copy of the keys, [units][rows][d] storage bits."""
    assert ipot.ipot_sync_status(h) == 0
    shape = (cfg.units, cfg.pot_size, cfg.d)
    return from_dev_bits(ipot.device_array(ipot.ipot_view_rope(h), shape, cfg.dtype)[:, :rows], cfg.dtype)


def check_rotated(got: np.ndarray, rows: np.ndarray, pos, rope, dtype: str) -> float:
    """got: rotated rows read from the GPU (storage bits), rows: the unrotated rows they were made from, both
    [..., n, d]; pos [n].  Asserts the bound above on every element and returns the fraction of bit-equal ones."""
    cos_t, sin_t, inter = rope
    ref, exact, mag = oracle.rope_rows(rows, pos, cos_t, sin_t, inter, with_exact=True)
    same = got == ref
    if not same.all():
        g = inputs.widen(got, dtype).astype(np.float64)
        big = np.maximum(np.abs(g), np.abs(exact))
        ulp = np.ldexp(1.0, np.floor(np.log2(np.maximum(big, 2.0 ** -120))).astype(np.int64) - (23 if dtype == "f32" else 7))
        bad = ~same & (np.abs(g - exact) > 0.5 * ulp * (1 + 1e-9) + 2.0 ** -23 * mag)
        assert not bad.any(), f"{int(bad.sum())} rotated elements outside the single-precision bound"
    frac = float(same.mean())
    assert frac >= (0.70 if dtype == "f32" else 0.999), f"only {frac:.4%} of the rotated elements bit-equal"
    return frac


def gpu_cycle(cfg: inputs.CcdConfig, t: dict, scorer=ipot.IPOT_SCORER_AUTO, n=None, deferred_from=None, tuning=None):
    """Fill a fresh pot with t['K'], t['V'] (first n rows), run one cycle, read everything back.
    deferred_from = s: rows [0, s) are appended the plain way, rows [s, n) as a deferred append.
    tuning: {IPOT_TUNE_*: value} launch parameters set before the cycle."""
    n = cfg.pot_size if n is None else n
    h = make_pot(cfg, max_cap_rows=t["Q"].shape[3])
    keep_alive = []
    try:
        ipot.ipot_set_scorer(h, scorer)
        for what, value in (tuning or {}).items():
            ipot.ipot_set_tuning(h, what, value)
        if t.get("rope") is not None:  # Sec. 3.4: t["K"] holds unrotated keys, the library keeps the rotated copy
            cos_t, sin_t, inter = t["rope"]
            keep_alive = [to_dev(cos_t, cfg.dtype), to_dev(sin_t, cfg.dtype)]
            ipot.ipot_enable_rope(h, keep_alive[0], keep_alive[1], ipot.IPOT_ROPE_INTERLEAVED if inter else ipot.IPOT_ROPE_HALF)
        Kd, Vd = to_dev(t["K"][:, :, :, :n], cfg.dtype), to_dev(t["V"][:, :, :, :n], cfg.dtype)
        Qd = to_dev(t["Q"], cfg.dtype)
        auxd = torch.from_numpy(np.ascontiguousarray(t["aux"][:, :n])).cuda()
        if deferred_from is None:
            ipot.ipot_append_chunk(h, Kd, Vd, n)
        else:
            s0 = deferred_from
            if s0 > 0:
                ipot.ipot_append_chunk(h, Kd[:, :, :, :s0].contiguous(), Vd[:, :, :, :s0].contiguous(), s0)
            Kd, Vd = Kd[:, :, :, s0:].contiguous(), Vd[:, :, :, s0:].contiguous()   # alive until the cycle has run
            ipot.ipot_set_deferred_append(h, True)
            ipot.ipot_append_chunk(h, Kd, Vd, n - s0)
        if t.get("K_cap") is not None:  # Appendix B listing: the CaP's own keys join the softmax
            ipot.ipot_score_and_compress_cap(h, Qd, to_dev(t["K_cap"], cfg.dtype), t["Q"].shape[3],
                                             auxd if cfg.nuc_slots > 0 else None)
        else:
            ipot.ipot_score_and_compress(h, Qd, t["Q"].shape[3], auxd if cfg.nuc_slots > 0 else None)
        res = read_results(h, cfg, n)
        if t.get("rope") is not None:
            res = res + (read_rotated(h, cfg, cfg.keep),)
        return res
    finally:
        ipot.ipot_destroy(h)


def check_unit(cfg, u_gpu, idx_gpu, K_gpu, V_gpu, K_in, V_in, ref_u, ref_idx, nuc, M, ref_K=None, ref_V=None):
    """Compare one unit.  Returns True if the index lists are identical."""
    floor = M * 2.0 ** -126
    err = np.abs(u_gpu.astype(np.float64) - ref_u)
    bad = err > REL * np.abs(ref_u) + floor
    assert not bad.any(), f"scores off: worst rel {np.max(err / (np.abs(ref_u) + floor)):.3e}"
    keep = cfg.keep
    assert idx_gpu.shape == (keep,) and (np.diff(idx_gpu) > 0).all()
    assert idx_gpu[0] >= 0 and idx_gpu[-1] < ref_u.shape[0]
    gs, rs = set(idx_gpu.tolist()), set(ref_idx.tolist())
    assert set(nuc.tolist()) <= gs, "a novelty slot was dropped"
    same = gs == rs
    if not same:
        cap = np.setdiff1d(ref_idx, nuc)
        beta = ref_u[cap].min()
        for j in gs ^ rs:
            assert abs(ref_u[j] - beta) <= REL * abs(beta) + floor, f"slot {j} differs outside the tie band"
    assert (K_gpu == K_in[idx_gpu]).all() and (V_gpu == V_in[idx_gpu]).all()
    if same and ref_K is not None:
        assert (K_gpu == ref_K).all() and (V_gpu == ref_V).all()
    return same


def compare_cycle(cfg, t, gpu, units=None, n=None):
    """gpu = (u, idx, K, V) over all units.  The checker runs on `units` (default all).
    Returns (units whose index list is identical to the checker's, units compared)."""
    n = cfg.pot_size if n is None else n
    K_in, V_in = t["K"][:, :, :, :n], t["V"][:, :, :, :n]
    ref = oracle.cycle(t["Q"], K_in, V_in, t["aux"][:, :n], cfg.keep, cfg.nuc_slots, units=units, K_cap=t.get("K_cap"),
                       rope=t.get("rope"))
    u, idx, K, V = gpu[:4]
    Kf, Vf = K_in.reshape(cfg.units, n, cfg.d), V_in.reshape(cfg.units, n, cfg.d)
    M = cfg.G * t["Q"].shape[3]
    nuc = [oracle.nuc_top(t["aux"][b, :n], cfg.nuc_slots) for b in range(cfg.batch)]
    identical = 0
    for k, unit in enumerate(ref["units"]):
        b = (unit // cfg.Hkv) % cfg.batch
        same = check_unit(cfg, u[unit], idx[unit], K[unit], V[unit], Kf[unit], Vf[unit],
                          ref["u"][k], ref["idx"][k], nuc[b], M, ref["K"][k], ref["V"][k])
        identical += same
        if t.get("rope") is not None:  # the rotated copy: the survivors rotated at their new slot numbers
            check_rotated(gpu[4][unit], Kf[unit][idx[unit]], np.arange(cfg.keep), t["rope"], cfg.dtype)
    return identical, len(ref["units"])
