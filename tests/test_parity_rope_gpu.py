"""GPU parity of the context-reset rotary mode (Sec. 3.4): unrotated keys in the pot, a rotated copy kept by the
row movers, scores from the rotated copy - against the CPU checker, through the C ABI.  The checker rotates in
float64 and rounds once; the rotated rows must lie within the error bound of the kernel's single-precision
evaluation and be bit-equal almost everywhere (tests/parity.py states both numbers); scores and index lists
under the tolerances of tests/parity.py."""
import numpy as np
import pytest
import torch

import oracle
from paper_2410_01518_b200 import inputs, ipot
from parity import check_rotated, compare_cycle, from_dev_bits, gpu_cycle, make_pot, read_results, read_rotated, to_dev

pytestmark = pytest.mark.gpu

SCORERS = [ipot.IPOT_SCORER_SIMT, ipot.IPOT_SCORER_TENSOR]


def with_rope(cfg, inter=False, cycle=0):
    t = inputs.make_cycle(cfg, cycle)
    cos_t, sin_t = inputs.make_rope_table(cfg.pot_size, cfg.d, cfg.dtype)
    t["rope"] = (cos_t, sin_t, inter)
    return t


SHAPES = [
    dict(pot_size=96, keep=40, nuc_slots=20, cap_rows=5, Hq=4, Hkv=2, d=64, dtype="f32"),
    dict(pot_size=333, keep=100, nuc_slots=37, cap_rows=7, Hq=6, Hkv=2, d=64, dtype="bf16"),
    dict(pot_size=200, keep=199, nuc_slots=1, cap_rows=3, Hq=2, Hkv=2, d=32, dtype="bf16"),     # one row dropped
    dict(pot_size=130, keep=1, nuc_slots=0, cap_rows=2, Hq=2, Hkv=1, d=32, dtype="f32"),        # one survivor
    dict(pot_size=700, keep=300, nuc_slots=100, cap_rows=16, Hq=8, Hkv=2, d=128, dtype="bf16", layers=2),
    dict(pot_size=512, keep=256, nuc_slots=128, cap_rows=8, Hq=4, Hkv=1, d=256, dtype="bf16", batch=2),
    dict(pot_size=300, keep=150, nuc_slots=75, cap_rows=4, Hq=2, Hkv=2, d=48, dtype="f32", batch=2),
]


@pytest.mark.parametrize("inter", [False, True])
@pytest.mark.parametrize("case", range(len(SHAPES)))
def test_rope_shapes(case, inter):
    cfg = inputs.small_config(cfg_id=700 + case, **SHAPES[case])
    t = with_rope(cfg, inter)
    gpu = gpu_cycle(cfg, t, ipot.IPOT_SCORER_AUTO)
    same, n = compare_cycle(cfg, t, gpu)
    assert n == cfg.units and same >= n - 1


@pytest.mark.parametrize("scorer", SCORERS)
def test_config2_mistral_layer_with_rope(scorer):
    cfg = inputs.CONFIGS[2].with_layers(1)
    cfg = inputs.small_config(**{**cfg.__dict__, "recipe": "normal", "cfg_id": 720})   # unrotated keys: no rope in the recipe
    t = with_rope(cfg)
    gpu = gpu_cycle(cfg, t, scorer)
    same, n = compare_cycle(cfg, t, gpu)
    assert n == cfg.units and same >= n - 1


def test_config3_full_size_with_rope_sampled_units():
    """All 32 layers in one call; the checker follows 8 sampled units, the rotated copy is checked on those."""
    cfg = inputs.CONFIGS[3]
    K0, V0 = inputs.make_kv(cfg, 2048, chunk=0)
    K1, V1 = inputs.make_kv(cfg, 2048, chunk=1)
    cos_t, sin_t = inputs.make_rope_table(cfg.pot_size, cfg.d, cfg.dtype)
    t = {"K": np.concatenate([K0, K1], axis=3), "V": np.concatenate([V0, V1], axis=3),
         "Q": inputs.make_q(cfg, 1), "aux": inputs.make_aux(cfg, 1), "rope": (cos_t, sin_t, False)}
    gpu = gpu_cycle(cfg, t, ipot.IPOT_SCORER_AUTO)
    units = np.linspace(0, cfg.units - 1, 8).astype(np.int32)
    same, cnt = compare_cycle(cfg, t, gpu, units=units)
    assert cnt == 8 and same >= 7


def test_stream_of_cycles_keeps_the_rotated_copy_current():
    """Three cycles with appends in between (device and host-buffer calls): after every step the rotated copy equals
    the unrotated pot rotated at the slot numbers, and every cycle agrees with the checker run on the pot's bytes."""
    cfg = inputs.small_config(cfg_id=730, pot_size=384, keep=128, nuc_slots=64, cap_rows=6, Hq=4, Hkv=2, d=64,
                              dtype="bf16", layers=2, batch=2)
    cos_t, sin_t = inputs.make_rope_table(cfg.pot_size, cfg.d, cfg.dtype)
    h = make_pot(cfg)
    tables = [to_dev(cos_t, "bf16"), to_dev(sin_t, "bf16")]
    shape = (cfg.units, cfg.pot_size, cfg.d)
    try:
        ipot.ipot_enable_rope(h, tables[0], tables[1], ipot.IPOT_ROPE_HALF)
        filled = 0
        for step in range(3):
            n_new = cfg.pot_size - filled
            Kn, Vn = inputs.make_kv(cfg, n_new, chunk=step)
            if step == 1:
                ipot.ipot_append_chunk_host(h, Kn, Vn, n_new)
            else:
                ipot.ipot_append_chunk(h, to_dev(Kn, "bf16"), to_dev(Vn, "bf16"), n_new)
            Kp, Vp, ln = ipot.ipot_view(h)
            assert ln == cfg.pot_size
            pot_k = from_dev_bits(ipot.device_array(Kp, shape, "bf16"), "bf16")
            pot_v = from_dev_bits(ipot.device_array(Vp, shape, "bf16"), "bf16")
            assert (pot_k[:, filled:] == Kn.reshape(cfg.units, n_new, cfg.d)).all()
            rot = read_rotated(h, cfg, cfg.pot_size)
            check_rotated(rot, pot_k, np.arange(cfg.pot_size), (cos_t, sin_t, False), "bf16")
            t = {"K": pot_k.reshape(cfg.layers, cfg.batch, cfg.Hkv, cfg.pot_size, cfg.d),
                 "V": pot_v.reshape(cfg.layers, cfg.batch, cfg.Hkv, cfg.pot_size, cfg.d),
                 "Q": inputs.make_q(cfg, step), "aux": inputs.make_aux(cfg, step), "rope": (cos_t, sin_t, False)}
            ipot.ipot_score_and_compress(h, to_dev(t["Q"], "bf16"), cfg.cap_rows, torch.from_numpy(t["aux"]).cuda())
            gpu = read_results(h, cfg, cfg.pot_size) + (read_rotated(h, cfg, cfg.keep),)
            same, n = compare_cycle(cfg, t, gpu)
            assert same >= n - 1
            filled = cfg.keep
    finally:
        ipot.ipot_destroy(h)


def test_enable_rope_argument_and_state_errors():
    cfg = inputs.small_config(cfg_id=731, pot_size=64, keep=16, nuc_slots=8, d=40, dtype="bf16")   # 80-byte rows
    cos_t, sin_t = inputs.make_rope_table(64, 64, "bf16")
    c, s = to_dev(cos_t, "bf16"), to_dev(sin_t, "bf16")
    L = ipot.lib()
    h = make_pot(cfg)
    try:
        assert L.ipot_enable_rope(h, c.data_ptr(), s.data_ptr(), ipot.IPOT_ROPE_HALF) == ipot.IPOT_E_INVALID   # row not 2 x 16k bytes
        assert L.ipot_view_rope(h, None) == ipot.IPOT_E_INVALID
    finally:
        ipot.ipot_destroy(h)
    cfg = inputs.small_config(cfg_id=732, pot_size=64, keep=16, nuc_slots=8, d=64, dtype="bf16")
    h = make_pot(cfg)
    try:
        import ctypes
        out = ctypes.c_void_p()
        assert L.ipot_view_rope(h, ctypes.byref(out)) == ipot.IPOT_E_STATE                        # mode is off
        for bad in ((None, s.data_ptr(), 1), (c.data_ptr(), None, 1), (c.data_ptr() + 2, s.data_ptr(), 1),
                    (c.data_ptr(), s.data_ptr(), 0), (c.data_ptr(), s.data_ptr(), 3)):
            assert L.ipot_enable_rope(h, *bad) == ipot.IPOT_E_INVALID
        K, V = inputs.make_kv(cfg, 32)
        ipot.ipot_append_chunk(h, to_dev(K, "bf16"), to_dev(V, "bf16"), 32)
        assert L.ipot_enable_rope(h, c.data_ptr(), s.data_ptr(), 1) == ipot.IPOT_E_STATE          # the pot is not empty
        ipot.ipot_reset(h)
        ipot.ipot_enable_rope(h, c, s, ipot.IPOT_ROPE_INTERLEAVED)
        ipot.ipot_append_chunk(h, to_dev(K, "bf16"), to_dev(V, "bf16"), 32)
        rot = read_rotated(h, cfg, 32)
        check_rotated(rot, K.reshape(cfg.units, 32, 64), np.arange(32), (cos_t, sin_t, True), "bf16")
    finally:
        ipot.ipot_destroy(h)
