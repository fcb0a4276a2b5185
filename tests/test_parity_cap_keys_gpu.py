"""GPU parity of the CaP-inclusive scoring variant (the PyTorch-style listing of
Appendix B read literally: the CaP's own keys join every row's softmax under the
causal mask and their columns are cut away) against the CPU checker, through the
C ABI.  Tolerances as in tests/parity.py."""
import numpy as np
import pytest

import oracle
from paper_2410_01518_b200 import inputs, ipot
from parity import compare_cycle, from_dev_bits, gpu_cycle, make_pot, to_dev

pytestmark = pytest.mark.gpu

SCORERS = [ipot.IPOT_SCORER_SIMT, ipot.IPOT_SCORER_TENSOR, ipot.IPOT_SCORER_WARP_MMA]


def with_cap_keys(cfg, cycle=0, scale=1.0):
    t = inputs.make_cycle(cfg, cycle)
    kc = inputs.make_kcap(cfg, cycle)
    if scale != 1.0:
        kc = inputs.store((inputs.widen(kc, cfg.dtype) * scale).astype(np.float32), cfg.dtype)
    t["K_cap"] = kc
    return t


def test_config1_tiny_f32_with_cap_keys():
    cfg = inputs.CONFIGS[1]
    t = with_cap_keys(cfg)
    gpu = gpu_cycle(cfg, t, ipot.IPOT_SCORER_SIMT)
    same, n = compare_cycle(cfg, t, gpu)
    assert n == cfg.units and same == n
    M = cfg.G * cfg.cap_rows
    assert (gpu[0].sum(axis=1) < M - 1e-3).all()   # the CaP columns took part of every row


@pytest.mark.parametrize("scorer", SCORERS)
def test_config2_mistral_layer_with_cap_keys(scorer):
    cfg = inputs.CONFIGS[2]
    t = with_cap_keys(cfg)
    gpu = gpu_cycle(cfg, t, scorer)
    same, n = compare_cycle(cfg, t, gpu)
    assert n == cfg.units and same >= n - 1


SHAPES = [
    # CaP lengths that do not divide the row tiles, rows of one head split over two row blocks, G = 1, P = 1
    dict(pot_size=96, keep=40, nuc_slots=20, cap_rows=5, Hq=6, Hkv=2, d=64, dtype="f32"),
    dict(pot_size=333, keep=100, nuc_slots=37, cap_rows=7, Hq=6, Hkv=2, d=64, dtype="bf16"),
    dict(pot_size=700, keep=300, nuc_slots=100, cap_rows=48, Hq=4, Hkv=1, d=128, dtype="bf16"),            # M = 192
    dict(pot_size=1025, keep=512, nuc_slots=0, cap_rows=33, Hq=8, Hkv=2, d=128, dtype="bf16", layers=2),   # M = 132
    dict(pot_size=2048, keep=1024, nuc_slots=512, cap_rows=64, Hq=8, Hkv=1, d=128, dtype="bf16", batch=2),  # M = 512
    dict(pot_size=300, keep=150, nuc_slots=75, cap_rows=1, Hq=2, Hkv=1, d=128, dtype="bf16"),              # one CaP row
    dict(pot_size=130, keep=65, nuc_slots=0, cap_rows=70, Hq=3, Hkv=3, d=40, dtype="f32"),                 # more CaP keys than a key tile
]


@pytest.mark.parametrize("case", range(len(SHAPES)))
@pytest.mark.parametrize("scorer", SCORERS)
def test_shapes_with_cap_keys(case, scorer):
    cfg = inputs.small_config(cfg_id=500 + case, **SHAPES[case])
    if scorer == ipot.IPOT_SCORER_TENSOR and not (cfg.dtype == "bf16" and cfg.d in (64, 128)):
        pytest.skip("the tensor scorer takes bf16 with d = 128 or 64")
    if scorer == ipot.IPOT_SCORER_WARP_MMA and not (cfg.dtype == "bf16" and cfg.d % 16 == 0):
        pytest.skip("the warp-level tensor-core scorer takes bf16 with d a multiple of 16")
    t = with_cap_keys(cfg)
    gpu = gpu_cycle(cfg, t, scorer)
    same, n = compare_cycle(cfg, t, gpu)
    assert n == cfg.units and same >= n - 1


def test_dominant_cap_keys_leave_almost_nothing_to_the_pot():
    """CaP keys with 6x the norm take nearly all of the mass: scores far below 1 still agree to 1e-3."""
    cfg = inputs.small_config(cfg_id=520, pot_size=600, keep=200, nuc_slots=50, cap_rows=16, Hq=8, Hkv=2, d=128,
                              dtype="bf16")
    t = with_cap_keys(cfg, scale=6.0)
    for scorer in SCORERS:
        gpu = gpu_cycle(cfg, t, scorer)
        same, n = compare_cycle(cfg, t, gpu)
        assert same >= n - 1
        assert gpu[0].sum(axis=1).max() < 0.9 * cfg.G * cfg.cap_rows


def test_config3_full_size_with_cap_keys_sampled_units():
    """All 32 layers in one call; the checker follows 8 sampled units."""
    cfg = inputs.CONFIGS[3]
    K0, V0 = inputs.make_kv(cfg, 2048, chunk=0)
    K1, V1 = inputs.make_kv(cfg, 2048, chunk=1)
    t = {"K": np.concatenate([K0, K1], axis=3), "V": np.concatenate([V0, V1], axis=3),
         "Q": inputs.make_q(cfg, 1), "aux": inputs.make_aux(cfg, 1), "K_cap": inputs.make_kcap(cfg, 1)}
    gpu = gpu_cycle(cfg, t, ipot.IPOT_SCORER_AUTO)
    units = np.linspace(0, cfg.units - 1, 8).astype(np.int32)
    same, cnt = compare_cycle(cfg, t, gpu, units=units)
    assert cnt == 8 and same >= 7
    u, idx = gpu[0], gpu[1]
    assert (u.sum(axis=1) < cfg.G * cfg.cap_rows).all()
    assert (np.diff(idx, axis=1) > 0).all() and idx.min() >= 0 and idx.max() < cfg.pot_size


def test_score_only_cap_and_argument_errors():
    cfg = inputs.small_config(cfg_id=521, pot_size=400, keep=100, nuc_slots=50, cap_rows=8, Hq=8, Hkv=2, d=128,
                              dtype="bf16")
    t = with_cap_keys(cfg)
    h = make_pot(cfg)
    try:
        Kd, Vd, Qd, Kc = (to_dev(t[k], "bf16") for k in ("K", "V", "Q", "K_cap"))
        ipot.ipot_append_chunk(h, Kd, Vd, 400)
        L = ipot.lib()
        assert L.ipot_score_only_cap(h, Qd.data_ptr(), None, 8, None) == ipot.IPOT_E_INVALID
        assert L.ipot_score_and_compress_cap(h, Qd.data_ptr(), None, 8, None) == ipot.IPOT_E_INVALID
        assert L.ipot_score_only_cap(h, Qd.data_ptr(), Kc.data_ptr() + 2, 8, None) == ipot.IPOT_E_INVALID
        assert L.ipot_score_only_cap(h, Qd.data_ptr(), Kc.data_ptr(), 9, None) == ipot.IPOT_E_INVALID
        ipot.ipot_score_only_cap(h, Qd, Kc, 8)
        assert ipot.ipot_sync_status(h) == 0
        sp, nb = ipot.ipot_last_scores(h)
        u = ipot.device_array(sp, (cfg.units, nb), "f32").cpu().numpy()
        Kp, Vp, ln = ipot.ipot_view(h)
        assert ln == 400 and nb == 400
        assert (from_dev_bits(ipot.device_array(Kp, (cfg.units, 400, 128), "bf16"), "bf16")
                == t["K"].reshape(cfg.units, 400, 128)).all()
        ref = oracle.cycle(t["Q"], t["K"], t["V"], t["aux"], cfg.keep, cfg.nuc_slots, with_kv=False, K_cap=t["K_cap"])
        np.testing.assert_allclose(u, ref["u"], rtol=1e-3, atol=1e-30)
        # the plain call afterwards is the context-only softmax again
        ipot.ipot_score_only(h, Qd, 8)
        assert ipot.ipot_sync_status(h) == 0
        u0 = ipot.device_array(ipot.ipot_last_scores(h)[0], (cfg.units, 400), "f32").cpu().numpy()
        assert abs(u0.sum(axis=1) - cfg.G * cfg.cap_rows).max() < 1e-2
    finally:
        ipot.ipot_destroy(h)


def test_host_buffer_call_matches_device_call():
    cfg = inputs.small_config(cfg_id=522, pot_size=512, keep=256, nuc_slots=128, cap_rows=12, Hq=8, Hkv=2, d=128,
                              dtype="bf16", layers=2)
    t = with_cap_keys(cfg)
    dev = gpu_cycle(cfg, t, ipot.IPOT_SCORER_AUTO)
    h = make_pot(cfg)
    try:
        ipot.ipot_append_chunk_host(h, t["K"], t["V"], cfg.pot_size)
        idx_host = np.full((cfg.units, cfg.keep), -1, dtype=np.int32)
        ipot.ipot_score_and_compress_cap_host(h, t["Q"], t["K_cap"], cfg.cap_rows, t["aux"], idx_host)
        assert ipot.ipot_sync_status(h) == 0
        assert (idx_host == dev[1]).all()
        Kp, _, ln = ipot.ipot_view(h)
        assert ln == cfg.keep
        got = from_dev_bits(ipot.device_array(Kp, (cfg.units, cfg.pot_size, cfg.d), "bf16")[:, :cfg.keep], "bf16")
        assert (got == dev[2]).all()
    finally:
        ipot.ipot_destroy(h)
