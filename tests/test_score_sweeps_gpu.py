"""GPU parity of the two-sweep tensor-core scorer (IPOT_SCORER_TENSOR_SWEEPS: row log-sum-exps in a first sweep over
the keys, probabilities and their column sums in a second one, inside thread-block clusters) against the CPU
checker, through the C ABI, under the tolerances of tests/parity.py.  Eq. 2, Sec. 3.3.1."""
import numpy as np
import pytest
import torch

import oracle
from paper_2410_01518_b200 import inputs, ipot
from parity import compare_cycle, gpu_cycle, make_pot, read_results, to_dev

pytestmark = pytest.mark.gpu
SW = ipot.IPOT_SCORER_TENSOR_SWEEPS

SHAPES = [
    # (pot_size, rows used, cap_rows, Hq, Hkv, layers, batch): 1..64 slabs per unit, ragged slabs, 1-4 row blocks
    # (the last one ragged), fewer and more units than clusters, fewer slabs than CTAs of a cluster
    (512, 512, 32, 4, 1, 1, 1), (640, 513, 16, 8, 2, 2, 1), (1536, 1500, 33, 8, 2, 1, 2), (2048, 2048, 64, 8, 2, 3, 1),
    (3000, 2999, 5, 6, 2, 1, 1), (4096, 3585, 64, 12, 2, 2, 1), (300, 129, 1, 1, 1, 1, 1), (8192, 8192, 64, 8, 2, 1, 2),
    (5000, 4097, 40, 4, 1, 20, 1), (4096, 4096, 64, 8, 1, 2, 1), (16384, 16001, 64, 8, 1, 1, 2), (4096, 4096, 32, 32, 8, 21, 1),
]


@pytest.mark.parametrize("cluster", [0, 1, 2, 4, 8])
@pytest.mark.parametrize("case", range(len(SHAPES)))
def test_sweeps_shapes_and_cluster_sizes(case, cluster):
    pot, n, P, Hq, Hkv, L, B = SHAPES[case]
    if cluster not in (0, 2) and case in (8, 10, 11):
        pytest.skip("the largest shapes run with the chosen and one fixed cluster size")
    cfg = inputs.small_config(cfg_id=450 + case, pot_size=pot, keep=n // 2, nuc_slots=n // 4, cap_rows=P, Hq=Hq,
                              Hkv=Hkv, d=128, dtype="bf16", layers=L, batch=B)
    t = inputs.make_cycle(cfg)
    gpu = gpu_cycle(cfg, t, SW, n=n, tuning={ipot.IPOT_TUNE_SWEEPS_CLUSTER: cluster})
    units = None if cfg.units <= 24 else np.linspace(0, cfg.units - 1, 24).astype(np.int32)
    same, cnt = compare_cycle(cfg, t, gpu, n=n, units=units)
    assert same >= cnt - 1


@pytest.mark.parametrize("eighths", [2, 3])
def test_sweeps_fma_pipe_share_and_64_channel_heads(eighths):
    """Both shares of the exponentials that go to the FMA pipe, on d = 64 (one 64-channel half per tile) and d = 128;
    the two settings agree with each other far inside the tolerance."""
    out = []
    for d in (64, 128):
        cfg = inputs.small_config(cfg_id=470 + d, pot_size=3000, keep=1400, nuc_slots=700, cap_rows=40, Hq=8, Hkv=2, d=d,
                                  dtype="bf16", layers=3, batch=2)
        t = inputs.make_cycle(cfg)
        gpu = gpu_cycle(cfg, t, SW, n=2999, tuning={ipot.IPOT_TUNE_SWEEPS_FMA_EIGHTHS: eighths})
        same, cnt = compare_cycle(cfg, t, gpu, n=2999)
        assert cnt == cfg.units and same >= cnt - 1
        simt = gpu_cycle(cfg, t, ipot.IPOT_SCORER_SIMT, n=2999)
        np.testing.assert_allclose(gpu[0], simt[0], rtol=2e-5, atol=1e-30)
        out.append(gpu[0])
    assert len(out) == 2


def test_sweeps_heavy_tails_outliers_and_duplicates():
    """Student-t keys with exactly duplicated tokens (logits far above the row's first ones: the row reference has to
    move), outlier channels, log-normal key norms."""
    for recipe, cid, kw in (("student_dup", 5, dict(pot_size=2300, keep=600, nuc_slots=300, cap_rows=16, batch=2)),
                            ("stream", 3, dict(pot_size=900, keep=450, nuc_slots=225, cap_rows=8, batch=2, chunk=900)),
                            ("lognorm", 4, dict(pot_size=900, keep=450, nuc_slots=225, cap_rows=8, batch=2))):
        cfg = inputs.small_config(cfg_id=cid, recipe=recipe, dtype="bf16", Hq=8, Hkv=2, d=128, **kw)
        t = inputs.make_cycle(cfg)
        for cluster in (1, 4):
            compare_cycle(cfg, t, gpu_cycle(cfg, t, SW, tuning={ipot.IPOT_TUNE_SWEEPS_CLUSTER: cluster}))


def test_sweeps_keys_far_above_the_first_ones():
    """The first 32 keys of every unit are tiny, later keys are 60 times larger: a reference taken from the first
    logits is hundreds of exponent steps too low for most rows and must be moved without losing a term."""
    cfg = inputs.small_config(cfg_id=480, pot_size=1024, keep=400, nuc_slots=0, cap_rows=32, Hq=4, Hkv=1, d=128, dtype="bf16", layers=2)
    t = inputs.make_cycle(cfg)
    K = inputs.widen(t["K"], "bf16").astype(np.float32)
    K[:, :, :, :32] *= 0.01
    K[:, :, :, 300:340] *= 60.0
    t["K"] = inputs.store(K, "bf16")
    same, cnt = compare_cycle(cfg, t, gpu_cycle(cfg, t, SW))
    assert cnt == cfg.units


def test_sweeps_with_cap_keys_rope_and_deferred_append():
    """The variants that reach the scorer through other entry points: CaP keys inside the softmax (Appendix B listing),
    the rotated key copy (Sec. 3.4), and keys of a deferred append read where they lie (whole 256-key slabs)."""
    cfg = inputs.small_config(cfg_id=481, pot_size=1536, keep=700, nuc_slots=300, cap_rows=24, Hq=8, Hkv=2, d=128,
                              dtype="bf16", layers=2, batch=2)
    t = inputs.make_cycle(cfg)
    plain = gpu_cycle(cfg, t, SW)
    same, cnt = compare_cycle(cfg, t, plain)
    assert same >= cnt - 1
    for first in (0, 512, 1280, 700):          # 700: not a slab boundary, the keys are copied first
        got = gpu_cycle(cfg, t, SW, deferred_from=first)
        assert all((a == b).all() for a, b in zip(got, plain)), first
    tc = dict(t)
    tc["K_cap"] = inputs.make_kcap(cfg)
    same, cnt = compare_cycle(cfg, tc, gpu_cycle(cfg, tc, SW))
    assert same >= cnt - 1
    tr = dict(t)
    cos_t, sin_t = inputs.make_rope_table(cfg.pot_size, cfg.d, cfg.dtype)
    tr["rope"] = (cos_t, sin_t, False)
    same, cnt = compare_cycle(cfg, tr, gpu_cycle(cfg, tr, SW))
    assert same >= cnt - 1


def test_sweeps_refuses_shapes_it_does_not_take():
    for kw in (dict(d=96, dtype="bf16", cap_rows=4), dict(d=128, dtype="f32", cap_rows=4), dict(d=128, dtype="bf16", cap_rows=130)):
        cfg = inputs.small_config(cfg_id=482, pot_size=300, keep=100, nuc_slots=0, Hq=4, Hkv=1, **kw)   # 130 rows x 4 heads > 512
        t = inputs.make_cycle(cfg)
        h = make_pot(cfg)
        try:
            ipot.ipot_set_scorer(h, SW)
            ipot.ipot_append_chunk(h, to_dev(t["K"], cfg.dtype), to_dev(t["V"], cfg.dtype), cfg.pot_size)
            assert ipot.lib().ipot_score_only(h, to_dev(t["Q"], cfg.dtype).data_ptr(), cfg.cap_rows, None) == ipot.IPOT_E_INVALID
            L = ipot.lib()
            for what, bad in ((ipot.IPOT_TUNE_SWEEPS_CLUSTER, 3), (ipot.IPOT_TUNE_SWEEPS_FMA_EIGHTHS, 5),
                              (ipot.IPOT_TUNE_WAIT_LIMIT_NS, 10), (ipot.IPOT_TUNE_TEST_WITHHOLD_RANK, 8), (99, 0)):
                assert L.ipot_set_tuning(h, what, bad) == ipot.IPOT_E_INVALID
        finally:
            ipot.ipot_destroy(h)


@pytest.mark.parametrize("scorer", [SW, ipot.IPOT_SCORER_TENSOR])
def test_a_wait_that_runs_out_ends_the_launch_with_a_status_and_the_pot_recovers(scorer):
    """One CTA (of every cluster, or of the one-sweep kernel's grid) never reports its statistics (a test hook: nothing
    is damaged, the others' wait for them simply cannot end) and the wait limit is 2 ms: the launch must end by
    itself, the status word must say IPOT_E_TIMEOUT, and after ipot_reset the same pot must run a correct cycle with
    the hook off."""
    cfg = inputs.small_config(cfg_id=483, pot_size=1024, keep=400, nuc_slots=100, cap_rows=16, Hq=8, Hkv=2, d=128,
                              dtype="bf16", layers=2)
    t = inputs.make_cycle(cfg)
    h = make_pot(cfg)
    try:
        ipot.ipot_set_scorer(h, scorer)
        ipot.ipot_set_tuning(h, ipot.IPOT_TUNE_SWEEPS_CLUSTER, 2)
        ipot.ipot_set_tuning(h, ipot.IPOT_TUNE_WAIT_LIMIT_NS, 2_000_000)
        ipot.ipot_set_tuning(h, ipot.IPOT_TUNE_TEST_WITHHOLD_RANK, 1)
        Kd, Vd, Qd = to_dev(t["K"], "bf16"), to_dev(t["V"], "bf16"), to_dev(t["Q"], "bf16")
        ipot.ipot_append_chunk(h, Kd, Vd, cfg.pot_size)
        ipot.ipot_score_only(h, Qd, cfg.cap_rows)
        assert ipot.ipot_sync_status(h) == ipot.IPOT_E_TIMEOUT
        ipot.ipot_reset(h)
        ipot.ipot_set_tuning(h, ipot.IPOT_TUNE_TEST_WITHHOLD_RANK, -1)
        ipot.ipot_set_tuning(h, ipot.IPOT_TUNE_WAIT_LIMIT_NS, 200_000_000)
        ipot.ipot_append_chunk(h, Kd, Vd, cfg.pot_size)
        ipot.ipot_score_and_compress(h, Qd, cfg.cap_rows, torch.from_numpy(t["aux"]).cuda())
        # the status word is sticky: read the results without the status assertion of read_results
        torch.cuda.synchronize()
        sp, nb = ipot.ipot_last_scores(h)
        u = ipot.device_array(sp, (cfg.units, nb), "f32").cpu().numpy()
        idx = ipot.device_array(ipot.ipot_last_indices(h), (cfg.units, cfg.keep), "i32").cpu().numpy()
        ref = oracle.cycle(t["Q"], t["K"], t["V"], t["aux"], cfg.keep, cfg.nuc_slots)
        M = cfg.G * cfg.cap_rows
        assert (np.abs(u - ref["u"]) <= 1e-3 * np.abs(ref["u"]) + M * 2.0 ** -126).all()
        assert sum((idx[i] == ref["idx"][i]).all() for i in range(cfg.units)) >= cfg.units - 1
    finally:
        ipot.ipot_destroy(h)


@pytest.mark.parametrize("cfg_id", [4, 5])
def test_sweeps_configs_4_and_5_full_size(cfg_id):
    """The Llama-3-8B-shaped batch (two row blocks) and the 70B-shaped layer (four row blocks, which the automatic
    choice gives to this kernel): whole configuration on the GPU, the checker follows 16 units."""
    cfg = inputs.CONFIGS[cfg_id]
    t = inputs.make_cycle(cfg)
    gpu = gpu_cycle(cfg, t, SW)
    units = np.linspace(0, cfg.units - 1, 16).astype(np.int32)
    same, cnt = compare_cycle(cfg, t, gpu, units=units)
    assert cnt == 16 and same >= 14
    M = cfg.G * cfg.cap_rows
    assert np.abs(gpu[0].sum(axis=1) - M).max() < 1e-4 * M
