"""GPU tests of the deferred append (ipot_set_deferred_append): the newest chunk stays
in the caller's buffers, the tensor-core scorer reads its keys there and the
compaction (Appendix B, "KV-cache compression") fetches the survivors from there.
The pot after the cycle must be the one the CPU checker computes, and bit for bit
the one the plain append gives, through the C ABI."""
import numpy as np
import pytest
import torch

from paper_2410_01518_b200 import inputs, ipot
from parity import compare_cycle, from_dev_bits, gpu_cycle, make_pot, to_dev

pytestmark = pytest.mark.gpu

CASES = [
    # (shape, scorers, fills before the deferred chunk)
    (dict(pot_size=1024, keep=512, nuc_slots=256, cap_rows=32, Hq=8, Hkv=2, d=128, dtype="bf16"),
     [ipot.IPOT_SCORER_TENSOR, ipot.IPOT_SCORER_WARP_MMA, ipot.IPOT_SCORER_SIMT], [0, 256, 512, 300, 1023]),
    (dict(pot_size=1500, keep=700, nuc_slots=100, cap_rows=16, Hq=4, Hkv=2, d=64, dtype="bf16", layers=2),
     [ipot.IPOT_SCORER_TENSOR], [0, 768, 700]),                       # ragged last slab inside the chunk
    (dict(pot_size=333, keep=100, nuc_slots=37, cap_rows=7, Hq=6, Hkv=2, d=64, dtype="f32"),
     [ipot.IPOT_SCORER_SIMT], [0, 100, 256]),                         # fp32: the keys are always copied first
    (dict(pot_size=2048, keep=1024, nuc_slots=512, cap_rows=64, Hq=8, Hkv=1, d=128, dtype="bf16", batch=2),
     [ipot.IPOT_SCORER_AUTO], [1024]),                                # M = 512: four row blocks
]


def identical(a, b):
    return all((x == y).all() for x, y in zip(a, b))


@pytest.mark.parametrize("case", range(len(CASES)))
def test_deferred_chunk_gives_the_checkers_pot(case):
    shape, scorers, fills = CASES[case]
    cfg = inputs.small_config(cfg_id=700 + case, **shape)
    t = inputs.make_cycle(cfg)
    for scorer in scorers:
        plain = gpu_cycle(cfg, t, scorer)
        for s0 in fills:
            got = gpu_cycle(cfg, t, scorer, deferred_from=s0)
            same, n = compare_cycle(cfg, t, got)
            assert n == cfg.units and same >= n - 1, (scorer, s0)
            assert identical(got, plain), (scorer, s0)   # same arithmetic in the same order: same bits


def test_deferred_with_cap_keys_and_with_rotary_mode():
    cfg = inputs.small_config(cfg_id=710, pot_size=1024, keep=512, nuc_slots=128, cap_rows=16, Hq=8, Hkv=2, d=128,
                              dtype="bf16")
    t = inputs.make_cycle(cfg)
    t["K_cap"] = inputs.make_kcap(cfg, 0)
    plain = gpu_cycle(cfg, t)
    for s0 in (0, 512, 700):
        got = gpu_cycle(cfg, t, deferred_from=s0)
        same, n = compare_cycle(cfg, t, got)
        assert same >= n - 1 and identical(got, plain)
    cfg = inputs.small_config(cfg_id=711, recipe="rope", pot_size=1024, keep=512, nuc_slots=256, cap_rows=32, Hq=8,
                              Hkv=2, d=128, dtype="bf16")
    t = inputs.make_cycle(cfg)
    plain = gpu_cycle(cfg, t)
    for s0 in (0, 512, 333):
        got = gpu_cycle(cfg, t, deferred_from=s0)      # values deferred, keys written (rotated copy) at append
        same, n = compare_cycle(cfg, t, got)
        assert same >= n - 1 and identical(got, plain)


def test_calls_between_append_and_cycle_see_the_rows():
    """ipot_view, a further append and ipot_sync_status put the deferred rows into the pot; after
    ipot_sync_status the chunk buffers may be overwritten."""
    cfg = inputs.small_config(cfg_id=712, pot_size=1024, keep=512, nuc_slots=256, cap_rows=8, Hq=8, Hkv=2, d=128,
                              dtype="bf16")
    t = inputs.make_cycle(cfg)
    plain = gpu_cycle(cfg, t)
    Kall, Vall = t["K"].reshape(cfg.units, cfg.pot_size, cfg.d), t["V"].reshape(cfg.units, cfg.pot_size, cfg.d)
    h = make_pot(cfg)
    try:
        ipot.ipot_set_deferred_append(h, True)
        parts = [(0, 256), (256, 600), (600, 1024)]
        bufs = []
        for a, b in parts:   # the second and third append copy the chunk before them
            Kd, Vd = to_dev(t["K"][:, :, :, a:b], "bf16"), to_dev(t["V"][:, :, :, a:b], "bf16")
            bufs.append((Kd, Vd))
            ipot.ipot_append_chunk(h, Kd, Vd, b - a)
        Kp, Vp, ln = ipot.ipot_view(h)               # copies the last chunk
        assert ln == 1024 and ipot.ipot_sync_status(h) == 0
        shape = (cfg.units, cfg.pot_size, cfg.d)
        assert (from_dev_bits(ipot.device_array(Kp, shape, "bf16"), "bf16") == Kall).all()
        assert (from_dev_bits(ipot.device_array(Vp, shape, "bf16"), "bf16") == Vall).all()
        ipot.ipot_reset(h)
        Kd, Vd = to_dev(t["K"], "bf16"), to_dev(t["V"], "bf16")
        ipot.ipot_append_chunk(h, Kd, Vd, 1024)
        assert ipot.ipot_sync_status(h) == 0         # from here on the library needs the buffers no more
        Kd.zero_()
        Vd.zero_()
        torch.cuda.synchronize()
        Qd = to_dev(t["Q"], "bf16")
        auxd = torch.from_numpy(np.ascontiguousarray(t["aux"])).cuda()
        ipot.ipot_score_and_compress(h, Qd, cfg.cap_rows, auxd)
        assert ipot.ipot_sync_status(h) == 0
        idx = ipot.device_array(ipot.ipot_last_indices(h), (cfg.units, cfg.keep), "i32").cpu().numpy()
        Kp, Vp, ln = ipot.ipot_view(h)
        assert ln == cfg.keep and (idx == plain[1]).all()
        assert (from_dev_bits(ipot.device_array(Kp, shape, "bf16")[:, :cfg.keep], "bf16") == plain[2]).all()
        assert (from_dev_bits(ipot.device_array(Vp, shape, "bf16")[:, :cfg.keep], "bf16") == plain[3]).all()
    finally:
        ipot.ipot_destroy(h)


def test_stream_of_cycles_matches_the_plain_append_and_decode_sees_deferred_rows():
    """Four chunks, a cycle after each: the pots of a deferred and a plain run stay bit-identical, and so does
    generation over a pot whose newest rows are still deferred."""
    cfg = inputs.small_config(cfg_id=713, pot_size=1024, keep=512, nuc_slots=256, cap_rows=16, Hq=8, Hkv=2, d=128,
                              dtype="bf16", layers=2)
    pots = [make_pot(cfg), make_pot(cfg)]
    try:
        ipot.ipot_set_deferred_append(pots[1], True)
        shape = (cfg.units, cfg.pot_size, cfg.d)
        keep_alive = []
        for step in range(4):
            n_new = cfg.pot_size if step == 0 else cfg.pot_size - cfg.keep
            K, V = inputs.make_kv(cfg, n_new, chunk=step)
            Kd, Vd = to_dev(K, "bf16"), to_dev(V, "bf16")
            Qd = to_dev(inputs.make_q(cfg, step), "bf16")
            auxd = torch.from_numpy(np.ascontiguousarray(inputs.make_aux(cfg, step))).cuda()
            qd = to_dev(np.ascontiguousarray(inputs.make_q(cfg, 100 + step)[:, :, :, 0]), "bf16")   # [L][B][Hq][d]
            keep_alive.append((Kd, Vd, Qd, auxd, qd))
            outs = []
            for h in pots:
                ipot.ipot_append_chunk(h, Kd, Vd, n_new)
                out = torch.zeros((cfg.layers, cfg.batch, cfg.Hq, cfg.d), dtype=torch.float32, device="cuda")
                lse = torch.zeros((cfg.layers, cfg.batch, cfg.Hq), dtype=torch.float32, device="cuda")
                if step == 2:
                    ipot.ipot_decode_attention(h, qd, out, lse)
                ipot.ipot_score_and_compress(h, Qd, cfg.cap_rows, auxd)
                assert ipot.ipot_sync_status(h) == 0
                Kp, Vp, ln = ipot.ipot_view(h)
                assert ln == cfg.keep
                outs.append((ipot.device_array(ipot.ipot_last_indices(h), (cfg.units, cfg.keep), "i32").cpu().numpy(),
                             from_dev_bits(ipot.device_array(Kp, shape, "bf16")[:, :cfg.keep], "bf16"),
                             from_dev_bits(ipot.device_array(Vp, shape, "bf16")[:, :cfg.keep], "bf16"),
                             out.cpu().numpy() if step == 2 else np.zeros(1), lse.cpu().numpy() if step == 2 else np.zeros(1)))
            assert identical(outs[0], outs[1]), step
    finally:
        for h in pots:
            ipot.ipot_destroy(h)


def test_full_size_stream_deferred_sampled_units():
    """The 32-layer configuration as the bench runs it (pot 4096 = 2048 kept + 2048 deferred)."""
    cfg = inputs.CONFIGS[3]
    K0, V0 = inputs.make_kv(cfg, 2048, chunk=0)
    K1, V1 = inputs.make_kv(cfg, 2048, chunk=1)
    t = {"K": np.concatenate([K0, K1], axis=3), "V": np.concatenate([V0, V1], axis=3),
         "Q": inputs.make_q(cfg, 1), "aux": inputs.make_aux(cfg, 1)}
    got = gpu_cycle(cfg, t, ipot.IPOT_SCORER_AUTO, deferred_from=2048)
    units = np.linspace(0, cfg.units - 1, 6).astype(np.int32)
    same, cnt = compare_cycle(cfg, t, got, units=units)
    assert cnt == 6 and same >= 5
    plain = gpu_cycle(cfg, t, ipot.IPOT_SCORER_AUTO)
    assert identical(got, plain)
