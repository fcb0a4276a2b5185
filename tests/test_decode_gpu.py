"""GPU parity of generation over the pot (ipot_decode_attention) against the CPU checker, through the C ABI.

Tolerance: the kernel keeps everything in fp32 (weights are never rounded to bf16), so per output element
|out_gpu - out_ref| <= 2e-4 * |out_ref| + 2e-5 (a weighted mean of O(1) values: fp32 rounding of the logits,
~4e-6, moves each weight by that much relatively) and |lse_gpu - lse_ref| <= 2e-4."""
import numpy as np
import pytest
import torch

import oracle
from paper_2410_01518_b200 import inputs, ipot
from parity import make_pot, to_dev

pytestmark = pytest.mark.gpu


def make_query(cfg, seed=0):
    g = np.random.default_rng(0xDEC0 + seed + cfg.cfg_id)
    return inputs.store(g.standard_normal((cfg.layers, cfg.batch, cfg.Hq, cfg.d), dtype=np.float32) * np.float32(1.5), cfg.dtype)


def run_decode(cfg, K, V, q, n, rope=None, with_lse=True, scorer=ipot.IPOT_SCORER_AUTO):
    h = make_pot(cfg)
    keep = []
    try:
        ipot.ipot_set_scorer(h, scorer)   # SIMT: the fp32-FMA stream; otherwise tensor cores where they apply
        if rope is not None:
            keep = [to_dev(rope[0], cfg.dtype), to_dev(rope[1], cfg.dtype)]
            ipot.ipot_enable_rope(h, keep[0], keep[1], ipot.IPOT_ROPE_INTERLEAVED if rope[2] else ipot.IPOT_ROPE_HALF)
        ipot.ipot_append_chunk(h, to_dev(K[:, :, :, :n], cfg.dtype), to_dev(V[:, :, :, :n], cfg.dtype), n)
        out = torch.full((cfg.layers, cfg.batch, cfg.Hq, cfg.d), float("nan"), device="cuda")
        lse = torch.full((cfg.layers, cfg.batch, cfg.Hq), float("nan"), device="cuda") if with_lse else None
        for _ in range(2):   # twice: the split counters must be back at zero after a call
            ipot.ipot_decode_attention(h, to_dev(q, cfg.dtype), out, lse)
        assert ipot.ipot_sync_status(h) == 0
        return out.cpu().numpy(), (lse.cpu().numpy() if with_lse else None)
    finally:
        ipot.ipot_destroy(h)


def check(out, lse, ref_out, ref_lse):
    assert np.isfinite(out).all()
    err = np.abs(out - ref_out)
    assert (err <= 2e-4 * np.abs(ref_out) + 2e-5).all(), f"worst {err.max():.3e}"
    if lse is not None:
        assert np.abs(lse - ref_lse).max() <= 2e-4


SHAPES = [
    # rows of 64 .. 512 bytes, 1 .. 8 query heads per KV head, ragged and tiny fills
    dict(pot_size=96, keep=40, Hq=4, Hkv=2, d=64, dtype="f32", n=96),
    dict(pot_size=333, keep=100, Hq=8, Hkv=2, d=128, dtype="bf16", n=333),
    dict(pot_size=1000, keep=500, Hq=2, Hkv=2, d=64, dtype="bf16", n=777, batch=2),
    dict(pot_size=700, keep=300, Hq=16, Hkv=2, d=32, dtype="bf16", n=700),
    dict(pot_size=2048, keep=1024, Hq=4, Hkv=1, d=256, dtype="bf16", n=2047, layers=2),
    dict(pot_size=512, keep=256, Hq=8, Hkv=1, d=128, dtype="f32", n=1),
    dict(pot_size=5000, keep=2500, Hq=4, Hkv=2, d=32, dtype="f32", n=4999, layers=3),
    dict(pot_size=300, keep=150, Hq=2, Hkv=1, d=128, dtype="bf16", n=65),
    dict(pot_size=3000, keep=1500, Hq=8, Hkv=1, d=64, dtype="bf16", n=2999, batch=2),      # 8 heads per KV head, 64 channels
    dict(pot_size=100, keep=50, Hq=1, Hkv=1, d=128, dtype="bf16", n=17),
]


def test_decode_three_heads_per_kv_head_needs_the_tensor_path():
    cfg = inputs.small_config(cfg_id=830, pot_size=500, keep=100, nuc_slots=0, cap_rows=1, Hq=6, Hkv=2, d=128, dtype="bf16")
    K, V = inputs.make_kv(cfg, 500)
    q = make_query(cfg)
    out, lse = run_decode(cfg, K, V, q, 500)
    check(out, lse, *oracle.decode_attention(q, K, V))


@pytest.mark.parametrize("scorer", [ipot.IPOT_SCORER_SIMT, ipot.IPOT_SCORER_AUTO])
@pytest.mark.parametrize("case", range(len(SHAPES)))
def test_decode_shapes(case, scorer):
    kw = dict(SHAPES[case])
    n = kw.pop("n")
    cfg = inputs.small_config(cfg_id=800 + case, nuc_slots=0, cap_rows=1, **kw)
    K, V = inputs.make_kv(cfg, cfg.pot_size)
    q = make_query(cfg)
    out, lse = run_decode(cfg, K, V, q, n, scorer=scorer)
    ref_out, ref_lse = oracle.decode_attention(q, K, V, n)
    check(out, lse, ref_out, ref_lse)


def test_decode_config3_full_size():
    """All 32 layers of the Mistral-7B-shaped pot in one call (the launch the benchmark times); the checker follows
    every fourth unit."""
    cfg = inputs.CONFIGS[3]
    K0, V0 = inputs.make_kv(cfg, 2048, chunk=0)
    K1, V1 = inputs.make_kv(cfg, 2048, chunk=1)
    K, V = np.concatenate([K0, K1], axis=3), np.concatenate([V0, V1], axis=3)
    q = make_query(cfg)
    out, lse = run_decode(cfg, K, V, q, 4096, with_lse=False)
    ref_out, _ = oracle.decode_attention(q[::4], K[::4], V[::4])
    check(out[::4], None, ref_out, None)


def test_decode_reads_the_rotated_keys_in_rotary_mode():
    cfg = inputs.small_config(cfg_id=820, pot_size=400, keep=100, nuc_slots=0, cap_rows=1, Hq=8, Hkv=2, d=128, dtype="bf16")
    K, V = inputs.make_kv(cfg, 400)
    q = make_query(cfg)
    cos_t, sin_t = inputs.make_rope_table(400, 128, "bf16")
    out, lse = run_decode(cfg, K, V, q, 400, rope=(cos_t, sin_t, False))
    Kr = oracle.rope_rows(K, np.arange(400), cos_t, sin_t)
    ref_out, ref_lse = oracle.decode_attention(q, Kr, V)
    check(out, lse, ref_out, ref_lse)
    plain, _ = oracle.decode_attention(q, K, V)
    assert np.abs(plain - ref_out).max() > 1e-2


def test_decode_after_a_cycle_and_argument_errors():
    cfg = inputs.small_config(cfg_id=821, pot_size=256, keep=64, nuc_slots=32, cap_rows=4, Hq=4, Hkv=2, d=64, dtype="bf16")
    t = inputs.make_cycle(cfg)
    q = make_query(cfg)
    L = ipot.lib()
    h = make_pot(cfg)
    try:
        out = torch.zeros((1, 1, 4, 64), device="cuda")
        qd = to_dev(q, "bf16")
        assert L.ipot_decode_attention(h, qd.data_ptr(), out.data_ptr(), None) == ipot.IPOT_E_STATE   # empty pot
        ipot.ipot_append_chunk(h, to_dev(t["K"], "bf16"), to_dev(t["V"], "bf16"), 256)
        ipot.ipot_score_and_compress(h, to_dev(t["Q"], "bf16"), 4, torch.from_numpy(t["aux"]).cuda())
        ipot.ipot_decode_attention(h, qd, out)
        assert ipot.ipot_sync_status(h) == 0
        ref = oracle.cycle(t["Q"], t["K"], t["V"], t["aux"], 64, 32)
        Kc = ref["K"].reshape(1, 1, 2, 64, 64)
        Vc = ref["V"].reshape(1, 1, 2, 64, 64)
        idx = ipot.device_array(ipot.ipot_last_indices(h), (cfg.units, 64), "i32").cpu().numpy()
        if (idx == ref["idx"]).all():                       # the distilled pot is what generation attends to
            check(out.cpu().numpy(), None, oracle.decode_attention(q, Kc, Vc)[0], None)
        for bad in ((None, out.data_ptr()), (qd.data_ptr(), None), (qd.data_ptr() + 2, out.data_ptr())):
            assert L.ipot_decode_attention(h, bad[0], bad[1], None) == ipot.IPOT_E_INVALID
    finally:
        ipot.ipot_destroy(h)
    odd = inputs.small_config(cfg_id=822, pot_size=64, keep=16, nuc_slots=0, Hq=6, Hkv=2, d=64, dtype="bf16")   # G = 3
    h = make_pot(odd)
    try:
        ipot.ipot_set_scorer(h, ipot.IPOT_SCORER_SIMT)      # the fp32-FMA stream takes 1, 2, 4 or 8 heads per KV head
        K, V = inputs.make_kv(odd, 64)
        ipot.ipot_append_chunk(h, to_dev(K, "bf16"), to_dev(V, "bf16"), 64)
        o = torch.zeros((1, 1, 6, 64), device="cuda")
        assert L.ipot_decode_attention(h, to_dev(make_query(odd), "bf16").data_ptr(), o.data_ptr(), None) == ipot.IPOT_E_INVALID
    finally:
        ipot.ipot_destroy(h)
