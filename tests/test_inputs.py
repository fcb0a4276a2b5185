"""The synthetic input generators: determinism, formats, recipe structure."""
import numpy as np
import pytest

from paper_2410_01518_b200 import inputs


def test_bf16_rounding_matches_library_conversion():
    torch = pytest.importorskip("torch")
    g = np.random.default_rng(0)
    x = np.concatenate([g.standard_normal(10000).astype(np.float32) * 10,
                        np.array([1.00390625, 1.01171875, -0.0, 3.0e38], dtype=np.float32)])
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = inputs.f32_to_bf16_bits(x)
    assert (got == want).all()
    back = inputs.bf16_bits_to_f32(got)
    assert (back == torch.from_numpy(x).to(torch.bfloat16).float().numpy()).all()


def test_streams_are_deterministic_and_layer_addressable():
    cfg = inputs.CONFIGS[3].with_layers(3)
    K1, V1 = inputs.make_kv(cfg, 64, chunk=5)
    K2, V2 = inputs.make_kv(cfg, 64, chunk=5, layers=[2])
    assert K1.dtype == np.uint16 and K1.shape == (3, 1, 8, 64, 128)
    assert (K1[2] == K2[0]).all() and (V1[2] == V2[0]).all()
    K3, _ = inputs.make_kv(cfg, 64, chunk=6)
    assert (K1 != K3).any()
    assert (inputs.make_q(cfg, 4) == inputs.make_q(cfg, 4)).all()


def test_config_table():
    for i, cfg in inputs.CONFIGS.items():
        assert cfg.cfg_id == i and cfg.Hq % cfg.Hkv == 0 and 0 < cfg.keep < cfg.pot_size
        assert 0 <= cfg.nuc_slots <= cfg.keep
    c1 = inputs.make_cycle(inputs.CONFIGS[1])
    assert c1["K"].dtype == np.float32 and c1["K"].shape == (1, 1, 2, 512, 64)
    assert c1["Q"].shape == (1, 1, 8, 16, 64) and c1["aux"].shape == (1, 512)
    assert 0 <= c1["aux"].min() and c1["aux"].max() < 1


def test_duplicate_recipe_has_exact_duplicates():
    cfg = inputs.small_config(cfg_id=5, recipe="student_dup", dtype="bf16", pot_size=400, batch=2,
                              Hq=4, Hkv=2, d=64)
    K, V = inputs.make_kv(cfg)
    for b, (dst, src) in enumerate(inputs._dup_plan(cfg, 400)):
        assert len(dst) == 20
        for t, s in zip(dst, src):
            assert s < t
            assert (K[0, b, :, t] == K[0, b, :, s]).all() and (V[0, b, :, t] == V[0, b, :, s]).all()


def test_outlier_channels_fixed_per_stream():
    cfg = inputs.CONFIGS[3].with_layers(1)
    s = inputs._outlier_scale(cfg, 0)
    assert set(np.unique(s).tolist()) <= {1.0, 8.0}
    assert (s == inputs._outlier_scale(cfg, 0)).all()


def test_cap_key_rows_are_seeded_and_shaped():
    cfg = inputs.small_config(cfg_id=130, layers=2, batch=2, Hq=4, Hkv=2, d=64, cap_rows=5, dtype="bf16")
    a, b = inputs.make_kcap(cfg, 3), inputs.make_kcap(cfg, 3)
    assert a.shape == (2, 2, 2, 5, 64) and a.dtype == np.uint16 and (a == b).all()
    assert not (a == inputs.make_kcap(cfg, 4)).all()
    assert (inputs.make_kcap(cfg, 3, layers=[1])[0] == a[1]).all()          # a layer subset is the same stream
    assert not (a[:, :, :, :, :] == inputs.make_q(cfg, 3)[:, :, :2]).all()  # independent of the queries


def test_logits_recipe():
    z, lab = inputs.make_logits(9, 200, 500, "bf16", chunk=2, ignored=0.1)
    z2, lab2 = inputs.make_logits(9, 200, 500, "bf16", chunk=2, ignored=0.1)
    assert z.shape == (200, 500) and z.dtype == np.uint16 and (z == z2).all() and (lab == lab2).all()
    assert lab.dtype == np.int32 and ((lab == -100) | ((lab >= 0) & (lab < 500))).all() and (lab == -100).any()
    assert not (inputs.make_logits(9, 200, 500, "bf16", chunk=3)[0] == z).all()
    zf = inputs.widen(z, "bf16")
    ok = lab >= 0
    assert (zf[ok, lab[ok]] > 5).mean() > 0.3      # about half of the labels are well predicted
