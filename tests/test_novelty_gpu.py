"""GPU parity of the token-novelty producer (Sec. 3.3.2, Eq. 3) against the CPU checker, through the C ABI.

Tolerance: |n_gpu - n_ref| <= 1e-4 + 1e-5 * |n_ref|.  The kernel works in fp32 on log2-scaled logits: the
scaling rounds each logit to 6e-8 relative (4e-6 absolute at |z| = 50), the exponentials and their sum carry
that into a few 1e-6 on the log-sum-exp; novelty is a difference of two such numbers, so the bound is
absolute, with a factor ~10 of margin.  NuC only ranks the largest values."""
import numpy as np
import pytest
import torch

import oracle
from paper_2410_01518_b200 import inputs, ipot
from parity import compare_cycle, make_pot, read_results, to_dev

pytestmark = pytest.mark.gpu


def close(got, ref):
    return np.abs(got.astype(np.float64) - ref) <= 1e-4 + 1e-5 * np.abs(ref)


def run_producer(batch, n, V, dtype, row_pad=0, slot0=0, extra=0, chunk=0, ignored=0.0, misalign=0):
    """Returns (gpu novelty [batch][n], checker novelty [batch][n], aux array, status)."""
    cfg = inputs.small_config(cfg_id=600, batch=batch, pot_size=max(64, slot0 + n + extra), keep=8, nuc_slots=4)
    z, lab = inputs.make_logits(0x5EED + V, batch * n, V, dtype, chunk, ignored)
    stride = V + row_pad
    zp = np.zeros((batch * n, stride), dtype=z.dtype)
    zp[:, :V] = z
    if row_pad:
        zp[:, V:] = inputs.store(np.full((batch * n, row_pad), 1e4, dtype=np.float32), dtype)  # must never be read
    flat = np.concatenate([np.zeros(misalign, dtype=z.dtype), zp.reshape(-1)])
    zd = to_dev(flat, dtype)[misalign:]
    labd = torch.from_numpy(lab).cuda()
    aux_stride = slot0 + n + extra
    aux = torch.full((batch, aux_stride), -7.0, device="cuda")
    h = make_pot(cfg)
    try:
        ipot.ipot_nuc_scores(h, zd, ipot.IPOT_F32 if dtype == "f32" else ipot.IPOT_BF16, stride, labd, n, V, aux,
                             aux_stride, slot0)
        status = ipot.ipot_sync_status(h)
    finally:
        ipot.ipot_destroy(h)
    a = aux.cpu().numpy()
    ref = oracle.token_novelty(inputs.widen(z, dtype), lab).reshape(batch, n)
    return a[:, slot0:slot0 + n], ref, a, status


SHAPES = [
    # (batch, tokens, vocab, dtype, row padding, misalignment in elements)
    (1, 5, 7, "f32", 0, 0), (1, 64, 1000, "f32", 0, 0), (2, 33, 8192, "bf16", 0, 0), (1, 40, 8193, "bf16", 7, 0),
    (1, 17, 50257, "bf16", 0, 0),      # odd vocabulary: most rows start off a 16-byte boundary
    (1, 9, 16384, "f32", 0, 1),        # every row misaligned
    (3, 11, 32000, "bf16", 64, 0), (1, 24, 128256, "bf16", 0, 0), (1, 6, 151936, "f32", 0, 0),
]


@pytest.mark.parametrize("case", range(len(SHAPES)))
def test_producer_shapes(case):
    batch, n, V, dtype, pad, mis = SHAPES[case]
    got, ref, _, status = run_producer(batch, n, V, dtype, row_pad=pad, misalign=mis)
    assert status == 0
    assert close(got, ref).all(), f"worst {np.abs(got - ref).max():.3e}"
    assert ref.min() < 3.0 and ref.max() > np.log(V) * 0.8   # the recipe spans confident and surprised tokens


def test_chunk_of_the_mistral_stream_goes_to_its_slots():
    """2048 new tokens over a 32000-word vocabulary, written behind 2048 survivors of a 4096-slot array."""
    got, ref, aux, status = run_producer(1, 2048, 32000, "bf16", slot0=2048, chunk=3)
    assert status == 0 and close(got, ref).all()
    assert (aux[:, :2048] == -7.0).all()                      # nothing outside [slot0, slot0 + n) is touched
    top = np.argsort(-ref[0], kind="stable")[:1024]           # the NuC ranking is the checker's
    assert set(np.argsort(-got[0], kind="stable")[:1000].tolist()) <= set(np.argsort(-ref[0], kind="stable")[:1048].tolist())
    assert len(top) == 1024


def test_ignored_and_out_of_range_labels():
    got, ref, _, status = run_producer(2, 50, 300, "f32", ignored=0.3)
    assert status == 0 and close(got, ref).all() and (got == 0).sum() >= 10
    cfg = inputs.small_config(cfg_id=601, pot_size=64, keep=8, nuc_slots=4)
    z, lab = inputs.make_logits(5, 4, 100, "f32")
    lab[2] = 100                                              # one past the vocabulary
    h = make_pot(cfg)
    try:
        aux = torch.zeros((1, 4), device="cuda")
        ipot.ipot_nuc_scores(h, to_dev(z, "f32"), ipot.IPOT_F32, 100, torch.from_numpy(lab).cuda(), 4, 100, aux, 4, 0)
        assert ipot.ipot_sync_status(h) == ipot.IPOT_E_BOUNDS
        a = aux.cpu().numpy()[0]
        assert a[2] == 0 and close(np.delete(a, 2), np.delete(oracle.token_novelty(z.astype(np.float64), lab), 2)).all()
        L = ipot.lib()
        zd, ld = to_dev(z, "f32"), torch.from_numpy(lab).cuda()
        args = lambda **k: [h, k.get("z", zd.data_ptr()), k.get("dt", 1), k.get("stride", 100), k.get("lab", ld.data_ptr()),
                            k.get("n", 4), k.get("V", 100), k.get("out", aux.data_ptr()), k.get("astride", 4), k.get("slot0", 0)]
        for bad in (dict(z=None), dict(lab=None), dict(out=None), dict(dt=5), dict(stride=99), dict(n=0), dict(V=0),
                    dict(slot0=1), dict(slot0=-1), dict(astride=3), dict(z=zd.data_ptr() + 2), dict(n=70000)):
            assert L.ipot_nuc_scores(*args(**bad)) == ipot.IPOT_E_INVALID, bad
    finally:
        ipot.ipot_destroy(h)


def test_produced_novelty_drives_a_cycle():
    """Producer -> aux array on the device -> ipot_score_and_compress, no host round trip; the checker gets the
    same aux bytes, so the whole cycle must agree with it."""
    cfg = inputs.small_config(cfg_id=602, pot_size=512, keep=256, nuc_slots=128, cap_rows=8, Hq=8, Hkv=2, d=128,
                              dtype="bf16", batch=2)
    t = inputs.make_cycle(cfg)
    z, lab = inputs.make_logits(77, cfg.batch * 512, 4000, "bf16")
    h = make_pot(cfg)
    try:
        aux = torch.empty((cfg.batch, 512), device="cuda")
        ipot.ipot_append_chunk(h, to_dev(t["K"], "bf16"), to_dev(t["V"], "bf16"), 512)
        ipot.ipot_nuc_scores(h, to_dev(z, "bf16"), ipot.IPOT_BF16, 4000, torch.from_numpy(lab).cuda(), 512, 4000, aux, 512, 0)
        ipot.ipot_score_and_compress(h, to_dev(t["Q"], "bf16"), cfg.cap_rows, aux)
        gpu = read_results(h, cfg, 512)
    finally:
        ipot.ipot_destroy(h)
    t["aux"] = aux.cpu().numpy()
    assert close(t["aux"], oracle.token_novelty(inputs.widen(z, "bf16"), lab).reshape(cfg.batch, 512)).all()
    same, n = compare_cycle(cfg, t, gpu)
    assert n == cfg.units and same >= n - 1
