"""The documented call sequence on ONE pot, every result against the CPU checker, through the C ABI:
token novelty (Sec. 3.3.2, Eq. 3) -> compression cycle (Sec. 3.2) -> generation over the distilled pot (Sec. 4.5),
then a novelty call with a larger vocabulary, which makes the library grow its novelty scratch, and generation
again.  The scratch buffers of the three calls belong to the same handle; each call must leave the others' alone."""
import numpy as np
import pytest
import torch

import oracle
from paper_2410_01518_b200 import inputs, ipot
from parity import compare_cycle, make_pot, read_results, to_dev
from test_decode_gpu import check as check_decode, make_query
from test_novelty_gpu import close as novelty_close

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("deferred", [False, True])
def test_novelty_cycle_generation_on_one_pot(deferred):
    cfg = inputs.small_config(cfg_id=900, pot_size=768, keep=256, nuc_slots=128, cap_rows=8, Hq=8, Hkv=2, d=128,
                              dtype="bf16", batch=2, layers=2)
    N = cfg.pot_size
    t = inputs.make_cycle(cfg)
    z, lab = inputs.make_logits(91, cfg.batch * N, 3000, "bf16")
    z2, lab2 = inputs.make_logits(92, cfg.batch * 40, 70000, "bf16")       # more scratch than the first call needed
    q = make_query(cfg)
    h = make_pot(cfg)
    try:
        Kd, Vd = to_dev(t["K"], "bf16"), to_dev(t["V"], "bf16")
        if deferred:
            ipot.ipot_set_deferred_append(h, True)
        ipot.ipot_append_chunk(h, Kd, Vd, N)
        aux = torch.empty((cfg.batch, N), device="cuda")
        ipot.ipot_nuc_scores(h, to_dev(z, "bf16"), ipot.IPOT_BF16, 3000, torch.from_numpy(lab).cuda(), N, 3000, aux, N, 0)
        ipot.ipot_score_and_compress(h, to_dev(t["Q"], "bf16"), cfg.cap_rows, aux)
        gpu = read_results(h, cfg, N)
        t["aux"] = aux.cpu().numpy()
        assert novelty_close(t["aux"], oracle.token_novelty(inputs.widen(z, "bf16"), lab).reshape(cfg.batch, N)).all()
        same, n = compare_cycle(cfg, t, gpu)
        assert n == cfg.units and same >= n - 1

        # generation attends to what the GPU kept (bytes already checked against the inputs above)
        shape = (cfg.layers, cfg.batch, cfg.Hkv, cfg.keep, cfg.d)
        Kc, Vc = gpu[2].reshape(shape), gpu[3].reshape(shape)
        ref_out, ref_lse = oracle.decode_attention(q, Kc, Vc)
        qd = to_dev(q, "bf16")
        out = torch.full((cfg.layers, cfg.batch, cfg.Hq, cfg.d), float("nan"), device="cuda")
        lse = torch.full((cfg.layers, cfg.batch, cfg.Hq), float("nan"), device="cuda")
        for _ in range(2):
            out.fill_(float("nan"))
            ipot.ipot_decode_attention(h, qd, out, lse)
            assert ipot.ipot_sync_status(h) == 0
            check_decode(out.cpu().numpy(), lse.cpu().numpy(), ref_out, ref_lse)

        # a larger vocabulary: the novelty scratch is re-allocated, nothing else may move
        aux2 = torch.full((cfg.batch, 64), -7.0, device="cuda")
        ipot.ipot_nuc_scores(h, to_dev(z2, "bf16"), ipot.IPOT_BF16, 70000, torch.from_numpy(lab2).cuda(), 40, 70000, aux2, 64, 8)
        assert ipot.ipot_sync_status(h) == 0
        a2 = aux2.cpu().numpy()
        assert novelty_close(a2[:, 8:48], oracle.token_novelty(inputs.widen(z2, "bf16"), lab2).reshape(cfg.batch, 40)).all()
        assert (a2[:, :8] == -7.0).all() and (a2[:, 48:] == -7.0).all()
        out.fill_(float("nan"))
        ipot.ipot_decode_attention(h, qd, out, lse)
        assert ipot.ipot_sync_status(h) == 0
        check_decode(out.cpu().numpy(), lse.cpu().numpy(), ref_out, ref_lse)

        # and the pot goes on: refill, second cycle with produced novelty for the new slots only
        n_new = N - cfg.keep
        Kn, Vn = inputs.make_kv(cfg, n_new, chunk=5)
        Knd, Vnd = to_dev(Kn, "bf16"), to_dev(Vn, "bf16")
        ipot.ipot_append_chunk(h, Knd, Vnd, n_new)
        t2 = {"K": np.concatenate([Kc, Kn], axis=3), "V": np.concatenate([Vc, Vn], axis=3),
              "Q": inputs.make_q(cfg, 1), "aux": inputs.make_aux(cfg, 1)}
        ipot.ipot_score_and_compress(h, to_dev(t2["Q"], "bf16"), cfg.cap_rows, torch.from_numpy(t2["aux"]).cuda())
        same, n = compare_cycle(cfg, t2, read_results(h, cfg, N))
        assert n == cfg.units and same >= n - 1
    finally:
        ipot.ipot_destroy(h)
