"""The allocation-free scoring entry point against the pot's own scoring.

Some users of this library cannot allocate device memory when they need CaP scores:
their framework took the whole device for its memory pool at start-up, or they sit in a
latency-critical loop where cudaMalloc would stall every stream.  For them
``ipot_cap_scores_noalloc`` keeps its scratch in a fixed array inside the library.
This file checks, through the C ABI, that it returns what ``ipot_score_only`` returns and
what the CPU checker computes (Eq. 2), twice in a row with different shapes (the array keeps
the first call's contents), that the device's free memory as the driver reports it does not
move across a call, and that it refuses work beyond the array's capacity.  It sorts last so that a run that
stops at the first failure has already run everything else.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2410_01518_b200 import inputs, ipot
from parity import REL, make_pot, to_dev

pytestmark = pytest.mark.gpu


def pot_scores(cfg, t, n):
    h = make_pot(cfg)
    try:
        ipot.ipot_set_scorer(h, ipot.IPOT_SCORER_SIMT)
        ipot.ipot_append_chunk(h, to_dev(t["K"][:, :, :, :n], cfg.dtype), to_dev(t["V"][:, :, :, :n], cfg.dtype), n)
        ipot.ipot_score_only(h, to_dev(t["Q"], cfg.dtype), cfg.cap_rows)
        assert ipot.ipot_sync_status(h) == 0
        sp, nb = ipot.ipot_last_scores(h)
        return ipot.device_array(sp, (cfg.units, nb), "f32").clone()
    finally:
        ipot.ipot_destroy(h)


def noalloc_scores(cfg, t, n, watch_memory):
    Q = to_dev(t["Q"], cfg.dtype)                       # [L][B][Hq][P][d] == [units][G*P][d]
    K = to_dev(t["K"], cfg.dtype)                       # [units][pot_size][d], first n rows scored
    out = torch.full((cfg.units, n), float("nan"), device="cuda")
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]          # the driver's figure: it sees any allocation, the library's too
    ipot.ipot_cap_scores_noalloc(Q, K, out, cfg.units, cfg.G * cfg.cap_rows, n, cfg.d, cfg.pot_size,
                                 ipot.IPOT_F32 if cfg.dtype == "f32" else ipot.IPOT_BF16,
                                 torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    if watch_memory:
        assert torch.cuda.mem_get_info()[0] == free_before
    return out


def test_noalloc_scores_match_pot_scores_and_the_checker_twice_in_a_row():
    first = inputs.small_config(cfg_id=290, pot_size=900, keep=300, nuc_slots=0, cap_rows=16, Hq=8, Hkv=2, d=128,
                                dtype="bf16", layers=3, batch=2)
    second = inputs.small_config(cfg_id=291, pot_size=333, keep=100, nuc_slots=0, cap_rows=5, Hq=4, Hkv=2, d=64,
                                 dtype="f32", layers=2)
    for k, (cfg, n) in enumerate(((first, 900), (second, 301), (first, 900))):
        t = inputs.make_cycle(cfg)
        want = pot_scores(cfg, t, n)
        # the first call on a device looks the array's address up and the first launch of a kernel loads its code:
        # the free-memory figure is watched from the second call on
        got = noalloc_scores(cfg, t, n, watch_memory=k > 0)
        assert torch.isfinite(got).all()
        # same kernels, same order of operations: the tests' score tolerance (1e-3 relative) is met exactly
        torch.testing.assert_close(got, want, rtol=1e-3, atol=1e-30)
        assert abs(got.sum(dim=1) - cfg.G * cfg.cap_rows).max().item() < 1e-2
        # Eq. 2 from the CPU checker, unit by unit, under the rule of tests/parity.py
        M = cfg.G * cfg.cap_rows
        Qw = inputs.widen(t["Q"], cfg.dtype).reshape(cfg.units, M, cfg.d)
        Kw = inputs.widen(t["K"], cfg.dtype).reshape(cfg.units, cfg.pot_size, cfg.d)[:, :n]
        g = got.cpu().numpy().astype(np.float64)
        for unit in range(cfg.units):
            ref = oracle.cap_scores(Qw[unit], Kw[unit])
            assert (np.abs(g[unit] - ref) <= REL * np.abs(ref) + M * 2.0 ** -126).all(), unit


def test_noalloc_refuses_more_rows_than_its_fixed_scratch_holds():
    L = ipot.lib()
    x = torch.zeros(64, device="cuda")
    units, rows = 1024, 65     # 66560 rows > 65536
    rc = L.ipot_cap_scores_noalloc(x.data_ptr(), x.data_ptr(), x.data_ptr(), units, rows, 8, 64, 8, ipot.IPOT_BF16, None)
    assert rc == ipot.IPOT_E_LIMIT and "scratch" in ipot.ipot_strerror(rc)
    rc = L.ipot_cap_scores_noalloc(None, x.data_ptr(), x.data_ptr(), 1, 1, 8, 64, 8, ipot.IPOT_BF16, None)
    assert rc == ipot.IPOT_E_INVALID
