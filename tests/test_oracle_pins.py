"""Pins for the CPU checker: what the paper and the mathematics fix, checked
against the checker (never the other way round)."""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def rnd(seed):
    return np.random.default_rng(seed)


# ---------------------------------------------------------------- Eq. 2
def test_worked_example_eq2():
    want = {}
    for line in open(os.path.join(GOLD, "eq2_worked_example.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, v = line.split("=")
        want[k.strip()] = float(sum(Fraction(t.strip()) for t in v.split("+")))
    Q = np.array([[2.0, 0, 0, 0], [-2.0, 0, 0, 0]])
    K = np.array([[0.0, 5, -1, 2], [np.log(2.0), 7, 0, 1], [np.log(3.0), -3, 4, 9]])
    u = oracle.cap_scores(Q, K)
    np.testing.assert_allclose(u, [want["u0"], want["u1"], want["u2"]], rtol=1e-14)


@pytest.mark.parametrize("M,N,d", [(1, 7, 4), (16, 64, 8), (64, 512, 64), (5, 33, 128)])
def test_rows_sum_to_one_and_total_is_M(M, N, d):
    g = rnd(1)
    Q, K = g.standard_normal((M, d)) * 3, g.standard_normal((N, d)) * 3
    u, rs = oracle.cap_scores(Q, K, return_row_sums=True)
    np.testing.assert_allclose(rs, 1.0, atol=1e-12)
    assert abs(u.sum() - M) <= 1e-10 * M
    assert (u >= 0).all()


def test_zero_queries_and_equal_keys_give_uniform():
    g = rnd(2)
    M, N, d = 6, 40, 16
    K = g.standard_normal((N, d))
    np.testing.assert_allclose(oracle.cap_scores(np.zeros((M, d)), K), M / N, rtol=1e-13)
    Q = g.standard_normal((M, d))
    Keq = np.tile(g.standard_normal((1, d)), (N, 1))
    np.testing.assert_allclose(oracle.cap_scores(Q, Keq), M / N, rtol=1e-13)


def test_single_key_takes_everything():
    g = rnd(3)
    Q = g.standard_normal((9, 32))
    np.testing.assert_allclose(oracle.cap_scores(Q, g.standard_normal((1, 32))), [9.0], rtol=1e-14)


def test_dominant_key_limit():
    g = rnd(4)
    d, N = 16, 50
    q = g.standard_normal((1, d))
    K = g.standard_normal((N, d))
    K[17] = 200.0 * q[0]
    u = oracle.cap_scores(q, K)
    assert u[17] > 1 - 1e-12 and abs(u.sum() - 1) < 1e-12


def test_key_shift_invariance():
    # adding one vector c to every key adds q.c/sqrt(d) to a whole row: softmax unchanged
    g = rnd(5)
    Q, K = g.standard_normal((8, 24)), g.standard_normal((70, 24))
    c = g.standard_normal((1, 24)) * 5
    np.testing.assert_allclose(oracle.cap_scores(Q, K + c), oracle.cap_scores(Q, K), rtol=1e-9)


def test_slot_permutation_equivariance():
    g = rnd(6)
    Q, K = g.standard_normal((8, 24)), g.standard_normal((70, 24))
    perm = g.permutation(70)
    np.testing.assert_allclose(oracle.cap_scores(Q, K[perm]), oracle.cap_scores(Q, K)[perm], rtol=1e-12)


def test_row_order_does_not_matter_but_rows_add():
    g = rnd(7)
    Q, K = g.standard_normal((6, 8)), g.standard_normal((20, 8))
    whole = oracle.cap_scores(Q, K)
    parts = sum(oracle.cap_scores(Q[i:i + 1], K) for i in range(6))
    np.testing.assert_allclose(whole, parts, rtol=1e-13)


def test_single_row_is_a_library_softmax():
    torch = pytest.importorskip("torch")
    from scipy.special import softmax
    g = rnd(8)
    d = 64
    q, K = g.standard_normal((1, d)), g.standard_normal((300, d))
    u = oracle.cap_scores(q, K)
    logits = (K @ q[0]) / np.sqrt(d)
    np.testing.assert_allclose(u, softmax(logits), rtol=1e-12)
    t = torch.softmax(torch.from_numpy(logits), dim=0).numpy()
    np.testing.assert_allclose(u, t, rtol=1e-12)


def test_many_rows_against_library_softmax():
    from scipy.special import softmax
    g = rnd(9)
    d = 32
    Q, K = g.standard_normal((12, d)) * 2, g.standard_normal((90, d)) * 2
    ref = softmax(Q @ K.T / np.sqrt(d), axis=1).sum(axis=0)
    np.testing.assert_allclose(oracle.cap_scores(Q, K), ref, rtol=1e-12)


def test_scale_is_one_over_sqrt_d():
    # d = 16: logits are q.k/4.  One row, two keys, q.k = (0, 4 ln 3) -> p = (1/4, 3/4)
    d = 16
    q = np.zeros((1, d)); q[0, 0] = 1.0
    K = np.zeros((2, d)); K[1, 0] = 4 * np.log(3.0)
    np.testing.assert_allclose(oracle.cap_scores(q, K), [0.25, 0.75], rtol=1e-14)


# ---------------------------------------------------------------- selection
def brute_best_subset(vals, cand, r):
    best, arg = None, None
    for sub in itertools.combinations(cand, r):
        s = sum(vals[j] for j in sub)
        if best is None or s > best:
            best, arg = s, sub
    return set(arg) if arg is not None else set()


@pytest.mark.parametrize("seed", range(12))
def test_selection_is_the_brute_force_maximiser(seed):
    g = rnd(100 + seed)
    N = int(g.integers(4, 13))
    keep = int(g.integers(1, N))
    T = int(g.integers(0, keep + 1))
    aux, u = g.random(N), g.random(N)
    nuc = oracle.nuc_top(aux, T)
    assert set(nuc.tolist()) == brute_best_subset(aux, range(N), T)
    assert list(nuc) == sorted(nuc)
    idx = oracle.select(u, nuc, keep)
    rest = [j for j in range(N) if j not in set(nuc.tolist())]
    want = set(nuc.tolist()) | brute_best_subset(u, rest, keep - T)
    assert set(idx.tolist()) == want
    assert len(idx) == keep and list(idx) == sorted(set(idx.tolist()))


def test_selection_invariants_large():
    g = rnd(20)
    N, keep, T = 1000, 400, 150
    aux, u = g.random(N), g.random(N)
    nuc = oracle.nuc_top(aux, T)
    idx = oracle.select(u, nuc, keep)
    assert len(idx) == keep and (np.diff(idx) > 0).all()
    assert set(nuc.tolist()) <= set(idx.tolist())
    assert aux[nuc].min() >= np.delete(aux, nuc).max()
    kept_cap = np.setdiff1d(idx, nuc)
    dropped = np.setdiff1d(np.arange(N), idx)
    assert len(kept_cap) == keep - T
    assert u[kept_cap].min() >= u[dropped].max()


def test_nuc_only_and_cap_only_special_cases():
    g = rnd(21)
    N, keep = 200, 60
    aux = g.random(N)
    # T = keep: every head keeps the same slots whatever its CaP scores (NuC is per token)
    nuc = oracle.nuc_top(aux, keep)
    a = oracle.select(g.random(N), nuc, keep)
    b = oracle.select(g.random(N), nuc, keep)
    assert (a == b).all() and (a == nuc).all()
    # T = 0: plain top-k of the CaP score (library sort as the reference)
    u = g.random(N)
    idx = oracle.select(u, np.empty(0, dtype=np.int32), keep)
    assert set(idx.tolist()) == set(np.argsort(-u, kind="stable")[:keep].tolist())


def test_fill_with_max_then_one_topk_gives_the_same_set():
    # Appendix B combines the two scores by raising the NuC slots to the tensor's
    # maximum and taking a single top-|C|; Sec. 3.3.3 describes two separate
    # rankings.  With at least one CaP slot and distinct scores they agree.
    g = rnd(22)
    N, keep, T = 300, 120, 50
    aux, u = g.random(N), g.random(N)
    nuc = oracle.nuc_top(aux, T)
    filled = u.copy()
    filled[nuc] = np.inf  # strictly above every CaP score: the NuC slots can never lose
    one_topk = set(np.argsort(-filled, kind="stable")[:keep].tolist())
    assert set(oracle.select(u, nuc, keep).tolist()) == one_topk


def test_ties_prefer_lower_slots():
    N = 50
    nuc = oracle.nuc_top(np.ones(N), 7)
    assert nuc.tolist() == list(range(7))
    idx = oracle.select(np.full(N, 0.5), nuc, 20)
    assert idx.tolist() == list(range(20))
    u = np.zeros(N); u[40:] = 1.0
    idx = oracle.select(u, np.array([3], dtype=np.int32), 13)
    assert idx.tolist() == [0, 1, 3] + list(range(40, 50))


# ---------------------------------------------------------------- gather
def test_gather_is_bytewise_row_copy():
    g = rnd(30)
    rows = g.integers(0, 65536, size=(64, 24), dtype=np.uint16)
    idx = np.sort(g.choice(64, 20, replace=False)).astype(np.int32)
    out = oracle.gather(rows, idx)
    assert out.dtype == rows.dtype and (out == rows[idx]).all()
    ident = oracle.gather(rows, np.arange(64, dtype=np.int32))
    assert (ident == rows).all()


# ---------------------------------------------------------------- whole cycle wiring
def test_cycle_wiring_gqa_streams_layers():
    g = rnd(40)
    L, B, Hq, Hkv, P, d, N, keep, T = 2, 3, 6, 2, 4, 8, 30, 12, 5
    G = Hq // Hkv
    Q = g.standard_normal((L, B, Hq, P, d)).astype(np.float32)
    K = g.standard_normal((L, B, Hkv, N, d)).astype(np.float32)
    V = g.standard_normal((L, B, Hkv, N, d)).astype(np.float32)
    aux = g.random((B, N)).astype(np.float32)
    out = oracle.cycle(Q, K, V, aux, keep, T)
    assert out["u"].shape == (L * B * Hkv, N)
    for l in range(L):
        for b in range(B):
            nuc = oracle.nuc_top(aux[b], T)
            for kv in range(Hkv):
                unit = (l * B + b) * Hkv + kv
                # query head h serves kv head h // G; its P rows add to the same score
                u = sum(oracle.cap_scores(Q[l, b, h].astype(np.float64), K[l, b, kv].astype(np.float64))
                        for h in range(Hq) if h // G == kv)
                np.testing.assert_allclose(out["u"][unit], u, rtol=1e-12)
                assert abs(out["u"][unit].sum() - G * P) < 1e-9
                idx = oracle.select(out["u"][unit], nuc, keep)
                assert (out["idx"][unit] == idx).all()
                assert (out["K"][unit] == K[l, b, kv][idx]).all()
                assert (out["V"][unit] == V[l, b, kv][idx]).all()
    # a subset of units gives the same rows
    sub = oracle.cycle(Q, K, V, aux, keep, T, units=[7, 2])
    assert (sub["idx"][0] == out["idx"][7]).all() and (sub["idx"][1] == out["idx"][2]).all()
    np.testing.assert_array_equal(sub["u"][1], out["u"][2])


def test_cycle_accepts_bf16_bit_patterns():
    torch = pytest.importorskip("torch")
    g = rnd(41)
    x = g.standard_normal((1, 1, 2, 3, 8)).astype(np.float32)
    bits = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    wide = oracle.widen_storage(bits)
    assert (wide == torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()).all()


# ---------------------------------------------------------------- Appendix B listing, CaP keys inside the softmax
def test_incl_zero_queries_closed_form():
    # all logits 0: CaP position i sees N + i + 1 columns, each pot column gets 1 / (N + i + 1)
    g = rnd(50)
    G, P, N, d = 3, 4, 7, 8
    u, pm = oracle.cap_scores_incl(np.zeros((G * P, d)), g.standard_normal((N, d)), g.standard_normal((P, d)), P, True)
    want = G * sum(Fraction(1, N + i + 1) for i in range(P))
    np.testing.assert_allclose(u, float(want), rtol=1e-14)
    np.testing.assert_allclose(pm, [N / (N + (r % P) + 1) for r in range(G * P)], rtol=1e-14)


def test_incl_against_masked_library_softmax():
    torch = pytest.importorskip("torch")
    g = rnd(51)
    G, P, N, d = 2, 5, 40, 16
    Q, K, Kc = g.standard_normal((G * P, d)) * 2, g.standard_normal((N, d)) * 2, g.standard_normal((P, d)) * 2
    logits = torch.from_numpy(np.concatenate([Q @ K.T, Q @ Kc.T], axis=1) / np.sqrt(d))
    pos = torch.arange(G * P) % P                                # CaP position of each row
    hidden = torch.arange(P)[None, :] > pos[:, None]             # CaP key i' is hidden from row i when i' > i
    logits[:, N:] = logits[:, N:].masked_fill(hidden, float("-inf"))
    p = torch.softmax(logits, dim=1).numpy()
    u, pm = oracle.cap_scores_incl(Q, K, Kc, P, True)
    np.testing.assert_allclose(u, p[:, :N].sum(axis=0), rtol=1e-12)
    np.testing.assert_allclose(pm, p[:, :N].sum(axis=1), rtol=1e-12)
    assert abs(u.sum() + p[:, N:].sum() - G * P) < 1e-10         # the CaP columns took the rest


def test_incl_far_away_cap_keys_reduce_to_eq2():
    g = rnd(52)
    G, P, N, d = 2, 3, 25, 8
    Q = np.abs(g.standard_normal((G * P, d))) + 0.1               # every q . (-c 1) is very negative
    K = g.standard_normal((N, d))
    Kc = -400.0 * np.ones((P, d))
    np.testing.assert_allclose(oracle.cap_scores_incl(Q, K, Kc, P), oracle.cap_scores(Q, K), rtol=1e-12)


def test_incl_is_causal_inside_the_cap():
    g = rnd(53)
    G, P, N, d = 2, 4, 12, 8
    Q, K, Kc = g.standard_normal((G * P, d)), g.standard_normal((N, d)), g.standard_normal((P, d))
    _, pm = oracle.cap_scores_incl(Q, K, Kc, P, True)
    Kc2 = Kc.copy()
    Kc2[2] += 3.0                                                 # only rows at CaP positions 2 and 3 may notice
    _, pm2 = oracle.cap_scores_incl(Q, K, Kc2, P, True)
    for r in range(G * P):
        assert (pm[r] == pm2[r]) == (r % P < 2)
    # a single CaP row (P = 1) sees exactly one CaP key: its own
    q, kc = Q[:1], Kc[:1]
    s = np.concatenate([K @ q[0], kc @ q[0]]) / np.sqrt(d)
    e = np.exp(s - s.max())
    np.testing.assert_allclose(oracle.cap_scores_incl(q, K, kc, 1), (e / e.sum())[:N], rtol=1e-12)


def test_cycle_with_cap_keys_wiring():
    g = rnd(54)
    L, B, Hq, Hkv, P, d, N, keep, T = 2, 2, 4, 2, 3, 8, 20, 9, 4
    G = Hq // Hkv
    Q = g.standard_normal((L, B, Hq, P, d)).astype(np.float32)
    K = g.standard_normal((L, B, Hkv, N, d)).astype(np.float32)
    V = g.standard_normal((L, B, Hkv, N, d)).astype(np.float32)
    Kc = g.standard_normal((L, B, Hkv, P, d)).astype(np.float32)
    aux = g.random((B, N)).astype(np.float32)
    out = oracle.cycle(Q, K, V, aux, keep, T, K_cap=Kc)
    for l in range(L):
        for b in range(B):
            for kv in range(Hkv):
                unit = (l * B + b) * Hkv + kv
                u = sum(oracle.cap_scores_incl(Q[l, b, h].astype(np.float64), K[l, b, kv].astype(np.float64),
                                               Kc[l, b, kv].astype(np.float64), P)
                        for h in range(Hq) if h // G == kv)
                np.testing.assert_allclose(out["u"][unit], u, rtol=1e-12)
                assert out["u"][unit].sum() < G * P
                assert (out["idx"][unit] == oracle.select(out["u"][unit], oracle.nuc_top(aux[b], T), keep)).all()
                assert (out["K"][unit] == K[l, b, kv][out["idx"][unit]]).all()
    base = oracle.cycle(Q, K, V, aux, keep, T)
    assert not np.allclose(base["u"], out["u"])


# ---------------------------------------------------------------- Eq. 3: token novelty
def test_novelty_closed_forms():
    V = 37
    out = oracle.token_novelty(np.full((3, V), 1.25), [0, 5, V - 1])
    np.testing.assert_allclose(out, np.log(V), rtol=1e-14)                  # uniform prediction
    z = np.array([[0.3, -1.1], [2.0, 2.0], [-4.0, 6.0]])
    lab = [0, 1, 0]
    want = [np.log1p(np.exp(z[i, 1 - lab[i]] - z[i, lab[i]])) for i in range(3)]   # V = 2: a softplus
    np.testing.assert_allclose(oracle.token_novelty(z, lab), want, rtol=1e-13)
    z = np.zeros((2, 50)); z[0, 7] = 60.0; z[1, 7] = -60.0                  # certain / hopeless
    out = oracle.token_novelty(z, [7, 7])
    assert 0 <= out[0] < 1e-20 and abs(out[1] - (60.0 + np.log(49))) < 1e-12
    assert (oracle.token_novelty(np.ones((2, 9)), [-100, 9]) == 0).all()    # ignored positions


def test_novelty_is_the_library_cross_entropy():
    torch = pytest.importorskip("torch")
    from scipy.special import logsumexp
    g = rnd(60)
    z = g.standard_normal((40, 513)) * 4
    lab = g.integers(0, 513, 40)
    out = oracle.token_novelty(z, lab)
    np.testing.assert_allclose(out, logsumexp(z, axis=1) - z[np.arange(40), lab], rtol=1e-12)
    ce = torch.nn.functional.cross_entropy(torch.from_numpy(z), torch.from_numpy(lab), reduction="none")
    np.testing.assert_allclose(out, ce.numpy(), rtol=1e-12)
    np.testing.assert_allclose(oracle.token_novelty(z + 123.0, lab), out, rtol=1e-9, atol=1e-11)  # shift invariance
    assert (out > 0).all()


# ---------------------------------------------------------------- Sec. 3.4: rotary embedding at pot positions
def _tables(positions, d, dtype="f32"):
    from paper_2410_01518_b200 import inputs
    return inputs.make_rope_table(positions, d, dtype)


def test_rope_exact_small_cases_and_identity():
    x = np.array([[1, 2, 3, 4]], dtype=np.float32)
    c = np.array([[1, 1], [0.5, 0.5], [0, 0]], dtype=np.float32)
    s = np.array([[0, 0], [0.5, 0.5], [1, 1]], dtype=np.float32)
    assert (oracle.rope_rows(x, [0], c, s) == x).all()                                  # angle 0
    assert (oracle.rope_rows(x, [1], c, s) == [[-1, -1, 2, 3]]).all()                   # pairs (1,3), (2,4)
    assert (oracle.rope_rows(x, [1], c, s, True) == [[-0.5, 1.5, -0.5, 3.5]]).all()     # pairs (1,2), (3,4)
    assert (oracle.rope_rows(x, [2], c, s) == [[-3, -4, 1, 2]]).all()                   # quarter turn
    cos_t, sin_t = _tables(16, 8)
    g = rnd(70)
    rows = g.standard_normal((3, 5, 8)).astype(np.float32)
    out = oracle.rope_rows(rows, [0, 0, 0, 0, 0], cos_t, sin_t)
    assert (out == rows).all()                                                          # position 0 everywhere


def test_rope_is_complex_multiplication():
    g = rnd(71)
    d, n = 16, 40
    cos_t, sin_t = _tables(64, d)
    rows = g.standard_normal((n, d)).astype(np.float32)
    pos = g.integers(0, 64, n)
    out, exact, mag = oracle.rope_rows(rows, pos, cos_t, sin_t, with_exact=True)
    z = rows[:, :d // 2].astype(np.float64) + 1j * rows[:, d // 2:].astype(np.float64)
    w = z * (cos_t[pos].astype(np.float64) + 1j * sin_t[pos].astype(np.float64))        # the library's complex product
    assert (exact[:, :d // 2] == w.real).all() and (exact[:, d // 2:] == w.imag).all()
    assert (out[:, :d // 2] == w.real.astype(np.float32)).all() and (out[:, d // 2:] == w.imag.astype(np.float32)).all()
    a, b = np.abs(rows[:, :d // 2].astype(np.float64)), np.abs(rows[:, d // 2:].astype(np.float64))
    c, s_ = np.abs(cos_t[pos].astype(np.float64)), np.abs(sin_t[pos].astype(np.float64))
    assert (mag[:, :d // 2] == a * c + b * s_).all() and (mag[:, d // 2:] == b * c + a * s_).all()
    # pair norms survive the rotation (up to the table's rounding)
    o = out.astype(np.float64)
    np.testing.assert_allclose(o[:, :d // 2] ** 2 + o[:, d // 2:] ** 2, np.abs(z) ** 2, rtol=1e-5)


def test_rope_rounds_the_exact_product_once_to_the_nearest_storage_value():
    """Exact rational arithmetic, then a brute-force search over every finite bf16 value for the nearest one
    (ties: even bit pattern).  A product rounded through float32 first would fail the constructed tie case."""
    from fractions import Fraction
    from paper_2410_01518_b200 import inputs
    g = rnd(75)
    d, n = 12, 9
    rows = g.standard_normal((n, d)).astype(np.float32)
    pos = g.integers(0, 32, n)
    rb, cb, sb = inputs.store(rows, "bf16"), *inputs.make_rope_table(32, d, "bf16")
    got = oracle.rope_rows(rb, pos, cb, sb)
    bits = np.arange(65536, dtype=np.uint32)
    with np.errstate(invalid="ignore"):
        vals = (bits << np.uint32(16)).view(np.float32).astype(np.float64)
    finite = np.isfinite(vals)

    def nearest(x: Fraction) -> int:
        xf = float(x)                                   # exact: a sum of two 16-bit products
        assert Fraction(xf) == x
        dist = np.where(finite, np.abs(vals - xf), np.inf)
        best = np.flatnonzero(dist == dist.min())
        if xf == 0.0:
            return 0
        best = [b for b in best if (vals[b] >= 0) == (xf >= 0) or vals[b] == 0]
        return int(min(best, key=lambda b: b & 1))      # a tie has one even and one odd neighbour

    w = lambda a: Fraction(float(inputs.widen(np.array([a], dtype=np.uint16), "bf16")[0]))
    for r in range(n):
        for c in range(d // 2):
            lo, hi, cs, sn = w(rb[r, c]), w(rb[r, c + d // 2]), w(cb[pos[r], c]), w(sb[pos[r], c])
            assert int(got[r, c]) == nearest(lo * cs - hi * sn)
            assert int(got[r, c + d // 2]) == nearest(hi * cs + lo * sn)
    # a case that rounding through float32 first gets wrong: lo cos - hi sin = (1 + 2^-7)(1 - 2^-8) + 145 * 113 * 2^-29
    # = 1 + 2^-8 + 2^-29, just above the midpoint of the bf16 neighbours 1 and 1 + 2^-7.  float32 drops the 2^-29,
    # lands on the midpoint and would then tie to even (1.0); one rounding from the exact value gives 1 + 2^-7.
    x = inputs.store(np.array([[1.0 + 2.0 ** -7, -145.0 * 2.0 ** -14]], dtype=np.float32), "bf16")
    ct = inputs.store(np.array([[1.0 - 2.0 ** -8]], dtype=np.float32), "bf16")
    st = inputs.store(np.array([[113.0 * 2.0 ** -15]], dtype=np.float32), "bf16")
    val = Fraction(1) + Fraction(1, 2 ** 8) + Fraction(1, 2 ** 29)
    assert w(x[0, 0]) * w(ct[0, 0]) - w(x[0, 1]) * w(st[0, 0]) == val
    assert nearest(val) == 0x3F81
    assert int(oracle.rope_rows(x, [0], ct, st)[0, 0]) == 0x3F81
    assert int(inputs.store(np.array([np.float32(float(val))]), "bf16")[0]) == 0x3F80   # the two-step route differs


def test_rope_scores_depend_on_the_position_difference():
    g = rnd(72)
    d = 32
    cos_t, sin_t = _tables(200, d)
    q = g.standard_normal((1, d)).astype(np.float32)
    k = g.standard_normal((1, d)).astype(np.float32)
    dots = [float(oracle.rope_rows(q, [m], cos_t, sin_t).astype(np.float64)[0]
                  @ oracle.rope_rows(k, [m - 17], cos_t, sin_t).astype(np.float64)[0]) for m in (17, 60, 199)]
    assert max(dots) - min(dots) < 1e-4 * max(1.0, abs(dots[0]))
    other = float(oracle.rope_rows(q, [60], cos_t, sin_t).astype(np.float64)[0]
                  @ oracle.rope_rows(k, [60 - 18], cos_t, sin_t).astype(np.float64)[0])
    assert abs(other - dots[0]) > 1e-3                                                  # and on nothing less


def test_rope_pairings_are_a_channel_permutation_apart():
    g = rnd(73)
    d, n = 12, 9
    rows = g.standard_normal((n, d)).astype(np.float32)
    cos_t, sin_t = _tables(32, d)
    pos = g.integers(0, 32, n)
    # interleaved channels 2c, 2c + 1 hold what the half layout keeps in channels c, c + d/2
    inter_in = np.empty_like(rows)
    inter_in[:, 0::2], inter_in[:, 1::2] = rows[:, :d // 2], rows[:, d // 2:]
    inter = oracle.rope_rows(inter_in, pos, cos_t, sin_t, True)
    ref = oracle.rope_rows(rows, pos, cos_t, sin_t, False)
    assert (inter[:, 0::2] == ref[:, :d // 2]).all() and (inter[:, 1::2] == ref[:, d // 2:]).all()


def test_cycle_with_rope_scores_rotated_keys_and_moves_unrotated_rows():
    from paper_2410_01518_b200 import inputs
    g = rnd(74)
    L, B, Hq, Hkv, P, d, N, keep, T = 1, 2, 4, 2, 3, 8, 20, 9, 4
    Q = g.standard_normal((L, B, Hq, P, d)).astype(np.float32)
    K = g.standard_normal((L, B, Hkv, N, d)).astype(np.float32)
    V = g.standard_normal((L, B, Hkv, N, d)).astype(np.float32)
    aux = g.random((B, N)).astype(np.float32)
    cos_t, sin_t = inputs.make_rope_table(N, d, "f32")
    out = oracle.cycle(Q, K, V, aux, keep, T, rope=(cos_t, sin_t, False))
    Kr = oracle.rope_rows(K, np.arange(N), cos_t, sin_t)
    plain = oracle.cycle(Q, Kr, V, aux, keep, T)
    np.testing.assert_array_equal(out["u"], plain["u"])
    assert (out["idx"] == plain["idx"]).all()
    for unit in range(L * B * Hkv):
        src = K.reshape(-1, N, d)[unit][out["idx"][unit]]
        assert (out["K"][unit] == src).all()                                           # unrotated rows move
        assert (out["K_rot"][unit] == oracle.rope_rows(src, np.arange(keep), cos_t, sin_t)).all()   # new positions
    assert not np.allclose(out["u"], oracle.cycle(Q, K, V, aux, keep, T)["u"])


# ---------------------------------------------------------------- generation over the pot
def test_decode_attention_closed_forms_and_library():
    torch = pytest.importorskip("torch")
    from scipy.special import logsumexp
    g = rnd(80)
    L, B, Hq, Hkv, d, N = 2, 2, 6, 2, 16, 37
    q = g.standard_normal((L, B, Hq, d)).astype(np.float32) * 2
    K = g.standard_normal((L, B, Hkv, N, d)).astype(np.float32)
    V = g.standard_normal((L, B, Hkv, N, d)).astype(np.float32)
    out, lse = oracle.decode_attention(q, K, V)
    G = Hq // Hkv
    for l in range(L):
        for b in range(B):
            for h in range(Hq):
                kv = h // G                                       # query head h reads KV head h // G
                s = K[l, b, kv].astype(np.float64) @ q[l, b, h].astype(np.float64) / np.sqrt(d)
                np.testing.assert_allclose(lse[l, b, h], logsumexp(s), rtol=1e-12)
                ref = torch.nn.functional.scaled_dot_product_attention(
                    torch.from_numpy(q[l, b, h].astype(np.float64))[None, None, :],
                    torch.from_numpy(K[l, b, kv].astype(np.float64))[None], torch.from_numpy(V[l, b, kv].astype(np.float64))[None])
                np.testing.assert_allclose(out[l, b, h], ref[0, 0].numpy(), rtol=1e-10, atol=1e-12)
    # one row: its value comes back; equal keys: the mean value; only the first n rows count
    o1, l1 = oracle.decode_attention(q, K, V, n=1)
    for h in range(Hq):
        np.testing.assert_allclose(o1[0, 0, h], V[0, 0, h // G, 0], rtol=1e-14)
    Ke = np.broadcast_to(K[:, :, :, :1], K.shape).copy()
    oe, le = oracle.decode_attention(q, Ke, V)
    np.testing.assert_allclose(oe[1, 1, 4], V[1, 1, 4 // G].astype(np.float64).mean(axis=0), rtol=1e-12)
    np.testing.assert_allclose(le - np.log(N), oracle.decode_attention(q, Ke, V, n=1)[1], rtol=1e-12)
    perm = g.permutation(N)                                       # the order of the slots does not matter
    op, lp = oracle.decode_attention(q, K[:, :, :, perm], V[:, :, :, perm])
    np.testing.assert_allclose(op, out, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(lp, lse, rtol=1e-12)
