"""Pins of the verification oracle (Section 3.2, Eq. 4-7, Algorithm 1's A).

Expected values come from closed forms, invariants, an fp64 library routine on
tiny inputs, published Philox vectors, and brute-force restatements written
here in plain Python; never from the oracle itself or the CUDA library.
"""
import math
import os

import numpy as np
import pytest
import scipy.special

from paper_2604_05250_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
TRUST, KL, CONF = 0, 1, 2
PROB, EMIT_DRAFTER = 0x100, 0x200


def bits(x):
    return synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def f64(b):
    return synth.bf16_bits_to_f32(b).astype(np.float64)


def golden(name):
    with open(os.path.join(GOLDEN, "closed_forms.txt")) as fh:
        for line in fh:
            if line.startswith(name + " "):
                return [float(t) for t in line.split()[1:]]
    raise KeyError(name)


def rand_rows(n, V, seed, sigma=2.0):
    rng = np.random.default_rng(seed)
    return bits(sigma * rng.standard_normal((n, V)))


# --------------------------------------------------------------------------- Philox


def test_philox_known_answers(oracle_mod):
    n = 0
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            w = [int(t, 16) for t in line.split()]
            out = oracle_mod.philox4x32_10(w[0:4], w[4:6])
            assert [int(x) for x in out] == w[6:10]
            n += 1
    assert n == 3


def test_uniform_mapping(oracle_mod):
    # u = (first word >> 8) * 2^-24 with counter (i, b, 0, 0) and key = seed halves
    seed = 0x0123456789ABCDEF
    for b, i in [(0, 0), (3, 17), (15, 255)]:
        w = oracle_mod.philox4x32_10([i, b, 0, 0], [seed & 0xFFFFFFFF, seed >> 32])
        assert oracle_mod.uniform(seed, b, i) == (int(w[0]) >> 8) / 2.0 ** 24
    us = np.array([oracle_mod.uniform(7, 0, i) for i in range(4000)])
    assert 0.0 <= us.min() and us.max() < 1.0
    assert abs(us.mean() - 0.5) < 0.02 and abs(us.var() - 1 / 12) < 0.01
    # distinct (b, i) and distinct seeds give distinct streams
    assert oracle_mod.uniform(7, 0, 1) != oracle_mod.uniform(7, 1, 0)
    assert oracle_mod.uniform(7, 0, 1) != oracle_mod.uniform(8, 0, 1)
    assert oracle_mod.uniform(1 << 32, 0, 1) != oracle_mod.uniform(1, 0, 1)


# --------------------------------------------------------------------------- per-position scores


def test_kl_of_identical_rows_is_zero(oracle_mod):
    rows = rand_rows(4, 300, 0)
    for r in rows:
        _, _, kl = oracle_mod.row_scores(r, r)
        assert kl == 0.0 or abs(kl) < 1e-15


def test_kl_nonnegative_and_asymmetric(oracle_mod):
    d = rand_rows(16, 257, 1)
    v = rand_rows(16, 257, 2)
    for i in range(16):
        kl_dv = oracle_mod.row_scores(d[i], v[i])[2]
        kl_vd = oracle_mod.row_scores(v[i], d[i])[2]
        assert kl_dv > 0 and kl_vd > 0
        assert abs(kl_dv - kl_vd) > 1e-6        # direction matters: KL(p_D || p_V)


def test_two_token_closed_forms(oracle_mod):
    a, c, kl = oracle_mod.row_scores(bits([1.0, 0.0]), bits([0.0, 0.0]))
    assert a == 0 and c == 0.5
    assert abs(kl - golden("kl_two_tokens")[0]) < 1e-15
    a, c, _ = oracle_mod.row_scores(None, bits([0.0, 2.0]))
    assert a == 1 and abs(c - golden("conf_two_tokens")[0]) < 1e-15
    # general two-token formula: a ln(a/b) + (1-a) ln((1-a)/(1-b)) with sigmoid probabilities
    for xd, xv in [(0.5, -1.0), (-3.0, 2.0), (4.0, 4.0)]:
        pa = 1 / (1 + math.exp(-xd))
        pb = 1 / (1 + math.exp(-xv))
        ref = pa * math.log(pa / pb) + (1 - pa) * math.log((1 - pa) / (1 - pb))
        kl = oracle_mod.row_scores(bits([xd, 0.0]), bits([xv, 0.0]))[2]
        assert abs(kl - ref) < 1e-14


def test_constant_logits(oracle_mod):
    V = 640
    a, c, kl = oracle_mod.row_scores(bits(np.full(V, 3.0)), bits(np.full(V, -1.0)))
    assert a == 0                                   # lowest index among exact ties
    assert abs(c - 1.0 / V) < 1e-15 and abs(kl) < 1e-13


def test_confidence_bounds_and_shift_invariance(oracle_mod):
    V = 512
    d = f64(rand_rows(8, V, 3)).astype(np.float32)
    v = f64(rand_rows(8, V, 4)).astype(np.float32)
    for i in range(8):
        a0, c0, k0 = oracle_mod.row_scores(bits(d[i]), bits(v[i]))
        assert 1.0 / V <= c0 <= 1.0
        # shifts by powers of two keep every entry representable in bf16 here? not in general,
        # so shift in integer steps on integer-valued rows
        di = np.round(d[i] * 4) / 4
        vi = np.round(v[i] * 4) / 4
        a1, c1, k1 = oracle_mod.row_scores(bits(di), bits(vi))
        a2, c2, k2 = oracle_mod.row_scores(bits(di + 8.0), bits(vi - 4.0))
        assert a1 == a2 and abs(c1 - c2) < 1e-13 and abs(k1 - k2) < 1e-12
        del a0, k0


@pytest.mark.parametrize("V", [2, 7, 1000])
def test_matches_library_log_softmax_and_rel_entr(oracle_mod, V):
    d = rand_rows(5, V, 5)
    v = rand_rows(5, V, 6)
    for i in range(5):
        a, c, kl = oracle_mod.row_scores(d[i], v[i])
        lp_d = scipy.special.log_softmax(f64(d[i]))
        lp_v = scipy.special.log_softmax(f64(v[i]))
        ref_kl = scipy.special.rel_entr(np.exp(lp_d), np.exp(lp_v)).sum()
        assert abs(kl - ref_kl) < 1e-12
        assert abs(c - np.exp(lp_v).max()) < 1e-14
        assert a == int(np.argmax(f64(v[i])))


def test_tokens_the_drafter_excludes_add_nothing(oracle_mod):
    """Logit -inf (a banned or padded vocabulary entry) is p(x) = 0.  Eq. 5 is a sum over the
    support of p_D (0 ln 0 = 0): an entry the drafter excludes contributes no term, an entry both
    models exclude might as well not exist, an entry only the verifier excludes makes the
    divergence infinite."""
    V = 40
    d = f64(rand_rows(1, V, 8)[0])
    v = f64(rand_rows(1, V, 9)[0])
    d[[3, 17, 30]] = -np.inf
    v[[17, 30]] = -np.inf               # excluded by both
    a, c, kl = oracle_mod.row_scores(bits(d), bits(v))
    lp_d = scipy.special.log_softmax(f64(bits(d)))
    lp_v = scipy.special.log_softmax(f64(bits(v)))
    ref = scipy.special.rel_entr(np.exp(lp_d), np.exp(lp_v)).sum()
    assert np.isfinite(kl) and abs(kl - ref) < 1e-12
    # without the entries both models exclude, the same rows give the same number
    keep = np.isfinite(d) | np.isfinite(v)
    assert keep.sum() == V - 2
    sub = oracle_mod.row_scores(bits(d[keep]), bits(v[keep]))[2]
    assert abs(kl - sub) < 1e-12
    assert abs(c - np.exp(lp_v).max()) < 1e-14 and a == int(np.argmax(f64(bits(v))))
    v[5] = -np.inf                      # p_D(5) > 0 = p_V(5)
    assert oracle_mod.row_scores(bits(d), bits(v))[2] == np.inf


def test_argmax_lowest_index_on_ties(oracle_mod):
    row = np.zeros(100, dtype=np.float32)
    row[[13, 57, 99]] = 9.0
    a, _, _ = oracle_mod.row_scores(None, bits(row))
    assert a == 13


# --------------------------------------------------------------------------- decisions


def tiny_case(P=12, V=64, seed=0, nflag=None):
    rng = np.random.default_rng(seed)
    ver = bits(2.0 * rng.standard_normal((1, P, V)))
    dra = bits(f64(ver) + rng.standard_normal((1, P, V)) * rng.uniform(0.1, 3.0, size=(1, P, 1)))
    tokens = rng.integers(0, V, size=(1, P)).astype(np.int32)
    flags = np.ones((1, P), dtype=np.uint8)
    if nflag is not None:
        flags[:] = 0
        flags[0, rng.choice(P, nflag, replace=False)] = 1
    return dra, ver, tokens, flags


def test_trust_mode_is_bruteforce_argmax_and_never_remasks(oracle_mod):
    dra, ver, tokens, flags = tiny_case(P=20, V=33, seed=1, nflag=13)
    ver_f = f64(ver)
    ver_f[0, 3, 5] = ver_f[0, 3, 20] = 50.0          # an exact tie at the maximum
    ver = bits(ver_f)
    r = oracle_mod.verify(dra, ver, tokens, flags, TRUST, 0.5, 4, 0)
    assert not r["out_mask"].any() and not r["exempt"].any()
    for i in range(20):
        if flags[0, i]:
            row = list(f64(ver)[0, i])
            assert r["out_tokens"][0, i] == row.index(max(row))
        else:
            assert r["out_tokens"][0, i] == tokens[0, i]
            assert r["out_score"][0, i] == 0.0
    if flags[0, 3]:
        assert r["out_tokens"][0, 3] == 5
    # Eq. 4 literally: the drafter's sequence comes back unchanged
    r = oracle_mod.verify(dra, ver, tokens, flags, TRUST | EMIT_DRAFTER, 0.5, 4, 0)
    np.testing.assert_array_equal(r["out_tokens"], tokens)
    assert not r["out_mask"].any()


def test_kl_threshold_rule_handbuilt(oracle_mod):
    # four positions, |V| = 2, verifier uniform; KL known from the two-token closed form
    V = 2
    xs = [0.0, 1.0, 3.0, 6.0]                        # drafter logit gaps
    dra = bits(np.array([[[x, 0.0] for x in xs]]))
    ver = bits(np.zeros((1, 4, V)))
    tokens = np.array([[1, 1, 1, 1]], dtype=np.int32)
    flags = np.ones((1, 4), dtype=np.uint8)
    kls = []
    for x in xs:
        a = 1 / (1 + math.exp(-x))
        kls.append(a * math.log(2 * a) + (1 - a) * math.log(2 * (1 - a)) if x else 0.0)
    tau = 0.3
    r = oracle_mod.verify(dra, ver, tokens, flags, KL, tau, 0, 0)
    np.testing.assert_allclose(r["out_score"][0], kls, atol=1e-14)
    assert list(r["out_mask"][0]) == [int(v > tau) for v in kls] == [0, 0, 1, 1]
    # remasked positions return the caller's token, kept ones the verifier argmax (index 0)
    assert list(r["out_tokens"][0]) == [0, 0, 1, 1]
    # equality keeps: "remask iff KL > tau" is strict
    tau_eq = float(np.float32(kls[2]))
    r = oracle_mod.verify(dra, ver, tokens, flags, KL, tau_eq, 0, 0)
    assert r["out_mask"][0, 2] == int(kls[2] > tau_eq)
    assert r["exempt"][0, 2] == 1 and r["exempt"][0, 0] == 0


def test_conf_threshold_rule_handbuilt(oracle_mod):
    gaps = [0.0, 1.0, 2.0, 4.0]
    ver = bits(np.array([[[0.0, g] for g in gaps]]))
    conf = [1 / (1 + math.exp(-g)) for g in gaps]
    tokens = np.zeros((1, 4), dtype=np.int32)
    flags = np.ones((1, 4), dtype=np.uint8)
    r = oracle_mod.verify(None, ver, tokens, flags, CONF, 0.8, 0, 0)
    np.testing.assert_allclose(r["out_score"][0], conf, atol=1e-14)
    assert list(r["out_mask"][0]) == [int(c < 0.8) for c in conf] == [1, 1, 0, 0]
    r = oracle_mod.verify(None, ver, tokens, flags, CONF, 0.5, 0, 0)
    assert r["out_mask"][0, 0] == 0                  # c == tau is kept: "c < tau" is strict


def test_threshold_monotonicity(oracle_mod):
    dra, ver, tokens, flags = tiny_case(P=40, V=50, seed=2)
    prev_kl, prev_conf = None, None
    for tau in [0.01, 0.05, 0.2, 0.5, 1.0, 3.0]:
        m_kl = oracle_mod.verify(dra, ver, tokens, flags, KL, tau, 0, 0)["out_mask"].astype(bool)
        m_cf = oracle_mod.verify(dra, ver, tokens, flags, CONF, min(tau, 1.0), 0, 0)["out_mask"].astype(bool)
        if prev_kl is not None:
            assert not (m_kl & ~prev_kl).any()       # raising tau_KL only shrinks the remask set
            assert not (prev_conf & ~m_cf).any()     # raising tau_conf only grows it
        prev_kl, prev_conf = m_kl, m_cf


def test_probabilistic_kl_matches_eq6(oracle_mod):
    dra, ver, tokens, flags = tiny_case(P=10, V=40, seed=3, nflag=6)
    kl = np.array([oracle_mod.row_scores(dra[0, i], ver[0, i])[2] if flags[0, i] else 0.0
                   for i in range(10)])
    pi = kl / kl.sum()
    assert abs(pi.sum() - 1.0) < 1e-12
    hits = np.zeros(10)
    n_seeds = 3000
    for seed in range(n_seeds):
        r = oracle_mod.verify(dra, ver, tokens, flags, KL | PROB, 0.5, 0, seed)
        expect = np.array([flags[0, i] and oracle_mod.uniform(seed, 0, i) < pi[i] for i in range(10)])
        np.testing.assert_array_equal(r["out_mask"][0].astype(bool), expect)
        hits += r["out_mask"][0]
    freq = hits / n_seeds
    sd = np.sqrt(pi * (1 - pi) / n_seeds)
    assert (np.abs(freq - pi) <= 4.5 * sd + 1e-9).all()
    assert hits[flags[0] == 0].sum() == 0


def test_probabilistic_conf_frequency(oracle_mod):
    gaps = [0.0, 1.0, 3.0]
    ver = bits(np.array([[[0.0, g] for g in gaps]]))
    conf = np.array([1 / (1 + math.exp(-g)) for g in gaps])
    tokens = np.zeros((1, 3), dtype=np.int32)
    flags = np.ones((1, 3), dtype=np.uint8)
    hits = np.zeros(3)
    n_seeds = 3000
    for seed in range(n_seeds):
        hits += oracle_mod.verify(None, ver, tokens, flags, CONF | PROB, 0.5, 0, seed)["out_mask"][0]
    p = 1 - conf
    assert (np.abs(hits / n_seeds - p) <= 4.5 * np.sqrt(p * (1 - p) / n_seeds)).all()


@pytest.mark.parametrize("mode", [KL, CONF])
@pytest.mark.parametrize("k", [0, 1, 3, 7, 50])
def test_min_keep_topk_bruteforce(oracle_mod, mode, k):
    """The reading of k: the k most reliable flagged positions are always kept."""
    dra, ver, tokens, flags = tiny_case(P=16, V=30, seed=4, nflag=9)
    # force an exact reliability tie between two flagged positions
    idx = np.flatnonzero(flags[0])
    ver[0, idx[3]] = ver[0, idx[1]]
    dra[0, idx[3]] = dra[0, idx[1]]
    tau = 0.05 if mode == KL else 0.99                # nearly everything fails the rule
    r = oracle_mod.verify(dra, ver, tokens, flags, mode, tau, k, 0)
    score = {}
    for i in idx:
        a, c, kl = oracle_mod.row_scores(dra[0, i], ver[0, i])
        score[i] = (kl, c, a)
    rel = {i: (-score[i][0] if mode == KL else score[i][1]) for i in idx}
    order = sorted(idx, key=lambda i: (-rel[i], i))
    keep = set(order[:k])
    for i in range(16):
        if not flags[0, i]:
            assert r["out_mask"][0, i] == 0 and r["out_tokens"][0, i] == tokens[0, i]
            continue
        fail = score[i][0] > float(np.float32(tau)) if mode == KL else score[i][1] < float(np.float32(tau))
        remask = fail and i not in keep
        assert r["out_mask"][0, i] == int(remask)
        assert r["out_tokens"][0, i] == (tokens[0, i] if remask else score[i][2])
    assert r["out_mask"].sum() <= max(0, len(idx) - k)


def test_exemption_flags_mark_topk_boundary(oracle_mod):
    ver = bits(np.array([[[0.0, 1.0], [0.0, 1.0], [0.0, 2.0], [0.0, 3.0]]]))
    tokens = np.zeros((1, 4), dtype=np.int32)
    flags = np.ones((1, 4), dtype=np.uint8)
    # all fail tau=0.999; k=3 keeps positions 3, 2 and (tie -> lower index) 0; position 1 is remasked
    r = oracle_mod.verify(None, ver, tokens, flags, CONF, 0.999, 3, 0)
    assert list(r["out_mask"][0]) == [0, 1, 0, 0]
    assert list(r["exempt"][0]) == [1, 1, 0, 0]       # the tied pair straddles the boundary


def test_well_separated_topk_boundary_is_not_exempt(oracle_mod):
    """Confidences 0.88, 0.73, 0.95, 0.62 (two-token rows with peaks 2, 1, 3, 0.5): every position
    fails tau = 0.999 and k = 2 keeps positions 2 and 0.  No reliability is within 1e-5 of the one
    across the boundary, so nothing is exempt, the positions at the boundary included."""
    ver = bits(np.array([[[0.0, 2.0], [0.0, 1.0], [0.0, 3.0], [0.0, 0.5]]]))
    tokens = np.zeros((1, 4), dtype=np.int32)
    flags = np.ones((1, 4), dtype=np.uint8)
    r = oracle_mod.verify(None, ver, tokens, flags, CONF, 0.999, 2, 0)
    assert list(r["out_mask"][0]) == [0, 1, 0, 1]
    assert list(r["exempt"][0]) == [0, 0, 0, 0]
    u = oracle_mod.unmask(ver, tokens, flags, np.inf, 2)
    assert list(u["out_mask"][0]) == [0, 1, 0, 1]
    assert list(u["exempt"][0]) == [0, 0, 0, 0]


# Seeds whose uniform for (b, i) = (0, 0) lies next to 1/2: found by a search over the Philox
# mapping pinned above; the tests re-check the distance before using them.
SEEDS_NEAR_HALF = {41794: -4.47e-6, 95032: 3.76e-6}       # inside the 1e-5 band
SEEDS_OFF_HALF = {1782: -4.31e-5, 3545: 2.84e-5}          # outside it


@pytest.mark.parametrize("seed,delta,inside", [(s, d, True) for s, d in SEEDS_NEAR_HALF.items()] +
                         [(s, d, False) for s, d in SEEDS_OFF_HALF.items()])
def test_probabilistic_rules_exemption_band(oracle_mod, seed, delta, inside):
    """The probabilistic rules flag a decision as exempt iff the uniform lies within 1e-5 of the
    remask probability (1 - c for confidence, Eq. 6's share for KL); both are 1/2 exactly here."""
    u0 = oracle_mod.uniform(seed, 0, 0)
    assert abs((u0 - 0.5) - delta) < 1e-7 and (abs(u0 - 0.5) <= 1e-5) == inside
    # confidence: two tokens with equal logits, c = 1/2, remask iff u < 1/2
    ver = bits(np.zeros((1, 1, 2)))
    tokens = np.array([[1]], dtype=np.int32)
    flags = np.ones((1, 1), dtype=np.uint8)
    r = oracle_mod.verify(None, ver, tokens, flags, CONF | PROB, 0.9, 0, seed)
    assert r["out_score"][0, 0] == 0.5
    assert r["out_mask"][0, 0] == (1 if u0 < 0.5 else 0)
    assert r["exempt"][0, 0] == (1 if inside else 0)
    # KL: two positions with the same pair of rows share Eq. 6's mass equally
    dra = bits(np.array([[[2.0, 0.0], [2.0, 0.0]]]))
    ver = bits(np.zeros((1, 2, 2)))
    tokens = np.array([[0, 0]], dtype=np.int32)
    flags = np.ones((1, 2), dtype=np.uint8)
    r = oracle_mod.verify(dra, ver, tokens, flags, KL | PROB, 0.0, 0, seed)
    assert r["out_score"][0, 0] == r["out_score"][0, 1] > 0
    u1 = oracle_mod.uniform(seed, 0, 1)
    assert abs(u1 - 0.5) > 1e-3                         # the second position is far from the boundary
    assert r["out_mask"][0].tolist() == [int(u0 < 0.5), int(u1 < 0.5)]
    assert r["exempt"][0].tolist() == [1 if inside else 0, 0]


def test_unknown_mode_rejected(oracle_mod):
    dra, ver, tokens, flags = tiny_case(P=2, V=4)
    with pytest.raises(ValueError):
        oracle_mod.verify(dra, ver, tokens, flags, 3, 0.5, 0, 0)
    with pytest.raises(ValueError):
        oracle_mod.verify(None, ver, tokens, flags, KL, 0.5, 0, 0)
