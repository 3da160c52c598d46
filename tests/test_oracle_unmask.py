"""Pins of the unmask oracle (Algorithm 1's Unmask: confidence threshold or fixed number per step).

Expected values are written down by hand for small cases or come from scipy's fp64 softmax
and numpy's sort on random inputs; none comes from the oracle or from the CUDA library.
"""
import numpy as np
import scipy.special

from paper_2604_05250_b200 import synth

MASK_ID = 99


def bits(x):
    return synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def f64(b):
    return synth.bf16_bits_to_f32(b).astype(np.float64)


def peaked_row(V, token, logit):
    row = np.zeros(V, dtype=np.float32)
    row[token] = logit
    return row


def hand_case():
    """One sequence, V = 4, five positions; confidences 1/(1+3e^-l) for a peak of height l."""
    V = 4
    peaks = [(2, 6.0), (0, 1.0), (3, 3.0), (1, 0.0), (2, 3.0)]      # (argmax token, peak logit)
    logits = bits(np.stack([peaked_row(V, t, l) for t, l in peaks])[None])
    conf = np.array([1.0 / (1.0 + 3.0 * np.exp(-l)) for _, l in peaks])   # 0.9926, 0.4754, 0.8700, 0.25, 0.8700
    tokens = np.full((1, 5), MASK_ID, dtype=np.int32)
    flags = np.array([[1, 1, 1, 1, 0]], dtype=np.uint8)
    tokens[0, 4] = 7                                                # already decoded: passes through
    return logits, tokens, flags, conf, [t for t, _ in peaks]


def test_threshold_rule_by_hand(oracle_mod):
    logits, tokens, flags, conf, best = hand_case()
    r = oracle_mod.unmask(logits, tokens, flags, tau=0.8, k=0)
    np.testing.assert_array_equal(r["out_mask"], [[0, 1, 0, 1, 0]])
    np.testing.assert_array_equal(r["out_tokens"], [[best[0], MASK_ID, best[2], MASK_ID, 7]])
    np.testing.assert_allclose(r["out_conf"][0, :4], conf[:4], rtol=0, atol=1e-12)
    assert r["out_conf"][0, 4] == 0.0
    # constant logits: the first token wins the tie, confidence 1/V
    r = oracle_mod.unmask(bits(np.zeros((1, 1, 4))), np.array([[MASK_ID]], dtype=np.int32),
                          np.array([[1]], dtype=np.uint8), tau=0.25, k=0)
    assert r["out_tokens"][0, 0] == 0 and r["out_mask"][0, 0] == 0 and r["out_conf"][0, 0] == 0.25


def test_fixed_number_per_step_by_hand(oracle_mod):
    logits, tokens, flags, conf, best = hand_case()
    # an unreachable threshold leaves the count rule alone: the two most confident masked positions
    r = oracle_mod.unmask(logits, tokens, flags, tau=np.inf, k=2)
    np.testing.assert_array_equal(r["out_mask"], [[0, 1, 0, 1, 0]])
    r = oracle_mod.unmask(logits, tokens, flags, tau=np.inf, k=3)
    np.testing.assert_array_equal(r["out_mask"], [[0, 0, 0, 1, 0]])
    # k beyond the number of masked positions unmasks them all; k = 0 with an unreachable tau none
    assert oracle_mod.unmask(logits, tokens, flags, tau=np.inf, k=9)["out_mask"].sum() == 0
    assert oracle_mod.unmask(logits, tokens, flags, tau=np.inf, k=0)["out_mask"].sum() == 4
    # a threshold that nothing reaches, with k = 1: the single most confident position makes progress
    r = oracle_mod.unmask(logits, tokens, flags, tau=0.999, k=1)
    np.testing.assert_array_equal(r["out_mask"], [[0, 1, 1, 1, 0]])


def test_equal_confidences_go_to_the_lower_position(oracle_mod):
    V = 4
    logits = bits(np.stack([peaked_row(V, 1, 2.0)] * 4)[None])
    tokens = np.full((1, 4), MASK_ID, dtype=np.int32)
    flags = np.ones((1, 4), dtype=np.uint8)
    r = oracle_mod.unmask(logits, tokens, flags, tau=np.inf, k=2)
    np.testing.assert_array_equal(r["out_mask"], [[0, 0, 1, 1]])


def test_random_inputs_against_library_softmax_and_sort(oracle_mod):
    rng = np.random.default_rng(5)
    B, P, V, k, tau = 3, 40, 50, 6, 0.35
    logits = bits(rng.standard_normal((B, P, V)) * 3.0)
    flags = (rng.random((B, P)) < 0.7).astype(np.uint8)
    tokens = np.full((B, P), MASK_ID, dtype=np.int32)
    r = oracle_mod.unmask(logits, tokens, flags, tau=tau, k=k)
    p = scipy.special.softmax(f64(logits), axis=-1)
    conf, best = p.max(-1), p.argmax(-1)
    tau32 = float(np.float32(tau))
    for b in range(B):
        idx = np.flatnonzero(flags[b])
        order = idx[np.lexsort((idx, -conf[b, idx]))]              # confidence descending, position ascending
        chosen = set(order[:k].tolist()) | set(idx[conf[b, idx] >= tau32].tolist())
        want_mask = np.array([1 if (flags[b, i] and i not in chosen) else 0 for i in range(P)])
        strict = r["exempt"][b] == 0
        np.testing.assert_array_equal(r["out_mask"][b][strict], want_mask[strict])
        unm = (want_mask == 0) & (flags[b] == 1) & strict
        np.testing.assert_array_equal(r["out_tokens"][b][unm], best[b][unm])
    np.testing.assert_allclose(r["out_conf"], conf * flags, rtol=1e-12, atol=0)
    assert r["exempt"].sum() <= 2


def test_raising_the_threshold_never_unmasks_more(oracle_mod):
    rng = np.random.default_rng(6)
    logits = bits(rng.standard_normal((2, 30, 20)) * 4.0)
    flags = np.ones((2, 30), dtype=np.uint8)
    tokens = np.full((2, 30), MASK_ID, dtype=np.int32)
    prev = None
    for tau in [0.0, 0.2, 0.5, 0.9, 1.0, np.inf]:
        m = oracle_mod.unmask(logits, tokens, flags, tau=tau, k=3)["out_mask"]
        if prev is not None:
            assert (m >= prev).all()
        prev = m
    assert oracle_mod.unmask(logits, tokens, flags, tau=0.0, k=0)["out_mask"].sum() == 0
    assert ((1 - prev).sum(axis=1) == 3).all()
