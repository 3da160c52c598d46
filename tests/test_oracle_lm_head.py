"""Pins of the oracle's language-model head and of the verification algorithm on fp64 logits
(Algorithm 1, verification phase: p_V(. | x^D) for all positions, then A(p_D, p_V, x^D)).

Expected values come from special cases that need no arithmetic (identity and one-hot weights),
from numpy's fp64 matmul, and from the bf16 form of the oracle where the logits are exactly
representable; never from the CUDA library."""
import numpy as np

from paper_2604_05250_b200 import synth

KL, CONF, PROB = 1, 2, 0x100


def bits(x):
    return synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def f64(b):
    return synth.bf16_bits_to_f32(b).astype(np.float64)


def test_identity_weights_return_the_hidden_state(oracle_mod):
    rng = np.random.default_rng(0)
    h = bits(rng.standard_normal((7, 48)))
    w = bits(np.eye(48))
    np.testing.assert_array_equal(oracle_mod.lm_head(h, w), f64(h))


def test_one_hot_weight_rows_pick_and_scale(oracle_mod):
    rng = np.random.default_rng(1)
    rows, K, V = 5, 32, 77
    h = bits(rng.standard_normal((rows, K)))
    pick = rng.integers(0, K, size=V)
    scale = np.array([0.5, -2.0, 4.0])[rng.integers(0, 3, size=V)]
    w = np.zeros((V, K), dtype=np.float32)
    w[np.arange(V), pick] = scale
    got = oracle_mod.lm_head(h, bits(w))
    np.testing.assert_array_equal(got, f64(h)[:, pick] * scale[None, :])      # exact: powers of two


def test_matches_numpy_matmul_and_skips_unflagged_rows(oracle_mod):
    rng = np.random.default_rng(2)
    rows, K, V = 9, 130, 61
    h = bits(rng.standard_normal((rows, K)))
    w = bits(rng.standard_normal((V, K)) / np.sqrt(K))
    ref = f64(h) @ f64(w).T
    got = oracle_mod.lm_head(h, w)
    assert np.abs(got - ref).max() < 1e-12
    # transposing the roles must change the result (a swapped operand would pass a symmetric case only)
    assert np.abs(oracle_mod.lm_head(h, w) - (f64(w) @ f64(h).T).T).max() < 1e-12
    flags = np.array([1, 0, 1, 1, 0, 0, 1, 1, 1], dtype=np.uint8)
    got = oracle_mod.lm_head(h, w, flags)
    assert (got[flags == 0] == 0).all() and np.abs(got[flags == 1] - ref[flags == 1]).max() < 1e-12


def test_fp64_form_of_the_algorithm_equals_the_bf16_form_on_representable_logits(oracle_mod):
    dra, ver, tokens, flags = synth.verify_inputs(2, 20, 96, 13, 0.3, seed=3)
    for mode, k in ((KL, 3), (CONF, 2), (KL | PROB, 0), (CONF | PROB, 4), (0, 0)):
        a = oracle_mod.verify(dra if (mode & 0xFF) == KL else None, ver, tokens, flags, mode, 0.5, k, 11)
        b = oracle_mod.verify_f64(f64(dra) if (mode & 0xFF) == KL else None, f64(ver), tokens, flags, mode, 0.5, k, 11)
        for key in ("out_tokens", "out_mask", "out_score", "exempt"):
            np.testing.assert_array_equal(a[key], b[key])


def test_head_then_verify_with_identity_weights_is_verify(oracle_mod):
    """hidden = the logits themselves, weight = identity: the fused form must give what the
    algorithm gives on those logits, in both the rounded and the unrounded reading."""
    V = 64
    dra, ver, tokens, flags = synth.verify_inputs(2, 10, V, 7, 0.3, seed=4)
    w = bits(np.eye(V))
    ref = oracle_mod.verify(dra, ver, tokens, flags, KL, 0.5, 2, 5)
    for rounded in (False, True):
        got = oracle_mod.lm_head_verify(dra, w, ver, w, tokens, flags, KL, 0.5, 2, 5, round_logits=rounded)
        for key in ("out_tokens", "out_mask", "out_score"):
            np.testing.assert_array_equal(got[key], ref[key])
    # the gap between the two largest verifier logits, by brute force
    lv = f64(ver)
    for b in range(2):
        for i in range(10):
            if flags[b, i]:
                top = np.sort(lv[b, i])[-2:]
                assert got["top2_gap"][b, i] == top[1] - top[0]


def test_rounding_the_logits_is_a_different_reading(oracle_mod):
    rng = np.random.default_rng(6)
    B, P, K, V = 1, 6, 64, 200
    hv = bits(rng.standard_normal((B, P, K)))
    wv = bits(rng.standard_normal((V, K)) * 0.3)
    tokens = np.zeros((B, P), dtype=np.int32)
    flags = np.ones((B, P), dtype=np.uint8)
    exact = oracle_mod.lm_head_verify(None, None, hv, wv, tokens, flags, CONF, 0.5, 0, 0)
    rounded = oracle_mod.lm_head_verify(None, None, hv, wv, tokens, flags, CONF, 0.5, 0, 0, round_logits=True)
    # confidences agree to about bf16 precision of the logits, not better
    rel = np.abs(exact["out_score"] - rounded["out_score"]) / exact["out_score"]
    assert 1e-6 < rel.max() < 5e-2
    # and the rounded path is exactly verify() on the rounded logits
    lv = oracle_mod.lm_head(hv.reshape(P, K), wv)
    ref = oracle_mod.verify(None, bits(lv).reshape(B, P, V), tokens, flags, CONF, 0.5, 0, 0)
    np.testing.assert_array_equal(rounded["out_score"], ref["out_score"])
