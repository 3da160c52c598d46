"""Pins of the attention oracle against what Eq. 3 and the mathematics fix.

None of the expected values here comes from the oracle or from the CUDA
library: they are invariants of a row-stochastic average, closed forms, and an
fp64 library softmax on tiny inputs.
"""
import os

import numpy as np
import pytest
import scipy.special

from paper_2604_05250_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


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


def rand_qkv(B, H, N, D, seed):
    return synth.attention_inputs(B, H, N, D, seed)


def test_softmax_rows_sum_to_one(oracle_mod):
    q, k, _ = rand_qkv(2, 3, 37, 16, 1)
    for (b, h, i) in [(0, 0, 0), (1, 2, 36), (0, 1, 17)]:
        p = oracle_mod.attention_probs(q, k, 0.25, b, h, i)
        assert abs(p.sum() - 1.0) < 1e-12
        assert (p >= 0).all()


def test_two_key_closed_form(oracle_mod):
    q = bits([[[[1.0, 0.0]]]])
    k = bits([[[[1.0, 0.0], [0.0, 0.0]]]])
    v = bits([[[[1.0, -2.0], [0.0, 4.0]]]])
    # N differs between q and k here, so build the N=2 problem with a dummy second query
    q2 = bits([[[[1.0, 0.0], [0.0, 0.0]]]])
    out = oracle_mod.attention(q2, k, v, 1.0)
    np.testing.assert_allclose(out[0, 0, 0], golden("attention_two_keys"), rtol=0, atol=1e-15)
    # the all-zero query weighs both keys equally
    np.testing.assert_allclose(out[0, 0, 1], [0.5, 1.0], rtol=0, atol=1e-15)
    del q


def test_constant_values_pass_through(oracle_mod):
    q, k, _ = rand_qkv(1, 2, 50, 8, 2)
    v = bits(np.full((1, 2, 50, 8), 1.5))
    out = oracle_mod.attention(q, k, v, 0.3)
    np.testing.assert_allclose(out, 1.5, rtol=0, atol=1e-12)


def test_single_key_returns_its_value(oracle_mod):
    q, k, v = rand_qkv(2, 2, 1, 8, 3)
    out = oracle_mod.attention(q, k, v, 0.7)
    np.testing.assert_array_equal(out, f64(v))


def test_zero_keys_give_column_mean(oracle_mod):
    q, _, v = rand_qkv(1, 2, 33, 8, 4)
    k = np.zeros_like(q)
    out = oracle_mod.attention(q, k, v, 1.0)
    mean = f64(v).mean(axis=2, keepdims=True)
    np.testing.assert_allclose(out, np.broadcast_to(mean, out.shape), rtol=0, atol=1e-12)


def test_joint_key_value_permutation_invariance(oracle_mod):
    q, k, v = rand_qkv(1, 2, 41, 16, 5)
    perm = np.random.default_rng(0).permutation(41)
    out = oracle_mod.attention(q, k, v, 0.25)
    out_p = oracle_mod.attention(q, k[:, :, perm], v[:, :, perm], 0.25)
    np.testing.assert_allclose(out_p, out, rtol=0, atol=1e-12)
    # permuting only the keys (not the values) must change the result
    out_bad = oracle_mod.attention(q, k[:, :, perm], v, 0.25)
    assert np.abs(out_bad - out).max() > 1e-3


def test_query_permutation_equivariance(oracle_mod):
    q, k, v = rand_qkv(1, 2, 29, 16, 6)
    perm = np.random.default_rng(1).permutation(29)
    out = oracle_mod.attention(q, k, v, 0.25)
    out_p = oracle_mod.attention(q[:, :, perm], k, v, 0.25)
    np.testing.assert_array_equal(out_p, out[:, :, perm])


def test_one_hot_limit_selects_a_value_row(oracle_mod):
    N = D = 16
    eye = np.eye(N, dtype=np.float32)
    perm = np.random.default_rng(2).permutation(N)
    k = bits(eye[None, None])
    q = bits(64.0 * eye[perm][None, None])          # q_i = 64 * k_{perm[i]}
    _, _, v = rand_qkv(1, 1, N, D, 7)
    out = oracle_mod.attention(q, k, v, 1.0)
    np.testing.assert_allclose(out[0, 0], f64(v)[0, 0][perm], rtol=0, atol=1e-12)


@pytest.mark.parametrize("B,H,N,D,scale", [(1, 1, 5, 3, 1.0), (2, 3, 19, 8, 0.35), (1, 2, 64, 32, 32 ** -0.5)])
def test_matches_library_softmax(oracle_mod, B, H, N, D, scale):
    q, k, v = rand_qkv(B, H, N, D, 8)
    out, lse = oracle_mod.attention(q, k, v, scale, return_lse=True)
    qf, kf, vf = f64(q), f64(k), f64(v)
    s = scale * np.einsum("bhid,bhjd->bhij", qf, kf)
    ref = np.einsum("bhij,bhjd->bhid", scipy.special.softmax(s, axis=-1), vf)
    np.testing.assert_allclose(out, ref, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, scipy.special.logsumexp(s, axis=-1), rtol=0, atol=1e-12)


def test_row_subset_equals_full(oracle_mod):
    q, k, v = rand_qkv(1, 2, 40, 8, 9)
    rows = np.array([0, 7, 39], dtype=np.int32)
    full = oracle_mod.attention(q, k, v, 0.5)
    sub = oracle_mod.attention(q, k, v, 0.5, rows=rows)
    np.testing.assert_array_equal(sub, full[:, :, rows])


def test_scale_is_applied_to_scores(oracle_mod):
    # scale -> 0 flattens the softmax: the output tends to the mean of V
    q, k, v = rand_qkv(1, 1, 20, 8, 10)
    out = oracle_mod.attention(q, k, v, 1e-9)
    np.testing.assert_allclose(out[0, 0], np.broadcast_to(f64(v)[0, 0].mean(0), (20, 8)), atol=1e-6)
