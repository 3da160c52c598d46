"""Pins of the block-attention oracle (Eq. 3 for a query block over stored keys).

Expected values come from numpy / scipy fp64 routines on the valid keys, from
truncated and transposed copies of the inputs, and from closed forms; none
comes from the oracle itself or from the CUDA library.
"""
import numpy as np
import pytest
import scipy.special

from paper_2604_05250_b200 import synth


def f64(b):
    return synth.bf16_bits_to_f32(b).astype(np.float64)


def rand_block(B, H, Nq, Nkv, D, seed):
    q, _, _ = synth.attention_inputs(B, H, Nq, D, seed)
    _, k, v = synth.attention_inputs(B, H, Nkv, D, seed + 1)
    return q, k, v


def library_reference(q, k, v, scale, kv_len):
    """softmax(scale q k^T) v over the first kv_len[b] keys, with scipy's softmax (bhnd)."""
    B = q.shape[0]
    out = np.zeros(q.shape, dtype=np.float64)
    for b in range(B):
        n = k.shape[2] if kv_len is None else int(np.clip(kv_len[b], 0, k.shape[2]))
        if n == 0:
            continue
        s = scale * np.einsum("hid,hjd->hij", f64(q[b]), f64(k[b, :, :n]))
        out[b] = np.einsum("hij,hjd->hid", scipy.special.softmax(s, axis=-1), f64(v[b, :, :n]))
    return out


@pytest.mark.parametrize("B,H,Nq,Nkv,D", [(1, 1, 3, 7, 4), (2, 3, 5, 19, 8), (2, 2, 33, 20, 16)])
def test_matches_library_softmax_on_a_query_block(oracle_mod, B, H, Nq, Nkv, D):
    q, k, v = rand_block(B, H, Nq, Nkv, D, 11)
    out = oracle_mod.block_attention(q, k, v, 0.4)
    np.testing.assert_allclose(out, library_reference(q, k, v, 0.4, None), rtol=0, atol=1e-12)


def test_padding_keys_never_contribute(oracle_mod):
    q, k, v = rand_block(3, 2, 6, 25, 8, 12)
    kv_len = np.array([25, 9, 1], dtype=np.int32)
    out = oracle_mod.block_attention(q, k, v, 0.3, kv_len=kv_len)
    np.testing.assert_allclose(out, library_reference(q, k, v, 0.3, kv_len), rtol=0, atol=1e-12)
    # whatever sits in the padding (here: huge keys and values) changes nothing
    k2, v2 = k.copy(), v.copy()
    k2[1, :, 9:] = synth.f32_to_bf16_bits(np.float32(1e30))
    v2[1, :, 9:] = synth.f32_to_bf16_bits(np.float32(-1e30))
    out2 = oracle_mod.block_attention(q, k2, v2, 0.3, kv_len=kv_len)
    np.testing.assert_array_equal(out2, out)
    # one valid key: the output is that key's value row
    np.testing.assert_array_equal(out[2], np.broadcast_to(f64(v)[2, :, :1], out[2].shape))


def test_lengths_are_clamped_and_zero_keys_give_zero(oracle_mod):
    q, k, v = rand_block(3, 1, 4, 10, 8, 13)
    out = oracle_mod.block_attention(q, k, v, 0.5, kv_len=np.array([0, 99, -3], dtype=np.int32))
    assert (out[0] == 0).all() and (out[2] == 0).all()
    np.testing.assert_allclose(out[1], library_reference(q, k, v, 0.5, None)[1], rtol=0, atol=1e-12)


def test_interleaved_head_layout_is_a_transpose(oracle_mod):
    q, k, v = rand_block(2, 3, 5, 12, 8, 14)
    kv_len = np.array([12, 7], dtype=np.int32)
    ref = library_reference(q, k, v, 0.35, kv_len)
    tr = lambda a: np.ascontiguousarray(a.transpose(0, 2, 1, 3))
    out = oracle_mod.block_attention(tr(q), tr(k), tr(v), 0.35, kv_len=kv_len, layout="bnhd")
    np.testing.assert_allclose(out, tr(ref), rtol=0, atol=1e-12)


def test_constant_values_pass_through(oracle_mod):
    q, k, _ = rand_block(1, 2, 9, 30, 8, 15)
    v = synth.f32_to_bf16_bits(np.full((1, 2, 30, 8), -2.25, dtype=np.float32))
    out = oracle_mod.block_attention(q, k, v, 0.3, kv_len=np.array([17], dtype=np.int32))
    np.testing.assert_allclose(out, -2.25, rtol=0, atol=1e-12)


def test_two_key_closed_form(oracle_mod):
    # q.k = (1, 0) -> weights e/(1+e), 1/(1+e)
    bits = synth.f32_to_bf16_bits
    q = bits(np.array([[[[1.0, 0.0]]]], dtype=np.float32))
    k = bits(np.array([[[[1.0, 0.0], [0.0, 0.0], [5.0, 5.0]]]], dtype=np.float32))
    v = bits(np.array([[[[1.0, -2.0], [0.0, 4.0], [100.0, 100.0]]]], dtype=np.float32))
    out = oracle_mod.block_attention(q, k, v, 1.0, kv_len=np.array([2], dtype=np.int32))
    w = np.e / (1.0 + np.e)
    np.testing.assert_allclose(out[0, 0, 0], [w, -2.0 * w + 4.0 * (1 - w)], rtol=0, atol=1e-15)
