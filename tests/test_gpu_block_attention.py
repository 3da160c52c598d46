"""dd_block_attention on the GPU against the fp64 CPU oracle, through the C ABI:
a block of queries over stored keys, ragged key counts, both memory layouts."""
import numpy as np
import pytest

from paper_2604_05250_b200 import synth
from tests._parity import Guarded, bf16_tensor_to_f64, check_attention, to_torch_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dd():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2604_05250_b200 import binding, build
    build.build()
    binding.lib()
    return binding


def block_inputs(B, H, Nq, Nkv, D, seed, planted=False):
    if planted:
        # queries and keys must share the planted subspace: one draw, the first Nq query rows
        assert Nq <= Nkv
        q, k, v = synth.attention_inputs(B, H, Nkv, D, seed, planted=True)
        return np.ascontiguousarray(q[:, :, :Nq]), k, v
    q, _, _ = synth.attention_inputs(B, H, Nq, D, seed)
    _, k, v = synth.attention_inputs(B, H, Nkv, D, seed + 1)
    return q, k, v


def run_gpu(dd, q, k, v, scale, kv_len=None, layout="bhnd"):
    import torch
    tq, tk, tv = (to_torch_bf16(x, "cuda") for x in (q, k, v))
    tl = None if kv_len is None else torch.from_numpy(np.asarray(kv_len, dtype=np.int32)).cuda()
    g = Guarded(tq.shape, torch.bfloat16)        # guard regions on both sides of the output
    out = dd.block_attention(tq, tk, tv, out=g.view, kv_len=tl, layout=layout, scale=scale)
    torch.cuda.synchronize()
    assert dd.attention_status() == 0
    g.check("block attention output")
    return bf16_tensor_to_f64(out)


# query blocks shorter than, equal to and longer than one and two 128-row tiles; key counts
# that end inside a tile, on a tile boundary and span several ring rounds
@pytest.mark.parametrize("B,H,Nq,Nkv,D", [
    (2, 3, 32, 1024, 128), (1, 4, 64, 1000, 128), (2, 2, 128, 130, 128), (1, 2, 200, 700, 64),
    (1, 3, 300, 257, 128), (3, 2, 1, 1, 64), (1, 2, 256, 2048, 128),
])
def test_query_block_over_stored_keys(dd, oracle_mod, B, H, Nq, Nkv, D):
    q, k, v = block_inputs(B, H, Nq, Nkv, D, 100 + Nq)
    scale = D ** -0.5
    got = run_gpu(dd, q, k, v, scale)
    check_attention(got, oracle_mod.block_attention(q, k, v, scale))


def test_ragged_key_counts_and_padding(dd, oracle_mod):
    B, H, Nq, Nkv, D = 6, 2, 96, 640, 128
    q, k, v = block_inputs(B, H, Nq, Nkv, D, 21)
    kv_len = np.array([640, 1, 128, 129, 0, 511], dtype=np.int32)
    # padding holds values that would dominate every row if it were read as keys
    for b in range(B):
        k[b, :, kv_len[b]:] = synth.f32_to_bf16_bits(np.float32(50.0))
        v[b, :, kv_len[b]:] = synth.f32_to_bf16_bits(np.float32(1000.0))
    got = run_gpu(dd, q, k, v, D ** -0.5, kv_len=kv_len)
    ref = oracle_mod.block_attention(q, k, v, D ** -0.5, kv_len=kv_len)
    check_attention(got, ref)
    assert (got[4] == 0).all()                      # no valid key: zero output
    # lengths outside [0, Nkv] are clamped
    got2 = run_gpu(dd, q, k, v, D ** -0.5, kv_len=np.array([9999, 1, 128, 129, -5, 511], dtype=np.int32))
    np.testing.assert_array_equal(got2, got)


@pytest.mark.parametrize("layout", ["bhnd", "bnhd"])
def test_padding_of_nan_and_inf_never_contributes(dd, oracle_mod, layout):
    """Keys and values beyond n_b are padding (Eq. 3 runs over the keys that exist): a cache
    that was never initialised there may hold any bit pattern, NaN and infinities included."""
    B, H, Nq, Nkv, D = 5, 2, 150, 520, 128
    q, k, v = block_inputs(B, H, Nq, Nkv, D, 23)
    kv_len = np.array([520, 1, 129, 383, 512], dtype=np.int32)
    junk = np.array([0x7FC0, 0x7F80, 0xFF80, 0xFFFF], dtype=np.uint16)       # NaN, +inf, -inf, NaN
    for b in range(B):
        n = Nkv - kv_len[b]
        k[b, :, kv_len[b]:] = junk[np.arange(n * D).reshape(n, D) % 4]
        v[b, :, kv_len[b]:] = junk[(np.arange(n * D).reshape(n, D) + 1) % 4]
    ref = oracle_mod.block_attention(q, k, v, D ** -0.5, kv_len=kv_len)
    assert np.isfinite(ref).all()
    if layout == "bnhd":
        q, k, v = (np.ascontiguousarray(a.transpose(0, 2, 1, 3)) for a in (q, k, v))
        ref = np.ascontiguousarray(ref.transpose(0, 2, 1, 3))
    got = run_gpu(dd, q, k, v, D ** -0.5, kv_len=kv_len, layout=layout)
    check_attention(got, ref)


@pytest.mark.parametrize("D", [64, 128])
def test_interleaved_head_layout(dd, oracle_mod, D):
    B, H, Nq, Nkv = 2, 5, 160, 384
    q, k, v = block_inputs(B, H, Nq, Nkv, D, 33)
    kv_len = np.array([384, 200], dtype=np.int32)
    tr = lambda a: np.ascontiguousarray(a.transpose(0, 2, 1, 3))
    got = run_gpu(dd, tr(q), tr(k), tr(v), D ** -0.5, kv_len=kv_len, layout="bnhd")
    ref = oracle_mod.block_attention(tr(q), tr(k), tr(v), D ** -0.5, kv_len=kv_len, layout="bnhd")
    check_attention(got, ref)
    # the same problem in the head-major layout gives the same bits
    got_hm = run_gpu(dd, q, k, v, D ** -0.5, kv_len=kv_len, layout="bhnd")
    np.testing.assert_array_equal(tr(got_hm), got)


def test_square_case_equals_bidirectional_attention(dd):
    """Nq = Nkv with every key valid: the general instantiation (forced by passing kv_len)
    gives the same bits as dd_bidir_attention where every CTA holds two query tiles; a CTA
    with a single query tile splits its keys between the softmax groups, which changes the
    order of the sums but not the result beyond rounding."""
    import torch
    for N, exact in ((512, True), (333, False)):
        q, k, v = synth.attention_inputs(2, 4, N, 128, 5)
        tq, tk, tv = (to_torch_bf16(x, "cuda") for x in (q, k, v))
        a = dd.bidir_attention(tq, tk, tv)
        b = dd.block_attention(tq, tk, tv)
        c = dd.block_attention(tq, tk, tv, kv_len=torch.tensor([N, N + 67], dtype=torch.int32, device="cuda"))
        torch.cuda.synchronize()
        assert dd.attention_status() == 0
        assert torch.equal(a, b)
        if exact:
            assert torch.equal(a, c)
        else:
            assert torch.equal(a[:, :, :256], c[:, :, :256])
            assert (a.float() - c.float()).abs().max().item() <= 4e-3


# ---- the drafter's shape with more (batch, head) items than SMs, key counts differing from
# sequence to sequence

@pytest.mark.parametrize("layout", ["bhnd", "bnhd"])
@pytest.mark.parametrize("D", [64, 128])
def test_many_heads_ragged_keys(dd, oracle_mod, layout, D):
    import torch
    B, H, Nq, Nkv = 12, 16, 32, 600            # 192 items
    assert B * H > torch.cuda.get_device_properties(0).multi_processor_count
    q, k, v = block_inputs(B, H, Nq, Nkv, D, 61)
    # no key, one key, one tile, one key more, an odd number of tiles, all keys; twice, so that
    # consecutive items of a CTA differ in every way
    kv_len = np.array([600, 0, 1, 128, 129, 300, 0, 0, 511, 257, 600, 64], dtype=np.int32)
    junk = np.array([0x7FC0, 0x7F80, 0xFF80, 0xFFFF], dtype=np.uint16)       # NaN, +inf, -inf, NaN
    for b in range(B):
        n = Nkv - kv_len[b]
        k[b, :, kv_len[b]:] = junk[np.arange(n * D).reshape(n, D) % 4]
        v[b, :, kv_len[b]:] = junk[(np.arange(n * D).reshape(n, D) + 1) % 4]
    ref = oracle_mod.block_attention(q, k, v, D ** -0.5, kv_len=kv_len)
    assert np.isfinite(ref).all()
    if layout == "bnhd":
        q, k, v = (np.ascontiguousarray(a.transpose(0, 2, 1, 3)) for a in (q, k, v))
        ref = np.ascontiguousarray(ref.transpose(0, 2, 1, 3))
    got = run_gpu(dd, q, k, v, D ** -0.5, kv_len=kv_len, layout=layout)
    check_attention(got, ref)
    zero = got[[1, 6, 7]] if layout == "bhnd" else got[[1, 6, 7]]
    assert (zero == 0).all()                        # sequences without keys: zero output


@pytest.mark.parametrize("Nq,Nkv", [(1, 1), (128, 1024), (100, 130), (7, 4096)])
def test_many_heads_shapes(dd, oracle_mod, Nq, Nkv):
    B, H, D = 5, 32, 128                        # 160 items, no kv_len: every key counts
    q, k, v = block_inputs(B, H, Nq, Nkv, D, 70 + Nq)
    got = run_gpu(dd, q, k, v, D ** -0.5)
    check_attention(got, oracle_mod.block_attention(q, k, v, D ** -0.5))


def test_peaked_rows_with_planted_structure(dd, oracle_mod):
    q, k, v = block_inputs(1, 2, 128, 1536, 128, 44, planted=True)
    got = run_gpu(dd, q, k, v, 128 ** -0.5, kv_len=np.array([1500], dtype=np.int32))
    check_attention(got, oracle_mod.block_attention(q, k, v, 128 ** -0.5, kv_len=np.array([1500], dtype=np.int32)))


def test_argument_errors(dd):
    import torch
    q = torch.zeros(1, 2, 16, 128, dtype=torch.bfloat16, device="cuda")
    k = torch.zeros(1, 2, 32, 128, dtype=torch.bfloat16, device="cuda")
    L = dd.lib()
    p = lambda t: t.data_ptr()
    assert L.dd_block_attention(p(q), p(k), p(k), p(q), 1, 2, 16, 32, 128, None, 7, 0.1, None) == dd.DD_ERR_INVALID_ARG
    assert L.dd_block_attention(p(q), p(k), p(k), p(q), 1, 2, 0, 32, 128, None, 0, 0.1, None) == dd.DD_ERR_INVALID_ARG
    assert L.dd_block_attention(p(q), p(k), p(k), p(q), 1, 2, 16, 32, 96, None, 0, 0.1, None) == dd.DD_ERR_UNSUPPORTED
    assert L.dd_block_attention(None, p(k), p(k), p(q), 1, 2, 16, 32, 128, None, 0, 0.1, None) == dd.DD_ERR_INVALID_ARG


@pytest.mark.parametrize("layout", ["bhnd", "bnhd"])
def test_drafter_shape_full_size(dd, oracle_mod, layout):
    """The drafter shape bench.py times: 32 queries over 1024 stored keys, B = 16, H = 32, D = 128."""
    B, H, Nq, Nkv, D = 16, 32, 32, 1024, 128
    q, k, v = block_inputs(B, H, Nq, Nkv, D, 77)
    kv_len = np.random.default_rng(3).integers(Nkv // 4, Nkv + 1, size=B).astype(np.int32)
    if layout == "bnhd":
        q, k, v = (np.ascontiguousarray(a.transpose(0, 2, 1, 3)) for a in (q, k, v))
    got = run_gpu(dd, q, k, v, D ** -0.5, kv_len=kv_len, layout=layout)
    check_attention(got, oracle_mod.block_attention(q, k, v, D ** -0.5, kv_len=kv_len, layout=layout))
