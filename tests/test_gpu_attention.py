"""dd_bidir_attention on the GPU against the fp64 CPU oracle, through the C ABI."""
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


def run_gpu(dd, q, k, v, scale, host=False):
    import torch
    dev = None if host else "cuda"
    tq, tk, tv = (to_torch_bf16(x, dev, pin=host) for x in (q, k, v))
    # the output sits between two guard regions that the kernel must leave alone
    g = Guarded(tq.shape, torch.bfloat16, device=dev, pin=host)
    out = dd.bidir_attention(tq, tk, tv, out=g.view, scale=scale, host=host)
    torch.cuda.synchronize()
    assert dd.attention_status() == 0
    g.check("attention output")
    return bf16_tensor_to_f64(out)


def sample_rows(N, per_tile=1):
    """Deterministic row sample that covers every 128-row query tile (so both tiles of every CTA):
    `per_tile` rows at varying offsets inside each tile, plus the first and last rows of the
    first and last tiles.  The same rows are compared in every head of every sequence."""
    fixed = {0, 1, 127, 128, N - 129, N - 128, N - 1, N // 2}
    rng = np.random.default_rng(N)
    rows = {r for r in fixed if 0 <= r < N}
    for t in range((N + 127) // 128):
        lo, hi = 128 * t, min(N, 128 * t + 128)
        rows |= set(int(r) for r in rng.integers(lo, hi, size=per_tile))
    return np.array(sorted(rows), dtype=np.int32)


@pytest.mark.parametrize("cfg", [0, 1])
def test_configs_full_compare(dd, oracle_mod, cfg):
    c = synth.ATTENTION_CONFIGS[cfg]
    q, k, v = synth.attention_config_inputs(cfg)
    scale = c["D"] ** -0.5
    got = run_gpu(dd, q, k, v, scale)
    ref = oracle_mod.attention(q, k, v, scale)
    check_attention(got, ref)


def test_config1_host_entry_point(dd, oracle_mod):
    q, k, v = synth.attention_config_inputs(1)
    rows = sample_rows(1024, 4)
    got = run_gpu(dd, q, k, v, 128 ** -0.5, host=True)
    ref = oracle_mod.attention(q, k, v, 128 ** -0.5, rows=rows)
    check_attention(got[:, :, rows], ref)


def test_config2_batched(dd, oracle_mod):
    q, k, v = synth.attention_config_inputs(2)
    got = run_gpu(dd, q, k, v, 128 ** -0.5)
    rows = sample_rows(512, 4)
    ref = oracle_mod.attention(q, k, v, 128 ** -0.5, rows=rows)
    check_attention(got[:, :, rows], ref)


def test_config3_long_context_planted_structure(dd, oracle_mod):
    q, k, v = synth.attention_config_inputs(3)
    got = run_gpu(dd, q, k, v, 128 ** -0.5)
    rows = sample_rows(8192, 2)          # every one of the 64 query tiles, all 32 heads
    assert len(set((rows // 128).tolist())) == 64
    ref = oracle_mod.attention(q, k, v, 128 ** -0.5, rows=rows)
    check_attention(got[:, :, rows], ref)
    # properties that hold at any size: finite everywhere, inside the convex hull of V per column
    vf = synth.bf16_bits_to_f32(v).astype(np.float64)
    assert np.isfinite(got).all()
    assert (got <= vf.max(axis=2, keepdims=True) + 1e-2).all()
    assert (got >= vf.min(axis=2, keepdims=True) - 1e-2).all()


@pytest.mark.parametrize("N", [256, 1024, 4096, 16384])
def test_config4_sweep(dd, oracle_mod, N):
    B = 16384 // N
    q, k, v = synth.attention_inputs(B, 32, N, 128, synth.config_seed(4))
    got = run_gpu(dd, q, k, v, 128 ** -0.5)
    # at least one row of every 128-row query tile, in all 32 heads of every sequence
    rows = sample_rows(N, 4 if N <= 1024 else 1)
    assert len(set((rows // 128).tolist())) == N // 128
    ref = oracle_mod.attention(q, k, v, 128 ** -0.5, rows=rows)
    check_attention(got[:, :, rows], ref)


@pytest.mark.parametrize("B,H,N,D", [(1, 1, 1, 64), (1, 2, 7, 128), (2, 3, 129, 64), (1, 2, 200, 128),
                                     (1, 1, 383, 128), (2, 2, 640, 64), (1, 3, 1000, 128)])
def test_ragged_and_small_shapes(dd, oracle_mod, B, H, N, D):
    q, k, v = synth.attention_inputs(B, H, N, D, seed=N)
    got = run_gpu(dd, q, k, v, D ** -0.5)
    ref = oracle_mod.attention(q, k, v, D ** -0.5)
    check_attention(got, ref)


def test_constant_values_and_scale_zero(dd, oracle_mod):
    q, k, v = synth.attention_inputs(1, 2, 300, 128, seed=5)
    vc = synth.f32_to_bf16_bits(np.full((1, 2, 300, 128), 1.5, dtype=np.float32))
    got = run_gpu(dd, q, k, vc, 128 ** -0.5)
    assert np.abs(got - 1.5).max() <= 1e-2
    got0 = run_gpu(dd, q, k, v, 0.0)
    ref0 = oracle_mod.attention(q, k, v, 0.0)
    check_attention(got0, ref0)


@pytest.mark.parametrize("strength", [6.0, 10.0])      # 8 % and 49 % of the rows move their reference point
def test_peaked_rows(dd, oracle_mod, strength):
    """One-hot-like scores: row maxima that outgrow the reference point of the row's first tile by
    more than the kernel's step (scores with a standard deviation of 13 nats), so the accumulator in
    tensor memory is rescaled.  A stress input beyond the workload's recipe (strength 3): see
    check_attention's stress bar."""
    q, k, v = synth.attention_inputs(1, 2, 512, 128, seed=6, planted=True, strength=strength)
    got = run_gpu(dd, q, k, v, 128 ** -0.5)
    ref = oracle_mod.attention(q, k, v, 128 ** -0.5)
    check_attention(got, ref, stress=True)


def test_bitwise_repeatability(dd):
    q, k, v = synth.attention_inputs(2, 4, 640, 128, seed=7)
    first = run_gpu(dd, q, k, v, 128 ** -0.5)
    for _ in range(3):
        assert np.array_equal(first, run_gpu(dd, q, k, v, 128 ** -0.5))


# ---- more (head, 256-row block) work items than SMs, each with few key tiles: dd_bidir_attention
# runs these on persistent CTAs that walk over several items

@pytest.mark.parametrize("B,H,N,D", [(6, 32, 200, 64), (5, 32, 440, 128), (3, 64, 256, 128), (2, 96, 130, 64)])
def test_many_short_items(dd, oracle_mod, B, H, N, D):
    import torch
    assert B * H * ((N + 255) // 256) > torch.cuda.get_device_properties(0).multi_processor_count
    q, k, v = synth.attention_inputs(B, H, N, D, seed=1000 + N)
    got = run_gpu(dd, q, k, v, D ** -0.5)
    check_attention(got, oracle_mod.attention(q, k, v, D ** -0.5))


def test_many_short_items_peaked_rows(dd, oracle_mod):
    """Rows whose maximum outgrows the reference point they inherit: the accumulator in tensor
    memory is rescaled in the middle of an item, on CTAs that carry their barriers' phases over
    from the items before.  Same bits as one CTA per item (one sequence per call), and the first
    heads of every sequence against the oracle."""
    import torch
    q, k, v = synth.attention_inputs(5, 32, 512, 128, seed=61, planted=True, strength=6.0)
    tq, tk, tv = (to_torch_bf16(x, "cuda") for x in (q, k, v))
    g = Guarded(tq.shape, torch.bfloat16)
    whole = dd.bidir_attention(tq, tk, tv, out=g.view, scale=128 ** -0.5)
    parts = torch.cat([dd.bidir_attention(tq[i:i + 1].contiguous(), tk[i:i + 1].contiguous(), tv[i:i + 1].contiguous(),
                                          scale=128 ** -0.5) for i in range(5)], dim=0)
    torch.cuda.synchronize()
    assert dd.attention_status() == 0
    g.check("attention output")
    assert torch.equal(whole, parts)
    sub = slice(0, 2)
    ref = oracle_mod.attention(np.ascontiguousarray(q[:, sub]), np.ascontiguousarray(k[:, sub]),
                               np.ascontiguousarray(v[:, sub]), 128 ** -0.5)
    check_attention(bf16_tensor_to_f64(whole[:, sub]), ref, stress=True)


def test_many_short_items_match_one_item_per_cta(dd):
    """The same 320 items in one call (persistent CTAs) and in four calls of 80 (one CTA per
    item): the same arithmetic in the same order, so the same bits."""
    import torch
    q, k, v = synth.attention_inputs(1, 160, 512, 128, seed=62)
    tq, tk, tv = (to_torch_bf16(x, "cuda") for x in (q, k, v))
    whole = dd.bidir_attention(tq, tk, tv)
    parts = [dd.bidir_attention(tq[:, i:i + 40].contiguous(), tk[:, i:i + 40].contiguous(), tv[:, i:i + 40].contiguous())
             for i in range(0, 160, 40)]
    torch.cuda.synchronize()
    assert dd.attention_status() == 0
    assert torch.equal(whole, torch.cat(parts, dim=1))
