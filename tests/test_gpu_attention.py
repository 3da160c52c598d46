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


def test_peaked_rows(dd, oracle_mod):
    """One-hot-like scores: large logits exercise the running-maximum update."""
    q, k, v = synth.attention_inputs(1, 2, 512, 128, seed=6, planted=True, strength=6.0)
    got = run_gpu(dd, q, k, v, 128 ** -0.5)
    ref = oracle_mod.attention(q, k, v, 128 ** -0.5)
    check_attention(got, ref)


def test_bitwise_repeatability(dd):
    q, k, v = synth.attention_inputs(2, 4, 640, 128, seed=7)
    first = run_gpu(dd, q, k, v, 128 ** -0.5)
    for _ in range(3):
        assert np.array_equal(first, run_gpu(dd, q, k, v, 128 ** -0.5))
