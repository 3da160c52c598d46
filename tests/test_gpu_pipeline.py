"""Algorithm 1 end to end: the library's loop (dd_unmask / dd_verify on the GPU) against the
oracle's loop on the CPU, with the same toy drafter and verifier on both sides."""
import numpy as np
import pytest

from paper_2604_05250_b200 import synth
from tests._toy_models import ToyModel
from tests._parity import to_torch_bf16

pytestmark = pytest.mark.gpu
TRUST, KL, CONF = 0, 1, 2
MASK_ID, V = 63, 64


@pytest.fixture(scope="module")
def dd():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2604_05250_b200 import binding, build
    build.build()
    binding.lib()
    return binding


def problem(seed, B=3, P=40, prompt=8):
    rng = np.random.default_rng(seed)
    target = rng.integers(0, V - 1, size=(B, P)).astype(np.int32)     # MASK_ID never is a target
    start = np.full((B, P), MASK_ID, dtype=np.int32)
    start[:, :prompt] = target[:, :prompt]
    drafter = ToyModel(target, V, MASK_ID, seed + 1, wrong_share=0.2, base=1.0, gain=4.0)
    verifier = ToyModel(target, V, MASK_ID, seed + 2, wrong_share=0.0, base=3.0, gain=6.0)
    return target, start, drafter, verifier


def on_device(model):
    def call(tokens):
        return to_torch_bf16(model(tokens.cpu().numpy()), "cuda")
    return call


@pytest.mark.parametrize("mode,tau,k,K", [(TRUST, 0.0, 0, 2), (KL, 0.5, 2, 3), (CONF, 0.6, 1, 4),
                                          (KL | 0x100, 0.0, 1, 2), (CONF | 0x200, 0.9, 3, 1)])
def test_loop_matches_oracle_loop(dd, oracle_mod, mode, tau, k, K):
    import torch
    from paper_2604_05250_b200.pipeline import dualdiffusion_generate
    target, start, drafter, verifier = problem(5)
    ref_x, ref_stats, near = oracle_mod.dualdiffusion_loop(drafter, verifier, start, MASK_ID, K, mode, tau, k,
                                                           seed=9, unmask_tau=0.7, unmask_k=2, max_cycles=200)
    assert near == 0, "the toy problem was meant to keep every decision away from its boundary"
    assert ref_stats["cycles"] < 200 and not (ref_x == MASK_ID).any()
    x, stats = dualdiffusion_generate(on_device(drafter), on_device(verifier), torch.from_numpy(start).cuda(),
                                      MASK_ID, K, mode, tau, k, seed=9, unmask_tau=0.7, unmask_k=2, max_cycles=200)
    assert dd.verify_status() == 0
    np.testing.assert_array_equal(x.cpu().numpy(), ref_x)
    for key in ("cycles", "drafter_calls", "verifier_calls", "unmasked_by_drafter", "remasked_by_verifier",
                "masked_after_cycle"):
        assert getattr(stats, key) == ref_stats[key], key
    if (mode & 0xFF) == TRUST:
        assert stats.remasked_by_verifier == 0
    if not mode & 0x200:
        # kept positions carry the verifier's token, and the toy verifier knows the target
        np.testing.assert_array_equal(x.cpu().numpy(), target)
