"""Algorithm 1 with the oracle's steps: properties that the paper's loop must have."""
import numpy as np

from paper_2604_05250_b200 import synth
from tests._toy_models import ToyModel

MASK_ID, V = 63, 64


def problem(seed, B=2, P=30, prompt=6, wrong=0.25):
    rng = np.random.default_rng(seed)
    target = rng.integers(0, V - 1, size=(B, P)).astype(np.int32)
    start = np.full((B, P), MASK_ID, dtype=np.int32)
    start[:, :prompt] = target[:, :prompt]
    drafter = ToyModel(target, V, MASK_ID, seed + 1, wrong_share=wrong, base=1.0, gain=4.0)
    verifier = ToyModel(target, V, MASK_ID, seed + 2, wrong_share=0.0, base=3.0, gain=6.0)
    return target, start, drafter, verifier


def test_trust_verifier_accepts_everything_and_needs_the_fewest_cycles(oracle_mod):
    target, start, drafter, verifier = problem(3)
    # fixed number per step: 2 positions per drafter step, K = 3 steps per cycle, 24 masked per sequence
    x, stats, _ = oracle_mod.dualdiffusion_loop(drafter, verifier, start, MASK_ID, 3, 0, 0.0, 0,
                                                unmask_tau=np.inf, unmask_k=2)
    assert not (x == MASK_ID).any() and stats["remasked_by_verifier"] == 0
    assert stats["cycles"] == 4 and stats["verifier_calls"] == 4 and stats["drafter_calls"] == 12
    assert stats["masked_after_cycle"] == [36, 24, 12, 0]
    # the prompt is never touched
    np.testing.assert_array_equal(x[:, :6], target[:, :6])


def test_kl_remasking_terminates_through_the_minimum_keep_and_repairs_the_drafter(oracle_mod):
    target, start, drafter, verifier = problem(4)
    assert (drafter.belief != target).any()
    x, stats, _ = oracle_mod.dualdiffusion_loop(drafter, verifier, start, MASK_ID, 2, 1, 0.5, 1,
                                                unmask_tau=np.inf, unmask_k=3, max_cycles=500)
    assert stats["cycles"] < 500 and not (x == MASK_ID).any()
    assert stats["remasked_by_verifier"] > 0
    np.testing.assert_array_equal(x, target)          # kept positions carry the verifier's token
    # without a minimum keep the same run cannot finish: the drafter's errors are remasked for ever
    x0, stats0, _ = oracle_mod.dualdiffusion_loop(drafter, verifier, start, MASK_ID, 2, 1, 0.5, 0,
                                                  unmask_tau=np.inf, unmask_k=3, max_cycles=60)
    assert stats0["cycles"] == 60 and (x0 == MASK_ID).any()


def test_more_drafter_steps_per_cycle_mean_fewer_verifier_calls(oracle_mod):
    target, start, drafter, verifier = problem(5, wrong=0.0)
    calls = []
    for K in (1, 2, 4, 8):
        _, stats, _ = oracle_mod.dualdiffusion_loop(drafter, verifier, start, MASK_ID, K, 2, 0.2, 1,
                                                    unmask_tau=np.inf, unmask_k=1)
        calls.append(stats["verifier_calls"])
    assert calls == sorted(calls, reverse=True) and calls[0] > calls[-1]
