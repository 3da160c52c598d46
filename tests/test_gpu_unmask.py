"""dd_unmask on the GPU against the CPU oracle, through the C ABI."""
import numpy as np
import pytest

from paper_2604_05250_b200 import synth
from tests._parity import SCORE_ABS_FLOOR, SCORE_REL, Guarded, to_torch_bf16

pytestmark = pytest.mark.gpu
MASK_ID = 126336


@pytest.fixture(scope="module")
def dd():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2604_05250_b200 import binding, build
    build.build()
    binding.lib()
    return binding


def compare(dd, oracle_mod, logits, flags, tau, k):
    import torch
    B, P, V = logits.shape
    tokens = np.full((B, P), MASK_ID, dtype=np.int32)
    tokens[flags == 0] = 5
    ref = oracle_mod.unmask(logits, tokens, flags, tau, k)
    g_tok, g_mask = Guarded((B, P), torch.int32), Guarded((B, P), torch.uint8)
    g_conf = Guarded((B, P), torch.float32)
    ot, om, oc = dd.unmask(to_torch_bf16(logits, "cuda"), torch.from_numpy(tokens).cuda(),
                           torch.from_numpy(flags).cuda(), tau, k, out_tokens=g_tok.view, out_mask=g_mask.view,
                           out_conf=g_conf.view)
    torch.cuda.synchronize()
    assert dd.verify_status() == 0
    g_tok.check("out_tokens"); g_mask.check("out_mask"); g_conf.check("out_conf")
    ot, om, oc = ot.cpu().numpy(), om.cpu().numpy(), oc.cpu().numpy().astype(np.float64)
    tol = np.maximum(SCORE_REL * np.abs(ref["out_conf"]), SCORE_ABS_FLOOR)
    assert (np.abs(oc - ref["out_conf"]) <= tol).all()
    strict = ref["exempt"] == 0
    assert (om[strict] == ref["out_mask"][strict]).all()
    assert (ot[strict] == ref["out_tokens"][strict]).all()
    # at exempt positions either decision stands, with the token that goes with it
    ex = ~strict
    if ex.any():
        p_best = np.where(ref["out_mask"] == 0, ref["out_tokens"], -1)
        ok = ((om == 1) & (ot == tokens)) | ((om == 0) & ((ot == p_best) | (p_best < 0)))
        assert ok[ex].all()
    assert (ot[flags == 0] == 5).all() and not om[flags == 0].any() and not oc[flags == 0].any()
    return ref, om


@pytest.mark.parametrize("tau,k", [(0.5, 0), (0.5, 1), (np.inf, 8), (0.02, 4), (0.0, 0), (2.0, 0)])
def test_llada_vocabulary(dd, oracle_mod, tau, k):
    _, logits, _, flags = synth.verify_inputs(2, 64, 126464, 48, 0.1, seed=71)
    ref, om = compare(dd, oracle_mod, logits, flags, tau, k)
    if np.isinf(tau):
        assert ((flags == 1) & (om == 0)).sum(axis=1).tolist() == [k, k]


@pytest.mark.parametrize("V", [1000, 1003, 8200, 32000])
def test_vocabulary_sizes_and_fixed_count(dd, oracle_mod, V):
    _, logits, _, flags = synth.verify_inputs(3, 128, V, 96, 0.1, seed=72 + V)
    compare(dd, oracle_mod, logits, flags, 0.3, 5)
    compare(dd, oracle_mod, logits, flags, np.inf, 17)


def test_nothing_masked_passes_through(dd, oracle_mod):
    _, logits, _, flags = synth.verify_inputs(2, 32, 1024, 16, 0.1, seed=73)
    flags[1] = 0
    ref, om = compare(dd, oracle_mod, logits, flags, 0.4, 2)
    assert not om[1].any()


def test_batched_serving_shape(dd, oracle_mod):
    """The cfg2 logits shape [16,256,126464] with 25-100 % of the positions masked per sequence."""
    _, logits, _, flags = synth.verify_config_inputs(2)
    ref, om = compare(dd, oracle_mod, logits, flags, 0.5, 16)
    assert ((flags == 1) & (om == 0)).sum(axis=1).min() >= 16
