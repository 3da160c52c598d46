"""dd_lm_head_verify on the GPU against the CPU oracle (fp64 head, then the verification algorithm
on the unrounded logits), through the C ABI."""
import numpy as np
import pytest

from paper_2604_05250_b200 import synth
from tests._parity import Guarded, check_verify, to_torch_bf16

pytestmark = pytest.mark.gpu

TRUST, KL, CONF, PROB, EMIT = 0, 1, 2, 0x100, 0x200
# The kernel accumulates the bf16 products in fp32 where the oracle uses fp64: a verifier token is
# only comparable where the two largest logits are further apart than that can blur.
TOP2_GAP = 1e-3
# KL scores (Eq. 4-5) are differences of quantities of size |logit| ~ 10: the fp32 accumulation of
# K bf16 products leaves each logit within about sqrt(K) * 2^-24 * |logit| ~ 4e-5 (K = 4096) of the
# oracle's fp64 value, and the score inherits an error of that size whatever its own magnitude.
KL_SCORE_ABS = 1e-4


@pytest.fixture(scope="module")
def dd():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2604_05250_b200 import binding, build
    build.build()
    binding.lib()
    return binding


def compare(dd, oracle_mod, hidden, weight, tokens, flags, mode, tau, k, seed, drafter=(None, None)):
    import torch
    B, P, K = hidden.shape
    ref = oracle_mod.lm_head_verify(drafter[0], drafter[1], hidden, weight, tokens, flags, mode, tau, k, seed)
    g_tok, g_mask, g_score = (Guarded((B, P), dt) for dt in (torch.int32, torch.uint8, torch.float32))
    t_dra = [None if x is None else to_torch_bf16(x, "cuda") for x in drafter]
    ot, om, osc = dd.lm_head_verify(t_dra[0], t_dra[1], to_torch_bf16(hidden, "cuda"), to_torch_bf16(weight, "cuda"),
                                    torch.from_numpy(tokens).cuda(), torch.from_numpy(flags).cuda(),
                                    mode, tau, k, seed, out_tokens=g_tok.view, out_mask=g_mask.view, out_score=g_score.view)
    torch.cuda.synchronize()
    assert dd.verify_status() == 0
    g_tok.check("out_tokens"); g_mask.check("out_mask"); g_score.check("out_score")
    ot, om, osc = ot.cpu().numpy(), om.cpu().numpy(), osc.cpu().numpy()
    # where the verifier's two best tokens are closer than fp32 accumulation resolves, either is right
    close = (ref["top2_gap"] <= TOP2_GAP) & flags.astype(bool) & (om == 0) & (ref["out_mask"] == 0)
    ref = dict(ref)
    ref["out_tokens"] = np.where(close, ot, ref["out_tokens"])
    n_exempt = check_verify(ot, om, osc, ref, flags, tokens,
                            **(dict(score_abs=KL_SCORE_ABS) if (mode & 0xFF) == KL else {}))
    return ref, (ot, om, osc), int(close.sum()), n_exempt


@pytest.mark.parametrize("B,P,K,V,flagged", [
    (1, 40, 128, 1000, 25),            # one row block, rows and vocabulary both ragged
    (2, 70, 256, 4100, 51),            # rows of two sequences share a 128-row tile
    (1, 300, 64, 8232, 300),           # two row blocks, a single k-step
    (3, 128, 512, 2048, "uniform_25_100"),
    (1, 1, 64, 8, 1),
])
@pytest.mark.parametrize("mode", [TRUST, CONF, CONF | PROB])
def test_small_shapes(dd, oracle_mod, B, P, K, V, flagged, mode):
    hidden, weight, tokens, flags = synth.lm_head_inputs(B, P, K, V, flagged, seed=B * 1000 + P)
    compare(dd, oracle_mod, hidden, weight, tokens, flags, mode, 0.05, 3, 7)


@pytest.mark.parametrize("B,P,K,V,flagged", [
    (1, 40, 128, 1000, 25),
    (2, 70, 256, 4100, 51),
    (1, 300, 64, 8232, 300),
    (3, 128, 512, 2048, "uniform_25_100"),
    (1, 1, 64, 8, 1),
])
@pytest.mark.parametrize("mode", [KL, KL | PROB, KL | EMIT])
def test_small_shapes_kl(dd, oracle_mod, B, P, K, V, flagged, mode):
    """Eq. 4-5 from both models' hidden states: two products per work item, one epilogue."""
    dh, dw, vh, vw, tokens, flags = synth.lm_head_pair_inputs(B, P, K, V, flagged, 0.2, seed=B * 1000 + P)
    ref, got, _, _ = compare(dd, oracle_mod, vh, vw, tokens, flags, mode, 0.5, 3, 7, drafter=(dh, dw))
    if P >= 40:        # the scores are those of two different distributions, and both outcomes occur
        fl = flags.astype(bool)
        assert (ref["out_score"][fl] > 1e-3).all()
        if not mode & PROB:
            assert ref["out_mask"][fl].any() and not ref["out_mask"][fl].all()


@pytest.mark.parametrize("P", [700, 1100, 2100])
def test_long_sequences(dd, oracle_mod, P):
    """Sequences longer than the register-resident decision stage holds (512 positions), longer
    than the general form keeps in registers (1024), and longer than the fold kernel's key area in
    shared memory (2048)."""
    hidden, weight, tokens, flags = synth.lm_head_inputs(2, P, 64, 520, "uniform_25_100", seed=P)
    compare(dd, oracle_mod, hidden, weight, tokens, flags, CONF | PROB, 0.05, 9, 11)
    dh, dw, vh, vw, tokens, flags = synth.lm_head_pair_inputs(2, P, 64, 520, "uniform_25_100", 0.2, seed=P + 1)
    compare(dd, oracle_mod, vh, vw, tokens, flags, KL, 0.5, 9, 11, drafter=(dh, dw))


def test_kl_tells_the_two_models_apart(dd, oracle_mod):
    """The drafter's pair and the verifier's pair swapped: D_KL(p_V || p_D) is another number."""
    dh, dw, vh, vw, tokens, flags = synth.lm_head_pair_inputs(1, 64, 128, 2000, 64, 0.2, seed=5)
    a, _, _, _ = compare(dd, oracle_mod, vh, vw, tokens, flags, KL, 0.5, 0, 0, drafter=(dh, dw))
    b, _, _, _ = compare(dd, oracle_mod, dh, dw, tokens, flags, KL, 0.5, 0, 0, drafter=(vh, vw))
    assert (np.abs(a["out_score"] - b["out_score"]) > 1e-3).sum() > 32
    # and a drafter equal to the verifier scores zero everywhere
    import torch
    t = [to_torch_bf16(x, "cuda") for x in (vh, vw)]
    out = dd.lm_head_verify(t[0], t[1], t[0], t[1], torch.from_numpy(tokens).cuda(), torch.from_numpy(flags).cuda(),
                            KL, 0.5, 0, 0)
    assert float(out[2].abs().max()) <= 1e-6 and int(out[1].sum()) == 0


def test_matches_the_unfused_path(dd, oracle_mod):
    """Logits by the oracle's head, rounded to bf16, through dd_verify: the same decisions wherever
    the confidence is far from the threshold (the two paths differ by the rounding of the logits)."""
    import torch
    B, P, K, V = 1, 64, 256, 4096
    hidden, weight, tokens, flags = synth.lm_head_inputs(B, P, K, V, 64, seed=9)
    logits = oracle_mod.lm_head(hidden.reshape(P, K), weight)
    bits = synth.f32_to_bf16_bits(logits.astype(np.float32)).reshape(B, P, V)
    a = dd.lm_head_verify(None, None, to_torch_bf16(hidden, "cuda"), to_torch_bf16(weight, "cuda"), torch.from_numpy(tokens).cuda(),
                          torch.from_numpy(flags).cuda(), CONF, 0.05, 0, 0)
    b = dd.verify(None, to_torch_bf16(bits, "cuda"), torch.from_numpy(tokens).cuda(), torch.from_numpy(flags).cuda(),
                  CONF, 0.05, 0, 0)
    torch.cuda.synchronize()
    sa, sb = a[2].cpu().numpy(), b[2].cpu().numpy()
    assert np.abs(sa - sb).max() <= 2e-2 * sb.max()
    far = np.abs(sb - 0.05) > 5e-3
    assert far.sum() > P // 2 and (a[1].cpu().numpy()[far] == b[1].cpu().numpy()[far]).all()


def test_llada_shaped_full_size(dd, oracle_mod):
    """cfg1's verification step from hidden states: 256 positions, K = 4096, V = 126464."""
    hidden, weight, tokens, flags = synth.lm_head_inputs(1, 256, 4096, 126464, "all", seed=1000)
    ref, got, n_close, _ = compare(dd, oracle_mod, hidden, weight, tokens, flags, CONF, 0.5, 32, 0)
    assert n_close <= 8
    kept = (flags.astype(bool) & ~ref["out_mask"].astype(bool)).sum()
    assert kept >= 32


def test_llada_shaped_full_size_kl(dd, oracle_mod):
    """The same step in the KL mode: both heads at K = 4096, V = 126464."""
    dh, dw, vh, vw, tokens, flags = synth.lm_head_pair_inputs(1, 256, 4096, 126464, "all", 0.2, seed=1001)
    ref, got, _, _ = compare(dd, oracle_mod, vh, vw, tokens, flags, KL, 0.5, 32, 0, drafter=(dh, dw))
    rejected = int(ref["out_mask"].sum())
    assert 20 <= rejected <= 120


def test_results_do_not_depend_on_the_grid(dd, oracle_mod):
    import torch
    hidden, weight, tokens, flags = synth.lm_head_inputs(2, 150, 128, 3000, 97, seed=12)
    dh, dw, _, _, _, _ = synth.lm_head_pair_inputs(2, 150, 128, 3000, 97, 0.2, seed=12)
    tail = (to_torch_bf16(hidden, "cuda"), to_torch_bf16(weight, "cuda"), torch.from_numpy(tokens).cuda(),
            torch.from_numpy(flags).cuda())
    for args in ((None, None) + tail + (CONF | PROB, 0.05, 4, 3),
                 (to_torch_bf16(dh, "cuda"), to_torch_bf16(dw, "cuda")) + tail + (KL | PROB, 0.5, 4, 3)):
        try:
            ref = [x.cpu().numpy() for x in dd.lm_head_verify(*args)]
            for cap in (1, 5, 37):
                dd.debug_set_max_ctas(cap)
                got = [x.cpu().numpy() for x in dd.lm_head_verify(*args)]
                for a, b in zip(ref, got):
                    assert np.array_equal(a, b), f"cap {cap}"
        finally:
            dd.debug_set_max_ctas(0)


def test_argument_errors(dd):
    import torch
    h = torch.zeros(1, 4, 64, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(16, 64, dtype=torch.bfloat16, device="cuda")
    t = torch.zeros(1, 4, dtype=torch.int32, device="cuda")
    f = torch.ones(1, 4, dtype=torch.uint8, device="cuda")
    o = torch.zeros(1, 4, dtype=torch.float32, device="cuda")
    L, p = dd.lib(), (lambda x: x.data_ptr())
    call = lambda mode, K: L.dd_lm_head_verify(None, None, p(h), p(w), p(t), p(f), mode, 0.5, 0, 0, p(t), p(f), p(o), 1, 4, K, 16, None)
    assert call(KL, 64) == dd.DD_ERR_INVALID_ARG           # the KL mode needs the drafter's pair
    assert L.dd_lm_head_verify(p(h), None, p(h), p(w), p(t), p(f), KL, 0.5, 0, 0, p(t), p(f), p(o), 1, 4, 64, 16, None) == dd.DD_ERR_INVALID_ARG
    assert L.dd_lm_head_verify(p(h) + 2, p(w), p(h), p(w), p(t), p(f), KL, 0.5, 0, 0, p(t), p(f), p(o), 1, 4, 64, 16, None) == dd.DD_ERR_UNSUPPORTED
    assert call(CONF, 48) == dd.DD_ERR_UNSUPPORTED
    assert call(CONF, 0) == dd.DD_ERR_INVALID_ARG
    assert call(7, 64) == dd.DD_ERR_INVALID_ARG
    assert L.dd_lm_head_verify(None, None, None, p(w), p(t), p(f), CONF, 0.5, 0, 0, p(t), p(f), p(o), 1, 4, 64, 16, None) == dd.DD_ERR_INVALID_ARG
