"""dd_verify on the GPU against the CPU oracle, through the C ABI."""
import numpy as np
import pytest

from paper_2604_05250_b200 import synth
from tests._parity import Guarded, check_verify, to_torch_bf16

pytestmark = pytest.mark.gpu

TRUST, KL, CONF = 0, 1, 2
PROB, EMIT = 0x100, 0x200


@pytest.fixture(scope="module")
def dd():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2604_05250_b200 import binding, build
    build.build()
    binding.lib()
    return binding


def run_gpu(dd, dra, ver, tokens, flags, mode, tau, k, seed, host=False):
    import torch
    dev = None if host else "cuda"
    t_ver = to_torch_bf16(ver, dev, pin=host)
    t_dra = None if dra is None else to_torch_bf16(dra, dev, pin=host)
    t_tok = torch.from_numpy(tokens)
    t_fl = torch.from_numpy(flags)
    if host:
        t_tok, t_fl = t_tok.pin_memory(), t_fl.pin_memory()
    else:
        t_tok, t_fl = t_tok.cuda(), t_fl.cuda()
    # each output sits between two guard regions that the kernels must leave alone
    g_tok = Guarded(tokens.shape, torch.int32, device=dev, pin=host)
    g_mask = Guarded(tokens.shape, torch.uint8, device=dev, pin=host)
    g_score = Guarded(tokens.shape, torch.float32, device=dev, pin=host)
    ot, om, osc = dd.verify(t_dra, t_ver, t_tok, t_fl, mode, tau, k, seed, out_tokens=g_tok.view,
                            out_mask=g_mask.view, out_score=g_score.view, host=host)
    torch.cuda.synchronize()
    assert dd.verify_status() == 0
    g_tok.check("out_tokens"); g_mask.check("out_mask"); g_score.check("out_score")
    return ot.cpu().numpy(), om.cpu().numpy(), osc.cpu().numpy()


def compare(dd, oracle_mod, dra, ver, tokens, flags, mode, tau, k, seed, host=False):
    algo = mode & 0xFF
    d_in = dra if algo == KL else None
    ref = oracle_mod.verify(d_in, ver, tokens, flags, mode, tau, k, seed)
    ot, om, osc = run_gpu(dd, d_in, ver, tokens, flags, mode, tau, k, seed, host=host)
    return check_verify(ot, om, osc, ref, flags, tokens), ref, (ot, om, osc)


ALL_MODES = [TRUST, KL, CONF, KL | PROB, CONF | PROB, KL | EMIT, TRUST | EMIT, CONF | PROB | EMIT]


@pytest.mark.parametrize("mode", ALL_MODES)
def test_config0_tiny(dd, oracle_mod, mode):
    c = synth.VERIFY_CONFIGS[0]
    dra, ver, tokens, flags = synth.verify_config_inputs(0)
    assert flags.sum() == 32
    compare(dd, oracle_mod, dra, ver, tokens, flags, mode, c["tau"], c["k"], c["seed"])


@pytest.mark.parametrize("V", [8, 1000, 1003, 8192, 8200, 8201, 20000, 32000])
@pytest.mark.parametrize("mode", [KL, CONF])
def test_vocab_sizes_and_ragged_tails(dd, oracle_mod, V, mode):
    """Several chunks plus a ragged tail; V % 8 != 0 takes the element-wise path."""
    dra, ver, tokens, flags = synth.verify_inputs(2, 24, V, 17, 0.2, seed=V)
    compare(dd, oracle_mod, dra, ver, tokens, flags, mode, 0.5, 4, 1)


def test_config1_llada_shaped_full_size(dd, oracle_mod):
    c = synth.VERIFY_CONFIGS[1]
    dra, ver, tokens, flags = synth.verify_config_inputs(1)
    n_ex, ref, _ = compare(dd, oracle_mod, dra, ver, tokens, flags, KL, c["tau"], c["k"], c["seed"])
    assert 5 <= ref["out_mask"].sum() <= 60           # ~10% drafter errors get remasked
    assert n_ex <= 4
    # probabilistic variant and the host-buffer entry point on the same data
    compare(dd, oracle_mod, dra, ver, tokens, flags, KL | PROB, c["tau"], c["k"], 3)
    compare(dd, oracle_mod, dra, ver, tokens, flags, KL, c["tau"], c["k"], c["seed"], host=True)


def test_config2_batched_full_size(dd, oracle_mod):
    c = synth.VERIFY_CONFIGS[2]
    dra, ver, tokens, flags = synth.verify_config_inputs(2)
    counts = flags.sum(axis=1)
    assert counts.min() >= 64 and counts.max() <= 256 and len(set(counts.tolist())) > 4
    _, ref, _ = compare(dd, oracle_mod, dra, ver, tokens, flags, CONF, c["tau"], c["k"], c["seed"])
    # every position fails c < 0.5 at this vocabulary size: the top-k rule decides
    kept = (flags.astype(bool) & ~ref["out_mask"].astype(bool)).sum(axis=1)
    assert (kept == c["k"]).all()
    compare(dd, oracle_mod, dra, ver, tokens, flags, CONF | PROB, c["tau"], c["k"], 5)


@pytest.mark.parametrize("mode", [TRUST, KL])
def test_config3_long_context(dd, oracle_mod, mode):
    c = synth.VERIFY_CONFIGS[3]
    dra, ver, tokens, flags = synth.verify_config_inputs(3)
    compare(dd, oracle_mod, dra, ver, tokens, flags, mode, c["tau"], c["k"], c["seed"])


@pytest.mark.parametrize("V,seeds", [(32000, (0, 1, 2, 3)), (126464, (0,))])
@pytest.mark.parametrize("err", [0.05, 0.20, 0.50])
def test_config4_sweep(dd, oracle_mod, V, seeds, err):
    sw = synth.VERIFY_SWEEP
    for seed in seeds:
        for nflag in sw["flagged"]:
            dra, ver, tokens, flags = synth.verify_inputs(1, sw["P"], V, nflag, err,
                                                          synth.config_seed(4, seed))
            k = 8 if nflag == 32 else 32
            for mode in (TRUST, KL, CONF) if seed == 0 else (KL,):
                compare(dd, oracle_mod, dra, ver, tokens, flags, mode, sw["tau"], k, seed)
            if seed == 0 and nflag == 128:
                compare(dd, oracle_mod, dra, ver, tokens, flags, KL | PROB, sw["tau"], k, seed)
                compare(dd, oracle_mod, dra, ver, tokens, flags, CONF | PROB, sw["tau"], k, seed)


def test_degenerate_cases(dd, oracle_mod):
    dra, ver, tokens, flags = synth.verify_inputs(3, 16, 256, 9, 0.3, seed=11)
    # nothing flagged anywhere: pure pass-through
    none = np.zeros_like(flags)
    compare(dd, oracle_mod, dra, ver, tokens, none, KL, 0.5, 4, 0)
    # one sequence empty, one full
    mixed = flags.copy(); mixed[0] = 0; mixed[1] = 1
    compare(dd, oracle_mod, dra, ver, tokens, mixed, KL, 0.5, 4, 0)
    # k = 0 (pure rule), k >= number flagged (keep all), unreachable thresholds
    compare(dd, oracle_mod, dra, ver, tokens, flags, KL, 0.05, 0, 0)
    _, ref, got = compare(dd, oracle_mod, dra, ver, tokens, flags, KL, 0.0, 1000, 0)
    assert not got[1].any()
    compare(dd, oracle_mod, dra, ver, tokens, flags, CONF, 2.0, 3, 0)
    compare(dd, oracle_mod, dra, ver, tokens, flags, KL, 1e9, 3, 0)
    # identical drafter and verifier: KL = 0 everywhere, nothing exceeds tau = 0
    _, ref, got = compare(dd, oracle_mod, ver, ver, tokens, flags, KL, 0.0, 0, 0)
    assert not got[1].any() and np.abs(got[2]).max() <= 1e-6
    # P = 1, V = 8
    d1, v1, t1, f1 = synth.verify_inputs(1, 1, 8, 1, 0.0, seed=12)
    compare(dd, oracle_mod, d1, v1, t1, f1, CONF, 0.5, 0, 0)


def test_many_short_rows_and_long_sequences(dd, oracle_mod):
    # more (row, chunk) units than the CTAs' tables hold at once (several rounds per CTA), and
    # sequences that exactly fill the decision stage's key area in shared memory (8192 keys)
    dra, ver, tokens, flags = synth.verify_inputs(15, 8192, 64, 5700, 0.2, seed=31)
    compare(dd, oracle_mod, dra, ver, tokens, flags, KL, 0.5, 40, 3)
    compare(dd, oracle_mod, dra, ver, tokens, flags, CONF | PROB, 0.5, 7, 3)
    # longer than what a lane keeps in registers (1024 keys), inside the key area
    dra, ver, tokens, flags = synth.verify_inputs(2, 1500, 4104, 900, 0.2, seed=32)
    compare(dd, oracle_mod, dra, ver, tokens, flags, KL, 0.5, 33, 1)
    # the element-wise kernel (V % 8 != 0): inside its key area (2048 keys) and beyond it, where
    # every pass of the decision stage re-reads the scores from memory (the streaming kernel's
    # area holds the longest sequence the library accepts)
    for P, nflag in ((1900, 1000), (2500, 1200)):
        dra, ver, tokens, flags = synth.verify_inputs(1, P, 203, nflag, 0.2, seed=P)
        compare(dd, oracle_mod, dra, ver, tokens, flags, KL | PROB, 0.5, 21, 5)


def test_exact_ties_in_verifier_row(dd, oracle_mod):
    dra, ver, tokens, flags = synth.verify_inputs(1, 8, 20000, 8, 0.0, seed=13)
    top = synth.f32_to_bf16_bits(np.array([30.0], dtype=np.float32))[0]
    ver[0, 0, [19999, 8191, 8192, 12345]] = top        # ties across chunk and warp boundaries
    ver[0, 1, [7, 3]] = top
    ver[0, 2, :] = top                                  # a constant row
    _, ref, got = compare(dd, oracle_mod, dra, ver, tokens, flags, TRUST, 0.5, 0, 0)
    assert got[0][0, 0] == 8191 and got[0][0, 1] == 3 and got[0][0, 2] == 0


def test_threshold_sweep_crosses_scores(dd, oracle_mod):
    """Thresholds placed on and next to actual scores exercise the exempt band."""
    dra, ver, tokens, flags = synth.verify_inputs(1, 32, 4096, 32, 0.3, seed=14)
    ref = oracle_mod.verify(dra, ver, tokens, flags, KL, 0.5, 0, 0)
    scores = np.sort(ref["out_score"][0])
    n_exempt = 0
    for s in scores[::4]:
        for tau in (s, s * (1 + 3e-6), s * (1 - 3e-6), s + 1e-3):
            n, _, _ = compare(dd, oracle_mod, dra, ver, tokens, flags, KL, float(tau), 0, 0)
            n_exempt += n
    assert n_exempt > 0


def test_out_tokens_may_alias_tokens_and_score_is_optional(dd, oracle_mod):
    import torch
    dra, ver, tokens, flags = synth.verify_inputs(2, 16, 1024, 10, 0.2, seed=15)
    ref = oracle_mod.verify(dra, ver, tokens, flags, KL, 0.5, 2, 0)
    t_tok = torch.from_numpy(tokens.copy()).cuda()
    ot, om, osc = dd.verify(to_torch_bf16(dra, "cuda"), to_torch_bf16(ver, "cuda"), t_tok,
                            torch.from_numpy(flags).cuda(), KL, 0.5, 2, 0,
                            out_tokens=t_tok, want_score=False)
    torch.cuda.synchronize()
    assert osc is None
    strict = ~ref["exempt"].astype(bool)
    assert (ot.cpu().numpy()[strict] == ref["out_tokens"][strict]).all()
    assert (om.cpu().numpy()[strict] == ref["out_mask"][strict]).all()


def test_bitwise_repeatability(dd, oracle_mod):
    dra, ver, tokens, flags = synth.verify_inputs(4, 64, 32000, "uniform_25_100", 0.2, seed=16)
    first = run_gpu(dd, dra, ver, tokens, flags, KL | PROB, 0.5, 8, 9)
    for _ in range(5):
        again = run_gpu(dd, dra, ver, tokens, flags, KL | PROB, 0.5, 8, 9)
        for a, b in zip(first, again):
            assert np.array_equal(a, b)


def test_philox_stream_matches_oracle(dd, oracle_mod):
    """With all verifier logits equal, c = 1/2 exactly at V = 2... use V = 8: c = 1/8, so
    CONF|PROB remasks iff u < 7/8: the GPU's uniforms must match the oracle's one by one."""
    B, P, V = 3, 200, 8
    ver = np.zeros((B, P, V), dtype=np.uint16)
    tokens = np.zeros((B, P), dtype=np.int32)
    flags = np.ones((B, P), dtype=np.uint8)
    for seed in (0, 1, 0xDEADBEEFCAFEF00D):
        ot, om, osc = run_gpu(dd, None, ver, tokens, flags, CONF | PROB, 0.5, 0, seed)
        expect = np.array([[oracle_mod.uniform(seed, b, i) < 0.875 for i in range(P)] for b in range(B)])
        assert np.array_equal(om.astype(bool), expect)


def test_scratch_survives_changing_shapes(dd, oracle_mod):
    """Calls of different (B, P, V) in a row reuse the library's scratch: the completion
    counters must not inherit stale data from a previous layout."""
    shapes = [(1, 8, 64), (4, 300, 1024), (2, 16, 20000), (6, 700, 256), (1, 8, 64), (3, 200, 8)]
    for n, (B, P, V) in enumerate(shapes):
        dra, ver, tokens, flags = synth.verify_inputs(B, P, V, max(1, P // 2), 0.2, seed=100 + n)
        compare(dd, oracle_mod, dra, ver, tokens, flags, KL, 0.5, 3, n)


@pytest.fixture
def cta_cap(dd):
    """Caps the streaming kernel's grid for one test and lifts the cap afterwards."""
    yield dd.debug_set_max_ctas
    dd.debug_set_max_ctas(0)


def test_results_do_not_depend_on_the_grid(dd, oracle_mod, cta_cap):
    """Same inputs on 1, 7, 37 CTAs and on every SM: tokens, masks and scores bit-identical (which
    warp computes a unit, and in which order units finish, must not matter)."""
    cases = [
        (synth.verify_config_inputs(0), KL | PROB, 0.5, 8, 0),
        (synth.verify_inputs(2, 40, 20000 + 8 * 37, 29, 0.2, seed=41), KL, 0.5, 4, 1),       # ragged last chunk
        (synth.verify_inputs(2, 40, 20000 + 8 * 37, 29, 0.2, seed=41), CONF | PROB, 0.5, 4, 2),
        (synth.verify_inputs(15, 8192, 64, 5700, 0.2, seed=31), KL, 0.5, 40, 3),              # many short rows
        (synth.verify_inputs(3, 96, 32000, 80, 0.3, seed=42), TRUST, 0.5, 0, 0),
    ]
    for (dra, ver, tokens, flags), mode, tau, k, seed in cases:
        d_in = dra if (mode & 0xFF) == KL else None
        cta_cap(0)
        ref = run_gpu(dd, d_in, ver, tokens, flags, mode, tau, k, seed)
        for cap in (1, 7, 37):
            cta_cap(cap)
            got = run_gpu(dd, d_in, ver, tokens, flags, mode, tau, k, seed)
            for a, b in zip(ref, got):
                assert np.array_equal(a, b), f"cap {cap}"
        cta_cap(0)
        check_verify(*ref, oracle_mod.verify(d_in, ver, tokens, flags, mode, tau, k, seed), flags, tokens)


@pytest.mark.parametrize("V", [20000, 1003])
def test_token_excluded_by_the_verifier_alone(dd, oracle_mod, V):
    """p_V(x) = 0 where p_D(x) > 0: the divergence of Eq. 5 is infinite, in the oracle and in both
    kernels (the streaming path meets the token as a finite logit of -3.4e38 and must notice)."""
    ninf = np.uint16(0xFF80)
    dra, ver, tokens, flags = synth.verify_inputs(2, 12, V, 12, 0.25, seed=77 + V)
    rng = np.random.default_rng(V + 1)
    ver[0, 2, rng.choice(V, size=5, replace=False)] = ninf            # five ordinary tokens
    top = int(np.argmax(synth.bf16_bits_to_f32(dra[1, 3])))
    ver[1, 3, top] = ninf                                              # the drafter's most likely token
    both = rng.choice(V, size=40, replace=False)
    dra[1, 4, both] = ninf; ver[1, 4, both] = ninf                     # a row that stays finite
    tokens[:] = np.argmax(synth.bf16_bits_to_f32(dra), axis=2)
    _, ref, got = compare(dd, oracle_mod, dra, ver, tokens, flags, KL, 0.5, 3, 7)
    inf_at = np.zeros((2, 12), dtype=bool)
    inf_at[0, 2] = inf_at[1, 3] = True
    assert np.isposinf(ref["out_score"][inf_at]).all() and np.isposinf(got[2][inf_at]).all()
    assert np.isfinite(ref["out_score"][~inf_at]).all() and np.isfinite(got[2][~inf_at]).all()


@pytest.mark.parametrize("V", [4096, 20000, 1003])
def test_excluded_tokens(dd, oracle_mod, V):
    """Logits of -inf (banned or padded vocabulary entries) at shared and at drafter-only
    indices: probability zero, no term in Eq. 5; the other rows are untouched by the detour."""
    ninf = np.uint16(0xFF80)
    if True:
        dra, ver, tokens, flags = synth.verify_inputs(2, 12, V, 12, 0.25, seed=51 + V)
        rng = np.random.default_rng(V)
        both = rng.choice(V, size=V // 16, replace=False)
        dra[0, 1, both] = ninf; ver[0, 1, both] = ninf                 # excluded by both models
        dra[0, 3, both[:50]] = ninf                                    # excluded by the drafter only
        run_end = 4000 if V > 4096 else 1000
        dra[1, 5, 8:run_end] = ninf; ver[1, 5, 8:run_end] = ninf       # a whole run of the row
        dra[1, 7, :V - 3] = ninf; ver[1, 7, :V - 3] = ninf             # nearly everything
        tokens[:] = np.argmax(synth.bf16_bits_to_f32(dra), axis=2)
        for mode in (KL, CONF, KL | PROB):
            _, ref, got = compare(dd, oracle_mod, dra, ver, tokens, flags, mode, 0.5, 3, 7)
            assert np.isfinite(ref["out_score"]).all() and np.isfinite(got[2]).all()
