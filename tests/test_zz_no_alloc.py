"""dd_verify_static, the entry point for callers that cannot allocate device memory
(a server that has given all free memory to its caches, code that must not hit the
implicit synchronisation of cudaMalloc, a process whose allocator belongs to another
runtime).  Its scratch is a fixed array inside the library, so it must give what
dd_verify gives, call after call, whatever the previous call left in that array,
and it must leave the amount of free device memory alone.

Collected last on purpose: a failure here cannot hide the result of any other test.
"""
import ctypes

import numpy as np
import pytest

from paper_2604_05250_b200 import synth
from tests._parity import SCORE_ABS_FLOOR, SCORE_REL, check_verify, to_torch_bf16

pytestmark = pytest.mark.gpu

KL, CONF, PROB = 1, 2, 0x100


def both_entry_points(dd, oracle_mod, shape, mode, seed):
    import torch
    B, P, V, nflag = shape
    dra, ver, tokens, flags = synth.verify_inputs(B, P, V, nflag, 0.2, seed=seed)
    t_dra, t_ver = to_torch_bf16(dra, "cuda"), to_torch_bf16(ver, "cuda")
    t_tok, t_fl = torch.from_numpy(tokens).cuda(), torch.from_numpy(flags).cuda()
    if (mode & 0xFF) != KL:
        t_dra, dra = None, None
    ref = dd.verify(t_dra, t_ver, t_tok, t_fl, mode, 0.5, 4, seed)
    outs = (torch.full((B, P), -7, dtype=torch.int32, device="cuda"),
            torch.full((B, P), 9, dtype=torch.uint8, device="cuda"),
            torch.full((B, P), -1.0, dtype=torch.float32, device="cuda"))
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    got = dd.verify(t_dra, t_ver, t_tok, t_fl, mode, 0.5, 4, seed, out_tokens=outs[0], out_mask=outs[1],
                    out_score=outs[2], static_scratch=True)
    torch.cuda.synchronize()
    free_after = torch.cuda.mem_get_info()[0]
    assert dd.verify_status() == 0
    r_tok, r_mask, r_score = (x.cpu().numpy() for x in ref)
    g_tok, g_mask, g_score = (x.cpu().numpy() for x in got)
    assert np.array_equal(g_tok, r_tok)
    assert np.array_equal(g_mask, r_mask)
    tol = np.maximum(SCORE_REL * np.abs(r_score), SCORE_ABS_FLOOR)
    assert (np.abs(g_score - r_score) <= tol).all()
    assert flags.sum() > 0 and (g_score[flags.astype(bool)] > 0).any()
    # and against the oracle, like every other entry point
    check_verify(g_tok, g_mask, g_score, oracle_mod.verify(dra, ver, tokens, flags, mode, 0.5, 4, seed), flags, tokens)
    return free_before, free_after


def test_static_scratch_matches_dd_verify_on_two_calls_in_a_row(oracle_mod):
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2604_05250_b200 import binding as dd
    from paper_2604_05250_b200 import build
    build.build()
    # consecutive calls with different shapes and modes: each one runs on whatever the previous
    # one left in the shared array
    both_entry_points(dd, oracle_mod, (2, 96, 20000, 61), KL | PROB, seed=21)
    frees = [both_entry_points(dd, oracle_mod, (3, 40, 126464, 33), KL, seed=22),
             both_entry_points(dd, oracle_mod, (1, 128, 1024, 32), CONF, seed=23),
             # V % 8 != 0: the element-wise kernel runs on the fixed array as well
             both_entry_points(dd, oracle_mod, (2, 50, 1003, 31), KL, seed=24)]
    # once the first call on the device has looked up the array, a call takes no device memory
    for before, after in frees:
        assert after == before


def test_static_scratch_at_its_size_limit():
    """B*P = 4096 rows of the LLaDA vocabulary fill the fixed array exactly (16 chunks of 8192
    logits per row): still served, with dd_verify's results."""
    import torch
    from paper_2604_05250_b200 import binding as dd
    B, P, V = 16, 256, 126464
    gen = torch.Generator(device="cuda").manual_seed(5)
    ver = (2.0 * torch.randn(B, P, V, generator=gen, device="cuda", dtype=torch.float32)).to(torch.bfloat16)
    tok = torch.zeros(B, P, dtype=torch.int32, device="cuda")
    fl = torch.ones(B, P, dtype=torch.uint8, device="cuda")
    ref = dd.verify(None, ver, tok, fl, CONF, 0.5, 16, 0)
    outs = dict(out_tokens=torch.empty_like(tok), out_mask=torch.empty_like(fl),
                out_score=torch.empty(B, P, dtype=torch.float32, device="cuda"))
    got = dd.verify(None, ver, tok, fl, CONF, 0.5, 16, 0, static_scratch=True, **outs)
    torch.cuda.synchronize()
    assert dd.verify_status() == 0
    assert torch.equal(got[0], ref[0]) and torch.equal(got[1], ref[1])
    assert torch.allclose(got[2], ref[2], rtol=SCORE_REL, atol=SCORE_ABS_FLOOR)
    assert int(got[1].sum()) == B * (P - 16)          # c << 0.5 everywhere: the 16 most confident are kept


def test_static_scratch_rejects_oversized_problems():
    import torch
    from paper_2604_05250_b200 import binding as dd
    B, P, V = 1, 4097, 8                       # one row more than the fixed array holds
    ver = torch.zeros(B, P, V, dtype=torch.bfloat16, device="cuda")
    tok = torch.zeros(B, P, dtype=torch.int32, device="cuda")
    fl = torch.ones(B, P, dtype=torch.uint8, device="cuda")
    outs = dict(out_tokens=torch.empty_like(tok), out_mask=torch.empty_like(fl),
                out_score=torch.empty(B, P, dtype=torch.float32, device="cuda"))
    with pytest.raises(dd.DualDiffError) as e:
        dd.verify(None, ver, tok, fl, CONF, 0.5, 0, 0, static_scratch=True, **outs)
    assert e.value.status == dd.DD_ERR_UNSUPPORTED
    # one chunk per row more than the array holds: 4096 rows x 17 chunks of 8192 logits.  The
    # sizes are rejected before any pointer is looked at, so no tensors of that size are needed.
    p, null = ctypes.c_void_p(16), ctypes.c_void_p(0)
    L = dd.lib()
    assert L.dd_verify_static(null, p, p, p, CONF, 0.5, 0, 0, p, p, p, 16, 256, 126464 + 8192, null) == dd.DD_ERR_UNSUPPORTED
    assert L.dd_verify_static(null, p, p, p, CONF, 0.5, 0, 0, p, p, p, 16, 256, 8 * 8192 * 2 + 8, null) == dd.DD_ERR_UNSUPPORTED
