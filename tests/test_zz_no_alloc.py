"""dd_verify_static, the entry point for callers that cannot allocate device memory
(a server that has given all free memory to its caches, code that must not hit the
implicit synchronisation of cudaMalloc, a process whose allocator belongs to another
runtime).  Its scratch is a fixed array inside the library, so it must give what
dd_verify gives, call after call, whatever the previous call left in that array.

Collected last on purpose: a failure here cannot hide the result of any other test.
"""
import numpy as np
import pytest

from paper_2604_05250_b200 import synth
from tests._parity import SCORE_ABS_FLOOR, SCORE_REL, to_torch_bf16

pytestmark = pytest.mark.gpu

KL, CONF, PROB = 1, 2, 0x100


def both_entry_points(dd, shape, mode, seed):
    import torch
    B, P, V, nflag = shape
    dra, ver, tokens, flags = synth.verify_inputs(B, P, V, nflag, 0.2, seed=seed)
    t_dra, t_ver = to_torch_bf16(dra, "cuda"), to_torch_bf16(ver, "cuda")
    t_tok, t_fl = torch.from_numpy(tokens).cuda(), torch.from_numpy(flags).cuda()
    if (mode & 0xFF) != KL:
        t_dra = None
    ref = dd.verify(t_dra, t_ver, t_tok, t_fl, mode, 0.5, 4, seed)
    outs = (torch.full((B, P), -7, dtype=torch.int32, device="cuda"),
            torch.full((B, P), 9, dtype=torch.uint8, device="cuda"),
            torch.full((B, P), -1.0, dtype=torch.float32, device="cuda"))
    got = dd.verify(t_dra, t_ver, t_tok, t_fl, mode, 0.5, 4, seed, out_tokens=outs[0], out_mask=outs[1],
                    out_score=outs[2], static_scratch=True)
    torch.cuda.synchronize()
    r_tok, r_mask, r_score = (x.cpu().numpy() for x in ref)
    g_tok, g_mask, g_score = (x.cpu().numpy() for x in got)
    assert np.array_equal(g_tok, r_tok)
    assert np.array_equal(g_mask, r_mask)
    tol = np.maximum(SCORE_REL * np.abs(r_score), SCORE_ABS_FLOOR)
    assert (np.abs(g_score - r_score) <= tol).all()
    assert flags.sum() > 0 and (g_score[flags.astype(bool)] > 0).any()


def test_static_scratch_matches_dd_verify_on_two_calls_in_a_row():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2604_05250_b200 import binding as dd
    from paper_2604_05250_b200 import build
    build.build()
    # two consecutive calls with different shapes and modes: the second one runs on whatever the
    # first left in the shared array
    both_entry_points(dd, (2, 96, 20000, 61), KL | PROB, seed=21)
    both_entry_points(dd, (3, 40, 126464, 33), KL, seed=22)
    both_entry_points(dd, (1, 128, 1024, 32), CONF, seed=23)


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
