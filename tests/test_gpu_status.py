"""Recorded timeouts: a launch whose bounded wait expired makes the next call fail fast, without a
synchronisation, until dd_clear_status() re-arms the kernel.  The expiry is produced by the test
hook (a one-thread kernel whose own short wait runs out): nothing stalls, nothing faults."""
import numpy as np
import pytest

from paper_2604_05250_b200 import synth
from tests._parity import bf16_tensor_to_f64, check_attention, check_verify, to_torch_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dd():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2604_05250_b200 import binding, build
    build.build()
    binding.lib()
    return binding


def test_attention_refuses_after_a_recorded_timeout_and_recovers(dd, oracle_mod):
    import torch
    q, k, v = synth.attention_inputs(1, 2, 200, 128, seed=3)
    tq, tk, tv = (to_torch_bf16(x, "cuda") for x in (q, k, v))
    dd.clear_status()
    dd.bidir_attention(tq, tk, tv)
    torch.cuda.synchronize()
    assert dd.attention_status() == dd.DD_OK
    try:
        dd.debug_expire_wait(0)
        torch.cuda.synchronize()
        out = torch.full_like(tq, 7.0)
        with pytest.raises(dd.DualDiffError) as e:
            dd.bidir_attention(tq, tk, tv, out=out)
        assert e.value.status == dd.DD_ERR_TIMEOUT
        with pytest.raises(dd.DualDiffError) as e:
            dd.block_attention(tq, tk, tv, out=out)
        assert e.value.status == dd.DD_ERR_TIMEOUT
        torch.cuda.synchronize()
        assert (out == 7.0).all()                       # nothing was launched
        assert dd.attention_status() == dd.DD_ERR_TIMEOUT
        assert dd.verify_status() == dd.DD_OK           # the other kernel's word is its own
    finally:
        dd.clear_status()
    assert dd.attention_status() == dd.DD_OK
    got = dd.bidir_attention(tq, tk, tv)
    torch.cuda.synchronize()
    check_attention(bf16_tensor_to_f64(got), oracle_mod.attention(q, k, v, 128 ** -0.5))


def test_verify_refuses_after_a_recorded_timeout_and_recovers(dd, oracle_mod):
    import torch
    dra, ver, tokens, flags = synth.verify_inputs(2, 24, 4096, 17, 0.2, seed=5)
    args = (to_torch_bf16(dra, "cuda"), to_torch_bf16(ver, "cuda"), torch.from_numpy(tokens).cuda(),
            torch.from_numpy(flags).cuda(), 1, 0.5, 3, 0)
    dd.clear_status()
    dd.verify(*args)
    torch.cuda.synchronize()
    try:
        dd.debug_expire_wait(1)
        torch.cuda.synchronize()
        for call in (lambda: dd.verify(*args), lambda: dd.unmask(args[1], args[2], args[3], 0.5, 1)):
            with pytest.raises(dd.DualDiffError) as e:
                call()
            assert e.value.status == dd.DD_ERR_TIMEOUT
        outs = dict(out_tokens=torch.empty_like(args[2]), out_mask=torch.empty_like(args[3]),
                    out_score=torch.empty(2, 24, dtype=torch.float32, device="cuda"))
        with pytest.raises(dd.DualDiffError) as e:
            dd.verify(*args, static_scratch=True, **outs)
        assert e.value.status == dd.DD_ERR_TIMEOUT
        assert dd.verify_status() == dd.DD_ERR_TIMEOUT and dd.attention_status() == dd.DD_OK
    finally:
        dd.clear_status()
    assert dd.verify_status() == dd.DD_OK
    ot, om, osc = dd.verify(*args)
    torch.cuda.synchronize()
    ref = oracle_mod.verify(dra, ver, tokens, flags, 1, 0.5, 3, 0)
    check_verify(ot.cpu().numpy(), om.cpu().numpy(), osc.cpu().numpy(), ref, flags, tokens)
    assert dd.lib().dd_debug_expire_wait(2, None) == dd.DD_ERR_INVALID_ARG
