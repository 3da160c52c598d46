"""A sample of the parity cases through the bounds-checked build of the library
(-DDD_BOUNDS_CHECK: every index the verification kernels form into a caller's tensor or into the
library's scratch is compared with its extent; a violation is recorded in the health word and
index 0 is used instead).  No memory checker can be run on these kernels here, so this build,
the guard regions around every output and the grid-size invariance tests are what speaks for
their addressing.  The checked build must report nothing and give the normal build's bits."""
import numpy as np
import pytest

from paper_2604_05250_b200 import synth
from tests._parity import to_torch_bf16

pytestmark = pytest.mark.gpu

TRUST, KL, CONF, PROB, EMIT = 0, 1, 2, 0x100, 0x200


@pytest.fixture(scope="module")
def libs():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2604_05250_b200 import binding, build
    build.build()
    return binding, build.build_check()


def both_builds(binding, check_path, call):
    """call() under the normal and under the checked build; the checked one must stay silent."""
    import torch
    normal = [x.cpu().numpy() for x in call()]
    torch.cuda.synchronize()
    assert binding.verify_status() == 0
    with binding.use_library(check_path):
        checked = [x.cpu().numpy() for x in call()]
        torch.cuda.synchronize()
        word = binding.verify_status()
        assert word == 0, f"bounds-checked build recorded {word:#x} (site {(word >> 8) & 0xF}, CTA {word & 0xFF})"
    for a, b in zip(normal, checked):
        assert np.array_equal(a, b)


@pytest.mark.parametrize("B,P,V,flagged,mode", [
    (1, 128, 1024, 32, KL),                      # cfg0
    (2, 96, 20000, 61, KL | PROB),               # ragged last chunk, rows cut by range boundaries
    (3, 40, 126464, 33, CONF),                   # the LLaDA vocabulary
    (2, 50, 1003, 31, KL),                       # V % 8 != 0: the element-wise kernel
    (15, 700, 64, 380, CONF | PROB),             # many short rows, sequences beyond the register-resident decision
    (1, 1500, 4104, 900, TRUST | EMIT),          # a sequence beyond the register-resident decision
    (4, 8, 8, 0, KL),                            # nothing flagged: every sequence passes through
])
def test_verify_addresses_stay_inside(libs, B, P, V, flagged, mode):
    import torch
    binding, check_path = libs
    dra, ver, tokens, flags = synth.verify_inputs(B, P, V, flagged, 0.2, seed=P + V)
    t = [to_torch_bf16(dra, "cuda") if (mode & 0xFF) == KL else None, to_torch_bf16(ver, "cuda"),
         torch.from_numpy(tokens).cuda(), torch.from_numpy(flags).cuda()]
    both_builds(binding, check_path, lambda: binding.verify(t[0], t[1], t[2], t[3], mode, 0.5, 4, 9))


def test_static_scratch_and_unmask(libs):
    import torch
    binding, check_path = libs
    dra, ver, tokens, flags = synth.verify_inputs(2, 96, 20000, 61, 0.2, seed=3)
    t = [to_torch_bf16(dra, "cuda"), to_torch_bf16(ver, "cuda"), torch.from_numpy(tokens).cuda(), torch.from_numpy(flags).cuda()]

    def static_call():
        outs = dict(out_tokens=torch.empty(2, 96, dtype=torch.int32, device="cuda"),
                    out_mask=torch.empty(2, 96, dtype=torch.uint8, device="cuda"),
                    out_score=torch.empty(2, 96, dtype=torch.float32, device="cuda"))
        return binding.verify(t[0], t[1], t[2], t[3], KL, 0.5, 4, 9, static_scratch=True, **outs)
    both_builds(binding, check_path, static_call)
    both_builds(binding, check_path, lambda: binding.unmask(t[1], t[2], t[3], 0.3, 2))


@pytest.mark.parametrize("mode", [CONF | PROB, KL])
def test_fused_heads(libs, mode):
    import torch
    binding, check_path = libs
    dh, dw, vh, vw, tokens, flags = synth.lm_head_pair_inputs(2, 300, 128, 4100, "uniform_25_100", 0.2, seed=8)
    t = [to_torch_bf16(x, "cuda") for x in (dh, dw, vh, vw)]
    tok, fl = torch.from_numpy(tokens).cuda(), torch.from_numpy(flags).cuda()
    d = t[:2] if mode == KL else [None, None]
    both_builds(binding, check_path, lambda: binding.lm_head_verify(d[0], d[1], t[2], t[3], tok, fl, mode, 0.3, 3, 5))
