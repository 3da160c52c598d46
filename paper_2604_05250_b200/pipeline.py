"""Algorithm 1 (the DualDiffusion loop) as host-side orchestration of the library's calls.

The drafter and the verifier are callables supplied by the user (the models themselves are
not part of this library): each maps the current token tensor [B,P] (int32, on the device)
to logits [B,P,V] (bfloat16, on the device).  Every step of the algorithm that touches logits
runs in the CUDA library: ``dd_unmask`` for the drafter's K unmasking steps, ``dd_verify`` for
the verification algorithm A.  What is left here is the control flow of Algorithm 1: which
positions are masked, which were decoded by the drafter in the current cycle, and when to stop.
"""
from __future__ import annotations

from dataclasses import dataclass, field

from . import binding as dd


@dataclass
class LoopStats:
    cycles: int = 0
    drafter_calls: int = 0
    verifier_calls: int = 0
    unmasked_by_drafter: int = 0
    remasked_by_verifier: int = 0
    masked_after_cycle: list = field(default_factory=list)


def dualdiffusion_generate(drafter, verifier, tokens, mask_id, K, mode, tau, k, seed=0,
                           unmask_tau=float("inf"), unmask_k=1, max_cycles=10_000):
    """Runs Algorithm 1 until no position holds ``mask_id`` (or ``max_cycles`` is reached).

    tokens: int32 [B,P] device tensor, ``mask_id`` where a token is still to be generated.
    K: drafter steps per cycle.  mode, tau, k, seed: as for ``dd_verify`` (the verification
    algorithm and its threshold, minimum-keep count and Philox seed; the seed is advanced by
    one per cycle).  unmask_tau, unmask_k: the drafter's unmasking rule as for ``dd_unmask``.
    In KL mode the drafter is evaluated once more on the drafted sequence, which is the
    distribution Eq. 5 names.  Returns (tokens, LoopStats).
    """
    import torch
    x = tokens.clone()
    stats = LoopStats()
    algo = mode & 0xFF
    while stats.cycles < max_cycles:
        masked = (x == mask_id)
        if not bool(masked.any()):
            break
        drafted = torch.zeros_like(masked)
        # ---- drafting phase: K unmasking steps of the fast model
        for _ in range(K):
            flags = masked.to(torch.uint8)
            if not bool(masked.any()):
                break
            logits_d = drafter(x)
            stats.drafter_calls += 1
            x_new, still, _ = dd.unmask(logits_d, x, flags, unmask_tau, unmask_k)
            newly = masked & (still == 0)
            drafted |= newly
            stats.unmasked_by_drafter += int(newly.sum())
            x = x_new
            masked = still.bool()
        # ---- verification phase: one step of the accurate model over the drafted positions
        logits_v = verifier(x)
        stats.verifier_calls += 1
        logits_d = None
        if algo == dd.DD_MODE_KL:
            logits_d = drafter(x)
            stats.drafter_calls += 1
        out_tokens, remask, _ = dd.verify(logits_d, logits_v, x, drafted.to(torch.uint8), mode, tau, k,
                                          seed + stats.cycles)
        remask = remask.bool()
        x = torch.where(remask, torch.full_like(out_tokens, mask_id), out_tokens)
        stats.remasked_by_verifier += int(remask.sum())
        stats.cycles += 1
        stats.masked_after_cycle.append(int((x == mask_id).sum()))
    return x, stats
