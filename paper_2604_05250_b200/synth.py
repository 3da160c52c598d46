"""Seeded synthetic inputs for one DualDiffusion verification step.

These generators feed identical arrays to the CUDA library and to the CPU
oracle.  They hold none of the method's arithmetic: only random draws, the
bf16 rounding of those draws, and the table of workload shapes.  The shapes
stand in for LLaDA-8B activations and logits (32 heads of 128, vocabulary
126464, 768 prompt + 256 generated positions), which are not available here.

bf16 tensors are numpy ``uint16`` bit patterns.
"""
from __future__ import annotations

import numpy as np

# ----------------------------------------------------------------------------
# bf16 <-> fp32 bit helpers (data formatting only)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


# ----------------------------------------------------------------------------
# workload table

ATTENTION_CONFIGS = {
    0: dict(B=1, H=4, N=128, D=64, planted=False),        # tiny
    1: dict(B=1, H=32, N=1024, D=128, planted=False),     # LLaDA-8B-shaped verify step
    2: dict(B=16, H=32, N=512, D=128, planted=False),     # batched serving
    3: dict(B=1, H=32, N=8192, D=128, planted=True),      # long context, rank-16 q.k structure
}
ATTENTION_SWEEP_N = (256, 1024, 4096, 16384)              # B*N fixed at 16384, H=32, D=128

MODE_TRUST, MODE_KL, MODE_CONF = 0, 1, 2
FLAG_PROBABILISTIC, FLAG_EMIT_DRAFTER = 0x100, 0x200

VERIFY_CONFIGS = {
    0: dict(B=1, P=128, V=1024, flagged=32, err=0.10, tau=0.5, k=8, seed=0,
            modes=(MODE_TRUST, MODE_KL, MODE_CONF)),
    1: dict(B=1, P=256, V=126464, flagged="all", err=0.10, tau=0.5, k=32, seed=0,
            modes=(MODE_KL,)),
    2: dict(B=16, P=256, V=126464, flagged="uniform_25_100", err=0.10, tau=0.5, k=16, seed=0,
            modes=(MODE_CONF,)),
    3: dict(B=1, P=512, V=126464, flagged="all", err=0.10, tau=0.5, k=32, seed=0,
            modes=(MODE_TRUST, MODE_KL)),
}
VERIFY_SWEEP = dict(V=(32000, 126464), flagged=(32, 128, 512), err=(0.05, 0.20, 0.50),
                    P=512, tau=0.5, seeds=(0, 1, 2, 3))


def config_seed(config_index: int, sweep_seed: int = 0) -> int:
    return config_index * 1000 + sweep_seed


# ----------------------------------------------------------------------------
# attention inputs


def attention_inputs(B, H, N, D, seed, planted=False, rank=16, strength=3.0):
    """q, k, v as [B,H,N,D] uint16 (bf16 bits), entries ~ N(0,1).

    planted=True adds a shared low-rank component to q and k: per head an
    orthonormal W [rank,D]; q_i += strength * z_i W, k_j += strength * z'_j W
    with z, z' ~ N(0,I).  Scores then have heavy, peaked rows.
    """
    rng = np.random.default_rng([int(seed), 0xA77])
    shape = (B, H, N, D)
    q = rng.standard_normal(shape, dtype=np.float32)
    k = rng.standard_normal(shape, dtype=np.float32)
    v = rng.standard_normal(shape, dtype=np.float32)
    if planted:
        for b in range(B):
            for h in range(H):
                g = rng.standard_normal((D, rank))
                w = np.linalg.qr(g)[0].T.astype(np.float32)          # [rank, D], orthonormal rows
                zq = rng.standard_normal((N, rank), dtype=np.float32)
                zk = rng.standard_normal((N, rank), dtype=np.float32)
                q[b, h] += np.float32(strength) * (zq @ w)
                k[b, h] += np.float32(strength) * (zk @ w)
    return f32_to_bf16_bits(q), f32_to_bf16_bits(k), f32_to_bf16_bits(v)


# ----------------------------------------------------------------------------
# verification inputs


def flag_counts(B, P, flagged, rng):
    if flagged == "all":
        return [P] * B
    if flagged == "uniform_25_100":
        return [int(round(float(f) * P)) for f in rng.uniform(0.25, 1.0, size=B)]
    return [min(int(flagged), P)] * B


def verify_inputs(B, P, V, flagged, err, seed, bump=8.0):
    """Drafter/verifier logits and the current sequence state.

    verifier logits ~ N(0, 2^2) with +bump at one random token per position;
    drafter = verifier (before rounding) + N(0, 0.5^2) on a (1-err) share of
    the positions and an independent N(0, 2^2) row (no bump) on the rest.
    tokens = the drafter row's first largest entry; flags mark the
    drafter-decoded set (a random subset of the P positions of each sequence).

    Returns (drafter u16 [B,P,V], verifier u16 [B,P,V], tokens i32 [B,P],
    flags u8 [B,P]).
    """
    rng = np.random.default_rng([int(seed), 0x7E1])
    counts = flag_counts(B, P, flagged, rng)
    drafter = np.empty((B, P, V), dtype=np.uint16)
    verifier = np.empty((B, P, V), dtype=np.uint16)
    tokens = np.empty((B, P), dtype=np.int32)
    flags = np.zeros((B, P), dtype=np.uint8)
    for b in range(B):
        flags[b, np.sort(rng.choice(P, size=counts[b], replace=False))] = 1
        lv = rng.standard_normal((P, V), dtype=np.float32)
        lv *= np.float32(2.0)
        hot = rng.integers(0, V, size=P)
        lv[np.arange(P), hot] += np.float32(bump)
        ld = rng.standard_normal((P, V), dtype=np.float32)
        wrong = rng.random(P) < err
        ld[wrong] *= np.float32(2.0)
        good = ~wrong
        ld[good] *= np.float32(0.5)
        ld[good] += lv[good]
        verifier[b] = f32_to_bf16_bits(lv)
        drafter[b] = f32_to_bf16_bits(ld)
        tokens[b] = np.argmax(bf16_bits_to_f32(drafter[b]), axis=1).astype(np.int32)
    return drafter, verifier, tokens, flags


def verify_config_inputs(config_index: int):
    c = VERIFY_CONFIGS[config_index]
    return verify_inputs(c["B"], c["P"], c["V"], c["flagged"], c["err"],
                         config_seed(config_index, c["seed"]))


def attention_config_inputs(config_index: int):
    c = ATTENTION_CONFIGS[config_index]
    return attention_inputs(c["B"], c["H"], c["N"], c["D"], config_seed(config_index),
                            planted=c["planted"])


# ----------------------------------------------------------------------------
# language-model head inputs


def lm_head_inputs(B, P, K, V, flagged, seed, bump=8.0):
    """Last hidden states [B,P,K] and output embedding [V,K] (uint16 bf16 bits) whose product has the
    statistics of verify_inputs' verifier logits: entries ~ N(0, 2^2), plus about `bump` at one random
    token per position (the hidden state leans towards that token's embedding).  Stands in for
    LLaDA-8B's final hidden states and tied output embedding (K = 4096, V = 126464).

    Returns (hidden u16 [B,P,K], weight u16 [V,K], tokens i32 [B,P], flags u8 [B,P])."""
    rng = np.random.default_rng([int(seed), 0x1E4D])
    counts = flag_counts(B, P, flagged, rng)
    weight = rng.standard_normal((V, K), dtype=np.float32)
    weight *= np.float32(2.0 / np.sqrt(K))
    hidden = rng.standard_normal((B, P, K), dtype=np.float32)
    hot = rng.integers(0, V, size=(B, P))
    hidden += np.float32(bump / 4.0) * weight[hot]               # |w|^2 ~ 4: logit of the hot token rises by ~bump
    tokens = rng.integers(0, V, size=(B, P)).astype(np.int32)
    flags = np.zeros((B, P), dtype=np.uint8)
    for b in range(B):
        flags[b, np.sort(rng.choice(P, size=counts[b], replace=False))] = 1
    return f32_to_bf16_bits(hidden), f32_to_bf16_bits(weight), tokens, flags


def lm_head_pair_inputs(B, P, K, V, flagged, err, seed, bump=8.0):
    """Both models' last hidden states and output embeddings, for the KL mode from hidden states.
    The verifier's pair is lm_head_inputs' (same seed, same values).  The drafter has an embedding
    of its own, the verifier's plus N(0, (0.1 * 2 / sqrt(K))^2) per entry; on a (1 - err) share of
    the positions its hidden state is the verifier's plus N(0, 0.25^2) per entry (logits that
    differ by about N(0, 0.5^2), as in verify_inputs) and the token is the position's hot token,
    on the rest it is an independent N(0, 1) vector (no hot token) and the token is random.

    Returns (drafter_hidden, drafter_weight, verifier_hidden, verifier_weight: uint16 bf16 bits,
    tokens i32 [B,P], flags u8 [B,P])."""
    rng = np.random.default_rng([int(seed), 0x1E4D])
    counts = flag_counts(B, P, flagged, rng)
    weight = rng.standard_normal((V, K), dtype=np.float32)
    weight *= np.float32(2.0 / np.sqrt(K))
    hidden = rng.standard_normal((B, P, K), dtype=np.float32)
    hot = rng.integers(0, V, size=(B, P))
    hidden += np.float32(bump / 4.0) * weight[hot]
    tokens = rng.integers(0, V, size=(B, P)).astype(np.int32)
    flags = np.zeros((B, P), dtype=np.uint8)
    for b in range(B):
        flags[b, np.sort(rng.choice(P, size=counts[b], replace=False))] = 1
    # everything above draws what lm_head_inputs draws, in its order; the drafter comes after
    weight_d = weight + np.float32(0.2 / np.sqrt(K)) * rng.standard_normal((V, K), dtype=np.float32)
    wrong = rng.random((B, P)) < err
    hidden_d = hidden + np.float32(0.25) * rng.standard_normal((B, P, K), dtype=np.float32)
    hidden_d[wrong] = rng.standard_normal((int(wrong.sum()), K), dtype=np.float32)
    tokens = np.where(wrong, tokens, hot).astype(np.int32)
    return (f32_to_bf16_bits(hidden_d), f32_to_bf16_bits(weight_d), f32_to_bf16_bits(hidden),
            f32_to_bf16_bits(weight), tokens, flags)
