"""Toy "models" for the Algorithm 1 loop tests: stand-ins for a drafter and a verifier network
(the repository holds no model).  Test fixture only."""
import numpy as np

from paper_2604_05250_b200.synth import f32_to_bf16_bits


class ToyModel:
    """Deterministic logits as a function of the token sequence: position i of sequence b gets
    fixed N(0,1) noise over the vocabulary plus a bump on the token the model believes in,
    ``base + gain * (share of the sequence that is already unmasked)``: like a real masked
    diffusion model it grows more confident as context fills in.  The drafter's beliefs differ
    from the target on a fixed set of positions (its errors); the verifier's do not.

    ``model(tokens)``: int32 [B,P] numpy -> uint16 [B,P,V] (bf16 bits).
    """

    def __init__(self, target, V, mask_id, seed, wrong_share=0.0, base=2.0, gain=6.0):
        assert mask_id == V - 1 and int(np.max(target)) < V - 1, "tokens 0..V-2, the mask id is V-1"
        rng = np.random.default_rng([int(seed), 0x70F])
        B, P = target.shape
        self.mask_id = int(mask_id)
        self.noise = rng.standard_normal((B, P, V), dtype=np.float32)
        self.belief = np.array(target, dtype=np.int64, copy=True)
        wrong = rng.random((B, P)) < wrong_share
        # a wrong belief is another ordinary token (the mask id, the last of the vocabulary, is none)
        shift = rng.integers(1, V - 1, size=(B, P))
        self.belief[wrong] = (self.belief[wrong] + shift[wrong]) % (V - 1)
        self.jitter = rng.random((B, P)).astype(np.float32)
        self.base, self.gain = np.float32(base), np.float32(gain)

    def __call__(self, tokens):
        B, P, V = self.noise.shape
        known = (np.asarray(tokens) != self.mask_id).mean(axis=1).astype(np.float32)      # [B]
        bump = self.base + self.gain * known[:, None] + self.jitter                          # [B,P]
        logits = self.noise.copy()
        b_idx, p_idx = np.meshgrid(np.arange(B), np.arange(P), indexing="ij")
        logits[b_idx, p_idx, self.belief] += bump
        return f32_to_bf16_bits(logits)
