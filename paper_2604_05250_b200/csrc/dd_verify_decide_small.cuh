// Decision stage for short sequences (P <= 32 R), run by one warp: the same rules and the
// same results as decide_sequence_impl, with everything a lane needs about its R positions --
// key, token, verifier argmax -- loaded once, in one batch of independent loads, and kept in
// registers.  Included by dd_verify_decide.cuh.
#pragma once

namespace ddv {

template <int R>
__device__ __noinline__ void decide_sequence_small(const VerifyParams params, int b, int dry)
{
    const int lane = threadIdx.x & 31;
    const unsigned full = 0xFFFFFFFFu;
    // every field used goes into a register once (the stores below are through generic pointers)
    const uint8_t *flags = params.flags;
    const int32_t *tokens = params.tokens;
    const float *row_score = params.row_score;
    const int *row_argmax = params.row_argmax;
    int32_t *out_tokens = params.out_tokens;
    uint8_t *out_mask = params.out_mask;
    float *out_score = params.out_score;
    const int P = params.P, k_keep = params.k, algo = params.algo;
    const bool probabilistic = params.probabilistic != 0, emit_drafter = params.emit_drafter != 0;
    const float tau = params.tau;
    const uint32_t seed_lo = params.seed_lo, seed_hi = params.seed_hi;
    const bool kl_mode = algo == DD_MODE_KL;
    // every access below is at base + i with i < P: one check of the sequence index covers them
    const long base = (long)checked(params, b, params.B, kSiteSeq) * P;

    // lane l owns positions l, l + 32, ...: key (order-preserving image of the reliability, 0
    // outside the set), token and verifier argmax
    uint32_t key[R];
    int32_t tok[R], top[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int i = lane + 32 * r, ic = min(i, P - 1);
        const uint8_t f = flags[base + ic];
        const float s = __ldcg(row_score + base + ic);
        tok[r] = tokens[base + ic];
        top[r] = __ldcg(row_argmax + base + ic);
        key[r] = (i < P && f) ? orderable(kl_mode ? 0.0f - s : s) : 0u;
    }
    auto score_of = [&](uint32_t kk) -> float {     // inverse of the key map (kk != 0)
        const float rel = __uint_as_float((kk & 0x80000000u) ? (kk ^ 0x80000000u) : ~kk);
        return kl_mode ? 0.0f - rel : rel;
    };
    // number of keys of the whole sequence above `bound`
    auto count_above = [&](uint32_t bound) -> int {
        int c0 = 0, c1 = 0;
#pragma unroll
        for (int r = 0; r < R; r += 2) { c0 += key[r] > bound; c1 += key[r + 1] > bound; }
        return __reduce_add_sync(full, c0 + c1);
    };

    const int n_flagged = count_above(0u);
    // Eq. 6 normaliser: sum of KL over the drafter-decoded set, in a fixed order
    double kl_sum = 0.0;
    if (kl_mode && probabilistic) {
        double part = 0.0;
#pragma unroll
        for (int r = 0; r < R; ++r) if (key[r]) part += (double)score_of(key[r]);
        kl_sum = warp_sum(part);
    }
    // which of the lane's positions fail the rule (bit r)
    unsigned fail_bits = 0u;
    if (algo != DD_MODE_TRUST) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
            if (key[r] == 0u) continue;
            const float s = score_of(key[r]);
            bool fail;
            if (!probabilistic) {
                fail = kl_mode ? (s > tau) : (s < tau);
            } else {
                const uint32_t w = philox_first_word((uint32_t)(lane + 32 * r), (uint32_t)b, seed_lo, seed_hi);
                const double u = (double)(w >> 8) * (1.0 / 16777216.0);
                const double prob = kl_mode ? (kl_sum > 0.0 ? (double)s / kl_sum : 0.0) : 1.0 - (double)s;
                fail = u < prob;
            }
            fail_bits |= fail ? 1u << r : 0u;
        }
    }
    const bool any_fail = k_keep > 0 && __any_sync(full, fail_bits != 0u);

    // minimum-keep top-k: k-th largest key by a bitwise search; ties to the lower index
    uint32_t thr = 0u;
    int quota = 0;
    bool topk_active = false, keep_all = false;
    if (any_fail) {
        if (n_flagged <= k_keep) {
            keep_all = true;
        } else {
            topk_active = true;
            // (a short rehearsal walks through two of the 32 steps: each waits for the one before
            // it, and the whole search is a third of this function's time)
            for (int bit = 31; bit >= (dry == kDryShort ? 30 : 0); --bit) {
                const uint32_t cand = thr | (1u << bit);
                if (count_above(cand - 1u) >= k_keep) thr = cand;      // keys >= cand
            }
            quota = k_keep - count_above(thr);
        }
    }

    int equal_seen = 0;         // positions equal to thr at lower indices
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int i = lane + 32 * r;
        const long t = base + i;
        const bool flagged = key[r] != 0u;
        bool protect = keep_all;
        if (topk_active) {
            const bool eq = flagged && key[r] == thr;
            const unsigned eq_mask = __ballot_sync(full, eq);
            const int my_rank = equal_seen + __popc(eq_mask & ((1u << lane) - 1u));
            equal_seen += __popc(eq_mask);
            protect = key[r] > thr || (eq && my_rank < quota);
        }
        if (i >= P || dry) continue;
        const bool remask = flagged && ((fail_bits >> r) & 1u) != 0u && !protect;
        out_mask[t] = remask ? 1 : 0;
        out_tokens[t] = (!flagged || remask || emit_drafter) ? tok[r] : top[r];
        if (out_score) out_score[t] = flagged ? score_of(key[r]) : 0.0f;
    }
}

}  // namespace ddv
