// Decision stage, row fold and partial publication of dd_verify (warp-level code).
// Included by dd_verify_common.cuh.
#pragma once

namespace ddv {

// ---------------------------------------------------------------------------
// Decision stage for one sequence, run by one warp (the one that completed it).
//
// Minimum-keep top-k without sorting: the k-th largest reliability t among the flagged
// positions is found by a bitwise binary search on the order-preserving integer image of
// the score; positions above t are kept, and those equal to t are kept lowest index first
// until k are kept in all.  This equals ranking by (reliability descending, index ascending).
//
// Lane l owns positions l, l+32, l+64, ...  The keys of a sequence that fits the caller's staging
// area are kept there (shared memory), and in registers as well while there are at most 32 per
// lane; longer sequences re-read them from memory on every pass (33 passes of dependent loads:
// two orders of magnitude slower, so callers size the area for the sequences they expect).
// The code runs once per sequence, from a cold instruction cache: it is written as short loops,
// not unrolled.
// The parameters come by value: only this rare call copies them to the stack.  dry: every
// load and every step, but no store.
constexpr int kDecideRegKeys = 1024;     // keys a warp can also hold in registers

// `dry` of the decision functions: 0 decides; a rehearsal makes every load and every step but no
// store, and the short one walks through only two steps of the threshold search.
constexpr int kDryFull = 1, kDryShort = 2;

struct DecideStage {            // one per deciding warp
    uint32_t *key;              // shared memory for `capacity` keys (at least 256: the rehearsal's table)
    int capacity;
};

__device__ __noinline__ void decide_sequence_impl(const VerifyParams params, int b, DecideStage *stage, int dry)
{
    // Every field goes into a register once: the stores below are through generic pointers, after
    // which the compiler would have to read the by-value structure again.
    struct {
        const uint8_t *flags; const int32_t *tokens; const float *row_score; const int *row_argmax;
        int32_t *out_tokens; uint8_t *out_mask; float *out_score;
        int P, k, algo, probabilistic, emit_drafter;
        float tau;
        uint32_t seed_lo, seed_hi;
    } p;
    p.flags = params.flags; p.tokens = params.tokens; p.row_score = params.row_score; p.row_argmax = params.row_argmax;
    p.out_tokens = params.out_tokens; p.out_mask = params.out_mask; p.out_score = params.out_score;
    p.P = params.P; p.k = params.k; p.algo = params.algo; p.probabilistic = params.probabilistic;
    p.emit_drafter = params.emit_drafter; p.tau = params.tau; p.seed_lo = params.seed_lo; p.seed_hi = params.seed_hi;

    const int lane = threadIdx.x & 31;
    const unsigned full = 0xFFFFFFFFu;
    // every access below is at base + i with i < P: one check of the sequence index covers them
    const long base = (long)checked(params, b, params.B, kSiteSeq) * p.P;
    const bool kl_mode = p.algo == DD_MODE_KL;
    const int nk = (p.P + 31) / 32;                 // positions per lane (upper bound)
    const bool staged = stage != nullptr && p.P <= stage->capacity;      // without a staging area: re-read from memory
    uint32_t *const skey = staged ? stage->key : nullptr;
    const bool in_regs = staged && p.P <= kDecideRegKeys;

    // key of position i: order-preserving image of its reliability, 0 outside the set.
    // Both loads are unconditional (the score slot exists for every position), so a pass
    // over the keys is a batch of independent loads.
    auto load_key = [&](int i) -> uint32_t {
        const int ic = min(i, p.P - 1);
        const uint8_t f = p.flags[base + ic];
        const float s = __ldcg(p.row_score + base + ic);
        return (i < p.P && f) ? orderable(kl_mode ? 0.0f - s : s) : 0u;
    };
    if (staged) {
        // eight positions per lane at a time: every load of the group first (independent, so
        // they overlap), then the stores
        for (int r0 = 0; r0 < nk; r0 += 8) {
            uint32_t k[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) k[u] = load_key(lane + 32 * (r0 + u));
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int i = lane + 32 * (r0 + u);
                if (r0 + u < nk) skey[i] = k[u];      // i < 32 nk <= capacity rounded up to 32 (the area is a multiple of 32)
            }
        }
        __syncwarp();
    }
    auto key_at = [&](int r) -> uint32_t { return staged ? skey[lane + 32 * r] : load_key(lane + 32 * r); };
    auto score_of = [&](uint32_t key) -> float {     // inverse of the key map (key != 0)
        const float rel = __uint_as_float((key & 0x80000000u) ? (key ^ 0x80000000u) : ~key);
        return kl_mode ? 0.0f - rel : rel;
    };
    // number of keys of the whole sequence with key >= cand, or key > cand.  The threshold search
    // below makes 33 passes: from registers (up to 32 keys per lane), else from the staging area,
    // else from memory.
    uint32_t kr[kDecideRegKeys / 32];
#pragma unroll
    for (int r = 0; r < kDecideRegKeys / 32; ++r) kr[r] = (in_regs && r < nk) ? skey[lane + 32 * r] : 0u;
    auto count_keys = [&](uint32_t cand, bool strictly) -> int {
        int c0 = 0, c1 = 0, c2 = 0, c3 = 0;
        const uint32_t bound = strictly ? cand : cand - 1u;      // cand >= 1 when not strict
        if (in_regs) {
            if (nk <= 8) {
#pragma unroll
                for (int r = 0; r < 8; r += 4) {
                    c0 += kr[r] > bound; c1 += kr[r + 1] > bound; c2 += kr[r + 2] > bound; c3 += kr[r + 3] > bound;
                }
            } else {
#pragma unroll
                for (int r = 0; r < kDecideRegKeys / 32; r += 4) {
                    c0 += kr[r] > bound; c1 += kr[r + 1] > bound; c2 += kr[r + 2] > bound; c3 += kr[r + 3] > bound;
                }
            }
        } else if (staged) {
            // slots past the sequence hold 0 (the staging loop wrote load_key's 0 there)
            // sixteen independent loads per step: a pass is bound by their issue, not their latency
            const uint32_t *kp = skey + lane;
            int r = 0;
            for (; r + 15 < nk; r += 16) {
#pragma unroll
                for (int u = 0; u < 16; u += 4) {
                    c0 += kp[32 * (r + u)] > bound; c1 += kp[32 * (r + u + 1)] > bound;
                    c2 += kp[32 * (r + u + 2)] > bound; c3 += kp[32 * (r + u + 3)] > bound;
                }
            }
            for (; r < nk; ++r) c0 += kp[32 * r] > bound;
        } else {
#pragma unroll 4
            for (int r = 0; r < nk; ++r) {
                const uint32_t k = load_key(lane + 32 * r);
                c0 += strictly ? (k > cand) : (k >= cand);
            }
        }
        return __reduce_add_sync(full, c0 + c1 + c2 + c3);
    };

    // Eq. 6 normaliser: sum of KL over the drafter-decoded set, in a fixed order
    const int n_flagged = count_keys(0u, true);
    double kl_sum = 0.0;
    if (kl_mode && p.probabilistic) {
        double part = 0.0;
        for (int r = 0; r < nk; ++r) {
            const uint32_t k = key_at(r);
            if (k) part += (double)score_of(k);
        }
        kl_sum = warp_sum(part);
    }
    auto fails = [&](int i, float s) -> bool {
        if (p.algo == DD_MODE_TRUST) return false;
        if (!p.probabilistic) return kl_mode ? (s > p.tau) : (s < p.tau);
        const uint32_t w = philox_first_word((uint32_t)i, (uint32_t)b, p.seed_lo, p.seed_hi);
        const double u = (double)(w >> 8) * (1.0 / 16777216.0);
        const double prob = kl_mode ? (kl_sum > 0.0 ? (double)s / kl_sum : 0.0) : 1.0 - (double)s;
        return u < prob;
    };

    bool any_fail = false;
    if (p.k > 0 && p.algo != DD_MODE_TRUST) {
        for (int r = 0; r < nk; ++r) {
            const uint32_t k = key_at(r);
            any_fail |= k != 0u && fails(lane + 32 * r, score_of(k));
        }
        any_fail = __any_sync(full, any_fail);
    }

    // top-k threshold, needed only if some position fails and fewer than all are protected
    uint32_t thr = 0u;          // k-th largest key
    int quota = 0;              // how many of the positions equal to thr are still kept
    bool topk_active = false, keep_all = false;
    if (any_fail) {
        if (n_flagged <= p.k) {
            keep_all = true;
        } else {
            topk_active = true;
            for (int bit = 31; bit >= 0; --bit) {
                const uint32_t cand = thr | (1u << bit);
                if (count_keys(cand, false) >= p.k) thr = cand;
            }
            quota = p.k - count_keys(thr, true);
        }
    }

    // final pass, eight positions per lane at a time: first every load of the group (they are
    // independent, so they overlap), then the decisions and the stores
    int equal_seen = 0;         // positions equal to thr at lower indices
    for (int r0 = 0; r0 < nk; r0 += 8) {
        uint32_t key[8];
        int32_t tok[8], top[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int i = lane + 32 * (r0 + u);
            const bool in = r0 + u < nk && i < p.P;
            key[u] = r0 + u < nk ? key_at(r0 + u) : 0u;
            tok[u] = in ? p.tokens[base + i] : 0;
            top[u] = (in && key[u] != 0u) ? __ldcg(p.row_argmax + base + i) : 0;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int r = r0 + u;
            if (r >= nk) break;                     // uniform
            const int i = lane + 32 * r;
            const long t = base + i;
            const bool flagged = key[u] != 0u;
            bool protect = keep_all;
            if (topk_active) {
                const bool eq = flagged && key[u] == thr;
                const unsigned eq_mask = __ballot_sync(full, eq);
                const int my_rank = equal_seen + __popc(eq_mask & ((1u << lane) - 1u));
                equal_seen += __popc(eq_mask);
                protect = key[u] > thr || (eq && my_rank < quota);
            }
            if (i >= p.P || dry) continue;
            if (!flagged) {
                p.out_tokens[t] = tok[u];
                p.out_mask[t] = 0;
                if (p.out_score) p.out_score[t] = 0.0f;
                continue;
            }
            const float s = score_of(key[u]);       // exactly the stored score
            const bool remask = fails(i, s) && !protect;
            p.out_mask[t] = remask ? 1 : 0;
            p.out_tokens[t] = (remask || p.emit_drafter) ? tok[u] : top[u];
            if (p.out_score) p.out_score[t] = s;
        }
    }
}

}  // namespace ddv

#include "dd_verify_decide_small.cuh"

namespace ddv {

// Short sequences are decided from registers, longer ones from the staging area.
__device__ __forceinline__ void decide_dispatch(const VerifyParams &p, int b, DecideStage *stage, int dry)
{
    if (p.P <= 256) decide_sequence_small<8>(p, b, dry);
    else if (p.P <= 512) decide_sequence_small<16>(p, b, dry);
    else decide_sequence_impl(p, b, stage, dry);
}

__device__ __forceinline__ void decide_sequence(const VerifyParams &p, int b, DecideStage *stage)
{
    decide_dispatch(p, b, stage, 0);
}

// Runs the decision code on sequence 0 without storing anything.  The decision runs once per
// sequence, at the very end of a launch that has streamed the instruction lines out of every
// cache; a warp with nothing to do yet calls this to bring them back in.
__device__ __forceinline__ void decide_sequence_rehearsal(const VerifyParams &p, DecideStage *stage, bool brief)
{
    decide_dispatch(p, 0, stage, brief ? kDryShort : kDryFull);
}

// One sequence has one more completed row; the warp that completes the sequence decides it.
__device__ __forceinline__ void row_done(const VerifyParams &p, int b, DecideStage *stage)
{
    const int lane = threadIdx.x & 31;
    int last = 0;
    if (lane == 0) {
        __threadfence();
        last = atomicAdd(p.seq_counter + checked(p, b, p.B, kSiteSeq), 1u) == (unsigned)(p.P - 1);
    }
    last = __shfl_sync(0xFFFFFFFFu, last, 0);
    if (!last) return;
    __threadfence();
    if (lane == 0) p.seq_counter[b] = 0u;      // ready for the next launch
    decide_sequence(p, b, stage);
}

// 16 bytes from shared or global memory, never from a stale cache line or register copy.
__device__ __forceinline__ float4 ld_volatile16(const void *ptr)
{
    float4 r;
    asm volatile("ld.volatile.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w) : "l"(ptr));
    return r;
}

// Folds n chunk partials of one row, in chunk order, in fp64 (warp-level; src may point to
// shared or global memory).  Every lane returns the row's score (KL_i of Eq. 5, or c_i of
// Eq. 7) and the lowest index of the verifier's maximum.
template <bool KL>
__device__ __noinline__ void fold_partials(const Partial *src, int n, float &score, int &argmax)
{
    const int lane = threadIdx.x & 31;
    float bm_v = -INFINITY, bm_d = -INFINITY;
    int bidx = 0x7FFFFFFF;
    for (int ch = lane; ch < n; ch += 32) {
        const float4 a = ld_volatile16(src + ch);
        const float mv = a.x, md = a.w;
        const int ix = __float_as_int(a.z);
        if (mv > bm_v || (mv == bm_v && ix < bidx)) { bm_v = mv; bidx = ix; }
        bm_d = fmaxf(bm_d, md);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float om = __shfl_xor_sync(0xFFFFFFFFu, bm_v, o);
        const int oi = __shfl_xor_sync(0xFFFFFFFFu, bidx, o);
        if (om > bm_v || (om == bm_v && oi < bidx)) { bm_v = om; bidx = oi; }
        bm_d = fmaxf(bm_d, __shfl_xor_sync(0xFFFFFFFFu, bm_d, o));
    }
    const float Mv = __fmul_rn(bm_v, kLog2e), Md = __fmul_rn(bm_d, kLog2e);
    double sv = 0.0, sd = 0.0, tt = 0.0;
    for (int ch = lane; ch < n; ch += 32) {
        const float4 a = ld_volatile16(src + ch);
        const float4 bq = ld_volatile16(reinterpret_cast<const float4 *>(src + ch) + 1);
        // the factor that moves a chunk's sums to the row's reference point is a power of two with a
        // fractional exponent: one ex2.approx (2^-22 relative, the accuracy of every term inside
        // the chunk sums), not a double-precision exp2 (a long software routine on this path,
        // which sits at the very end of a launch).  The product is rounded on its own (no fused
        // multiply-add), as Mv and Md were: the maximum's chunk gets the factor 2^0 exactly.
        sv += (double)a.y * (double)ex2_approx(__fmul_rn(a.x, kLog2e) - Mv);
        if (KL) {
            const double f = (double)ex2_approx(__fmul_rn(a.w, kLog2e) - Md);
            sd += (double)bq.x * f;
            tt += (double)bq.y * f;
        }
    }
    sv = warp_sum(sv);
    if (KL) { sd = warp_sum(sd); tt = warp_sum(tt); }
    float sc = 0.f;
    if (KL) {
        // lane 0 takes the verifier's logarithm while lane 1 takes the drafter's
        const double lse = (lane == 0 ? (double)Mv : (double)Md) * kLn2 + log(lane == 0 ? sv : sd);
        const double lse_d = __shfl_sync(0xFFFFFFFFu, lse, 1);
        if (lane == 0) {
            const double kl = tt / sd - lse_d + lse;
            sc = (float)fmax(kl, 0.0);
        }
    } else if (lane == 0) {
        // the maximum's own term is 2^(m*log2e - M), not exactly 1
        sc = (float)(exp2((double)bm_v * (double)kLog2e - (double)Mv) / sv);
    }
    score = __shfl_sync(0xFFFFFFFFu, sc, 0);
    argmax = bidx;
}

// The calling warp saw the row's last chunk published to global memory: fold the row, store
// its score and argmax, and report the row to its sequence.
template <bool KL>
__device__ __forceinline__ void fold_row(const VerifyParams &p, int row, DecideStage *stage)
{
    const int lane = threadIdx.x & 31;
    __threadfence();
    float score;
    int argmax;
    const long n_rows = (long)p.B * p.P;
    fold_partials<KL>(p.partials + checked_run(p, (long)row * p.nchunks, p.nchunks, n_rows * p.nchunks, kSitePartial),
                      p.nchunks, score, argmax);
    if (lane == 0) {
        const size_t row_at = checked(p, row, n_rows, kSiteRow);
        __stcg(p.row_score + row_at, score);
        __stcg(p.row_argmax + row_at, argmax);
        p.row_counter[row_at] = 0u;      // ready for the next launch
    }
    __syncwarp();
    row_done(p, row / p.P, stage);
}

// Publishes up to 32 finished (row, chunk) partials at once -- lane l holds entry l, its row in
// pad0 and its chunk in pad1 (as integer bits) -- with one fence for the whole batch; the rows
// whose last chunk was among them are then folded one after the other.  An entry with a
// negative chunk stands for an unflagged row, which is only reported to its sequence.
template <bool KL>
__device__ __forceinline__ void publish_batch(const VerifyParams &p, const Partial &c, int n, DecideStage *stage)
{
    const int lane = threadIdx.x & 31;
    const unsigned full = 0xFFFFFFFFu;
    const int row = __float_as_int(c.pad0), chunk = __float_as_int(c.pad1);
    const bool mine = lane < n;
    if (mine && chunk >= 0) {
        Partial *dst = p.partials + checked(p, (long)row * p.nchunks + chunk, (long)p.B * p.P * p.nchunks, kSitePartial);
        const float4 a = make_float4(c.m_v, c.s_v, __int_as_float(c.idx), c.m_d);
        const float4 bq = make_float4(c.s_d, c.t, 0.f, 0.f);
        __stcg(reinterpret_cast<float4 *>(dst), a);
        __stcg(reinterpret_cast<float4 *>(dst) + 1, bq);
    }
    __threadfence();
    bool last = false;
    if (mine && chunk >= 0)
        last = atomicAdd(p.row_counter + checked(p, row, (long)p.B * p.P, kSiteRow), 1u) == (unsigned)(p.nchunks - 1);
    unsigned todo = __ballot_sync(full, last);
    while (todo) {
        const int src = __ffs(todo) - 1;
        todo &= todo - 1;
        fold_row<KL>(p, __shfl_sync(full, row, src), stage);
    }
    todo = __ballot_sync(full, mine && chunk < 0);
    while (todo) {
        const int src = __ffs(todo) - 1;
        todo &= todo - 1;
        row_done(p, __shfl_sync(full, row, src) / p.P, stage);
    }
}

// One partial, held by every lane alike.
template <bool KL>
__device__ __forceinline__ void chunk_done(const VerifyParams &p, int row, int chunk, Partial c, DecideStage *stage)
{
    c.pad0 = __int_as_float(row);
    c.pad1 = __int_as_float(chunk);
    publish_batch<KL>(p, c, 1, stage);
}

}  // namespace ddv
