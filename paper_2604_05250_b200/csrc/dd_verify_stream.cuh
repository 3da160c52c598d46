// Streaming kernel of dd_verify (V % 8 == 0, 16-byte aligned logits).
//
// One persistent CTA per SM: fifteen streaming warps and one publishing warp.
//
// Work.  A flagged row is cut into chunks of a fixed number of logits (a multiple of the stage
// size); the (row, chunk) units of all flagged rows, numbered in row order, are cut into equal
// contiguous ranges, one per CTA (more, taken in rounds, when a range would not fit the CTA's
// table).  A unit is the work of one streaming warp and yields one partial; inside the CTA the
// range's units go to whichever warp asks next.  Which warp computes a unit never changes the
// unit's partial, and rows are folded from their partials in chunk order, so the results
// depend neither on the grid nor on timing.
//
// Data path.  Every streaming warp owns a ring of two 4 KB stages in shared memory.  One lane
// issues bulk asynchronous copies from global memory into a stage (1024 logits of both
// tensors, or 2048 of the verifier alone), completing on the stage's mbarrier; the warp waits
// for the stage, loads its eight 16-byte vectors per lane, and as soon as the first pass has
// consumed the registers the same lane re-arms the stage with the piece two steps ahead.
// The copy instructions run on the warp-uniform datapath: issued by one lane they cost a few
// dozen cycles per piece, issued by a separate warp on behalf of fifteen others they
// serialised into thousands.  No lane computes a global address in the arithmetic.
//
// Arithmetic.  Within a chunk every lane keeps its own state: packed bf16x2 running maxima of
// the verifier with the ordinal of the word where each half first rose (the lowest index of
// the maximum without a second look at the data), and fp32 pair sums S_V, S_D,
// T = sum 2^(..)(l_D - l_V) against reference points fixed by the lane's first piece of the
// chunk (any reference works as long as it is reused; an overflow of the range shows up as a
// non-finite sum and sends the chunk to a careful scalar path, as do logits of -inf).  Lanes
// talk to each other only when the chunk ends: the 32 lane states become one partial in the
// CTA's table in shared memory.
//
// Rows.  The warp that stores the last chunk of a row's share of the range folds the row
// there, in chunk order in fp64 (Eq. 5, Eq. 7): a row that lies inside one range costs no
// global round trip.  The two rows a range may share with its neighbours go through global
// memory (their partials, one fence and one counter update per range; the last arriver folds
// the same partials in the same order), and their units are handed out first, so that they are
// complete long before the range is.  The publishing warp takes finished rows from a queue in
// shared memory, stores their scores, counts them per sequence (one fence and one counter
// update per sequence and range) and decides the sequences it completes (Section 3.2).
#pragma once

#include "dd_verify_common.cuh"

namespace ddv {

constexpr int kSConsumers = 15;                               // warps that stream
constexpr int kSPublisherWarp = kSConsumers;                  // one warp that publishes finished rows
constexpr int kSWarps = kSConsumers + 1;
constexpr int kSThreads = kSWarps * 32;
constexpr int kSStages = 2;                                   // ring slots per streaming warp (three gain nothing)
constexpr int kSStageBytes = 4096;
constexpr int kSRingBytes = kSConsumers * kSStages * kSStageBytes;
constexpr int kSDecideKeys = 8192;                            // keys of one sequence the publishing warp can keep in shared memory
constexpr int kSQueue = 64;                                   // finished-row queue slots
constexpr int kSTable = 640;                                  // chunk partials a CTA keeps per range
constexpr int kPiece = 32 * kVecPerThread * 8;                // 1024 logits per tensor per stage (KL)
constexpr int kMaxPiecesPerChunk = 8;
constexpr int kSChunk = kPiece * kMaxPiecesPerChunk;          // coarsest cut of a row: 8192 logits
constexpr unsigned kErrWaitQueue = 0x800, kErrWaitFull = 0x900;

// Logits per tensor in one stage.  Without a drafter tensor (TRUST, CONF) the half of the stage
// that would hold the drafter's logits holds 1024 more of the verifier's.
template <bool KL>
struct PieceOf {
    static constexpr int value = KL ? kPiece : 2 * kPiece;
};

// ---- mbarrier and bulk-copy wrappers (shared::cta addresses as 32-bit integers) ----------------
__device__ __forceinline__ uint32_t s_addr(const void *ptr) { return (uint32_t)__cvta_generic_to_shared(ptr); }
__device__ __forceinline__ void sbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
// Named barrier of the CTA over `count` threads (a multiple of 32; id 0 is __syncthreads): wait, or
// arrive without waiting (the waiting side counts the arrival).
__device__ __forceinline__ void cta_bar_sync(uint32_t id, uint32_t count)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
__device__ __forceinline__ void cta_bar_arrive(uint32_t id, uint32_t count)
{
    asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(count) : "memory");
}

__device__ __forceinline__ void sbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void sbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool sbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// L2 policy for data that is read once: first in line for eviction.  Without it the streamed
// logits push everything else out of the L2, and the kernel that runs next (the attention of the
// following step) was measured 4.5 us slower.
__device__ __forceinline__ uint64_t l2_evict_first_policy()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
// bytes (a multiple of 16) from global to shared memory, both 16-byte aligned; completes on `bar`
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar, uint64_t policy)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy) : "memory");
}

// Running state of one lane over the pieces of a chunk.
// Packed bf16x2 maximum of two words.
__device__ __forceinline__ uint32_t bf16x2_max(uint32_t a, uint32_t b)
{
    const __nv_bfloat162 m = __hmax2(*reinterpret_cast<const __nv_bfloat162 *>(&a), *reinterpret_cast<const __nv_bfloat162 *>(&b));
    return *reinterpret_cast<const uint32_t *>(&m);
}

// A chunk whose sum T = sum e (l_D - l_V) exceeds this many times its sum of weights S_D cannot come
// from logits of any model (an average difference of 10^4 nats); it is what a token excluded by
// the verifier alone leaves behind once -inf has been raised to the lowest finite bf16
// (3.4e38 times the token's weight).  Such a chunk goes to the scalar routine, which returns the
// infinite divergence.  A token the drafter gives a probability below 10^4 / 3.4e38 = 3e-35
// of the chunk's mass escapes the test and counts as excluded by both models.
constexpr float kExcludedExcess = 1e4f;

struct LaneState {
    uint32_t max2_v;           // packed bf16x2 running maxima of the verifier (even / odd logits of the lane's words)
    uint32_t where2_v;         // per half: ordinal of the word that first attained that maximum
    uint32_t max2_d;           // drafter: packed maxima of the lane's first piece (its reference point)
    float M_v, M_d;            // reference points: maximum of the lane's first piece * log2e
    float2 s_v, s_d, t;        // sums of the even / odd logits
};

__device__ __forceinline__ void lane_reset(LaneState &L)
{
    L.max2_v = L.max2_d = 0xFF80FF80u;     // -inf, -inf
    L.where2_v = 0u;
    L.M_v = L.M_d = -INFINITY;
    L.s_v = L.s_d = L.t = make_float2(0.f, 0.f);
}

// First pass over a piece: the verifier's packed running maxima and where they rose.  Lane's
// vector j covers logits (lane + 32 j) * 8 ..+7 of the piece.  KL: rv / rd are the verifier's /
// drafter's vectors 0..3; otherwise rv holds the verifier's vectors 0..3 and rd its vectors 4..7.
// Absent vectors hold -inf.  `first`: the piece opens a chunk and fixes the lane's reference points.
template <bool KL>
__device__ __forceinline__ void lane_pass1(LaneState &L, const uint4 (&rv)[kVecPerThread],
                                           const uint4 (&rd)[kVecPerThread], int ordinal, bool first)
{
    uint32_t max2_v = L.max2_v, where2 = 0u;
#pragma unroll
    for (int j = 0; j < (KL ? 1 : 2) * kVecPerThread; ++j) {
        // words are visited in the order of their logits, so a maximum that occurs twice keeps its first place
        const uint4 &x = j < kVecPerThread ? rv[j] : rd[j - kVecPerThread];
        const uint32_t wv[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int h = 0; h < 4; ++h) {
            const __nv_bfloat162 w = *reinterpret_cast<const __nv_bfloat162 *>(&wv[h]);
            const __nv_bfloat162 m = *reinterpret_cast<const __nv_bfloat162 *>(&max2_v);
            const uint32_t rose = __hgt2_mask(w, m);                  // 0xFFFF per half that rises
            const __nv_bfloat162 m_new = __hmax2(m, w);
            max2_v = *reinterpret_cast<const uint32_t *>(&m_new);
            const uint32_t q2 = (uint32_t)(j * 4 + h) * 0x00010001u;
            where2 = (where2 & ~rose) | (q2 & rose);
        }
    }
    {
        // halves that rose during this piece take (piece ordinal, word ordinal)
        const __nv_bfloat162 before = *reinterpret_cast<const __nv_bfloat162 *>(&L.max2_v);
        const __nv_bfloat162 after = *reinterpret_cast<const __nv_bfloat162 *>(&max2_v);
        const uint32_t rose = __hgt2_mask(after, before);
        const uint32_t q2 = where2 + (uint32_t)(ordinal * (KL ? 16 : 32)) * 0x00010001u;
        L.where2_v = (L.where2_v & ~rose) | (q2 & rose);
        L.max2_v = max2_v;
    }
    if (first) {
        L.M_v = fmaxf(bf16lo(max2_v), bf16hi(max2_v)) * kLog2e;
        if (KL) {
            uint32_t max2_d = 0xFF80FF80u;
#pragma unroll
            for (int j = 0; j < kVecPerThread; ++j) {
                const uint32_t wd[4] = {rd[j].x, rd[j].y, rd[j].z, rd[j].w};
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    const __nv_bfloat162 md = __hmax2(*reinterpret_cast<const __nv_bfloat162 *>(&max2_d),
                                                      *reinterpret_cast<const __nv_bfloat162 *>(&wd[h]));
                    max2_d = *reinterpret_cast<const uint32_t *>(&md);
                }
            }
            L.max2_d = max2_d;
            L.M_d = fmaxf(bf16lo(max2_d), bf16hi(max2_d)) * kLog2e;
        }
    }
}

// Second pass: one ex2 per logit against the lane's reference points.  kFull: no vector is absent;
// otherwise the piece has n logits (a multiple of 8) and vectors beyond them are skipped.
template <bool KL, bool kFull>
__device__ __forceinline__ void lane_pass2(LaneState &L, const uint4 (&rv)[kVecPerThread],
                                           const uint4 (&rd)[kVecPerThread], int n, int lane)
{
    const float2 log2e2 = make_float2(kLog2e, kLog2e);
    const float2 nMv2 = make_float2(-L.M_v, -L.M_v), nMd2 = make_float2(-L.M_d, -L.M_d);
    const float2 neg1 = make_float2(-1.f, -1.f);
    float2 s_v = L.s_v, s_d = L.s_d, t = L.t;
#pragma unroll
    for (int j = 0; j < kVecPerThread; ++j) {
        if (kFull || (lane + j * 32) * 8 < n) {
            uint32_t wv[4] = {rv[j].x, rv[j].y, rv[j].z, rv[j].w};
            uint32_t wd[4] = {rd[j].x, rd[j].y, rd[j].z, rd[j].w};
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                if (KL) {
                    // An excluded token (logit -inf) has weight 2^(-inf) = 0 either way, but in
                    // e * (d - v) it would be 0 * inf: both logits are raised to the lowest finite
                    // bf16 first, so the term of a token the drafter excludes is an exact 0
                    // whatever the verifier says.  (A token only the verifier excludes then adds
                    // e * 3.4e38 instead of infinity: kExcludedExcess below catches that.)
                    wv[h] = bf16x2_max(wv[h], 0xFF7FFF7Fu);
                    wd[h] = bf16x2_max(wd[h], 0xFF7FFF7Fu);
                }
                const float2 v2 = make_float2(bf16lo(wv[h]), bf16hi(wv[h]));
                const float2 a = __ffma2_rn(v2, log2e2, nMv2);
                s_v = __fadd2_rn(s_v, make_float2(ex2_approx(a.x), ex2_approx(a.y)));
                if (KL) {
                    const float2 d2 = make_float2(bf16lo(wd[h]), bf16hi(wd[h]));
                    const float2 b = __ffma2_rn(d2, log2e2, nMd2);
                    const float2 e2 = make_float2(ex2_approx(b.x), ex2_approx(b.y));
                    s_d = __fadd2_rn(s_d, e2);
                    t = __ffma2_rn(e2, __ffma2_rn(v2, neg1, d2), t);          // e * (d - v)
                }
            }
        }
    }
    if (!KL) {
#pragma unroll
        for (int j = 0; j < kVecPerThread; ++j) {
            if (kFull || (lane + (kVecPerThread + j) * 32) * 8 < n) {
                const uint32_t wd[4] = {rd[j].x, rd[j].y, rd[j].z, rd[j].w};
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    const float2 v2 = make_float2(bf16lo(wd[h]), bf16hi(wd[h]));
                    const float2 a = __ffma2_rn(v2, log2e2, nMv2);
                    s_v = __fadd2_rn(s_v, make_float2(ex2_approx(a.x), ex2_approx(a.y)));
                }
            }
        }
    }
    L.s_v = s_v; L.s_d = s_d; L.t = t;
}

// The chunk has ended: the 32 lane states become one partial (the same bits in every lane):
// the warp's maxima first, then every lane's sums moved to them and added up.  The drafter's
// "maximum" is the largest of the lanes' reference points: the sums only need a common one.
template <bool KL>
__device__ __forceinline__ Partial lanes_to_partial(const LaneState &L, int chunk_begin, int lane)
{
    Partial c;
    const float lo_m = bf16lo(L.max2_v), hi_m = bf16hi(L.max2_v);
    auto element_of = [&](uint32_t q, int odd) {     // q = piece * 16 + j * 4 + h (KL), piece * 32 + j * 4 + h
        const int piece = KL ? (int)(q >> 4) : (int)(q >> 5);
        const int vec = KL ? (int)((q >> 2) & 3u) : (int)((q >> 2) & 7u);
        return chunk_begin + piece * PieceOf<KL>::value + (lane + 32 * vec) * 8 + 2 * (int)(q & 3u) + odd;
    };
    const int e_lo = element_of(L.where2_v & 0xFFFFu, 0), e_hi = element_of(L.where2_v >> 16, 1);
    const float my_m = fmaxf(lo_m, hi_m);
    const int my_idx = lo_m > hi_m ? e_lo : (hi_m > lo_m ? e_hi : min(e_lo, e_hi));
    c.m_v = warp_max(my_m);
    c.idx = __reduce_min_sync(0xFFFFFFFFu, my_m == c.m_v ? my_idx : 0x7FFFFFFF);
    c.s_v = warp_sum((L.s_v.x + L.s_v.y) * rescale_factor(L.M_v, c.m_v * kLog2e));
    c.m_d = 0.f; c.s_d = 0.f; c.t = 0.f;
    if (KL) {
        c.m_d = warp_max(fmaxf(bf16lo(L.max2_d), bf16hi(L.max2_d)));
        const float f = rescale_factor(L.M_d, c.m_d * kLog2e);
        c.s_d = warp_sum((L.s_d.x + L.s_d.y) * f);
        c.t = warp_sum((L.t.x + L.t.y) * f);
    }
    c.pad0 = c.pad1 = 0.f;
    return c;
}

// The same partial computed one logit at a time, straight from global memory, with every special
// case spelled out: a logit of -inf is probability zero and contributes no term (Eq. 5 runs over
// the support of p_D), a token only the verifier excludes makes the divergence infinite, and the
// reference points are the true maxima.  Rare: a chunk comes here only when the packed path
// produced a non-finite sum.
template <bool KL>
__device__ __noinline__ Partial careful_chunk_partial(const uint16_t *verifier_row, const uint16_t *drafter_row,
                                                      int begin, int end)
{
    const int lane = threadIdx.x & 31;
    float mv = -INFINITY, md = -INFINITY;
    int idx = 0x7FFFFFFF;
    for (int e = begin + lane; e < end; e += 32) {
        const float v = bf16lo((uint32_t)verifier_row[e]);
        if (v > mv) { mv = v; idx = e; }
        if (KL) md = fmaxf(md, bf16lo((uint32_t)drafter_row[e]));
    }
    Partial c;
    c.m_v = warp_max(mv);
    c.idx = __reduce_min_sync(0xFFFFFFFFu, (mv == c.m_v && idx != 0x7FFFFFFF) ? idx : 0x7FFFFFFF);
    if (c.idx == 0x7FFFFFFF) c.idx = begin;               // every logit is -inf: the lowest index
    c.m_d = KL ? warp_max(md) : 0.f;
    const float Mv = c.m_v * kLog2e, Md = c.m_d * kLog2e;
    float sv = 0.f, sd = 0.f, t = 0.f;
    for (int e = begin + lane; e < end; e += 32) {
        const float v = bf16lo((uint32_t)verifier_row[e]);
        if (v != -INFINITY) sv += ex2_approx(fmaf(v, kLog2e, -Mv));
        if (KL) {
            const float d = bf16lo((uint32_t)drafter_row[e]);
            if (d != -INFINITY) {
                const float ed = ex2_approx(fmaf(d, kLog2e, -Md));
                sd += ed;
                if (ed > 0.f) t = fmaf(ed, d - v, t);
            }
        }
    }
    c.s_v = warp_sum(sv);
    c.s_d = KL ? warp_sum(sd) : 0.f;
    c.t = KL ? warp_sum(t) : 0.f;
    c.pad0 = c.pad1 = 0.f;
    return c;
}

// A finished row (or a range's share of a row cut by a range boundary), handed from a
// streaming warp to the publishing warp.
struct __align__(16) RowEvent {
    int row;
    int whole;        // 1: the row lay inside the range and is folded: score and argmax are final
    float score;
    int argmax;
    int first_slot;   // whole == 0: the range's chunks of this row are table slots first_slot ..
    int first_chunk;  //             and chunks first_chunk .. of the row,
    int count;        //             count of them
    int pad;
};

// Queue of row events between the streaming warps (many producers) and the publishing warp
// (one consumer), in shared memory.
struct EventQueue {
    RowEvent entry[kSQueue];
    unsigned int ready[kSQueue];     // sequence number + 1 of the entry the slot holds
    unsigned int tail;               // next sequence number to hand out
    unsigned int head;               // entries below this have been taken
    unsigned int done;               // streaming warps that have finished the current range
    unsigned int next_unit;          // units of the current range handed out so far
};

// One lane of a streaming warp hands over an entry.  False if the queue stayed full.
__device__ __forceinline__ bool queue_push(EventQueue &q, const RowEvent &e)
{
    const unsigned int seq = atomicAdd(&q.tail, 1u);
    volatile unsigned int *head = &q.head;
    unsigned it = 0;
    while (seq - *head >= (unsigned)kSQueue) {
        if (++it > (1u << 22)) return false;
        __nanosleep(64);
    }
    q.entry[seq % kSQueue] = e;
    __threadfence_block();
    *(volatile unsigned int *)&q.ready[seq % kSQueue] = seq + 1u;
    return true;
}

}  // namespace ddv

#include "dd_verify_stream_kernel.cuh"
