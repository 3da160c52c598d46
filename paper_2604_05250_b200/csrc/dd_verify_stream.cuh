// Streaming kernel of dd_verify (V % 8 == 0, 16-byte aligned logits).
//
// One persistent CTA per SM: fifteen warps stream, one warp publishes.  The flagged rows'
// (row, chunk) units (3 to 8 pieces of 1024 logits, chosen per launch so that the units of a
// range come out in whole rounds of the streaming warps) are numbered in row order and cut into equal
// contiguous ranges, one per CTA (more when a range would not fit the CTA's table).  The
// range's units go to the streaming warps in turn.  A warp walks its unit in pieces of 1024
// logits per tensor (2048 of the verifier when there is no drafter tensor): every lane holds
// four 16-byte vectors per tensor of the current piece (eight of the verifier)
// in registers and has the loads of the next piece in flight while it computes (the
// measured copy bandwidth is reached with this depth; a shared-memory ring fed by bulk
// copies reached it too but cost about four times the instructions per piece).  Within a
// chunk every lane keeps its own running maxima, reference points and sums (packed bf16x2
// maxima, packed fp32 pairs); lanes talk to each other only when the chunk ends.  The
// chunk's partial goes into a table in shared memory; the warp that stores a row's last
// chunk folds the row there, so a row that lies inside one range costs no global round
// trip.  Rows cut by a range boundary go through global memory as chunk partials plus one
// counter update per range.  The publishing warp takes finished rows from a shared-memory
// queue, stores their scores, updates the sequence counters in batches (one fence per
// batch) and decides completed sequences, so the streaming warps never wait for global
// memory other than their logits.
#pragma once

#include "dd_verify_common.cuh"

namespace ddv {

constexpr int kSStreamWarps = 15;                             // warps that stream
constexpr int kSWarps = kSStreamWarps + 1;                    // + one that publishes finished chunks
constexpr int kSThreads = kSWarps * 32;
constexpr int kSQueue = 64;                                   // finished-chunk queue slots
constexpr int kPiece = 32 * kVecPerThread * 8;                // 1024 logits per tensor per step of a warp
constexpr int kMinPiecesPerChunk = 3, kMaxPiecesPerChunk = 8; // a (row, chunk) unit is 3072 .. 8192 logits
constexpr int kSChunk = kPiece * kMaxPiecesPerChunk;
constexpr int kSTable = 768;                                  // chunk partials a CTA keeps per range
constexpr unsigned kErrWaitQueue = 0x800;

// Logits per tensor in one step of a warp.  Without a drafter tensor (TRUST, CONF) the registers
// that would hold the drafter's vectors hold four more vectors of the verifier: the piece is twice
// as long, so that a warp has as many bytes in flight as in KL mode.
template <bool KL>
struct PieceOf {
    static constexpr int value = KL ? kPiece : 2 * kPiece;
};

__device__ __forceinline__ uint4 ld_stream(const uint4 *ptr)
{
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(ptr));
    return r;
}

// Running state of one lane over the pieces of a chunk.
struct LaneState {
    uint32_t max2_v, max2_d;   // packed bf16x2 running maxima (even / odd logits of the lane's words)
    uint32_t where2_v;         // per half: ordinal of the word that first attained the verifier's maximum
    float M_v, M_d;            // reference points: lane maximum * log2e
    float2 s_v, s_d, t;        // sums of the even / odd logits
};

__device__ __forceinline__ void lane_reset(LaneState &L)
{
    L.max2_v = L.max2_d = 0xFF80FF80u;     // -inf, -inf
    L.where2_v = 0u;
    L.M_v = L.M_d = -INFINITY;
    L.s_v = L.s_d = L.t = make_float2(0.f, 0.f);
}

// One piece (n logits, a multiple of 8; lane's vector j covers logits (lane + 32 j) * 8 ..+7).
// KL: rv / rd are the verifier's / drafter's vectors 0..3.  Otherwise rv holds the verifier's
// vectors 0..3 and rd its vectors 4..7.  kFull: no vector is absent.
template <bool KL, bool kFull>
__device__ __forceinline__ void lane_piece(LaneState &L, const uint4 (&rv)[kVecPerThread],
                                           const uint4 (&rd)[kVecPerThread], int n, int lane, int ordinal)
{
    // pass 1: packed running maxima; the word ordinal (within this piece) where a half first rose
    uint32_t max2_v = L.max2_v, max2_d = L.max2_d, where2 = 0u;
#pragma unroll
    for (int j = 0; j < kVecPerThread; ++j) {
        const uint32_t wv[4] = {rv[j].x, rv[j].y, rv[j].z, rv[j].w};
        const uint32_t wd[4] = {rd[j].x, rd[j].y, rd[j].z, rd[j].w};
#pragma unroll
        for (int h = 0; h < 4; ++h) {
            const __nv_bfloat162 w = *reinterpret_cast<const __nv_bfloat162 *>(&wv[h]);
            const __nv_bfloat162 m = *reinterpret_cast<const __nv_bfloat162 *>(&max2_v);
            const uint32_t rose = __hgt2_mask(w, m);                  // 0xFFFF per half that rises
            const __nv_bfloat162 m_new = __hmax2(m, w);
            max2_v = *reinterpret_cast<const uint32_t *>(&m_new);
            const uint32_t q2 = (uint32_t)(j * 4 + h) * 0x00010001u;
            where2 = (where2 & ~rose) | (q2 & rose);
            if (KL) {
                const __nv_bfloat162 d = *reinterpret_cast<const __nv_bfloat162 *>(&wd[h]);
                const __nv_bfloat162 md = __hmax2(*reinterpret_cast<const __nv_bfloat162 *>(&max2_d), d);
                max2_d = *reinterpret_cast<const uint32_t *>(&md);
            }
        }
    }
    if (!KL) {
        // the verifier's vectors 4..7, after 0..3: words are visited in the order of their logits,
        // so a maximum that occurs twice keeps its first place
#pragma unroll
        for (int j = 0; j < kVecPerThread; ++j) {
            const uint32_t wd[4] = {rd[j].x, rd[j].y, rd[j].z, rd[j].w};
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                const __nv_bfloat162 w = *reinterpret_cast<const __nv_bfloat162 *>(&wd[h]);
                const __nv_bfloat162 m = *reinterpret_cast<const __nv_bfloat162 *>(&max2_v);
                const uint32_t rose = __hgt2_mask(w, m);
                const __nv_bfloat162 m_new = __hmax2(m, w);
                max2_v = *reinterpret_cast<const uint32_t *>(&m_new);
                const uint32_t q2 = (uint32_t)((kVecPerThread + j) * 4 + h) * 0x00010001u;
                where2 = (where2 & ~rose) | (q2 & rose);
            }
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
        L.max2_d = max2_d;
    }
    // move the reference points; the sums follow
    const float M_v = fmaxf(bf16lo(max2_v), bf16hi(max2_v)) * kLog2e;
    {
        const float f = rescale_factor(L.M_v, M_v);
        L.s_v = __fmul2_rn(L.s_v, make_float2(f, f));
        L.M_v = M_v;
    }
    float M_d = 0.f;
    if (KL) {
        M_d = fmaxf(bf16lo(max2_d), bf16hi(max2_d)) * kLog2e;
        const float f = rescale_factor(L.M_d, M_d);
        L.s_d = __fmul2_rn(L.s_d, make_float2(f, f));
        L.t = __fmul2_rn(L.t, make_float2(f, f));
        L.M_d = M_d;
    }
    // pass 2: one ex2 per logit against the lane's reference
    const float2 log2e2 = make_float2(kLog2e, kLog2e);
    const float2 nMv2 = make_float2(-M_v, -M_v), nMd2 = make_float2(-M_d, -M_d);
    const float2 neg1 = make_float2(-1.f, -1.f);
    float2 s_v = L.s_v, s_d = L.s_d, t = L.t;
#pragma unroll
    for (int j = 0; j < kVecPerThread; ++j) {
        if (kFull || (lane + j * 32) * 8 < n) {
            const uint32_t wv[4] = {rv[j].x, rv[j].y, rv[j].z, rv[j].w};
            const uint32_t wd[4] = {rd[j].x, rd[j].y, rd[j].z, rd[j].w};
#pragma unroll
            for (int h = 0; h < 4; ++h) {
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
// the warp's maxima first, then every lane's sums moved to them and added up.
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
    int idx = my_m == c.m_v ? my_idx : 0x7FFFFFFF;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) idx = min(idx, __shfl_xor_sync(0xFFFFFFFFu, idx, o));
    c.idx = idx;
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

// A finished row (or a range's share of a row cut by a range boundary), handed from a
// streaming warp to the publishing warp.
struct RowEvent {
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
    unsigned int pad;
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
