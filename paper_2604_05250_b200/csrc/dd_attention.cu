// dd_bidir_attention: full-sequence bidirectional attention (Section 2.2; Eq. 3
// evaluated over the whole key range) for sm_100a, and dd_block_attention: the same
// equation for a block of Nq queries against Nkv (cached) keys, with a per-sequence
// number of valid keys and either memory layout.  One kernel serves both.
//
// One CTA owns two tiles of 128 query rows of one (batch, head) and walks over
// the keys in tiles of 128.  The CTA is warp-specialised:
//   warps 0-3   softmax of query tile 0 (thread = query row = TMEM lane)
//   warps 4-7   softmax of query tile 1
//   warp  8     one thread feeds a ring of K/V tiles by TMA (tensor maps over
//               (D, N, B*H) or, heads interleaved, (D, N, H, B); 128-byte swizzle;
//               rows past N read as zero)
//   warp  9     one thread issues every tcgen05 MMA
// S_g = Q_g K^T goes to tensor memory; the softmax thread reads its row, keeps the
// running maximum and sum in fp32 (online softmax in base 2, scale*log2e folded
// into one FMA), writes P = 2^(S - m) as bf16 over the first half of the S columns,
// and O_g += P V is a second MMA whose A operand is read from tensor memory.  While
// one tile's softmax runs, the tensor core works on the other tile.  The reference
// point m of a row only moves when the row maximum has outgrown it by more than 2^24
// (a power-of-two factor common to P and to the row sum changes neither bf16's nor
// fp32's relative precision; the step only has to leave fp32 its range); only then
// is O rescaled in tensor memory.  O is normalised by the row sum at the end and
// rounded to bf16 once.
#include <cuda.h>
#include <cuda_bf16.h>
#include <math.h>

#include <mutex>

#include "dd_common.cuh"
#include "dd_ptx.cuh"

namespace {

using namespace ddptx;

constexpr int kBlockM = 128;        // query rows per tile
constexpr int kQTiles = 2;          // query tiles per CTA
constexpr int kBlockN = 128;        // keys per step
constexpr int kStages = 5;          // K/V ring slots (one tile each)
constexpr int kThreads = 384;
constexpr int kSoftmaxWarps = 8;
constexpr int kLoadWarp = 8, kMmaWarp = 9;
constexpr uint32_t kTmemCols = 512; // S_0 [0,128)  S_1 [128,256)  O_0 [256,256+D)  O_1 [256+D,256+2D)
// log2 of the largest P tolerated before the reference point moves.  A move costs the row's warp a
// wait for the previous P V product, a pass over the accumulator in tensor memory and a second
// weighting of the tile: with a step of 8, rows whose scores are peaked (a planted low-rank
// component; trained heads) moved often enough to cost 25-40 % of the throughput.  With 24 the sum
// of a row's weights stays below N * 2^24 and fp32 holds O for |v| * N < 2^100.
constexpr float kRescaleStep = 24.f;

enum : unsigned { kErrWaitQ = 0x100, kErrWaitKV = 0x200, kErrWaitS = 0x300, kErrWaitO = 0x400,
                  kErrWaitP = 0x500, kErrWaitSlot = 0x600 };

struct AttnParams {
    int BH, H, Nq, Nkv, D;
    int m_blocks;              // CTAs per (batch, head) = ceil(Nq / 256)
    const int *kv_len;         // [B] keys of each sequence that exist (clamped to 0..Nkv), or null: Nkv
    int head_major;            // 1: [B,H,N,D], tensor maps are 3-D over (D, N, B*H); 0: [B,N,H,D], 4-D maps (D, N, H, B)
    float scale_log2;          // scale * log2(e)
    unsigned int *status;      // health word of the attention kernel on this device
    unsigned int *mirror;      // its copy in mapped host memory (written only when a wait expires)
};

template <int D>
struct Smem {
    static constexpr int kTileBytes = kBlockN * D * 2;             // one 128 x D bf16 tile
    static constexpr int kQ = 0;                                   // two query tiles
    static constexpr int kRing = kQTiles * kTileBytes;             // kStages K/V tiles
    static constexpr int kBars = kRing + kStages * kTileBytes;
    // barriers (8 bytes each): q_full[2], kv_full[kStages], kv_empty[kStages], s_full[2], p_full[2], o_full[2]
    static constexpr int kNumBars = 2 + 2 * kStages + 6;
    static constexpr int kTmemSlot = kBars + 8 * kNumBars;
    static constexpr int kTotal = kTmemSlot + 16;
    // every tile starts on the 1024-byte boundary the 128-byte swizzle needs, the barriers on 8 bytes,
    // and the whole layout plus the alignment slack fits what one CTA may ask for
    static_assert(kTileBytes % 1024 == 0 && kBars % 8 == 0, "tiles on swizzle boundaries, barriers on 8 bytes");
    static_assert(kTotal + 1024 <= 227 * 1024, "shared memory of one CTA");
};

__device__ __forceinline__ void report(const AttnParams &p, unsigned code)
{
    const unsigned word = code | (unsigned)(blockIdx.x & 0xFF);
    if (atomicCAS(p.status, 0u, word) == 0u && p.mirror) {
        *reinterpret_cast<volatile unsigned int *>(p.mirror) = word;      // the host sees it without a synchronisation
        __threadfence_system();
    }
}

// One key tile of the online softmax for one query row; s[] holds the raw scores.
// Row maximum of the raw scores (keys past the sequence end excluded).
template <bool kMasked>
__device__ __forceinline__ float row_max(const float (&s)[kBlockN], int valid)
{
    float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
    for (int i = 0; i < kBlockN; i += 4) {
        if (!kMasked || i + 0 < valid) m0 = fmaxf(m0, s[i + 0]);
        if (!kMasked || i + 1 < valid) m1 = fmaxf(m1, s[i + 1]);
        if (!kMasked || i + 2 < valid) m2 = fmaxf(m2, s[i + 2]);
        if (!kMasked || i + 3 < valid) m3 = fmaxf(m3, s[i + 3]);
    }
    return fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
}

// Weights P = 2^(s*c - m_ref) of the tile as packed bf16 into tensor memory, 32 keys (16
// columns) at a time; returns the sum of the weights as rounded, and through mx the row
// maximum of the raw scores seen on the way (so the caller can tell afterwards whether
// m_ref was still a good reference point).  Two values per instruction where the
// hardware has a packed form.
template <bool kMasked>
__device__ __forceinline__ float weights_to_tmem(const float (&s)[kBlockN], int valid, float c, float m_ref,
                                                 uint32_t tmem_p, float &mx)
{
    const float2 c2 = make_float2(c, c), nm2 = make_float2(-m_ref, -m_ref);
    float2 sum2 = make_float2(0.f, 0.f);
    float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
    for (int q = 0; q < kBlockN / 32; ++q) {
        uint32_t pk[16];
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
            const int e = q * 32 + i;
            const float2 a = __ffma2_rn(make_float2(s[e], s[e + 1]), c2, nm2);
            float p0 = ex2(a.x), p1 = ex2(a.y);
            if (kMasked) {
                // keys past the end of the sequence get weight zero (a select, not -inf arithmetic: scale may be 0)
                p0 = e < valid ? p0 : 0.f;
                p1 = e + 1 < valid ? p1 : 0.f;
                if (e < valid) m0 = fmaxf(m0, s[e]);
                if (e + 1 < valid) m1 = fmaxf(m1, s[e + 1]);
            } else {
                m0 = fmaxf(m0, s[e]);
                m1 = fmaxf(m1, s[e + 1]);
            }
            __nv_bfloat162 b = __floats2bfloat162_rn(p0, p1);
            const uint32_t w = *reinterpret_cast<uint32_t *>(&b);
            pk[i / 2] = w;
            // the row sum takes the weights as rounded, so that O / l is an exact convex combination
            sum2 = __fadd2_rn(sum2, make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u)));
        }
        tmem_st16(tmem_p + q * 16, pk);
    }
    mx = fmaxf(m0, m1);
    return sum2.x + sum2.y;
}

// One key tile of one query row, shared by both attention kernels: reads the row's 128 scores
// from tensor memory (the S product has completed), weights them against the reference point the
// row inherits (the first tile of a row takes its own maximum) and writes P over S.  Only a row
// whose maximum turns out to have grown past the reference point by more than the allowed step
// moves it, rescales O in tensor memory (which holds the sum over the earlier tiles once the
// barrier o_full_bar has completed the phase o_parity) and weights the tile again.  Returns 0, or
// the error code of the wait that expired.  The caller hands P over (wait for the stores, fence,
// arrive).
template <int D>
__device__ __forceinline__ unsigned softmax_tile(uint32_t tS, uint32_t tO, uint32_t o_full_bar, uint32_t o_parity,
                                                 bool first, int valid, float c, float &m_ref, float &l_run)
{
    float s[kBlockN];
#pragma unroll
    for (int cb = 0; cb < kBlockN / 32; ++cb)
        tmem_ld32(tS + cb * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[cb * 32]));
    tmem_wait_ld();
    const bool masked = valid < kBlockN;
    if (first) m_ref = (masked ? row_max<true>(s, valid) : row_max<false>(s, valid)) * c;
    float mx;
    float sum = masked ? weights_to_tmem<true>(s, valid, c, m_ref, tS, mx)
                       : weights_to_tmem<false>(s, valid, c, m_ref, tS, mx);
    const bool move = mx * c > m_ref + kRescaleStep;
    if (__any_sync(0xffffffffu, move)) {
        const float m_new = move ? mx * c : m_ref;
        const float alpha = ex2(m_ref - m_new);       // 1 where the row does not move
        m_ref = m_new;
        l_run *= alpha;
        if (!mbar_wait(o_full_bar, o_parity)) return kErrWaitO;
        tc_fence_after();
#pragma unroll
        for (int cb = 0; cb < D / 32; ++cb) {
            uint32_t r[32];
            tmem_ld32(tO + cb * 32, r);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
            tmem_st32(tO + cb * 32, r);
        }
        tmem_wait_st();                               // the first weights are overwritten next
        sum = masked ? weights_to_tmem<true>(s, valid, c, m_ref, tS, mx)
                     : weights_to_tmem<false>(s, valid, c, m_ref, tS, mx);
    }
    l_run += sum;
    return 0;
}

// 32 columns of one output row, scaled, rounded to bf16 and written to the staging tile in the
// 128-byte-swizzled layout of the output tensor map (`stage` = the row's first byte in the tile,
// r = the row, cb = which 32 columns).
__device__ __forceinline__ void columns_to_staging(const uint32_t *acc, float f, uint32_t stage, int r, int cb)
{
    constexpr uint32_t kBoxBytes = 128 * 128;
    const uint32_t box = stage + (cb / 2) * kBoxBytes;   // 64 columns per box
#pragma unroll
    for (int i = 0; i < 32; i += 8) {
        uint32_t w[4];
#pragma unroll
        for (int h = 0; h < 4; ++h) {
            __nv_bfloat162 v = __floats2bfloat162_rn(__uint_as_float(acc[i + 2 * h]) * f, __uint_as_float(acc[i + 2 * h + 1]) * f);
            w[h] = *reinterpret_cast<uint32_t *>(&v);
        }
        const int chunk = (cb % 2) * 4 + i / 8;          // 16-byte chunk of the 128-byte row
        st_shared_v4(box + ((chunk ^ (r & 7)) << 4), w[0], w[1], w[2], w[3]);
    }
}

// kBlock = false: the square, head-major, unpadded case of dd_bidir_attention with nothing of the
// general case compiled in.
template <int D, bool kBlock>
__global__ void __launch_bounds__(kThreads, 1)
attention_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                 const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
                 const AttnParams p)
{
    extern __shared__ __align__(1024) unsigned char smem_dyn[];
    // 128-byte-swizzled tiles must start on a 1024-byte boundary
    const uint32_t smem_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char *smem_gen = smem_dyn + (smem_base - smem_u32(smem_dyn));
    constexpr uint32_t kTileBytes = Smem<D>::kTileBytes;
    const uint32_t sQ = smem_base + Smem<D>::kQ, sRing = smem_base + Smem<D>::kRing;
    const uint32_t bars = smem_base + Smem<D>::kBars;
    auto bar_q = [&](int g) { return bars + 8u * g; };
    auto bar_kv_full = [&](int s) { return bars + 8u * (2 + s); };
    auto bar_kv_empty = [&](int s) { return bars + 8u * (2 + kStages + s); };
    auto bar_s_full = [&](int g) { return bars + 8u * (2 + 2 * kStages + g); };
    auto bar_p_full = [&](int g) { return bars + 8u * (4 + 2 * kStages + g); };
    auto bar_o_full = [&](int g) { return bars + 8u * (6 + 2 * kStages + g); };
    const uint32_t tmem_slot = smem_base + Smem<D>::kTmemSlot;
    volatile uint32_t *tmem_slot_gen = reinterpret_cast<volatile uint32_t *>(smem_gen + Smem<D>::kTmemSlot);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bh = blockIdx.x / p.m_blocks;
    const int mb = blockIdx.x - bh * p.m_blocks;
    const int row0 = mb * (kQTiles * kBlockM);
    const int b_idx = kBlock ? bh / p.H : 0, h_idx = kBlock ? bh - b_idx * p.H : 0;
    const bool hm = !kBlock || p.head_major != 0;
    // one tile of 128 rows x 64 columns of head (b_idx, h_idx), rows from n0
    auto load_box = [&](uint32_t dst, const CUtensorMap *tm, uint32_t bar, int c0, int n0) {
        if (hm) tma_load_3d(dst, tm, bar, c0, n0, bh);
        else tma_load_4d(dst, tm, bar, c0, n0, h_idx, b_idx);
    };
    const int keys = (kBlock && p.kv_len) ? min(max(p.kv_len[b_idx], 0), p.Nkv) : p.Nkv;   // keys that exist
    const int nkv = (keys + kBlockN - 1) / kBlockN;       // 0: the sequence has no key, the output is zero
    const int ntiles = (p.Nq - row0 > kBlockM) ? 2 : 1;   // query tiles of this CTA that hold rows
    // A CTA with a single query tile (a short query block) gives its key tiles to the two softmax
    // groups in turn: both keep a copy of the query tile and an accumulator of their own, and the
    // two partial results are combined at the end.  The tensor core then works for one group
    // while the other computes its weights, as with two query tiles.
    const bool split = kBlock && ntiles == 1 && nkv >= 2;
    const int groups = split ? 2 : ntiles;                // softmax groups at work
    constexpr int kBoxes = D / 64;                 // 64-column (128-byte) boxes per tile row
    constexpr uint32_t kBoxBytes = 128 * 128;      // 128 rows x 128 bytes
    constexpr uint32_t kColS = 0, kColO = 256;

    // The producer thread sets up the barriers its copies complete on and sends the first copies
    // on their way (Q tile 0, K tile 0; not for a sequence without keys, whose Q buffers only stage
    // zeros) before the CTA's first barrier: they travel while tensor memory is allocated and the
    // other barriers are set up (cfg1: 22.9 -> 22.0 us).  Nothing else in the CTA touches those
    // buffers or barriers before the __syncthreads below.
    const bool early = warp == kLoadWarp && lane == 0 && (!kBlock || nkv > 0);
    bool early_sent = false;
    if (warp == kLoadWarp && lane == 0) {
        prefetch_tmap(&tm_q); prefetch_tmap(&tm_k); prefetch_tmap(&tm_v);
        mbar_init(bar_q(0), 1); mbar_init(bar_q(1), 1);
        for (int s = 0; s < kStages; ++s) mbar_init(bar_kv_full(s), 1);
        fence_mbar_init();
        // (also when an earlier wait has expired and the CTA will do nothing: such a CTA lingers at
        // its end until copies in flight have landed)
        if (early) {
            mbar_expect_tx(bar_q(0), kTileBytes);
#pragma unroll
            for (int cx = 0; cx < kBoxes; ++cx) load_box(sQ + cx * kBoxBytes, &tm_q, bar_q(0), cx * 64, row0);
            mbar_expect_tx(bar_kv_full(0), kTileBytes);
#pragma unroll
            for (int cx = 0; cx < kBoxes; ++cx) load_box(sRing + cx * kBoxBytes, &tm_k, bar_kv_full(0), cx * 64, 0);
            early_sent = true;
        }
    }
    if (tid == 0) {
        prefetch_tmap(&tm_o);
        for (int s = 0; s < kStages; ++s) mbar_init(bar_kv_empty(s), 1);
        for (int g = 0; g < kQTiles; ++g) {
            mbar_init(bar_s_full(g), 1);
            mbar_init(bar_p_full(g), kBlockM);
            mbar_init(bar_o_full(g), 1);
        }
        fence_mbar_init();
        // a wait that expired in an earlier CTA or launch stops the rest from queueing up behind it
        tmem_slot_gen[1] = *reinterpret_cast<volatile unsigned int *>(p.status);
    }
    if (warp == 0) { tmem_alloc(tmem_slot, kTmemCols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot_gen;
    const bool healthy = tmem_slot_gen[1] == 0;

    if (!healthy) {
        // nothing to do
    } else if (warp < kSoftmaxWarps) {
        // =================================================================== softmax warpgroups
        reg_inc<216>();
        const int g = warp >> 2;
        const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;   // this warp's 32 TMEM lanes
        const uint32_t tS = tmem + lane_off + kColS + g * kBlockN;
        const uint32_t tO = tmem + lane_off + kColO + g * D;
        const float c = p.scale_log2;
        float m_ref = -INFINITY, l_run = 0.f;
        unsigned err = 0;

        // key tiles of this group: j_first, j_first + j_step, ...
        const int j_first = split ? g : 0, j_step = split ? 2 : 1;
        const int my_tiles = nkv > j_first ? (nkv - j_first + j_step - 1) / j_step : 0;
        if (g < groups) {
            for (int i = 0; i < my_tiles; ++i) {
                const int j = j_first + i * j_step;
                if (!mbar_wait(bar_s_full(g), i & 1)) { err = kErrWaitS; break; }
                tc_fence_after();
                const int valid = keys - j * kBlockN;      // keys of this tile that exist
                const bool masked = valid < kBlockN;
                // O_g holds the sum over tiles < j once the previous P V has completed
                err = softmax_tile<D>(tS, tO, bar_o_full(g), (uint32_t)(i - 1) & 1, i == 0, valid, c, m_ref, l_run);
                if (err) break;
                if (kBlock && masked) {
                    // Keys past the end of the sequence have weight zero, but 0 x NaN is NaN in the
                    // product P V, and padding may hold any bit pattern: clear their value rows in
                    // the ring slot (whole 128-byte rows, which the swizzle maps onto themselves)
                    // before the weights are handed over.  The slot cannot be refilled before this
                    // group's product has read it.
                    const int item_v = 2 * j + 1, slot_v = item_v % kStages;
                    if (!mbar_wait(bar_kv_full(slot_v), (item_v / kStages) & 1)) { err = kErrWaitKV; break; }
                    const int r = (warp & 3) * 32 + lane;
                    if (r >= valid) {
                        const uint32_t row = sRing + slot_v * kTileBytes + r * 128;
#pragma unroll
                        for (int cx = 0; cx < kBoxes; ++cx)
#pragma unroll
                            for (int c16 = 0; c16 < 8; ++c16)
                                st_shared_v4(row + cx * kBoxBytes + c16 * 16, 0u, 0u, 0u, 0u);
                    }
                    fence_proxy_async_smem();
                }
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(bar_p_full(g));
            }
            if (err == 0 && (!kBlock || nkv > 0) && !mbar_wait(bar_o_full(g), (my_tiles - 1) & 1)) err = kErrWaitO;
            // ---- split keys: group 1 hands its reference point and row sum to group 0 (through its
            // own Q buffer, which no MMA reads any more) and is done; group 0 adds group 1's
            // accumulator, read from tensor memory, to its own.  Every thread of both groups takes
            // part in the hand-over, also after an expired wait.
            float scale_own = 1.f, scale_other = 0.f;
            float2 *hand_over = reinterpret_cast<float2 *>(smem_gen + Smem<D>::kQ + kTileBytes);
            if (kBlock && split) {
                const int r = (warp & 3) * 32 + lane;
                if (g == 1) {
                    hand_over[r] = make_float2(m_ref, l_run);
                    __threadfence_block();
                    named_bar_arrive(3, 2 * kBlockM);
                } else {
                    named_bar_sync(3, 2 * kBlockM);
                    const float2 other = hand_over[r];
                    if (err == 0 && !mbar_wait(bar_o_full(1), ((nkv / 2) - 1) & 1)) err = kErrWaitO;
                    const float m_all = fmaxf(m_ref, other.x);
                    scale_own = ex2(m_ref - m_all);
                    scale_other = ex2(other.x - m_all);
                    l_run = l_run * scale_own + other.y * scale_other;
                }
            }
            if (err != 0) report(p, err);
            const bool stores = !(kBlock && split && g == 1);
            if (stores && err == 0) {
                // ---- epilogue: O / l -> bf16 -> this tile's Q buffer (every MMA that read it has
                // completed), in the swizzled layout of the tensor map, -> global by TMA (rows past N
                // are clipped by the map)
                tc_fence_after();
                const int r = (warp & 3) * 32 + lane;                 // row within the tile
                const float inv = (!kBlock || nkv > 0) ? 1.f / l_run : 0.f;
                const float w_own = scale_own * inv, w_other = scale_other * inv;
                const uint32_t stage = sQ + g * kTileBytes + r * 128;
                if constexpr (!kBlock) {
                    // the whole accumulator row in one go: every load is in flight before the first is waited for
                    uint32_t acc[D];
#pragma unroll
                    for (int cb = 0; cb < D / 32; ++cb)
                        tmem_ld32(tO + cb * 32, *reinterpret_cast<uint32_t(*)[32]>(&acc[cb * 32]));
                    tmem_wait_ld();
#pragma unroll
                    for (int cb = 0; cb < D / 32; ++cb) columns_to_staging(&acc[cb * 32], inv, stage, r, cb);
                } else
#pragma unroll
                for (int cb = 0; cb < D / 32; ++cb) {
                    uint32_t acc[32];
                    if (!kBlock || nkv > 0) {
                        tmem_ld32(tO + cb * 32, acc);
                        tmem_wait_ld();
                        if (kBlock && split) {
                            uint32_t acc1[32];
                            tmem_ld32(tO + D + cb * 32, acc1);          // group 1's accumulator, same rows
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i)
                                acc[i] = __float_as_uint(__uint_as_float(acc[i]) * w_own + __uint_as_float(acc1[i]) * w_other);
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) acc[i] = 0u;       // no key: nothing was accumulated
                    }
                    columns_to_staging(acc, (kBlock && split) ? 1.f : inv, stage, r, cb);      // split: already weighted
                }
                fence_proxy_async_smem();
            }
            // every thread of the warpgroup comes here, also after an expired wait
            named_bar_sync(1 + g, kBlockM);
            if (stores && err == 0 && (warp & 3) == 0 && lane == 0) {
#pragma unroll
                for (int cx = 0; cx < kBoxes; ++cx)
                    if (hm) tma_store_3d(&tm_o, sQ + g * kTileBytes + cx * kBoxBytes, cx * 64, row0 + g * kBlockM, bh);
                    else tma_store_4d(&tm_o, sQ + g * kTileBytes + cx * kBoxBytes, cx * 64, row0 + g * kBlockM, h_idx, b_idx);
                tma_store_commit();
                tma_store_wait_read();
            }
        }
    } else {
        reg_dec<72>();
        if (warp == kLoadWarp && lane == 0) {
            // =============================================================== TMA producer
            // what the first MMA needs comes first: Q tile 0, K tile 0, then Q tile 1
            // buffer g takes query tile g, or, with split keys, a second copy of tile 0
            auto load_q = [&](int g) {
                mbar_expect_tx(bar_q(g), kTileBytes);
#pragma unroll
                for (int cx = 0; cx < kBoxes; ++cx)
                    load_box(sQ + g * kTileBytes + cx * kBoxBytes, &tm_q, bar_q(g), cx * 64,
                             row0 + (split ? 0 : g * kBlockM));
            };
            if (!early_sent && (!kBlock || nkv > 0)) load_q(0);      // without keys the Q buffers only stage the zero output
            // ring items: 2j = K tile j, 2j+1 = V tile j
            for (int item = early_sent ? 1 : 0; item < 2 * nkv; ++item) {
                if (item == 1 && groups > 1) load_q(1);
                const int slot = item % kStages, use = item / kStages;
                if (use > 0 && !mbar_wait(bar_kv_empty(slot), (use - 1) & 1)) { report(p, kErrWaitSlot); break; }
                const uint32_t dst = sRing + slot * kTileBytes;
                const CUtensorMap *tm = (item & 1) ? &tm_v : &tm_k;
                mbar_expect_tx(bar_kv_full(slot), kTileBytes);
#pragma unroll
                for (int cx = 0; cx < kBoxes; ++cx)
                    load_box(dst + cx * kBoxBytes, tm, bar_kv_full(slot), cx * 64, (item >> 1) * kBlockN);
            }
        } else if (warp == kMmaWarp && lane == 0) {
            // =============================================================== MMA issuer
            constexpr uint32_t kIdescS = idesc_bf16(kBlockM, kBlockN, false);
            constexpr uint32_t kIdescO = idesc_bf16(kBlockM, D, true);
            // descriptors of a tile are the tile's base descriptor plus the byte offset / 16
            const uint64_t desc_q0 = smem_desc_sw128(sQ, 16, 1024);
            const uint64_t desc_k0 = smem_desc_sw128(sRing, 16, 1024);            // K-major operand (K tile)
            const uint64_t desc_v0 = smem_desc_sw128(sRing, kBoxBytes, 1024);     // MN-major operand (V tile)
            unsigned err = 0;
            // S_g = Q_g K^T for the K tile in `slot`
            auto issue_s = [&](int g, int slot) {
                const uint64_t a = desc_q0 + (uint64_t)(g * (kTileBytes >> 4));
                const uint64_t b = desc_k0 + (uint64_t)(slot * (kTileBytes >> 4));
                const uint32_t tS = tmem + kColS + g * kBlockN;
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t off = ((ks / 4) * kBoxBytes + (ks % 4) * 32) >> 4;   // 16 bf16 = 32 bytes per k-step
                    mma_ss(tS, a + off, b + off, kIdescS, ks > 0);
                }
                mma_commit(bar_s_full(g));
            };
            // O_g (+)= P_g V for the V tile in `slot`
            auto issue_o = [&](int g, int slot, bool first) {
                const uint64_t b = desc_v0 + (uint64_t)(slot * (kTileBytes >> 4));
                const uint32_t tS = tmem + kColS + g * kBlockN, tO = tmem + kColO + g * D;
#pragma unroll
                for (int ks = 0; ks < kBlockN / 16; ++ks) {
                    // 16 keys = two 8-row groups of 1024 bytes; column blocks of 64 are one box apart
                    mma_ts(tO, tS + ks * 8, b + (uint32_t)(ks * (2048 >> 4)), kIdescO, (!first || ks > 0));
                }
                mma_commit(bar_o_full(g));
            };
            auto wait_item = [&](int item) {
                return mbar_wait(bar_kv_full(item % kStages), (item / kStages) & 1);
            };
            // Split keys: key tile t belongs to group t & 1.  S_0(0), S_1(1), then per tile t:
            // O_g (+)= P_g V_t, S_g(t + 2).  Every ring item is read by one group only.
            if (kBlock && split) {
                do {
                    for (int g = 0; g < 2; ++g) {
                        if (!mbar_wait(bar_q(g), 0)) { err = kErrWaitQ; break; }
                        if (!wait_item(2 * g)) { err = kErrWaitKV; break; }
                        tc_fence_after();
                        issue_s(g, (2 * g) % kStages);
                        mma_commit(bar_kv_empty((2 * g) % kStages));
                    }
                    for (int t = 0; t < nkv && err == 0; ++t) {
                        const int g = t & 1, i = t >> 1;
                        const int item_v = 2 * t + 1, item_k = 2 * (t + 2);
                        if (!wait_item(item_v)) { err = kErrWaitKV; break; }
                        if (!mbar_wait(bar_p_full(g), i & 1)) { err = kErrWaitP; break; }
                        tc_fence_after();
                        issue_o(g, item_v % kStages, i == 0);
                        mma_commit(bar_kv_empty(item_v % kStages));
                        if (t + 2 < nkv) {
                            if (!wait_item(item_k)) { err = kErrWaitKV; break; }
                            tc_fence_after();
                            issue_s(g, item_k % kStages);
                            mma_commit(bar_kv_empty(item_k % kStages));
                        }
                    }
                } while (false);
            } else
            do {
                if (kBlock && nkv == 0) break;
                if (!mbar_wait(bar_q(0), 0)) { err = kErrWaitQ; break; }
                if (!wait_item(0)) { err = kErrWaitKV; break; }
                tc_fence_after();
                issue_s(0, 0);
                if (ntiles > 1) {
                    if (!mbar_wait(bar_q(1), 0)) { err = kErrWaitQ; break; }
                    tc_fence_after();
                    issue_s(1, 0);
                }
                mma_commit(bar_kv_empty(0));
                for (int j = 0; j < nkv && err == 0; ++j) {
                    const int item_v = 2 * j + 1, item_k = 2 * j + 2;
                    const bool more = j + 1 < nkv;
                    // both tiles this round reads are waited for here, not between two groups of MMAs:
                    // a wait in between lets the tensor core run dry
                    if (!wait_item(item_v)) { err = kErrWaitKV; break; }
                    if (more && !wait_item(item_k)) { err = kErrWaitKV; break; }
                    for (int g = 0; g < ntiles; ++g) {
                        if (!mbar_wait(bar_p_full(g), j & 1)) { err = kErrWaitP; break; }
                        tc_fence_after();
                        issue_o(g, item_v % kStages, j == 0);
                        if (more) issue_s(g, item_k % kStages);
                    }
                    if (err) break;
                    mma_commit(bar_kv_empty(item_v % kStages));
                    if (more) mma_commit(bar_kv_empty(item_k % kStages));
                }
            } while (false);
            if (err) report(p, err);
        }
    }

    __syncwarp();
    if (*reinterpret_cast<volatile unsigned int *>(p.status) != 0) {
        // a wait expired somewhere: give copies that may still be in flight time to land before the
        // shared memory is released
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) { __syncwarp(); tmem_dealloc(tmem, kTmemCols); }
}

#include "dd_attention_persistent.cuh"

// ---------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// bf16 view of a [B,H,N,D] tensor as (D, N, B*H) (head_major: batch and head merge into one
// dimension) or of a [B,N,H,D] tensor as (D, N, H, B); box = 64 columns x 128 rows x 1 (x 1),
// 128-byte swizzle, zero fill: a tile never reaches into the next head or sequence, and rows
// past N read as zero / are not written.
int make_tmap(CUtensorMap *m, const void *base, int B, int H, int N, int D, bool head_major)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return dd::cuda_fail(cudaErrorSymbolNotFound, "cuTensorMapEncodeTiled entry point");
    const cuuint64_t row = (cuuint64_t)D * 2;
    const cuuint32_t box[4] = {64, 128, 1, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r;
    if (head_major) {
        const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)N, (cuuint64_t)B * H};
        const cuuint64_t strides[2] = {row, row * N};
        r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    } else {
        const cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)N, (cuuint64_t)H, (cuuint64_t)B};
        const cuuint64_t strides[3] = {row * H, row, row * N * H};      // between rows, heads, sequences
        r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    }
    if (r != CUDA_SUCCESS) return dd::cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
    return DD_OK;
}

template <int D, bool kBlock>
int launch(const CUtensorMap &tq, const CUtensorMap &tk, const CUtensorMap &tv, const CUtensorMap &to,
           const AttnParams &p, cudaStream_t s)
{
    static bool attr_done[64] = {};
    static std::mutex attr_mu;
    int dev = 0;
    DD_CUDA_TRY(cudaGetDevice(&dev));
    const int smem = Smem<D>::kTotal + 1024;
    {
        std::lock_guard<std::mutex> lock(attr_mu);
        if (dev >= 0 && dev < 64 && !attr_done[dev]) {
            DD_CUDA_TRY(cudaFuncSetAttribute(attention_kernel<D, kBlock>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
            attr_done[dev] = true;
        }
    }
    const long grid = (long)p.BH * p.m_blocks;
    attention_kernel<D, kBlock><<<(unsigned)grid, kThreads, smem, s>>>(tq, tk, tv, to, p);
    DD_CUDA_TRY(cudaGetLastError());
    dd::count_launch();
    return DD_OK;
}

// The persistent kernel: one CTA per SM (or per item, if there are fewer).
template <int D>
int launch_persistent(const CUtensorMap &tq, const CUtensorMap &tk, const CUtensorMap &tv, const CUtensorMap &to,
                      const AttnParams &p, int sms, cudaStream_t s)
{
    static bool attr_done[64] = {};
    static std::mutex attr_mu;
    int dev = 0;
    DD_CUDA_TRY(cudaGetDevice(&dev));
    const int smem = SmemP<D>::kTotal + 1024;
    {
        std::lock_guard<std::mutex> lock(attr_mu);
        if (dev >= 0 && dev < 64 && !attr_done[dev]) {
            DD_CUDA_TRY(cudaFuncSetAttribute(attention_persistent_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
            attr_done[dev] = true;
        }
    }
    const long items = (long)p.BH * p.m_blocks;
    const unsigned grid = (unsigned)(items < sms ? items : sms);
    attention_persistent_kernel<D><<<grid, kThreads, smem, s>>>(tq, tk, tv, to, p);
    DD_CUDA_TRY(cudaGetLastError());
    dd::count_launch();
    return DD_OK;
}

int sm_count(int *out)
{
    static int cached[64] = {};
    static std::mutex mu;
    int dev = 0;
    DD_CUDA_TRY(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lock(mu);
    if (dev < 0 || dev >= 64) return DD_ERR_UNSUPPORTED;
    if (cached[dev] == 0) DD_CUDA_TRY(cudaDeviceGetAttribute(&cached[dev], cudaDevAttrMultiProcessorCount, dev));
    *out = cached[dev];
    return DD_OK;
}

int attention_impl(const void *q, const void *k, const void *v, void *out, int B, int H, int Nq, int Nkv, int D,
                   const int32_t *kv_len, int layout, float scale, void *stream)
{
    if (!q || !k || !v || !out) return DD_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || Nq <= 0 || Nkv <= 0 || D <= 0) return DD_ERR_INVALID_ARG;
    if (layout != DD_LAYOUT_BHND && layout != DD_LAYOUT_BNHD) return DD_ERR_INVALID_ARG;
    if (!isfinite(scale)) return DD_ERR_INVALID_ARG;
    if (scale < 0.f) return DD_ERR_UNSUPPORTED;
    if (D != 64 && D != 128) return DD_ERR_UNSUPPORTED;
    if ((((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)out) & 15) != 0) return DD_ERR_UNSUPPORTED;
    const long BH = (long)B * H;
    const int m_blocks = (Nq + kQTiles * kBlockM - 1) / (kQTiles * kBlockM);
    if (BH * m_blocks >= (1L << 31) || BH >= (1L << 31)) return DD_ERR_UNSUPPORTED;

    dd::DeviceCtx *ctx = dd::current_ctx();
    if (!ctx) return DD_ERR_CUDA;
    int rc = dd::ensure_mirror(ctx);
    if (rc != DD_OK) return rc;
    if ((rc = dd::check_mirror(ctx, 0)) != DD_OK) return rc;      // an earlier launch gave up a wait: nothing is launched
    if (!ctx->attn_status) {
        DD_CUDA_TRY(cudaMalloc(&ctx->attn_status, 256));
        DD_CUDA_TRY(cudaMemset(ctx->attn_status, 0, 256));
    }
    const bool head_major = layout == DD_LAYOUT_BHND;
    CUtensorMap tq, tk, tv, to;
    if ((rc = make_tmap(&tq, q, B, H, Nq, D, head_major)) != DD_OK) return rc;
    if ((rc = make_tmap(&tk, k, B, H, Nkv, D, head_major)) != DD_OK) return rc;
    if ((rc = make_tmap(&tv, v, B, H, Nkv, D, head_major)) != DD_OK) return rc;
    if ((rc = make_tmap(&to, out, B, H, Nq, D, head_major)) != DD_OK) return rc;

    AttnParams p;
    p.BH = (int)BH; p.H = H; p.Nq = Nq; p.Nkv = Nkv; p.D = D;
    p.m_blocks = m_blocks;
    p.kv_len = kv_len;
    p.head_major = head_major ? 1 : 0;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.status = ctx->attn_status;
    p.mirror = ctx->mirror_dev;
    cudaStream_t s = (cudaStream_t)stream;
    const bool general = kv_len != nullptr || !head_major || Nq != Nkv;
    if (general) return D == 64 ? launch<64, true>(tq, tk, tv, to, p, s) : launch<128, true>(tq, tk, tv, to, p, s);
    // Many short items (more than one per SM, at most sixteen key tiles each, two query tiles in
    // every item): the persistent kernel overlaps each item's start and end with its neighbours.
    int sms = 0;
    if ((rc = sm_count(&sms)) != DD_OK) return rc;
    const int nkv = (Nkv + kBlockN - 1) / kBlockN;
    if (BH * m_blocks > sms && nkv <= 16 && (Nq - 1) % (kQTiles * kBlockM) >= kBlockM)
        return D == 64 ? launch_persistent<64>(tq, tk, tv, to, p, sms, s) : launch_persistent<128>(tq, tk, tv, to, p, sms, s);
    return D == 64 ? launch<64, false>(tq, tk, tv, to, p, s) : launch<128, false>(tq, tk, tv, to, p, s);
}

}  // namespace

extern "C" int dd_bidir_attention(const void *q, const void *k, const void *v, void *out,
                                  int B, int H, int N, int D, float scale, void *stream)
{
    return attention_impl(q, k, v, out, B, H, N, N, D, nullptr, DD_LAYOUT_BHND, scale, stream);
}

extern "C" int dd_block_attention(const void *q, const void *k, const void *v, void *out,
                                  int B, int H, int Nq, int Nkv, int D,
                                  const int32_t *kv_len, int layout, float scale, void *stream)
{
    return attention_impl(q, k, v, out, B, H, Nq, Nkv, D, kv_len, layout, scale, stream);
}
