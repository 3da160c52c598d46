// Language-model heads fused with the verification algorithm (Algorithm 1, verification phase:
// the verifier's distribution p_V(. | x^D) at every position goes straight into A(p_D, p_V, x^D)).
//
// logits[t, x] = sum_k hidden[t, k] * weight[x, k] is a [rows, K] x [K, V] product whose result,
// 253 KB per position at the LLaDA vocabulary, is only ever reduced: per row its maximum, the
// lowest index of the maximum and the softmax normaliser (Eq. 7), and in the KL mode the sums of
// Eq. 4-5 over the drafter's logits, which are a second product of the same shape.  The kernel
// therefore keeps the products in tensor memory and never stores a logit: a persistent CTA takes
// work items of 256 rows x N vocabulary entries, accumulates them with tcgen05 MMAs (accumulators
// of 128 rows, fp32) from operand tiles that a TMA producer streams through a three-stage ring,
// and its epilogue warps turn every accumulator row into one partial (maximum, first index,
// sum 2^(l*log2e - M); KL: also the drafter's maximum, sum and the weighted logit differences) of
// the same form as the streaming kernel's chunk partials, stored in the same global table ("chunk"
// = vocabulary tile).  A second, small kernel behind it on the stream (lm_head_fold_kernel) folds
// every flagged row's partials in fp64 with the streaming kernel's fold and runs dd_verify's
// decision stage per sequence.
//
// Tensor memory (512 columns): TRUST/CONF, N <= 256: the verifier's two accumulators at columns 0
// and 256.  KL, N <= 128: the drafter's at 0 and 128, the verifier's at 256 and 384; a work item
// runs the k loop over the drafter's operands first, then over the verifier's.
//
//   warps 0-3   epilogue of rows 0-127 of the item (thread = row = tensor-memory lane)
//   warps 4-7   epilogue of rows 128-255
//   warp  8     one thread feeds the ring: per 64-wide k-step the two 128-row tiles of the hidden
//               states and the N-row tile of the weights (2-D tensor maps, 128-byte swizzle, rows
//               past the end read as zero; no multicast)
//   warp  9     one thread issues the MMAs and commits them to the ring's and the accumulators'
//               barriers
// Included by dd_verify.cu.
#pragma once

#include <cuda.h>

#include "dd_ptx.cuh"
#include "dd_verify_common.cuh"

namespace ddlm {

using namespace ddptx;

constexpr int kThreads = 320;
constexpr int kEpilogueWarps = 8;
constexpr int kLoadWarp = 8, kMmaWarp = 9;
constexpr int kRowsPerItem = 256;          // two accumulators of 128 rows
constexpr int kBlockK = 64;                // one 128-byte swizzled box per k-step
constexpr int kStages = 3;
constexpr int kMaxN = 256;
constexpr uint32_t kTmemCols = 512;        // see the layout above
constexpr int kATileBytes = 128 * kBlockK * 2;                        // 16 KB: 128 rows x 64 bf16
constexpr int kStageBytes = 2 * kATileBytes + kMaxN * kBlockK * 2;    // 64 KB
constexpr int kSmemBytes = kStages * kStageBytes + 1024 + 256;
constexpr unsigned kErrLmFull = 0xC00, kErrLmEmpty = 0xD00, kErrLmAcc = 0xE00;

struct LmParams {
    int rows, K, V;            // rows = B * P
    int N;                     // vocabulary entries per work item (a multiple of 32, <= 256; KL: <= 128)
    int n_tiles;               // ceil(V / N): the "chunks" of a row
    int row_blocks;            // ceil(rows / 256)
};

// One row's partial of one vocabulary tile into the global table.  Nothing else happens in this
// kernel: rows are folded and sequences decided by lm_head_fold_kernel, launched behind it on the
// same stream.  (Folding in here, by whichever warp stores a row's last tile, put every fold of the
// launch on the one CTA that finishes last: all rows of a row block complete together, with the
// last tile.  170 of 217 us on a 256-row, 143-tile problem were that CTA folding alone.)
__device__ __forceinline__ void store_partial(const ddv::VerifyParams &p, const ddv::Partial &c, int row, int tile)
{
    ddv::Partial *dst = p.partials + ddv::checked(p, (long)row * p.nchunks + tile, (long)p.B * p.P * p.nchunks, ddv::kSitePartial);
    __stcg(reinterpret_cast<float4 *>(dst), make_float4(c.m_v, c.s_v, __int_as_float(c.idx), c.m_d));
    __stcg(reinterpret_cast<float4 *>(dst) + 1, make_float4(c.s_d, c.t, 0.f, 0.f));
}

// n more rows of sequence b are accounted for (warp-level); the warp that accounts for the last
// of the P rows decides the sequence.
__device__ __forceinline__ void rows_done(const ddv::VerifyParams &p, int b, int n, ddv::DecideStage *stage)
{
    const int lane = threadIdx.x & 31;
    int last = 0;
    if (lane == 0) {
        __threadfence();
        last = atomicAdd(p.seq_counter + ddv::checked(p, b, p.B, ddv::kSiteSeq), (unsigned)n) + (unsigned)n == (unsigned)p.P;
    }
    last = __shfl_sync(0xFFFFFFFFu, last, 0);
    if (!last) return;
    __threadfence();
    if (lane == 0) p.seq_counter[b] = 0u;      // ready for the next launch
    ddv::decide_sequence(p, b, stage);
}

// Second launch of dd_lm_head_verify: one warp per row folds the row's tile partials (fp64, tile
// order: the streaming kernel's fold) and stores score and argmax; one warp per sequence accounts
// for the rows that are not flagged; the warp that accounts for a sequence's last row runs the
// decision stage.  The partials were written by the previous kernel on the stream.
constexpr int kFoldThreads = 128;
constexpr int kFoldDecideKeys = 2048;      // keys of one sequence each warp can keep in shared memory
template <bool KL>
__global__ void __launch_bounds__(kFoldThreads) lm_head_fold_kernel(const ddv::VerifyParams p, int rows)
{
    __shared__ uint32_t s_keys[kFoldThreads / 32][kFoldDecideKeys];
    ddv::DecideStage stage;
    stage.key = s_keys[threadIdx.x >> 5];
    stage.capacity = kFoldDecideKeys;
    const int w = blockIdx.x * (kFoldThreads / 32) + (threadIdx.x >> 5);     // rows first, then sequences
    if (w < rows) {
        if (!p.flags[w]) return;
        float score;
        int argmax;
        ddv::fold_partials<KL>(p.partials + ddv::checked_run(p, (long)w * p.nchunks, p.nchunks, (long)rows * p.nchunks, ddv::kSitePartial),
                               p.nchunks, score, argmax);
        if ((threadIdx.x & 31) == 0) {
            const size_t row_at = ddv::checked(p, w, (long)p.B * p.P, ddv::kSiteRow);
            __stcg(p.row_score + row_at, score);
            __stcg(p.row_argmax + row_at, argmax);
        }
        __syncwarp();
        rows_done(p, w / p.P, 1, &stage);
    } else {
        const int b = w - rows;
        if (b >= p.B) return;
        const int unflagged = p.P - ddv::count_flagged(p, b);
        if (unflagged > 0) rows_done(p, b, unflagged, &stage);
    }
}

// Epilogue warps: every accumulator row becomes one partial.  Columns are visited in index order
// with a strict comparison, so the index kept is the lowest index of the maximum.  KL (Eq. 4-5):
// the drafter's accumulator is read beside the verifier's, and the row also keeps the drafter's
// running maximum m_d, s_d = sum 2^(d*log2e - M_d) and t = sum 2^(d*log2e - M_d) * (d - v), both
// rescaled whenever the maximum moves.
template <bool KL>
__device__ __forceinline__ void epilogue(const LmParams &q, const ddv::VerifyParams &p, uint32_t tmem,
                                         uint32_t bar_acc_full, uint32_t bar_acc_empty,
                                         volatile uint32_t *abort_flag, int n_items)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int acc = warp >> 2;
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;          // this warp's 32 tensor-memory lanes
    const uint32_t tacc = tmem + lane_off + (KL ? 256u + (uint32_t)acc * 128u : (uint32_t)acc * 256u);   // verifier
    const uint32_t dacc = tmem + lane_off + (uint32_t)acc * 128u;                                          // drafter (KL)
    uint32_t n_done = 0;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++n_done) {
        const int tile = item / q.row_blocks, rb = item - tile * q.row_blocks;
        const int row = rb * kRowsPerItem + acc * 128 + (warp & 3) * 32 + lane, col0 = tile * q.N;
        bool arrived = false;
        for (uint32_t it = 0; it < (1u << 22); ++it) {
            if (mbar_try_wait(bar_acc_full, n_done & 1)) { arrived = true; break; }
            if (it > 64) {
                __nanosleep(64);
                if (*abort_flag) break;
            }
        }
        if (!arrived) {
            if (lane == 0) {
                *abort_flag = 1u;
                ddv::report_expired(p, kErrLmAcc);
            }
            return;
        }
        tc_fence_after();
        float m = -INFINITY, M = -INFINITY, s = 0.f;
        float m_d = -INFINITY, M_d = -INFINITY, s_d = 0.f, t = 0.f;
        int idx = 0x7FFFFFFF;
        for (int cb = 0; cb < q.N / 32; ++cb) {
            uint32_t r[32], rd[32];              // rd: the drafter's logits, KL only
            tmem_ld32(tacc + cb * 32, r);
            if constexpr (KL) tmem_ld32(dacc + cb * 32, rd);
            tmem_wait_ld();
            const int valid = q.V - (col0 + cb * 32);                 // columns of this group that exist
            if (valid <= 0) break;
            float cm = -INFINITY;
            int ci = 0;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const float v = __uint_as_float(r[i]);
                if (i < valid && v > cm) { cm = v; ci = i; }
            }
            if (cm > m) {
                const float M_new = cm * ddv::kLog2e;
                s *= ddv::rescale_factor(M, M_new);
                m = cm; M = M_new;
                idx = col0 + cb * 32 + ci;
            }
#pragma unroll
            for (int i = 0; i < 32; ++i)
                if (i < valid) s += ddv::ex2_approx(fmaf(__uint_as_float(r[i]), ddv::kLog2e, -M));
            if constexpr (KL) {
                float cd = -INFINITY;
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    if (i < valid) cd = fmaxf(cd, __uint_as_float(rd[i]));
                if (cd > m_d) {
                    const float M_new = cd * ddv::kLog2e;
                    const float f = ddv::rescale_factor(M_d, M_new);
                    s_d *= f; t *= f;
                    m_d = cd; M_d = M_new;
                }
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    if (i < valid) {
                        const float d = __uint_as_float(rd[i]);
                        const float e = ddv::ex2_approx(fmaf(d, ddv::kLog2e, -M_d));
                        s_d += e;
                        t = fmaf(e, d - __uint_as_float(r[i]), t);
                    }
            }
        }
        // both accumulators may be overwritten once every epilogue warp has read its lanes
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_acc_empty);

        ddv::Partial c;
        c.m_v = m; c.s_v = s; c.idx = idx;
        c.m_d = KL ? m_d : 0.f; c.s_d = s_d; c.t = t; c.pad0 = c.pad1 = 0.f;
        if (row < q.rows && p.flags[row]) store_partial(p, c, row, tile);
    }
}

// KL: every work item runs the k loop twice, first over the drafter's hidden states and weights
// into accumulators [0,N) and [128,128+N), then over the verifier's into [256,..) and [384,..)
// (N <= 128); the epilogue reads both.  Otherwise only the verifier's maps are used and the
// accumulators are [0,N) and [256,256+N) (N <= 256).
template <bool KL>
__global__ void __launch_bounds__(kThreads, 1)
lm_head_kernel(const __grid_constant__ CUtensorMap tm_h, const __grid_constant__ CUtensorMap tm_w,
               const __grid_constant__ CUtensorMap tm_hd, const __grid_constant__ CUtensorMap tm_wd,
               const LmParams q, const ddv::VerifyParams p)
{
    extern __shared__ __align__(1024) unsigned char smem_dyn[];
    const uint32_t smem_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;     // swizzled tiles: 1024-byte aligned
    unsigned char *smem_gen = smem_dyn + (smem_base - smem_u32(smem_dyn));
    const uint32_t bars = smem_base + kStages * kStageBytes;
    auto bar_full = [&](int s) { return bars + 8u * s; };
    auto bar_empty = [&](int s) { return bars + 8u * (kStages + s); };
    const uint32_t bar_acc_full = bars + 8u * (2 * kStages), bar_acc_empty = bars + 8u * (2 * kStages + 1);
    const uint32_t tmem_slot = bars + 8u * (2 * kStages + 2);
    volatile uint32_t *tmem_slot_gen = reinterpret_cast<volatile uint32_t *>(smem_gen + kStages * kStageBytes + 8 * (2 * kStages + 2));
    volatile uint32_t *abort_flag = tmem_slot_gen + 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_items = q.n_tiles * q.row_blocks;
    const int k_steps = q.K / kBlockK;

    if (tid == 0) {
        prefetch_tmap(&tm_h); prefetch_tmap(&tm_w);
        if (KL) { prefetch_tmap(&tm_hd); prefetch_tmap(&tm_wd); }
        for (int s = 0; s < kStages; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_empty(s), 1); }
        mbar_init(bar_acc_full, 1);
        mbar_init(bar_acc_empty, kEpilogueWarps);
        fence_mbar_init();
        *abort_flag = 0u;
    }
    if (warp == 0) { tmem_alloc(tmem_slot, kTmemCols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot_gen;

    // a wait that gives up: the code goes to the health word, every role winds down
    auto give_up = [&](unsigned code) {
        *abort_flag = 1u;
        ddv::report_expired(p, code);
    };
    auto wait = [&](uint32_t bar, uint32_t parity) {
        for (uint32_t it = 0; it < (1u << 22); ++it) {
            if (mbar_try_wait(bar, parity)) return true;
            if (it > 64) {
                __nanosleep(32);
                if (*abort_flag) return false;
            }
        }
        return false;
    };

    if (warp == kLoadWarp && lane == 0) {
        // ===================================================================== TMA producer
        uint32_t step = 0;                                    // k-steps issued over all items
        for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
            const int tile = item / q.row_blocks, rb = item - tile * q.row_blocks;
            const int row0 = rb * kRowsPerItem, col0 = tile * q.N;
            bool ok = true;
            for (int ks2 = 0; ks2 < (KL ? 2 : 1) * k_steps; ++ks2, ++step) {
                const int s = step % kStages;
                const uint32_t use = step / kStages;
                if (use > 0 && !wait(bar_empty(s), (use - 1) & 1)) { give_up(kErrLmEmpty); ok = false; break; }
                const uint32_t dst = smem_base + s * kStageBytes;
                const bool drafter = KL && ks2 < k_steps;                 // the drafter's pass comes first
                const int ks = ks2 < k_steps ? ks2 : ks2 - k_steps;
                const CUtensorMap *mh = drafter ? &tm_hd : &tm_h, *mw = drafter ? &tm_wd : &tm_w;
                mbar_expect_tx(bar_full(s), (uint32_t)(2 * kATileBytes + q.N * kBlockK * 2));
                tma_load_2d(dst, mh, bar_full(s), ks * kBlockK, row0);
                tma_load_2d(dst + kATileBytes, mh, bar_full(s), ks * kBlockK, row0 + 128);
                tma_load_2d(dst + 2 * kATileBytes, mw, bar_full(s), ks * kBlockK, col0);
            }
            if (!ok) break;
        }
    } else if (warp == kMmaWarp && lane == 0) {
        // ===================================================================== MMA issuer
        const uint32_t idesc = idesc_bf16(128, q.N, false);
        uint32_t step = 0, n_done = 0;                        // k-steps consumed, items finished
        for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++n_done) {
            // the epilogue of the previous item has read both accumulators
            if (n_done > 0 && !wait(bar_acc_empty, (n_done - 1) & 1)) { give_up(kErrLmAcc); break; }
            tc_fence_after();
            bool ok = true;
            for (int ks2 = 0; ks2 < (KL ? 2 : 1) * k_steps; ++ks2, ++step) {
                const int s = step % kStages;
                if (!wait(bar_full(s), (step / kStages) & 1)) { give_up(kErrLmFull); ok = false; break; }
                tc_fence_after();
                const int ks = ks2 < k_steps ? ks2 : ks2 - k_steps;
                // accumulator columns of this pass: see the layout above
                const uint32_t acc0 = tmem + ((KL && ks2 >= k_steps) ? 256u : 0u), acc1 = acc0 + (KL ? 128u : 256u);
                const uint32_t base = smem_base + s * kStageBytes;
                const uint64_t a0 = smem_desc_sw128(base, 16, 1024), a1 = smem_desc_sw128(base + kATileBytes, 16, 1024);
                const uint64_t b = smem_desc_sw128(base + 2 * kATileBytes, 16, 1024);
#pragma unroll
                for (int kk = 0; kk < kBlockK / 16; ++kk) {
                    const uint32_t off = (uint32_t)(kk * 32) >> 4;            // 16 bf16 = 32 bytes per MMA
                    mma_ss(acc0, a0 + off, b + off, idesc, (ks > 0 || kk > 0));
                    mma_ss(acc1, a1 + off, b + off, idesc, (ks > 0 || kk > 0));
                }
                mma_commit(bar_empty(s));                                      // the stage is free once these have run
            }
            if (!ok) break;
            mma_commit(bar_acc_full);
        }
    } else if (warp < kEpilogueWarps) {
        epilogue<KL>(q, p, tmem, bar_acc_full, bar_acc_empty, abort_flag, n_items);
    }

    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        // a wait expired: give copies that may still be in flight time to land before the shared
        // memory is released
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    }
    if (warp == 0) { __syncwarp(); tmem_dealloc(tmem, kTmemCols); }
}

}  // namespace ddlm
