// Persistent form of the attention kernel for many short work items (Section 2.2; Eq. 3): the
// square, head-major case of dd_bidir_attention when there are more (head, 256-row block) items
// than SMs and each item has few key tiles.  A CTA of the one-item kernel spends 5-6 us per item
// outside its steady state: Q and the first K tile have to arrive, the first S product and the
// first softmax run with nothing to overlap them, and at the end the tensor core waits for the
// epilogue.  With four key tiles per item (N = 512) that is a third of the item.
//
// Here one CTA per SM walks over items blockIdx.x, blockIdx.x + gridDim.x, ...  The roles and the
// arithmetic are those of attention_kernel (same softmax code, same MMA shapes); what changes:
//   * four Q buffers, two per item parity: the producer loads the next item's Q tiles and first
//     K/V tiles while the current item is still being worked on (ring of three K/V tiles);
//   * barriers, ring positions and tensor memory live across items, every phase is a running
//     count;
//   * the MMA thread issues the next item's first S products right behind the current item's last
//     P V, so that the softmax groups find scores waiting when their epilogue is done; the first
//     P V of an item waits until the group has read the previous accumulator out of tensor memory
//     (o_free);
//   * the output tile is staged in the item's own Q buffer as before; the buffer is handed back
//     to the producer (q_free) once the TMA store has read it, which the storing thread checks
//     after its next key tile, not before.
// Every wait is bounded and reports to the attention health word.  Included by dd_attention.cu
// (inside its unnamed namespace, after the softmax helpers).
#pragma once

constexpr int kPStages = 3;          // K/V ring slots of the persistent kernel

template <int D>
struct SmemP {
    static constexpr int kTileBytes = kBlockN * D * 2;
    static constexpr int kQ = 0;                                    // q[parity][group]: four tiles
    static constexpr int kRing = 4 * kTileBytes;
    static constexpr int kBars = kRing + kPStages * kTileBytes;
    // q_full[4], q_free[4], kv_full[3], kv_empty[3], s_full[2], p_full[2], o_full[2], o_free[2]
    static constexpr int kNumBars = 8 + 2 * kPStages + 8;
    static constexpr int kTmemSlot = kBars + 8 * kNumBars;
    static constexpr int kTotal = kTmemSlot + 16;
    static_assert(kTileBytes % 1024 == 0 && kBars % 8 == 0, "tiles on swizzle boundaries, barriers on 8 bytes");
    static_assert(kTotal + 1024 <= 227 * 1024, "shared memory of one CTA");
};

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
attention_persistent_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                            const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
                            const AttnParams p)
{
    extern __shared__ __align__(1024) unsigned char smem_dyn[];
    const uint32_t smem_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char *smem_gen = smem_dyn + (smem_base - smem_u32(smem_dyn));
    constexpr uint32_t kTileBytes = SmemP<D>::kTileBytes;
    const uint32_t sQ = smem_base + SmemP<D>::kQ, sRing = smem_base + SmemP<D>::kRing;
    const uint32_t bars = smem_base + SmemP<D>::kBars;
    auto bar_q_full = [&](int par, int g) { return bars + 8u * (par * 2 + g); };
    auto bar_q_free = [&](int par, int g) { return bars + 8u * (4 + par * 2 + g); };
    auto bar_kv_full = [&](int s) { return bars + 8u * (8 + s); };
    auto bar_kv_empty = [&](int s) { return bars + 8u * (8 + kPStages + s); };
    auto bar_s_full = [&](int g) { return bars + 8u * (8 + 2 * kPStages + g); };
    auto bar_p_full = [&](int g) { return bars + 8u * (10 + 2 * kPStages + g); };
    auto bar_o_full = [&](int g) { return bars + 8u * (12 + 2 * kPStages + g); };
    auto bar_o_free = [&](int g) { return bars + 8u * (14 + 2 * kPStages + g); };
    const uint32_t tmem_slot = smem_base + SmemP<D>::kTmemSlot;
    volatile uint32_t *tmem_slot_gen = reinterpret_cast<volatile uint32_t *>(smem_gen + SmemP<D>::kTmemSlot);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_items = p.BH * p.m_blocks;
    const int nkv = (p.Nkv + kBlockN - 1) / kBlockN;            // key tiles per item (>= 1)
    constexpr int kBoxes = D / 64;
    constexpr uint32_t kBoxBytes = 128 * 128;
    constexpr uint32_t kColS = 0, kColO = 256;
    auto q_buf = [&](int par, int g) { return sQ + (uint32_t)(par * 2 + g) * kTileBytes; };

    if (tid == 0) {
        prefetch_tmap(&tm_q); prefetch_tmap(&tm_k); prefetch_tmap(&tm_v); prefetch_tmap(&tm_o);
        for (int i = 0; i < 4; ++i) { mbar_init(bars + 8u * i, 1); mbar_init(bars + 8u * (4 + i), 1); }
        for (int s = 0; s < kPStages; ++s) { mbar_init(bar_kv_full(s), 1); mbar_init(bar_kv_empty(s), 1); }
        for (int g = 0; g < kQTiles; ++g) {
            mbar_init(bar_s_full(g), 1);
            mbar_init(bar_p_full(g), kBlockM);
            mbar_init(bar_o_full(g), 1);
            mbar_init(bar_o_free(g), kBlockM);
        }
        fence_mbar_init();
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
        const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + lane_off + kColS + g * kBlockN;
        const uint32_t tO = tmem + lane_off + kColO + g * D;
        const float c = p.scale_log2;
        const bool storer = (warp & 3) == 0 && lane == 0;
        unsigned err = 0;
        uint32_t t_run = 0;              // key tiles of this group so far, over all items: phase of s/p/o_full
        int pending_free = -1;           // parity of the Q buffer whose store this thread has committed
        int n = 0;
        for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++n) {
            const int par = n & 1;
            const int bh = item / p.m_blocks, mb = item - bh * p.m_blocks;
            const int row0 = mb * (kQTiles * kBlockM);
            float m_ref = -INFINITY, l_run = 0.f;
            for (int j = 0; j < nkv; ++j, ++t_run) {
                if (!mbar_wait(bar_s_full(g), t_run & 1)) { err = kErrWaitS; break; }
                tc_fence_after();
                // O_g holds the sum over this item's tiles < j once the previous P V has completed
                err = softmax_tile<D>(tS, tO, bar_o_full(g), (t_run - 1) & 1, j == 0, p.Nkv - j * kBlockN, c, m_ref, l_run);
                if (err) break;
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(bar_p_full(g));
                if (storer && pending_free >= 0) {
                    // the previous item's store has long read its staging buffer: hand it back
                    tma_store_wait_read();
                    mbar_arrive(bar_q_free(pending_free, g));
                    pending_free = -1;
                }
            }
            if (err == 0 && !mbar_wait(bar_o_full(g), (t_run - 1) & 1)) err = kErrWaitO;
            if (err != 0) report(p, err);
            if (err == 0) {
                // ---- epilogue: O / l -> bf16 -> this item's Q buffer (every MMA that read it has
                // completed) in the swizzled layout of the tensor map -> global by TMA
                tc_fence_after();
                const int r = (warp & 3) * 32 + lane;
                const float inv = 1.f / l_run;
                const uint32_t stage = q_buf(par, g) + r * 128;
                // the whole accumulator row in one go; once it is in registers the next item's first
                // P V may overwrite the accumulator
                uint32_t acc[D];
#pragma unroll
                for (int cb = 0; cb < D / 32; ++cb)
                    tmem_ld32(tO + cb * 32, *reinterpret_cast<uint32_t(*)[32]>(&acc[cb * 32]));
                tmem_wait_ld();
                tc_fence_before();
                mbar_arrive(bar_o_free(g));
#pragma unroll
                for (int cb = 0; cb < D / 32; ++cb) columns_to_staging(&acc[cb * 32], inv, stage, r, cb);
                fence_proxy_async_smem();
            }
            // every thread of the warpgroup comes here, also after an expired wait
            named_bar_sync(1 + g, kBlockM);
            if (err != 0) break;
            if (storer) {
#pragma unroll
                for (int cx = 0; cx < kBoxes; ++cx)
                    tma_store_3d(&tm_o, q_buf(par, g) + cx * kBoxBytes, cx * 64, row0 + g * kBlockM, bh);
                tma_store_commit();
                pending_free = par;
            }
        }
        if (storer) tma_store_wait_read();          // shared memory must outlive the last store's reads
    } else {
        reg_dec<72>();
        if (warp == kLoadWarp && lane == 0) {
            // =============================================================== TMA producer
            uint32_t ring = 0;           // ring items so far, over all items
            int n = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++n) {
                const int par = n & 1;
                const int bh = item / p.m_blocks, mb = item - bh * p.m_blocks;
                const int row0 = mb * (kQTiles * kBlockM);
                auto load_q = [&](int g) -> bool {
                    // the buffer staged the output of item n - 2
                    if (n >= 2 && !mbar_wait(bar_q_free(par, g), ((n >> 1) - 1) & 1)) return false;
                    mbar_expect_tx(bar_q_full(par, g), kTileBytes);
#pragma unroll
                    for (int cx = 0; cx < kBoxes; ++cx)
                        tma_load_3d(q_buf(par, g) + cx * kBoxBytes, &tm_q, bar_q_full(par, g), cx * 64, row0 + g * kBlockM, bh);
                    return true;
                };
                if (!load_q(0)) { report(p, kErrWaitSlot); break; }
                for (int it = 0; it < 2 * nkv; ++it, ++ring) {
                    if (it == 1 && !load_q(1)) { report(p, kErrWaitSlot); ok = false; break; }
                    const int slot = ring % kPStages;
                    const uint32_t use = ring / kPStages;
                    if (use > 0 && !mbar_wait(bar_kv_empty(slot), (use - 1) & 1)) { report(p, kErrWaitSlot); ok = false; break; }
                    const uint32_t dst = sRing + slot * kTileBytes;
                    const CUtensorMap *tm = (it & 1) ? &tm_v : &tm_k;
                    mbar_expect_tx(bar_kv_full(slot), kTileBytes);
#pragma unroll
                    for (int cx = 0; cx < kBoxes; ++cx)
                        tma_load_3d(dst + cx * kBoxBytes, tm, bar_kv_full(slot), cx * 64, (it >> 1) * kBlockN, bh);
                }
            }
        } else if (warp == kMmaWarp && lane == 0) {
            // =============================================================== MMA issuer
            constexpr uint32_t kIdescS = idesc_bf16(kBlockM, kBlockN, false);
            constexpr uint32_t kIdescO = idesc_bf16(kBlockM, D, true);
            const uint64_t desc_q0 = smem_desc_sw128(sQ, 16, 1024);
            const uint64_t desc_k0 = smem_desc_sw128(sRing, 16, 1024);
            const uint64_t desc_v0 = smem_desc_sw128(sRing, kBoxBytes, 1024);
            unsigned err = 0;
            auto issue_s = [&](int par, int g, int slot) {
                const uint64_t a = desc_q0 + (uint64_t)((par * 2 + g) * (kTileBytes >> 4));
                const uint64_t b = desc_k0 + (uint64_t)(slot * (kTileBytes >> 4));
                const uint32_t tS = tmem + kColS + g * kBlockN;
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t off = ((ks / 4) * kBoxBytes + (ks % 4) * 32) >> 4;
                    mma_ss(tS, a + off, b + off, kIdescS, ks > 0);
                }
                mma_commit(bar_s_full(g));
            };
            auto issue_o = [&](int g, int slot, bool first) {
                const uint64_t b = desc_v0 + (uint64_t)(slot * (kTileBytes >> 4));
                const uint32_t tS = tmem + kColS + g * kBlockN, tO = tmem + kColO + g * D;
#pragma unroll
                for (int ks = 0; ks < kBlockN / 16; ++ks)
                    mma_ts(tO, tS + ks * 8, b + (uint32_t)(ks * (2048 >> 4)), kIdescO, (!first || ks > 0));
                mma_commit(bar_o_full(g));
            };
            uint32_t ring = 0;           // ring items consumed so far, over all items
            uint32_t t_run = 0;          // key tiles so far (the same for both groups)
            auto wait_ring = [&](uint32_t r) { return mbar_wait(bar_kv_full(r % kPStages), (r / kPStages) & 1); };
            int n = 0;
            for (int item = blockIdx.x; item < n_items && err == 0; item += gridDim.x, ++n) {
                const int par = n & 1;
                const uint32_t q_phase = (uint32_t)(n >> 1) & 1;
                // ring items of this work item: ring + 2j = K tile j, ring + 2j + 1 = V tile j
                if (!mbar_wait(bar_q_full(par, 0), q_phase)) { err = kErrWaitQ; break; }
                if (!wait_ring(ring)) { err = kErrWaitKV; break; }
                tc_fence_after();
                issue_s(par, 0, ring % kPStages);
                if (!mbar_wait(bar_q_full(par, 1), q_phase)) { err = kErrWaitQ; break; }
                tc_fence_after();
                issue_s(par, 1, ring % kPStages);
                mma_commit(bar_kv_empty(ring % kPStages));
                for (int j = 0; j < nkv && err == 0; ++j, ++t_run) {
                    const uint32_t r_v = ring + 2 * j + 1, r_k = ring + 2 * j + 2;
                    const bool more = j + 1 < nkv;
                    if (!wait_ring(r_v)) { err = kErrWaitKV; break; }
                    if (more && !wait_ring(r_k)) { err = kErrWaitKV; break; }
                    for (int g = 0; g < kQTiles; ++g) {
                        if (!mbar_wait(bar_p_full(g), t_run & 1)) { err = kErrWaitP; break; }
                        // the first product of an item overwrites the accumulator: the group must
                        // have read the previous item's result out of it
                        if (j == 0 && n > 0 && !mbar_wait(bar_o_free(g), (uint32_t)(n - 1) & 1)) { err = kErrWaitO; break; }
                        tc_fence_after();
                        issue_o(g, r_v % kPStages, j == 0);
                        if (more) issue_s(par, g, r_k % kPStages);
                    }
                    if (err) break;
                    mma_commit(bar_kv_empty(r_v % kPStages));
                    if (more) mma_commit(bar_kv_empty(r_k % kPStages));
                }
                ring += 2 * (uint32_t)nkv;
            }
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
