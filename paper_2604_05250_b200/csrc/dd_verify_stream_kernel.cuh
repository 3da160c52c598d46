// The streaming kernel itself.  Included by dd_verify_stream.cuh.
#pragma once

namespace ddv {

// Number of flagged rows of sequence b (warp-level; every lane gets the result).
__device__ __forceinline__ int count_flagged(const VerifyParams &p, int b)
{
    const int lane = threadIdx.x & 31;
    const uint8_t *f = p.flags + (size_t)b * p.P;
    int n = 0;
    for (int i = lane; i < p.P; i += 32) n += f[i] != 0;
    return __reduce_add_sync(0xFFFFFFFFu, n);
}

// The publishing warp's view of the sequence whose rows it is counting.
struct SeqTally {
    int b;          // sequence, -1: none yet
    int target;     // its number of flagged rows
};

// cnt more rows of sequence b are complete (their scores are stored); the warp that completes
// the sequence decides it.  The caller has fenced its stores.
__device__ __forceinline__ void rows_done(const VerifyParams &p, SeqTally &tally, int b, int cnt, DecideStage *stage)
{
    const int lane = threadIdx.x & 31;
    if (tally.b != b) {
        tally.b = b;
        tally.target = count_flagged(p, b);
    }
    int last = 0;
    if (lane == 0) last = atomicAdd(p.seq_counter + b, (unsigned)cnt) + (unsigned)cnt == (unsigned)tally.target;
    last = __shfl_sync(0xFFFFFFFFu, last, 0);
    if (!last) return;
    __threadfence();
    if (lane == 0) p.seq_counter[b] = 0u;      // ready for the next launch
    decide_sequence(p, b, stage);
}

template <bool KL>
__global__ void __launch_bounds__(kSThreads, 1) verify_stream_kernel(const VerifyParams p)
{
    extern __shared__ __align__(128) unsigned char ring_raw[];
    __shared__ __align__(8) unsigned long long s_bar[kSStreamWarps][kSStages];
    __shared__ __align__(16) PieceDesc s_desc[kSStreamWarps][kSStages];
    __shared__ __align__(16) Partial s_table[kSTable];          // chunk partials of the current range
    __shared__ int s_rows[kSTable + 2];                          // flagged rows the range touches
    __shared__ unsigned int s_rowcnt[kSTable + 2];               // their chunks stored so far
    __shared__ __align__(16) EventQueue s_queue;
    __shared__ unsigned int s_next;
    __shared__ int s_scan[kSWarps];
    __shared__ DecideStage s_decide;                              // decision stage (publishing warp only)

    constexpr int kTensorBytes = kPiece * 2;                      // one piece of one tensor
    constexpr int kStageBytes = (KL ? 2 : 1) * kTensorBytes;
    const unsigned full = 0xFFFFFFFFu;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nch = p.nchunks;

    if (warp < kSStreamWarps && lane == 0) {
        for (int s = 0; s < kSStages; ++s) mbar_init(smem_u32(&s_bar[warp][s]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }

    // ---- every thread counts the flagged rows of its contiguous slice of the B*P rows; the block
    // scan gives each thread the number of flagged rows before its slice, and the total
    const long n_rows = (long)p.B * p.P;
    const long slice = (n_rows + kSThreads - 1) / kSThreads;
    const long my_begin = min(n_rows, (long)tid * slice), my_end = min(n_rows, my_begin + slice);
    int my_count = 0;
    for (long r = my_begin; r < my_end; ++r) my_count += p.flags[r] != 0;
    long my_prefix, total_flagged;
    {
        int incl = my_count;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(full, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) s_scan[warp] = incl;
        __syncthreads();
        int before = 0, all = 0;
        for (int w = 0; w < kSWarps; ++w) {
            const int v = s_scan[w];
            if (w < warp) before += v;
            all += v;
        }
        my_prefix = (long)before + incl - my_count;
        total_flagged = all;
    }
    const long total_units = total_flagged * nch;
    // equal ranges, each small enough for the table, their number a multiple of the CTAs
    const long per_cta = (total_units + gridDim.x - 1) / gridDim.x;
    const long rounds = per_cta > kSTable ? (per_cta + kSTable - 1) / kSTable : 1;
    const long n_ranges = rounds * gridDim.x;

    SeqTally tally;
    tally.b = -1;
    tally.target = 0;
    __shared__ float s_rehearsal[2];
    if (warp == kSStreamWarps) {
        // sequences without a single flagged row pass through; this CTA's share of them
        for (int b = blockIdx.x; b < p.B; b += gridDim.x)
            if (count_flagged(p, b) == 0) decide_sequence(p, b, &s_decide);
    }

    bool rehearsed = false;
    unsigned ring_uses = 0;       // streaming warps: pieces taken from the ring so far
    bool wait_ok = true, queue_ok = true;

    for (long range = blockIdx.x; range < n_ranges; range += gridDim.x) {
        const long lo = total_units * range / n_ranges, hi = total_units * (range + 1) / n_ranges;
        if (hi <= lo) continue;                                   // uniform over the CTA
        const int n_units = (int)(hi - lo);
        const long f_lo = lo / nch, f_hi = (hi - 1) / nch;        // flagged-row ordinals the range touches

        __syncthreads();                                          // the previous range is fully drained
        {
            long ord = my_prefix;
            for (long r = my_begin; r < my_end && ord <= f_hi; ++r) {
                if (p.flags[r]) {
                    if (ord >= f_lo) s_rows[ord - f_lo] = (int)r;
                    ++ord;
                }
            }
            for (int i = tid; i < (int)(f_hi - f_lo + 1); i += kSThreads) s_rowcnt[i] = 0u;
            if (tid < kSQueue) s_queue.ready[tid] = 0u;
            if (tid == 0) {
                s_next = 0u;
                s_queue.tail = s_queue.head = s_queue.done = 0u;
            }
        }
        __syncthreads();

        if (warp == kSStreamWarps) {
            // =============================================================== publishing warp
            if (!rehearsed) {
                // nothing is finished yet: bring the code of the row fold and of the decision stage
                // into the instruction caches now, not at the end of the launch
                rehearsed = true;
                float sc;
                int am;
                Partial *fake = reinterpret_cast<Partial *>(s_decide.key);      // free until a sequence ends
                {
                    Partial f;
                    f.m_v = 1.f + lane; f.s_v = 1.5f; f.idx = lane; f.m_d = 0.5f * lane; f.s_d = 1.25f; f.t = 0.125f;
                    f.pad0 = f.pad1 = 0.f;
                    fake[lane] = f;
                }
                __syncwarp();
                fold_partials<KL>(fake, 32, sc, am);
                if (lane == 0) { s_rehearsal[0] = sc; s_rehearsal[1] = __int_as_float(am); }
                decide_sequence_rehearsal(p, &s_decide);
            }
            unsigned int head = 0;
            for (unsigned idle = 0;;) {
                const unsigned int mine = head + lane;
                const bool ready = *(volatile unsigned int *)&s_queue.ready[mine % kSQueue] == mine + 1u;
                const unsigned mask = __ballot_sync(full, ready);
                const int n = mask == full ? 32 : __ffs(~mask) - 1;      // contiguous ready entries
                if (n == 0) {
                    const unsigned int done = *(volatile unsigned int *)&s_queue.done;
                    const unsigned int tail = *(volatile unsigned int *)&s_queue.tail;
                    if (done == (unsigned)kSStreamWarps && tail == head) break;
                    if (++idle > (1u << 24)) {     // the streaming warps never finished
                        if (lane == 0 && p.status) atomicCAS(p.status, 0u, kErrWaitQueue | (blockIdx.x & 0xFF));
                        break;
                    }
                    __nanosleep(100);
                    continue;
                }
                idle = 0;
                __threadfence_block();
                RowEvent e = s_queue.entry[(lane < n ? mine : head) % kSQueue];
                __syncwarp();
                head += n;
                if (lane == 0) *(volatile unsigned int *)&s_queue.head = head;
                const bool mine_ok = lane < n;

                // rows cut by a range boundary: this range's chunk partials go to global memory
                unsigned parts = __ballot_sync(full, mine_ok && !e.whole);
                for (unsigned m = parts; m; m &= m - 1) {
                    const int src = __ffs(m) - 1;
                    const int row = __shfl_sync(full, e.row, src), slot0 = __shfl_sync(full, e.first_slot, src);
                    const int chunk0 = __shfl_sync(full, e.first_chunk, src), cnt = __shfl_sync(full, e.count, src);
                    Partial *dst = p.partials + (size_t)row * nch + chunk0;
                    for (int i = lane; i < 2 * cnt; i += 32)
                        __stcg(reinterpret_cast<float4 *>(dst) + i, reinterpret_cast<const float4 *>(s_table + slot0)[i]);
                }
                if (parts) {
                    __threadfence();
                    bool complete = false;
                    if (mine_ok && !e.whole)
                        complete = atomicAdd(p.row_counter + e.row, (unsigned)e.count) + (unsigned)e.count == (unsigned)nch;
                    unsigned fold = __ballot_sync(full, complete);
                    if (fold) __threadfence();
                    for (unsigned m = fold; m; m &= m - 1) {
                        const int src = __ffs(m) - 1;
                        const int row = __shfl_sync(full, e.row, src);
                        float score;
                        int argmax;
                        fold_partials<KL>(p.partials + (size_t)row * nch, nch, score, argmax);
                        if (lane == src) {
                            e.whole = 1;
                            e.score = score;
                            e.argmax = argmax;
                            p.row_counter[row] = 0u;      // ready for the next launch
                        }
                    }
                }
                // finished rows: store, fence once, count them per sequence
                const bool finished = mine_ok && e.whole;
                if (finished) {
                    __stcg(p.row_score + e.row, e.score);
                    __stcg(p.row_argmax + e.row, e.argmax);
                }
                unsigned fin = __ballot_sync(full, finished);
                if (fin) __threadfence();
                while (fin) {
                    const int src = __ffs(fin) - 1;
                    const int b = __shfl_sync(full, e.row, src) / p.P;
                    const unsigned same = __ballot_sync(full, finished && e.row / p.P == b) & fin;
                    fin &= ~same;
                    rows_done(p, tally, b, __popc(same), &s_decide);
                }
            }
            continue;       // next range
        }

        // =================================================================== streaming warps
        const uint32_t ring = smem_u32(ring_raw) + warp * (kSStages * kStageBytes);
        const uint32_t bars = smem_u32(&s_bar[warp][0]);

        // ---- producer side (all lanes follow, lane 0 issues): the unit being fed into the ring
        int pu_row = 0, pu_chunk = 0, pu_e = 0, pu_begin = 0, pu_end = 0, pu_slot = 0, pu_local = 0;
        bool pu_done = !wait_ok;          // after an expired wait this warp only reports itself done
        auto produce = [&](int stage) {
            for (;;) {
                if (pu_done) {
                    if (lane == 0) s_desc[warp][stage].row = -1;
                    return;
                }
                if (pu_e < pu_end) {
                    const int n = min(kPiece, pu_end - pu_e);
                    if (lane == 0) {
                        PieceDesc d;
                        d.row = pu_row; d.chunk = pu_chunk; d.e_begin = pu_e; d.n = n;
                        d.ordinal = (pu_e - pu_begin) / kPiece; d.last = pu_e + n >= pu_end;
                        d.slot = pu_slot; d.local_row = pu_local;
                        s_desc[warp][stage] = d;
                        const uint32_t bytes = (uint32_t)n * 2u;
                        const uint32_t bar = bars + 8 * stage, dst = ring + stage * kStageBytes;
                        const size_t off = (size_t)pu_row * p.V + pu_e;
                        mbar_expect_tx(bar, KL ? 2 * bytes : bytes);
                        bulk_load(dst, p.verifier + off, bytes, bar);
                        if (KL) bulk_load(dst + kTensorBytes, p.drafter + off, bytes, bar);
                    }
                    pu_e += n;
                    return;
                }
                // next unit of the range
                unsigned int t = 0;
                if (lane == 0) t = atomicAdd(&s_next, 1u);
                t = __shfl_sync(full, t, 0);
                if (t >= (unsigned)n_units) { pu_done = true; continue; }
                const long unit = lo + t;
                const long f = unit / nch;
                pu_chunk = (int)(unit - f * nch);
                pu_local = (int)(f - f_lo);
                pu_row = s_rows[pu_local];
                pu_slot = (int)t;
                pu_begin = pu_e = pu_chunk * kSChunk;
                pu_end = min(p.V, pu_begin + kSChunk);
            }
        };

        // the ring is empty here; its stages continue in order across ranges
        for (int s = 0; s < kSStages; ++s) produce((ring_uses + s) % kSStages);
        __syncwarp();

        LaneState L;
        lane_reset(L);
        for (;; ++ring_uses) {
            const int stage = ring_uses % kSStages;
            const uint32_t parity = (ring_uses / kSStages) & 1u;
            const PieceDesc d = s_desc[warp][stage];
            if (d.row < 0) break;

            // bounded, warp-uniform wait for the stage's copies
            bool landed = false;
            for (unsigned it = 0; it < (1u << 22); ++it) {
                landed = mbar_try_wait(bars + 8 * stage, parity);
                if (__all_sync(full, landed)) { landed = true; break; }
                landed = false;
                if (it > 64) __nanosleep(32);
            }
            if (!landed) { wait_ok = false; break; }

            uint4 rv[kVecPerThread], rd[kVecPerThread];
            const uint32_t src = ring + stage * kStageBytes;
            const bool whole_piece = d.n == kPiece;
#pragma unroll
            for (int j = 0; j < kVecPerThread; ++j) {
                const int e0 = (lane + j * 32) * 8;
                if (whole_piece || e0 < d.n) {
                    rv[j] = lds128(src + e0 * 2);
                    if (KL) rd[j] = lds128(src + kTensorBytes + e0 * 2);
                    else rd[j] = make_uint4(0u, 0u, 0u, 0u);
                } else {
                    rv[j] = make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);
                    rd[j] = rv[j];
                }
            }
            __syncwarp();          // every lane has its vectors: the stage can be refilled
            produce(stage);
            __syncwarp();

            if (whole_piece) lane_piece<KL, true>(L, rv, rd, d.n, lane, d.ordinal);
            else lane_piece<KL, false>(L, rv, rd, d.n, lane, d.ordinal);
            if (!d.last) continue;

            // ---- the chunk is complete: into the table; the warp that completes the range's share
            // of a row hands the row on
            const Partial part = lanes_to_partial<KL>(L, d.chunk * kSChunk, lane);
            lane_reset(L);
            const long f = f_lo + d.local_row;
            const long first_unit = max(lo, f * nch), end_unit = min(hi, (f + 1) * nch);
            const int share = (int)(end_unit - first_unit);
            int complete = 0;
            if (lane == 0) {
                s_table[d.slot] = part;
                __threadfence_block();
                complete = atomicAdd(&s_rowcnt[d.local_row], 1u) + 1u == (unsigned)share;
            }
            complete = __shfl_sync(full, complete, 0);
            if (!complete) continue;
            __threadfence_block();
            RowEvent e;
            e.row = d.row;
            e.whole = share == nch;
            e.score = 0.f;
            e.argmax = 0;
            e.first_slot = (int)(first_unit - lo);
            e.first_chunk = (int)(first_unit - f * nch);
            e.count = share;
            e.pad = 0;
            if (e.whole) fold_partials<KL>(s_table + e.first_slot, nch, e.score, e.argmax);
            if (lane == 0) queue_ok &= queue_push(s_queue, e);
        }
        if (lane == 0) {
            __threadfence_block();
            atomicAdd(&s_queue.done, 1u);
        }
    }

    if (warp < kSStreamWarps && (!wait_ok || !queue_ok)) {
        if (lane == 0 && p.status)
            atomicCAS(p.status, 0u, (wait_ok ? kErrWaitQueue : kErrWaitPiece) | (blockIdx.x & 0xFF));
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);   // copies still in flight may land in the ring
    }
}

}  // namespace ddv
