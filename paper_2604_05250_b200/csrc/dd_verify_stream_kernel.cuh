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

// Finished rows are counted per sequence.  The publishing warp collects the counts of a range
// (lane i holds one sequence and its count) and reports them together when the range ends: one
// fence and one counter update per sequence and range instead of one per batch of rows.
struct Pending {
    int b;          // this lane's sequence, -1: none
    int cnt;        // finished rows of that sequence not reported yet
    int target;     // flagged rows of that sequence (counted when the sequence first shows up)
    int used;       // lanes in use (the same in every lane)
};

// Reports every pending count; a sequence whose last rows these were is decided on the spot.
// The scores of the rows counted have been stored (not yet fenced) by this warp.
__device__ __forceinline__ void pending_flush(const VerifyParams &p, Pending &pend, DecideStage *stage)
{
    const unsigned full = 0xFFFFFFFFu;
    if (pend.used == 0) return;
    __threadfence();
    unsigned int before = 0u;
    if (pend.b >= 0) before = atomicAdd(p.seq_counter + checked(p, pend.b, p.B, kSiteSeq), (unsigned)pend.cnt);
    for (int e = 0; e < pend.used; ++e) {
        const int b = __shfl_sync(full, pend.b, e);
        const unsigned after = __shfl_sync(full, before, e) + (unsigned)__shfl_sync(full, pend.cnt, e);
        if (after != (unsigned)__shfl_sync(full, pend.target, e)) continue;
        __threadfence();
        if ((threadIdx.x & 31) == 0) p.seq_counter[b] = 0u;      // ready for the next launch
        decide_sequence(p, b, stage);
    }
    pend.b = -1;
    pend.cnt = 0;
    pend.target = 0;
    pend.used = 0;
}

// cnt more rows of sequence b are finished.
__device__ __forceinline__ void pending_add(const VerifyParams &p, Pending &pend, int b, int cnt, DecideStage *stage)
{
    const unsigned full = 0xFFFFFFFFu;
    const int lane = threadIdx.x & 31;
    const unsigned holder = __ballot_sync(full, pend.b == b);
    if (holder) {
        if (pend.b == b) pend.cnt += cnt;
        return;
    }
    if (pend.used == 32) pending_flush(p, pend, stage);
    const int target = count_flagged(p, b);
    if (lane == pend.used) {
        pend.b = b;
        pend.cnt = cnt;
        pend.target = target;
    }
    ++pend.used;
}

template <bool KL>
__global__ void __launch_bounds__(kSThreads, 1) verify_stream_kernel(const VerifyParams p)
{
    extern __shared__ __align__(128) unsigned char s_ring[];     // [warp][stage][kSStageBytes]
    __shared__ __align__(8) unsigned long long s_full[kSConsumers][kSStages];    // mbarriers: the stage holds data
    __shared__ __align__(16) int4 s_meta[kSConsumers][kSStages];  // what the stage holds
    // chunk partials of the current range; between ranges (every streaming warp has finished, every
    // row event has been taken) the same memory holds the keys of the sequence being decided
    constexpr int kTableSlots = kSDecideKeys * 4 / (int)sizeof(Partial);
    static_assert(kTableSlots >= kSTable, "the table fits the area");
    __shared__ __align__(16) Partial s_table[kTableSlots];       // kSTable slots in use as a table
    __shared__ __align__(16) Partial s_fake[32];                   // the rehearsal's partials
    __shared__ int s_rows[kSTable + 2];                           // flagged rows the range touches
    __shared__ unsigned int s_rowcnt[kSTable + 2];                // their chunks stored so far
    __shared__ __align__(16) EventQueue s_queue;
    __shared__ int s_scan[kSWarps];
    __shared__ int s_abort;                                       // a bounded wait expired somewhere in the CTA
    __shared__ int s_setup;                                       // 1: the flag scan is complete, 2: the first range is set up
    // Decision stage of the publishing warp at the end of a range.  Anywhere else (sequences
    // without a flagged row at the kernel's start; a flush in the middle of a range, which only
    // ranges over more than 32 sequences, hence short ones, ever need) the table is in use and the
    // decision runs without a key area.
    DecideStage s_decide, s_no_area;
    s_decide.key = reinterpret_cast<uint32_t *>(s_table);
    s_decide.capacity = kSDecideKeys;
    s_no_area.key = nullptr;
    s_no_area.capacity = 0;

    const unsigned full = 0xFFFFFFFFu;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nch = p.nchunks;
    constexpr int kStep = PieceOf<KL>::value;                    // logits per stage

    // ---- every thread counts the flagged rows of its contiguous slice of the B*P rows; the block
    // scan gives each thread the number of flagged rows before its slice, and the total
    // The publishing warp takes no part in the scan or in the set-up of the CTA's first range: it
    // spends that time (and the first microseconds of streaming) on the rehearsal below, and learns
    // through s_setup how far the streaming warps have come.
    constexpr int kScanThreads = kSConsumers * 32;
    const bool publisher = warp == kSPublisherWarp;
    volatile int *setup_flag = &s_setup;
    volatile int *abort_flag = &s_abort;
    const long n_rows = (long)p.B * p.P;
    if (publisher) {
        if (lane == 0) *setup_flag = 0;
        __threadfence_block();
        __syncwarp();
        cta_bar_arrive(1, kSThreads);         // the streaming warps pass this barrier after the flag is zero
    }
    if (publisher && lane < kSConsumers) {
        // Before anything is known about the flags: ask the L2 (and with it the address translation)
        // for the first lines this CTA would stream if every row were flagged, one unit per
        // streaming warp.  The first copies of a launch otherwise arrive up to 4 us apart, and a
        // CTA that starts late finishes late.  A prefetch has no effect on any result; where the
        // guess is wrong it is wasted.
        const unsigned units = (unsigned)n_rows * (unsigned)nch, per = (units + gridDim.x - 1) / gridDim.x;
        if (per <= (unsigned)kSTable) {
            const unsigned lo = blockIdx.x * (units / gridDim.x) + min(blockIdx.x, units % gridDim.x);
            const unsigned hi = lo + units / gridDim.x + (blockIdx.x < units % gridDim.x ? 1u : 0u);
            if (hi > lo) {
                const unsigned f_hi = (hi - 1) / (unsigned)nch;
                unsigned t = (unsigned)lane;
                if (f_hi > lo / (unsigned)nch && hi < (f_hi + 1) * (unsigned)nch) t += f_hi * (unsigned)nch - lo;
                if (t >= hi - lo) t -= hi - lo;
                if (t < hi - lo) {
                    const unsigned g = lo + t, f = g / (unsigned)nch;
                    const size_t off = (size_t)f * p.V + (size_t)(g - f * (unsigned)nch) * p.chunk;
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(p.verifier + off));
                    if (KL) asm volatile("prefetch.global.L2 [%0];" ::"l"(p.drafter + off));
                }
            }
        }
    }
    const long slice = (n_rows + kScanThreads - 1) / kScanThreads;
    const long my_begin = publisher ? n_rows : min(n_rows, (long)tid * slice);
    const long my_end = publisher ? n_rows : min(n_rows, my_begin + slice);
    long my_prefix = 0, total_flagged = 0;
    bool setup_lost = false;          // publishing warp: the streaming warps never reported
    if (!publisher) {
        int my_count = 0;
        for (long r = my_begin; r < my_end; ++r) my_count += p.flags[r] != 0;
        int incl = my_count;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(full, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) s_scan[warp] = incl;
        if (tid < kSConsumers * kSStages) sbar_init(s_addr(&s_full[0][0] + tid), 1);
        if (tid == 0) s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        cta_bar_sync(1, kSThreads);
        int before = 0, all = 0;
        for (int w = 0; w < kSConsumers; ++w) {
            const int v = s_scan[w];
            if (w < warp) before += v;
            all += v;
        }
        my_prefix = (long)before + incl - my_count;
        total_flagged = all;
        if (tid == 0) {
            __threadfence_block();
            *setup_flag = 1;
        }
    } else {
        // nothing is finished yet: bring the code of the row fold and of the decision stage into the
        // instruction caches now, not at the end of the launch, and decide the sequences without a
        // single flagged row (this CTA's share of them)
        __shared__ float s_rehearsal[2];
        float sc;
        int am;
        Partial *fake = s_fake;
        {
            Partial f;
            f.m_v = 1.f + lane; f.s_v = 1.5f; f.idx = lane; f.m_d = 0.5f * lane; f.s_d = 1.25f; f.t = 0.125f;
            f.pad0 = f.pad1 = 0.f;
            fake[lane] = f;
        }
        __syncwarp();
        fold_partials<KL>(fake, 32, sc, am);
        if (lane == 0) { s_rehearsal[0] = sc; s_rehearsal[1] = __int_as_float(am); }
        for (int b = blockIdx.x; b < p.B; b += gridDim.x)
            if (count_flagged(p, b) == 0) decide_sequence(p, b, &s_no_area);
        // the scan's result
        int seen = 0;
        for (unsigned spin = 0; spin < (1u << 22); ++spin) {
            seen = __shfl_sync(full, *setup_flag, 0);             // the same answer in every lane
            if (seen >= 1) break;
            __nanosleep(64);
        }
        __threadfence_block();
        if (seen >= 1) {
            int all = 0;
            for (int w = 0; w < kSConsumers; ++w) all += s_scan[w];
            total_flagged = all;
        } else {
            setup_lost = true;        // no range for this warp; reported below
        }
        // The decision stage (only its register-resident forms: the general form for longer
        // sequences is short loops written for a cold start, and a walk through it costs as much as
        // the decision itself).  Where the launch has so little to stream (less than a unit for
        // every other streaming warp of the grid) that its rows finish within microseconds, the
        // walk is the short one: finished rows wait while this warp rehearses.
        if (p.P <= 512)
            decide_sequence_rehearsal(p, &s_decide, 2L * total_flagged * nch <= (long)kSConsumers * gridDim.x);
    }
    // equal ranges, each small enough for the table, their number a multiple of the CTAs
    const unsigned total_units = (unsigned)(total_flagged * nch);          // fits 31 bits (checked by the host)
    const unsigned per_cta = (total_units + gridDim.x - 1) / gridDim.x;
    const unsigned rounds = per_cta > (unsigned)kSTable ? (per_cta + kSTable - 1) / kSTable : 1u;
    const unsigned n_ranges = rounds * gridDim.x;
    const unsigned range_len = total_units / n_ranges, range_extra = total_units % n_ranges;
    auto range_begin = [&](unsigned r) { return r * range_len + min(r, range_extra); };

    unsigned it = 0;                  // streaming warp: stages taken (across ranges)
    Pending pend;
    pend.b = -1;
    pend.cnt = 0;
    pend.target = 0;
    pend.used = 0;
    if (setup_lost && lane == 0) {
        *abort_flag = 1;
        report_expired(p, kErrWaitQueue);
    }
    bool first_range = true;

    for (unsigned range = blockIdx.x; range < n_ranges; range += gridDim.x) {
        const unsigned lo = range_begin(range), hi = range_begin(range + 1);
        if (hi <= lo) continue;                                   // uniform over the CTA
        const int n_units = (int)(hi - lo);
        const unsigned f_lo = lo / (unsigned)nch, f_hi = (hi - 1) / (unsigned)nch;   // flagged-row ordinals the range touches

        if (first_range && publisher) {
            // the streaming warps set the CTA's first range up among themselves
            int seen = 0;
            for (unsigned spin = 0; spin < (1u << 22); ++spin) {
                seen = __shfl_sync(full, *setup_flag, 0);
                if (seen >= 2) break;
                __nanosleep(64);
            }
            __threadfence_block();
            if (seen < 2) {
                if (lane == 0) {
                    *abort_flag = 1;
                    report_expired(p, kErrWaitQueue);
                }
                break;                                            // this warp only: the others see the flag
            }
        } else {
            if (!first_range) __syncthreads();                    // the previous range is fully drained
            long ord = my_prefix;
            for (long r = my_begin; r < my_end && ord <= (long)f_hi; ++r) {
                if (p.flags[r]) {
                    if (ord >= (long)f_lo) s_rows[ord - f_lo] = (int)r;
                    ++ord;
                }
            }
            const int helpers = first_range ? kScanThreads : kSThreads;       // tid < helpers here
            for (int i = tid; i < (int)(f_hi - f_lo + 1); i += helpers) s_rowcnt[i] = 0u;
            if (tid < kSQueue) s_queue.ready[tid] = 0u;
            if (tid == 0) s_queue.tail = s_queue.head = s_queue.done = s_queue.next_unit = 0u;
            if (first_range) {
                // no wait can have expired yet
                cta_bar_sync(2, kScanThreads);
                if (tid == 0) {
                    __threadfence_block();
                    *setup_flag = 2;
                }
            } else if (__syncthreads_or(*abort_flag)) {
                break;                                            // the same answer in every thread
            }
        }
        first_range = false;

        if (warp < kSConsumers) {
            // ================================================================= streaming warps
            const unsigned char *ring_gen = s_ring + warp * kSStages * kSStageBytes;
            const uint32_t ring = s_addr(s_ring) + (uint32_t)(warp * kSStages * kSStageBytes);
            const int chunk_pieces = p.chunk / kStep;
            const int last_pieces = (p.V - (nch - 1) * p.chunk + kStep - 1) / kStep;     // of a row's last chunk
            // The order in which the range's units are handed out starts with the range's share of
            // its last row, then its share of its first row (the two rows it may share with a
            // neighbour), then everything in between.
            int first_t = 0;
            if (f_hi > f_lo && hi < (f_hi + 1) * (unsigned)nch) first_t = (int)(f_hi * (unsigned)nch - lo);

            // ---- lane 0 feeds the ring: the piece it will issue next
            int i_row = 0, i_chunk = 0, i_piece = 0, i_npieces = 0, i_where = 0;
            bool i_more = true;               // false once the end marker has been posted
            const uint64_t policy = l2_evict_first_policy();
            auto issue = [&](unsigned stage) {
                if (!i_more) return;
                const uint32_t bar = s_addr(&s_full[warp][stage]);
                if (i_piece == i_npieces) {
                    // next unit of the range, or the end marker
                    const int u = (int)atomicAdd(&s_queue.next_unit, 1u);
                    if (u >= n_units) {
                        s_meta[warp][stage] = make_int4(0, 0, 0, 0);
                        sbar_arrive(bar);
                        i_more = false;
                        return;
                    }
                    int t = u + first_t;
                    if (t >= n_units) t -= n_units;
                    const unsigned g = lo + (unsigned)t, f = g / (unsigned)nch;
                    i_chunk = (int)(g - f * (unsigned)nch);
                    const int local_row = (int)(f - f_lo);
                    i_row = s_rows[local_row];
                    i_where = t | (local_row << 16);
                    i_npieces = i_chunk == nch - 1 ? last_pieces : chunk_pieces;
                    i_piece = 0;
                }
                const int e_begin = i_chunk * p.chunk + i_piece * kStep;
                const int n = min(kStep, p.V - e_begin);
                const int fl = n | (i_piece == 0 ? 1 << 16 : 0) | (i_piece == i_npieces - 1 ? 1 << 17 : 0) | (i_piece << 20);
                s_meta[warp][stage] = make_int4(fl, i_where, i_row, i_chunk);
                const uint32_t bytes = (uint32_t)n * 2u;
                const uint32_t dst = ring + stage * kSStageBytes;
                const size_t off = checked_run(p, (long)i_row * p.V + e_begin, n, n_rows * p.V, kSiteLogit);
                sbar_expect_tx(bar, KL ? 2u * bytes : bytes);
                bulk_load(dst, p.verifier + off, bytes, bar, policy);
                if (KL) bulk_load(dst + kSStageBytes / 2, p.drafter + off, bytes, bar, policy);
                ++i_piece;
            };
            if (lane == 0) {
#pragma unroll 1
                for (unsigned s = 0; s < (unsigned)kSStages; ++s) issue((it + s) % kSStages);
            }
            __syncwarp();

            unsigned err = 0;
            LaneState L;
            lane_reset(L);
            for (;; ++it) {
                const unsigned stage = it % kSStages, use = it / kSStages;
                {
                    const uint32_t bar = s_addr(&s_full[warp][stage]);
                    bool arrived = false;
                    for (unsigned spin = 0; spin < (1u << 22); ++spin) {
                        if (sbar_try_wait(bar, use & 1)) { arrived = true; break; }
                        if (spin > 32) {
                            __nanosleep(64);
                            if (*abort_flag) break;
                        }
                    }
                    if (!arrived) { err = kErrWaitFull; break; }
                }
                // n logits | first << 16 | last << 17 | piece << 20;  slot | local row << 16;  row;  chunk
                const int4 meta = s_meta[warp][stage];
                const int n = meta.x & 0xFFFF;
                if (n == 0) { ++it; break; }                      // the range has no more units for this warp
                const bool first = (meta.x & (1 << 16)) != 0, last = (meta.x & (1 << 17)) != 0;
                uint4 rv[kVecPerThread], rd[kVecPerThread];
                {
                    const uint4 *sv = reinterpret_cast<const uint4 *>(ring_gen + stage * kSStageBytes) + lane;
                    const uint4 *sd = sv + (kSStageBytes / 2) / 16;
#pragma unroll
                    for (int j = 0; j < kVecPerThread; ++j) {
                        rv[j] = sv[32 * j];
                        rd[j] = sd[32 * j];
                    }
                    if (n < kStep) {
                        // what lies beyond the row's end in the stage is stale: -inf instead
                        const uint4 ninf = make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);
#pragma unroll
                        for (int j = 0; j < kVecPerThread; ++j) {
                            if ((lane + 32 * j) * 8 >= n) rv[j] = ninf;
                            if ((lane + 32 * (KL ? j : kVecPerThread + j)) * 8 >= n) rd[j] = ninf;
                        }
                    }
                }
                lane_pass1<KL>(L, rv, rd, (meta.x >> 20) & 0xF, first);
                // every lane's vectors are in registers (the first pass has used them): the stage is
                // re-armed with the piece kSStages steps ahead
                __syncwarp();
                if (lane == 0) issue(stage);
                if (n == kStep) lane_pass2<KL, true>(L, rv, rd, n, lane);
                else lane_pass2<KL, false>(L, rv, rd, n, lane);
                if (!last) continue;

                // ---- the chunk is complete: into the table; the warp that completes the range's share
                // of a row hands the row on
                Partial part = lanes_to_partial<KL>(L, meta.w * p.chunk, lane);
                lane_reset(L);
                if (!(isfinite(part.s_v) && isfinite(part.s_d) && isfinite(part.t) && part.m_v > -INFINITY) ||
                    (KL && fabsf(part.t) > kExcludedExcess * part.s_d)) {
                    const int begin = meta.w * p.chunk;
                    const size_t row_off = checked_run(p, (long)meta.z * p.V, p.V, n_rows * p.V, kSiteLogit);
                    part = careful_chunk_partial<KL>(p.verifier + row_off, KL ? p.drafter + row_off : nullptr,
                                                     begin, min(p.V, begin + p.chunk));
                }
                const int slot = meta.y & 0xFFFF, local_row = meta.y >> 16;
                const unsigned row_first = (f_lo + (unsigned)local_row) * (unsigned)nch;   // the row's unit 0
                const unsigned first_unit = max(lo, row_first), end_unit = min(hi, row_first + (unsigned)nch);
                const int share = (int)(end_unit - first_unit);
                int complete = 0;
                if (lane == 0) {
                    s_table[slot] = part;
                    __threadfence_block();
                    complete = atomicAdd(&s_rowcnt[local_row], 1u) + 1u == (unsigned)share;
                }
                complete = __shfl_sync(full, complete, 0);
                if (!complete) continue;
                __threadfence_block();
                RowEvent e;
                e.row = meta.z;
                e.whole = share == nch;
                e.score = 0.f;
                e.argmax = 0;
                e.first_slot = (int)(first_unit - lo);
                e.first_chunk = (int)(first_unit - row_first);
                e.count = share;
                e.pad = 0;
                if (e.whole) fold_partials<KL>(s_table + e.first_slot, nch, e.score, e.argmax);
                int pushed = 1;
                if (lane == 0) pushed = queue_push(s_queue, e);
                if (!__shfl_sync(full, pushed, 0)) { err = kErrWaitQueue; break; }
            }
            if (lane == 0) {
                if (err) {
                    *abort_flag = 1;
                    report_expired(p, err);
                }
                __threadfence_block();
                atomicAdd(&s_queue.done, 1u);
            }
        } else {
            // ================================================================= publishing warp
            unsigned int head = 0;
            for (unsigned idle = 0;;) {
                const unsigned int mine = head + lane;
                const bool ready = *(volatile unsigned int *)&s_queue.ready[mine % kSQueue] == mine + 1u;
                const unsigned mask = __ballot_sync(full, ready);
                const int n = mask == full ? 32 : __ffs(~mask) - 1;      // contiguous ready entries
                if (n == 0) {
                    const unsigned int done = *(volatile unsigned int *)&s_queue.done;
                    const unsigned int tail = *(volatile unsigned int *)&s_queue.tail;
                    if (done == (unsigned)kSConsumers && tail == head) {
                        pending_flush(p, pend, &s_decide);          // the range is complete
                        break;
                    }
                    if (++idle > (1u << 23)) {     // the streaming warps never finished
                        if (lane == 0) {
                            *abort_flag = 1;
                            report_expired(p, kErrWaitQueue);
                        }
                        break;
                    }
                    __nanosleep(32);
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
                const unsigned parts = __ballot_sync(full, mine_ok && !e.whole);
                for (unsigned m = parts; m; m &= m - 1) {
                    const int from = __ffs(m) - 1;
                    const int row = __shfl_sync(full, e.row, from), slot0 = __shfl_sync(full, e.first_slot, from);
                    const int chunk0 = __shfl_sync(full, e.first_chunk, from), cnt = __shfl_sync(full, e.count, from);
                    Partial *dst = p.partials + checked_run(p, (long)row * nch + chunk0, cnt, n_rows * nch, kSitePartial);
                    for (int i = lane; i < 2 * cnt; i += 32)
                        __stcg(reinterpret_cast<float4 *>(dst) + i, reinterpret_cast<const float4 *>(s_table + slot0)[i]);
                }
                if (parts) {
                    __threadfence();
                    bool complete = false;
                    if (mine_ok && !e.whole)
                        complete = atomicAdd(p.row_counter + checked(p, e.row, n_rows, kSiteRow), (unsigned)e.count) + (unsigned)e.count == (unsigned)nch;
                    const unsigned fold = __ballot_sync(full, complete);
                    if (fold) __threadfence();
                    for (unsigned m = fold; m; m &= m - 1) {
                        const int from = __ffs(m) - 1;
                        const int row = __shfl_sync(full, e.row, from);
                        float score;
                        int argmax;
                        fold_partials<KL>(p.partials + checked_run(p, (long)row * nch, nch, n_rows * nch, kSitePartial), nch, score, argmax);
                        if (lane == from) {
                            e.whole = 1;
                            e.score = score;
                            e.argmax = argmax;
                            p.row_counter[row] = 0u;      // ready for the next launch
                        }
                    }
                }
                // finished rows: store, and count them per sequence
                const bool finished = mine_ok && e.whole;
                if (finished) {
                    const size_t row_at = checked(p, e.row, n_rows, kSiteRow);
                    __stcg(p.row_score + row_at, e.score);
                    __stcg(p.row_argmax + row_at, e.argmax);
                }
                unsigned fin = __ballot_sync(full, finished);
                while (fin) {
                    const int from = __ffs(fin) - 1;
                    const int b = __shfl_sync(full, e.row, from) / p.P;
                    const unsigned same = __ballot_sync(full, finished && e.row / p.P == b) & fin;
                    fin &= ~same;
                    pending_add(p, pend, b, __popc(same), &s_no_area);
                }
            }
        }
    }

    __syncthreads();
    if (*abort_flag) {
        // a wait expired: give copies that may still be in flight time to land before the shared
        // memory is released
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    }
}

}  // namespace ddv
