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
    extern __shared__ __align__(128) unsigned char s_ring[];     // [consumer][stage][kSStageBytes]
    __shared__ __align__(8) unsigned long long s_full[kSConsumers][kSStages];    // mbarriers: the stage holds data
    __shared__ __align__(8) unsigned long long s_empty[kSConsumers][kSStages];   // mbarriers: the stage is free
    __shared__ __align__(16) int4 s_meta[kSConsumers][kSStages];  // what the stage holds
    __shared__ __align__(8) unsigned long long s_mailbox[kSConsumers][2];       // (unit index + 1) << 32 | ticket
    __shared__ __align__(16) EventQueue s_queue;
    __shared__ int s_prefix[kSThreads + 1];                       // flagged rows before each thread's slice
    __shared__ int s_scan[kSWarps];
    __shared__ int s_abort;                                       // a bounded wait expired somewhere in the CTA
    __shared__ DecideStage s_decide;                              // decision stage (publishing warp only)

    const unsigned full = 0xFFFFFFFFu;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nch = p.nchunks;
    constexpr int kStep = PieceOf<KL>::value;                    // logits per stage

    // ---- every thread counts the flagged rows of its contiguous slice of the B*P rows; the block
    // scan gives each thread the number of flagged rows before its slice, and the total
    const long n_rows = (long)p.B * p.P;
    const long slice = (n_rows + kSThreads - 1) / kSThreads;
    const long my_begin = min(n_rows, (long)tid * slice), my_end = min(n_rows, my_begin + slice);
    int my_count = 0;
    for (long r = my_begin; r < my_end; ++r) my_count += p.flags[r] != 0;
    long total_flagged;
    {
        int incl = my_count;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(full, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) s_scan[warp] = incl;
        if (tid < kSQueue) s_queue.ready[tid] = 0u;
        if (tid == 0) {
            s_queue.tail = s_queue.head = s_queue.done = 0u;
            s_abort = 0;
            for (int w = 0; w < kSConsumers; ++w) {
                for (int s = 0; s < kSStages; ++s) {
                    sbar_init(s_addr(&s_full[w][s]), 1);
                    sbar_init(s_addr(&s_empty[w][s]), 1);
                }
                s_mailbox[w][0] = s_mailbox[w][1] = 0ull;
            }
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        __syncthreads();
        int before = 0, all = 0;
        for (int w = 0; w < kSWarps; ++w) {
            const int v = s_scan[w];
            if (w < warp) before += v;
            all += v;
        }
        s_prefix[tid] = before + incl - my_count;
        if (tid == 0) s_prefix[kSThreads] = all;
        total_flagged = all;
    }
    __syncthreads();
    const long total_units = total_flagged * nch;
    volatile int *abort_flag = &s_abort;

    if (warp < kSConsumers) {
        // ===================================================================== consumer warps
        const uint32_t ring = s_addr(s_ring) + (uint32_t)(warp * kSStages * kSStageBytes);
        const unsigned char *ring_gen = s_ring + warp * kSStages * kSStageBytes;
        unsigned int ticket = 0;          // lane 0: drawn at the start of unit j for unit j + 2
        unsigned units = 0;               // units started
        unsigned err = 0;
        LaneState L;
        lane_reset(L);
        for (unsigned it = 0;; ++it) {
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
            const int4 meta = s_meta[warp][stage];            // n logits, flags | piece << 8, row, chunk
            const int n = meta.x;
            if (n == 0) break;                                // no more units for this warp
            const bool first = (meta.y & 1) != 0, last = (meta.y & 2) != 0;
            if (first) {
                if (lane == 0) {
                    // the unit after this one becomes known to the producer; the one after that is drawn
                    if (units >= 1)
                        *(volatile unsigned long long *)&s_mailbox[warp][(units + 1) & 1] =
                            ((unsigned long long)(units + 2) << 32) | ticket;
                    ticket = atomicAdd(p.ticket, 1u);
                }
                ++units;
            }
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
            lane_pass1<KL>(L, rv, rd, meta.y >> 8, first);
            // every lane's vectors are in registers (the first pass has used them): the stage goes back
            __syncwarp();
            if (lane == 0) sbar_arrive(s_addr(&s_empty[warp][stage]));
            if (n == kStep) lane_pass2<KL, true>(L, rv, rd, n, lane);
            else lane_pass2<KL, false>(L, rv, rd, n, lane);
            if (!last) continue;

            // ---- the chunk is complete: one partial, handed to the publishing warp
            Partial part = lanes_to_partial<KL>(L, meta.w * p.chunk, lane);
            lane_reset(L);
            if (!(isfinite(part.s_v) && isfinite(part.s_d) && isfinite(part.t) && part.m_v > -INFINITY)) {
                const int begin = meta.w * p.chunk;
                part = careful_chunk_partial<KL>(p.verifier + (size_t)meta.z * p.V,
                                                 KL ? p.drafter + (size_t)meta.z * p.V : nullptr,
                                                 begin, min(p.V, begin + p.chunk));
            }
            if (!queue_push(s_queue, meta.z, meta.w, part, lane)) { err = kErrWaitQueue; break; }
        }
        if (lane == 0) {
            if (err) {
                *abort_flag = 1;
                if (p.status) atomicCAS(p.status, 0u, err | (blockIdx.x & 0xFF));
            }
            __threadfence_block();
            atomicAdd(&s_queue.done, 1u);
        }
    } else if (warp == kSProducerWarp) {
        // ===================================================================== producer warp
        // lane w feeds consumer w; lanes poll in lockstep and never block on one consumer
        const int w = lane;
        enum { kNeed, kHave, kLast, kDone };
        int state = w < kSConsumers ? kNeed : kDone;
        unsigned it = 0;                  // stages issued to this consumer
        unsigned k = 0;                   // units taken for this consumer
        int row = 0, chunk = 0, piece = 0, npieces = 0;
        unsigned stuck = 0;
        const long static0 = (long)blockIdx.x * kSConsumers + w;
        const long static1 = (long)gridDim.x * kSConsumers + static0;
        const long ticket_base = 2L * gridDim.x * kSConsumers;
        const int chunk_pieces = p.chunk / kStep;
        const int last_pieces = (p.V - (nch - 1) * p.chunk + kStep - 1) / kStep;         // of a row's last chunk
        const uint32_t ring = s_addr(s_ring) + (uint32_t)(w * kSStages * kSStageBytes);
        while (__any_sync(full, state != kDone)) {
            bool progress = false;
            if (state == kNeed) {
                long unit = -2;                                   // -2: not known yet
                if (k == 0) unit = static0;
                else if (k == 1) unit = static1;
                else {
                    const unsigned long long m = *(volatile unsigned long long *)&s_mailbox[w][k & 1];
                    if ((unsigned)(m >> 32) == k + 1u) unit = ticket_base + (long)(unsigned)m;
                }
                if (unit != -2) {
                    if (unit >= total_units) {
                        state = kLast;
                    } else {
                        const int f = (int)(unit / nch);          // ordinal of the flagged row
                        chunk = (int)(unit - (long)f * nch);
                        // the thread slice that holds flagged row f, then the row within it
                        int lo = 0, hi = kSThreads - 1;
                        while (lo < hi) {
                            const int mid = (lo + hi + 1) >> 1;
                            if (s_prefix[mid] <= f) lo = mid; else hi = mid - 1;
                        }
                        long r = (long)lo * slice;
                        const long r_end = min(n_rows, r + slice);
                        int ord = s_prefix[lo];
                        for (; r < r_end; ++r) {
                            if (p.flags[r]) {
                                if (ord == f) break;
                                ++ord;
                            }
                        }
                        row = (int)r;
                        npieces = chunk == nch - 1 ? last_pieces : chunk_pieces;
                        piece = 0;
                        state = kHave;
                    }
                    ++k;
                    progress = true;
                }
            }
            if (state == kHave || state == kLast) {
                const unsigned stage = it % kSStages, use = it / kSStages;
                if (use == 0 || sbar_try_wait(s_addr(&s_empty[w][stage]), (use - 1) & 1)) {
                    const uint32_t bar = s_addr(&s_full[w][stage]);
                    if (state == kLast) {
                        s_meta[w][stage] = make_int4(0, 0, 0, 0);
                        sbar_arrive(bar);
                        state = kDone;
                    } else {
                        const int e_begin = chunk * p.chunk + piece * kStep;
                        const int n = min(kStep, p.V - e_begin);
                        const int fl = (piece == 0 ? 1 : 0) | (piece == npieces - 1 ? 2 : 0) | (piece << 8);
                        s_meta[w][stage] = make_int4(n, fl, row, chunk);
                        const uint32_t bytes = (uint32_t)n * 2u;
                        const uint32_t dst = ring + stage * kSStageBytes;
                        const size_t off = (size_t)row * p.V + e_begin;
                        sbar_expect_tx(bar, KL ? 2u * bytes : bytes);
                        bulk_load(dst, p.verifier + off, bytes, bar);
                        if (KL) bulk_load(dst + kSStageBytes / 2, p.drafter + off, bytes, bar);
                        if (++piece == npieces) state = kNeed;
                    }
                    ++it;
                    progress = true;
                }
            }
            if (progress) {
                stuck = 0;
            } else if (state != kDone && ++stuck > (1u << 21)) {
                // the consumer never freed a stage or never named its next unit
                *abort_flag = 1;
                if (p.status) atomicCAS(p.status, 0u, (state == kNeed ? kErrWaitUnit : kErrWaitEmpty) | (blockIdx.x & 0xFF));
                state = kDone;
            }
            if (*abort_flag) break;
            if (!__any_sync(full, progress)) __nanosleep(100);
        }
    } else {
        // ===================================================================== publishing warp
        SeqTally tally;
        tally.b = -1;
        tally.target = 0;
        {
            // nothing is finished yet: bring the code of the row fold and of the decision stage
            // into the instruction caches now, not at the end of the launch
            __shared__ float s_rehearsal[2];
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
            // sequences without a single flagged row pass through; this CTA's share of them
            for (int b = blockIdx.x; b < p.B; b += gridDim.x)
                if (count_flagged(p, b) == 0) decide_sequence(p, b, &s_decide);
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
                if (done == (unsigned)kSConsumers && tail == head) break;
                if (++idle > (1u << 23)) {     // the consumer warps never finished
                    if (lane == 0) {
                        *abort_flag = 1;
                        if (p.status) atomicCAS(p.status, 0u, kErrWaitQueue | (blockIdx.x & 0xFF));
                    }
                    break;
                }
                __nanosleep(200);
                continue;
            }
            idle = 0;
            __threadfence_block();
            const bool mine_ok = lane < n;
            const UnitEvent *src = &s_queue.entry[(mine_ok ? mine : head) % kSQueue];
            const float4 e0 = reinterpret_cast<const float4 *>(src)[0];
            const float4 e1 = reinterpret_cast<const float4 *>(src)[1];
            const float4 e2 = reinterpret_cast<const float4 *>(src)[2];
            const int row = __float_as_int(e0.x), chunk = __float_as_int(e0.y);
            __syncwarp();
            head += n;
            if (lane == 0) *(volatile unsigned int *)&s_queue.head = head;

            // the partials go to global memory; one fence for the batch, then one count per unit
            if (mine_ok) {
                float4 *dst = reinterpret_cast<float4 *>(p.partials + (size_t)row * nch + chunk);
                __stcg(dst, e1);
                __stcg(dst + 1, e2);
            }
            __threadfence();
            bool complete = false;
            if (mine_ok) complete = atomicAdd(p.row_counter + row, 1u) + 1u == (unsigned)nch;
            const unsigned fold = __ballot_sync(full, complete);
            if (fold == 0u) continue;
            __threadfence();
            float my_score = 0.f;
            int my_argmax = 0;
            for (unsigned m = fold; m; m &= m - 1) {
                const int from = __ffs(m) - 1;
                const int r = __shfl_sync(full, row, from);
                float score;
                int argmax;
                fold_partials<KL>(p.partials + (size_t)r * nch, nch, score, argmax);
                if (lane == from) {
                    my_score = score;
                    my_argmax = argmax;
                    p.row_counter[r] = 0u;      // ready for the next launch
                }
            }
            // finished rows: store, fence once, count them per sequence
            if (complete) {
                __stcg(p.row_score + row, my_score);
                __stcg(p.row_argmax + row, my_argmax);
            }
            __threadfence();
            unsigned fin = fold;
            while (fin) {
                const int from = __ffs(fin) - 1;
                const int b = __shfl_sync(full, row, from) / p.P;
                const unsigned same = __ballot_sync(full, complete && row / p.P == b) & fin;
                fin &= ~same;
                rows_done(p, tally, b, __popc(same), &s_decide);
            }
        }
    }

    // ---- the ticket counter goes back to zero once every CTA has drawn its last ticket
    __syncthreads();
    if (*abort_flag) {
        // a wait expired: give copies that may still be in flight time to land before the shared
        // memory is released
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
        __syncthreads();
    }
    if (tid == 0) {
        __threadfence();
        if (atomicAdd(p.ctas_done, 1u) == gridDim.x - 1) {
            *p.ticket = 0u;
            __threadfence();
            *p.ctas_done = 0u;
        }
    }
}

}  // namespace ddv
