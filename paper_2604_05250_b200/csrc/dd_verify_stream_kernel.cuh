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
    __shared__ __align__(16) Partial s_table[kSTable];          // chunk partials of the current range
    __shared__ int s_rows[kSTable + 2];                          // flagged rows the range touches
    __shared__ unsigned int s_rowcnt[kSTable + 2];               // their chunks stored so far
    __shared__ __align__(16) EventQueue s_queue;
    __shared__ int s_scan[kSWarps];
    __shared__ DecideStage s_decide;                              // decision stage (publishing warp only)

    const unsigned full = 0xFFFFFFFFu;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nch = p.nchunks;

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
    // sequences without a single flagged row pass through; this CTA's share of them
    auto pass_through = [&]() {
        for (int b = blockIdx.x; b < p.B; b += gridDim.x)
            if (count_flagged(p, b) == 0) decide_sequence(p, b, &s_decide);
    };
    bool rehearsed = false;
    bool queue_ok = true;

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
                pass_through();
            }
            {
                // the sequence this range ends in: its size is needed when its rows are counted
                const int b_last = s_rows[(int)(f_hi - f_lo)] / p.P;
                if (tally.b != b_last) {
                    tally.b = b_last;
                    tally.target = count_flagged(p, b_last);
                }
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
                    __nanosleep(250);
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
        const unsigned ulo = (unsigned)lo, uhi = (unsigned)hi, uflo = (unsigned)f_lo;   // units fit 31 bits
        constexpr int kStep = PieceOf<KL>::value;                                        // logits per piece
        const int chunk_len = p.chunk, chunk_pieces = p.chunk / kStep;                  // logits, pieces per chunk
        const int last_pieces = (p.V - (nch - 1) * chunk_len + kStep - 1) / kStep;         // of a row's last chunk

        // Units of the range go to the streaming warps in turn: warp w takes units w, w + 15, ...
        // A cursor walks one warp's pieces in order (all lanes hold the same values).
        struct Cursor {
            int t;              // unit within the range (= its table slot); >= n_units: past the end
            int local_row;      // the unit's row, numbered within the range
            int chunk, piece, npieces, row;
        };
        auto enter_unit = [&](Cursor &c) {
            if (c.t >= n_units) return;
            c.npieces = c.chunk == nch - 1 ? last_pieces : chunk_pieces;
            c.row = s_rows[c.local_row];
        };
        auto advance = [&](Cursor &c) {
            if (++c.piece < c.npieces) return;
            c.piece = 0;
            c.t += kSStreamWarps;
            c.chunk += kSStreamWarps;
            if (c.chunk >= nch) {
                const int q = c.chunk / nch;
                c.chunk -= q * nch;
                c.local_row += q;
            }
            enter_unit(c);
        };
        // the lane's vectors of the cursor's piece, -inf where the row has ended: four per tensor, or
        // (no drafter tensor) eight of the verifier, the second four in d
        auto fetch = [&](const Cursor &c, uint4 (&v)[kVecPerThread], uint4 (&d)[kVecPerThread]) {
            const int e_begin = c.chunk * chunk_len + c.piece * kStep;
            const int n = p.V - e_begin;                      // logits left in the row
            const size_t off = (size_t)c.row * p.V + e_begin;
            const uint4 *gv = reinterpret_cast<const uint4 *>(p.verifier + off) + lane;
            const uint4 *gd = KL ? reinterpret_cast<const uint4 *>(p.drafter + off) + lane : gv + 32 * kVecPerThread;
            if (n >= kStep) {
#pragma unroll
                for (int j = 0; j < kVecPerThread; ++j) {
                    v[j] = ld_stream(gv + 32 * j);
                    d[j] = ld_stream(gd + 32 * j);
                }
            } else {
#pragma unroll
                for (int j = 0; j < kVecPerThread; ++j) {
                    v[j] = make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);
                    d[j] = v[j];
                    if ((lane + 32 * j) * 8 < n) v[j] = ld_stream(gv + 32 * j);
                    if ((lane + 32 * (KL ? j : kVecPerThread + j)) * 8 < n) d[j] = ld_stream(gd + 32 * j);
                }
            }
        };

        Cursor cc;
        {
            cc.t = warp;
            cc.piece = 0; cc.npieces = 0; cc.row = 0;
            const unsigned unit = ulo + (unsigned)warp, f = unit / (unsigned)nch;
            cc.chunk = (int)(unit - f * (unsigned)nch);
            cc.local_row = (int)(f - uflo);
            enter_unit(cc);
        }
        Cursor nc = cc;                                       // the piece whose loads are in flight
        uint4 nv[kVecPerThread], nd[kVecPerThread];
        if (nc.t < n_units) fetch(nc, nv, nd);

        LaneState L;
        lane_reset(L);
        while (cc.t < n_units) {
            uint4 rv[kVecPerThread], rd[kVecPerThread];
#pragma unroll
            for (int j = 0; j < kVecPerThread; ++j) { rv[j] = nv[j]; rd[j] = nd[j]; }
            advance(nc);
            if (nc.t < n_units) fetch(nc, nv, nd);            // in flight while this piece is computed

            const int n = min(kStep, p.V - (cc.chunk * chunk_len + cc.piece * kStep));
            if (n == kStep) lane_piece<KL, true>(L, rv, rd, n, lane, cc.piece);
            else lane_piece<KL, false>(L, rv, rd, n, lane, cc.piece);
            const bool chunk_ends = cc.piece == cc.npieces - 1;
            const Cursor done = cc;
            advance(cc);
            if (!chunk_ends) continue;

            // ---- the chunk is complete: into the table; the warp that completes the range's share
            // of a row hands the row on
            const Partial part = lanes_to_partial<KL>(L, done.chunk * chunk_len, lane);
            lane_reset(L);
            const unsigned row_first = (uflo + (unsigned)done.local_row) * (unsigned)nch;   // the row's unit 0
            const unsigned first_unit = max(ulo, row_first), end_unit = min(uhi, row_first + (unsigned)nch);
            const int share = (int)(end_unit - first_unit);
            int complete = 0;
            if (lane == 0) {
                s_table[done.t] = part;
                __threadfence_block();
                complete = atomicAdd(&s_rowcnt[done.local_row], 1u) + 1u == (unsigned)share;
            }
            complete = __shfl_sync(full, complete, 0);
            if (!complete) continue;
            __threadfence_block();
            RowEvent e;
            e.row = done.row;
            e.whole = share == nch;
            e.score = 0.f;
            e.argmax = 0;
            e.first_slot = (int)(first_unit - ulo);
            e.first_chunk = (int)(first_unit - row_first);
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

    if (warp == kSStreamWarps && !rehearsed) pass_through();      // this CTA had no range
    if (warp < kSStreamWarps && !queue_ok && lane == 0 && p.status)
        atomicCAS(p.status, 0u, kErrWaitQueue | (blockIdx.x & 0xFF));
}

}  // namespace ddv
