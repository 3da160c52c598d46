// The streaming kernel itself.  Included by dd_verify_stream.cuh.
#pragma once

namespace ddv {

template <bool KL>
__global__ void __launch_bounds__(kSThreads, 1) verify_stream_kernel(const VerifyParams p)
{
    extern __shared__ __align__(128) unsigned char ring_raw[];
    __shared__ __align__(8) unsigned long long s_bar[kSStreamWarps][kSStages];
    __shared__ __align__(16) PieceDesc s_desc[kSStreamWarps][kSStages];
    __shared__ __align__(16) ChunkQueue s_queue;
    __shared__ unsigned int s_next;

    constexpr int kTensorBytes = kPiece * 2;                      // one piece of one tensor
    constexpr int kStageBytes = (KL ? 2 : 1) * kTensorBytes;
    const unsigned full = 0xFFFFFFFFu;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    if (threadIdx.x == 0) {
        s_next = 0u;
        s_queue.tail = s_queue.head = s_queue.done = 0u;
    }
    if (threadIdx.x < kSQueue) s_queue.ready[threadIdx.x] = 0u;
    if (warp < kSStreamWarps && lane == 0) {
        for (int s = 0; s < kSStages; ++s) mbar_init(smem_u32(&s_bar[warp][s]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    if (warp == kSStreamWarps) {
        // =================================================================== publishing warp
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
                __nanosleep(200);
                continue;
            }
            idle = 0;
            __threadfence_block();
            const Partial e = s_queue.entry[(lane < n ? mine : head) % kSQueue];
            __syncwarp();
            head += n;
            if (lane == 0) *(volatile unsigned int *)&s_queue.head = head;
            publish_batch<KL>(p, e, n);
        }
        return;
    }

    // ======================================================================= streaming warps
    const uint32_t ring = smem_u32(ring_raw) + warp * (kSStages * kStageBytes);
    const uint32_t bars = smem_u32(&s_bar[warp][0]);

    // this CTA's share of the (row, chunk) units: blockIdx.x, blockIdx.x + gridDim.x, ...
    const long units = (long)p.B * p.P * p.nchunks;
    const long n_local = units > (long)blockIdx.x ? (units - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    bool queue_ok = true;

    // ---- producer side (all lanes follow, lane 0 issues): the unit being fed into the ring
    int pu_row = 0, pu_chunk = 0, pu_e = 0, pu_begin = 0, pu_end = 0;
    bool pu_done = false;
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
                    d.ordinal = (pu_e - pu_begin) / kPiece; d.last = pu_e + n >= pu_end; d.pad0 = d.pad1 = 0;
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
            // next unit of this CTA
            unsigned int t = 0;
            if (lane == 0) t = atomicAdd(&s_next, 1u);
            t = __shfl_sync(full, t, 0);
            if ((long)t >= n_local) { pu_done = true; continue; }
            const long u = (long)blockIdx.x + (long)t * gridDim.x;
            const int row = (int)(u / p.nchunks), chunk = (int)(u - (long)row * p.nchunks);
            if (!p.flags[row]) {
                // unflagged rows cost nothing; their chunk-0 unit has the row reported as complete
                if (chunk == 0 && lane == 0) {
                    Partial e;
                    e.m_v = e.s_v = e.m_d = e.s_d = e.t = 0.f;
                    e.idx = 0;
                    e.pad0 = __int_as_float(row);
                    e.pad1 = __int_as_float(-1);
                    queue_ok &= queue_push(s_queue, e);
                }
                continue;
            }
            pu_row = row; pu_chunk = chunk;
            pu_begin = pu_e = chunk * kSChunk;
            pu_end = min(p.V, pu_begin + kSChunk);
        }
    };

    for (int s = 0; s < kSStages; ++s) produce(s);
    __syncwarp();

    LaneState L;
    lane_reset(L);
    bool wait_ok = true;
    for (unsigned c = 0;; ++c) {
        const int stage = c % kSStages;
        const uint32_t parity = (c / kSStages) & 1u;
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
#pragma unroll
        for (int j = 0; j < kVecPerThread; ++j) {
            const int e0 = (lane + j * 32) * 8;
            if (e0 < d.n) {
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

        lane_piece<KL>(L, rv, rd, d.n, lane, d.ordinal);
        if (d.last) {
            Partial part = lanes_to_partial<KL>(L, d.chunk * kSChunk, lane);
            lane_reset(L);
            if (lane == 0) {
                part.pad0 = __int_as_float(d.row);
                part.pad1 = __int_as_float(d.chunk);
                queue_ok &= queue_push(s_queue, part);
            }
        }
    }
    if (lane == 0) {
        if ((!wait_ok || !queue_ok) && p.status)
            atomicCAS(p.status, 0u, (wait_ok ? kErrWaitQueue : kErrWaitPiece) | (blockIdx.x & 0xFF));
        __threadfence_block();
        atomicAdd(&s_queue.done, 1u);
    }
    if (!wait_ok) {
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);   // copies still in flight may land in the ring
    }
}

}  // namespace ddv
