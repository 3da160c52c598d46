// dd_verify: the verification algorithm A(p_D, p_V, x^D) of Algorithm 1
// (Section 3.2) as one memory-bound kernel launch.
//
// Work decomposition.  A flagged row (one position of the drafter-decoded set)
// is V logits from the verifier and, in KL mode, V from the drafter.  The row is
// cut into `nchunks` equal chunks of at most 8192 logits; one CTA of 256 threads
// streams one (row, chunk): every thread holds four 16-byte vectors per tensor in
// registers, so a CTA has 32 KB (64 KB in KL mode) of loads in flight and each
// logit is read from HBM exactly once.  Per chunk the CTA produces
//     m_V, S_V = sum 2^(l_V*log2e - M_V), lowest index of the maximum,
//     m_D, S_D = sum 2^(l_D*log2e - M_D), T = sum 2^(l_D*log2e - M_D) (l_D - l_V)
// (M = m*log2e rounded once; any reference works as long as it is reused).
// The last CTA to finish a row folds the row's chunk partials in chunk order in
// fp64 into  c_i = 2^(..)/S_V  (Eq. 7)  and
//     KL_i = T/S_D - lse_D + lse_V                                   (Eq. 5)
// and the last CTA to finish a sequence runs the decision stage for it:
// Eq. 6 normaliser, Philox uniforms, threshold / probabilistic rule, the
// minimum-keep top-k, and the emitted tokens.  "Last" is decided with
// __threadfence + atomic counters that the last arriver resets to zero, so the
// scratch is ready for the next launch; every fold runs in a fixed order, so the
// result does not depend on the order in which CTAs finish.
#include <cuda_bf16.h>
#include <math.h>

#include "dd_common.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kVecPerThread = 4;                              // 16-byte vectors per thread per tensor
constexpr int kMaxChunk = kThreads * kVecPerThread * 8;       // 8192 logits
constexpr int kMaxP = 8192;
constexpr float kLog2e = 1.4426950408889634f;
constexpr double kLn2 = 0.69314718055994530942;

struct __align__(16) Partial {   // one per (row, chunk); 32 bytes
    float m_v, s_v;
    int idx;
    float m_d;
    float s_d, t, pad0, pad1;
};

struct VerifyParams {
    const uint16_t *drafter;
    const uint16_t *verifier;
    const int32_t *tokens;
    const uint8_t *flags;
    int32_t *out_tokens;
    uint8_t *out_mask;
    float *out_score;
    int B, P, V;
    int nchunks, chunk;
    int algo, probabilistic, emit_drafter;
    float tau;
    int k;
    uint32_t seed_lo, seed_hi;
    // scratch
    unsigned int *row_counter;   // [B*P]
    unsigned int *seq_counter;   // [B]
    float *row_score;            // [B*P]
    int *row_argmax;             // [B*P]
    Partial *partials;           // [B*P*nchunks]
};

__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

__device__ __forceinline__ uint4 ld_stream(const uint4 *p)
{
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}

// Philox4x32-10 (Salmon et al., SC'11): first output word for counter (c0,c1,0,0).
__device__ __forceinline__ uint32_t philox_first_word(uint32_t c0, uint32_t c1, uint32_t k0, uint32_t k1)
{
    uint32_t c2 = 0, c3 = 0;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        c0 = hi1 ^ c1 ^ k0;
        c1 = lo1;
        c2 = hi0 ^ c3 ^ k1;
        c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return c0;
}

// Monotone map float -> uint32 (larger float, larger integer).
__device__ __forceinline__ uint32_t orderable(float f)
{
    const uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Loads the thread's share of a chunk: vectors t, t+256, t+512, t+768 (8 logits each).
// VEC: 16-byte loads (row base and chunk are multiples of 8 logits, pointer aligned).
// Otherwise element-wise loads with -inf beyond the chunk's end.
template <bool VEC>
__device__ __forceinline__ void load_chunk(const uint16_t *row, int n, int tid, uint4 (&r)[kVecPerThread])
{
#pragma unroll
    for (int j = 0; j < kVecPerThread; ++j) {
        const int e0 = (tid + j * kThreads) * 8;
        if (VEC) {
            if (e0 < n) r[j] = ld_stream(reinterpret_cast<const uint4 *>(row + e0));
            else r[j] = make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);
        } else {
            uint32_t w[4];
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                const int a = e0 + 2 * h, b = a + 1;
                const uint32_t lo = a < n ? (uint32_t)__ldg(row + a) : 0xFF80u;
                const uint32_t hi = b < n ? (uint32_t)__ldg(row + b) : 0xFF80u;
                w[h] = lo | (hi << 16);
            }
            r[j] = make_uint4(w[0], w[1], w[2], w[3]);
        }
    }
}

__device__ __forceinline__ float chunk_max(const uint4 (&r)[kVecPerThread])
{
    __nv_bfloat162 m = __halves2bfloat162(__ushort_as_bfloat16(0xFF80), __ushort_as_bfloat16(0xFF80));
#pragma unroll
    for (int j = 0; j < kVecPerThread; ++j) {
        const uint32_t w[4] = {r[j].x, r[j].y, r[j].z, r[j].w};
#pragma unroll
        for (int h = 0; h < 4; ++h) m = __hmax2(m, *reinterpret_cast<const __nv_bfloat162 *>(&w[h]));
    }
    const uint32_t mw = *reinterpret_cast<uint32_t *>(&m);
    return fmaxf(bf16lo(mw), bf16hi(mw));
}

__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}
__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// ---------------------------------------------------------------------------
// Decision stage for one sequence, run by the whole CTA that completed it.
__device__ void decide_sequence(const VerifyParams &p, int b, unsigned long long *keys, double *red)
{
    const int tid = threadIdx.x;
    const long base = (long)b * p.P;
    const bool kl_mode = p.algo == DD_MODE_KL;

    // reliability keys of the flagged positions (0 for the others: they rank below every real key)
    double kl_part = 0.0;
    for (int i = tid; i < p.P; i += kThreads) {
        unsigned long long key = 0ull;
        if (p.flags[base + i]) {
            const float s = __ldcg(p.row_score + base + i);
            const float rel = kl_mode ? 0.0f - s : s;
            key = ((unsigned long long)orderable(rel) << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)i);
            kl_part += (double)s;
        }
        keys[i] = key;
    }
    // Eq. 6 normaliser: sum of KL over the drafter-decoded set, folded in a fixed order
    double kl_sum = 0.0;
    if (kl_mode && p.probabilistic) {
        const double w = warp_sum(kl_part);
        if ((tid & 31) == 0) red[tid >> 5] = w;
        __syncthreads();
        for (int wi = 0; wi < kWarps; ++wi) kl_sum += red[wi];
    }
    __syncthreads();

    for (int i = tid; i < p.P; i += kThreads) {
        const long t = base + i;
        const int32_t tok = p.tokens[t];
        if (!p.flags[t]) {
            p.out_tokens[t] = tok;
            p.out_mask[t] = 0;
            if (p.out_score) p.out_score[t] = 0.0f;
            continue;
        }
        const float s = __ldcg(p.row_score + t);
        bool fail = false;
        if (p.algo != DD_MODE_TRUST) {
            if (!p.probabilistic) {
                fail = kl_mode ? (s > p.tau) : (s < p.tau);
            } else {
                const uint32_t w = philox_first_word((uint32_t)i, (uint32_t)b, p.seed_lo, p.seed_hi);
                const double u = (double)(w >> 8) * (1.0 / 16777216.0);
                const double prob = kl_mode ? (kl_sum > 0.0 ? (double)s / kl_sum : 0.0) : 1.0 - (double)s;
                fail = u < prob;
            }
        }
        bool remask = false;
        if (fail) {
            remask = true;
            if (p.k > 0) {
                // rank = number of positions with a strictly larger key; kept if rank < k
                const unsigned long long mine = keys[i];
                int better = 0;
                for (int j = 0; j < p.P && better < p.k; ++j) better += keys[j] > mine;
                remask = better >= p.k;
            }
        }
        p.out_mask[t] = remask ? 1 : 0;
        p.out_tokens[t] = (remask || p.emit_drafter) ? tok : __ldcg(p.row_argmax + t);
        if (p.out_score) p.out_score[t] = s;
    }
}

// ---------------------------------------------------------------------------
template <bool KL, bool VEC>
__global__ void __launch_bounds__(kThreads, KL ? 3 : 4) verify_kernel(const VerifyParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    unsigned long long *keys = reinterpret_cast<unsigned long long *>(smem_raw);  // [P], decision stage
    __shared__ Partial warp_part[kWarps];
    __shared__ double red[kWarps];
    __shared__ int s_flag;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int row = blockIdx.x / p.nchunks;
    const int chunk = blockIdx.x - row * p.nchunks;
    const int b = row / p.P;

    bool seq_done = false;

    if (!p.flags[row]) {
        // Unflagged rows cost nothing; their chunk-0 CTA reports the row as complete.
        if (chunk != 0) return;
        if (tid == 0) {
            __threadfence();
            s_flag = atomicAdd(p.seq_counter + b, 1u) == (unsigned)(p.P - 1);
        }
        __syncthreads();
        seq_done = s_flag != 0;
    } else {
        const int e_begin = chunk * p.chunk;
        const int n = min(p.chunk, p.V - e_begin);
        const size_t off = (size_t)row * p.V + e_begin;

        uint4 rv[kVecPerThread], rd[kVecPerThread];
        load_chunk<VEC>(p.verifier + off, n, tid, rv);
        if (KL) load_chunk<VEC>(p.drafter + off, n, tid, rd);

        // pass 1 (registers): warp-wide maxima, lowest index of the verifier's maximum
        const float m_v = warp_max(chunk_max(rv));
        float m_d = 0.f;
        if (KL) m_d = warp_max(chunk_max(rd));
        int idx = 0x7FFFFFFF;
#pragma unroll
        for (int j = kVecPerThread - 1; j >= 0; --j) {
            const uint32_t w[4] = {rv[j].x, rv[j].y, rv[j].z, rv[j].w};
#pragma unroll
            for (int h = 3; h >= 0; --h) {
                const int e = e_begin + (tid + j * kThreads) * 8 + 2 * h;
                if (bf16hi(w[h]) == m_v) idx = e + 1;
                if (bf16lo(w[h]) == m_v) idx = e;
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) idx = min(idx, __shfl_xor_sync(0xFFFFFFFFu, idx, o));

        // pass 2 (registers): one ex2 per logit against the warp's reference
        const float M_v = m_v * kLog2e, M_d = m_d * kLog2e;
        float s_v0 = 0.f, s_v1 = 0.f, s_d0 = 0.f, s_d1 = 0.f, t0 = 0.f, t1 = 0.f;
#pragma unroll
        for (int j = 0; j < kVecPerThread; ++j) {
            const int e0 = (tid + j * kThreads) * 8;
            if (e0 < n) {
                const uint32_t wv[4] = {rv[j].x, rv[j].y, rv[j].z, rv[j].w};
                uint32_t wd[4] = {0u, 0u, 0u, 0u};
                if (KL) { wd[0] = rd[j].x; wd[1] = rd[j].y; wd[2] = rd[j].z; wd[3] = rd[j].w; }
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    const bool ok0 = VEC || (e0 + 2 * h < n), ok1 = VEC || (e0 + 2 * h + 1 < n);
                    const float v0 = bf16lo(wv[h]), v1 = bf16hi(wv[h]);
                    if (ok0) s_v0 += ex2_approx(fmaf(v0, kLog2e, -M_v));
                    if (ok1) s_v1 += ex2_approx(fmaf(v1, kLog2e, -M_v));
                    if (KL) {
                        const float d0 = bf16lo(wd[h]), d1 = bf16hi(wd[h]);
                        if (ok0) {
                            const float e = ex2_approx(fmaf(d0, kLog2e, -M_d));
                            s_d0 += e;
                            t0 = fmaf(e, d0 - v0, t0);
                        }
                        if (ok1) {
                            const float e = ex2_approx(fmaf(d1, kLog2e, -M_d));
                            s_d1 += e;
                            t1 = fmaf(e, d1 - v1, t1);
                        }
                    }
                }
            }
        }
        const float s_v = warp_sum(s_v0 + s_v1);
        float s_d = 0.f, t = 0.f;
        if (KL) {
            s_d = warp_sum(s_d0 + s_d1);
            t = warp_sum(t0 + t1);
        }
        if (lane == 0) {
            Partial w;
            w.m_v = m_v; w.s_v = s_v; w.idx = idx; w.m_d = m_d; w.s_d = s_d; w.t = t; w.pad0 = w.pad1 = 0.f;
            warp_part[warp] = w;
        }
        __syncthreads();

        // fold the eight warp partials (fixed order), publish the chunk partial, count the chunk
        if (tid == 0) {
            Partial c = warp_part[0];
#pragma unroll
            for (int w = 1; w < kWarps; ++w) {
                const Partial o = warp_part[w];
                if (o.m_v > c.m_v) {
                    c.s_v = c.s_v * ex2_approx(c.m_v * kLog2e - o.m_v * kLog2e) + o.s_v;
                    c.m_v = o.m_v;
                    c.idx = o.idx;
                } else {
                    c.s_v += o.s_v * ex2_approx(o.m_v * kLog2e - c.m_v * kLog2e);
                    if (o.m_v == c.m_v) c.idx = min(c.idx, o.idx);
                }
                if (KL) {
                    if (o.m_d > c.m_d) {
                        const float f = ex2_approx(c.m_d * kLog2e - o.m_d * kLog2e);
                        c.s_d = c.s_d * f + o.s_d;
                        c.t = c.t * f + o.t;
                        c.m_d = o.m_d;
                    } else {
                        const float f = ex2_approx(o.m_d * kLog2e - c.m_d * kLog2e);
                        c.s_d += o.s_d * f;
                        c.t += o.t * f;
                    }
                }
            }
            Partial *dst = p.partials + (size_t)row * p.nchunks + chunk;
            const float4 a = make_float4(c.m_v, c.s_v, __int_as_float(c.idx), c.m_d);
            const float4 bq = make_float4(c.s_d, c.t, 0.f, 0.f);
            __stcg(reinterpret_cast<float4 *>(dst), a);
            __stcg(reinterpret_cast<float4 *>(dst) + 1, bq);
            __threadfence();
            s_flag = atomicAdd(p.row_counter + row, 1u) == (unsigned)(p.nchunks - 1);
        }
        __syncthreads();
        if (!s_flag) return;
        __syncthreads();   // everyone has read s_flag before it is reused below

        // ---- this CTA finished the row: fold its chunk partials in chunk order (warp 0, fp64)
        if (warp == 0) {
            __threadfence();
            const Partial *src = p.partials + (size_t)row * p.nchunks;
            float bm_v = -INFINITY, bm_d = -INFINITY;
            int bidx = 0x7FFFFFFF;
            for (int c = lane; c < p.nchunks; c += 32) {
                const float4 a = __ldcg(reinterpret_cast<const float4 *>(src + c));
                const float mv = a.x, md = a.w;
                const int ix = __float_as_int(a.z);
                if (mv > bm_v || (mv == bm_v && ix < bidx)) { bm_v = mv; bidx = ix; }
                bm_d = fmaxf(bm_d, md);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float om = __shfl_xor_sync(0xFFFFFFFFu, bm_v, o);
                const int oi = __shfl_xor_sync(0xFFFFFFFFu, bidx, o);
                if (om > bm_v || (om == bm_v && oi < bidx)) { bm_v = om; bidx = oi; }
                bm_d = fmaxf(bm_d, __shfl_xor_sync(0xFFFFFFFFu, bm_d, o));
            }
            const float Mv = bm_v * kLog2e, Md = bm_d * kLog2e;
            double sv = 0.0, sd = 0.0, tt = 0.0;
            for (int c = lane; c < p.nchunks; c += 32) {
                const float4 a = __ldcg(reinterpret_cast<const float4 *>(src + c));
                const float4 bq = __ldcg(reinterpret_cast<const float4 *>(src + c) + 1);
                sv += (double)a.y * exp2((double)(a.x * kLog2e) - (double)Mv);
                if (KL) {
                    const double f = exp2((double)(a.w * kLog2e) - (double)Md);
                    sd += (double)bq.x * f;
                    tt += (double)bq.y * f;
                }
            }
            sv = warp_sum(sv);
            if (KL) { sd = warp_sum(sd); tt = warp_sum(tt); }
            if (lane == 0) {
                float score;
                if (KL) {
                    const double lse_v = (double)Mv * kLn2 + log(sv);
                    const double lse_d = (double)Md * kLn2 + log(sd);
                    const double kl = tt / sd - lse_d + lse_v;
                    score = (float)fmax(kl, 0.0);
                } else {
                    // the maximum's own term is 2^(m*log2e - M), not exactly 1
                    score = (float)(exp2((double)bm_v * (double)kLog2e - (double)Mv) / sv);
                }
                __stcg(p.row_score + row, score);
                __stcg(p.row_argmax + row, bidx);
                p.row_counter[row] = 0u;      // ready for the next launch
                __threadfence();
                s_flag = atomicAdd(p.seq_counter + b, 1u) == (unsigned)(p.P - 1);
            }
        }
        __syncthreads();
        seq_done = s_flag != 0;
    }

    if (!seq_done) return;
    // ---- this CTA finished the sequence: decision stage
    __threadfence();
    if (tid == 0) p.seq_counter[b] = 0u;      // ready for the next launch
    decide_sequence(p, b, keys, red);
}

// Counters live in their own allocation: it holds nothing else, so it is all zero whenever no
// launch is in flight, whatever (B, P) the previous call used.
size_t counter_bytes(int B, int P)
{
    const size_t bp = (size_t)B * P;
    return ((bp * 4 + 255) & ~size_t(255)) + (((size_t)B * 4 + 255) & ~size_t(255));
}

size_t workspace_bytes(int B, int P, int nchunks)
{
    const size_t bp = (size_t)B * P;
    size_t bytes = 0;
    bytes += (bp * 4 + 255) & ~size_t(255);           // row_score
    bytes += (bp * 4 + 255) & ~size_t(255);           // row_argmax
    bytes += bp * nchunks * sizeof(Partial);
    return bytes;
}

void chunking(int V, int *nchunks, int *chunk)
{
    const int n = (V + kMaxChunk - 1) / kMaxChunk;
    int c = (V + n - 1) / n;
    c = (c + 7) & ~7;
    *nchunks = (V + c - 1) / c;
    *chunk = c;
}

template <bool KL, bool VEC>
int launch(const VerifyParams &p, size_t smem, cudaStream_t stream)
{
    static bool attr_done[64] = {};
    int dev = 0;
    DD_CUDA_TRY(cudaGetDevice(&dev));
    if (dev >= 0 && dev < 64 && !attr_done[dev]) {
        DD_CUDA_TRY(cudaFuncSetAttribute(verify_kernel<KL, VEC>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         kMaxP * (int)sizeof(unsigned long long)));
        attr_done[dev] = true;
    }
    const long grid = (long)p.B * p.P * p.nchunks;
    verify_kernel<KL, VEC><<<(unsigned)grid, kThreads, smem, stream>>>(p);
    DD_CUDA_TRY(cudaGetLastError());
    dd::count_launch();
    return DD_OK;
}

}  // namespace

extern "C" size_t dd_verify_workspace_bytes(int B, int P, int V)
{
    if (B <= 0 || P <= 0 || V <= 0) return 0;
    int nchunks, chunk;
    chunking(V, &nchunks, &chunk);
    return workspace_bytes(B, P, nchunks) + counter_bytes(B, P);
}

extern "C" int dd_verify(const void *drafter_logits, const void *verifier_logits,
                         const int32_t *tokens, const uint8_t *mask_flags,
                         int mode, float tau, int k, uint64_t seed,
                         int32_t *out_tokens, uint8_t *out_mask, float *out_score,
                         int B, int P, int V, void *stream)
{
    const int algo = mode & 0xFF;
    if (!verifier_logits || !tokens || !mask_flags || !out_tokens || !out_mask) return DD_ERR_INVALID_ARG;
    if (B <= 0 || P <= 0 || V <= 0 || k < 0) return DD_ERR_INVALID_ARG;
    if (algo != DD_MODE_TRUST && algo != DD_MODE_KL && algo != DD_MODE_CONF) return DD_ERR_INVALID_ARG;
    if (mode & ~(0xFF | DD_FLAG_PROBABILISTIC | DD_FLAG_EMIT_DRAFTER)) return DD_ERR_INVALID_ARG;
    if (algo == DD_MODE_KL && !drafter_logits) return DD_ERR_INVALID_ARG;
    if (tau != tau) return DD_ERR_INVALID_ARG;
    if (P > kMaxP) return DD_ERR_UNSUPPORTED;
    if ((long)V >= (1L << 30)) return DD_ERR_UNSUPPORTED;

    VerifyParams p;
    chunking(V, &p.nchunks, &p.chunk);
    if ((long)B * P * p.nchunks >= (1L << 31)) return DD_ERR_UNSUPPORTED;

    dd::DeviceCtx *ctx = dd::current_ctx();
    if (!ctx) return DD_ERR_CUDA;
    int rc = dd::ensure_bytes(&ctx->verify_ws, &ctx->verify_ws_bytes, workspace_bytes(B, P, p.nchunks));
    if (rc != DD_OK) return rc;
    rc = dd::ensure_bytes(&ctx->verify_cnt, &ctx->verify_cnt_bytes, counter_bytes(B, P));
    if (rc != DD_OK) return rc;

    const size_t bp = (size_t)B * P;
    p.row_counter = (unsigned int *)ctx->verify_cnt;
    p.seq_counter = (unsigned int *)((char *)ctx->verify_cnt + ((bp * 4 + 255) & ~size_t(255)));
    char *w = (char *)ctx->verify_ws;
    p.row_score = (float *)w;          w += (bp * 4 + 255) & ~size_t(255);
    p.row_argmax = (int *)w;           w += (bp * 4 + 255) & ~size_t(255);
    p.partials = (Partial *)w;

    p.drafter = (const uint16_t *)drafter_logits;
    p.verifier = (const uint16_t *)verifier_logits;
    p.tokens = tokens;
    p.flags = mask_flags;
    p.out_tokens = out_tokens;
    p.out_mask = out_mask;
    p.out_score = out_score;
    p.B = B; p.P = P; p.V = V;
    p.algo = algo;
    p.probabilistic = (mode & DD_FLAG_PROBABILISTIC) != 0;
    p.emit_drafter = (mode & DD_FLAG_EMIT_DRAFTER) != 0;
    p.tau = tau;
    p.k = k;
    p.seed_lo = (uint32_t)(seed & 0xFFFFFFFFu);
    p.seed_hi = (uint32_t)(seed >> 32);

    const bool kl = algo == DD_MODE_KL;
    const bool vec = (V % 8 == 0) && (((uintptr_t)verifier_logits & 15) == 0) &&
                     (!kl || ((uintptr_t)drafter_logits & 15) == 0);
    const size_t smem = (size_t)P * sizeof(unsigned long long);
    cudaStream_t s = (cudaStream_t)stream;
    if (kl) return vec ? launch<true, true>(p, smem, s) : launch<true, false>(p, smem, s);
    return vec ? launch<false, true>(p, smem, s) : launch<false, false>(p, smem, s);
}

// ---------------------------------------------------------------------------
// dd_verify_static: the same kernel with its scratch in a fixed device array.
//
// Some callers must not allocate device memory at all: code running inside a
// pre-sized memory budget (an inference server that has handed every free byte
// to its KV cache), code that may not trigger the implicit device
// synchronisation of cudaMalloc/cudaFree, or a process whose allocator is owned
// by another runtime.  For them the partials, row results and completion
// counters live in the file-scope array below, which every GPU that loads this
// library holds until the process exits.
namespace {

constexpr int kStaticMaxRows = 4096;          // B * P
constexpr int kStaticMaxPartials = 65536;     // B * P * ceil(V / 8192)
constexpr size_t kStaticCounterBytes = (((size_t)kStaticMaxRows * 4 + 255) & ~size_t(255)) +
                                       (((size_t)kStaticMaxRows * 4 + 255) & ~size_t(255));   // rows + sequences
constexpr size_t kStaticRowBytes = 2 * (((size_t)kStaticMaxRows * 4 + 255) & ~size_t(255));  // score + argmax
constexpr size_t kStaticScratchBytes = kStaticCounterBytes + kStaticRowBytes +
                                       (size_t)kStaticMaxPartials * sizeof(Partial);

// In host code this name is only a handle for cudaGetSymbolAddress, never an address to pass on.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// Device address of g_static_scratch per device, resolved on the first call made on that device.
unsigned char *g_static_ptr[64] = {};

}  // namespace

extern "C" int dd_verify_static(const void *drafter_logits, const void *verifier_logits,
                                const int32_t *tokens, const uint8_t *mask_flags,
                                int mode, float tau, int k, uint64_t seed,
                                int32_t *out_tokens, uint8_t *out_mask, float *out_score,
                                int B, int P, int V, void *stream)
{
    const int algo = mode & 0xFF;
    if (!verifier_logits || !tokens || !mask_flags || !out_tokens || !out_mask) return DD_ERR_INVALID_ARG;
    if (B <= 0 || P <= 0 || V <= 0 || k < 0) return DD_ERR_INVALID_ARG;
    if (algo != DD_MODE_TRUST && algo != DD_MODE_KL && algo != DD_MODE_CONF) return DD_ERR_INVALID_ARG;
    if (mode & ~(0xFF | DD_FLAG_PROBABILISTIC | DD_FLAG_EMIT_DRAFTER)) return DD_ERR_INVALID_ARG;
    if (algo == DD_MODE_KL && !drafter_logits) return DD_ERR_INVALID_ARG;
    if (tau != tau) return DD_ERR_INVALID_ARG;
    if (P > kMaxP) return DD_ERR_UNSUPPORTED;
    if ((long)V >= (1L << 30)) return DD_ERR_UNSUPPORTED;

    VerifyParams p;
    chunking(V, &p.nchunks, &p.chunk);
    // the fixed scratch bounds the problem size
    if ((long)B * P > kStaticMaxRows || (long)B * P * p.nchunks > kStaticMaxPartials) return DD_ERR_UNSUPPORTED;

    int dev = -1;
    DD_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return dd::cuda_fail(cudaErrorInvalidDevice, "dd_verify_static: device index");
    if (!g_static_ptr[dev]) {
        // set-up, once per device, with that device current
        void *ptr = nullptr;
        DD_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_scratch));
        g_static_ptr[dev] = static_cast<unsigned char *>(ptr);
    }
    unsigned char *base = g_static_ptr[dev];
    const size_t bp = (size_t)B * P;
    const size_t rows_slot = ((size_t)kStaticMaxRows * 4 + 255) & ~size_t(255);
    p.row_counter = (unsigned int *)base;
    p.seq_counter = (unsigned int *)(base + rows_slot);
    p.row_score = (float *)(base + kStaticCounterBytes);
    p.row_argmax = (int *)(base + kStaticCounterBytes + rows_slot);
    p.partials = (Partial *)(base + kStaticCounterBytes + kStaticRowBytes);

    p.drafter = (const uint16_t *)drafter_logits;
    p.verifier = (const uint16_t *)verifier_logits;
    p.tokens = tokens;
    p.flags = mask_flags;
    p.out_tokens = out_tokens;
    p.out_mask = out_mask;
    p.out_score = out_score;
    p.B = B; p.P = P; p.V = V;
    p.algo = algo;
    p.probabilistic = (mode & DD_FLAG_PROBABILISTIC) != 0;
    p.emit_drafter = (mode & DD_FLAG_EMIT_DRAFTER) != 0;
    p.tau = tau;
    p.k = k;
    p.seed_lo = (uint32_t)(seed & 0xFFFFFFFFu);
    p.seed_hi = (uint32_t)(seed >> 32);

    cudaStream_t s = (cudaStream_t)stream;
    // The array keeps whatever the previous call left: the counters must start at zero.
    DD_CUDA_TRY(cudaMemsetAsync(p.row_counter, 0, bp * 4, s));
    DD_CUDA_TRY(cudaMemsetAsync(p.seq_counter, 0, (size_t)B * 4, s));

    const bool kl = algo == DD_MODE_KL;
    const bool vec = (V % 8 == 0) && (((uintptr_t)verifier_logits & 15) == 0) &&
                     (!kl || ((uintptr_t)drafter_logits & 15) == 0);
    const size_t smem = (size_t)P * sizeof(unsigned long long);
    if (kl) return vec ? launch<true, true>(p, smem, s) : launch<true, false>(p, smem, s);
    return vec ? launch<false, true>(p, smem, s) : launch<false, false>(p, smem, s);
}
