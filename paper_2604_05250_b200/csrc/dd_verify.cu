// dd_verify: the verification algorithm A(p_D, p_V, x^D) of Algorithm 1
// (Section 3.2) as one memory-bound kernel launch.
//
// Work decomposition.  A flagged row (one position of the drafter-decoded set)
// is V logits from the verifier and, in KL mode, V from the drafter.  The row is
// cut into chunks; every (row, chunk) yields one partial
//     m_V, S_V = sum 2^(l_V*log2e - M_V), lowest index of the maximum,
//     m_D, S_D = sum 2^(l_D*log2e - M_D), T = sum 2^(l_D*log2e - M_D) (l_D - l_V)
// (M = m*log2e rounded once; any reference works as long as it is reused), and
// each logit is read from HBM exactly once.
//
// Streaming kernel (V % 8 == 0, 16-byte aligned logits; dd_verify_stream.cuh):
// persistent CTAs; a producer warp feeds per-warp rings in shared memory with bulk
// asynchronous copies, consumer warps accumulate chunks of up to 8192 logits from
// them, a publishing warp counts, folds and decides.
// Element-wise kernel (any V, any alignment; this file): one CTA of 256 threads
// per chunk of at most 8192 logits, 2-byte loads with bounds checks.
//
// The warp that sees a row's last chunk folds the row's chunk partials in chunk
// order in fp64 into  c_i = 2^(..)/S_V  (Eq. 7)  and
//     KL_i = T/S_D - lse_D + lse_V                                   (Eq. 5)
// and the warp that sees a sequence's last row runs the decision stage for it:
// Eq. 6 normaliser, Philox uniforms, threshold / probabilistic rule, the
// minimum-keep top-k, and the emitted tokens.  "Last" is decided with
// __threadfence + atomic counters that the last arriver resets to zero, so the
// scratch is ready for the next launch; every fold runs in a fixed order, so the
// result does not depend on the order in which warps finish.
#include <stdio.h>

#include <atomic>
#include <mutex>

#include "dd_verify_stream.cuh"
#include "dd_lm_head_kernel.cuh"

namespace {

using namespace ddv;

// ---------------------------------------------------------------------------
// Element-wise kernel.
constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxChunk = kThreads * kVecPerThread * 8;       // 8192 logits

// The thread's share of a chunk of n logits: vectors t, t+256, t+512, t+768 (8 logits each),
// -inf beyond the chunk's end.
__device__ __forceinline__ void load_chunk_elementwise(const uint16_t *row, int n, int tid,
                                                       uint4 (&r)[kVecPerThread])
{
#pragma unroll
    for (int j = 0; j < kVecPerThread; ++j) {
        const int e0 = (tid + j * kThreads) * 8;
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

__device__ __forceinline__ float vectors_max(const uint4 (&r)[kVecPerThread])
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

// Warp-level partial of the vectors the 32 lanes hold (thread t of kThreads; the chunk has n
// logits and starts at logit e_begin of the row).
template <bool KL>
__device__ __forceinline__ void warp_partial(const uint4 (&rv)[kVecPerThread], const uint4 (&rd)[kVecPerThread],
                                             int n, int e_begin, int t, Partial &out)
{
    const float m_v = warp_max(vectors_max(rv));
    float m_d = 0.f;
    if (KL) m_d = warp_max(vectors_max(rd));
    int idx = 0x7FFFFFFF;
#pragma unroll
    for (int j = kVecPerThread - 1; j >= 0; --j) {
        const uint32_t w[4] = {rv[j].x, rv[j].y, rv[j].z, rv[j].w};
#pragma unroll
        for (int h = 3; h >= 0; --h) {
            const int e = e_begin + (t + j * kThreads) * 8 + 2 * h;
            if (bf16hi(w[h]) == m_v) idx = e + 1;
            if (bf16lo(w[h]) == m_v) idx = e;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) idx = min(idx, __shfl_xor_sync(0xFFFFFFFFu, idx, o));

    // one ex2 per logit against the warp's reference
    const float M_v = m_v * kLog2e, M_d = m_d * kLog2e;
    float s_v0 = 0.f, s_v1 = 0.f, s_d0 = 0.f, s_d1 = 0.f, t0 = 0.f, t1 = 0.f;
#pragma unroll
    for (int j = 0; j < kVecPerThread; ++j) {
        const int e0 = (t + j * kThreads) * 8;
        if (e0 < n) {
            const uint32_t wv[4] = {rv[j].x, rv[j].y, rv[j].z, rv[j].w};
            uint32_t wd[4] = {0u, 0u, 0u, 0u};
            if (KL) { wd[0] = rd[j].x; wd[1] = rd[j].y; wd[2] = rd[j].z; wd[3] = rd[j].w; }
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                const bool ok0 = e0 + 2 * h < n, ok1 = e0 + 2 * h + 1 < n;
                const float v0 = bf16lo(wv[h]), v1 = bf16hi(wv[h]);
                // a logit of -inf is probability zero: no term (also when every logit of the warp is -inf)
                if (ok0 && v0 != -INFINITY) s_v0 += ex2_approx(fmaf(v0, kLog2e, -M_v));
                if (ok1 && v1 != -INFINITY) s_v1 += ex2_approx(fmaf(v1, kLog2e, -M_v));
                if (KL) {
                    const float d0 = bf16lo(wd[h]), d1 = bf16hi(wd[h]);
                    if (ok0 && d0 != -INFINITY) {
                        const float e = ex2_approx(fmaf(d0, kLog2e, -M_d));
                        s_d0 += e;
                        if (e > 0.f) t0 = fmaf(e, d0 - v0, t0);      // p_D = 0 contributes no term
                    }
                    if (ok1 && d1 != -INFINITY) {
                        const float e = ex2_approx(fmaf(d1, kLog2e, -M_d));
                        s_d1 += e;
                        if (e > 0.f) t1 = fmaf(e, d1 - v1, t1);
                    }
                }
            }
        }
    }
    out.m_v = m_v;
    out.s_v = warp_sum(s_v0 + s_v1);
    out.idx = idx;
    out.m_d = m_d;
    out.s_d = 0.f;
    out.t = 0.f;
    if (KL) {
        out.s_d = warp_sum(s_d0 + s_d1);
        out.t = warp_sum(t0 + t1);
    }
    out.pad0 = out.pad1 = 0.f;
}

constexpr int kEDecideKeys = 2048;      // keys of one sequence the element-wise kernel's deciding warp keeps in shared memory

template <bool KL>
__global__ void __launch_bounds__(kThreads, 3) verify_elementwise_kernel(const VerifyParams p)
{
    __shared__ Partial warp_part[kWarps];
    __shared__ uint32_t s_decide_keys[kEDecideKeys];   // decision stage (warp 0 only)
    DecideStage s_decide;
    s_decide.key = s_decide_keys;
    s_decide.capacity = kEDecideKeys;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int row = (int)checked(p, blockIdx.x / p.nchunks, (long)p.B * p.P, kSiteFlag);
    const int chunk = blockIdx.x - row * p.nchunks;

    if (!p.flags[row]) {
        // Unflagged rows cost nothing; warp 0 of their chunk-0 CTA reports the row as complete.
        if (chunk == 0 && warp == 0) row_done(p, row / p.P, &s_decide);
        return;
    }
    const int e_begin = chunk * p.chunk;
    const int n = min(p.chunk, p.V - e_begin);
    const size_t off = checked_run(p, (long)row * p.V + e_begin, n, (long)p.B * p.P * p.V, kSiteLogit);

    uint4 rv[kVecPerThread], rd[kVecPerThread];
    load_chunk_elementwise(p.verifier + off, n, tid, rv);
    if (KL) load_chunk_elementwise(p.drafter + off, n, tid, rd);
    Partial part;
    warp_partial<KL>(rv, rd, n, e_begin, tid, part);
    if (lane == 0) warp_part[warp] = part;
    __syncthreads();
    if (warp != 0) return;

    // warp 0 folds the eight warp partials in warp order (every lane the same arithmetic)
    Partial c = warp_part[0];
#pragma unroll
    for (int w = 1; w < kWarps; ++w) merge_partial<KL>(c, warp_part[w]);
    chunk_done<KL>(p, row, chunk, c, &s_decide);
}

// ---------------------------------------------------------------------------
// Host side.

// Counters live in their own allocation: it holds nothing else, so it is all zero whenever no
// launch is in flight, whatever (B, P) the previous call used.  Its last 256 bytes hold the
// streaming kernel's health word.
constexpr size_t kControlBytes = 256;
constexpr size_t kStatusOffset = 0;

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

bool streaming_path(const void *drafter, const void *verifier, int V, bool kl)
{
    return (V % 8 == 0) && (((uintptr_t)verifier & 15) == 0) && (!kl || ((uintptr_t)drafter & 15) == 0);
}

// Streaming path: stages per chunk (a chunk is the work of one warp and yields one partial).
// Four stages (16 KB of logits) keep the cost of ending a chunk small; fewer when the rows are
// too few to give every streaming warp of `sms` CTAs a couple of units; eight where every warp
// has many units anyway, or where the partials would not fit `max_partials` (0: no limit).
// The choice depends on the device, never on the grid actually launched.
int pick_pieces(int V, long rows, int sms, long max_partials, bool kl)
{
    const long step = kl ? kPiece : 2 * kPiece;
    auto chunks_of = [&](int k) { return (V + k * step - 1) / (k * step); };
    const int k_max = kl ? kMaxPiecesPerChunk : kMaxPiecesPerChunk / 2;      // 8192 logits either way
    int k = 4;
    const long want = 2L * kSConsumers * sms;
    while (k > 1 && rows * chunks_of(k) < want) k >>= 1;
    // The coarsest cut costs least (half the chunk ends, half the partials to fold and to publish)
    // as long as every CTA still gets about two units per streaming warp: cfg2 shape 5.95 against
    // 5.76 TB/s, cfg1 35.0 against 36.8 us; below that the ranges no longer balance (512 rows of a
    // 32000-entry vocabulary: 30.0 against 27.5 us).
    if (k == 4 && k_max == 8 && rows * chunks_of(8) >= 24L * sms) k = 8;
    while (max_partials > 0 && k < k_max && rows * chunks_of(k) > max_partials) k <<= 1;
    return k;
}

void chunking(int V, bool streaming, bool kl, int pieces, int *nchunks, int *chunk)
{
    if (streaming) {
        *chunk = pieces * (kl ? kPiece : 2 * kPiece);
        *nchunks = (V + *chunk - 1) / *chunk;
        return;
    }
    const int n = (V + kMaxChunk - 1) / kMaxChunk;
    int c = (V + n - 1) / n;
    c = (c + 7) & ~7;
    *nchunks = (V + c - 1) / c;
    *chunk = c;
}

std::mutex g_mu;                 // guards the per-device caches below
int g_sm_count[64] = {};
bool g_smem_attr_done[64][2] = {};
std::atomic<int> g_max_ctas{0};  // 0: one CTA per SM; otherwise a cap on the streaming kernel's grid

// Number of SMs of the current device (cached), or a negative status.
int sm_count_of_current_device()
{
    int dev = 0;
    DD_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return dd::cuda_fail(cudaErrorInvalidDevice, "dd_verify: device index");
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_sm_count[dev]) DD_CUDA_TRY(cudaDeviceGetAttribute(&g_sm_count[dev], cudaDevAttrMultiProcessorCount, dev));
    return g_sm_count[dev];
}

template <bool KL>
int launch_stream(const VerifyParams &p, cudaStream_t stream)
{
    const int sms = sm_count_of_current_device();
    if (sms < 0) return sms;
    int dev = 0;
    DD_CUDA_TRY(cudaGetDevice(&dev));
    {
        std::lock_guard<std::mutex> lock(g_mu);
        if (!g_smem_attr_done[dev][KL ? 1 : 0]) {
            DD_CUDA_TRY(cudaFuncSetAttribute(verify_stream_kernel<KL>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             kSRingBytes));
            // the same split of the SM's memory as the attention kernel that runs before and after
            DD_CUDA_TRY(cudaFuncSetAttribute(verify_stream_kernel<KL>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                             cudaSharedmemCarveoutMaxShared));
            g_smem_attr_done[dev][KL ? 1 : 0] = true;
        }
    }
    const long units = (long)p.B * p.P * p.nchunks;
    long grid = units < sms ? units : sms;
    const int cap = g_max_ctas.load(std::memory_order_relaxed);
    if (cap > 0 && grid > cap) grid = cap;
    verify_stream_kernel<KL><<<(unsigned)grid, kSThreads, kSRingBytes, stream>>>(p);
    DD_CUDA_TRY(cudaGetLastError());
    dd::count_launch();
    return DD_OK;
}

template <bool KL>
int launch_elementwise(const VerifyParams &p, cudaStream_t stream)
{
    const long grid = (long)p.B * p.P * p.nchunks;
    verify_elementwise_kernel<KL><<<(unsigned)grid, kThreads, 0, stream>>>(p);
    DD_CUDA_TRY(cudaGetLastError());
    dd::count_launch();
    return DD_OK;
}

int launch(const VerifyParams &p, bool streaming, cudaStream_t s)
{
    const bool kl = p.algo == DD_MODE_KL;
    if (streaming) return kl ? launch_stream<true>(p, s) : launch_stream<false>(p, s);
    return kl ? launch_elementwise<true>(p, s) : launch_elementwise<false>(p, s);
}

int check_args(const void *drafter_logits, const void *verifier_logits, const int32_t *tokens,
               const uint8_t *mask_flags, int mode, float tau, int k, const int32_t *out_tokens,
               const uint8_t *out_mask, int B, int P, int V)
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
    return DD_OK;
}

void fill_params(VerifyParams &p, const void *drafter_logits, const void *verifier_logits,
                 const int32_t *tokens, const uint8_t *mask_flags, int mode, float tau, int k, uint64_t seed,
                 int32_t *out_tokens, uint8_t *out_mask, float *out_score, int B, int P, int V)
{
    p.drafter = (const uint16_t *)drafter_logits;
    p.verifier = (const uint16_t *)verifier_logits;
    p.tokens = tokens;
    p.flags = mask_flags;
    p.out_tokens = out_tokens;
    p.out_mask = out_mask;
    p.out_score = out_score;
    p.B = B; p.P = P; p.V = V;
    p.algo = mode & 0xFF;
    p.probabilistic = (mode & DD_FLAG_PROBABILISTIC) != 0;
    p.emit_drafter = (mode & DD_FLAG_EMIT_DRAFTER) != 0;
    p.tau = tau;
    p.k = k;
    p.seed_lo = (uint32_t)(seed & 0xFFFFFFFFu);
    p.seed_hi = (uint32_t)(seed >> 32);
}

}  // namespace

extern "C" size_t dd_verify_workspace_bytes(int B, int P, int V)
{
    if (B <= 0 || P <= 0 || V <= 0) return 0;
    int nchunks, chunk;
    chunking(V, V % 8 == 0, true, 1, &nchunks, &chunk);       // the finest cut a launch may choose
    return workspace_bytes(B, P, nchunks) + counter_bytes(B, P) + kControlBytes;
}

extern "C" int dd_verify(const void *drafter_logits, const void *verifier_logits,
                         const int32_t *tokens, const uint8_t *mask_flags,
                         int mode, float tau, int k, uint64_t seed,
                         int32_t *out_tokens, uint8_t *out_mask, float *out_score,
                         int B, int P, int V, void *stream)
{
    int rc = check_args(drafter_logits, verifier_logits, tokens, mask_flags, mode, tau, k, out_tokens, out_mask,
                        B, P, V);
    if (rc != DD_OK) return rc;
    const bool kl = (mode & 0xFF) == DD_MODE_KL;
    const bool streaming = streaming_path(drafter_logits, verifier_logits, V, kl);

    VerifyParams p;
    int pieces = 4;
    if (streaming) {
        const int sms = sm_count_of_current_device();
        if (sms < 0) return sms;
        pieces = pick_pieces(V, (long)B * P, sms, 0, kl);
    }
    chunking(V, streaming, kl, pieces, &p.nchunks, &p.chunk);
    if ((long)B * P * p.nchunks >= (1L << 31) - (1L << 24)) return DD_ERR_UNSUPPORTED;

    dd::DeviceCtx *ctx = dd::current_ctx();
    if (!ctx) return DD_ERR_CUDA;
    if ((rc = dd::ensure_mirror(ctx)) != DD_OK) return rc;
    if ((rc = dd::check_mirror(ctx, 1)) != DD_OK) return rc;      // an earlier launch gave up a wait: nothing is launched
    rc = dd::ensure_bytes(&ctx->verify_ws, &ctx->verify_ws_bytes, workspace_bytes(B, P, p.nchunks));
    if (rc != DD_OK) return rc;
    rc = dd::ensure_bytes(&ctx->verify_cnt, &ctx->verify_cnt_bytes, counter_bytes(B, P) + kControlBytes);
    if (rc != DD_OK) return rc;

    const size_t bp = (size_t)B * P;
    p.row_counter = (unsigned int *)ctx->verify_cnt;
    p.seq_counter = (unsigned int *)((char *)ctx->verify_cnt + ((bp * 4 + 255) & ~size_t(255)));
    char *control = (char *)ctx->verify_cnt + ctx->verify_cnt_bytes - kControlBytes;
    p.status = (unsigned int *)(control + kStatusOffset);
    p.mirror = ctx->mirror_dev + 1;
    char *w = (char *)ctx->verify_ws;
    p.row_score = (float *)w;          w += (bp * 4 + 255) & ~size_t(255);
    p.row_argmax = (int *)w;           w += (bp * 4 + 255) & ~size_t(255);
    p.partials = (Partial *)w;

    fill_params(p, drafter_logits, verifier_logits, tokens, mask_flags, mode, tau, k, seed,
                out_tokens, out_mask, out_score, B, P, V);
    return launch(p, streaming, (cudaStream_t)stream);
}

// Unmask(p, x) of Algorithm 1's drafting phase: the confidence rule of dd_verify on one logits
// tensor.  "Stays masked" is "fails the threshold and is not among the k most confident": the
// CONF-mode decision with the roles of the outputs renamed, so it runs the same launch.
extern "C" int dd_unmask(const void *logits, const int32_t *tokens, const uint8_t *mask_flags,
                         float tau, int k, int32_t *out_tokens, uint8_t *out_mask, float *out_conf,
                         int B, int P, int V, void *stream)
{
    return dd_verify(nullptr, logits, tokens, mask_flags, DD_MODE_CONF, tau, k, 0, out_tokens, out_mask, out_conf,
                     B, P, V, stream);
}

extern "C" int dd_debug_set_max_ctas(int max_ctas)
{
    if (max_ctas < 0) return DD_ERR_INVALID_ARG;
    g_max_ctas.store(max_ctas, std::memory_order_relaxed);
    return DD_OK;
}

// ---------------------------------------------------------------------------
// dd_lm_head_verify: the verifier's language-model head fused with the verification algorithm.
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

// bf16 matrix [n_rows, K], K innermost, as a 2-D tensor map with boxes of 64 columns x box_rows rows,
// 128-byte swizzle; rows past the end read as zero.
int make_matrix_tmap(CUtensorMap *m, const void *base, long n_rows, int K, int box_rows)
{
    static EncodeTiledFn fn = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mu);
        if (!fn) {
            void *sym = nullptr;
            cudaDriverEntryPointQueryResult qr;
            if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qr) == cudaSuccess &&
                qr == cudaDriverEntryPointSuccess)
                fn = reinterpret_cast<EncodeTiledFn>(sym);
        }
    }
    if (!fn) return dd::cuda_fail(cudaErrorSymbolNotFound, "cuTensorMapEncodeTiled entry point");
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)n_rows};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return dd::cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
    return DD_OK;
}

// Vocabulary entries per work item: the multiple of 32 (at most `max_n`, at least half of it) for
// which the slowest CTA of `ctas` finishes first.  A work item of n entries takes about
// (fixed + n) units of time: the hidden-state tiles it loads and the MMAs' shared-memory reads of
// them do not shrink with n.  Measured at K = 4096 (time per item against n, tile widths forced):
// fixed = 140 for one product per item, 157 for the KL mode's two.  Counting n alone picked tiles
// of 128 entries at 4096 rows, 25 % slower than 256.
int pick_tile_n(int V, long row_blocks, int ctas, int max_n, int fixed)
{
    int best = max_n;
    long best_cost = -1;
    for (int n = max_n; n >= max_n / 2; n -= 32) {
        const long items = ((V + n - 1) / n) * row_blocks;
        const long cost = ((items + ctas - 1) / ctas) * (fixed + n);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = n; }
    }
    return best;
}

}  // namespace

extern "C" int dd_lm_head_verify(const void *drafter_hidden, const void *drafter_weight,
                                 const void *verifier_hidden, const void *verifier_weight,
                                 const int32_t *tokens, const uint8_t *mask_flags,
                                 int mode, float tau, int k, uint64_t seed,
                                 int32_t *out_tokens, uint8_t *out_mask, float *out_score,
                                 int B, int P, int K, int V, void *stream)
{
    if (!verifier_hidden || !verifier_weight) return DD_ERR_INVALID_ARG;
    if (K <= 0) return DD_ERR_INVALID_ARG;
    const bool kl = (mode & 0xFF) == DD_MODE_KL;
    if (kl && !drafter_weight) return DD_ERR_INVALID_ARG;
    int rc = check_args(kl ? drafter_hidden : nullptr, verifier_hidden, tokens, mask_flags, mode, tau, k, out_tokens,
                        out_mask, B, P, V);
    if (rc != DD_OK) return rc;
    if (K % ddlm::kBlockK != 0) return DD_ERR_UNSUPPORTED;
    if ((((uintptr_t)verifier_hidden | (uintptr_t)verifier_weight) & 15) != 0) return DD_ERR_UNSUPPORTED;
    if (kl && (((uintptr_t)drafter_hidden | (uintptr_t)drafter_weight) & 15) != 0) return DD_ERR_UNSUPPORTED;
    const long rows = (long)B * P;
    const int sms = sm_count_of_current_device();
    if (sms < 0) return sms;
    int cap = g_max_ctas.load(std::memory_order_relaxed);
    const int ctas = cap > 0 && cap < sms ? cap : sms;

    ddlm::LmParams q;
    q.rows = (int)rows; q.K = K; q.V = V;
    q.row_blocks = (int)((rows + ddlm::kRowsPerItem - 1) / ddlm::kRowsPerItem);
    q.N = kl ? pick_tile_n(V, q.row_blocks, sms, ddlm::kMaxN / 2, 157) : pick_tile_n(V, q.row_blocks, sms, ddlm::kMaxN, 140);
    q.n_tiles = (V + q.N - 1) / q.N;
    if (rows * q.n_tiles >= (1L << 31) - (1L << 24)) return DD_ERR_UNSUPPORTED;

    VerifyParams p;
    p.nchunks = q.n_tiles;
    p.chunk = q.N;
    dd::DeviceCtx *ctx = dd::current_ctx();
    if (!ctx) return DD_ERR_CUDA;
    if ((rc = dd::ensure_mirror(ctx)) != DD_OK) return rc;
    if ((rc = dd::check_mirror(ctx, 1)) != DD_OK) return rc;
    rc = dd::ensure_bytes(&ctx->verify_ws, &ctx->verify_ws_bytes, workspace_bytes(B, P, p.nchunks));
    if (rc != DD_OK) return rc;
    rc = dd::ensure_bytes(&ctx->verify_cnt, &ctx->verify_cnt_bytes, counter_bytes(B, P) + kControlBytes);
    if (rc != DD_OK) return rc;
    const size_t bp = (size_t)rows;
    p.row_counter = (unsigned int *)ctx->verify_cnt;
    p.seq_counter = (unsigned int *)((char *)ctx->verify_cnt + ((bp * 4 + 255) & ~size_t(255)));
    p.status = (unsigned int *)((char *)ctx->verify_cnt + ctx->verify_cnt_bytes - kControlBytes + kStatusOffset);
    p.mirror = ctx->mirror_dev + 1;
    char *w = (char *)ctx->verify_ws;
    p.row_score = (float *)w;          w += (bp * 4 + 255) & ~size_t(255);
    p.row_argmax = (int *)w;           w += (bp * 4 + 255) & ~size_t(255);
    p.partials = (Partial *)w;
    fill_params(p, nullptr, nullptr, tokens, mask_flags, mode, tau, k, seed, out_tokens, out_mask, out_score, B, P, V);

    CUtensorMap tm_h, tm_w, tm_hd, tm_wd;
    if ((rc = make_matrix_tmap(&tm_h, verifier_hidden, rows, K, 128)) != DD_OK) return rc;
    if ((rc = make_matrix_tmap(&tm_w, verifier_weight, V, K, q.N)) != DD_OK) return rc;
    tm_hd = tm_h; tm_wd = tm_w;                    // not read outside the KL mode
    if (kl) {
        if ((rc = make_matrix_tmap(&tm_hd, drafter_hidden, rows, K, 128)) != DD_OK) return rc;
        if ((rc = make_matrix_tmap(&tm_wd, drafter_weight, V, K, q.N)) != DD_OK) return rc;
    }

    int dev = 0;
    DD_CUDA_TRY(cudaGetDevice(&dev));
    {
        static bool attr_done[64] = {};
        std::lock_guard<std::mutex> lock(g_mu);
        if (!attr_done[dev]) {
            DD_CUDA_TRY(cudaFuncSetAttribute(ddlm::lm_head_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             ddlm::kSmemBytes));
            DD_CUDA_TRY(cudaFuncSetAttribute(ddlm::lm_head_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             ddlm::kSmemBytes));
            attr_done[dev] = true;
        }
    }
    const long items = (long)q.n_tiles * q.row_blocks;
    const unsigned grid = (unsigned)(items < ctas ? items : ctas);
    if (kl)
        ddlm::lm_head_kernel<true><<<grid, ddlm::kThreads, ddlm::kSmemBytes, (cudaStream_t)stream>>>(tm_h, tm_w, tm_hd, tm_wd, q, p);
    else
        ddlm::lm_head_kernel<false><<<grid, ddlm::kThreads, ddlm::kSmemBytes, (cudaStream_t)stream>>>(tm_h, tm_w, tm_hd, tm_wd, q, p);
    DD_CUDA_TRY(cudaGetLastError());
    dd::count_launch();
    // one warp per row, then one per sequence
    const unsigned fold_grid = (unsigned)((rows + B + ddlm::kFoldThreads / 32 - 1) / (ddlm::kFoldThreads / 32));
    if (kl)
        ddlm::lm_head_fold_kernel<true><<<fold_grid, ddlm::kFoldThreads, 0, (cudaStream_t)stream>>>(p, (int)rows);
    else
        ddlm::lm_head_fold_kernel<false><<<fold_grid, ddlm::kFoldThreads, 0, (cudaStream_t)stream>>>(p, (int)rows);
    DD_CUDA_TRY(cudaGetLastError());
    dd::count_launch();
    return DD_OK;
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
constexpr size_t kStaticRowsSlot = ((size_t)kStaticMaxRows * 4 + 255) & ~size_t(255);
constexpr size_t kStaticCounterBytes = 2 * kStaticRowsSlot + kControlBytes;   // rows, sequences, control words
constexpr size_t kStaticRowBytes = 2 * kStaticRowsSlot;                       // score + argmax
constexpr size_t kStaticScratchBytes = kStaticCounterBytes + kStaticRowBytes +
                                       (size_t)kStaticMaxPartials * sizeof(Partial);

// In host code this name is only a handle for cudaGetSymbolAddress, never an address to pass on.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// Device address of g_static_scratch per device, resolved on the first call made on that device
// (guarded by g_mu).
unsigned char *g_static_ptr[64] = {};

// The array's address on the current device (null if no call has resolved it yet).
unsigned char *static_scratch_if_resolved()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(g_mu);
    return g_static_ptr[dev];
}

}  // namespace

extern "C" int dd_verify_static(const void *drafter_logits, const void *verifier_logits,
                                const int32_t *tokens, const uint8_t *mask_flags,
                                int mode, float tau, int k, uint64_t seed,
                                int32_t *out_tokens, uint8_t *out_mask, float *out_score,
                                int B, int P, int V, void *stream)
{
    int rc = check_args(drafter_logits, verifier_logits, tokens, mask_flags, mode, tau, k, out_tokens, out_mask,
                        B, P, V);
    if (rc != DD_OK) return rc;
    const bool kl = (mode & 0xFF) == DD_MODE_KL;
    const bool streaming = streaming_path(drafter_logits, verifier_logits, V, kl);

    VerifyParams p;
    // the fixed scratch bounds the problem size (stated for chunks of 8192 logits; a finer cut is
    // only chosen where its partials still fit)
    const long coarse_chunks = (V + kSChunk - 1) / kSChunk;
    if ((long)B * P > kStaticMaxRows || (long)B * P * coarse_chunks > kStaticMaxPartials) return DD_ERR_UNSUPPORTED;
    int pieces = 4;
    if (streaming) {
        const int sms = sm_count_of_current_device();
        if (sms < 0) return sms;
        pieces = pick_pieces(V, (long)B * P, sms, kStaticMaxPartials, kl);
    }
    chunking(V, streaming, kl, pieces, &p.nchunks, &p.chunk);
    if ((long)B * P * p.nchunks > kStaticMaxPartials) return DD_ERR_UNSUPPORTED;

    int dev = -1;
    DD_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return dd::cuda_fail(cudaErrorInvalidDevice, "dd_verify_static: device index");
    unsigned char *base = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mu);
        if (!g_static_ptr[dev]) {
            // set-up, once per device, with that device current
            void *ptr = nullptr;
            DD_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_scratch));
            g_static_ptr[dev] = static_cast<unsigned char *>(ptr);
        }
        base = g_static_ptr[dev];
    }
    const size_t bp = (size_t)B * P;
    unsigned char *control = base + 2 * kStaticRowsSlot;
    p.row_counter = (unsigned int *)base;
    p.seq_counter = (unsigned int *)(base + kStaticRowsSlot);
    p.status = (unsigned int *)(control + kStatusOffset);
    {
        // the host copy of the health word is used if an earlier call of another entry point made
        // it; this entry point allocates nothing, not even pinned host memory
        dd::DeviceCtx *ctx = dd::current_ctx();
        if (!ctx) return DD_ERR_CUDA;
        if ((rc = dd::check_mirror(ctx, 1)) != DD_OK) return rc;
        p.mirror = ctx->mirror_dev ? ctx->mirror_dev + 1 : nullptr;
    }
    p.row_score = (float *)(base + kStaticCounterBytes);
    p.row_argmax = (int *)(base + kStaticCounterBytes + kStaticRowsSlot);
    p.partials = (Partial *)(base + kStaticCounterBytes + kStaticRowBytes);

    fill_params(p, drafter_logits, verifier_logits, tokens, mask_flags, mode, tau, k, seed,
                out_tokens, out_mask, out_score, B, P, V);

    cudaStream_t s = (cudaStream_t)stream;
    // The array keeps whatever the previous call left: the counters must start at zero (the
    // health word is left alone: it is sticky, like dd_verify's).
    DD_CUDA_TRY(cudaMemsetAsync(p.row_counter, 0, bp * 4, s));
    DD_CUDA_TRY(cudaMemsetAsync(p.seq_counter, 0, (size_t)B * 4, s));
    return launch(p, streaming, s);
}

extern "C" int dd_verify_status(void)
{
    dd::DeviceCtx *ctx = dd::current_ctx();
    if (!ctx) return DD_ERR_CUDA;
    unsigned char *fixed = static_scratch_if_resolved();
    if (!ctx->verify_cnt && !fixed) return DD_OK;
    unsigned int word = 0, word_fixed = 0;
    DD_CUDA_TRY(cudaDeviceSynchronize());
    if (ctx->verify_cnt)
        DD_CUDA_TRY(cudaMemcpy(&word, (char *)ctx->verify_cnt + ctx->verify_cnt_bytes - kControlBytes + kStatusOffset,
                               sizeof word, cudaMemcpyDeviceToHost));
    if (fixed)
        DD_CUDA_TRY(cudaMemcpy(&word_fixed, fixed + 2 * kStaticRowsSlot + kStatusOffset, sizeof word_fixed,
                               cudaMemcpyDeviceToHost));
    if (word == 0) word = word_fixed;
    if (word != 0) {
        char text[96];
        snprintf(text, sizeof text, "verify kernel: bounded wait expired, code 0x%08x", word);
        dd::set_error_text(text);
        return DD_ERR_TIMEOUT;
    }
    return DD_OK;
}

// ---------------------------------------------------------------------------
// Recovery and its test hook.

namespace {

// One thread waits on an mbarrier that nothing will ever complete, gives up after a few hundred
// polls and records the expiry exactly as the real kernels do.  The launch ends by itself within
// microseconds: this is how the error path is exercised without stalling a GPU.
__global__ void expire_wait_kernel(unsigned int *status, unsigned int *mirror, unsigned code)
{
    __shared__ __align__(8) unsigned long long bar;
    const uint32_t b = ddv::s_addr(&bar);
    ddv::sbar_init(b, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    bool arrived = false;
    for (int spin = 0; spin < 512 && !arrived; ++spin) arrived = ddv::sbar_try_wait(b, 0);
    if (!arrived && atomicCAS(status, 0u, code) == 0u && mirror) {
        *reinterpret_cast<volatile unsigned int *>(mirror) = code;
        __threadfence_system();
    }
}

}  // namespace

extern "C" int dd_debug_expire_wait(int which, void *stream)
{
    if (which != 0 && which != 1) return DD_ERR_INVALID_ARG;
    dd::DeviceCtx *ctx = dd::current_ctx();
    if (!ctx) return DD_ERR_CUDA;
    int rc = dd::ensure_mirror(ctx);
    if (rc != DD_OK) return rc;
    unsigned int *word = nullptr;
    if (which == 0) {
        if (!ctx->attn_status) {
            DD_CUDA_TRY(cudaMalloc(&ctx->attn_status, 256));
            DD_CUDA_TRY(cudaMemset(ctx->attn_status, 0, 256));
        }
        word = ctx->attn_status;
    } else {
        rc = dd::ensure_bytes(&ctx->verify_cnt, &ctx->verify_cnt_bytes, counter_bytes(1, 1) + kControlBytes);
        if (rc != DD_OK) return rc;
        word = (unsigned int *)((char *)ctx->verify_cnt + ctx->verify_cnt_bytes - kControlBytes + kStatusOffset);
    }
    expire_wait_kernel<<<1, 1, 0, (cudaStream_t)stream>>>(word, ctx->mirror_dev + which, 0xE000u + (unsigned)which);
    DD_CUDA_TRY(cudaGetLastError());
    return DD_OK;
}

extern "C" int dd_clear_status(void)
{
    dd::DeviceCtx *ctx = dd::current_ctx();
    if (!ctx) return DD_ERR_CUDA;
    DD_CUDA_TRY(cudaDeviceSynchronize());
    if (ctx->attn_status) DD_CUDA_TRY(cudaMemset(ctx->attn_status, 0, sizeof(unsigned int)));
    if (ctx->verify_cnt)
        DD_CUDA_TRY(cudaMemset((char *)ctx->verify_cnt + ctx->verify_cnt_bytes - kControlBytes + kStatusOffset, 0,
                               sizeof(unsigned int)));
    if (unsigned char *fixed = static_scratch_if_resolved())
        DD_CUDA_TRY(cudaMemset(fixed + 2 * kStaticRowsSlot + kStatusOffset, 0, sizeof(unsigned int)));
    if (ctx->mirror) ctx->mirror[0] = ctx->mirror[1] = 0u;
    return DD_OK;
}
