// dd_bidir_attention: full-sequence bidirectional attention (Section 2.2; Eq. 3
// evaluated over the whole key range) for sm_100a.
//
// One CTA owns a tile of 128 query rows of one (batch, head) and walks over the
// keys in tiles of 128.  Q, K and V tiles arrive in shared memory by TMA (3-D
// tensor maps over [B*H, N, D], 128-byte swizzle; rows past N read as zero).
// S = Q K^T is a tcgen05 MMA into tensor memory; each of the 128 threads owns one
// query row (= one TMEM lane), reads its 128 scores, keeps the running row
// maximum and sum in fp32 (online softmax, base 2 with scale*log2e folded in),
// writes P = 2^(S - m) as bf16 back into the same TMEM columns, and O += P V is a
// second tcgen05 MMA whose A operand is read from TMEM.  O is rescaled in TMEM
// when the row maximum moves, normalised by the row sum at the end and rounded to
// bf16 once.
#include <cuda.h>
#include <cuda_bf16.h>
#include <math.h>

#include "dd_common.cuh"
#include "dd_ptx.cuh"

namespace {

using namespace ddptx;

constexpr int kBlockM = 128;   // query rows per CTA
constexpr int kBlockN = 128;   // keys per step
constexpr int kThreads = 128;
constexpr uint32_t kTmemCols = 256;       // S: [0,128)  O: [128,128+D)
constexpr uint32_t kColS = 0, kColO = 128;

enum : unsigned { kErrWaitQ = 0x100, kErrWaitKV = 0x200, kErrWaitS = 0x300, kErrWaitO = 0x400 };

struct AttnParams {
    __nv_bfloat16 *out;
    int BH, N, D;
    int m_blocks;
    float scale_log2;          // scale * log2(e)
    unsigned int *status;
    float *dbg;                // bring-up only: raw scores of the first key tile of CTA 0
};

template <int D>
struct Smem {
    static constexpr int kTileBytes = kBlockN * D * 2;     // one 128 x D bf16 tile
    static constexpr int kQ = 0;
    static constexpr int kK = kTileBytes;
    static constexpr int kV = 2 * kTileBytes;
    static constexpr int kBars = 3 * kTileBytes;           // 3 mbarriers + tmem slot
    static constexpr int kTotal = kBars + 64;
};

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
attention_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                 const __grid_constant__ CUtensorMap tm_v, const AttnParams p)
{
    extern __shared__ __align__(1024) unsigned char smem_dyn[];
    // 128-byte-swizzled tiles must start on a 1024-byte boundary
    const uint32_t smem_base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base + Smem<D>::kQ, sK = smem_base + Smem<D>::kK, sV = smem_base + Smem<D>::kV;
    const uint32_t bar_q = smem_base + Smem<D>::kBars, bar_kv = bar_q + 8, bar_mma = bar_q + 16;
    const uint32_t tmem_slot = bar_q + 24;
    unsigned char *smem_gen = smem_dyn + (smem_base - smem_u32(smem_dyn));
    volatile uint32_t *tmem_slot_gen = reinterpret_cast<volatile uint32_t *>(smem_gen + Smem<D>::kBars + 24);

    const int tid = threadIdx.x, warp = tid >> 5;
    const int bh = blockIdx.x / p.m_blocks;
    const int mb = blockIdx.x - bh * p.m_blocks;
    const int row0 = mb * kBlockM;
    const int nkv = (p.N + kBlockN - 1) / kBlockN;
    constexpr int kBoxes = D / 64;                 // 64-column (128-byte) boxes per tile row
    constexpr uint32_t kBoxBytes = 128 * 128;      // 128 rows x 128 bytes

    if (tid == 0) {
        prefetch_tmap(&tm_q); prefetch_tmap(&tm_k); prefetch_tmap(&tm_v);
        mbar_init(bar_q, 1); mbar_init(bar_kv, 1); mbar_init(bar_mma, 1);
        fence_mbar_init();
    }
    if (warp == 0) { tmem_alloc(tmem_slot, kTmemCols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot_gen;
    const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);   // this warp's 32 TMEM lanes

    if (tid == 0) {
        mbar_expect_tx(bar_q, Smem<D>::kTileBytes);
#pragma unroll
        for (int c = 0; c < kBoxes; ++c) tma_load_3d(sQ + c * kBoxBytes, &tm_q, bar_q, c * 64, row0, bh);
    }

    constexpr uint32_t kIdescS = idesc_bf16(kBlockM, kBlockN, false);
    constexpr uint32_t kIdescO = idesc_bf16(kBlockM, D, true);

    float m_run = -INFINITY, l_run = 0.f;
    uint32_t mma_phase = 0;
    unsigned err = 0;

    for (int j = 0; j < nkv && err == 0; ++j) {
        if (tid == 0) {
            mbar_expect_tx(bar_kv, 2 * Smem<D>::kTileBytes);
#pragma unroll
            for (int c = 0; c < kBoxes; ++c) {
                tma_load_3d(sK + c * kBoxBytes, &tm_k, bar_kv, c * 64, j * kBlockN, bh);
                tma_load_3d(sV + c * kBoxBytes, &tm_v, bar_kv, c * 64, j * kBlockN, bh);
            }
        }
        if (j == 0 && !mbar_wait(bar_q, 0)) { err = kErrWaitQ; break; }
        if (!mbar_wait(bar_kv, j & 1)) { err = kErrWaitKV; break; }
        __syncwarp();

        // ---- S = Q K^T
        if (tid == 0) {
            tc_fence_after();
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                const uint32_t off = (ks / 4) * kBoxBytes + (ks % 4) * 32;   // 16 bf16 = 32 bytes per k-step
                mma_ss(tmem + kColS, smem_desc_sw128(sQ + off, 16, 1024), smem_desc_sw128(sK + off, 16, 1024),
                       kIdescS, ks > 0);
            }
            mma_commit(bar_mma);
        }
        if (!mbar_wait(bar_mma, mma_phase)) { err = kErrWaitS; break; }
        mma_phase ^= 1;
        __syncwarp();
        tc_fence_after();

        // ---- online softmax on this thread's row
        float s[kBlockN];
#pragma unroll
        for (int c = 0; c < kBlockN / 32; ++c) {
            uint32_t r[32];
            tmem_ld32(lane_base + kColS + c * 32, r);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) s[c * 32 + i] = __uint_as_float(r[i]);
        }
        if (p.dbg && blockIdx.x == 0 && j == 0) {
            for (int i = 0; i < kBlockN; ++i) p.dbg[tid * kBlockN + i] = s[i];
        }
        const int valid = p.N - j * kBlockN;       // keys of this tile that exist
        float mx = -INFINITY;
#pragma unroll
        for (int i = 0; i < kBlockN; ++i) {
            if (i < valid) mx = fmaxf(mx, s[i]);
        }
        const float m_new = fmaxf(m_run, mx * p.scale_log2);
        const float alpha = ex2(m_run - m_new);
        float sum = 0.f;
        uint32_t pk[kBlockN / 2];
#pragma unroll
        for (int i = 0; i < kBlockN; i += 2) {
            // keys past the end of the sequence get weight zero (no -inf arithmetic: scale may be 0)
            const float p0 = i < valid ? ex2(fmaf(s[i], p.scale_log2, -m_new)) : 0.f;
            const float p1 = i + 1 < valid ? ex2(fmaf(s[i + 1], p.scale_log2, -m_new)) : 0.f;
            sum += p0 + p1;
            __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
            pk[i / 2] = *reinterpret_cast<uint32_t *>(&h);
        }
        l_run = l_run * alpha + sum;
        m_run = m_new;

        // rescale this row of O
        if (j > 0) {
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t r[32];
                tmem_ld32(lane_base + kColO + c * 32, r);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
                tmem_st32(lane_base + kColO + c * 32, r);
            }
        }
        // P (bf16, two per 32-bit column) over the first 64 columns of S
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            uint32_t r[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = pk[c * 32 + i];
            tmem_st32(lane_base + kColS + c * 32, r);
        }
        tmem_wait_st();
        tc_fence_before();
        __syncthreads();

        // ---- O += P V
        if (tid == 0) {
            tc_fence_after();
#pragma unroll
            for (int ks = 0; ks < kBlockN / 16; ++ks) {
                // 16 keys = two 8-row groups of 1024 bytes; column blocks of 64 are one box apart
                mma_ts(tmem + kColO, tmem + kColS + ks * 8, smem_desc_sw128(sV + ks * 2048, kBoxBytes, 1024),
                       kIdescO, (j > 0 || ks > 0));
            }
            mma_commit(bar_mma);
        }
        if (!mbar_wait(bar_mma, mma_phase)) { err = kErrWaitO; break; }
        mma_phase ^= 1;
        __syncwarp();
        tc_fence_after();
    }

    __syncwarp();
    if (err != 0) {
        atomicCAS(p.status, 0u, err | (unsigned)(blockIdx.x & 0xFF));
        // give copies that may still be in flight time to land before the shared memory is released
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    } else {
        // ---- epilogue: O / l -> bf16 -> global
        const int row = row0 + tid;
        const float inv = 1.f / l_run;
        __nv_bfloat16 *dst = p.out + ((size_t)bh * p.N + row) * D;
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
            uint32_t r[32];
            tmem_ld32(lane_base + kColO + c * 32, r);
            tmem_wait_ld();
            if (row < p.N) {
#pragma unroll
                for (int i = 0; i < 32; i += 8) {
                    uint32_t w[4];
#pragma unroll
                    for (int h = 0; h < 4; ++h) {
                        __nv_bfloat162 v = __floats2bfloat162_rn(__uint_as_float(r[i + 2 * h]) * inv,
                                                                 __uint_as_float(r[i + 2 * h + 1]) * inv);
                        w[h] = *reinterpret_cast<uint32_t *>(&v);
                    }
                    *reinterpret_cast<uint4 *>(dst + c * 32 + i) = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

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

// [BH, N, D] bf16, D innermost; box = 64 columns x 128 rows x 1, 128-byte swizzle, zero fill.
int make_tmap(CUtensorMap *m, const void *base, int BH, int N, int D)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return dd::cuda_fail(cudaErrorSymbolNotFound, "cuTensorMapEncodeTiled entry point");
    const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)N, (cuuint64_t)BH};
    const cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)N * D * 2};
    const cuuint32_t box[3] = {64, 128, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return dd::cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
    return DD_OK;
}

template <int D>
int launch(const CUtensorMap &tq, const CUtensorMap &tk, const CUtensorMap &tv, const AttnParams &p, cudaStream_t s)
{
    static bool attr_done[64] = {};
    int dev = 0;
    DD_CUDA_TRY(cudaGetDevice(&dev));
    const int smem = Smem<D>::kTotal + 1024;
    if (dev >= 0 && dev < 64 && !attr_done[dev]) {
        DD_CUDA_TRY(cudaFuncSetAttribute(attention_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        attr_done[dev] = true;
    }
    const long grid = (long)p.BH * p.m_blocks;
    attention_kernel<D><<<(unsigned)grid, kThreads, smem, s>>>(tq, tk, tv, p);
    DD_CUDA_TRY(cudaGetLastError());
    dd::count_launch();
    return DD_OK;
}

int attention_impl(const void *q, const void *k, const void *v, void *out, int B, int H, int N, int D,
                   float scale, void *stream, float *dbg)
{
    if (!q || !k || !v || !out) return DD_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || N <= 0 || D <= 0) return DD_ERR_INVALID_ARG;
    if (!isfinite(scale)) return DD_ERR_INVALID_ARG;
    if (scale < 0.f) return DD_ERR_UNSUPPORTED;
    if (D != 64 && D != 128) return DD_ERR_UNSUPPORTED;
    if ((((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)out) & 15) != 0) return DD_ERR_UNSUPPORTED;
    const long BH = (long)B * H;
    const int m_blocks = (N + kBlockM - 1) / kBlockM;
    if (BH * m_blocks >= (1L << 31) || BH >= (1L << 31)) return DD_ERR_UNSUPPORTED;

    dd::DeviceCtx *ctx = dd::current_ctx();
    if (!ctx) return DD_ERR_CUDA;
    if (!ctx->attn_status) {
        DD_CUDA_TRY(cudaMalloc(&ctx->attn_status, 256));
        DD_CUDA_TRY(cudaMemset(ctx->attn_status, 0, 256));
    }
    CUtensorMap tq, tk, tv;
    int rc;
    if ((rc = make_tmap(&tq, q, (int)BH, N, D)) != DD_OK) return rc;
    if ((rc = make_tmap(&tk, k, (int)BH, N, D)) != DD_OK) return rc;
    if ((rc = make_tmap(&tv, v, (int)BH, N, D)) != DD_OK) return rc;

    AttnParams p;
    p.out = (__nv_bfloat16 *)out;
    p.BH = (int)BH; p.N = N; p.D = D;
    p.m_blocks = m_blocks;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.status = ctx->attn_status;
    p.dbg = dbg;
    cudaStream_t s = (cudaStream_t)stream;
    return D == 64 ? launch<64>(tq, tk, tv, p, s) : launch<128>(tq, tk, tv, p, s);
}

}  // namespace

extern "C" int dd_bidir_attention(const void *q, const void *k, const void *v, void *out,
                                  int B, int H, int N, int D, float scale, void *stream)
{
    return attention_impl(q, k, v, out, B, H, N, D, scale, stream, nullptr);
}

// Bring-up aid (not part of the public header): also dumps the raw fp32 scores
// S = Q K^T of the first key tile of the first CTA into dbg[128*128].
extern "C" int dd_debug_attention(const void *q, const void *k, const void *v, void *out,
                                  int B, int H, int N, int D, float scale, void *stream, float *dbg)
{
    return attention_impl(q, k, v, out, B, H, N, D, scale, stream, dbg);
}
