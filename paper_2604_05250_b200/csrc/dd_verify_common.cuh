// Shared device code of the dd_verify kernels: the per-(row, chunk) partial, the
// row fold (Eq. 5, Eq. 7) and the decision stage (Section 3.2 rules, Eq. 6,
// minimum-keep top-k, Philox uniforms).  Both kernels end a chunk the same way:
// publish its partial, count it; the warp that sees a row's last chunk folds the
// row, and the warp that sees a sequence's last row decides the sequence.
#pragma once

#include <cuda_bf16.h>
#include <math.h>
#include <stdint.h>

#include "dd_common.cuh"

namespace ddv {

constexpr int kVecPerThread = 4;                              // 16-byte vectors per thread per tensor
constexpr int kMaxP = 8192;
constexpr float kLog2e = 1.4426950408889634f;
constexpr double kLn2 = 0.69314718055994530942;

struct __align__(16) Partial {   // one per (row, chunk); 32 bytes
    float m_v, s_v;              // verifier: maximum, sum 2^(l*log2e - M) with M = m*log2e rounded once
    int idx;                     // lowest index of the verifier's maximum
    float m_d;                   // drafter: reference point of its sums (at most its maximum)
    float s_d, t;                // drafter: sum 2^(..), sum 2^(..) (l_D - l_V)
    float pad0, pad1;            // in flight inside a kernel: row and chunk as integer bits
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
    unsigned int *status;        // one word: first expired wait of the streaming kernel (may be null)
    unsigned int *mirror;        // its copy in mapped host memory, written only when a wait expires (may be null)
};

// Records the first expired wait of a launch: in the device word and, so that the host sees it
// without a synchronisation, in its host copy.
__device__ __forceinline__ void report_expired(const VerifyParams &p, unsigned code)
{
    const unsigned word = code | (unsigned)(blockIdx.x & 0xFF);
    if (p.status && atomicCAS(p.status, 0u, word) == 0u && p.mirror) {
        *reinterpret_cast<volatile unsigned int *>(p.mirror) = word;
        __threadfence_system();
    }
}

// Bounds-checked build (-DDD_BOUNDS_CHECK, `python -m paper_2604_05250_b200.build --check`): every
// index these kernels form into a caller's tensor or into the library's scratch goes through
// checked(), which compares it with the extent, records kErrBounds | site << 8 in the health word
// and substitutes index 0 (a legal one) on a violation, so that the launch finishes and the host
// reads the word.  In the normal build checked() is the identity.  (The attention kernels address
// global memory through tensor maps only, which the hardware clips.)
constexpr unsigned kErrBounds = 0xB000;
enum : unsigned { kSitePartial = 1, kSiteRow = 2, kSiteSeq = 3, kSiteLogit = 4, kSiteOut = 5, kSiteFlag = 6 };
#ifdef DD_BOUNDS_CHECK
constexpr bool kBoundsChecked = true;
#else
constexpr bool kBoundsChecked = false;
#endif
__device__ __forceinline__ size_t checked(const VerifyParams &p, long index, long extent, unsigned site)
{
    if (kBoundsChecked && (index < 0 || index >= extent)) {
        report_expired(p, kErrBounds | (site << 8));
        return 0;
    }
    return (size_t)index;
}
// the last element of a run of n starting at index (n >= 1) is checked as well
__device__ __forceinline__ size_t checked_run(const VerifyParams &p, long index, long n, long extent, unsigned site)
{
    if (kBoundsChecked && (index < 0 || n < 1 || index + n > extent)) {
        report_expired(p, kErrBounds | (site << 8));
        return 0;
    }
    return (size_t)index;
}

__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// 2^(M_old - M_new) for moving a sum to a new reference point; M_old = -inf gives 0, and two
// equal references (also both -inf) give 1.
__device__ __forceinline__ float rescale_factor(float M_old, float M_new)
{
    return M_new == M_old ? 1.f : ex2_approx(M_old - M_new);
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

// Monotone map float -> uint32 (larger float, larger integer); never 0 for a non-NaN input.
__device__ __forceinline__ uint32_t orderable(float f)
{
    const uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
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

// c <- c (+) o for two partials of disjoint logits, tolerant of empty ones (maximum -inf,
// sums 0).  Ties of the maximum keep the lower index.
template <bool KL>
__device__ __forceinline__ void merge_partial(Partial &c, const Partial &o)
{
    if (o.m_v > c.m_v) {
        c.s_v = c.s_v * rescale_factor(c.m_v * kLog2e, o.m_v * kLog2e) + o.s_v;
        c.m_v = o.m_v;
        c.idx = o.idx;
    } else if (o.m_v == c.m_v) {
        c.s_v += o.s_v;
        c.idx = min(c.idx, o.idx);
    } else {
        c.s_v += o.s_v * rescale_factor(o.m_v * kLog2e, c.m_v * kLog2e);
    }
    if (KL) {
        if (o.m_d > c.m_d) {
            const float f = rescale_factor(c.m_d * kLog2e, o.m_d * kLog2e);
            c.s_d = c.s_d * f + o.s_d;
            c.t = c.t * f + o.t;
            c.m_d = o.m_d;
        } else {
            const float f = rescale_factor(o.m_d * kLog2e, c.m_d * kLog2e);
            c.s_d += o.s_d * f;
            c.t += o.t * f;
        }
    }
}

}  // namespace ddv

#include "dd_verify_decide.cuh"
