/*
 * dualdiff.h -- C ABI of the B200 (sm_100a) library for the data-parallel core
 * of one DualDiffusion verification step (speculative decoding for masked
 * diffusion language models):
 *
 *   dd_bidir_attention : full-sequence bidirectional multi-head attention, the
 *                        O(L^2)-per-step cost of Section 2.2 (Eq. 3 evaluated
 *                        over the whole key range, no causal mask, no cache).
 *   dd_verify          : the verification algorithm A(p_D, p_V, x^D) of
 *                        Algorithm 1 / Section 3.2: Trust Verifier (Eq. 4),
 *                        KL-divergence remasking (Eq. 5, Eq. 6) and
 *                        confidence remasking (Eq. 7).
 *
 * Conventions shared by every entry point
 *   - Pointers named without a prefix are DEVICE pointers owned by the caller;
 *     the *_host entry points take HOST pointers (pinned memory if the copies
 *     are to be asynchronous).  Tensors are contiguous, innermost dimension
 *     last.  bf16 tensors are passed as void* to raw bf16 storage.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     All work is enqueued on it; no entry point synchronises the stream.
 *   - The return value is a dd_status; 0 is success.  On any error nothing is
 *     launched and no output is written.  The library never falls back to a
 *     CPU computation.
 *   - The library keeps a small per-device scratch area (partial results and
 *     completion counters of dd_verify, staging buffers of the *_host calls).
 *     It is allocated with cudaMalloc the first time a call on that device
 *     needs it, or needs more than before, which synchronises the device: make
 *     one call of the intended size before relying on asynchrony.  Two calls
 *     that may run concurrently on the same device (different streams, no
 *     ordering between them) would share this scratch and are not supported.
 *     dd_release() frees it.
 */
#ifndef DUALDIFF_H_
#define DUALDIFF_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DD_OK = 0,
    DD_ERR_INVALID_ARG = -1, /* null pointer, non-positive size, unknown mode, NaN tau, k < 0 */
    DD_ERR_UNSUPPORTED = -2, /* valid request outside what the kernels implement          */
    DD_ERR_CUDA = -3,        /* a CUDA runtime/driver call failed; see dd_last_cuda_error  */
    DD_ERR_TIMEOUT = -4      /* a bounded device-side wait expired (see dd_clear_status)    */
} dd_status;

/* `mode` argument of dd_verify: algorithm in the low 8 bits, flag bits above. */
enum {
    DD_MODE_TRUST = 0,             /* Eq. 4: nothing is remasked                              */
    DD_MODE_KL = 1,                /* Eq. 5 score; remask if KL > tau (threshold rule)        */
    DD_MODE_CONF = 2,              /* Eq. 7 score; remask if c_V < tau (threshold rule)       */
    DD_FLAG_PROBABILISTIC = 0x100, /* KL: remask w.p. Eq. 6; CONF: remask w.p. 1 - c_V        */
    DD_FLAG_EMIT_DRAFTER = 0x200   /* kept positions keep tokens[i] instead of the verifier's
                                      most likely token (Eq. 4 taken literally)               */
};

/*
 * Bidirectional attention (Section 2.2; Eq. 3 with the key range 1..L):
 *     out[b,h,i,:] = sum_j softmax_j(scale * q[b,h,i,:] . k[b,h,j,:]) v[b,h,j,:],
 * j over all N positions.  q, k, v, out: [B,H,N,D] bf16, D innermost, 16-byte
 * aligned, out not overlapping the inputs.  Scores and the softmax are
 * accumulated in fp32 (weights relative to a per-row reference point that may lag the
 * row maximum by a factor of up to 2^24: the result is finite for |v| * N < 2^100);
 * the result is rounded to bf16 once.
 * Supported: D in {64,128}; any N >= 1; scale >= 0; B*H*ceil(N/128) < 2^31.
 * Errors: DD_ERR_INVALID_ARG (null pointer, B/H/N/D <= 0, scale not finite),
 * DD_ERR_UNSUPPORTED (other D, negative scale, misaligned pointer), DD_ERR_CUDA.
 */
int dd_bidir_attention(const void *q, const void *k, const void *v, void *out,
                       int B, int H, int N, int D, float scale, void *stream);

/*
 * Verification algorithm A(p_D, p_V, x^D) (Algorithm 1, verification phase;
 * Section 3.2).  For every position i of sequence b with mask_flags[b,i] != 0
 * (the drafter-decoded set D of the sequence):
 *   a_i   = argmax_x verifier_logits[b,i,x], lowest index among ties
 *   c_i   = max_x softmax(verifier_logits[b,i,:])                    (Eq. 7)
 *   KL_i  = KL(softmax(drafter_logits[b,i,:]) || softmax(verifier_logits[b,i,:]))
 *           in nats                                                   (Eq. 5)
 *   fail_i: TRUST never; KL: KL_i > tau, or u_i < KL_i / sum_{j in D} KL_j with
 *           DD_FLAG_PROBABILISTIC (Eq. 6); CONF: c_i < tau, or u_i < 1 - c_i with
 *           DD_FLAG_PROBABILISTIC.  u_i = (w >> 8) * 2^-24 where w is the first
 *           word of Philox4x32-10 with key (seed low, seed high) and counter
 *           (i, b, 0, 0).
 *   The k positions of the sequence with the highest reliability (-KL_i or c_i,
 *   ties to the lower i) are kept whatever fail_i says; k = 0 disables this.
 *   out_mask[b,i]   = 1 if fail_i and not among those k, else 0
 *   out_tokens[b,i] = tokens[b,i] if remasked (the caller overlays its [MASK]
 *                     id) or if DD_FLAG_EMIT_DRAFTER; otherwise a_i
 *   out_score[b,i]  = KL_i (KL mode) or c_i (CONF and TRUST modes)
 * Positions with mask_flags == 0 pass through: out_tokens = tokens,
 * out_mask = 0, out_score = 0, and their logits are never read.
 * A logit of -inf is an excluded token (probability 0, an ordinary input: a banned or
 * padded vocabulary entry, the mask token): it contributes no term to Eq. 5 where the
 * drafter excludes it (the sum runs over the support of p_D), and KL_i = +inf where
 * only the verifier does.  In the streaming path that last case is recognised as long
 * as the drafter gives the token at least 3e-35 of the probability mass of its stretch
 * of 4096-8192 logits; below that the token counts as excluded by both.
 *
 * drafter_logits, verifier_logits: [B,P,V] bf16 (drafter_logits may be NULL
 * unless the mode is KL); tokens int32 [B,P]; mask_flags uint8 [B,P];
 * out_tokens int32 [B,P] (may alias tokens); out_mask uint8 [B,P]; out_score
 * fp32 [B,P], nullable.  The streaming path needs V % 8 == 0 and 16-byte
 * aligned logits; otherwise a slower element-wise path is taken.
 * Supported: P <= 8192; V < 2^31 / 2.
 * Errors: DD_ERR_INVALID_ARG (null required pointer, B/P/V <= 0, k < 0, unknown
 * mode or flag bit, tau NaN), DD_ERR_UNSUPPORTED (P too large), DD_ERR_CUDA.
 */
int dd_verify(const void *drafter_logits, const void *verifier_logits,
              const int32_t *tokens, const uint8_t *mask_flags,
              int mode, float tau, int k, uint64_t seed,
              int32_t *out_tokens, uint8_t *out_mask, float *out_score,
              int B, int P, int V, void *stream);

/*
 * Unmask(p, x): one confidence-based unmasking step of a masked diffusion
 * model, the operation the drafter applies K times per cycle (Algorithm 1,
 * drafting phase; Section 2.1; Section 2.3 for the threshold rule versus a
 * fixed number per step).  For every position with mask_flags == 1 (currently
 * [MASK]): a_i = argmax_x logits[b,i,x] (lowest index), c_i = softmax(logits[b,i,:])(a_i).
 * The position is unmasked iff c_i >= tau, or it is one of the k most confident
 * masked positions of its sequence (ties to the lower i).  tau = +infinity
 * unmasks exactly min(k, masked) positions per sequence; k = 1 guarantees
 * progress under a threshold; k = 0 leaves the threshold alone.
 *   out_tokens[b,i] = a_i if unmasked, else tokens[b,i] (the caller's [MASK] id)
 *   out_mask[b,i]   = 1 if the position stays masked, else 0
 *   out_conf[b,i]   = c_i (nullable)
 * Positions with mask_flags == 0 pass through (out_tokens = tokens, out_mask = 0,
 * out_conf = 0) and their logits are never read.  Shapes, supported sizes,
 * scratch and errors as for dd_verify, whose confidence rule (Eq. 7) this is,
 * applied to one logits tensor: the same kernel launch.
 */
int dd_unmask(const void *logits, const int32_t *tokens, const uint8_t *mask_flags,
              float tau, int k, int32_t *out_tokens, uint8_t *out_mask, float *out_conf,
              int B, int P, int V, void *stream);

/*
 * The language-model heads fused with the verification algorithm (Algorithm 1, verification
 * phase: p_V(. | x^D) is computed at every position and handed to A(p_D, p_V, x^D); Section 3.1).
 * Instead of logits the caller passes last hidden states and output embeddings:
 *     verifier logits[b,i,x] = sum_j verifier_hidden[b,i,j] * verifier_weight[x,j]
 *     drafter  logits[b,i,x] = sum_j drafter_hidden[b,i,j]  * drafter_weight[x,j]     (DD_MODE_KL only)
 * (fp32 accumulation of bf16 products on the tensor cores, never rounded to bf16, never stored), and
 * the call gives what dd_verify gives on those logits, in every mode and with DD_FLAG_PROBABILISTIC /
 * DD_FLAG_EMIT_DRAFTER as there.  DD_MODE_TRUST and DD_MODE_CONF need the verifier only: the drafter's
 * pair is not read and may be NULL.  DD_MODE_KL (Eq. 4-5) needs both pairs (DD_ERR_INVALID_ARG if one
 * is NULL); the drafter's distribution is then the one its head gives on the same positions.
 * verifier_hidden, drafter_hidden: [B,P,K] bf16; verifier_weight, drafter_weight: [V,K] bf16 (row x =
 * output embedding of token x); all contiguous, K innermost, 16-byte aligned, the same K for both
 * models.  The other arguments, outputs, scratch and errors are dd_verify's.  The hidden states of
 * positions with mask_flags == 0 are read (they share tiles with their neighbours) but nothing is
 * computed from them.  Two kernels per call, in stream order: the products with their per-tile
 * reductions, then a small one that combines the tiles of every row and decides the sequences.
 * Supported: K a multiple of 64; any V >= 1; P <= 8192.
 */
int dd_lm_head_verify(const void *drafter_hidden, const void *drafter_weight,
                      const void *verifier_hidden, const void *verifier_weight,
                      const int32_t *tokens, const uint8_t *mask_flags,
                      int mode, float tau, int k, uint64_t seed,
                      int32_t *out_tokens, uint8_t *out_mask, float *out_score,
                      int B, int P, int K, int V, void *stream);

/* `layout` argument of dd_block_attention. */
enum {
    DD_LAYOUT_BHND = 0, /* q, out [B,H,Nq,D]; k, v [B,H,Nkv,D]                     */
    DD_LAYOUT_BNHD = 1  /* q, out [B,Nq,H,D]; k, v [B,Nkv,H,D] (heads interleaved) */
};

/*
 * Attention of a block of queries over cached keys and values (Section 2.2,
 * Eq. 3 as written: the queries of the positions being computed against the
 * stored K and V of the whole context; the shape of the drafter's step with a
 * block-wise KV cache, Section 2.3).  No mask among the valid keys:
 *     out[b,h,i,:] = sum_{j < n_b} softmax_j(scale * q[b,h,i,:] . k[b,h,j,:]) v[b,h,j,:]
 * for i in [0,Nq), where n_b = Nkv if kv_len is NULL, else kv_len[b] clamped to
 * [0,Nkv] (keys at and beyond n_b are padding and never contribute).  A
 * sequence with n_b = 0 gets out = 0.  dd_bidir_attention is the case
 * Nq = Nkv, kv_len = NULL, DD_LAYOUT_BHND, and runs the same kernel.
 * q, k, v, out: bf16 in the given layout, D innermost, contiguous, 16-byte
 * aligned, out not overlapping the inputs; kv_len: int32 [B] DEVICE pointer or
 * NULL, read by the kernel when it runs.
 * Supported and errors: as dd_bidir_attention, with Nq, Nkv >= 1;
 * DD_ERR_INVALID_ARG for an unknown layout.
 */
int dd_block_attention(const void *q, const void *k, const void *v, void *out,
                       int B, int H, int Nq, int Nkv, int D,
                       const int32_t *kv_len, int layout, float scale, void *stream);

/*
 * Host-buffer forms of dd_bidir_attention and dd_verify (same definitions, same errors).
 * Every pointer is a HOST pointer.  The call enqueues, on `stream`, the
 * host-to-device copies into library-owned staging memory, the kernel, and the
 * device-to-host copies of the outputs; the outputs are valid once the stream
 * has been synchronised by the caller.
 */
int dd_bidir_attention_host(const void *q, const void *k, const void *v, void *out,
                            int B, int H, int N, int D, float scale, void *stream);
int dd_verify_host(const void *drafter_logits, const void *verifier_logits,
                   const int32_t *tokens, const uint8_t *mask_flags,
                   int mode, float tau, int k, uint64_t seed,
                   int32_t *out_tokens, uint8_t *out_mask, float *out_score,
                   int B, int P, int V, void *stream);

/*
 * dd_verify for callers that must not allocate device memory (the paper has no
 * counterpart to this entry point; it is the same computation as dd_verify, with
 * the same arguments, outputs and errors).  Meant for code that runs inside a
 * fixed memory budget, that may not trigger the device-wide synchronisation of
 * cudaMalloc/cudaFree, or that does not own the allocator of its process: this
 * call performs no cudaMalloc, cudaFree or other allocating routine.  Its scratch
 * (chunk partials, row results, completion counters, and a health word of its
 * own that dd_verify_status reads as well) is a fixed array of about 2.1 MB
 * inside the library, held by every GPU that loads the library until the
 * process exits.
 * Limits: B*P <= 4096 and B*P*ceil(V/8192) <= 65536; larger problems return
 * DD_ERR_UNSUPPORTED and launch nothing.
 * The first call on each device looks up the array's device address; make that
 * first call outside any stream capture.  All calls on a device share the one
 * array: each call clears the counters it needs on `stream` before its kernel,
 * and two calls that may overlap on the GPU (different streams without ordering)
 * race on the scratch and give undefined results.
 */
int dd_verify_static(const void *drafter_logits, const void *verifier_logits,
                     const int32_t *tokens, const uint8_t *mask_flags,
                     int mode, float tau, int k, uint64_t seed,
                     int32_t *out_tokens, uint8_t *out_mask, float *out_score,
                     int B, int P, int V, void *stream);

/*
 * Test hook: caps the number of CTAs the streaming kernel of dd_verify / dd_unmask /
 * dd_verify_static launches (0 = no cap, one CTA per SM).  Outputs, scores included, are
 * bit-identical for every cap: which warp computes a (row, chunk) unit never changes the
 * unit's partial result, and rows are folded from their partials in a fixed order (Eq. 5 and
 * Eq. 7 are sums over the vocabulary; only the order of their evaluation is at stake).
 * Process-wide.  Returns DD_OK, or DD_ERR_INVALID_ARG for a negative cap.
 */
int dd_debug_set_max_ctas(int max_ctas);

/* Bytes of per-device scratch dd_verify needs for this shape (informational). */
size_t dd_verify_workspace_bytes(int B, int P, int V);

/*
 * Health of the kernels.  Every device-side wait is bounded; a wait that expires records a code in
 * a per-device health word (one for the attention kernel, one for dd_verify / dd_unmask /
 * dd_verify_static) and the affected outputs of that launch are undefined.  The word is sticky:
 *   - the code is also written to a host copy, so the NEXT call of an entry point of that kernel
 *     on the device returns DD_ERR_TIMEOUT without launching anything and without synchronising
 *     (dd_verify_static consults the host copy only if another entry point has created it);
 *   - dd_attention_status() / dd_verify_status() synchronise the device and read the word itself:
 *     DD_OK, DD_ERR_TIMEOUT (dd_last_cuda_error() names the code) or DD_ERR_CUDA;
 *   - dd_clear_status() synchronises the device and re-arms both words (the scratch stays
 *     allocated); dd_release() frees everything.
 */
int dd_attention_status(void);
int dd_verify_status(void);
int dd_clear_status(void);

/*
 * Test hook for the above: launches, on `stream`, a one-thread kernel that waits on a barrier
 * nothing completes, gives up after a few hundred polls (microseconds) and records the expiry in
 * the health word of the attention kernel (which = 0) or of dd_verify (which = 1) exactly as those
 * kernels would.  It stalls nothing and faults nothing.  DD_ERR_INVALID_ARG for another `which`.
 */
int dd_debug_expire_wait(int which, void *stream);

/* Number of kernels launched by this library in this process (all devices). */
uint64_t dd_launch_count(void);

/* Frees the current device's scratch.  The next call re-allocates it. */
int dd_release(void);

/* Text of a dd_status; the last CUDA error text recorded by this thread. */
const char *dd_status_string(int status);
const char *dd_last_cuda_error(void);

/* Library version: major * 10000 + minor * 100 + patch. */
int dd_version(void);

#ifdef __cplusplus
}
#endif
#endif /* DUALDIFF_H_ */
