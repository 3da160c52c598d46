// Host-side plumbing: per-device scratch, error text, launch counter, and the
// host-buffer forms of the two entry points (copies + the device entry point).
#include <atomic>
#include <cstdio>
#include <cstring>
#include <mutex>

#include "dd_common.cuh"

namespace dd {

namespace {
constexpr int kMaxDevices = 64;
DeviceCtx g_ctx[kMaxDevices];
bool g_ctx_live[kMaxDevices] = {};
std::mutex g_mu;
std::atomic<uint64_t> g_launches{0};
thread_local char g_err[256] = "";
}  // namespace

int cuda_fail(cudaError_t e, const char *where)
{
    snprintf(g_err, sizeof g_err, "%s: %s (%s)", where, cudaGetErrorName(e), cudaGetErrorString(e));
    (void)cudaGetLastError();  // clear the sticky-free error state
    return DD_ERR_CUDA;
}

void set_error_text(const char *text) { snprintf(g_err, sizeof g_err, "%s", text); }

void count_launch(unsigned n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

DeviceCtx *current_ctx(int *device_out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        cuda_fail(e == cudaSuccess ? cudaErrorInvalidDevice : e, "cudaGetDevice");
        return nullptr;
    }
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_ctx_live[dev]) {
        g_ctx[dev] = DeviceCtx();
        g_ctx_live[dev] = true;
    }
    if (device_out) *device_out = dev;
    return &g_ctx[dev];
}

int ensure_mirror(DeviceCtx *ctx)
{
    std::lock_guard<std::mutex> lock(g_mu);
    if (ctx->mirror) return DD_OK;
    void *host = nullptr, *dev = nullptr;
    DD_CUDA_TRY(cudaHostAlloc(&host, 64, cudaHostAllocMapped));
    memset(host, 0, 64);
    DD_CUDA_TRY(cudaHostGetDevicePointer(&dev, host, 0));
    ctx->mirror_dev = static_cast<unsigned int *>(dev);
    ctx->mirror = static_cast<volatile unsigned int *>(host);
    return DD_OK;
}

int check_mirror(const DeviceCtx *ctx, int which)
{
    if (!ctx->mirror) return DD_OK;
    const unsigned int word = ctx->mirror[which];
    if (word == 0) return DD_OK;
    snprintf(g_err, sizeof g_err, "%s kernel: a bounded wait expired earlier on this device (code 0x%08x); "
             "dd_clear_status() re-arms it", which == 0 ? "attention" : "verify", word);
    return DD_ERR_TIMEOUT;
}

int ensure_bytes(void **ptr, size_t *have, size_t need)
{
    if (need <= *have && *ptr) return DD_OK;
    if (*ptr) {
        DD_CUDA_TRY(cudaDeviceSynchronize());  // earlier launches may still use the old block
        DD_CUDA_TRY(cudaFree(*ptr));
        *ptr = nullptr;
        *have = 0;
    }
    size_t bytes = (need + 255) & ~size_t(255);
    DD_CUDA_TRY(cudaMalloc(ptr, bytes));
    DD_CUDA_TRY(cudaMemset(*ptr, 0, bytes));
    DD_CUDA_TRY(cudaDeviceSynchronize());
    *have = bytes;
    return DD_OK;
}

}  // namespace dd

using namespace dd;

extern "C" {

const char *dd_status_string(int status)
{
    switch (status) {
        case DD_OK: return "ok";
        case DD_ERR_INVALID_ARG: return "invalid argument";
        case DD_ERR_UNSUPPORTED: return "unsupported shape or alignment";
        case DD_ERR_CUDA: return "CUDA call failed";
        case DD_ERR_TIMEOUT: return "a bounded device-side wait expired";
        default: return "unknown status";
    }
}

const char *dd_last_cuda_error(void) { return g_err; }

int dd_version(void) { return 100; }

uint64_t dd_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int dd_release(void)
{
    DeviceCtx *ctx = current_ctx();
    if (!ctx) return DD_ERR_CUDA;
    DD_CUDA_TRY(cudaDeviceSynchronize());
    if (ctx->verify_ws) DD_CUDA_TRY(cudaFree(ctx->verify_ws));
    if (ctx->verify_cnt) DD_CUDA_TRY(cudaFree(ctx->verify_cnt));
    if (ctx->staging) DD_CUDA_TRY(cudaFree(ctx->staging));
    if (ctx->attn_status) DD_CUDA_TRY(cudaFree(ctx->attn_status));
    if (ctx->mirror) DD_CUDA_TRY(cudaFreeHost(const_cast<unsigned int *>(ctx->mirror)));
    *ctx = DeviceCtx();
    return DD_OK;
}

int dd_attention_status(void)
{
    DeviceCtx *ctx = current_ctx();
    if (!ctx) return DD_ERR_CUDA;
    if (!ctx->attn_status) return DD_OK;
    unsigned int word = 0;
    DD_CUDA_TRY(cudaDeviceSynchronize());
    DD_CUDA_TRY(cudaMemcpy(&word, ctx->attn_status, sizeof word, cudaMemcpyDeviceToHost));
    if (word != 0) {
        snprintf(g_err, sizeof g_err, "attention kernel: bounded wait expired, code 0x%08x", word);
        return DD_ERR_TIMEOUT;
    }
    return DD_OK;
}

// ---------------------------------------------------------------------------
// Host-buffer forms: stage through library-owned device memory on `stream`.

static size_t align256(size_t x) { return (x + 255) & ~size_t(255); }

int dd_bidir_attention_host(const void *q, const void *k, const void *v, void *out,
                            int B, int H, int N, int D, float scale, void *stream)
{
    if (!q || !k || !v || !out || B <= 0 || H <= 0 || N <= 0 || D <= 0) return DD_ERR_INVALID_ARG;
    DeviceCtx *ctx = current_ctx();
    if (!ctx) return DD_ERR_CUDA;
    const size_t bytes = (size_t)B * H * N * D * 2;
    const size_t slot = align256(bytes);
    int rc = ensure_bytes(&ctx->staging, &ctx->staging_bytes, 4 * slot);
    if (rc != DD_OK) return rc;
    char *base = (char *)ctx->staging;
    cudaStream_t s = (cudaStream_t)stream;
    DD_CUDA_TRY(cudaMemcpyAsync(base + 0 * slot, q, bytes, cudaMemcpyHostToDevice, s));
    DD_CUDA_TRY(cudaMemcpyAsync(base + 1 * slot, k, bytes, cudaMemcpyHostToDevice, s));
    DD_CUDA_TRY(cudaMemcpyAsync(base + 2 * slot, v, bytes, cudaMemcpyHostToDevice, s));
    rc = dd_bidir_attention(base, base + slot, base + 2 * slot, base + 3 * slot, B, H, N, D, scale, stream);
    if (rc != DD_OK) return rc;
    DD_CUDA_TRY(cudaMemcpyAsync(out, base + 3 * slot, bytes, cudaMemcpyDeviceToHost, s));
    return DD_OK;
}

int dd_verify_host(const void *drafter_logits, const void *verifier_logits,
                   const int32_t *tokens, const uint8_t *mask_flags,
                   int mode, float tau, int k, uint64_t seed,
                   int32_t *out_tokens, uint8_t *out_mask, float *out_score,
                   int B, int P, int V, void *stream)
{
    if (!verifier_logits || !tokens || !mask_flags || !out_tokens || !out_mask ||
        B <= 0 || P <= 0 || V <= 0)
        return DD_ERR_INVALID_ARG;
    if ((mode & 0xFF) == DD_MODE_KL && !drafter_logits) return DD_ERR_INVALID_ARG;
    DeviceCtx *ctx = current_ctx();
    if (!ctx) return DD_ERR_CUDA;
    const size_t bp = (size_t)B * P;
    const size_t logit_bytes = bp * V * 2;
    const size_t s_logit = align256(logit_bytes);
    const size_t s_i32 = align256(bp * 4), s_u8 = align256(bp);
    const bool need_drafter = (mode & 0xFF) == DD_MODE_KL;
    // layout: [verifier][drafter?][tokens][flags][out_tokens][out_mask][out_score]
    const size_t total = s_logit * (need_drafter ? 2 : 1) + 3 * s_i32 + 2 * s_u8;
    int rc = ensure_bytes(&ctx->staging, &ctx->staging_bytes, total);
    if (rc != DD_OK) return rc;
    char *p = (char *)ctx->staging;
    char *d_ver = p; p += s_logit;
    char *d_dra = nullptr;
    if (need_drafter) { d_dra = p; p += s_logit; }
    char *d_tok = p; p += s_i32;
    char *d_flag = p; p += s_u8;
    char *d_otok = p; p += s_i32;
    char *d_omask = p; p += s_u8;
    char *d_oscore = p;
    cudaStream_t s = (cudaStream_t)stream;
    DD_CUDA_TRY(cudaMemcpyAsync(d_ver, verifier_logits, logit_bytes, cudaMemcpyHostToDevice, s));
    if (need_drafter)
        DD_CUDA_TRY(cudaMemcpyAsync(d_dra, drafter_logits, logit_bytes, cudaMemcpyHostToDevice, s));
    DD_CUDA_TRY(cudaMemcpyAsync(d_tok, tokens, bp * 4, cudaMemcpyHostToDevice, s));
    DD_CUDA_TRY(cudaMemcpyAsync(d_flag, mask_flags, bp, cudaMemcpyHostToDevice, s));
    rc = dd_verify(d_dra, d_ver, (const int32_t *)d_tok, (const uint8_t *)d_flag, mode, tau, k, seed,
                   (int32_t *)d_otok, (uint8_t *)d_omask, (float *)d_oscore, B, P, V, stream);
    if (rc != DD_OK) return rc;
    DD_CUDA_TRY(cudaMemcpyAsync(out_tokens, d_otok, bp * 4, cudaMemcpyDeviceToHost, s));
    DD_CUDA_TRY(cudaMemcpyAsync(out_mask, d_omask, bp, cudaMemcpyDeviceToHost, s));
    if (out_score) DD_CUDA_TRY(cudaMemcpyAsync(out_score, d_oscore, bp * 4, cudaMemcpyDeviceToHost, s));
    return DD_OK;
}

}  // extern "C"
