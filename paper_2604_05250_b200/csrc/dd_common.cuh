// Shared host-side plumbing of the library: status codes, per-device scratch,
// CUDA error capture, launch counting.  No kernel arithmetic lives here.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/dualdiff.h"

namespace dd {

// Per-device scratch owned by the library.
struct DeviceCtx {
    void *verify_ws = nullptr;      // dd_verify chunk partials and row results
    size_t verify_ws_bytes = 0;
    void *verify_cnt = nullptr;     // dd_verify completion counters: all zero between launches
    size_t verify_cnt_bytes = 0;
    void *staging = nullptr;        // device copies of host buffers (the *_host calls)
    size_t staging_bytes = 0;
    unsigned int *attn_status = nullptr;  // one word: first expired wait of the attention kernel
    // Host copy of the two health words (pinned, mapped): [0] attention, [1] verify.  A kernel that
    // records an expired wait writes the code here as well, so the next call sees it without a
    // device synchronisation.
    volatile unsigned int *mirror = nullptr;
    unsigned int *mirror_dev = nullptr;   // the same two words as the kernels address them
};

// Returns the context of the current device (creating it on first use), or
// nullptr after recording a CUDA error.
DeviceCtx *current_ctx(int *device_out = nullptr);

// Allocates the host copy of the health words on first use (pinned host memory, no device memory).
int ensure_mirror(DeviceCtx *ctx);

// DD_ERR_TIMEOUT (with error text) if the host copy shows that kernel `which` (0 attention,
// 1 verify) has recorded an expired wait on this device; DD_OK otherwise.
int check_mirror(const DeviceCtx *ctx, int which);

// Grows (never shrinks) a scratch buffer; new memory is zero-filled.
int ensure_bytes(void **ptr, size_t *have, size_t need);

// Records a CUDA error text for dd_last_cuda_error() and returns DD_ERR_CUDA.
int cuda_fail(cudaError_t e, const char *where);

// Sets the text dd_last_cuda_error() returns.
void set_error_text(const char *text);

void count_launch(unsigned n = 1);

#define DD_CUDA_TRY(expr)                                         \
    do {                                                          \
        cudaError_t _e = (expr);                                  \
        if (_e != cudaSuccess) return ::dd::cuda_fail(_e, #expr); \
    } while (0)

}  // namespace dd
