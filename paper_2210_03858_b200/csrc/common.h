// Host-side helpers shared by the translation units of the library (no device code here).
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/bcq.h"

#define BCQ_MAX_Q 8
#define BCQ_MAX_QUANT_G 32768

namespace bcq {

// cudaError_t of the last failing CUDA call on this thread (read by bcq_last_cuda_error()).
void set_last_cuda_error(int e);

// Called once per kernel launch (bcq_kernel_launches()).
void count_launch();

inline bcq_status cuda_fail(cudaError_t e) {
    set_last_cuda_error((int)e);
    return BCQ_ERR_CUDA;
}

#define BCQ_CUDA_TRY(expr)                                  \
    do {                                                    \
        cudaError_t e__ = (expr);                           \
        if (e__ != cudaSuccess) return bcq::cuda_fail(e__); \
    } while (0)

// Shape rules shared by every entry point (see include/bcq.h).
inline bcq_status check_shape(int d_out, int d_in, int q, int g) {
    if (d_out < 1 || d_in < 1 || q < 1 || g < 1 || g > d_in) return BCQ_ERR_SHAPE;
    if (q > BCQ_MAX_Q) return BCQ_ERR_UNSUPPORTED;
    if (g != d_in && (g % 32) != 0) return BCQ_ERR_UNSUPPORTED;
    return BCQ_OK;
}

// Number of SMs of the current device (148 on a B200; that value is also the answer when no device
// can be asked, e.g. for size queries on a machine without a GPU).
inline int sm_count() {
    static int cached = 0;
    if (cached == 0) {
        int dev = 0, n = 0;
        if (cudaGetDevice(&dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0)
            cached = n;
        else
            return 148;  // not cached, so a later call with a device present asks again
    }
    return cached;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

}  // namespace bcq
