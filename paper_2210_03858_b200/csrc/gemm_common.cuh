// Pieces shared by the tcgen05 kernels: CTA geometry, the mbarrier control block with
// time-limited waits, and the host helpers that build TMA descriptors.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "common.h"
#include "ptx.cuh"

namespace bcq {

constexpr int kThreads = 320;       // warp 0: TMA, warp 1: UMMA + TMEM, warps 2..9: workers
constexpr int kWorkerWarp0 = 2;
constexpr int kWorkerWarps = 8;
constexpr int kWorkers = kWorkerWarps * 32;
constexpr int kBlockM = 128;
constexpr int kBlockK = 64;
constexpr uint32_t kABytes = kBlockM * kBlockK * 2;  // one 16-bit A tile: 16 KiB
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

struct Ctl {
    uint32_t full;    // + 8*s : TMA bytes of the stage have landed
    uint32_t aready;  // + 8*s : worker-written tiles of the stage are complete
    uint32_t empty;   // + 8*s : the UMMAs that read the stage have completed
    uint32_t accum;   // accumulator complete
    uint32_t spare;   // only used when giving up
    volatile int* abort_flag;  // CTA-wide "somebody timed out"
    int* device_flag;          // library-wide flag in global memory
};

// Waits for the phase with the given parity.  Gives up after kWaitLimitNs (or as soon as another
// thread of the CTA gave up), records `code` in the device flag and returns false.
// Between polls the warp sleeps for `nap_ns`: a warp that spins on try_wait keeps winning issue
// slots from the warps that do the work (measured: about half of all instructions a kernel issued
// were polls), while a sleeping warp costs nothing; the price is up to nap_ns of extra latency
// when the phase completes, so waits on the critical path take a short nap and long, off-path
// waits (an epilogue waiting for a whole tile) a longer one.
#ifndef BCQ_NAP_NS
#define BCQ_NAP_NS 128u
#endif
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, const Ctl& ctl, int code,
                                         uint32_t nap_ns = BCQ_NAP_NS) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = ptx::globaltimer_ns();
    uint32_t spins = 0;
    while (true) {
        if (ptx::mbar_try_wait(bar, parity)) return true;
        __nanosleep(nap_ns);
        if ((++spins & 7u) == 0u) {
            if (*ctl.abort_flag) return false;
            if (ptx::globaltimer_ns() - t0 > kWaitLimitNs) {
                *ctl.abort_flag = 1;
                atomicExch(ctl.device_flag, code);
                return false;
            }
        }
    }
}

// The same for a whole (converged) warp: lane 0 polls, the outcome is broadcast, and the warp
// barrier orders the other lanes' later reads after lane 0's acquire.  Keeps the number of threads
// polling shared-memory barriers small.
__device__ __forceinline__ bool warp_wait_bar(uint32_t bar, uint32_t parity, const Ctl& ctl, int code) {
    int ok = 1;
    if ((threadIdx.x & 31) == 0) ok = wait_bar(bar, parity, ctl, code) ? 1 : 0;
    ok = __shfl_sync(0xffffffffu, ok, 0);
    __syncwarp();
    return ok != 0;
}

template <int TN>
struct TmemCols {
    static constexpr uint32_t value = TN < 32 ? 32 : TN;
};

// ------------------------------------------------------------------------------------------
// host helpers
// ------------------------------------------------------------------------------------------

// Raises a kernel's dynamic shared memory limit, once per (kernel, device) (the attribute call is
// not free, and callers that launch eagerly would pay it on every call).  Defined in api.cu.
bcq_status ensure_dynamic_smem_impl(const void* kern, size_t bytes);
template <typename Kern>
inline bcq_status ensure_dynamic_smem(Kern kern, size_t bytes) {
    return ensure_dynamic_smem_impl(reinterpret_cast<const void*>(kern), bytes);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// 16-bit matrix [outer][pitch_elems] with `inner` valid elements per row; box = 64 x box_outer,
// 128-byte swizzle, out-of-range elements read as zero.
inline bcq_status make_tmap_16bit(CUtensorMap* m, const void* base, int is_fp16, int inner, int outer,
                                  size_t pitch_elems, int box_outer) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) {
        set_last_cuda_error((int)cudaErrorNotSupported);
        return BCQ_ERR_CUDA;
    }
    cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
    cuuint64_t strides[1] = {(cuuint64_t)pitch_elems * 2};
    cuuint32_t box[2] = {64u, (cuuint32_t)box_outer};
    cuuint32_t estr[2] = {1u, 1u};
    CUresult r = fn(m, is_fp16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                    const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_last_cuda_error((int)cudaErrorInvalidValue);
        return BCQ_ERR_CUDA;
    }
    return BCQ_OK;
}

// bf16 output [outer][pitch_elems] with `inner` valid elements per row, written in boxes of
// 32 x 16 elements whose 64-byte rows are 64-byte swizzled in shared memory.
inline bcq_status make_tmap_out_bf16(CUtensorMap* m, void* base, int inner, int outer, size_t pitch_elems) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) {
        set_last_cuda_error((int)cudaErrorNotSupported);
        return BCQ_ERR_CUDA;
    }
    cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
    cuuint64_t strides[1] = {(cuuint64_t)pitch_elems * 2};
    cuuint32_t box[2] = {32u, 16u};
    cuuint32_t estr[2] = {1u, 1u};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_last_cuda_error((int)cudaErrorInvalidValue);
        return BCQ_ERR_CUDA;
    }
    return BCQ_OK;
}

// The packed planes uint32 [q][d_out][pitch] as a 3-D tensor; box = 4 words (128 weights) x
// box_rows x q, no swizzle; rows or words out of range read as zero.
inline bcq_status make_tmap_bits(CUtensorMap* m, const uint32_t* bits, int d_out, int pitch_words, int q,
                                 int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) {
        set_last_cuda_error((int)cudaErrorNotSupported);
        return BCQ_ERR_CUDA;
    }
    cuuint64_t dims[3] = {(cuuint64_t)pitch_words, (cuuint64_t)d_out, (cuuint64_t)q};
    cuuint64_t strides[2] = {(cuuint64_t)pitch_words * 4, (cuuint64_t)pitch_words * 4 * (cuuint64_t)d_out};
    cuuint32_t box[3] = {4u, (cuuint32_t)box_rows, (cuuint32_t)q};
    cuuint32_t estr[3] = {1u, 1u, 1u};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, const_cast<uint32_t*>(bits), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_last_cuda_error((int)cudaErrorInvalidValue);
        return BCQ_ERR_CUDA;
    }
    return BCQ_OK;
}

inline bcq_status check_act(const void* ptr, size_t ld, int cols) {
    if (ptr == nullptr) return BCQ_ERR_NULL;
    if (ld < (size_t)cols) return BCQ_ERR_SHAPE;
    if (!aligned16(ptr) || (ld % 8) != 0) return BCQ_ERR_ALIGN;
    return BCQ_OK;
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// per-TU device timeout flags
bcq_status expand_timeout_flag(int* flag_out, int reset);
bcq_status dalpha_timeout_flag(int* flag_out, int reset);
bcq_status decode_timeout_flag(int* flag_out, int reset);

// workspace sizes (defined next to the kernels that use them)
size_t fwd_workspace_bytes(int d_out, int d_in, int q, int g, int n);
size_t decode_workspace_bytes(int d_out, int d_in, int q, int g, int n);
size_t bwd_x_workspace_bytes(int d_out, int d_in, int q, int g, int n);
size_t bwd_alpha_workspace_bytes(int d_out, int d_in, int q, int g, int n);
size_t decode_packed_workspace_bytes(int d_out, int d_in, int q, int g, int n);

}  // namespace bcq
