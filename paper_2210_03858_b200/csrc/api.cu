// Host-only entry points: size helpers of the container format, status strings, error state.
#include <map>
#include <mutex>
#include <utility>

#include "gemm_common.cuh"

namespace bcq {
static thread_local int t_last_cuda_error = 0;
static thread_local unsigned long long t_launches = 0;
void set_last_cuda_error(int e) { t_last_cuda_error = e; }
void count_launch() { ++t_launches; }

bcq_status ensure_dynamic_smem_impl(const void* kern, size_t bytes) {
    static std::mutex lock;
    static std::map<std::pair<const void*, int>, size_t> configured;  // (kernel, device) -> bytes granted
    int dev = 0;
    BCQ_CUDA_TRY(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> guard(lock);
    size_t& have = configured[std::make_pair(kern, dev)];
    if (have < bytes) {
        BCQ_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes));
        have = bytes;
    }
    return BCQ_OK;
}
}  // namespace bcq

extern "C" size_t bcq_pitch_words(int d_in) {
    return d_in < 1 ? 0 : 4 * (((size_t)d_in + 127) / 128);
}

extern "C" size_t bcq_bits_bytes(int d_out, int d_in, int q) {
    if (d_out < 1 || q < 1) return 0;
    return (size_t)q * (size_t)d_out * bcq_pitch_words(d_in) * sizeof(uint32_t);
}

extern "C" size_t bcq_num_groups(int d_in, int g) {
    return (g < 1 || d_in < 1) ? 0 : ((size_t)d_in + (size_t)g - 1) / (size_t)g;
}

extern "C" size_t bcq_alpha_count(int d_out, int d_in, int q, int g) {
    if (d_out < 1 || q < 1) return 0;
    return (size_t)q * (size_t)d_out * bcq_num_groups(d_in, g);
}

extern "C" size_t bcq_payload_bits(int d_out, int d_in, int q, int g) {
    if (d_out < 1 || d_in < 1 || q < 1 || g < 1) return 0;
    return (size_t)q * (size_t)d_out * (size_t)d_in + 32 * bcq_alpha_count(d_out, d_in, q, g);
}

extern "C" const char* bcq_status_string(int status) {
    switch (status) {
        case BCQ_OK: return "ok";
        case BCQ_ERR_NULL: return "a required pointer is NULL";
        case BCQ_ERR_SHAPE: return "a size or pitch is out of range";
        case BCQ_ERR_ALIGN: return "a pointer or pitch is not aligned as required";
        case BCQ_ERR_UNSUPPORTED: return "shape not covered by the kernels (q > 8, or g neither d_in nor a multiple of 32)";
        case BCQ_ERR_WORKSPACE: return "workspace smaller than bcq_workspace_bytes()";
        case BCQ_ERR_CUDA: return "a CUDA call failed (see bcq_last_cuda_error)";
        case BCQ_ERR_DEVICE_TIMEOUT: return "a kernel gave up on a bounded wait";
        default: return "unknown status";
    }
}

extern "C" unsigned long long bcq_kernel_launches(void) { return bcq::t_launches; }

extern "C" int bcq_last_cuda_error(void) { return bcq::t_last_cuda_error; }

extern "C" bcq_status bcq_device_timeout_flag(int* flag_out, int reset) {
    if (flag_out == nullptr) return BCQ_ERR_NULL;
    BCQ_CUDA_TRY(cudaDeviceSynchronize());
    int a = 0, b = 0, c = 0;
    bcq_status st = bcq::expand_timeout_flag(&a, reset);
    if (st != BCQ_OK) return st;
    st = bcq::dalpha_timeout_flag(&b, reset);
    if (st != BCQ_OK) return st;
    st = bcq::decode_timeout_flag(&c, reset);
    if (st != BCQ_OK) return st;
    *flag_out = a != 0 ? a : (b != 0 ? b : c);
    return BCQ_OK;
}

extern "C" bcq_status bcq_check_device(void) {
    int flag = 0;
    const bcq_status st = bcq_device_timeout_flag(&flag, 0);
    if (st != BCQ_OK) return st;
    return flag != 0 ? BCQ_ERR_DEVICE_TIMEOUT : BCQ_OK;
}

extern "C" size_t bcq_workspace_bytes(int op, int d_out, int d_in, int q, int g, int n) {
    if (bcq::check_shape(d_out, d_in, q, g) != BCQ_OK) return 0;
    if (op != BCQ_OP_QUANTIZE && n < 1) return 0;
    switch (op) {
        case BCQ_OP_FWD: return bcq::fwd_workspace_bytes(d_out, d_in, q, g, n);
        case BCQ_OP_DECODE: return n > 16 ? 0 : bcq::decode_workspace_bytes(d_out, d_in, q, g, n);
        case BCQ_OP_BWD_X: return bcq::bwd_x_workspace_bytes(d_out, d_in, q, g, n);
        case BCQ_OP_BWD_ALPHA: return bcq::bwd_alpha_workspace_bytes(d_out, d_in, q, g, n);
        case BCQ_OP_DECODE_PACKED: return n > 16 ? 0 : bcq::decode_packed_workspace_bytes(d_out, d_in, q, g, n);
        default: return 0;
    }
}
