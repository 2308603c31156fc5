// The AlphaTuning update: AdamW on the trainable scales, and the scale-only checkpoint.
//
// Only alpha is trained (Section "AlphaTuning: Efficient Fine-Tuning of Quantized Models"; the
// experiments train alpha_1 alone), with AdamW under a linear-decay learning rate (Appendix
// "Experimental Details") and the gradient of Eq. 4, which carries the empirical factor 1/g_L.
// The scales, their gradients and the two moments of ALL linears of a model live in flat fp32
// arrays with the same indexing, so one launch updates every trained scale: the trained part is
// described by segments (one per trained plane of each linear: planes are the outermost index of
// alpha[q][d_out][G], so a plane is one contiguous run), each with its own gradient scale.
// The same segments drive the checkpoint: the paper's per-task checkpoint is just the trained
// scales, gathered into one compact array.
#include "common.h"

namespace {

struct Segments {
    int nseg;
    const long long* begin;   // [nseg]   first element of the segment in the flat arrays
    const long long* prefix;  // [nseg+1] running count of elements before each segment
    const float* scale;       // [nseg]   gradient scale of the segment, or null (1)
};

// Segment that holds compact index e (prefix[s] <= e < prefix[s + 1]).
__device__ __forceinline__ int find_segment(const long long* __restrict__ prefix, int nseg, long long e) {
    int lo = 0, hi = nseg - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (__ldg(prefix + mid) <= e) lo = mid; else hi = mid - 1;
    }
    return lo;
}

struct AdamParams {
    float lr_wd_keep;   // 1 - lr * weight_decay
    float beta1, beta2, eps;
    float om_beta1, om_beta2;  // 1 - beta, formed in fp64 on the host (1 - 0.999f in fp32 is off by 1e-5)
    float step_size;    // lr / (1 - beta1^t)
    float inv_sqrt_bc2; // 1 / sqrt(1 - beta2^t)
    float grad_scale;   // applied on top of the per-segment scale
};

__global__ void __launch_bounds__(256)
alpha_adamw_kernel(long long count, Segments sg, AdamParams h, float* __restrict__ alpha,
                   const float* __restrict__ grad, float* __restrict__ m, float* __restrict__ v) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < count; e += stride) {
        long long idx = e;
        float gs = h.grad_scale;
        if (sg.nseg > 0) {
            const int s = find_segment(sg.prefix, sg.nseg, e);
            idx = __ldg(sg.begin + s) + (e - __ldg(sg.prefix + s));
            if (sg.scale != nullptr) gs *= __ldg(sg.scale + s);
        }
        const float g = gs * grad[idx];
        const float mm = h.beta1 * m[idx] + h.om_beta1 * g;
        const float vv = h.beta2 * v[idx] + h.om_beta2 * g * g;
        const float denom = sqrtf(vv) * h.inv_sqrt_bc2 + h.eps;
        alpha[idx] = alpha[idx] * h.lr_wd_keep - h.step_size * (mm / denom);
        m[idx] = mm;
        v[idx] = vv;
    }
}

// to_compact != 0: compact[e] = flat[...]; else flat[...] = compact[e].
__global__ void __launch_bounds__(256)
alpha_gather_kernel(long long count, Segments sg, int to_compact, float* __restrict__ flat,
                    float* __restrict__ compact) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < count; e += stride) {
        const int s = find_segment(sg.prefix, sg.nseg, e);
        const long long idx = __ldg(sg.begin + s) + (e - __ldg(sg.prefix + s));
        if (to_compact) compact[e] = flat[idx]; else flat[idx] = compact[e];
    }
}

unsigned grid_for(long long count) {
    long long blocks = (count + 255) / 256;
    const long long cap = (long long)bcq::sm_count() * 8;
    if (blocks > cap) blocks = cap;
    return (unsigned)(blocks < 1 ? 1 : blocks);
}

}  // namespace

extern "C" float bcq_lr_linear_decay(float lr0, long long step, long long warmup_steps, long long total_steps) {
    if (total_steps <= 0 || step < 0) return 0.0f;
    if (warmup_steps > 0 && step < warmup_steps) return (float)((double)lr0 * (double)step / (double)warmup_steps);
    if (step >= total_steps) return 0.0f;
    const long long w = warmup_steps > 0 ? warmup_steps : 0;
    return (float)((double)lr0 * (double)(total_steps - step) / (double)(total_steps - w));
}

extern "C" bcq_status bcq_alpha_adamw(long long count, int nseg, const long long* seg_begin,
                                      const long long* seg_prefix, const float* seg_scale, float* alpha,
                                      const float* dalpha, float* m, float* v, long long step, float lr,
                                      float beta1, float beta2, float eps, float weight_decay, float grad_scale,
                                      void* stream) {
    if (count < 0 || nseg < 0 || step < 1) return BCQ_ERR_SHAPE;
    if (!(beta1 >= 0.0f && beta1 < 1.0f && beta2 >= 0.0f && beta2 < 1.0f)) return BCQ_ERR_SHAPE;
    if (!alpha || !dalpha || !m || !v) return BCQ_ERR_NULL;
    if (nseg > 0 && (!seg_begin || !seg_prefix)) return BCQ_ERR_NULL;
    if (count == 0) return BCQ_OK;
    Segments sg{nseg, seg_begin, seg_prefix, seg_scale};
    AdamParams h;
    h.lr_wd_keep = 1.0f - lr * weight_decay;
    h.beta1 = beta1; h.beta2 = beta2; h.eps = eps;
    h.om_beta1 = (float)(1.0 - (double)beta1);
    h.om_beta2 = (float)(1.0 - (double)beta2);
    h.step_size = (float)((double)lr / (1.0 - pow((double)beta1, (double)step)));
    h.inv_sqrt_bc2 = (float)(1.0 / sqrt(1.0 - pow((double)beta2, (double)step)));
    h.grad_scale = grad_scale;
    alpha_adamw_kernel<<<grid_for(count), 256, 0, (cudaStream_t)stream>>>(count, sg, h, alpha, dalpha, m, v);
    bcq::count_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return bcq::cuda_fail(e);
    return BCQ_OK;
}

static bcq_status gather_common(long long count, int nseg, const long long* seg_begin, const long long* seg_prefix,
                                int to_compact, float* flat, float* compact, void* stream) {
    if (count < 0 || nseg < 1) return BCQ_ERR_SHAPE;
    if (!seg_begin || !seg_prefix || !flat || !compact) return BCQ_ERR_NULL;
    if (count == 0) return BCQ_OK;
    Segments sg{nseg, seg_begin, seg_prefix, nullptr};
    alpha_gather_kernel<<<grid_for(count), 256, 0, (cudaStream_t)stream>>>(count, sg, to_compact, flat, compact);
    bcq::count_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return bcq::cuda_fail(e);
    return BCQ_OK;
}

extern "C" bcq_status bcq_alpha_pack(long long count, int nseg, const long long* seg_begin,
                                     const long long* seg_prefix, const float* alpha_flat, float* packed,
                                     void* stream) {
    return gather_common(count, nseg, seg_begin, seg_prefix, 1, const_cast<float*>(alpha_flat), packed, stream);
}

extern "C" bcq_status bcq_alpha_unpack(long long count, int nseg, const long long* seg_begin,
                                       const long long* seg_prefix, const float* packed, float* alpha_flat,
                                       void* stream) {
    return gather_common(count, nseg, seg_begin, seg_prefix, 0, alpha_flat, const_cast<float*>(packed), stream);
}
