// BCQ post-training quantizer (greedy and alternating) and the dequantize helper.
//
// One "team" of threads owns one (row, group) problem and keeps the group's residual in
// registers: thread `tid` of a team of NT threads holds elements e*NT + tid, e < EPT.  A team is
// one warp for g <= 1024 and a whole CTA above that.  Sums are fp64 and are reduced in a fixed
// tree order (shuffles inside a warp, then a sequential pass over the per-warp partials), so a
// result never depends on scheduling.  Sign bits leave the team as __ballot words, which is
// exactly the container format: 32 consecutive weights of one plane per 32-bit word.
//
// Appendix "Details on BCQ Format": Eq. ap:1-ap:3 (greedy), Eq. ap:4 and the following
// paragraph (alternating).
#include "common.h"

namespace {

struct QuantParams {
    int d_out, d_in, q, g, G, alt_iters;
    long long ldw;
    int pitch;
    const float* W;
    uint32_t* bits;
    float* alpha;
    double* sq_err;
    long long items;  // d_out * G
};

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Sum over the team.  TW == 1: the warp.  TW > 1: the CTA (all threads must call).
template <int TW>
__device__ __forceinline__ double team_sum(double v, double* scratch) {
    v = warp_sum(v);
    if (TW == 1) return v;
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    double t = 0.0;
#pragma unroll 1
    for (int w = 0; w < TW; ++w) t += scratch[w];
    return t;
}

// Sum of small non-negative counts over the team, as a double.  A warp adds them with one
// integer reduction (exact, like the fp64 tree: the values are integers far below 2^53).
template <int TW>
__device__ __forceinline__ double team_count(int v, double* scratch) {
    if (TW == 1) return (double)__reduce_add_sync(0xffffffffu, v);
    return team_sum<TW>((double)v, scratch);
}

template <int TW>
__device__ __forceinline__ void team_sync() {
    if (TW == 1)
        __syncwarp();
    else
        __syncthreads();
}

// Least-squares scales for fixed signs (Eq. ap:4): solve (B^T B) x = B^T w by Gaussian
// elimination with partial pivoting.  Every thread of the team runs the same arithmetic on the
// same numbers.  Products and differences are rounded separately (no fused multiply-add).
// Returns false (alpha untouched) when a pivot is below 1e-12 * m.
__device__ bool solve_ls(int q, double m, double (*A)[BCQ_MAX_Q + 1], float* alpha) {
    const double tiny = 1e-12 * m;
    for (int col = 0; col < q; ++col) {
        int piv = col;
        for (int r = col + 1; r < q; ++r)
            if (fabs(A[r][col]) > fabs(A[piv][col])) piv = r;
        if (fabs(A[piv][col]) < tiny) return false;
        if (piv != col)
            for (int l = 0; l <= q; ++l) {
                double tmp = A[col][l];
                A[col][l] = A[piv][l];
                A[piv][l] = tmp;
            }
        for (int r = col + 1; r < q; ++r) {
            const double f = __ddiv_rn(A[r][col], A[col][col]);
            for (int l = col; l <= q; ++l) A[r][l] = __dsub_rn(A[r][l], __dmul_rn(f, A[col][l]));
        }
    }
    double x[BCQ_MAX_Q];
    for (int r = q - 1; r >= 0; --r) {
        double s = A[r][q];
        for (int l = r + 1; l < q; ++l) s = __dsub_rn(s, __dmul_rn(A[r][l], x[l]));
        x[r] = __ddiv_rn(s, A[r][r]);
    }
    for (int i = 0; i < q; ++i) alpha[i] = (float)x[i];
    return true;
}

// The same elimination for a plane count known at compile time: every index is static, so the
// matrix stays in registers (the pivot row is found by value and swapped in by predicated moves).
// Same operations in the same order as solve_ls, hence the same result.
template <int Q>
__device__ __forceinline__ bool solve_ls_static(double m, double (&A)[Q][Q + 1], float (&alpha)[Q]) {
    const double tiny = 1e-12 * m;
#pragma unroll
    for (int col = 0; col < Q; ++col) {
        int piv = col;
        double best = fabs(A[col][col]);
#pragma unroll
        for (int r = col + 1; r < Q; ++r) {
            const double v = fabs(A[r][col]);
            if (v > best) { best = v; piv = r; }
        }
        if (best < tiny) return false;
#pragma unroll
        for (int r = col + 1; r < Q; ++r) {
            if (r == piv) {
#pragma unroll
                for (int l = 0; l <= Q; ++l) {
                    const double tmp = A[col][l];
                    A[col][l] = A[r][l];
                    A[r][l] = tmp;
                }
            }
        }
#pragma unroll
        for (int r = col + 1; r < Q; ++r) {
            const double f = __ddiv_rn(A[r][col], A[col][col]);
#pragma unroll
            for (int l = col; l <= Q; ++l) A[r][l] = __dsub_rn(A[r][l], __dmul_rn(f, A[col][l]));
        }
    }
    double x[Q];
#pragma unroll
    for (int r = Q - 1; r >= 0; --r) {
        double s = A[r][Q];
#pragma unroll
        for (int l = r + 1; l < Q; ++l) s = __dsub_rn(s, __dmul_rn(A[r][l], x[l]));
        x[r] = __ddiv_rn(s, A[r][r]);
    }
#pragma unroll
    for (int i = 0; i < Q; ++i) alpha[i] = (float)x[i];
    return true;
}

// QT > 0: the number of planes as a compile-time constant (alternating path for q = 2, 3, 4: the
// scales and the normal equations then live in registers); QT = 0: p.q at run time.
template <int EPT, int TW, bool ALT, int QT>
__global__ void __launch_bounds__(TW == 1 ? 128 : TW * 32)
quantize_kernel(const QuantParams p) {
    constexpr int QN = QT > 0 ? QT : BCQ_MAX_Q;
    const int q = QT > 0 ? QT : p.q;
    constexpr int NT = TW * 32;
    constexpr int TEAMS = (TW == 1) ? 4 : 1;
    __shared__ double red_scratch[32];
    __shared__ double level_smem[TEAMS][ALT ? (1 << BCQ_MAX_Q) : 1];

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int team = (TW == 1) ? warp : 0;
    const int tid = (TW == 1) ? lane : (int)threadIdx.x;  // index inside the team
    const int twarp = (TW == 1) ? 0 : warp;               // warp index inside the team
    double* levels = level_smem[team];

    const long long first = (long long)blockIdx.x * TEAMS + team;
    const long long stride = (long long)gridDim.x * TEAMS;
    // TW > 1 uses __syncthreads(): every team of the CTA is the CTA, so the trip count is uniform.
    for (long long item = first; item < p.items; item += stride) {
        const int j = (int)(item / p.G);
        const int c = (int)(item - (long long)j * p.G);
        const int k0 = c * p.g;
        const int m = min(p.g, p.d_in - k0);
        const double md = (double)m;
        const bool m_pow2 = (m & (m - 1)) == 0;
        const double inv_m = 1.0 / md;

        double r[EPT];
        float w[ALT ? EPT : 1];
        uint32_t code[ALT ? EPT : 1];
        const float* wrow = p.W + (long long)j * p.ldw + k0;
#pragma unroll
        for (int e = 0; e < EPT; ++e) {
            const int kl = e * NT + tid;
            const float v = (kl < m) ? __ldg(wrow + kl) : 0.0f;
            r[e] = (double)v;
            if (ALT) {
                w[e] = v;
                code[e] = 0u;
            }
        }

        float a[QN];
        // ---- greedy planes (q is a constant for QT > 0: the loops over planes unroll by themselves)
        for (int i = 0; i < q; ++i) {
            double local = 0.0;
#pragma unroll
            for (int e = 0; e < EPT; ++e)
                if (e * NT + tid < m) local += fabs(r[e]);
            const double S = team_sum<TW>(local, red_scratch);
            // a power-of-two group size divides exactly by multiplying with its reciprocal
            a[i] = (float)(m_pow2 ? __dmul_rn(S, inv_m) : __ddiv_rn(S, md));
            const double ad = (double)a[i];
            uint32_t* brow = p.bits + ((long long)i * p.d_out + j) * p.pitch + (k0 >> 5);
#pragma unroll
            for (int e = 0; e < EPT; ++e) {
                const int kl = e * NT + tid;
                const bool valid = kl < m;
                const bool pos = r[e] >= 0.0;
                const uint32_t word = __ballot_sync(0xffffffffu, valid && pos);
                if (!ALT && lane == 0 && (e * NT + twarp * 32) < m) brow[e * TW + twarp] = word;
                if (valid) r[e] = pos ? r[e] - ad : r[e] + ad;
                if (ALT && pos) code[e] |= (1u << i);
            }
        }

        if (ALT) {
            const int ncodes = 1 << q;
            for (int it = 0; it <= p.alt_iters; ++it) {
                // ---- least-squares alpha for the current signs
                double A[QN][QN + 1];
                for (int i = 0; i < q; ++i) {
                    double local = 0.0;
#pragma unroll
                    for (int e = 0; e < EPT; ++e)
                        if (e * NT + tid < m) local += ((code[e] >> i) & 1u) ? (double)w[e] : -(double)w[e];
                    A[i][q] = team_sum<TW>(local, red_scratch);
                    A[i][i] = md;
                    for (int l = i + 1; l < q; ++l) {
                        int cnt = 0;
#pragma unroll
                        for (int e = 0; e < EPT; ++e)
                            if (e * NT + tid < m) cnt += (int)(((code[e] >> i) ^ (code[e] >> l)) & 1u);
                        const double mism = team_count<TW>(cnt, red_scratch);
                        A[i][l] = md - 2.0 * mism;
                        A[l][i] = A[i][l];
                    }
                }
                if constexpr (QT > 0) solve_ls_static<QT>(md, A, a);
                else solve_ls(q, md, A, a);
                if (it == p.alt_iters) break;  // the last pass is the final refit only
                // ---- every weight moves to the nearest level; largest code wins ties
                team_sync<TW>();
                for (int s = tid; s < ncodes; s += NT) {
                    double L = 0.0;
                    for (int i = 0; i < q; ++i) L = ((s >> i) & 1) ? L + (double)a[i] : L - (double)a[i];
                    levels[s] = L;
                }
                team_sync<TW>();
#pragma unroll
                for (int e = 0; e < EPT; ++e) {
                    const double wv = (double)w[e];
                    int best = ncodes - 1;
                    double dbest = fabs(wv - levels[best]);
#pragma unroll 1
                    for (int s = ncodes - 2; s >= 0; --s) {
                        const double d = fabs(wv - levels[s]);
                        if (d < dbest) {
                            dbest = d;
                            best = s;
                        }
                    }
                    code[e] = (uint32_t)best;
                }
            }
            // ---- write the planes
            for (int i = 0; i < q; ++i) {
                uint32_t* brow = p.bits + ((long long)i * p.d_out + j) * p.pitch + (k0 >> 5);
#pragma unroll
                for (int e = 0; e < EPT; ++e) {
                    const bool valid = (e * NT + tid) < m;
                    const uint32_t word = __ballot_sync(0xffffffffu, valid && ((code[e] >> i) & 1u));
                    if (lane == 0 && (e * NT + twarp * 32) < m) brow[e * TW + twarp] = word;
                }
            }
        }

        // ---- scales, zero padding words of the row, optional squared error
        if constexpr (QT > 0) {
#pragma unroll
            for (int i = 0; i < QT; ++i)
                if (tid == i) p.alpha[((long long)i * p.d_out + j) * p.G + c] = a[i];
        } else {
            if (tid < q) p.alpha[((long long)tid * p.d_out + j) * p.G + c] = a[tid];
        }
        if (c == p.G - 1) {
            const int first_pad = (p.d_in + 31) >> 5;
            const int npad = p.pitch - first_pad;  // 0..3
            for (int t = tid; t < npad * q; t += NT) {
                const int i = t / npad, wdx = t - i * npad;
                p.bits[((long long)i * p.d_out + j) * p.pitch + first_pad + wdx] = 0u;
            }
        }
        if (p.sq_err != nullptr) {
            double local = 0.0;
            if (ALT) {
#pragma unroll
                for (int e = 0; e < EPT; ++e)
                    if (e * NT + tid < m) {
                        double wh = 0.0;
                        for (int i = 0; i < q; ++i)
                            wh = ((code[e] >> i) & 1u) ? wh + (double)a[i] : wh - (double)a[i];
                        const double d = (double)w[e] - wh;
                        local += d * d;
                    }
            } else {
#pragma unroll
                for (int e = 0; e < EPT; ++e)
                    if (e * NT + tid < m) local += r[e] * r[e];
            }
            const double E = team_sum<TW>(local, red_scratch);
            if (tid == 0) p.sq_err[(long long)j * p.G + c] = E;
        }
    }
}

template <int EPT, int TW>
cudaError_t launch_quantize(const QuantParams& p, cudaStream_t stream) {
    constexpr int TEAMS = (TW == 1) ? 4 : 1;
    const int threads = (TW == 1) ? 128 : TW * 32;
    long long blocks = (p.items + TEAMS - 1) / TEAMS;
    const long long cap = (long long)bcq::sm_count() * 64;  // grid-stride beyond this
    if (blocks > cap) blocks = cap;
    if (p.alt_iters > 0) {
        if (p.q == 2) quantize_kernel<EPT, TW, true, 2><<<(unsigned)blocks, threads, 0, stream>>>(p);
        else if (p.q == 3) quantize_kernel<EPT, TW, true, 3><<<(unsigned)blocks, threads, 0, stream>>>(p);
        else if (p.q == 4) quantize_kernel<EPT, TW, true, 4><<<(unsigned)blocks, threads, 0, stream>>>(p);
        else quantize_kernel<EPT, TW, true, 0><<<(unsigned)blocks, threads, 0, stream>>>(p);
    } else {
        quantize_kernel<EPT, TW, false, 0><<<(unsigned)blocks, threads, 0, stream>>>(p);
    }
    bcq::count_launch();
    return cudaGetLastError();
}

__global__ void dequantize_kernel(int d_out, int d_in, int q, int g, int G, int pitch,
                                  const uint32_t* __restrict__ bits,
                                  const float* __restrict__ alpha, float* __restrict__ W_hat,
                                  long long ldw) {
    const int j = blockIdx.y;
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= d_in) return;
    const int c = k / g;
    float s = 0.0f;
    for (int i = 0; i < q; ++i) {
        const uint32_t word = __ldg(bits + ((long long)i * d_out + j) * pitch + (k >> 5));
        const float a = __ldg(alpha + ((long long)i * d_out + j) * G + c);
        s += ((word >> (k & 31)) & 1u) ? a : -a;
    }
    W_hat[(long long)j * ldw + k] = s;
}

}  // namespace

extern "C" bcq_status bcq_quantize(int d_out, int d_in, int q, int g, const float* W, size_t ldw,
                                   int alt_iters, uint32_t* bits, float* alpha, double* sq_err,
                                   void* stream) {
    bcq_status st = bcq::check_shape(d_out, d_in, q, g);
    if (st != BCQ_OK) return st;
    if (!W || !bits || !alpha) return BCQ_ERR_NULL;
    if (ldw < (size_t)d_in || alt_iters < 0) return BCQ_ERR_SHAPE;
    if (g > BCQ_MAX_QUANT_G) return BCQ_ERR_UNSUPPORTED;
    if (!bcq::aligned16(bits)) return BCQ_ERR_ALIGN;
    QuantParams p;
    p.d_out = d_out; p.d_in = d_in; p.q = q; p.g = g;
    p.G = (int)bcq_num_groups(d_in, g);
    p.alt_iters = alt_iters;
    p.ldw = (long long)ldw;
    p.pitch = (int)bcq_pitch_words(d_in);
    p.W = W; p.bits = bits; p.alpha = alpha; p.sq_err = sq_err;
    p.items = (long long)d_out * p.G;
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e;
    if (g <= 128) e = launch_quantize<4, 1>(p, s);
    else if (g <= 256) e = launch_quantize<8, 1>(p, s);
    else if (g <= 512) e = launch_quantize<16, 1>(p, s);
    else if (g <= 1024) e = launch_quantize<32, 1>(p, s);
    else if (g <= 2048) e = launch_quantize<8, 8>(p, s);
    else if (g <= 4096) e = launch_quantize<16, 8>(p, s);
    else if (g <= 8192) e = launch_quantize<32, 8>(p, s);
    else e = launch_quantize<32, 32>(p, s);
    if (e != cudaSuccess) return bcq::cuda_fail(e);
    return BCQ_OK;
}

extern "C" bcq_status bcq_dequantize(int d_out, int d_in, int q, int g, const uint32_t* bits,
                                     const float* alpha, float* W_hat, size_t ldw, void* stream) {
    bcq_status st = bcq::check_shape(d_out, d_in, q, g);
    if (st != BCQ_OK) return st;
    if (!bits || !alpha || !W_hat) return BCQ_ERR_NULL;
    if (ldw < (size_t)d_in) return BCQ_ERR_SHAPE;
    if (d_out > 65535 * 1) {
        // grid.y limit: fold rows is not needed for the layer sizes this library targets
        if (d_out > 65535) return BCQ_ERR_UNSUPPORTED;
    }
    dim3 grid((unsigned)bcq::ceil_div(d_in, 256), (unsigned)d_out);
    dequantize_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>(
        d_out, d_in, q, g, (int)bcq_num_groups(d_in, g), (int)bcq_pitch_words(d_in), bits, alpha,
        W_hat, (long long)ldw);
    bcq::count_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return bcq::cuda_fail(e);
    return BCQ_OK;
}
