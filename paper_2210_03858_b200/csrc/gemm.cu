// tcgen05 / TMEM kernels of the BCQ linear layer: forward (Eq. 2), input gradient (Eq. 3),
// scale gradient (Eq. 4) and the skinny decode case of the forward.
//
// All three contractions are 128 x TN x 64 UMMA tiles with fp32 accumulators in tensor memory:
//
//   forward   D[j, t] = sum_k  W_hat[j, k] * X[t, k]      A = W_hat tile, expanded on the fly
//   dX        D[k, t] = sum_j  W_hat[j, k] * dY[t, j]     A = W_hat tile, expanded on the fly
//   dalpha    D[j, k] = sum_t  dY[t, j]    * X[t, k]      A, B = TMA tiles of dY and X
//
// W_hat = sum_i alpha_i b_i (Eq. 1) never exists in global memory.  For the first two, eight
// "worker" warps read 32 weights per plane as one 32-bit word, rebuild the 32 scaled weights in
// fp32 registers, round once to bf16 and store them into the 128-byte-swizzled shared-memory
// layout the tensor core reads: with the weight row j as the M index and k contiguous for the
// forward (K-major A), and as "one 128-byte line of 64 k per row j" for dX, which is exactly the
// MN-major operand layout when k is the M index and j the K index.  The token-side operand
// (X or dY) arrives by TMA.  For dalpha both operands are MN-major TMA tiles (tokens are the K
// index) and the epilogue applies the signs of B_i to the accumulator tile and reduces it over
// each group, so the d_out x d_in product dY^T X never leaves the chip.
//
// Warp roles in a CTA of 320 threads: warp 0 = TMA producer (one elected lane), warp 1 = UMMA
// issuer (one lane) and owner of the TMEM allocation, warps 2..9 = workers (expansion during the
// main loop, then the epilogue: warp w reads TMEM lanes 32*(w%4).., the two warps that share a
// lane quarter split the columns).  Stages are handed around with mbarriers; every wait is
// bounded in time and a timeout raises a flag instead of hanging.
#include <cuda.h>
#include <cuda_bf16.h>

#include "common.h"
#include "ptx.cuh"

namespace {

using namespace bcq;

constexpr int kThreads = 320;
constexpr int kWorkerWarp0 = 2;
constexpr int kWorkerWarps = 8;
constexpr int kBlockM = 128;
constexpr int kBlockK = 64;
constexpr uint32_t kABytes = kBlockM * kBlockK * 2;  // 16 KiB per stage
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

__device__ int g_timeout_flag = 0;

enum { MODE_FWD = 0, MODE_BWDX = 1 };

struct ExpandParams {
    int d_out, d_in, q, g, G, pitch, n;
    int Mdim;            // rows of the output tile dimension: d_out (fwd) or d_in (dX)
    int num_kb;          // K blocks of 64 over d_in (fwd) or d_out (dX)
    int kb_per_split;    // K blocks per blockIdx.z
    int splits;
    const uint32_t* bits;
    const float* alpha;
    const float* bias;   // fwd only, may be null
    void* out;           // [n][ldo] (fp32 or bf16) when splits == 1
    long long ldo;
    int out_bf16;
    float* partial;      // [splits][n][Mdim] fp32 when splits > 1
};

struct DalphaParams {
    int d_out, d_in, q, g, G, pitch, n;
    int num_kb;          // K blocks of 64 tokens
    int kb_per_split;
    int splits;
    int n_subtiles;      // column sub-tiles of width TN/2 over d_in
    int slots;           // partial slots per sub-tile
    uint32_t plane_mask;
    const uint32_t* bits;
    float* partial;      // [splits][n_subtiles][q][slots][d_out]
};

// ------------------------------------------------------------------------------------------
// shared-memory control block and bounded waits
// ------------------------------------------------------------------------------------------

struct Ctl {
    uint32_t full;    // + 8*s : operand tiles landed (TMA bytes)
    uint32_t aready;  // + 8*s : expanded A tile written (one arrival per worker thread)
    uint32_t empty;   // + 8*s : UMMAs reading the stage have completed
    uint32_t accum;   // accumulator complete
    uint32_t spare;   // used only when giving up
    volatile int* abort_flag;
};

__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, const Ctl& ctl, int code) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = ptx::globaltimer_ns();
    uint32_t spins = 0;
    while (true) {
        if (ptx::mbar_try_wait(bar, parity)) return true;
        if ((++spins & 63u) == 0u) {
            if (*ctl.abort_flag) return false;
            if (ptx::globaltimer_ns() - t0 > kWaitLimitNs) {
                *ctl.abort_flag = 1;
                atomicExch(&g_timeout_flag, code);
                return false;
            }
        }
    }
}

// Rebuilds 32 consecutive weights of one row, W_hat = sum_i (+-alpha_i), from one 32-bit word per
// plane, rounds to bf16 and stores them as four 16-byte chunks of a 128-byte swizzled line.
//   nw[i]  : complement of the plane word (bit p clear <=> b_i = +1)
//   a[i]   : the scale of this (row, group)
//   line   : shared address of the 128-byte line;  lx = line index & 7 (the swizzle key)
//   chunk0 : first of the four chunk slots (0 or 4)
__device__ __forceinline__ void expand32(const uint32_t (&nw)[BCQ_MAX_Q], const float (&a)[BCQ_MAX_Q],
                                         int q, uint32_t line, uint32_t lx, uint32_t chunk0) {
    float v[32];
#pragma unroll
    for (int p = 0; p < 32; ++p) v[p] = 0.0f;
#pragma unroll
    for (int i = 0; i < BCQ_MAX_Q; ++i) {
        if (i < q) {
            const uint32_t ai = __float_as_uint(a[i]);
            const uint32_t w = nw[i];
#pragma unroll
            for (int p = 0; p < 32; ++p)
                v[p] += __uint_as_float(ai ^ ((w << (31 - p)) & 0x80000000u));
        }
    }
#pragma unroll
    for (int cc = 0; cc < 4; ++cc) {
        uint32_t o[4];
#pragma unroll
        for (int h = 0; h < 4; ++h) {
            __nv_bfloat162 t = __floats2bfloat162_rn(v[cc * 8 + 2 * h], v[cc * 8 + 2 * h + 1]);
            o[h] = *reinterpret_cast<uint32_t*>(&t);
        }
        ptx::st_shared_v4(line + (((chunk0 + cc) ^ lx) << 4), o[0], o[1], o[2], o[3]);
    }
}

template <int TN>
struct TmemCols {
    static constexpr uint32_t value = TN < 32 ? 32 : TN;
};

// ------------------------------------------------------------------------------------------
// forward / dX: A expanded from the bit-planes, B by TMA
// ------------------------------------------------------------------------------------------

template <int MODE, int TN, int STAGES>
__global__ void __launch_bounds__(kThreads, 1)
expand_gemm_kernel(const __grid_constant__ CUtensorMap tmap_b, const ExpandParams p) {
    constexpr uint32_t kBBytes = TN * kBlockK * 2;
    constexpr uint32_t kStageBytes = kABytes + kBBytes;
    constexpr uint32_t kIdesc = ptx::make_idesc_bf16(kBlockM, TN, MODE == MODE_BWDX ? 1 : 0, 0);

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
    const uint32_t ctl_base = smem_base + STAGES * kStageBytes;
    uint8_t* ctl_gen = smem_gen + STAGES * kStageBytes;

    Ctl ctl;
    ctl.full = ctl_base;
    ctl.aready = ctl_base + 8 * STAGES;
    ctl.empty = ctl_base + 16 * STAGES;
    ctl.accum = ctl_base + 24 * STAGES;
    ctl.spare = ctl.accum + 8;
    volatile uint32_t* tmem_holder = reinterpret_cast<volatile uint32_t*>(ctl_gen + 24 * STAGES + 16);
    ctl.abort_flag = reinterpret_cast<volatile int*>(ctl_gen + 24 * STAGES + 20);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int m0 = blockIdx.x * kBlockM;
    const int t0 = blockIdx.y * TN;
    const int kb_begin = blockIdx.z * p.kb_per_split;
    const int kb_end = min(p.num_kb, kb_begin + p.kb_per_split);
    const int iters = kb_end - kb_begin;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(ctl.full + 8 * s, 1);
            ptx::mbar_init(ctl.aready + 8 * s, kWorkerWarps * 32);
            ptx::mbar_init(ctl.empty + 8 * s, 1);
        }
        ptx::mbar_init(ctl.accum, 1);
        ptx::mbar_init(ctl.spare, 1);
        *ctl.abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tmap_b);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(const_cast<uint32_t*>(tmem_holder)), TmemCols<TN>::value);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_holder;

    if (warp == 0) {
        // ---------------- TMA producer
        if (lane == 0) {
            bool ok = true;
            int issued = 0;
            for (int it = 0; it < iters && ok; ++it) {
                const int s = it % STAGES;
                const uint32_t ph = (it / STAGES) & 1;
                ok = wait_bar(ctl.empty + 8 * s, ph ^ 1u, ctl, 1);
                if (!ok) break;
                ptx::mbar_arrive_expect_tx(ctl.full + 8 * s, kBBytes);
                ptx::tma_load_2d(smem_base + s * kStageBytes + kABytes, &tmap_b,
                                 (kb_begin + it) * kBlockK, t0, ctl.full + 8 * s);
                issued = it + 1;
            }
            if (!ok) {
                // giving up: let the copies already issued land before the CTA exits
                for (int it = max(0, issued - STAGES); it < issued; ++it)
                    wait_bar(ctl.full + 8 * (it % STAGES), (it / STAGES) & 1, ctl, 2);
            }
        }
    } else if (warp == 1) {
        // ---------------- UMMA issuer
        if (lane == 0) {
            bool ok = true;
            for (int it = 0; it < iters && ok; ++it) {
                const int s = it % STAGES;
                const uint32_t ph = (it / STAGES) & 1;
                ok = wait_bar(ctl.full + 8 * s, ph, ctl, 3) && wait_bar(ctl.aready + 8 * s, ph, ctl, 4);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint32_t sa = smem_base + s * kStageBytes;
                const uint32_t sb = sa + kABytes;
#pragma unroll
                for (int kk = 0; kk < kBlockK / 16; ++kk) {
                    uint64_t da, db;
                    if (MODE == MODE_FWD)
                        da = ptx::make_smem_desc(sa + kk * 32, 16, 1024);
                    else
                        da = ptx::make_smem_desc(sa + kk * 2048, 8192, 1024);
                    db = ptx::make_smem_desc(sb + kk * 32, 16, 1024);
                    ptx::umma_bf16(tmem_base, da, db, kIdesc, (it > 0 || kk > 0) ? 1u : 0u);
                }
                ptx::umma_commit(ctl.empty + 8 * s);
            }
            if (ok) {
                ptx::umma_commit(ctl.accum);
            } else {
                ptx::umma_commit(ctl.spare);
                wait_bar(ctl.spare, 0, ctl, 5);
            }
        }
    } else {
        // ---------------- workers: expansion, then epilogue
        const int e = threadIdx.x - kWorkerWarp0 * 32;  // 0..255
        int row_j, kw_off, line_idx;
        uint32_t line_off, chunk0;
        if (MODE == MODE_FWD) {
            // thread = (weight row m0 + (e & 127), 32-wide half of the 64 k of the stage)
            line_idx = e & 127;
            row_j = m0 + line_idx;
            kw_off = e >> 7;
            line_off = line_idx * 128;
            chunk0 = (e >> 7) * 4;
        } else {
            // thread = (K index j = 64*kb + (e & 63), 32-wide quarter of the 128 k of the tile)
            line_idx = e & 63;
            row_j = line_idx;  // + 64 * kb below
            kw_off = (m0 >> 5) + (e >> 6);
            line_off = ((e >> 7) * 8192) + line_idx * 128;
            chunk0 = ((e >> 6) & 1) * 4;
        }
        const uint32_t lx = line_idx & 7;
        const long long plane_words = (long long)p.d_out * p.pitch;
        const long long plane_alpha = (long long)p.d_out * p.G;

        uint32_t nw[BCQ_MAX_Q];
        float al[BCQ_MAX_Q];
        bool valid = false;
        auto fetch = [&](int kb) {
            int j, kw;
            if (MODE == MODE_FWD) {
                j = row_j;
                kw = kb * 2 + kw_off;
            } else {
                j = kb * kBlockK + row_j;
                kw = kw_off;
            }
            valid = (j < p.d_out) && (kw < p.pitch);
            const int c = min((kw * 32) / p.g, p.G - 1);
#pragma unroll
            for (int i = 0; i < BCQ_MAX_Q; ++i) {
                if (i < p.q && valid) {
                    nw[i] = ~__ldg(p.bits + i * plane_words + (long long)j * p.pitch + kw);
                    al[i] = __ldg(p.alpha + i * plane_alpha + (long long)j * p.G + c);
                } else {
                    nw[i] = 0u;
                    al[i] = 0.0f;
                }
            }
        };

        bool ok = true;
        if (iters > 0) fetch(kb_begin);
        for (int it = 0; it < iters; ++it) {
            const int s = it % STAGES;
            const uint32_t ph = (it / STAGES) & 1;
            uint32_t cnw[BCQ_MAX_Q];
            float cal[BCQ_MAX_Q];
#pragma unroll
            for (int i = 0; i < BCQ_MAX_Q; ++i) {
                cnw[i] = nw[i];
                cal[i] = al[i];
            }
            if (it + 1 < iters) fetch(kb_begin + it + 1);  // in flight while this stage is built
            ok = wait_bar(ctl.empty + 8 * s, ph ^ 1u, ctl, 6);
            if (!ok) break;
            expand32(cnw, cal, p.q, smem_base + s * kStageBytes + line_off, lx, chunk0);
            ptx::fence_proxy_async_smem();
            ptx::mbar_arrive(ctl.aready + 8 * s);
        }

        // epilogue: D[row, col] -> out[t0 + col][m0 + row]
        if (ok) ok = wait_bar(ctl.accum, 0, ctl, 7);
        if (ok) {
            ptx::tc_fence_after_sync();
            const int quarter = warp & 3;
            const int half = (warp - kWorkerWarp0) >> 2;
            constexpr int HN = TN / 2;
            constexpr int CH = HN < 16 ? 8 : 16;
            const int m = m0 + quarter * 32 + lane;
            const bool m_ok = m < p.Mdim;
            const float bias = (MODE == MODE_FWD && p.bias != nullptr && p.splits == 1 && m_ok)
                                   ? __ldg(p.bias + m) : 0.0f;
#pragma unroll 1
            for (int cb = 0; cb < HN; cb += CH) {
                const int col = half * HN + cb;
                if (t0 + col >= p.n) break;  // uniform in the warp
                uint32_t v[CH];
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)col;
                if (CH == 8)
                    ptx::tmem_ld_x8(taddr, v);
                else
                    ptx::tmem_ld_x16(taddr, v);
                ptx::tmem_ld_wait();
                if (m_ok) {
#pragma unroll
                    for (int cidx = 0; cidx < CH; ++cidx) {
                        const int t = t0 + col + cidx;
                        if (t < p.n) {
                            const float val = __uint_as_float(v[cidx]);
                            if (p.splits > 1) {
                                p.partial[((long long)blockIdx.z * p.n + t) * p.Mdim + m] = val;
                            } else if (p.out_bf16) {
                                reinterpret_cast<__nv_bfloat16*>(p.out)[(long long)t * p.ldo + m] =
                                    __float2bfloat16_rn(val + bias);
                            } else {
                                reinterpret_cast<float*>(p.out)[(long long)t * p.ldo + m] = val + bias;
                            }
                        }
                    }
                }
            }
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, TmemCols<TN>::value);
    }
}

// out[t][m] = sum_z partial[z][t][m] (+ bias[m]), in the order z = 0, 1, ...
__global__ void splitk_reduce_kernel(int n, int Mdim, int splits, const float* __restrict__ partial,
                                     const float* __restrict__ bias, void* out, long long ldo,
                                     int out_bf16) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long total = (long long)n * Mdim;
    if (idx >= total) return;
    const int t = (int)(idx / Mdim);
    const int m = (int)(idx - (long long)t * Mdim);
    float s = 0.0f;
    for (int z = 0; z < splits; ++z) s += __ldg(partial + (long long)z * total + idx);
    if (bias != nullptr) s += __ldg(bias + m);
    if (out_bf16)
        reinterpret_cast<__nv_bfloat16*>(out)[(long long)t * ldo + m] = __float2bfloat16_rn(s);
    else
        reinterpret_cast<float*>(out)[(long long)t * ldo + m] = s;
}

// ------------------------------------------------------------------------------------------
// dalpha: D[j, k] = sum_t dY[t, j] X[t, k], sign-weighted group sums in the epilogue
// ------------------------------------------------------------------------------------------

template <int TN, int STAGES>
__global__ void __launch_bounds__(kThreads, 1)
dalpha_kernel(const __grid_constant__ CUtensorMap tmap_dy, const __grid_constant__ CUtensorMap tmap_x,
              const DalphaParams p) {
    constexpr uint32_t kBBytes = TN * kBlockK * 2;
    constexpr uint32_t kStageBytes = kABytes + kBBytes;
    constexpr uint32_t kIdesc = ptx::make_idesc_bf16(kBlockM, TN, 1, 1);
    constexpr int HN = TN / 2;
    constexpr int NCH = HN / 32;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
    const uint32_t ctl_base = smem_base + STAGES * kStageBytes;
    uint8_t* ctl_gen = smem_gen + STAGES * kStageBytes;

    Ctl ctl;
    ctl.full = ctl_base;
    ctl.aready = 0;
    ctl.empty = ctl_base + 8 * STAGES;
    ctl.accum = ctl_base + 16 * STAGES;
    ctl.spare = ctl.accum + 8;
    volatile uint32_t* tmem_holder = reinterpret_cast<volatile uint32_t*>(ctl_gen + 16 * STAGES + 16);
    ctl.abort_flag = reinterpret_cast<volatile int*>(ctl_gen + 16 * STAGES + 20);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int j0 = blockIdx.x * kBlockM;
    const int k0 = blockIdx.y * TN;
    const int kb_begin = blockIdx.z * p.kb_per_split;
    const int kb_end = min(p.num_kb, kb_begin + p.kb_per_split);
    const int iters = kb_end - kb_begin;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(ctl.full + 8 * s, 1);
            ptx::mbar_init(ctl.empty + 8 * s, 1);
        }
        ptx::mbar_init(ctl.accum, 1);
        ptx::mbar_init(ctl.spare, 1);
        *ctl.abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tmap_dy);
        ptx::prefetch_tmap(&tmap_x);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(const_cast<uint32_t*>(tmem_holder)), TmemCols<TN>::value);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_holder;

    if (warp == 0) {
        if (lane == 0) {
            bool ok = true;
            int issued = 0;
            for (int it = 0; it < iters && ok; ++it) {
                const int s = it % STAGES;
                const uint32_t ph = (it / STAGES) & 1;
                ok = wait_bar(ctl.empty + 8 * s, ph ^ 1u, ctl, 11);
                if (!ok) break;
                const uint32_t sa = smem_base + s * kStageBytes;
                const int tok = (kb_begin + it) * kBlockK;
                ptx::mbar_arrive_expect_tx(ctl.full + 8 * s, kStageBytes);
                // A: two blocks of 64 rows j (inner) x 64 tokens; B: TN/64 blocks of 64 k x 64 tokens
                ptx::tma_load_2d(sa, &tmap_dy, j0, tok, ctl.full + 8 * s);
                ptx::tma_load_2d(sa + 8192, &tmap_dy, j0 + 64, tok, ctl.full + 8 * s);
#pragma unroll
                for (int b = 0; b < TN / 64; ++b)
                    ptx::tma_load_2d(sa + kABytes + b * 8192, &tmap_x, k0 + b * 64, tok, ctl.full + 8 * s);
                issued = it + 1;
            }
            if (!ok) {
                for (int it = max(0, issued - STAGES); it < issued; ++it)
                    wait_bar(ctl.full + 8 * (it % STAGES), (it / STAGES) & 1, ctl, 12);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            bool ok = true;
            for (int it = 0; it < iters && ok; ++it) {
                const int s = it % STAGES;
                const uint32_t ph = (it / STAGES) & 1;
                ok = wait_bar(ctl.full + 8 * s, ph, ctl, 13);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint32_t sa = smem_base + s * kStageBytes;
                const uint32_t sb = sa + kABytes;
#pragma unroll
                for (int kk = 0; kk < kBlockK / 16; ++kk) {
                    const uint64_t da = ptx::make_smem_desc(sa + kk * 2048, 8192, 1024);
                    const uint64_t db = ptx::make_smem_desc(sb + kk * 2048, 8192, 1024);
                    ptx::umma_bf16(tmem_base, da, db, kIdesc, (it > 0 || kk > 0) ? 1u : 0u);
                }
                ptx::umma_commit(ctl.empty + 8 * s);
            }
            if (ok) {
                ptx::umma_commit(ctl.accum);
            } else {
                ptx::umma_commit(ctl.spare);
                wait_bar(ctl.spare, 0, ctl, 15);
            }
        }
    } else {
        // ---------------- epilogue: thread = (row j, HN columns of the tile)
        const int quarter = warp & 3;
        const int half = (warp - kWorkerWarp0) >> 2;
        const int j = j0 + quarter * 32 + lane;
        const bool j_ok = j < p.d_out;
        const int kbase = k0 + half * HN;
        const int subtile = blockIdx.y * 2 + half;
        const long long plane_words = (long long)p.d_out * p.pitch;

        // the sign words do not depend on the accumulator: fetch them while the main loop runs
        uint32_t nw[NCH][BCQ_MAX_Q];
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch) {
            const int kw = (kbase >> 5) + ch;
#pragma unroll
            for (int i = 0; i < BCQ_MAX_Q; ++i) {
                const bool act = (i < p.q) && ((p.plane_mask >> i) & 1u) && j_ok && (kw < p.pitch);
                nw[ch][i] = act ? ~__ldg(p.bits + i * plane_words + (long long)j * p.pitch + kw) : 0u;
            }
        }

        bool ok = wait_bar(ctl.accum, 0, ctl, 16);
        if (ok && kbase < p.d_in) {
            ptx::tc_fence_after_sync();
            const int c_first = min(kbase / p.g, p.G - 1);
            float acc[BCQ_MAX_Q];
#pragma unroll
            for (int i = 0; i < BCQ_MAX_Q; ++i) acc[i] = 0.0f;
            int cur_c = c_first;
            auto flush = [&](int c) {
                if (!j_ok) return;
                const int slot = c - c_first;
#pragma unroll
                for (int i = 0; i < BCQ_MAX_Q; ++i) {
                    if (i < p.q && ((p.plane_mask >> i) & 1u)) {
                        const long long idx =
                            ((((long long)blockIdx.z * p.n_subtiles + subtile) * p.q + i) * p.slots + slot) *
                                p.d_out + j;
                        p.partial[idx] = acc[i];
                    }
                }
            };
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) {
                const int kg = kbase + ch * 32;
                if (kg < p.d_in) {  // uniform in the warp
                    const int c = min(kg / p.g, p.G - 1);
                    if (c != cur_c) {
                        flush(cur_c);
                        cur_c = c;
#pragma unroll
                        for (int i = 0; i < BCQ_MAX_Q; ++i) acc[i] = 0.0f;
                    }
                    uint32_t v[32];
                    ptx::tmem_ld_x32(tmem_base + ((uint32_t)(quarter * 32) << 16) +
                                         (uint32_t)(half * HN + ch * 32), v);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < BCQ_MAX_Q; ++i) {
                        if (i < p.q && ((p.plane_mask >> i) & 1u)) {
                            const uint32_t w = nw[ch][i];
                            float s = 0.0f;
#pragma unroll
                            for (int b = 0; b < 32; ++b)
                                s += __uint_as_float(v[b] ^ ((w << (31 - b)) & 0x80000000u));
                            acc[i] += s;
                        }
                    }
                }
            }
            flush(cur_c);
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, TmemCols<TN>::value);
    }
}

// dalpha[i][j][c] (+)= scale * sum over splits and over the sub-tiles that meet group c.
__global__ void dalpha_reduce_kernel(int d_out, int d_in, int q, int g, int G, int HN, int splits,
                                     int n_subtiles, int slots, uint32_t plane_mask, float scale,
                                     int accumulate, const float* __restrict__ partial,
                                     float* __restrict__ dalpha) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long total = (long long)q * G * d_out;
    if (idx >= total) return;
    const int j = (int)(idx % d_out);
    const long long r = idx / d_out;
    const int c = (int)(r % G);
    const int i = (int)(r / G);
    if (!((plane_mask >> i) & 1u)) return;
    const int k_lo = c * g;
    const int k_hi = min(k_lo + g, d_in) - 1;
    float s = 0.0f;
    for (int z = 0; z < splits; ++z)
        for (int st = k_lo / HN; st <= k_hi / HN; ++st) {
            const int slot = c - min((st * HN) / g, G - 1);
            s += __ldg(partial + ((((long long)z * n_subtiles + st) * q + i) * slots + slot) * d_out + j);
        }
    float* dst = dalpha + ((long long)i * d_out + j) * G + c;
    *dst = accumulate ? (*dst + scale * s) : (scale * s);
}

// ------------------------------------------------------------------------------------------
// host side: plans, tensor maps, launches
// ------------------------------------------------------------------------------------------

int sm_count() {
    static int cached = 0;
    if (cached == 0) {
        int dev = 0, n = 0;
        if (cudaGetDevice(&dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0)
            cached = n;
        else
            return 148;  // B200; not cached so that a later call with a device present asks again
    }
    return cached;
}

struct ExpandPlan {
    int TN, splits, kb_per_split, num_kb, m_tiles, n_tiles;
};

// Tile width over tokens and the K split.  Wide token tiles amortise the expansion of a weight
// tile over more tokens; the K split fills the SMs when the output has few tiles.
ExpandPlan plan_expand(int Mdim, int Kdim, int n) {
    ExpandPlan pl;
    const int sms = sm_count();
    pl.m_tiles = ceil_div(Mdim, kBlockM);
    pl.num_kb = ceil_div(Kdim, kBlockK);
    int tn;
    if (n <= 16) tn = 16;
    else if (n <= 32) tn = 32;
    else if (n <= 64) tn = 64;
    else if (n <= 128) tn = 128;
    else {
        tn = 256;
        if (pl.m_tiles * ceil_div(n, 256) < sms) tn = 128;
    }
    pl.TN = tn;
    pl.n_tiles = ceil_div(n, tn);
    const int tiles = pl.m_tiles * pl.n_tiles;
    int target = (tn <= 32) ? 2 * sms : sms;  // narrow tiles fit several CTAs per SM
    int splits = target / tiles;
    if (splits < 1) splits = 1;
    const int max_splits = (pl.num_kb + 3) / 4;  // at least 4 K blocks per CTA
    if (splits > max_splits) splits = max_splits;
    if (splits > 32) splits = 32;
    pl.kb_per_split = ceil_div(pl.num_kb, splits);
    pl.splits = ceil_div(pl.num_kb, pl.kb_per_split);
    return pl;
}

struct DalphaPlan {
    int TN, HN, splits, kb_per_split, num_kb, m_tiles, n_tiles, n_subtiles, slots;
};

DalphaPlan plan_dalpha(int d_out, int d_in, int g, int n) {
    DalphaPlan pl;
    const int sms = sm_count();
    pl.m_tiles = ceil_div(d_out, kBlockM);
    pl.num_kb = ceil_div(n, kBlockK);
    pl.TN = 256;
    if (d_in <= 128 || pl.m_tiles * ceil_div(d_in, 256) < sms) pl.TN = 128;
    pl.HN = pl.TN / 2;
    pl.n_tiles = ceil_div(d_in, pl.TN);
    pl.n_subtiles = pl.n_tiles * 2;
    if (g % pl.HN == 0) pl.slots = 1;
    else if (pl.HN % g == 0) pl.slots = pl.HN / g;
    else pl.slots = pl.HN / g + 2;
    const int tiles = pl.m_tiles * pl.n_tiles;
    int splits = sms / tiles;
    if (splits < 1) splits = 1;
    const int max_splits = (pl.num_kb + 3) / 4;
    if (splits > max_splits) splits = max_splits;
    if (splits > 32) splits = 32;
    pl.kb_per_split = ceil_div(pl.num_kb, splits);
    pl.splits = ceil_div(pl.num_kb, pl.kb_per_split);
    return pl;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
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

// bf16 matrix [outer][pitch_elems] with `inner` valid elements per row; box = 64 x box_outer,
// 128-byte swizzle, out-of-range elements read as zero.
bcq_status make_tmap(CUtensorMap* m, const void* base, int inner, int outer, size_t pitch_elems,
                     int box_outer) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) {
        set_last_cuda_error((int)cudaErrorNotSupported);
        return BCQ_ERR_CUDA;
    }
    cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
    cuuint64_t strides[1] = {(cuuint64_t)pitch_elems * 2};
    cuuint32_t box[2] = {64u, (cuuint32_t)box_outer};
    cuuint32_t estr[2] = {1u, 1u};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
                    estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_last_cuda_error((int)cudaErrorInvalidValue);
        return BCQ_ERR_CUDA;
    }
    return BCQ_OK;
}

template <int TN>
constexpr int stages_for() {
    return TN == 256 ? 4 : (TN == 128 ? 6 : 4);
}

template <int TN>
constexpr size_t smem_for() {
    return (size_t)stages_for<TN>() * (kABytes + TN * kBlockK * 2) + 1024 + 256;
}

template <int MODE, int TN>
bcq_status launch_expand(const CUtensorMap& tm, const ExpandParams& p, const ExpandPlan& pl,
                         cudaStream_t stream) {
    constexpr int ST = stages_for<TN>();
    constexpr size_t smem = smem_for<TN>();
    auto kern = expand_gemm_kernel<MODE, TN, ST>;
    BCQ_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    dim3 grid((unsigned)pl.m_tiles, (unsigned)pl.n_tiles, (unsigned)pl.splits);
    kern<<<grid, kThreads, smem, stream>>>(tm, p);
    BCQ_CUDA_TRY(cudaGetLastError());
    return BCQ_OK;
}

template <int MODE>
bcq_status run_expand(int d_out, int d_in, int q, int g, int n, const void* act, size_t ldact,
                      const uint32_t* bits, const float* alpha, const float* bias, void* out, size_t ldo,
                      int out_dtype, void* ws, size_t ws_bytes, void* stream, size_t need_ws,
                      const ExpandPlan& pl) {
    const int Mdim = (MODE == MODE_FWD) ? d_out : d_in;
    const int Kdim = (MODE == MODE_FWD) ? d_in : d_out;
    if (need_ws > 0) {
        if (ws == nullptr) return BCQ_ERR_NULL;
        if (ws_bytes < need_ws) return BCQ_ERR_WORKSPACE;
        if (!aligned16(ws)) return BCQ_ERR_ALIGN;
    }
    CUtensorMap tm;
    bcq_status st = make_tmap(&tm, act, Kdim, n, ldact, pl.TN);
    if (st != BCQ_OK) return st;
    ExpandParams p;
    p.d_out = d_out; p.d_in = d_in; p.q = q; p.g = g;
    p.G = (int)bcq_num_groups(d_in, g);
    p.pitch = (int)bcq_pitch_words(d_in);
    p.n = n; p.Mdim = Mdim; p.num_kb = pl.num_kb; p.kb_per_split = pl.kb_per_split; p.splits = pl.splits;
    p.bits = bits; p.alpha = alpha; p.bias = bias; p.out = out; p.ldo = (long long)ldo;
    p.out_bf16 = (out_dtype == BCQ_BF16);
    p.partial = reinterpret_cast<float*>(ws);
    cudaStream_t s = (cudaStream_t)stream;
    switch (pl.TN) {
        case 16: st = launch_expand<MODE, 16>(tm, p, pl, s); break;
        case 32: st = launch_expand<MODE, 32>(tm, p, pl, s); break;
        case 64: st = launch_expand<MODE, 64>(tm, p, pl, s); break;
        case 128: st = launch_expand<MODE, 128>(tm, p, pl, s); break;
        default: st = launch_expand<MODE, 256>(tm, p, pl, s); break;
    }
    if (st != BCQ_OK) return st;
    if (pl.splits > 1) {
        const long long total = (long long)n * Mdim;
        splitk_reduce_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(
            n, Mdim, pl.splits, p.partial, bias, out, (long long)ldo, p.out_bf16);
        BCQ_CUDA_TRY(cudaGetLastError());
    }
    return BCQ_OK;
}

bcq_status check_act(const void* ptr, size_t ld, int cols) {
    if (ptr == nullptr) return BCQ_ERR_NULL;
    if (ld < (size_t)cols) return BCQ_ERR_SHAPE;
    if (!aligned16(ptr) || (ld % 8) != 0) return BCQ_ERR_ALIGN;
    return BCQ_OK;
}

size_t expand_ws_bytes(const ExpandPlan& pl, int n, int Mdim) {
    return pl.splits > 1 ? (size_t)pl.splits * n * Mdim * sizeof(float) : 0;
}

size_t dalpha_ws_bytes(const DalphaPlan& pl, int d_out, int q) {
    return (size_t)pl.splits * pl.n_subtiles * q * pl.slots * d_out * sizeof(float);
}

bcq_status fwd_common(int decode, int d_out, int d_in, int q, int g, int n, const void* X, size_t ldx,
                      const uint32_t* bits, const float* alpha, const float* bias, void* Y, size_t ldy,
                      int y_dtype, void* ws, size_t ws_bytes, void* stream) {
    bcq_status st = check_shape(d_out, d_in, q, g);
    if (st != BCQ_OK) return st;
    if (n < 1 || (decode && n > 16)) return BCQ_ERR_SHAPE;
    if (!bits || !alpha || !Y) return BCQ_ERR_NULL;
    if ((st = check_act(X, ldx, d_in)) != BCQ_OK) return st;
    if (ldy < (size_t)d_out) return BCQ_ERR_SHAPE;
    if (y_dtype != BCQ_F32 && y_dtype != BCQ_BF16) return BCQ_ERR_SHAPE;
    if (!aligned16(bits)) return BCQ_ERR_ALIGN;
    const ExpandPlan pl = plan_expand(d_out, d_in, n);
    return run_expand<MODE_FWD>(d_out, d_in, q, g, n, X, ldx, bits, alpha, bias, Y, ldy, y_dtype, ws,
                                ws_bytes, stream, expand_ws_bytes(pl, n, d_out), pl);
}

}  // namespace

namespace bcq {
bcq_status gemm_timeout_flag(int* flag_out, int reset) {
    if (flag_out == nullptr) return BCQ_ERR_NULL;
    BCQ_CUDA_TRY(cudaDeviceSynchronize());
    int v = 0;
    BCQ_CUDA_TRY(cudaMemcpyFromSymbol(&v, g_timeout_flag, sizeof(int)));
    *flag_out = v;
    if (reset && v != 0) {
        const int zero = 0;
        BCQ_CUDA_TRY(cudaMemcpyToSymbol(g_timeout_flag, &zero, sizeof(int)));
    }
    return BCQ_OK;
}
}  // namespace bcq

extern "C" size_t bcq_workspace_bytes(int op, int d_out, int d_in, int q, int g, int n) {
    if (bcq::check_shape(d_out, d_in, q, g) != BCQ_OK) return 0;
    switch (op) {
        case BCQ_OP_FWD:
        case BCQ_OP_DECODE:
            if (n < 1) return 0;
            return expand_ws_bytes(plan_expand(d_out, d_in, n), n, d_out);
        case BCQ_OP_BWD_X:
            if (n < 1) return 0;
            return expand_ws_bytes(plan_expand(d_in, d_out, n), n, d_in);
        case BCQ_OP_BWD_ALPHA:
            if (n < 1) return 0;
            return dalpha_ws_bytes(plan_dalpha(d_out, d_in, g, n), d_out, q);
        default:
            return 0;
    }
}

extern "C" bcq_status bcq_linear_fwd(int d_out, int d_in, int q, int g, int n, const void* X, size_t ldx,
                                     const uint32_t* bits, const float* alpha, const float* bias, void* Y,
                                     size_t ldy, int y_dtype, void* ws, size_t ws_bytes, void* stream) {
    return fwd_common(0, d_out, d_in, q, g, n, X, ldx, bits, alpha, bias, Y, ldy, y_dtype, ws, ws_bytes,
                      stream);
}

extern "C" bcq_status bcq_linear_decode(int d_out, int d_in, int q, int g, int n, const void* X,
                                        size_t ldx, const uint32_t* bits, const float* alpha,
                                        const float* bias, void* Y, size_t ldy, int y_dtype, void* ws,
                                        size_t ws_bytes, void* stream) {
    return fwd_common(1, d_out, d_in, q, g, n, X, ldx, bits, alpha, bias, Y, ldy, y_dtype, ws, ws_bytes,
                      stream);
}

extern "C" bcq_status bcq_linear_bwd_x(int d_out, int d_in, int q, int g, int n, const void* dY,
                                       size_t lddy, const uint32_t* bits, const float* alpha, void* dX,
                                       size_t lddx, int dx_dtype, void* ws, size_t ws_bytes,
                                       void* stream) {
    bcq_status st = check_shape(d_out, d_in, q, g);
    if (st != BCQ_OK) return st;
    if (n < 1) return BCQ_ERR_SHAPE;
    if (!bits || !alpha || !dX) return BCQ_ERR_NULL;
    if ((st = check_act(dY, lddy, d_out)) != BCQ_OK) return st;
    if (lddx < (size_t)d_in) return BCQ_ERR_SHAPE;
    if (dx_dtype != BCQ_F32 && dx_dtype != BCQ_BF16) return BCQ_ERR_SHAPE;
    if (!aligned16(bits)) return BCQ_ERR_ALIGN;
    const ExpandPlan pl = plan_expand(d_in, d_out, n);
    return run_expand<MODE_BWDX>(d_out, d_in, q, g, n, dY, lddy, bits, alpha, nullptr, dX, lddx, dx_dtype,
                                 ws, ws_bytes, stream, expand_ws_bytes(pl, n, d_in), pl);
}

extern "C" bcq_status bcq_linear_bwd_alpha(int d_out, int d_in, int q, int g, int n, const void* dY,
                                           size_t lddy, const void* X, size_t ldx, const uint32_t* bits,
                                           uint32_t plane_mask, float scale, int accumulate,
                                           float* dalpha, void* ws, size_t ws_bytes, void* stream) {
    bcq_status st = check_shape(d_out, d_in, q, g);
    if (st != BCQ_OK) return st;
    if (n < 1) return BCQ_ERR_SHAPE;
    if (!bits || !dalpha) return BCQ_ERR_NULL;
    if ((st = check_act(dY, lddy, d_out)) != BCQ_OK) return st;
    if ((st = check_act(X, ldx, d_in)) != BCQ_OK) return st;
    if (!aligned16(bits)) return BCQ_ERR_ALIGN;
    plane_mask &= (1u << q) - 1u;
    if (plane_mask == 0) return BCQ_OK;
    const DalphaPlan pl = plan_dalpha(d_out, d_in, g, n);
    const size_t need = dalpha_ws_bytes(pl, d_out, q);
    if (ws == nullptr) return BCQ_ERR_NULL;
    if (ws_bytes < need) return BCQ_ERR_WORKSPACE;
    if (!aligned16(ws)) return BCQ_ERR_ALIGN;

    CUtensorMap tm_dy, tm_x;
    if ((st = make_tmap(&tm_dy, dY, d_out, n, lddy, 64)) != BCQ_OK) return st;
    if ((st = make_tmap(&tm_x, X, d_in, n, ldx, 64)) != BCQ_OK) return st;
    DalphaParams p;
    p.d_out = d_out; p.d_in = d_in; p.q = q; p.g = g;
    p.G = (int)bcq_num_groups(d_in, g);
    p.pitch = (int)bcq_pitch_words(d_in);
    p.n = n; p.num_kb = pl.num_kb; p.kb_per_split = pl.kb_per_split; p.splits = pl.splits;
    p.n_subtiles = pl.n_subtiles; p.slots = pl.slots; p.plane_mask = plane_mask;
    p.bits = bits; p.partial = reinterpret_cast<float*>(ws);
    cudaStream_t s = (cudaStream_t)stream;
    dim3 grid((unsigned)pl.m_tiles, (unsigned)pl.n_tiles, (unsigned)pl.splits);
    if (pl.TN == 256) {
        auto kern = dalpha_kernel<256, stages_for<256>()>;
        BCQ_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          (int)smem_for<256>()));
        kern<<<grid, kThreads, smem_for<256>(), s>>>(tm_dy, tm_x, p);
    } else {
        auto kern = dalpha_kernel<128, stages_for<128>()>;
        BCQ_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          (int)smem_for<128>()));
        kern<<<grid, kThreads, smem_for<128>(), s>>>(tm_dy, tm_x, p);
    }
    BCQ_CUDA_TRY(cudaGetLastError());
    const long long total = (long long)q * p.G * d_out;
    dalpha_reduce_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(
        d_out, d_in, q, g, p.G, pl.HN, pl.splits, pl.n_subtiles, pl.slots, plane_mask, scale, accumulate,
        p.partial, dalpha);
    BCQ_CUDA_TRY(cudaGetLastError());
    return BCQ_OK;
}
