// Scale gradient of the BCQ linear layer (Eq. 4):
//     dalpha_i[j, c] = scale * sum_{k in group c} b_i[j,k] * (dY^T X)[j,k].
//
// D[j, k] = sum_t dY[t, j] X[t, k] is a 128 x TN x 64 UMMA tile product with both operands
// MN-major (tokens are the K index; dY and X rows are contiguous in j and k), loaded by TMA in
// 64 x 64 boxes.  The epilogue never writes D: thread = (row j, half of the tile's columns) reads
// its accumulator row from tensor memory 32 columns at a time, applies the signs of every
// requested plane from one 32-bit word of the packed planes, and sums per group.  Partial sums
// (one per split over tokens, column sub-tile and group piece) go to the workspace and a second
// kernel adds them in a fixed order, so the result does not depend on scheduling.  When every
// output has exactly one partial (no token split and a group per column sub-tile, e.g. g = 128)
// the epilogue writes dalpha itself and the second kernel is not launched.
#include "gemm_common.cuh"

namespace {

using namespace bcq;

__device__ int g_timeout_flag = 0;

struct DalphaParams {
    int d_out, d_in, q, g, G, pitch, n;
    int num_kb;          // K blocks of 64 tokens
    int kb_per_split;
    int splits;
    int m_tiles, n_tiles;
    int n_subtiles;      // column sub-tiles of width TN/2 over d_in
    int slots;           // partial slots per sub-tile
    uint32_t plane_mask;
    const uint32_t* bits;
    float* partial;      // [splits][n_subtiles][q][slots][d_out]
    // direct != 0: every output has exactly one partial (no token split, one group per column
    // sub-tile), so the epilogue writes dalpha itself and no second kernel runs
    int direct, accumulate;
    float scale;
    float* dalpha;       // [q][d_out][G]
};


// ------------------------------------------------------------------------------------------
// dalpha: D[j, k] = sum_t dY[t, j] X[t, k], sign-weighted group sums in the epilogue
// ------------------------------------------------------------------------------------------

// Persistent: every CTA walks over (row tile, column tile, token split) tiles; two accumulators
// in tensor memory, so the sign-and-sum epilogue of one tile runs under the main loop of the next.
//   warp 0      TMA producer (dY and X boxes of every K block of 64 tokens)
//   warp 1      UMMA issuer, owner of the tensor-memory allocation
//   warps 2..9  epilogue: thread = (row j, half of the tile's columns)
template <int TN, int STAGES>
__global__ void __launch_bounds__(kThreads, 1)
dalpha_kernel(const __grid_constant__ CUtensorMap tmap_dy, const __grid_constant__ CUtensorMap tmap_x,
              const DalphaParams p) {
    constexpr uint32_t kBBytes = TN * kBlockK * 2;
    constexpr uint32_t kStageBytes = kABytes + kBBytes;
    constexpr int HN = TN / 2;
    constexpr int NCH = HN / 32;
    constexpr uint32_t kAccCols = TmemCols<TN>::value;
    constexpr uint32_t kTmemCols = 2 * kAccCols;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
    const uint32_t ctl_base = smem_base + STAGES * kStageBytes;
    uint8_t* ctl_gen = smem_gen + STAGES * kStageBytes;

    Ctl ctl;
    ctl.full = ctl_base;
    ctl.aready = 0;
    ctl.empty = ctl_base + 8 * STAGES;
    ctl.accum = ctl_base + 16 * STAGES;         // + 8c : accumulator c complete
    const uint32_t acc_empty = ctl.accum + 16;  // + 8c : accumulator c drained
    ctl.spare = ctl.accum + 32;
    volatile uint32_t* tmem_holder = reinterpret_cast<volatile uint32_t*>(ctl_gen + 16 * STAGES + 40);
    ctl.abort_flag = reinterpret_cast<volatile int*>(ctl_gen + 16 * STAGES + 44);
    ctl.device_flag = &g_timeout_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int num_tiles = p.m_tiles * p.n_tiles * p.splits;
    // row tile fastest: CTAs running together share the X boxes of a column tile in L2
    auto tile_coords = [&](int tile, int& j0, int& k0, int& z, int& kb_begin, int& iters) {
        const int mt = tile % p.m_tiles;
        const int rest = tile / p.m_tiles;
        j0 = mt * kBlockM;
        k0 = (rest % p.n_tiles) * TN;
        z = rest / p.n_tiles;
        kb_begin = z * p.kb_per_split;
        iters = min(p.num_kb, kb_begin + p.kb_per_split) - kb_begin;
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(ctl.full + 8 * s, 1);
            ptx::mbar_init(ctl.empty + 8 * s, 1);
        }
        for (int c = 0; c < 2; ++c) {
            ptx::mbar_init(ctl.accum + 8 * c, 1);
            ptx::mbar_init(acc_empty + 8 * c, kWorkerWarps);
        }
        ptx::mbar_init(ctl.spare, 1);
        *ctl.abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tmap_dy);
        ptx::prefetch_tmap(&tmap_x);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(const_cast<uint32_t*>(tmem_holder)), kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_holder;

    if (warp == 0) {
        if (lane == 0) {
            bool ok = true;
            int s = 0, in_flight = 0;
            uint32_t ph = 0;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                int j0, k0, z, kb_begin, iters;
                tile_coords(tile, j0, k0, z, kb_begin, iters);
                // a column tile that reaches past d_in brings (and multiplies) only the 64-column
                // blocks that hold columns of the matrix
                const int boxes = min(TN / 64, (p.d_in - k0 + 63) / 64);
                for (int it = 0; it < iters; ++it) {
                    ok = wait_bar(ctl.empty + 8 * s, ph ^ 1u, ctl, 11);
                    if (!ok) break;
                    const uint32_t sa = smem_base + s * kStageBytes;
                    const int tok = (kb_begin + it) * kBlockK;
                    ptx::mbar_arrive_expect_tx(ctl.full + 8 * s, kABytes + (uint32_t)boxes * 8192u);
                    // A: two blocks of 64 rows j (inner) x 64 tokens; B: TN/64 blocks of 64 k x 64 tokens
                    ptx::tma_load_2d(sa, &tmap_dy, j0, tok, ctl.full + 8 * s);
                    ptx::tma_load_2d(sa + 8192, &tmap_dy, j0 + 64, tok, ctl.full + 8 * s);
#pragma unroll
                    for (int b = 0; b < TN / 64; ++b)
                        if (b < boxes) ptx::tma_load_2d(sa + kABytes + b * 8192, &tmap_x, k0 + b * 64, tok, ctl.full + 8 * s);
                    in_flight = min(in_flight + 1, STAGES);
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
            }
            if (!ok) {
                int bs = s;
                uint32_t bph = ph;
                for (int i = 0; i < in_flight; ++i) {
                    if (bs == 0) { bs = STAGES; bph ^= 1u; }
                    --bs;
                    wait_bar(ctl.full + 8 * bs, bph, ctl, 12);
                }
            }
        }
    } else if (warp == 1) {
        // One elected thread runs the whole loop: between two stages it has a barrier check, a
        // fence, four UMMAs and a commit to get through in less time than the tensor core needs
        // for a stage, so nothing warp-wide (election, reconvergence) is left inside the loop.
        if (ptx::elect_one()) {
            bool ok = true;
            int s = 0, lt = 0;
            uint32_t ph = 0;
            // descriptor halves (128-byte swizzle, MN-major: leading offset 8192 B between blocks of 64
            // rows, stride 1024 B between groups of eight token lines); a UMMA steps the start by 2048 B
            constexpr uint32_t kHi = (1024u >> 4) | (1u << 14) | (2u << 29);
            constexpr uint32_t kLoExtra = (8192u >> 4) << 16;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++lt) {
                int j0, k0, z, kb_begin, iters;
                tile_coords(tile, j0, k0, z, kb_begin, iters);
                const int acc = lt & 1;
                ok = wait_bar(acc_empty + 8 * acc, (uint32_t)((lt >> 1) & 1) ^ 1u, ctl, 17);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + (uint32_t)acc * kAccCols;
                const int boxes = min(TN / 64, (p.d_in - k0 + 63) / 64);
                const uint32_t idesc = ptx::make_idesc_bf16(kBlockM, boxes * 64, 1, 1);  // the UMMA is as wide as the tile's columns
                for (int it = 0; it < iters; ++it) {
                    ok = wait_bar(ctl.full + 8 * s, ph, ctl, 13, 32u);
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    const uint32_t a_lo = (((smem_base + (uint32_t)s * kStageBytes) >> 4) & 0x3FFFu) | kLoExtra;
                    const uint32_t b_lo = a_lo + (kABytes >> 4);
#pragma unroll
                    for (int kk = 0; kk < kBlockK / 16; ++kk)
                        ptx::umma_f16_halves(d_tmem, a_lo + kk * (2048u >> 4), kHi, b_lo + kk * (2048u >> 4), kHi, idesc,
                                             (it > 0 || kk > 0) ? 1u : 0u);
                    ptx::umma_commit(ctl.empty + 8 * s);
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
                if (ok) ptx::umma_commit(ctl.accum + 8 * acc);
            }
            if (!ok) {
                ptx::umma_commit(ctl.spare);
                wait_bar(ctl.spare, 0, ctl, 15);
            }
        }
        __syncwarp();
    } else {
        // ---------------- epilogue: thread = (row j, HN columns of the tile)
        const int quarter = warp & 3;
        const int half = (warp - kWorkerWarp0) >> 2;
        const long long plane_words = (long long)p.d_out * p.pitch;
        bool ok = true;
        int lt = 0;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++lt) {
            int j0, k0, z, kb_begin, iters;
            tile_coords(tile, j0, k0, z, kb_begin, iters);
            const int acc = lt & 1;
            const int j = j0 + quarter * 32 + lane;
            const bool j_ok = j < p.d_out;
            const int kbase = k0 + half * HN;
            const int subtile = (k0 / TN) * 2 + half;

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

            ok = wait_bar(ctl.accum + 8 * acc, (uint32_t)(lt >> 1) & 1u, ctl, 16, 512u);
            if (!ok) break;
            ptx::tc_fence_after_sync();
            if (kbase < p.d_in) {
                const int c_first = min(kbase / p.g, p.G - 1);
                float accs[BCQ_MAX_Q];
#pragma unroll
                for (int i = 0; i < BCQ_MAX_Q; ++i) accs[i] = 0.0f;
                int cur_c = c_first;
                auto flush = [&](int c) {
                    if (!j_ok) return;
                    const int slot = c - c_first;
#pragma unroll
                    for (int i = 0; i < BCQ_MAX_Q; ++i) {
                        if (i < p.q && ((p.plane_mask >> i) & 1u)) {
                            if (p.direct) {
                                float* dst = p.dalpha + ((long long)i * p.d_out + j) * p.G + c;
                                *dst = p.accumulate ? (*dst + p.scale * accs[i]) : (p.scale * accs[i]);
                            } else {
                                const long long idx =
                                    ((((long long)z * p.n_subtiles + subtile) * p.q + i) * p.slots + slot) * p.d_out + j;
                                p.partial[idx] = accs[i];
                            }
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
                            for (int i = 0; i < BCQ_MAX_Q; ++i) accs[i] = 0.0f;
                        }
                        uint32_t v[32];
                        ptx::tmem_ld_x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)acc * kAccCols +
                                             (uint32_t)(half * HN + ch * 32), v);
                        ptx::tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < BCQ_MAX_Q; ++i) {
                            if (i < p.q && ((p.plane_mask >> i) & 1u)) {
                                const uint32_t w = nw[ch][i];
                                float sum = 0.0f;
#pragma unroll
                                for (int b = 0; b < 32; ++b)
                                    sum += __uint_as_float(v[b] ^ ((w << (31 - b)) & 0x80000000u));
                                accs[i] += sum;
                            }
                        }
                    }
                }
                flush(cur_c);
            }
            // the accumulator may be overwritten by the tile after next
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(acc_empty + 8 * acc);
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}

// dalpha[i][j][c] (+)= scale * sum over splits and over the sub-tiles that meet group c.
// Block = 32 consecutive rows j x 8 parts: part y adds every 8th partial of its output (so that
// eight loads per output are in flight at once), then the eight sums are added in order 0..7.
__global__ void __launch_bounds__(256)
dalpha_reduce_kernel(int d_out, int d_in, int q, int g, int G, int HN, int splits, int n_subtiles, int slots,
                     uint32_t plane_mask, float scale, int accumulate, const float* __restrict__ partial,
                     float* __restrict__ dalpha) {
    __shared__ float sums[8][32];
    const int jx = threadIdx.x & 31, part = threadIdx.x >> 5;
    const int jblocks = (d_out + 31) / 32;
    const int jb = blockIdx.x % jblocks;
    const int r = blockIdx.x / jblocks;  // (plane, group)
    const int c = r % G;
    const int i = r / G;
    const int j = jb * 32 + jx;
    if (!((plane_mask >> i) & 1u)) return;  // uniform in the block
    const int k_lo = c * g;
    const int k_hi = min(k_lo + g, d_in) - 1;
    const int st_lo = k_lo / HN, st_n = k_hi / HN - st_lo + 1;
    const int total = splits * st_n;
    float s = 0.0f;
    if (j < d_out) {
        for (int e = part; e < total; e += 8) {
            const int z = e / st_n, st = st_lo + (e - z * st_n);
            const int slot = c - min((st * HN) / g, G - 1);
            s += __ldg(partial + ((((long long)z * n_subtiles + st) * q + i) * slots + slot) * d_out + j);
        }
    }
    sums[part][jx] = s;
    __syncthreads();
    if (part == 0 && j < d_out) {
        float t = 0.0f;
#pragma unroll
        for (int y = 0; y < 8; ++y) t += sums[y][jx];
        float* dst = dalpha + ((long long)i * d_out + j) * G + c;
        *dst = accumulate ? (*dst + scale * t) : (scale * t);
    }
}

struct DalphaPlan {
    int TN, HN, splits, kb_per_split, num_kb, m_tiles, n_tiles, n_subtiles, slots;
};

DalphaPlan plan_dalpha(int d_out, int d_in, int g, int n) {
    DalphaPlan pl;
    const int sms = sm_count();
    pl.m_tiles = ceil_div(d_out, kBlockM);
    pl.num_kb = ceil_div(n, kBlockK);
    // The UMMA-issuing thread needs about 0.3 us per 64-token stage whatever the tile width, more
    // than a 128 x 128 x 64 UMMA group takes to execute, so wide tiles (and a token split when
    // they do not fill the SMs) beat twice as many narrow ones.
    pl.TN = (d_in <= 128) ? 128 : 256;
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


template <int TN>
constexpr int stages_for() {
    return TN == 256 ? 4 : 6;
}

template <int TN>
constexpr size_t smem_for() {
    return (size_t)stages_for<TN>() * (kABytes + TN * kBlockK * 2) + 1024 + 256;
}

size_t dalpha_ws_bytes(const DalphaPlan& pl, int d_out, int q) {
    return (size_t)pl.splits * pl.n_subtiles * q * pl.slots * d_out * sizeof(float);
}

}  // namespace

namespace bcq {
bcq_status dalpha_timeout_flag(int* flag_out, int reset) {
    int v = 0;
    BCQ_CUDA_TRY(cudaMemcpyFromSymbol(&v, g_timeout_flag, sizeof(int)));
    *flag_out = v;
    if (reset && v != 0) {
        const int zero = 0;
        BCQ_CUDA_TRY(cudaMemcpyToSymbol(g_timeout_flag, &zero, sizeof(int)));
    }
    return BCQ_OK;
}

size_t bwd_alpha_workspace_bytes(int d_out, int d_in, int q, int g, int n) {
    return dalpha_ws_bytes(plan_dalpha(d_out, d_in, g, n), d_out, q);
}
}  // namespace bcq

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
    if ((st = make_tmap_16bit(&tm_dy, dY, 0, d_out, n, lddy, 64)) != BCQ_OK) return st;
    if ((st = make_tmap_16bit(&tm_x, X, 0, d_in, n, ldx, 64)) != BCQ_OK) return st;
    DalphaParams p;
    p.d_out = d_out; p.d_in = d_in; p.q = q; p.g = g;
    p.G = (int)bcq_num_groups(d_in, g);
    p.pitch = (int)bcq_pitch_words(d_in);
    p.n = n; p.num_kb = pl.num_kb; p.kb_per_split = pl.kb_per_split; p.splits = pl.splits;
    p.m_tiles = pl.m_tiles; p.n_tiles = pl.n_tiles;
    p.n_subtiles = pl.n_subtiles; p.slots = pl.slots; p.plane_mask = plane_mask;
    p.bits = bits; p.partial = reinterpret_cast<float*>(ws);
    p.direct = (pl.splits == 1 && g == pl.HN) ? 1 : 0;
    p.accumulate = accumulate; p.scale = scale; p.dalpha = dalpha;
    cudaStream_t s = (cudaStream_t)stream;
    // persistent, one CTA per SM; every CTA gets the same number of tiles (as many as the busiest
    // would get anyway), which leaves whole SMs to other kernels instead of a ragged last wave
    const int tiles = pl.m_tiles * pl.n_tiles * pl.splits;
    const int per_cta = ceil_div(tiles, sm_count());
    const unsigned grid = (unsigned)ceil_div(tiles, per_cta);
    if (pl.TN == 256) {
        auto kern = dalpha_kernel<256, stages_for<256>()>;
        if ((st = ensure_dynamic_smem(kern, smem_for<256>())) != BCQ_OK) return st;
        kern<<<grid, kThreads, smem_for<256>(), s>>>(tm_dy, tm_x, p);
    } else {
        auto kern = dalpha_kernel<128, stages_for<128>()>;
        if ((st = ensure_dynamic_smem(kern, smem_for<128>())) != BCQ_OK) return st;
        kern<<<grid, kThreads, smem_for<128>(), s>>>(tm_dy, tm_x, p);
    }
    bcq::count_launch();
    BCQ_CUDA_TRY(cudaGetLastError());
    if (p.direct) return BCQ_OK;
    const long long rblocks = (long long)q * p.G * ((d_out + 31) / 32);
    dalpha_reduce_kernel<<<(unsigned)rblocks, 256, 0, s>>>(
        d_out, d_in, q, g, p.G, pl.HN, pl.splits, pl.n_subtiles, pl.slots, plane_mask, scale, accumulate,
        p.partial, dalpha);
    bcq::count_launch();
    BCQ_CUDA_TRY(cudaGetLastError());
    return BCQ_OK;
}
