// Decode (1..16 tokens) from a packed copy of the frozen weights: bcq_decode_pack and
// bcq_linear_decode_packed.
//
// Decode streams every weight once and uses it for at most 16 tokens, so the time is set by how
// cheaply a weight gets from its bits into a tensor-core operand (Section "Inference Speed": the
// cost of a small-batch layer is moving its weights).  B and, at inference, alpha are frozen, so
// everything that does not depend on the activations is done once, when the pack is written:
//
//   codes   for every weight the index of its level among the 2^q sums +-alpha_1 .. +-alpha_q of
//           its (row, group), as a 4-bit selector nibble for PRMT, eight consecutive weights per
//           32-bit word (q = 4: three index bits, mirrored when b_4 = -1, plus a sign flag; q = 3:
//           the fourth selector word of 32 weights is spread over the spare bit of the other
//           three; q = 2, 1: two or four selector words share a stored word).  q bits per weight,
//           as in the canonical planes.
//   tables  for every (row, group) the eight fp16 levels as the byte-wise lookup table the
//           workers keep in four registers (16 bytes = the four fp32 scales they replace at
//           q = 4), pre-multiplied by a power of two per row that brings q * max|alpha| of the
//           row to [2^13, 2^14).
//
// Both are stored in the order the kernel consumes them: per 128-row tile and per 128-wide step
// along d_in one contiguous chunk, fetched with a single bulk copy into a shared-memory ring.
//
// The kernel is persistent, one CTA per SM.  The (row tile, k step) units of the whole matrix are
// dealt to the CTAs as contiguous, equally long ranges, so the SMs finish together whatever the
// shape.  A range that ends inside a row tile leaves a partial sum: it goes to the workspace, and
// the last CTA to arrive at a tile (a counter in the pack) adds the tile's partial sums in a fixed
// order and writes Y.  No CTA ever waits for another.
//
//   warps 0..3    epilogue: accumulator rows -> Y or partial sums (warp w reads tensor-memory
//                 lanes 32w .. 32w + 31)
//   warp 4        UMMA issuer, owner of the tensor-memory allocation (two accumulators)
//   warps 5, 6    producers: bulk copies of the code chunks / of the table chunks
//   warp 7        only helps with the activation scan at the start
//   warps 8..23   workers, all on the same step: a thread expands 32 weights of one row (selector
//                 words and table from shared memory, PRMT lookups, four 16-byte stores into the
//                 swizzled A operand slot) and writes 4 of the step's activations as fp16
//                 (per-token power of two) into the B operand slot.  Working on one step
//                 together, the workers wait only when the memory or the tensor core is behind.
//
// The kernel may start while the previous kernel of the stream is finishing (programmatic
// dependent launch): the weights are frozen, so the copies and the expansion of the first
// operand slots run before the grid dependency wait; the activations and every global write
// come after it.
#include <algorithm>

#include "gemm_common.cuh"
#include "lut.cuh"

namespace {

using namespace bcq;

__device__ int g_timeout_flag = 0;

constexpr int kDpThreads = 768;
constexpr int kDpEpiWarps = 4;
constexpr int kDpMmaWarp = 4;
constexpr int kDpProdWarp0 = 5;  // 5: codes, 6: tables
constexpr int kDpXWarp = 7;
constexpr int kDpWorkerWarp0 = 8;
constexpr int kDpWorkerWarps = 16;
constexpr int kDpScanWarps = 21;  // every warp but the UMMA issuer and the producers
constexpr int kDpStepK = 128;     // weights of a row per step: two 64-wide UMMA K blocks
constexpr int kDpTN = 16;
constexpr int kDpASlots = 4;
constexpr uint32_t kDpABytes = 2 * kABytes;             // 32 KiB: two 128 x 64 fp16 tiles
constexpr uint32_t kDpBBytes = 2 * kDpTN * 128;         // 4 KiB: two 16 x 64 fp16 tiles
constexpr uint32_t kDpTableBytes = 128 * 16;            // one table chunk: 128 rows x 16 bytes
constexpr uint32_t kDpCtlBytes = 512;
constexpr uint32_t kDpTmemCols = 64;                    // two accumulators of 32 columns
constexpr int kDpMaxRing = 8;

// ------------------------------------------------------------------------------------------
// pack layout (host and device)
// ------------------------------------------------------------------------------------------

struct PackLayout {
    int m_tiles, steps, Q, parts, G;
    uint32_t code_bytes;  // codes of one unit: 128 rows x 128 weights x q bits
    size_t off_cnt, off_rinv, off_tables, off_codes, total;
};

__host__ __device__ inline int dp_parts(int d_in, int g, int G) {
    if (G == 1 || g % 128 == 0) return 1;
    if (g % 64 == 0) return 2;
    return 4;
}

PackLayout pack_layout(int d_out, int d_in, int q, int g) {
    PackLayout L;
    L.m_tiles = ceil_div(d_out, 128);
    L.steps = ceil_div(d_in, kDpStepK);
    L.Q = q;
    L.G = (int)bcq_num_groups(d_in, g);
    L.parts = dp_parts(d_in, g, L.G);
    L.code_bytes = (uint32_t)q * 2048u;
    L.off_cnt = 0;
    L.off_rinv = align_up((size_t)L.m_tiles * 4, 128);
    L.off_tables = align_up(L.off_rinv + (size_t)L.m_tiles * 128 * 4, 128);
    L.off_codes = align_up(L.off_tables + (size_t)L.m_tiles * L.G * kDpTableBytes, 128);
    L.total = L.off_codes + (size_t)L.m_tiles * L.steps * L.code_bytes;
    return L;
}

// ------------------------------------------------------------------------------------------
// writing the pack
// ------------------------------------------------------------------------------------------

// One thread per weight row: the power of two of the row and its inverse.
__global__ void pack_rowscale_kernel(int d_out, int q, int G, int rows_padded, const float* __restrict__ alpha,
                                     float* __restrict__ rinv) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= rows_padded) return;
    float inv = 1.0f;
    if (j < d_out) {
        uint32_t am = 0u;
        for (int i = 0; i < q; ++i)
            for (int c = 0; c < G; ++c)
                am = max(am, __float_as_uint(__ldg(alpha + ((long long)i * d_out + j) * G + c)) & 0x7FFFFFFFu);
        inv = pow2f(-shift_for(exponent_of_bits(__float_as_uint(__uint_as_float(am) * (float)q)), 13));
    }
    rinv[j] = inv;
}

// One thread per (row tile, group, row): the lookup table of the row's levels in that group.
__global__ void pack_tables_kernel(int d_out, int q, int G, int m_tiles, const float* __restrict__ alpha,
                                   const float* __restrict__ rinv, uint4* __restrict__ tables) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)m_tiles * G * 128) return;
    const int row = (int)(idx & 127);
    const int c = (int)((idx >> 7) % G);
    const int mt = (int)((idx >> 7) / G);
    const int j = mt * 128 + row;
    uint4 out = make_uint4(0u, 0u, 0u, 0u);  // rows past d_out expand to zeros
    if (j < d_out) {
        const float wscale = 1.0f / __ldg(rinv + j);  // a power of two
        float a[4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
            a[i] = (i < q) ? __ldg(alpha + ((long long)i * d_out + j) * G + c) * wscale : 0.0f;
        const Lut t = build_lut(a[0], a[1], a[2], a[3]);  // q <= 3: a[3] = 0 is the base
        out = make_uint4(t.tl0, t.tl1, t.th0, t.th1);
    }
    tables[idx] = out;
}

// One thread per (unit, quarter of the step, row): the selector words of 32 weights.
//   selector word r, nibble e  <->  weight 8r + e of the 32;  nibble = level index (bit i <=> b_i =
//   +1), for q = 4 the index of (b_1..b_3) mirrored when b_4 = -1 and bit 3 set in that case.
__global__ void pack_codes_kernel(int d_out, int pitch, int q, int m_tiles, int steps,
                                  const uint32_t* __restrict__ bits, uint32_t* __restrict__ codes) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long total = (long long)m_tiles * steps * 512;
    if (idx >= total) return;
    const int row = (int)(idx & 127);
    const int qd = (int)((idx >> 7) & 3);
    const long long unit = idx >> 9;
    const int st = (int)(unit % steps);
    const int mt = (int)(unit / steps);
    const int j = mt * 128 + row;
    const int word = st * 4 + qd;  // 32-weight block of the row: k = 128 st + 32 qd
    uint32_t w[4] = {0u, 0u, 0u, 0u};
    const bool valid = (j < d_out) && (word < pitch);
    for (int i = 0; i < q; ++i)
        if (valid) w[i] = __ldg(bits + ((long long)i * d_out + j) * pitch + word);
    uint32_t S[4];
    selectors_from_planes(w, q, S);
    if (!valid)
        for (int r = 0; r < 4; ++r) S[r] = 0u;
    uint32_t* dst = codes + idx * q;  // [unit][quarter][row][q words]
    switch (q) {
        case 4: pack_selectors<4>(S, dst); break;
        case 3: pack_selectors<3>(S, dst); break;
        case 2: pack_selectors<2>(S, dst); break;
        default: pack_selectors<1>(S, dst); break;
    }
}

// ------------------------------------------------------------------------------------------
// the decode kernel
// ------------------------------------------------------------------------------------------

struct DecPackedParams {
    int d_out, d_in, q, g, G, n;
    int m_tiles, steps, parts, ring;
    int slots_max;                 // partial-sum slots per row tile in the workspace
    int per, rem;                  // units per CTA and remainder (see range_begin)
    uint32_t code_bytes, chunk_bytes;
    const __nv_bfloat16* X;
    long long ldx;
    const uint8_t* codes;
    const uint8_t* tables;
    const float* rinv;
    unsigned int* counters;
    const float* bias;
    void* out;
    long long ldo;
    int out_bf16;
    float* partial;                // [m_tiles][slots_max][n][128]
};

// `units` units dealt to the CTAs as contiguous ranges: with per = units / ctas and rem = units %
// ctas, CTA c takes per + 1 units if c < rem, else per; its first unit is c * per + min(c, rem).
__host__ __device__ inline int range_begin(int c, int per, int rem) { return c * per + (c < rem ? c : rem); }
// The CTA whose range holds unit u.
__host__ __device__ inline int unit_owner(int u, int per, int rem) {
    const int big = rem * (per + 1);
    return u < big ? u / (per + 1) : rem + (u - big) / per;
}

__device__ __forceinline__ uint32_t max_mag_bf16x8_masked(const uint4& x, int k0, int K) {
    const uint32_t xs[4] = {x.x, x.y, x.z, x.w};
    uint32_t m = 0u;
#pragma unroll
    for (int e = 0; e < 8; ++e)
        if (k0 + e < K) m = max(m, (xs[e >> 1] >> ((e & 1) * 16)) & 0x7FFFu);
    return m;
}

template <int Q>
__global__ void __launch_bounds__(kDpThreads, 1)
decode_packed_kernel(const DecPackedParams p) {
    constexpr uint32_t kIdesc = ptx::make_idesc_bf16(kBlockM, kDpTN, 0, 0) & ~((1u << 7) | (1u << 10));  // fp16 x fp16

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
    const int RING = p.ring;
    const uint32_t a_base = smem_base;                                   // kDpASlots x 32 KiB
    const uint32_t b_base = a_base + kDpASlots * kDpABytes;              // kDpASlots x 4 KiB
    const uint32_t ring_base = b_base + kDpASlots * kDpBBytes;           // RING x chunk_bytes
    const uint32_t ctl_base = ring_base + (uint32_t)RING * p.chunk_bytes;
    uint8_t* ctl_gen = smem_gen + (ctl_base - smem_base);

    Ctl ctl;
    ctl.full = ctl_base;                        // + 8r : chunk r of the ring has landed
    const uint32_t wempty = ctl_base + 64;      // + 8r : its worker group has read it
    ctl.aready = ctl_base + 128;                // + 8a : both operands of slot a are written
    ctl.empty = ctl_base + 160;                 // + 8a : the UMMAs reading slot a are done
    ctl.accum = ctl_base + 192;                 // + 8c : accumulator c complete
    const uint32_t acc_empty = ctl_base + 208;  // + 8c : accumulator c drained
    ctl.spare = ctl_base + 224;
    volatile uint32_t* tmem_holder = reinterpret_cast<volatile uint32_t*>(ctl_gen + 232);
    ctl.abort_flag = reinterpret_cast<volatile int*>(ctl_gen + 236);
    ctl.device_flag = &g_timeout_flag;
    volatile int* last_flag = reinterpret_cast<volatile int*>(ctl_gen + 240);
    uint32_t* tok_max = reinterpret_cast<uint32_t*>(ctl_gen + 256);  // [16] bit patterns of bf16 magnitudes

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    // this CTA's range of units; unit u = (row tile u / steps, k step u % steps)
    const int u_begin = range_begin((int)blockIdx.x, p.per, p.rem);
    const int T = p.per + ((int)blockIdx.x < p.rem ? 1 : 0);
    const int mt0 = u_begin / p.steps;
    const int st0 = u_begin - mt0 * p.steps;

    // ---------------- prologue.  Nothing below the two requests that follow depends on anything but
    // the kernel's arguments, so they go out first and their latency hides the set-up:
    //   * the producers initialise the ring's barriers themselves and start copying at once;
    //   * every other warp but the UMMA issuer requests its share of the activations for the
    //     per-token scale (largest magnitude over the k range this CTA touches).
    // The kernel is launched so that it may start while the kernel before it in the stream is
    // still finishing (and lets its own successor do the same): the weights are frozen, so the
    // producers' first copies need not wait; everything that may depend on the previous kernel --
    // the activations, and every global write -- comes after the grid dependency wait below.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const bool scanner = (warp != kDpMmaWarp && warp != kDpProdWarp0 && warp != kDpProdWarp0 + 1);
    const int pw = (warp < kDpEpiWarps) ? warp : (warp == kDpXWarp ? kDpEpiWarps : warp - 3);  // 0..20
    const int cnt = min(T, p.steps);  // steps touched, starting at st0 and wrapping
    const int nchunks = cnt * 16;     // 16-byte pieces of one token's range
    const int items = p.n * nchunks;  // (token, piece) pairs, token-major
    constexpr int kScanRound = kDpScanWarps * 32 * 4;
    uint4 sx[4];
    int sk[4], stok[4];
    auto scan_request = [&](int base) {
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int idx = base + (r * kDpScanWarps + pw) * 32 + lane;
            stok[r] = idx / nchunks;
            const int ci = idx - stok[r] * nchunks;
            int st = st0 + (ci >> 4);
            if (st >= p.steps) st -= p.steps;
            sk[r] = st * kDpStepK + (ci & 15) * 8;
            sx[r] = (idx < items && sk[r] < p.d_in)
                        ? __ldg(reinterpret_cast<const uint4*>(p.X + (long long)stok[r] * p.ldx + sk[r]))
                        : make_uint4(0u, 0u, 0u, 0u);
            if (idx >= items) stok[r] = -1;
        }
    };
    auto scan_reduce = [&]() {
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            uint32_t m = max_mag_bf16x8_masked(sx[r], sk[r], p.d_in);
            // a warp's 32 consecutive pieces belong to one token, or to two at a boundary
            const int t_lo = __shfl_sync(0xffffffffu, stok[r], 0);
            if (__all_sync(0xffffffffu, stok[r] == t_lo)) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
                if (lane == 0 && t_lo >= 0) atomicMax(&tok_max[t_lo], m);
            } else if (stok[r] >= 0) {
                atomicMax(&tok_max[stok[r]], m);
            }
        }
    };

    if (warp == kDpProdWarp0) {
        if (lane < RING) {
            ptx::mbar_init(ctl.full + 8 * lane, 1 + p.parts);
            ptx::mbar_init(wempty + 8 * lane, kDpWorkerWarps);
        } else if (lane == 31) {
            *ctl.abort_flag = 0;
        }
        ptx::fence_mbar_init();
    }
    if (warp == kDpProdWarp0 || warp == kDpProdWarp0 + 1)
        asm volatile("bar.sync 3, 64;" ::: "memory");  // the ring's barriers exist: both producers may start
    if (warp == 0) {
        if (lane >= 8 && lane < 8 + kDpASlots) {
            ptx::mbar_init(ctl.aready + 8 * (lane - 8), kDpWorkerWarps);
            ptx::mbar_init(ctl.empty + 8 * (lane - 8), 1);
        } else if (lane >= 16 && lane < 18) {
            ptx::mbar_init(ctl.accum + 8 * (lane - 16), 1);
            ptx::mbar_init(acc_empty + 8 * (lane - 16), kDpEpiWarps);
        } else if (lane == 18) {
            ptx::mbar_init(ctl.spare, 1);
        }
        if (lane < 16) tok_max[lane] = 0u;
        ptx::fence_mbar_init();
    }
    if (warp == kDpMmaWarp) {
        ptx::tmem_alloc(ptx::smem_u32(const_cast<uint32_t*>(tmem_holder)), kDpTmemCols);
        ptx::tmem_relinquish();
    }
    uint32_t tmem_base = 0;
    auto cta_ready = [&]() {  // every warp passes here exactly once
        ptx::tc_fence_before_sync();
        __syncthreads();
        ptx::tc_fence_after_sync();
        tmem_base = *tmem_holder;
    };
    // power of two of token t (and its inverse), once the scan is complete
    auto token_shift = [&](int t) { return shift_for(exponent_of_bits(tok_max[t] << 16), 14); };

    // per-token scale: after the grid dependency wait (the activations may come from the previous
    // kernel), every scanner warp takes its share; the workers get here after filling the first
    // operand slots
    auto scan_tokens = [&]() {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        for (int base = 0; base < items; base += kScanRound) {
            scan_request(base);
            scan_reduce();
        }
        asm volatile("bar.sync 1, %0;" ::"n"(kDpScanWarps * 32) : "memory");
    };
    if (scanner) {
        cta_ready();
        if (warp < kDpWorkerWarp0) scan_tokens();
    }

    if (warp == kDpProdWarp0 || warp == kDpProdWarp0 + 1) {
        // ---------------- producers: warp 5 the code chunk of every step, warp 6 its table chunks
        // (lane a = part a).  Each arrives on the chunk's barrier with the bytes it brings.  The
        // first ring of copies needs no wait and leaves before the CTA-wide start.
        const bool codes_role = (warp == kDpProdWarp0);
        const bool active = lane < (codes_role ? 1 : p.parts);
        int r = 0, in_flight = 0, gs = 0;
        uint32_t ph = 0;
        int mt = mt0, st = st0;
        const uint8_t* src = p.codes + (size_t)u_begin * p.code_bytes;
        const int kspan = kDpStepK / p.parts;
        auto issue = [&]() {
            const uint32_t bar = ctl.full + 8 * r;
            const uint32_t dst = ring_base + (uint32_t)r * p.chunk_bytes;
            if (codes_role) {
                ptx::mbar_arrive_expect_tx(bar, p.code_bytes);
                ptx::bulk_load(dst, src, p.code_bytes, bar);
                src += p.code_bytes;
            } else {
                const int c = min((st * kDpStepK + lane * kspan) / p.g, p.G - 1);
                ptx::mbar_arrive_expect_tx(bar, kDpTableBytes);
                ptx::bulk_load(dst + p.code_bytes + lane * kDpTableBytes,
                               p.tables + ((size_t)mt * p.G + c) * kDpTableBytes, kDpTableBytes, bar);
                if (++st == p.steps) { st = 0; ++mt; }
            }
            in_flight = min(in_flight + 1, RING);
            if (++r == RING) { r = 0; ph ^= 1u; }
        };
        // (issuing a bulk copy takes a thread a few hundred cycles, and the whole CTA waits for this
        // warp at the start: two chunks now, the rest of the ring right after)
        if (active)
            for (; gs < min(T, 2); ++gs) issue();
        __syncwarp();
        cta_ready();
        if (active) {
            bool ok = true;
            for (; gs < T; ++gs) {
                if (gs >= RING) {  // the ring's first round needs no wait
                    ok = wait_bar(wempty + 8 * r, ph ^ 1u, ctl, 31);
                    if (!ok) break;
                }
                issue();
            }
            if (!ok) {
                int br = r;
                uint32_t bph = ph;
                for (int i = 0; i < in_flight; ++i) {
                    if (br == 0) { br = RING; bph ^= 1u; }
                    --br;
                    wait_bar(ctl.full + 8 * br, bph, ctl, 32);
                }
            }
        }
    } else if (warp == kDpMmaWarp) {
        // ---------------- UMMA issuer
        cta_ready();
        bool ok = true;
        int a = 0, seg = 0, st = st0;
        uint32_t ph = 0;
        constexpr uint32_t kHi = (1024u >> 4) | (1u << 14) | (2u << 29);  // stride 1024 B, version 1, 128-byte swizzle
        constexpr uint32_t kLoExtra = (16u >> 4) << 16;
        bool first = true;
        for (int gs = 0; gs < T && ok; ++gs) {
            const int acc = seg & 1;
            if (first) {
                ok = wait_bar(acc_empty + 8 * acc, (uint32_t)((seg >> 1) & 1) ^ 1u, ctl, 33);
                if (!ok) break;
                ptx::tc_fence_after_sync();
            }
            ok = wait_bar(ctl.aready + 8 * a, ph, ctl, 34);
            if (!ok) break;
            ptx::tc_fence_after_sync();
            const bool last = (st == p.steps - 1) || (gs == T - 1);
            if (ptx::elect_one()) {
                const uint32_t d_tmem = tmem_base + (uint32_t)acc * 32u;
                const uint32_t a_lo = (((a_base + (uint32_t)a * kDpABytes) >> 4) & 0x3FFFu) | kLoExtra;
                const uint32_t b_lo = (((b_base + (uint32_t)a * kDpBBytes) >> 4) & 0x3FFFu) | kLoExtra;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)  // two K blocks of four 16-wide UMMAs
                    ptx::umma_f16_halves(d_tmem, a_lo + (kk >> 2) * (kABytes >> 4) + (kk & 3) * 2, kHi,
                                         b_lo + (kk >> 2) * ((kDpTN * 128u) >> 4) + (kk & 3) * 2, kHi, kIdesc,
                                         (!first || kk > 0) ? 1u : 0u);
                ptx::umma_commit(ctl.empty + 8 * a);
                if (last) ptx::umma_commit(ctl.accum + 8 * acc);
            }
            __syncwarp();
            first = false;
            if (last) { ++seg; first = true; }
            if (++st == p.steps) st = 0;
            if (++a == kDpASlots) { a = 0; ph ^= 1u; }
        }
        if (!ok) {
            if (ptx::elect_one()) ptx::umma_commit(ctl.spare);
            __syncwarp();
            wait_bar(ctl.spare, 0, ctl, 35);
        }
    } else if (warp >= kDpWorkerWarp0) {
        // ---------------- workers: thread = (row, quarter qd of the step: k offset 32 qd, i.e. K
        // block qd / 2, chunks 4 (qd % 2) .. + 3 of the row's 128-byte line).  The eight lanes that
        // share a shared-memory transaction hold eight consecutive rows of one quarter, so their
        // 16-byte accesses fall on different banks (codes, tables, and the swizzled stores).
        const int wl = warp - kDpWorkerWarp0;           // 0..15
        const int qd = lane >> 3;
        const int row = wl * 8 + (lane & 7);
        const uint32_t line_off = (uint32_t)(qd >> 1) * kABytes + (uint32_t)row * 128u;
        const uint32_t lx = row & 7;
        const uint32_t chunk0 = (uint32_t)(qd & 1) * 4u;
        const uint32_t code_off = (uint32_t)((qd * 128 + row) * Q) * 4u;
        const uint32_t table_off = p.code_bytes + (uint32_t)(qd * p.parts / 4) * kDpTableBytes + (uint32_t)row * 16u;
        // activations (the B operand): 16 tokens x 128 k as fp16, 8 bytes (4 values) per thread:
        // token xt, 16-byte piece xpc of the step (K block xpc / 8), half xh of the piece.  Token
        // rows past n stay zero (written once per slot), columns past d_in are zeros.
        const int xe = wl * 32 + lane;
        const int xt = xe >> 5, xpc = (xe >> 1) & 15, xh = xe & 1;
        const __nv_bfloat16* xrow = p.X + (long long)xt * p.ldx + xpc * 8 + xh * 4;
        const uint32_t x_off = (uint32_t)(xpc >> 3) * (kDpTN * 128u) + (uint32_t)xt * 128u +
                               (uint32_t)(((xpc & 7) ^ (xt & 7)) << 4) + (uint32_t)xh * 8u;
        float xscale = 0.0f;

        bool ok = true;
        int r = 0, a = 0, st = st0;
        uint32_t rph = 0, aph = 0;
        uint2 xv = make_uint2(0u, 0u);
        auto request_x = [&](int step) {
            const int xk = step * kDpStepK + xpc * 8 + xh * 4;
            xv = make_uint2(0u, 0u);
            if (xt < p.n && xk < p.d_in) xv = __ldg(reinterpret_cast<const uint2*>(xrow + step * kDpStepK));
        };
        // A operand of step gs (ring slot r) into operand slot a
        auto expand_step = [&]() {
            ok = wait_bar(ctl.full + 8 * r, rph, ctl, 37);
            if (!ok) return;
            const uint32_t chunk = ring_base + (uint32_t)r * p.chunk_bytes;
            uint32_t v[Q];
            load_codes<Q>(chunk + code_off, v);
            Lut t;
            asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(t.tl0), "=r"(t.tl1), "=r"(t.th0), "=r"(t.th1)
                         : "r"(chunk + table_off) : "memory");
            ok = wait_bar(ctl.empty + 8 * a, aph ^ 1u, ctl, 38);
            if (!ok) return;
            uint32_t S[4];
            selectors<Q>(v, S);
            expand32_codes<Q>(S, t, a_base + (uint32_t)a * kDpABytes + line_off, lx, chunk0);
            // the chunk goes back to the producer only now that what was loaded from it has been
            // consumed: a load that has merely been issued may still be reading shared memory when
            // the next bulk copy (another proxy) overwrites the slot
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(wempty + 8 * r);
            if (++r == RING) { r = 0; rph ^= 1u; }
        };
        // B operand of the step whose activations are in xv, then the slot is complete
        auto finish_step = [&](int step, int gs) {
            if (xt < p.n) {
                const int xk = step * kDpStepK + xpc * 8 + xh * 4;
                float f0 = __uint_as_float(xv.x << 16) * xscale, f1 = __uint_as_float(xv.x & 0xFFFF0000u) * xscale;
                float f2 = __uint_as_float(xv.y << 16) * xscale, f3 = __uint_as_float(xv.y & 0xFFFF0000u) * xscale;
                if (xk + 4 > p.d_in) {
                    if (xk + 1 >= p.d_in) f1 = 0.0f;
                    if (xk + 2 >= p.d_in) f2 = 0.0f;
                    if (xk + 3 >= p.d_in) f3 = 0.0f;
                    if (xk >= p.d_in) f0 = 0.0f;
                }
                asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(b_base + (uint32_t)a * kDpBBytes + x_off),
                             "r"(pack_half2(f0, f1)), "r"(pack_half2(f2, f3)) : "memory");
            } else if (gs < kDpASlots) {
                asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(b_base + (uint32_t)a * kDpBBytes + x_off),
                             "r"(0u), "r"(0u) : "memory");
            }
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ctl.aready + 8 * a);
            if (++a == kDpASlots) { a = 0; aph ^= 1u; }
        };
        auto next_step = [&](int step) { return step + 1 == p.steps ? 0 : step + 1; };

        // before the grid dependency wait: the A operands of the first steps (every slot is free)
        const int early = min(T, kDpASlots);
        for (int gs = 0; gs < early && ok; ++gs) {
            expand_step();
            if (++a == kDpASlots) { a = 0; aph ^= 1u; }
        }
        a = 0;
        aph = 0;
        scan_tokens();
        xscale = pow2f(token_shift(xt));
        {
            // the early steps' activations, all requested at once
            uint2 xq[kDpASlots];
            int sq = st;
#pragma unroll
            for (int gs = 0; gs < kDpASlots; ++gs) {
                xq[gs] = make_uint2(0u, 0u);
                if (gs < early) {
                    request_x(sq);
                    xq[gs] = xv;
                    sq = next_step(sq);
                }
            }
#pragma unroll
            for (int gs = 0; gs < kDpASlots; ++gs) {
                if (gs < early && ok) {
                    xv = xq[gs];
                    finish_step(st, gs);
                    st = next_step(st);
                }
            }
        }
        // steady state: the activations are requested first, the load flies during the waits
        for (int gs = early; gs < T && ok; ++gs) {
            request_x(st);
            expand_step();
            if (!ok) break;
            finish_step(st, gs);
            st = next_step(st);
        }
    } else if (warp < kDpEpiWarps) {
        // ---------------- epilogue warps: one segment (the steps of one row tile inside this CTA's
        // range) at a time
        const int quarter = warp;
        const int row = quarter * 32 + lane;
        bool ok = true;
        int seg = 0, mt = mt0, st = st0;
        for (int gs = 0; gs < T && ok; ++seg) {
            const int len = min(p.steps - st, T - gs);
            const bool whole = (len == p.steps);
            const int acc = seg & 1;
            ok = wait_bar(ctl.accum + 8 * acc, (uint32_t)(seg >> 1) & 1u, ctl, 39, 1024u);
            if (!ok) break;
            ptx::tc_fence_after_sync();
            uint32_t v[16];
            ptx::tmem_ld_x16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)acc * 32u, v);
            ptx::tmem_ld_wait();
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(acc_empty + 8 * acc);
            const int j = mt * 128 + row;
            const float rinv = __ldg(p.rinv + j);
            const float bias = (p.bias != nullptr && j < p.d_out) ? __ldg(p.bias + j) : 0.0f;
            auto store_out = [&](int t, float val) {
                if (j < p.d_out) {
                    if (p.out_bf16)
                        reinterpret_cast<__nv_bfloat16*>(p.out)[(long long)t * p.ldo + j] = __float2bfloat16_rn(val + bias);
                    else
                        reinterpret_cast<float*>(p.out)[(long long)t * p.ldo + j] = val + bias;
                }
            };
            if (whole) {
#pragma unroll
                for (int t = 0; t < 16; ++t)
                    if (t < p.n) store_out(t, __uint_as_float(v[t]) * (rinv * pow2f(-token_shift(t))));
            } else {
                // contributors of this row tile: the CTAs owning its first .. last unit, in order
                const int c_first = unit_owner(mt * p.steps, p.per, p.rem);
                const int c_last = unit_owner(mt * p.steps + p.steps - 1, p.per, p.rem);
                const int count = c_last - c_first + 1;
                float* mine = p.partial + (((size_t)mt * p.slots_max + ((int)blockIdx.x - c_first)) * p.n) * 128 + row;
#pragma unroll
                for (int t = 0; t < 16; ++t)
                    if (t < p.n) mine[(size_t)t * 128] = __uint_as_float(v[t]) * (rinv * pow2f(-token_shift(t)));
                // publish: the barrier orders the four warps' stores before thread 0's fence, and the
                // fence before its arrival at the counter; the last CTA to arrive fences again
                // before any of its threads (ordered by the second barrier) reads the other CTAs' sums
                asm volatile("bar.sync 2, %0;" ::"n"(kDpEpiWarps * 32) : "memory");
                if (threadIdx.x == 0) {
                    __threadfence();
                    const int is_last = (atomicAdd(p.counters + mt, 1u) == (unsigned)(count - 1)) ? 1 : 0;
                    __threadfence();
                    *last_flag = is_last;
                }
                asm volatile("bar.sync 2, %0;" ::"n"(kDpEpiWarps * 32) : "memory");
                if (*last_flag) {
                    const float* base = p.partial + ((size_t)mt * p.slots_max * p.n) * 128 + row;
                    // all tokens' loads of one contributor in flight together; contributors in order
                    float sum[16];
#pragma unroll
                    for (int t = 0; t < 16; ++t) sum[t] = 0.0f;
                    for (int c = 0; c < count; ++c) {
                        float pv[16];
#pragma unroll
                        for (int t = 0; t < 16; ++t)
                            pv[t] = (t < p.n) ? __ldcg(base + ((size_t)c * p.n + t) * 128) : 0.0f;
#pragma unroll
                        for (int t = 0; t < 16; ++t) sum[t] += pv[t];
                    }
#pragma unroll
                    for (int t = 0; t < 16; ++t)
                        if (t < p.n) store_out(t, sum[t]);
                    if (threadIdx.x == 0) p.counters[mt] = 0u;  // ready for the next call
                }
                asm volatile("bar.sync 2, %0;" ::"n"(kDpEpiWarps * 32) : "memory");  // last_flag may be rewritten
            }
            gs += len;
            st += len;
            if (st == p.steps) { st = 0; ++mt; }
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == kDpMmaWarp) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, kDpTmemCols);
    }
}

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------

struct DecPackedPlan {
    int ctas, ring, slots_max, per, rem;
    uint32_t chunk_bytes;
    size_t smem, ws_bytes;
};

DecPackedPlan plan_decode_packed(const PackLayout& L, int n) {
    DecPackedPlan pl;
    const int units = L.m_tiles * L.steps;
    pl.ctas = std::min(sm_count(), units);
    pl.per = units / pl.ctas;
    pl.rem = units % pl.ctas;
    pl.chunk_bytes = L.code_bytes + (uint32_t)L.parts * kDpTableBytes;
    const size_t fixed = 1024 + (size_t)kDpASlots * (kDpABytes + kDpBBytes) + kDpCtlBytes;
    int ring = (int)((232448 - fixed) / pl.chunk_bytes);
    pl.ring = ring > kDpMaxRing ? kDpMaxRing : ring;
    pl.smem = fixed + (size_t)pl.ring * pl.chunk_bytes;
    // most CTAs that can meet in one row tile
    int most = 1;
    for (int mt = 0; mt < L.m_tiles; ++mt) {
        const int c0 = unit_owner(mt * L.steps, pl.per, pl.rem);
        const int c1 = unit_owner(mt * L.steps + L.steps - 1, pl.per, pl.rem);
        most = std::max(most, c1 - c0 + 1);
    }
    pl.slots_max = most;
    pl.ws_bytes = most > 1 ? (size_t)L.m_tiles * most * n * 128 * sizeof(float) : 0;
    return pl;
}

template <int Q>
bcq_status launch_decode_packed(const DecPackedParams& p, const DecPackedPlan& pl, cudaStream_t s) {
    auto kern = decode_packed_kernel<Q>;
    bcq_status st0 = ensure_dynamic_smem(kern, pl.smem);
    if (st0 != BCQ_OK) return st0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)pl.ctas);
    cfg.blockDim = dim3(kDpThreads);
    cfg.dynamicSmemBytes = pl.smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    BCQ_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, p));
    bcq::count_launch();
    BCQ_CUDA_TRY(cudaGetLastError());
    return BCQ_OK;
}

bcq_status check_pack_shape(int d_out, int d_in, int q, int g) {
    bcq_status st = check_shape(d_out, d_in, q, g);
    if (st != BCQ_OK) return st;
    if (q > 4) return BCQ_ERR_UNSUPPORTED;
    return BCQ_OK;
}

}  // namespace

namespace bcq {
bcq_status decode_timeout_flag(int* flag_out, int reset) {
    int v = 0;
    BCQ_CUDA_TRY(cudaMemcpyFromSymbol(&v, g_timeout_flag, sizeof(int)));
    *flag_out = v;
    if (reset && v != 0) {
        const int zero = 0;
        BCQ_CUDA_TRY(cudaMemcpyToSymbol(g_timeout_flag, &zero, sizeof(int)));
    }
    return BCQ_OK;
}

size_t decode_packed_workspace_bytes(int d_out, int d_in, int q, int g, int n) {
    if (check_pack_shape(d_out, d_in, q, g) != BCQ_OK) return 0;
    return plan_decode_packed(pack_layout(d_out, d_in, q, g), n).ws_bytes;
}
}  // namespace bcq

extern "C" size_t bcq_decode_pack_bytes(int d_out, int d_in, int q, int g) {
    if (check_pack_shape(d_out, d_in, q, g) != BCQ_OK) return 0;
    return pack_layout(d_out, d_in, q, g).total;
}

extern "C" bcq_status bcq_decode_pack(int d_out, int d_in, int q, int g, const uint32_t* bits,
                                      const float* alpha, void* pack, size_t pack_bytes, void* stream) {
    bcq_status st = check_pack_shape(d_out, d_in, q, g);
    if (st != BCQ_OK) return st;
    if (!bits || !alpha || !pack) return BCQ_ERR_NULL;
    if (!aligned16(bits) || (reinterpret_cast<uintptr_t>(pack) & 127u) != 0) return BCQ_ERR_ALIGN;
    const PackLayout L = pack_layout(d_out, d_in, q, g);
    if (pack_bytes < L.total) return BCQ_ERR_WORKSPACE;
    cudaStream_t s = (cudaStream_t)stream;
    uint8_t* pk = reinterpret_cast<uint8_t*>(pack);
    BCQ_CUDA_TRY(cudaMemsetAsync(pk + L.off_cnt, 0, L.off_rinv - L.off_cnt, s));
    float* rinv = reinterpret_cast<float*>(pk + L.off_rinv);
    const int rows_padded = L.m_tiles * 128;
    pack_rowscale_kernel<<<ceil_div(rows_padded, 128), 128, 0, s>>>(d_out, q, L.G, rows_padded, alpha, rinv);
    bcq::count_launch();
    BCQ_CUDA_TRY(cudaGetLastError());
    const long long nt = (long long)L.m_tiles * L.G * 128;
    pack_tables_kernel<<<(unsigned)((nt + 255) / 256), 256, 0, s>>>(d_out, q, L.G, L.m_tiles, alpha, rinv,
                                                                   reinterpret_cast<uint4*>(pk + L.off_tables));
    bcq::count_launch();
    BCQ_CUDA_TRY(cudaGetLastError());
    const long long nc = (long long)L.m_tiles * L.steps * 512;
    pack_codes_kernel<<<(unsigned)((nc + 255) / 256), 256, 0, s>>>(d_out, (int)bcq_pitch_words(d_in), q, L.m_tiles,
                                                                  L.steps, bits,
                                                                  reinterpret_cast<uint32_t*>(pk + L.off_codes));
    bcq::count_launch();
    BCQ_CUDA_TRY(cudaGetLastError());
    return BCQ_OK;
}

extern "C" bcq_status bcq_linear_decode_packed(int d_out, int d_in, int q, int g, int n, const void* X,
                                               size_t ldx, void* pack, const float* bias, void* Y, size_t ldy,
                                               int y_dtype, void* ws, size_t ws_bytes, void* stream) {
    bcq_status st = check_pack_shape(d_out, d_in, q, g);
    if (st != BCQ_OK) return st;
    if (n < 1 || n > 16) return BCQ_ERR_SHAPE;
    if (!pack || !Y) return BCQ_ERR_NULL;
    if ((st = check_act(X, ldx, d_in)) != BCQ_OK) return st;
    if (ldy < (size_t)d_out) return BCQ_ERR_SHAPE;
    if (y_dtype != BCQ_F32 && y_dtype != BCQ_BF16) return BCQ_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(pack) & 127u) != 0) return BCQ_ERR_ALIGN;
    const PackLayout L = pack_layout(d_out, d_in, q, g);
    const DecPackedPlan pl = plan_decode_packed(L, n);
    if (pl.ws_bytes > 0) {
        if (ws == nullptr) return BCQ_ERR_NULL;
        if (ws_bytes < pl.ws_bytes) return BCQ_ERR_WORKSPACE;
        if (!aligned16(ws)) return BCQ_ERR_ALIGN;
    }
    uint8_t* pk = reinterpret_cast<uint8_t*>(pack);
    DecPackedParams p;
    p.d_out = d_out; p.d_in = d_in; p.q = q; p.g = g; p.G = L.G; p.n = n;
    p.m_tiles = L.m_tiles; p.steps = L.steps; p.parts = L.parts; p.ring = pl.ring;
    p.slots_max = pl.slots_max;
    p.per = pl.per; p.rem = pl.rem;
    p.code_bytes = L.code_bytes; p.chunk_bytes = pl.chunk_bytes;
    p.X = reinterpret_cast<const __nv_bfloat16*>(X); p.ldx = (long long)ldx;
    p.codes = pk + L.off_codes; p.tables = pk + L.off_tables;
    p.rinv = reinterpret_cast<const float*>(pk + L.off_rinv);
    p.counters = reinterpret_cast<unsigned int*>(pk + L.off_cnt);
    p.bias = bias; p.out = Y; p.ldo = (long long)ldy; p.out_bf16 = (y_dtype == BCQ_BF16);
    p.partial = reinterpret_cast<float*>(ws);
    cudaStream_t s = (cudaStream_t)stream;
    switch (q) {
        case 1: return launch_decode_packed<1>(p, pl, s);
        case 2: return launch_decode_packed<2>(p, pl, s);
        case 3: return launch_decode_packed<3>(p, pl, s);
        default: return launch_decode_packed<4>(p, pl, s);
    }
}
