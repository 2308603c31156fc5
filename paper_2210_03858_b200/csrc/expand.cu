// Forward (Eq. 2), input gradient (Eq. 3) and decode kernels of the BCQ linear layer.
//
//   forward / decode   D[j, t] = sum_k  W_hat[j, k] * X[t, k]
//   dX                 D[k, t] = sum_j  W_hat[j, k] * dY[t, j]
//
// W_hat = sum_i alpha_i b_i (Eq. 1) never exists in global memory: worker warps rebuild it tile by
// tile from the packed planes, straight into the 128-byte-swizzled shared-memory operand layout of
// tcgen05.mma (K-major for the forward, where j is the M index; MN-major for dX, where k is the M
// index and one 128-byte line holds 64 consecutive k of one row j).  Accumulators live in tensor
// memory (128 lanes x TN fp32 columns).
//
// Number format.  A scaled weight rounded to bf16 (8 significant bits) alone already costs about
// 1.7e-3 relative error on the outputs, so both operands are fp16 (11 bits):
//   * the scaled weight takes one of 2^q values per (row, group).  For q <= 4 the workers build
//     a byte-wise lookup table of the fp16 levels in four registers and index it with PRMT: the
//     selector nibbles are the plane bits of four weights, gathered with shifts and masks.  For
//     q = 4 the table holds the eight levels with b_4 = +1; b_4 = -1 mirrors the index and flips
//     the sign.  q > 4 falls back to fp32 sums of +-alpha_i.
//   * activations are bf16 at the interface.  A short pre-pass writes them to the workspace as
//     fp16, each token row multiplied by a power of two that brings its largest magnitude to
//     2^14..2^15 (exact; undone in the epilogue), so neither large activations nor small
//     gradients leave the fp16 range.  The same pre-pass finds max|alpha|, from which a power of
//     two for the weights is derived.  Decode (<= 16 tokens) has no pre-pass: every CTA converts
//     the X slice it needs itself and scales per (token, K-slice) and per weight row.
//   * one PRMT pair emits the weights of a byte of a plane word in the order 0,4,1,5,2,6,3,7.
//     For the forward and dX the pre-pass, which regroups the plane words anyway, stores the bits
//     of every byte as 0,2,4,6,1,3,5,7, so that the expanded tile is in natural k order.  Decode
//     has no pre-pass: there the tile keeps the PRMT order and the workers write the activations
//     in the same order.
#include <mutex>

#include "gemm_common.cuh"
#include "lut.cuh"

namespace {

using namespace bcq;

__device__ int g_timeout_flag = 0;

enum { MODE_FWD = 0, MODE_BWDX = 1 };
enum { QM_LUT3 = 0, QM_LUT4 = 1, QM_GENERIC = 2 };
constexpr int kPrefetch = 3;  // stages between the global loads of a task and its use

// 16 weights of one row (bits 0..15 of the plane words w0..w3) through the lookup table, stored
// as two 16-byte chunks (slots chunk0, chunk0 + 1) of the 128-byte line at `line` (swizzle key
// lx).  Chunk u holds weights 8u..8u+7 in the order 0,4,1,5,2,6,3,7.
template <bool Q4>
__device__ __forceinline__ void expand16_lut(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t w3,
                                             const Lut& t, uint32_t line, uint32_t lx, uint32_t chunk0) {
    uint32_t x0 = w0, x1 = w1, x2 = w2, nf = 0u;
    if (Q4) {
        // b_4 = -1 (bit clear): value = -level[~index]
        nf = ~w3;
        x0 = ~(w0 ^ w3);
        x1 = ~(w1 ^ w3);
        x2 = ~(w2 ^ w3);
    }
    constexpr uint32_t M = 0x11111111u;
    uint32_t R[4][2];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        // nibble n of S = 3-bit level index of weight 4n + r
        const uint32_t a = x0 >> r;
        const uint32_t b = (r >= 1) ? (x1 >> (r >= 1 ? r - 1 : 0)) : (x1 << 1);
        const uint32_t c = (r >= 2) ? (x2 >> (r >= 2 ? r - 2 : 0)) : (x2 << (r >= 2 ? 0 : 2 - r));
        const uint32_t S = (a & M) | (b & (M << 1)) | (c & (M << 2));  // PRMT reads the low 16 bits
        uint32_t hb = prmt(t.th0, t.th1, S);
        const uint32_t lb = prmt(t.tl0, t.tl1, S);
        if (Q4) {
            // bytes of `flip` = 0xFF where the weight's b_4 is -1: bring the four bits (weights r,
            // r+4, r+8, r+12) to byte MSBs, two per copy, and replicate them with PRMT
            const uint32_t s02 = nf << (7 - r);
            const uint32_t s13 = nf << (3 - r);
            const uint32_t flip = prmt(s02, s13, 0xD9C8u);
            hb ^= flip & 0x80808080u;
        }
        R[r][0] = prmt(lb, hb, 0x5140u);  // weights r, r + 4
        R[r][1] = prmt(lb, hb, 0x7362u);  // weights r + 8, r + 12
    }
#pragma unroll
    for (int u = 0; u < 2; ++u)
        ptx::st_shared_v4(line + (((chunk0 + u) ^ lx) << 4), R[0][u], R[1][u], R[2][u], R[3][u]);
}

// 32 weights (whole plane words): the selector word S of residue r serves both halves, low 16 bits
// for weights 0..15 and high 16 bits for weights 16..31.  Four chunks, slots chunk0..chunk0+3.
template <bool Q4>
__device__ __forceinline__ void expand32_lut(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t w3,
                                             const Lut& t, uint32_t line, uint32_t lx, uint32_t chunk0) {
    uint32_t x0 = w0, x1 = w1, x2 = w2, nf = 0u;
    if (Q4) {
        nf = ~w3;
        x0 = ~(w0 ^ w3);
        x1 = ~(w1 ^ w3);
        x2 = ~(w2 ^ w3);
    }
    constexpr uint32_t M = 0x11111111u;
    uint32_t R[4][2][2];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const uint32_t a = x0 >> r;
        const uint32_t b = (r >= 1) ? (x1 >> (r >= 1 ? r - 1 : 0)) : (x1 << 1);
        const uint32_t c = (r >= 2) ? (x2 >> (r >= 2 ? r - 2 : 0)) : (x2 << (r >= 2 ? 0 : 2 - r));
        const uint32_t S = (a & M) | (b & (M << 1)) | (c & (M << 2));
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t sel = h ? (S >> 16) : S;  // weights 16h + 4m + r, m = 0..3
            uint32_t hb = prmt(t.th0, t.th1, sel);
            const uint32_t lb = prmt(t.tl0, t.tl1, sel);
            if (Q4) {
                const int p0 = 16 * h + r;  // bit of weight m = 0; m = 2 is 8 bits up, m = 1, 3 are 4 bits up
                const uint32_t s02 = (p0 <= 7) ? (nf << (p0 <= 7 ? 7 - p0 : 0)) : (nf >> (p0 > 7 ? p0 - 7 : 0));
                const uint32_t s13 = (p0 <= 3) ? (nf << (p0 <= 3 ? 3 - p0 : 0)) : (nf >> (p0 > 3 ? p0 - 3 : 0));
                const uint32_t flip = prmt(s02, s13, 0xD9C8u);
                hb ^= flip & 0x80808080u;
            }
            R[r][h][0] = prmt(lb, hb, 0x5140u);
            R[r][h][1] = prmt(lb, hb, 0x7362u);
        }
    }
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int u = 0; u < 2; ++u)
            ptx::st_shared_v4(line + (((chunk0 + 2 * h + u) ^ lx) << 4), R[0][h][u], R[1][h][u], R[2][h][u],
                              R[3][h][u]);
}

// Same result through fp32 sums, any q <= 8.  w[i] = plane words (bits 0..15 used), a[i] = scales.
__device__ __forceinline__ void expand16_sum(const uint32_t (&w)[BCQ_MAX_Q], const float (&a)[BCQ_MAX_Q],
                                             int q, uint32_t line, uint32_t lx, uint32_t chunk0) {
    float v[16];
#pragma unroll
    for (int p = 0; p < 16; ++p) v[p] = 0.0f;
#pragma unroll
    for (int i = 0; i < BCQ_MAX_Q; ++i) {
        if (i < q) {
            const uint32_t ai = __float_as_uint(a[i]);
            const uint32_t nw = ~w[i];
#pragma unroll
            for (int p = 0; p < 16; ++p) v[p] += __uint_as_float(ai ^ ((nw << (31 - p)) & 0x80000000u));
        }
    }
#pragma unroll
    for (int cc = 0; cc < 2; ++cc)
        ptx::st_shared_v4(line + (((chunk0 + cc) ^ lx) << 4), pack_half2(v[8 * cc + 0], v[8 * cc + 4]),
                          pack_half2(v[8 * cc + 1], v[8 * cc + 5]), pack_half2(v[8 * cc + 2], v[8 * cc + 6]),
                          pack_half2(v[8 * cc + 3], v[8 * cc + 7]));
}

template <int QM>
struct NumWords {
    static constexpr int value = (QM == QM_GENERIC) ? BCQ_MAX_Q : 4;
};

// Stored words per 32 weights when the planes are kept as selector codes (q <= 4): the q = 4
// packing for four planes, the q = 3 packing for one to three (missing planes read as index bits 0).
template <int QM>
struct CodeWords {
    static constexpr int value = (QM == QM_LUT4) ? 4 : 3;
};

// The scales of one (row, group), already multiplied by the weight scale; loaded ahead of use.
template <int QM>
struct AlphaSet {
    float a[NumWords<QM>::value];
    int key;  // row * G + group, or -1 for a row outside the matrix (expands to zeros)
};

template <int QM>
__device__ __forceinline__ void load_alpha(AlphaSet<QM>& s, const float* __restrict__ alpha,
                                           long long plane_alpha, int G, int q, int j, int c, bool valid,
                                           float wscale) {
    s.key = valid ? j * G + c : -1;
#pragma unroll
    for (int i = 0; i < NumWords<QM>::value; ++i)
        s.a[i] = (i < q && valid) ? __ldg(alpha + i * plane_alpha + (long long)j * G + c) * wscale : 0.0f;
}

// Expands the 16 weights that start at bit `bit_shift` (0 or 16) of the plane words in shared
// memory at bits_addr + i * plane_stride.
template <int QM>
__device__ __forceinline__ void expand_task(const AlphaSet<QM>& as, uint32_t bits_addr, uint32_t plane_stride,
                                            uint32_t bit_shift, Lut& lut, int& lut_key, int q, uint32_t line,
                                            uint32_t lx, uint32_t chunk0) {
    uint32_t w[NumWords<QM>::value];
#pragma unroll
    for (int i = 0; i < NumWords<QM>::value; ++i)
        w[i] = (i < q) ? (ptx::ld_shared_u32(bits_addr + i * plane_stride) >> bit_shift) : 0u;
    if (QM == QM_GENERIC) {
        uint32_t w8[BCQ_MAX_Q];
        float a8[BCQ_MAX_Q];
#pragma unroll
        for (int i = 0; i < BCQ_MAX_Q; ++i) {
            w8[i] = w[i % NumWords<QM>::value];
            a8[i] = as.a[i % NumWords<QM>::value];
        }
        expand16_sum(w8, a8, q, line, lx, chunk0);
    } else {
        if (as.key != lut_key) {
            lut = (QM == QM_LUT4) ? build_lut(as.a[0], as.a[1], as.a[2], as.a[3])
                                  : build_lut(as.a[0], as.a[1], as.a[2], 0.0f);
            lut_key = as.key;
        }
        expand16_lut<QM == QM_LUT4>(w[0], w[1], w[2], w[3], lut, line, lx, chunk0);
    }
}

// 32 weights (one whole plane word per plane): two 16-weight halves from one set of loads.
template <int QM>
__device__ __forceinline__ void expand_task32(const AlphaSet<QM>& as, uint32_t bits_addr, uint32_t plane_stride,
                                              Lut& lut, int& lut_key, int q, uint32_t line, uint32_t lx,
                                              uint32_t chunk0) {
    uint32_t w[NumWords<QM>::value];
#pragma unroll
    for (int i = 0; i < NumWords<QM>::value; ++i)
        w[i] = (i < q) ? ptx::ld_shared_u32(bits_addr + i * plane_stride) : 0u;
    if (QM == QM_GENERIC) {
        uint32_t w8[BCQ_MAX_Q];
        float a8[BCQ_MAX_Q];
#pragma unroll
        for (int i = 0; i < BCQ_MAX_Q; ++i) {
            w8[i] = w[i % NumWords<QM>::value];
            a8[i] = as.a[i % NumWords<QM>::value];
        }
        expand16_sum(w8, a8, q, line, lx, chunk0);
#pragma unroll
        for (int i = 0; i < BCQ_MAX_Q; ++i) w8[i] >>= 16;
        expand16_sum(w8, a8, q, line, lx, chunk0 + 2);
    } else {
        if (as.key != lut_key) {
            lut = (QM == QM_LUT4) ? build_lut(as.a[0], as.a[1], as.a[2], as.a[3])
                                  : build_lut(as.a[0], as.a[1], as.a[2], 0.0f);
            lut_key = as.key;
        }
        expand32_lut<QM == QM_LUT4>(w[0], w[1], w[2], w[3], lut, line, lx, chunk0);
    }
}

// ------------------------------------------------------------------------------------------
// pre-pass: activations -> fp16 with a per-token power-of-two scale; max |alpha|
// ------------------------------------------------------------------------------------------

constexpr int kMaxAlphaBlocks = 124;

// Head of the forward / dX workspace: max |alpha| of each pre-pass block that scanned alpha (bit
// patterns; the consumer takes the maximum over the first `nblocks`).  No zero-initialisation.
struct WsHeader {
    uint32_t nblocks;
    uint32_t pad[3];
    uint32_t block_max[kMaxAlphaBlocks];
};

// Power of two for the weights: q * max|alpha| lands in [2^13, 2^14).  Called by whole warps.
__device__ __forceinline__ int weight_shift(const WsHeader* hdr, int q) {
    const int nb = (int)__ldg(&hdr->nblocks);
    uint32_t m = 0u;
    for (int b = threadIdx.x & 31; b < nb; b += 32) m = max(m, __ldg(&hdr->block_max[b]));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
    return shift_for(exponent_of_bits(__float_as_uint(__uint_as_float(m) * (float)q)), 13);
}

struct PrepParams {
    int n, K, act_blocks;
    long long ld_in, ld_out;
    const __nv_bfloat16* in;
    __half* out;
    float* tok_inv_scale;  // [n]
    const float* alpha;
    long long alpha_count;
    WsHeader* hdr;
    // Weights regrouped into the chunks one pipeline stage consumes, each chunk contiguous so that
    // a single bulk copy brings it into shared memory (rows past d_out are written as zeros):
    //   forward  bits_t  [m_tile][kb][q][128 rows][2 words]   the 64 k of stage kb
    //            alpha_t [m_tile][G][q][128 rows]
    //   dX       bits_t  [u][jb][q][64 rows][4 words]         u = 128-wide k tile, jb = 64-row block
    //            alpha_t [jb][G][q][64 rows]
    int mode, d_out, q, G, pitch, num_kb, amax_blocks, bits_blocks;
    int row_tiles;   // ceil(d_out / 128)
    int bits_cblk;   // ceil(pitch / 32): 32-word column blocks of the plane words
    int alpha_cblk;  // ceil(G / 32)
    const uint32_t* bits;
    float* alpha_t;
    uint32_t* bits_t;
};

// One warp per token row; VPL = 16-byte vectors a lane keeps in registers between finding the
// row's largest magnitude and writing the scaled fp16 row (VPL = 0: the row is read twice).
// Blocks past the activation blocks scan alpha instead.
constexpr int kPrepTokensPerBlock = 8;

__device__ __forceinline__ uint32_t max_mag_bf16x8(const uint4& x, int k0, int K) {
    if (k0 + 8 <= K) {
        // whole vector inside the row: magnitudes are 15-bit integers, compared two per word
        const uint32_t a = __vmaxu2(x.x & 0x7FFF7FFFu, x.y & 0x7FFF7FFFu);
        const uint32_t b = __vmaxu2(x.z & 0x7FFF7FFFu, x.w & 0x7FFF7FFFu);
        const uint32_t c = __vmaxu2(a, b);
        return max(c & 0xFFFFu, c >> 16);
    }
    const uint32_t xs[4] = {x.x, x.y, x.z, x.w};
    uint32_t m = 0u;
#pragma unroll
    for (int e = 0; e < 8; ++e)
        if (k0 + e < K) m = max(m, (xs[e >> 1] >> ((e & 1) * 16)) & 0x7FFFu);
    return m;
}

__device__ __forceinline__ uint4 scale_to_fp16x8(const uint4& x, int k0, int K, float scale) {
    const uint32_t xs[4] = {x.x, x.y, x.z, x.w};
    if (k0 + 8 <= K) {
        // bf16 -> fp32 is a shift (low half) or a mask (high half); the product with a power of two
        // is exact and one conversion packs two of them
        uint4 o;
        uint32_t* ow = &o.x;
#pragma unroll
        for (int w = 0; w < 4; ++w)
            ow[w] = pack_half2(__uint_as_float(xs[w] << 16) * scale, __uint_as_float(xs[w] & 0xFFFF0000u) * scale);
        return o;
    }
    float f[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        const uint32_t b = (xs[e >> 1] >> ((e & 1) * 16)) & 0xFFFFu;
        f[e] = (k0 + e < K) ? __uint_as_float(b << 16) * scale : 0.0f;
    }
    uint4 o;
    o.x = pack_half2(f[0], f[1]);
    o.y = pack_half2(f[2], f[3]);
    o.z = pack_half2(f[4], f[5]);
    o.w = pack_half2(f[6], f[7]);
    return o;
}

template <int VPL>
__global__ void __launch_bounds__(256) prepare_kernel(const PrepParams p) {
    __shared__ uint32_t red[8];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // roles by block id: tokens, then max|alpha|, then the regrouping blocks.  The hardware starts
    // blocks in index order, and the short, latency-bound regrouping blocks should not queue
    // behind the register-heavy token blocks, so the ids run backwards.
    const int bid = (int)gridDim.x - 1 - (int)blockIdx.x;
    if (bid >= p.act_blocks + p.amax_blocks) {
        // ---- regroup a block of 128 rows x 32 columns (plane words or scales) of one plane:
        // coalesced reads into shared memory, then coalesced writes of the stage chunks
        __shared__ uint32_t tile[128][33];
        int b = bid - p.act_blocks - p.amax_blocks;
        const bool is_alpha = b >= p.bits_blocks;
        if (is_alpha) b -= p.bits_blocks;
        if (is_alpha) {
            // ---- scales of one plane and one tile of 128 rows: alpha[i][j][c] is contiguous over
            // (j, c), so the block reads it as one coalesced run and scatters the values to their
            // places in the regrouped array (rows past d_out become zeros)
            const int rt = b % p.row_tiles;
            const int i = b / p.row_tiles;
            const float* src = p.alpha + ((long long)i * p.d_out + (long long)rt * 128) * p.G;
            const int count = 128 * p.G;
            const int rows_left = p.d_out - rt * 128;
            for (int e = threadIdx.x; e < count; e += 256) {
                const int r = e / p.G, c = e - r * p.G;
                const float v = (r < rows_left) ? __ldg(src + e) : 0.0f;
                long long o;
                if (p.mode == MODE_FWD) {
                    o = (((long long)rt * p.G + c) * p.q + i) * 128 + r;
                } else {
                    const int jb = rt * 2 + (r >> 6), rr = r & 63;
                    if (jb >= p.num_kb) continue;
                    o = (((long long)jb * p.G + c) * p.q + i) * 64 + rr;
                }
                p.alpha_t[o] = v;
            }
            return;
        }
        const int cblks = is_alpha ? p.alpha_cblk : p.bits_cblk;
        const int cb = b % cblks;
        const int rt = (b / cblks) % p.row_tiles;
        const int i = b / (cblks * p.row_tiles);
        const int ncols = is_alpha ? p.G : p.pitch;
        const uint32_t* src = is_alpha ? reinterpret_cast<const uint32_t*>(p.alpha) : p.bits;
        src += (long long)i * p.d_out * ncols;
        // all sixteen loads of a thread in flight at once: the block's time is one memory latency
        uint32_t held[16];
        const int col_l = cb * 32 + lane;
#pragma unroll
        for (int pass = 0; pass < 16; ++pass) {
            const int j = rt * 128 + pass * 8 + warp;
            held[pass] = (j < p.d_out && col_l < ncols) ? __ldg(src + (long long)j * ncols + col_l) : 0u;
        }
#pragma unroll
        for (int pass = 0; pass < 16; ++pass) {
            uint32_t v = held[pass];
            if (!is_alpha) {
                // even bits of every byte to its low nibble, odd bits to the high nibble: one PRMT
                // pair of the expansion emits weights 0,4,1,5,2,6,3,7 of a byte, so with the bits
                // stored as 0,2,4,6,1,3,5,7 the expanded tile comes out in natural k order
                uint32_t t = (v ^ (v >> 1)) & 0x22222222u;
                v ^= t ^ (t << 1);
                t = (v ^ (v >> 2)) & 0x0C0C0C0Cu;
                v ^= t ^ (t << 2);
            }
            tile[pass * 8 + warp][lane] = v;
        }
        __syncthreads();
        const int t = threadIdx.x;
        uint32_t* dst = is_alpha ? reinterpret_cast<uint32_t*>(p.alpha_t) : p.bits_t;
#pragma unroll 4
        for (int pass = 0; pass < 16; ++pass) {
            int r, cl;
            if (is_alpha) { r = t & 127; cl = pass * 2 + (t >> 7); }
            else if (p.mode == MODE_FWD) { r = t >> 1; cl = pass * 2 + (t & 1); }
            else { r = (pass & 1) * 64 + (t >> 2); cl = (pass >> 1) * 4 + (t & 3); }
            const int col = cb * 32 + cl;
            if (col >= ncols) continue;
            long long o;
            if (p.mode == MODE_FWD) {
                if (is_alpha) {
                    o = (((long long)rt * p.G + col) * p.q + i) * 128 + r;
                } else {
                    const int kb = col >> 1;
                    if (kb >= p.num_kb) continue;
                    o = ((((long long)rt * p.num_kb + kb) * p.q + i) * 128 + r) * 2 + (col & 1);
                }
            } else {
                const int jb = rt * 2 + (r >> 6), rr = r & 63;
                if (jb >= p.num_kb) continue;
                if (is_alpha) o = (((long long)jb * p.G + col) * p.q + i) * 64 + rr;
                else o = ((((long long)(col >> 2) * p.num_kb + jb) * p.q + i) * 64 + rr) * 4 + (col & 3);
            }
            dst[o] = tile[r][cl];
        }
        return;
    }
    if (bid >= p.act_blocks) {
        // ---- max |alpha| of this block's share of the scales
        const long long nb = p.amax_blocks;
        uint32_t m = 0u;
        for (long long o = ((long long)bid - p.act_blocks) * 256 + threadIdx.x; o < p.alpha_count;
             o += nb * 256)
            m = max(m, __float_as_uint(__ldg(p.alpha + o)) & 0x7FFFFFFFu);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
        if (lane == 0) red[warp] = m;
        __syncthreads();
        if (threadIdx.x == 0) {
#pragma unroll
            for (int w = 0; w < 8; ++w) m = max(m, red[w]);
            p.hdr->block_max[bid - p.act_blocks] = m;
            if (bid == p.act_blocks) p.hdr->nblocks = (uint32_t)nb;
        }
        return;
    }
    const int t = bid * kPrepTokensPerBlock + warp;
    if (t >= p.n) return;
    const uint4* src = reinterpret_cast<const uint4*>(p.in + (long long)t * p.ld_in);
    uint4* dst = reinterpret_cast<uint4*>(p.out + (long long)t * p.ld_out);
    const int nvec = (p.K + 7) / 8;
    uint32_t m = 0u;
    uint4 held[VPL > 0 ? VPL : 1];
    if (VPL > 0) {
#pragma unroll
        for (int i = 0; i < VPL; ++i) {
            const int v = lane + 32 * i;
            held[i] = (v < nvec) ? __ldg(src + v) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int i = 0; i < VPL; ++i) m = max(m, max_mag_bf16x8(held[i], (lane + 32 * i) * 8, p.K));
    } else {
        // long rows: four loads of a lane in flight at a time
        for (int v0 = lane; v0 < nvec; v0 += 128) {
            uint4 x[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                x[u] = (v0 + 32 * u < nvec) ? __ldg(src + v0 + 32 * u) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
            for (int u = 0; u < 4; ++u) m = max(m, max_mag_bf16x8(x[u], (v0 + 32 * u) * 8, p.K));
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
    const int sh = shift_for(exponent_of_bits(m << 16), 14);
    const float scale = pow2f(sh);
    if (lane == 0) p.tok_inv_scale[t] = pow2f(-sh);
    if (VPL > 0) {
#pragma unroll
        for (int i = 0; i < VPL; ++i) {
            const int v = lane + 32 * i;
            if (v < nvec) dst[v] = scale_to_fp16x8(held[i], v * 8, p.K, scale);
        }
    } else {
        for (int v0 = lane; v0 < nvec; v0 += 128) {
            uint4 x[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                x[u] = (v0 + 32 * u < nvec) ? __ldg(src + v0 + 32 * u) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (v0 + 32 * u < nvec) dst[v0 + 32 * u] = scale_to_fp16x8(x[u], (v0 + 32 * u) * 8, p.K, scale);
        }
    }
}

// Selector codes of the planes (q <= 4) in the chunk order of the GEMM kernel; one thread per (row,
// 32-weight block).  The planes are frozen, so this runs once per layer (bcq_prepare_planes); a call
// that is not given prepared planes runs it into its workspace.
//   forward  codes [m_tile][kb][128 rows][2 halves][NW words]    NW = CodeWords
//   dX       codes [u][jb][64 rows][4 quarters][NW words]
// Rows past d_out and blocks past the row pitch are written as zeros (their levels are zero or
// meet zero activations).
template <int NW>
__global__ void __launch_bounds__(256) code_planes_kernel(int mode, int d_out, int pitch, int q, int rows_padded,
                                                           int words_padded, int num_kb, const uint32_t* __restrict__ bits,
                                                           uint32_t* __restrict__ codes) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)rows_padded * words_padded) return;
    const int wd = (int)(idx % words_padded);
    const int j = (int)(idx / words_padded);
    uint32_t w[4] = {0u, 0u, 0u, 0u};
    const bool valid = (j < d_out) && (wd < pitch);
    for (int i = 0; i < q; ++i)
        if (valid) w[i] = __ldg(bits + ((long long)i * d_out + j) * pitch + wd);
    uint32_t S[4];
    selectors_from_planes(w, q, S);
    if (!valid)
        for (int r = 0; r < 4; ++r) S[r] = 0u;
    long long o;
    if (mode == MODE_FWD)
        o = ((((long long)(j >> 7) * num_kb + (wd >> 1)) * 128 + (j & 127)) * 2 + (wd & 1)) * NW;
    else
        o = ((((long long)(wd >> 2) * num_kb + (j >> 6)) * 64 + (j & 63)) * 4 + (wd & 3)) * NW;
    pack_selectors<NW>(S, codes + o);
}

// ------------------------------------------------------------------------------------------
// forward / dX for n > 16: A expanded from the bit-planes, B (fp16 activations) by TMA
// ------------------------------------------------------------------------------------------

struct ExpandParams {
    int d_out, d_in, q, g, G, pitch, n;
    int Mdim;          // d_out (fwd) or d_in (dX)
    int num_kb;        // K blocks of 64 over d_in (fwd) or d_out (dX)
    int kb_per_split;
    int splits;
    int m_tiles, n_tiles;
    int tn;                // token tile width
    uint32_t acc_cols;     // tensor-memory columns per accumulator
    // pipeline geometry (chosen on the host)
    int a_slots;           // ring of expanded weight tiles (16 KiB each), >= the number of worker groups
    int b_slots;           // ring of activation tiles (TN x 128 B each), filled by TMA
    int epi_bufs;          // staging buffers per epilogue warp: 1 or 2
    uint32_t chunk_words;  // words of one stage's chunk of the regrouped planes
    const uint32_t* bits_t;      // regrouped plane words (see PrepParams)
    const float* alpha_t;        // regrouped scales
    const float* bias;           // fwd only, may be null
    const WsHeader* hdr;         // max |alpha| per pre-pass block
    const float* tok_inv_scale;  // [n]
    void* out;                   // [n][ldo]
    long long ldo;
    int out_bf16;
    int fast_epi;                // bf16 output written by TMA stores (aligned base and pitch, no K split)
    int helpers;                 // the worker warps share the epilogue of a CTA's last tile (see run_expand)
    float* partial;              // [splits][n][Mdim] when splits > 1
};

// One pipeline stage in shared memory: | A tile 16 KiB | B tile TN x 128 B | plane words |.
// The plane words arrive by TMA as [plane][row][4 words]: 128 weights of `rows` rows, where rows
// = 128 weight rows for the forward and decode (the stage uses 64 of the 128 weights) and the 64
// rows j of the K block for dX (the four words are the tile's 128 k).
template <int MODE, int TN, int QM>
struct StageLayout {
    static constexpr int kBitRows = (MODE == MODE_BWDX) ? 64 : 128;
    static constexpr uint32_t kBBytes = TN * kBlockK * 2;
    static constexpr uint32_t kBitsOff = kABytes + kBBytes;
    static constexpr uint32_t kPlaneBytes = kBitRows * 16;
    static constexpr uint32_t kBitsBytes = NumWords<QM>::value * kPlaneBytes;
    static constexpr uint32_t kStageBytes = kBitsOff + kBitsBytes;
};

// Prefill kernel.  Persistent: every CTA walks over output tiles (m-tile fastest, so that CTAs
// running at the same time share activation tiles in L2).  32 warps:
//   warps 0..11   workers in three groups of four; group g takes the pipeline stages whose running
//                 index is g mod 3.  A thread expands 64 weights of one row per stage (one 128-byte
//                 line of the operand tile), so a group rebuilds one 128 x 64 weight tile.  The
//                 thread reads its selector codes (or plane words) and scales straight from the
//                 regrouped arrays in global memory, one task ahead of the one it expands, so the
//                 loads are hidden behind a whole turn of the group
//   warp 12       UMMA issuer, owner of the tensor-memory allocation (two accumulators)
//   warp 13       producer of the activation tiles (TMA)
//   warps 16..19  epilogue: drain one accumulator while the main loop fills the other (warp w
//                 reaches the tensor-memory lanes 32 * (w % 4) .. + 31)
// Shared memory: a ring of weight tiles (16 KiB each; few, the workers refill one as soon as the
// tensor core is done with it), a deeper ring of activation tiles (TN x 128 B each; a TMA load
// takes about a microsecond to land), the epilogue's staging, barriers and output scales.
constexpr int kPfGroups = 3;
constexpr int kPfGroupWarps = 4;
constexpr int kPfWorkerWarps = kPfGroups * kPfGroupWarps;  // 12
constexpr int kPfMmaWarp = kPfWorkerWarps;                 // 12
constexpr int kPfProdWarp = kPfMmaWarp + 1;                // 13
constexpr int kPfEpiWarp0 = 16;
constexpr int kPfEpiWarps = 4;
constexpr int kPfWarps = kPfEpiWarp0 + kPfEpiWarps;        // 20
constexpr int kPfThreads = kPfWarps * 32;                  // 640
static_assert(kPfEpiWarp0 % 4 == 0, "epilogue warp e must sit on tensor-memory lane quarter e");
__device__ __forceinline__ int pf_worker_index(int warp) { return warp < kPfWorkerWarps ? warp : -1; }
__device__ __forceinline__ int pf_epilogue_index(int warp) { return warp >= kPfEpiWarp0 ? warp - kPfEpiWarp0 : -1; }
constexpr int kPfMaxSlots = 8;                                // per ring
constexpr uint32_t kPfGroupBar0 = 4;                           // named barriers 4, 5, 6: one per worker group
constexpr uint32_t kPfCtlBytes = 384;                          // barriers, TMEM handle, abort flag
constexpr uint32_t kPfScaleBytes = 256 * 4;                    // [TN] output scales of the tile being drained
constexpr uint32_t kPfStagingBuf = kPfEpiWarps * 1024;         // per epilogue warp one 1 KiB buffer of 32 rows x 16 bf16 (8 fp32) tokens; one or two such sets

template <int MODE, int QM>
__global__ void __launch_bounds__(kPfThreads, 1)
expand_gemm_kernel(const __grid_constant__ CUtensorMap tmap_b, const __grid_constant__ CUtensorMap tmap_out,
                   const ExpandParams p) {
    const int TN = p.tn;                                   // token tile: a multiple of 16, <= 256
    const uint32_t kBBytes = (uint32_t)TN * kBlockK * 2;
    const uint32_t kAccCols = p.acc_cols;                  // tensor-memory columns of one accumulator
    const uint32_t kTmemCols = 2 * kAccCols;               // a power of two >= 32
    constexpr int kRows = (MODE == MODE_FWD) ? 128 : 64;  // weight rows of one stage
    constexpr int kUnit = (MODE == MODE_FWD) ? 2 : 4;     // 32-weight blocks per row and stage
    constexpr int NW = NumWords<QM>::value;
    // fp16 x fp16 -> fp32; A is MN-major for dX
    const uint32_t kIdesc = (ptx::make_idesc_bf16(kBlockM, TN, MODE == MODE_BWDX ? 1 : 0, 0)) &
                            ~((1u << 7) | (1u << 10));

    extern __shared__ uint8_t smem_raw[];
    const int NA = p.a_slots, NB = p.b_slots;
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
    const uint32_t b_base = smem_base + NA * kABytes;
    const uint32_t staging_base = b_base + NB * kBBytes;  // 1 KiB aligned: the output boxes are swizzled
    const uint32_t staging_bytes = (uint32_t)p.epi_bufs * kPfStagingBuf;
    const uint32_t ctl_base = staging_base + staging_bytes;
    uint8_t* ctl_gen = smem_gen + NA * kABytes + NB * kBBytes + staging_bytes;

    Ctl ctl;
    ctl.aready = ctl_base;                      // + 8*s : the workers have written weight slot s
    ctl.empty = ctl_base + 8 * kPfMaxSlots;     // + 8*s : the UMMAs that read weight slot s are done
    ctl.full = ctl_base + 16 * kPfMaxSlots;     // + 8*s : the activation tile of slot s has landed
    const uint32_t b_empty = ctl_base + 24 * kPfMaxSlots;  // + 8*s : the UMMAs that read activation slot s are done
    ctl.accum = ctl_base + 32 * kPfMaxSlots;    // accumulator full [2]
    const uint32_t acc_empty = ctl.accum + 16;  // accumulator drained [2]
    ctl.spare = acc_empty + 16;
    volatile uint32_t* tmem_holder = reinterpret_cast<volatile uint32_t*>(ctl_gen + 32 * kPfMaxSlots + 40);
    ctl.abort_flag = reinterpret_cast<volatile int*>(ctl_gen + 32 * kPfMaxSlots + 44);
    ctl.device_flag = &g_timeout_flag;
    float* scale = reinterpret_cast<float*>(ctl_gen + kPfCtlBytes);  // [TN]: 1 / (weight scale * token scale)
    const uint32_t scale_addr = ctl_base + kPfCtlBytes;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (warp == 0) {
        // the barriers are initialised by the lanes of one warp side by side (one after the other
        // they cost a few tenths of a microsecond before any copy can start)
        if (lane < NA) {
            ptx::mbar_init(ctl.aready + 8 * lane, kPfGroupWarps);
            ptx::mbar_init(ctl.empty + 8 * lane, 1);
        } else if (lane >= 8 && lane < 8 + NB) {
            ptx::mbar_init(ctl.full + 8 * (lane - 8), 1);
            ptx::mbar_init(b_empty + 8 * (lane - 8), 1);
        } else if (lane >= 16 && lane < 18) {
            ptx::mbar_init(ctl.accum + 8 * (lane - 16), 1);
            ptx::mbar_init(acc_empty + 8 * (lane - 16), kPfEpiWarps);
        } else if (lane == 18) {
            ptx::mbar_init(ctl.spare, 1);
            *ctl.abort_flag = 0;
        } else if (lane == 19) {
            ptx::prefetch_tmap(&tmap_b);
            if (p.fast_epi) ptx::prefetch_tmap(&tmap_out);
        }
        ptx::fence_mbar_init();
    }
    if (warp == kPfMmaWarp) {
        ptx::tmem_alloc(ptx::smem_u32(const_cast<uint32_t*>(tmem_holder)), kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_holder;

    // every role walks the same sequence of tiles and pipeline stages
    const int num_tiles = p.m_tiles * p.n_tiles * p.splits;
    auto tile_coords = [&](int tile, int& m0, int& t0, int& z, int& kb_begin, int& iters) {
        const int mt = tile % p.m_tiles;
        const int rest = tile / p.m_tiles;
        m0 = mt * kBlockM;
        t0 = (rest % p.n_tiles) * TN;
        z = rest / p.n_tiles;
        kb_begin = z * p.kb_per_split;
        iters = min(p.num_kb, kb_begin + p.kb_per_split) - kb_begin;
    };

    // bf16 output through TMA stores, 16 tokens x 32 rows at a time: the accumulator is read as MMA
    // fragments (thread t: rows g = t/4 and g + 8 of each half of the warp's 32 lanes, token pairs
    // 2(t%4)), scaled, packed to bf16 pairs and transposed by stmatrix into a 64-byte-swizzled
    // [16 tokens][32 rows] box at `buf`, which one lane then hands to the TMA.  s0*, s1* are the
    // output scales of the thread's tokens in the first and second group of eight.
    auto store_box = [&](uint32_t t_row, int col, uint32_t buf, float s0x, float s0y, float s1x, float s1y,
                         const float (&b4)[4], int x, int y) {
        const int tok = ((lane >> 4) << 3) + (lane & 7);  // token row this lane addresses
        const uint32_t st_off = (uint32_t)tok * 64u;
        const uint32_t st_sw = (uint32_t)((tok >> 1) & 3);
        const uint32_t jb = (uint32_t)((lane >> 3) & 1);
        uint32_t va[8], vb[8];
        ptx::tmem_ld_16x256b_x2(t_row + (uint32_t)col, va);
        ptx::tmem_ld_16x256b_x2(t_row + (16u << 16) + (uint32_t)col, vb);
        ptx::tmem_ld_wait();
        auto pk = [](uint32_t u, uint32_t v, float sx, float sy, float b) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(u) * sx + b, __uint_as_float(v) * sy + b);
            return *reinterpret_cast<const uint32_t*>(&h);
        };
        const uint32_t a0 = pk(va[0], va[1], s0x, s0y, b4[0]), a1 = pk(va[2], va[3], s0x, s0y, b4[1]);
        const uint32_t a2 = pk(va[4], va[5], s1x, s1y, b4[0]), a3 = pk(va[6], va[7], s1x, s1y, b4[1]);
        const uint32_t c0 = pk(vb[0], vb[1], s0x, s0y, b4[2]), c1 = pk(vb[2], vb[3], s0x, s0y, b4[3]);
        const uint32_t c2 = pk(vb[4], vb[5], s1x, s1y, b4[2]), c3 = pk(vb[6], vb[7], s1x, s1y, b4[3]);
        ptx::stmatrix_x4_trans(buf + st_off + ((jb ^ st_sw) << 4), a0, a1, a2, a3);
        ptx::stmatrix_x4_trans(buf + st_off + (((jb + 2u) ^ st_sw) << 4), c0, c1, c2, c3);
        ptx::fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
            ptx::tma_store_2d(&tmap_out, x, y, buf);
            ptx::bulk_commit_group();
        }
    };
    // On the last tile of a CTA the worker warps have nothing left to expand, so they share its
    // epilogue: of the four warps on a tensor-memory lane quarter (one epilogue warp, three workers)
    // warp h takes the boxes h, h + 4, ...
    constexpr int kPfHelpers = 1 + kPfWorkerWarps / 4;  // 4
    auto is_last_tile = [&](int tile) { return tile + (int)gridDim.x >= num_tiles; };

    if (warp == kPfProdWarp) {
        // ---------------- producer: the activation tile of every stage (TMA), into a ring of its
        // own that runs as far ahead of the tensor core as shared memory allows
        if (lane == 0) {
            bool ok = true;
            int s = 0, in_flight = 0;
            uint32_t ph = 0;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                int m0, t0, z, kb_begin, iters;
                tile_coords(tile, m0, t0, z, kb_begin, iters);
                for (int it = 0; it < iters; ++it) {
                    ok = wait_bar(b_empty + 8 * s, ph ^ 1u, ctl, 1, 256u);
                    if (!ok) break;
                    const uint32_t bar = ctl.full + 8 * s;
                    ptx::mbar_arrive_expect_tx(bar, kBBytes);
                    ptx::tma_load_2d(b_base + s * kBBytes, &tmap_b, (kb_begin + it) * kBlockK, t0, bar);
                    in_flight = min(in_flight + 1, NB);
                    if (++s == NB) { s = 0; ph ^= 1u; }
                }
            }
            if (!ok) {
                // giving up: let the copies already issued land before the CTA exits.  The last
                // `in_flight` slots before (s, ph) were issued with the phase they had then.
                int bs = s;
                uint32_t bph = ph;
                for (int i = 0; i < in_flight; ++i) {
                    if (bs == 0) { bs = NB; bph ^= 1u; }
                    --bs;
                    wait_bar(ctl.full + 8 * bs, bph, ctl, 2);
                }
            }
        }
    } else if (warp == kPfMmaWarp) {
        // ---------------- UMMA issuer.  One elected thread runs the whole loop: per stage it has
        // to get through two barrier checks, a fence, four UMMAs and two commits in less time
        // than the tensor core needs for the stage (512 cycles at the full width), so nothing
        // warp-wide (election, reconvergence) is left inside the loop and the two barrier checks
        // are issued together.
        if (ptx::elect_one()) {
            bool ok = true;
            int sa = 0, sb = 0, lt = 0;
            uint32_t pha = 0, phb = 0;
            // shared-memory descriptor halves (128-byte swizzle, version 1): low = start address >> 4 and
            // leading offset >> 4 at bit 16, high = stride offset >> 4, version at bit 14, swizzle at bit 29
            constexpr uint32_t kHiCommon = (1024u >> 4) | (1u << 14) | (2u << 29);
            constexpr uint32_t kAHi = kHiCommon, kBHi = kHiCommon;
            constexpr uint32_t kALoExtra = ((MODE == MODE_FWD) ? (16u >> 4) : (8192u >> 4)) << 16;  // leading offset of A
            constexpr uint32_t kBLoExtra = (16u >> 4) << 16;
            constexpr uint32_t kAStep = (MODE == MODE_FWD) ? (32u >> 4) : (2048u >> 4);
            const uint32_t a_lo0 = ((smem_base >> 4) & 0x3FFFu) | kALoExtra;
            const uint32_t b_lo0 = ((b_base >> 4) & 0x3FFFu) | kBLoExtra;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++lt) {
                int m0, t0, z, kb_begin, iters;
                tile_coords(tile, m0, t0, z, kb_begin, iters);
                const int acc = lt & 1;
                const uint32_t acc_ph = (lt >> 1) & 1;
                ok = wait_bar(acc_empty + 8 * acc, acc_ph ^ 1u, ctl, 8);  // the epilogue has drained it
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + (uint32_t)acc * kAccCols;
                for (int it = 0; it < iters; ++it) {
                    // both operands of the stage in place?  (the common case: yes, both at once)
                    const bool fb = ptx::mbar_try_wait(ctl.full + 8 * sb, phb);
                    const bool fa = ptx::mbar_try_wait(ctl.aready + 8 * sa, pha);
                    if (!fb) ok = wait_bar(ctl.full + 8 * sb, phb, ctl, 4, 32u);
                    if (!fa && ok) ok = wait_bar(ctl.aready + 8 * sa, pha, ctl, 3, 32u);
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    // descriptors: only the start-address field changes, by 32 bytes (K-major) or
                    // 2048 bytes (MN-major A) per UMMA
                    const uint32_t a_lo = a_lo0 + (uint32_t)sa * (kABytes >> 4);
                    const uint32_t b_lo = b_lo0 + (uint32_t)sb * (kBBytes >> 4);
#pragma unroll
                    for (int kk = 0; kk < kBlockK / 16; ++kk)
                        ptx::umma_f16_halves(d_tmem, a_lo + kk * kAStep, kAHi, b_lo + kk * 2, kBHi, kIdesc,
                                             (it > 0 || kk > 0) ? 1u : 0u);
                    ptx::umma_commit(ctl.empty + 8 * sa);
                    ptx::umma_commit(b_empty + 8 * sb);
                    if (++sa == NA) { sa = 0; pha ^= 1u; }
                    if (++sb == NB) { sb = 0; phb ^= 1u; }
                }
                if (ok) ptx::umma_commit(ctl.accum + 8 * acc);
            }
            if (!ok) {
                ptx::umma_commit(ctl.spare);
                wait_bar(ctl.spare, 0, ctl, 5);
            }
        }
        __syncwarp();
    } else if (pf_worker_index(warp) >= 0) {
        // ---------------- workers
        const int wid = pf_worker_index(warp);  // 0..11
        const int group = wid / kPfGroupWarps;  // takes the stages whose running index is `group` mod kPfGroups
        const int wl = wid % kPfGroupWarps;
        const float wscale = pow2f(weight_shift(p.hdr, p.q));

        // A task is one 128-byte line of the weight tile: 64 weights of one row.
        // fwd : (weight row m0 + row, the stage's 64 k); a warp takes 32 consecutive rows
        // dX  : (K index j = 64*kb + row, 64-wide half of the tile's 128 k); the two halves of a row
        //       sit in adjacent lanes
        // Either way the 32 lanes of a warp write their 16-byte chunks to all banks evenly.
        const int row = (MODE == MODE_FWD) ? wl * 32 + lane : wl * 16 + (lane >> 1);
        const int half = (MODE == MODE_FWD) ? 0 : (lane & 1);
        const uint32_t line_off = (uint32_t)half * 8192u + (uint32_t)row * 128u;
        const uint32_t lx = row & 7;
        constexpr int NWC = CodeWords<QM>::value;
        constexpr int NL = (QM == QM_GENERIC) ? NW : NWC;   // words a 32-weight block loads
        constexpr int NSC = (QM == QM_GENERIC) ? NW : 4;    // scales a task loads
        // the task's words within a chunk [m_tile][kb] (fwd) or [u][jb] (dX) of the regrouped planes:
        // q <= 4 selector codes [row][block][NWC], q > 4 plane words [plane][row][block]; its two
        // 32-weight blocks are neighbours
        const uint32_t block0 = (uint32_t)(row * kUnit + half * 2);
        const uint32_t word_off = (QM == QM_GENERIC) ? block0 : block0 * NWC;
        const uint32_t chunk_words = p.chunk_words;
        const uint32_t alpha_block = (uint32_t)p.q * kRows;  // floats per (row block, group): [plane][row]

        // The task stream of this thread: the stages whose running index over all tiles of the CTA
        // is `group` mod kPfGroups.  A cursor names one of them.
        struct Cur {
            int tile, it, iters, kb_begin, mt;
            int c, kpos, next_edge;  // group index of the task's first 32 k (forward: advances with the stage)
            uint32_t code_idx;       // this thread's first word of the task in the regrouped planes
            uint32_t alpha_idx;      // its first scale (plane 0, group c) in the regrouped scales
            bool split;              // the second 32 k belong to the next group (g not a multiple of 64)
            bool fresh;              // the scales differ from the previous task's: load them, rebuild the table
            bool valid;
        };
        auto enter_tile = [&](Cur& x) {
            int m0, t0, z;
            tile_coords(x.tile, m0, t0, z, x.kb_begin, x.iters);
            x.mt = m0 >> 7;
        };
        const uint32_t code_step = kPfGroups * chunk_words;
        const uint32_t alpha_step = kPfGroups * (uint32_t)p.G * alpha_block;  // dX: the next task's rows
        auto locate = [&](Cur& x) {  // group index and array positions at (tile, it), from scratch
            x.kpos = (MODE == MODE_FWD) ? (x.kb_begin + x.it) * kBlockK : x.mt * kBlockM + half * 64;
            x.c = min(x.kpos / p.g, p.G - 1);
            x.next_edge = (x.c + 1) * p.g;
            x.split = (x.kpos + 32 >= x.next_edge) && (x.c < p.G - 1);
            x.code_idx = (uint32_t)(x.mt * p.num_kb + x.kb_begin + x.it) * chunk_words + word_off;
            const int blk = (MODE == MODE_FWD) ? x.mt : x.kb_begin + x.it;
            x.alpha_idx = (uint32_t)(blk * p.G + x.c) * alpha_block + (uint32_t)row;
        };
        // to the next task: kPfGroups stages on
        auto advance = [&](Cur& x) {
            x.it += kPfGroups;
            bool moved = false;
            while (x.it >= x.iters) {
                x.it -= x.iters;
                x.tile += gridDim.x;
                if (x.tile >= num_tiles) { x.valid = false; return; }
                enter_tile(x);
                moved = true;
            }
            if (moved) {
                locate(x);
                x.fresh = true;
            } else if (MODE == MODE_FWD) {
                const int c0 = x.c;
                x.kpos += kPfGroups * kBlockK;
                while (x.kpos >= x.next_edge && x.c < p.G - 1) { ++x.c; x.next_edge += p.g; }
                x.split = (x.kpos + 32 >= x.next_edge) && (x.c < p.G - 1);
                x.fresh = (QM == QM_GENERIC) || (x.c != c0) || x.split;
                x.code_idx += code_step;
                x.alpha_idx += (uint32_t)(x.c - c0) * alpha_block;
            } else {
                x.fresh = true;  // dX: every stage brings other rows
                x.code_idx += code_step;
                x.alpha_idx += alpha_step;
            }
        };
        // global loads of a task: its plane words or codes and, when they change, its scales
        auto issue = [&](const Cur& x, uint32_t (&cv)[2][NL], float (&av)[NSC]) {
            const uint32_t* src = p.bits_t + x.code_idx;
            if (QM == QM_GENERIC) {
#pragma unroll
                for (int i = 0; i < NL; ++i) {
                    if (i < p.q) {
                        const uint2 v = ptx::ldg_nc_v2(src + i * (kRows * kUnit));
                        cv[0][i] = v.x; cv[1][i] = v.y;
                    } else {
                        cv[0][i] = 0u; cv[1][i] = 0u;
                    }
                }
            } else if (NWC == 4) {
                const uint4 v0 = ptx::ldg_nc_v4(src), v1 = ptx::ldg_nc_v4(src + 4);
                cv[0][0] = v0.x; cv[0][1] = v0.y; cv[0][2] = v0.z; cv[0][NL - 1] = v0.w;
                cv[1][0] = v1.x; cv[1][1] = v1.y; cv[1][2] = v1.z; cv[1][NL - 1] = v1.w;
            } else {
                // six words, 8-byte aligned
                const uint2 v0 = ptx::ldg_nc_v2(src), v1 = ptx::ldg_nc_v2(src + 2), v2 = ptx::ldg_nc_v2(src + 4);
                cv[0][0] = v0.x; cv[0][1] = v0.y; cv[0][2] = v1.x;
                cv[1][0] = v1.y; cv[1][1] = v2.x; cv[1][2] = v2.y;
            }
            if (x.fresh) {
                const float* ap = p.alpha_t + x.alpha_idx;
#pragma unroll
                for (int i = 0; i < NSC; ++i)
                    av[i] = (i < p.q) ? __uint_as_float(ptx::ldg_nc_u32(ap + i * kRows)) : 0.0f;
            }
        };

        Lut lut = {0u, 0u, 0u, 0u};
        bool ok = true;
        int s = group;  // weight slot of the current task (a_slots >= kPfGroups)
        uint32_t ph = 0;
        // One task: wait until the UMMAs that read the slot's previous contents are done (the first
        // warp of the group polls the barrier, the others park on a hardware barrier: a polling
        // warp takes issue slots from the warps that expand), expand, publish.
        auto process = [&](const Cur& x, const uint32_t (&cv)[2][NL], const float (&av)[NSC]) -> bool {
            if (wl == 0) wait_bar(ctl.empty + 8 * s, ph ^ 1u, ctl, 9, 256u);  // a timeout shows in the abort flag
            ptx::named_bar_sync(kPfGroupBar0 + group, kPfGroupWarps * 32);
            if (*ctl.abort_flag) return false;
            const uint32_t line = smem_base + (uint32_t)s * kABytes + line_off;
            float a2[NSC];  // scales of the second 32 weights when they belong to the next group
            if (x.split) {
                const float* ap = p.alpha_t + x.alpha_idx + alpha_block;  // group c + 1
#pragma unroll
                for (int i = 0; i < NSC; ++i)
                    a2[i] = (i < p.q) ? __uint_as_float(ptx::ldg_nc_u32(ap + i * kRows)) : 0.0f;
            }
#pragma unroll
            for (int b = 0; b < 2; ++b) {
                const bool second = (b == 1) && x.split;
                if (QM == QM_GENERIC) {
                    float a8[BCQ_MAX_Q];
                    uint32_t w8[BCQ_MAX_Q];
#pragma unroll
                    for (int i = 0; i < BCQ_MAX_Q; ++i) {
                        a8[i] = (second ? a2[i % NSC] : av[i % NSC]) * wscale;
                        w8[i] = cv[b][i % NL];
                    }
                    expand16_sum(w8, a8, p.q, line, lx, 4 * b);
#pragma unroll
                    for (int i = 0; i < BCQ_MAX_Q; ++i) w8[i] >>= 16;
                    expand16_sum(w8, a8, p.q, line, lx, 4 * b + 2);
                } else {
                    if ((b == 0 && x.fresh) || second) {
                        float a[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) a[i] = (second ? a2[i % NSC] : av[i % NSC]) * wscale;
                        lut = (QM == QM_LUT4) ? build_lut(a[0], a[1], a[2], a[3]) : build_lut(a[0], a[1], a[2], 0.0f);
                    }
                    uint32_t cw[NWC], S[4];
#pragma unroll
                    for (int i = 0; i < NWC; ++i) cw[i] = cv[b][i % NL];
                    selectors<NWC>(cw, S);
                    expand32_codes<NWC>(S, lut, line, lx, 4 * b);
                }
            }
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ctl.aready + 8 * s);
            s += kPfGroups;
            if (s >= NA) { s -= NA; ph ^= 1u; }
            return true;
        };

        Cur cur;
        cur.tile = (int)blockIdx.x;
        cur.valid = cur.tile < num_tiles;
        cur.fresh = true;
        cur.split = false;
        cur.it = group;
        cur.iters = 0; cur.kb_begin = 0; cur.mt = 0; cur.c = 0; cur.kpos = 0; cur.next_edge = 0;
        cur.code_idx = 0; cur.alpha_idx = 0;
        if (cur.valid) {
            enter_tile(cur);
            while (cur.it >= cur.iters) {
                cur.it -= cur.iters;
                cur.tile += gridDim.x;
                if (cur.tile >= num_tiles) { cur.valid = false; break; }
                enter_tile(cur);
            }
            if (cur.valid) locate(cur);
        }
        uint32_t cvA[2][NL], cvB[2][NL];
        float avA[NSC], avB[NSC];
        if (QM == QM_GENERIC) {
            // q > 4: one set of registers, loaded at the head of the task (under the wait for the slot)
            while (cur.valid && ok) {
                issue(cur, cvA, avA);
                ok = process(cur, cvA, avA);
                advance(cur);
            }
        } else {
            // q <= 4: the loads of the next task are in flight while this one is expanded (two
            // register sets, so that nothing has to wait for a load in order to be moved)
            if (cur.valid) issue(cur, cvA, avA);
            while (cur.valid && ok) {
                Cur nxt = cur;
                advance(nxt);
                if (nxt.valid) issue(nxt, cvB, avB);
                ok = process(cur, cvA, avA);
                cur = nxt;
                if (!cur.valid || !ok) break;
                advance(nxt);
                if (nxt.valid) issue(nxt, cvA, avA);
                ok = process(cur, cvB, avB);
                cur = nxt;
            }
        }
        if (p.helpers && ok && (int)blockIdx.x < num_tiles) {
            // share the epilogue of this CTA's last tile.  Its operand slots are free once the
            // accumulator is complete, so each warp stages its boxes in 1 KiB of the first slots.
            const int lt = (num_tiles - 1 - (int)blockIdx.x) / (int)gridDim.x;
            const int tile = (int)blockIdx.x + lt * (int)gridDim.x;
            int m0, t0, z, kb_begin, iters;
            tile_coords(tile, m0, t0, z, kb_begin, iters);
            const int acc = lt & 1;
            ok = wait_bar(ctl.accum + 8 * acc, (uint32_t)(lt >> 1) & 1u, ctl, 10);
            if (ok) {
                ptx::tc_fence_after_sync();
                const int quarter = warp & 3, helper = 1 + (warp >> 2);  // 1..3
                const int m0w = m0 + quarter * 32;
                const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)acc * kAccCols;
                const uint32_t buf = smem_base + (uint32_t)warp * 1024u;
                const float winv = 1.0f / wscale;  // a power of two
                const int g = lane >> 2, tq = lane & 3;
                float b4[4];
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    b4[i] = (MODE == MODE_FWD && p.bias != nullptr && m0w + g + 8 * i < p.Mdim) ? __ldg(p.bias + m0w + g + 8 * i) : 0.0f;
                bool stored = false;
#pragma unroll 1
                for (int col = 16 * helper; col < TN; col += 16 * kPfHelpers) {
                    if (t0 + col >= p.n || m0w >= p.Mdim) break;  // uniform in the warp
                    if (stored && lane == 0) ptx::bulk_wait_group_read<0>();
                    __syncwarp();
                    const int ta = t0 + col + 2 * tq, tb = ta + 8;
                    const float s0x = (ta < p.n) ? winv * __ldg(p.tok_inv_scale + ta) : 0.0f;
                    const float s0y = (ta + 1 < p.n) ? winv * __ldg(p.tok_inv_scale + ta + 1) : 0.0f;
                    const float s1x = (tb < p.n) ? winv * __ldg(p.tok_inv_scale + tb) : 0.0f;
                    const float s1y = (tb + 1 < p.n) ? winv * __ldg(p.tok_inv_scale + tb + 1) : 0.0f;
                    store_box(t_row, col, buf, s0x, s0y, s1x, s1y, b4, m0w, t0 + col);
                    stored = true;
                }
                if (lane == 0) ptx::bulk_wait_group<0>();
            }
        }
    } else if (pf_epilogue_index(warp) >= 0) {
        // ---------------- epilogue warps: D[row, col] -> out[t0 + col][m0 + row]
        const int ew = pf_epilogue_index(warp);  // 0..3
        const int quarter = warp & 3;       // TMEM lanes 32 * quarter .. + 31
        const int et = ew * 32 + lane;      // 0..127
        const float winv = pow2f(-weight_shift(p.hdr, p.q));
        const uint32_t stg = staging_base + ew * 1024;  // this warp's staging: [tokens][32 rows], 1 KiB (a second one kPfStagingBuf further)
        const int esz = (p.splits > 1 || !p.out_bf16) ? 4 : 2;  // bytes per stored element
        uint8_t* out_base = (p.splits > 1) ? reinterpret_cast<uint8_t*>(p.partial) : reinterpret_cast<uint8_t*>(p.out);
        const long long out_ld = (p.splits > 1) ? (long long)p.Mdim : p.ldo;
        // 16-byte stores need an aligned base and pitch
        const bool vec_ok = ((reinterpret_cast<uintptr_t>(out_base) & 15u) == 0) && ((out_ld * esz) % 16 == 0);
        bool ok = true;
        int lt = 0;
        uint32_t chunks = 0;  // output boxes stored so far (fast path): selects the staging buffer
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++lt) {
            int m0, t0, z, kb_begin, iters;
            tile_coords(tile, m0, t0, z, kb_begin, iters);
            const int acc = lt & 1;
            const uint32_t acc_ph = (lt >> 1) & 1;
            for (int i = et; i < TN; i += kPfEpiWarps * 32)
                scale[i] = (t0 + i < p.n) ? winv * __ldg(p.tok_inv_scale + t0 + i) : 0.0f;
            // one warp polls the accumulator's barrier (a whole tile away), the others park on the
            // hardware barrier that also publishes the scale row; a timeout shows in the abort flag
            if (ew == 0) wait_bar(ctl.accum + 8 * acc, acc_ph, ctl, 7, 1000u);
            asm volatile("bar.sync 2, %0;" ::"n"(kPfEpiWarps * 32) : "memory");
            if (*ctl.abort_flag) { ok = false; break; }
            ptx::tc_fence_after_sync();
            // accumulator row `lane` of this warp's quarter is output column m0w + lrow
            const int m0w = m0 + quarter * 32;
            const int lrow = lane;
            const float bias = (MODE == MODE_FWD && p.bias != nullptr && p.splits == 1 && m0w + lrow < p.Mdim)
                                   ? __ldg(p.bias + m0w + lrow) : 0.0f;
            uint8_t* tile_out = out_base + ((p.splits > 1) ? (long long)z * p.n * p.Mdim * 4 : 0);
            const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)acc * kAccCols;
            const bool full_rows = vec_ok && (m0w + 32 <= p.Mdim);
            if (p.fast_epi) {
                const int g = lane >> 2, tq = lane & 3;
                float b4[4];
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    b4[i] = (MODE == MODE_FWD && p.bias != nullptr && m0w + g + 8 * i < p.Mdim) ? __ldg(p.bias + m0w + g + 8 * i) : 0.0f;
                const int cstep = (p.helpers && is_last_tile(tile)) ? 16 * kPfHelpers : 16;  // the workers take the other boxes
#pragma unroll 1
                for (int col = 0; col < TN; col += cstep) {
                    if (t0 + col >= p.n || m0w >= p.Mdim) break;  // uniform in the warp
                    // the store that last read this buffer has to be done with it
                    if (p.epi_bufs == 2) {
                        if (chunks >= 2 && lane == 0) ptx::bulk_wait_group_read<1>();
                    } else {
                        if (chunks >= 1 && lane == 0) ptx::bulk_wait_group_read<0>();
                    }
                    __syncwarp();
                    const uint32_t buf = stg + ((p.epi_bufs == 2) ? (chunks & 1u) * kPfStagingBuf : 0u);
                    float s0x, s0y, s1x, s1y;
                    asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(s0x), "=f"(s0y) : "r"(scale_addr + (col + 2 * tq) * 4) : "memory");
                    asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(s1x), "=f"(s1y) : "r"(scale_addr + (col + 8 + 2 * tq) * 4) : "memory");
                    store_box(t_row, col, buf, s0x, s0y, s1x, s1y, b4, m0w, t0 + col);
                    ++chunks;
                }
            }
            // one token's 32 rows are 64 (bf16) or 128 (fp32) bytes: `pieces` 16-byte vectors
            const int pieces = 2 * esz;
            const int toks = 1024 / (32 * esz);  // tokens per staging round: 16 (bf16) or 8 (fp32)
#pragma unroll 1
            for (int col = 0; col < TN && !p.fast_epi; col += 16) {
                if (t0 + col >= p.n) break;  // uniform in the warp
                uint32_t v[16];
                ptx::tmem_ld_x16(t_row + (uint32_t)col, v);
                ptx::tmem_ld_wait();
                // transpose through shared memory: staging[token][row], then 16-byte pieces of one
                // token's 32 rows go out as coalesced vector stores
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    if (esz == 2) {
                        if (half == 1) break;
#pragma unroll
                        for (int c = 0; c < 16; ++c) {
                            const __nv_bfloat16 h = __float2bfloat16_rn(__uint_as_float(v[c]) * scale[col + c] + bias);
                            asm volatile("st.shared.b16 [%0], %1;" ::"r"(stg + c * 64 + lrow * 2),
                                         "h"(*reinterpret_cast<const unsigned short*>(&h)) : "memory");
                        }
                    } else {
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            const float f = __uint_as_float(v[8 * half + c]) * scale[col + 8 * half + c] + bias;
                            asm volatile("st.shared.b32 [%0], %1;" ::"r"(stg + c * 128 + lrow * 4), "f"(f) : "memory");
                        }
                    }
                    __syncwarp();
                    const int tbase = t0 + col + ((esz == 4) ? 8 * half : 0);
                    for (int pc = lane; pc < toks * pieces; pc += 32) {
                        const int c = pc / pieces, seg = pc - c * pieces;
                        const int t = tbase + c;
                        if (t >= p.n) continue;
                        uint32_t r0, r1, r2, r3;
                        asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                                     : "r"(stg + pc * 16) : "memory");
                        uint8_t* dst = tile_out + ((long long)t * out_ld + m0w) * esz + seg * 16;
                        if (full_rows) {
                            *reinterpret_cast<uint4*>(dst) = make_uint4(r0, r1, r2, r3);
                        } else {
                            const uint32_t rr[4] = {r0, r1, r2, r3};
                            const int per = 16 / esz;  // elements in this piece
#pragma unroll
                            for (int e2 = 0; e2 < 8; ++e2) {
                                if (e2 < per && m0w + seg * per + e2 < p.Mdim) {
                                    if (esz == 2)
                                        reinterpret_cast<unsigned short*>(dst)[e2] =
                                            (unsigned short)(rr[e2 >> 1] >> ((e2 & 1) * 16));
                                    else
                                        reinterpret_cast<uint32_t*>(dst)[e2] = rr[e2 & 3];
                                }
                            }
                        }
                    }
                    __syncwarp();
                }
            }
            // the accumulator (and this tile's scale row) may be reused
            ptx::tc_fence_before_sync();
            asm volatile("bar.sync 2, %0;" ::"n"(kPfEpiWarps * 32) : "memory");
            if (lane == 0) ptx::mbar_arrive(acc_empty + 8 * acc);
        }
        if (p.fast_epi && lane == 0) ptx::bulk_wait_group<0>();  // all output boxes written before the CTA ends
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == kPfMmaWarp) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, kTmemCols);
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
// decode: n <= 16 tokens, no pre-pass; the workers write both operands
// ------------------------------------------------------------------------------------------

struct DecodeParams {
    int d_out, d_in, q, g, G, pitch, n;
    int num_kb, kb_per_split, splits;
    const float* alpha;
    const float* bias;
    const __nv_bfloat16* X;
    long long ldx;
    void* out;
    long long ldo;
    int out_bf16;
    float* partial;  // [splits][n][d_out]
};

constexpr int kDecTN = 16;
constexpr int kDecStages = 4;

// Scale of one weight row in decode: the largest |alpha| of the row over every plane and every
// group inside the CTA's K slice, times q (a bound on any level sum_i +-alpha_i), is brought to
// [2^13, 2^14), so no level of the slice can leave the fp16 range.
__device__ __forceinline__ int decode_row_shift(const float* __restrict__ alpha, long long plane_alpha, int G,
                                                int q, int j, int c_lo, int c_hi) {
    uint32_t am = 0u;
    for (int i = 0; i < q; ++i)
        for (int c = c_lo; c <= c_hi; ++c)
            am = max(am, __float_as_uint(__ldg(alpha + i * plane_alpha + (long long)j * G + c)) & 0x7FFFFFFFu);
    return shift_for(exponent_of_bits(__float_as_uint(__uint_as_float(am) * (float)q)), 13);
}

template <int QM>
__global__ void __launch_bounds__(kThreads, 2)
decode_kernel(const __grid_constant__ CUtensorMap tmap_bits, const DecodeParams p) {
    using L = StageLayout<MODE_FWD, kDecTN, QM>;
    constexpr int STAGES = kDecStages;
    constexpr uint32_t kStageBytes = L::kStageBytes;
    constexpr uint32_t kIdesc = ptx::make_idesc_bf16(kBlockM, kDecTN, 0, 0) & ~((1u << 7) | (1u << 10));

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
    ctl.device_flag = &g_timeout_flag;
    float* tok_scale = reinterpret_cast<float*>(ctl_gen + 24 * STAGES + 32);  // [16] scale, [16] inverse

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int m0 = blockIdx.x * kBlockM;
    const int kb_begin = blockIdx.y * p.kb_per_split;
    const int kb_end = min(p.num_kb, kb_begin + p.kb_per_split);
    const int iters = kb_end - kb_begin;
    const int k_lo = kb_begin * kBlockK;
    const int k_hi = min(kb_end * kBlockK, p.d_in);
    const int c_lo = min(k_lo / p.g, p.G - 1), c_hi = min((k_hi - 1) / p.g, p.G - 1);
    const long long plane_alpha = (long long)p.d_out * p.G;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(ctl.full + 8 * s, 1);
            ptx::mbar_init(ctl.aready + 8 * s, kWorkerWarps);
            ptx::mbar_init(ctl.empty + 8 * s, 1);
        }
        ptx::mbar_init(ctl.accum, 1);
        ptx::mbar_init(ctl.spare, 1);
        *ctl.abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tmap_bits);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(const_cast<uint32_t*>(tmem_holder)), TmemCols<kDecTN>::value);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_holder;

    if (warp == 0) {
        // ---------------- TMA producer: plane words only
        if (lane == 0) {
            bool ok = true;
            int issued = 0;
            const uint32_t tx = (uint32_t)p.q * L::kPlaneBytes;
            for (int it = 0; it < iters && ok; ++it) {
                const int s = it % STAGES;
                const uint32_t ph = (it / STAGES) & 1;
                const int kb = kb_begin + it;
                ok = wait_bar(ctl.empty + 8 * s, ph ^ 1u, ctl, 20);
                if (!ok) break;
                ptx::mbar_arrive_expect_tx(ctl.full + 8 * s, tx);
                ptx::tma_load_3d(smem_base + s * kStageBytes + L::kBitsOff, &tmap_bits, (kb >> 1) * 4, m0, 0,
                                 ctl.full + 8 * s);
                issued = it + 1;
            }
            if (!ok)
                for (int it = max(0, issued - STAGES); it < issued; ++it)
                    wait_bar(ctl.full + 8 * (it % STAGES), (it / STAGES) & 1, ctl, 25);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            bool ok = true;
            for (int it = 0; it < iters && ok; ++it) {
                const int s = it % STAGES;
                const uint32_t ph = (it / STAGES) & 1;
                ok = wait_bar(ctl.aready + 8 * s, ph, ctl, 21);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint32_t sa = smem_base + s * kStageBytes;
                const uint32_t sb = sa + kABytes;
#pragma unroll
                for (int kk = 0; kk < kBlockK / 16; ++kk)
                    ptx::umma_bf16(tmem_base, ptx::make_smem_desc(sa + kk * 32, 16, 1024),
                                   ptx::make_smem_desc(sb + kk * 32, 16, 1024), kIdesc,
                                   (it > 0 || kk > 0) ? 1u : 0u);
                ptx::umma_commit(ctl.empty + 8 * s);
            }
            if (ok) {
                ptx::umma_commit(ctl.accum);
            } else {
                ptx::umma_commit(ctl.spare);
                wait_bar(ctl.spare, 0, ctl, 22);
            }
        }
    } else {
        const int wid = warp - kWorkerWarp0;
        const int e = wid * 32 + lane;  // 0..255
        const int row = wid * 16 + (lane >> 1);
        const int half = lane & 1;
        const int j = m0 + row;
        const bool valid = j < p.d_out;
        const uint32_t lx = row & 7;

        // ---- per-token scale over this CTA's K slice: thread = (token e / 16, every 16th vector)
        {
            const int t = e >> 4, sub = e & 15;
            uint32_t m = 0u;
            if (t < p.n) {
                const __nv_bfloat16* xrow = p.X + (long long)t * p.ldx;
                for (int k = k_lo + sub * 8; k < k_hi; k += 128) {
                    const uint4 x = __ldg(reinterpret_cast<const uint4*>(xrow + k));
                    const uint32_t xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                    for (int el = 0; el < 8; ++el)
                        if (k + el < p.d_in) m = max(m, (xs[el >> 1] >> ((el & 1) * 16)) & 0x7FFFu);
                }
            }
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
            if (sub == 0) {
                const int sh = shift_for(exponent_of_bits(m << 16), 14);
                tok_scale[t] = pow2f(sh);
                tok_scale[16 + t] = pow2f(-sh);
            }
        }
        const float wscale = valid ? pow2f(decode_row_shift(p.alpha, plane_alpha, p.G, p.q, j, c_lo, c_hi)) : 1.0f;
        asm volatile("bar.sync 1, %0;" ::"n"(kWorkers) : "memory");  // tok_scale visible to all workers

        // activation task of threads e < 128: (token e / 8, 8 consecutive k = one 16-byte chunk)
        const int xt = e >> 3, xch = e & 7;
        const bool x_task = e < 128;
        const float xscale = x_task ? tok_scale[xt] : 0.0f;
        auto fetch_x = [&](uint4& slot, int kb) {
            const int k = kb * kBlockK + xch * 8;
            slot = make_uint4(0u, 0u, 0u, 0u);
            if (x_task && xt < p.n && k < p.d_in)
                slot = __ldg(reinterpret_cast<const uint4*>(p.X + (long long)xt * p.ldx + k));
        };

        const int cstep = max(1, kBlockK / p.g);
        auto group_of = [&](int kb) { return min((kb * kBlockK + half * 32) / p.g, p.G - 1); };
        AlphaSet<QM> cur, nxt;
        int c_cur = (iters > 0) ? group_of(kb_begin) : 0;
        load_alpha<QM>(cur, p.alpha, plane_alpha, p.G, p.q, j, c_cur, valid, wscale);
        load_alpha<QM>(nxt, p.alpha, plane_alpha, p.G, p.q, j, min(c_cur + cstep, p.G - 1), valid, wscale);
        uint4 xring[kPrefetch];
#pragma unroll
        for (int d = 0; d < kPrefetch; ++d)
            if (d < iters) fetch_x(xring[d], kb_begin + d);

        Lut lut = {0u, 0u, 0u, 0u};
        int lut_key = -2;
        bool ok = true;
        for (int it0 = 0; it0 < iters && ok; it0 += kPrefetch) {
#pragma unroll
            for (int d = 0; d < kPrefetch; ++d) {
                const int it = it0 + d;
                if (it < iters && ok) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1;
                    const int kb = kb_begin + it;
                    const uint4 xcur = xring[d];
                    if (it + kPrefetch < iters) fetch_x(xring[d], kb + kPrefetch);
                    const int c = group_of(kb);
                    if (c != c_cur) {
                        cur = nxt;
                        c_cur = c;
                        load_alpha<QM>(nxt, p.alpha, plane_alpha, p.G, p.q, j, min(c + cstep, p.G - 1), valid, wscale);
                    }
                    ok = wait_bar(ctl.full + 8 * s, ph, ctl, 23);
                    if (ok) {
                        const uint32_t st = smem_base + s * kStageBytes;
                        const uint32_t baddr = st + L::kBitsOff + row * 16 + (((kb & 1) * 2 + half) << 2);
                        expand_task32<QM>(cur, baddr, L::kPlaneBytes, lut, lut_key, p.q, st + row * 128, lx, half * 4);
                        if (x_task) {
                            const uint32_t xs[4] = {xcur.x, xcur.y, xcur.z, xcur.w};
                            float f[8];
#pragma unroll
                            for (int el = 0; el < 8; ++el) {
                                const uint32_t b = (xs[el >> 1] >> ((el & 1) * 16)) & 0xFFFFu;
                                f[el] = (kb * kBlockK + xch * 8 + el < p.d_in) ? __uint_as_float(b << 16) * xscale
                                                                             : 0.0f;
                            }
                            ptx::st_shared_v4(st + kABytes + xt * 128 + ((xch ^ (xt & 7)) << 4),
                                              pack_half2(f[0], f[4]), pack_half2(f[1], f[5]),
                                              pack_half2(f[2], f[6]), pack_half2(f[3], f[7]));
                        }
                        ptx::fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(ctl.aready + 8 * s);
                    }
                }
            }
        }

        // ---- epilogue: thread = (TMEM lane = weight row, tokens 8*eh .. 8*eh+7)
        if (ok) ok = wait_bar(ctl.accum, 0, ctl, 24);
        const int quarter = warp & 3, eh = wid >> 2;
        if (ok && eh * 8 < p.n) {
            ptx::tc_fence_after_sync();
            uint32_t v[8];
            ptx::tmem_ld_x8(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(eh * 8), v);
            ptx::tmem_ld_wait();
            const int je = m0 + quarter * 32 + lane;
            if (je < p.d_out) {
                const float winv = pow2f(-decode_row_shift(p.alpha, plane_alpha, p.G, p.q, je, c_lo, c_hi));
                const float bias = (p.bias != nullptr && p.splits == 1) ? __ldg(p.bias + je) : 0.0f;
#pragma unroll
                for (int cidx = 0; cidx < 8; ++cidx) {
                    const int t = eh * 8 + cidx;
                    if (t < p.n) {
                        const float val = __uint_as_float(v[cidx]) * (winv * tok_scale[16 + t]);
                        if (p.splits > 1)
                            p.partial[((long long)blockIdx.y * p.n + t) * p.d_out + je] = val;
                        else if (p.out_bf16)
                            reinterpret_cast<__nv_bfloat16*>(p.out)[(long long)t * p.ldo + je] =
                                __float2bfloat16_rn(val + bias);
                        else
                            reinterpret_cast<float*>(p.out)[(long long)t * p.ldo + je] = val + bias;
                    }
                }
            }
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, TmemCols<kDecTN>::value);
    }
}

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------

struct ExpandPlan {
    int TN, splits, kb_per_split, num_kb, m_tiles, n_tiles;
    int a_slots, b_slots, epi_bufs;
    uint32_t bits_bytes, alpha_bytes;                                    // one stage's chunk of the planes; the scales of one (row block, group)
    size_t planes_bytes;                                                 // the regrouped planes (codes for q <= 4)
    size_t smem;                                                         // dynamic shared memory of the GEMM kernel
    size_t off_tok, off_act, off_alpha, off_bits, off_partial, total;  // workspace layout (bytes)
    int ld_act;                                                          // pitch of the fp16 activations (elements)
};

constexpr int kPfStageFixed = 224;                                     // fixed cost of a pipeline stage, in token-tile columns
constexpr size_t kSmemLimit = 232448;                                   // 227 KiB per CTA
constexpr size_t kPfFixedBytes = 1024 + kPfCtlBytes + kPfScaleBytes;   // alignment slack, barriers, output scales

// Tile width over tokens, the K split and the pipeline geometry.  Wide token tiles amortise the
// expansion of a weight tile over more tokens; the K split fills the SMs when the output has few
// tiles.
ExpandPlan plan_expand(int mode, int d_out, int d_in, int q, int g, int n) {
    ExpandPlan pl;
    const int sms = sm_count();
    const int Mdim = (mode == MODE_FWD) ? d_out : d_in;
    const int Kdim = (mode == MODE_FWD) ? d_in : d_out;
    const int G = (int)bcq_num_groups(d_in, g);
    pl.m_tiles = ceil_div(Mdim, kBlockM);
    pl.num_kb = ceil_div(Kdim, kBlockK);
    int tn;
    if (n <= 32) tn = 32;
    else if (n <= 64) tn = 64;
    else if (n <= 128) tn = 128;
    else {
        // Any multiple of 16 up to 256 is a legal UMMA width.  A stage of the kernel takes a fixed
        // time (barriers, UMMA issue, the expansion of one weight tile whatever the width) plus a
        // time in proportion to the width (the UMMAs themselves); measured, the fixed part is worth
        // about kPfStageFixed columns.  The kernel is persistent with ceil(tiles / SMs) tiles per
        // CTA, so a narrower tile can shorten the call (fewer tiles per CTA, less padding past n)
        // but costs SM time that kernels running beside this one would have used.  The width
        // that minimises call time x SM time wins; ties go to the wider tile.
        long long best = -1;
        tn = 256;
        for (int c = 256; c >= 128; c -= 16) {
            const long long tiles = (long long)pl.m_tiles * ceil_div(n, c);
            const long long per_cta = (tiles + sms - 1) / sms;
            const long long stage = c + kPfStageFixed;
            const long long cost = (per_cta * stage) * (tiles * stage);
            if (best < 0 || cost < best) { best = cost; tn = c; }
        }
    }
    pl.TN = tn;
    pl.n_tiles = ceil_div(n, tn);
    const int tiles = pl.m_tiles * pl.n_tiles;
    // The K split goes through fp32 partials, a slower epilogue and a second kernel: only for
    // problems that would otherwise leave most of the SMs idle.
    int splits = (4 * tiles <= sms) ? sms / tiles : 1;
    if (splits < 1) splits = 1;
    const int max_splits = (pl.num_kb + 3) / 4;  // at least 4 K blocks per CTA
    if (splits > max_splits) splits = max_splits;
    if (splits > 32) splits = 32;
    pl.kb_per_split = ceil_div(pl.num_kb, splits);
    pl.splits = ceil_div(pl.num_kb, pl.kb_per_split);

    const int rows = (mode == MODE_FWD) ? 128 : 64;
    pl.bits_bytes = (q <= 3 ? 3u : (uint32_t)q) * 1024u;  // q <= 4: selector codes (3 or 4 words per 32 weights)
    pl.alpha_bytes = (uint32_t)(q * rows * 4);
    // Shared memory.  A worker group takes a few hundred nanoseconds from "the tensor core is done
    // with my slot" to "the slot holds the next tile", and a TMA load about a microsecond to land;
    // both rings must be deep enough to cover that at one stage per ~0.3 us.  First choice that fits:
    const size_t b_bytes = (size_t)tn * kBlockK * 2;
    auto smem_of = [&](int a_slots, int b_slots, int epi_bufs) {
        return a_slots * (size_t)kABytes + b_slots * b_bytes + epi_bufs * (size_t)kPfStagingBuf + kPfFixedBytes;
    };
    const int rings[8][2] = {{6, 5}, {5, 5}, {6, 4}, {5, 4}, {4, 4}, {4, 3}, {3, 3}, {3, 2}};
    pl.epi_bufs = 2;
    pl.a_slots = kPfGroups;
    pl.b_slots = 2;
    for (int r = 0; r < 8; ++r)
        if (smem_of(rings[r][0], rings[r][1], pl.epi_bufs) <= kSmemLimit) {
            pl.a_slots = rings[r][0];
            pl.b_slots = rings[r][1];
            break;
        }
    pl.smem = smem_of(pl.a_slots, pl.b_slots, pl.epi_bufs);

    const size_t chunks_bits = (size_t)pl.m_tiles * pl.num_kb;                       // [m_tile][kb] or [u][jb]
    const size_t blocks_alpha = (size_t)((mode == MODE_FWD) ? pl.m_tiles : pl.num_kb) * G;  // [m_tile][G] or [jb][G]
    pl.ld_act = (int)align_up((size_t)Kdim, 8);
    pl.off_tok = align_up(sizeof(WsHeader), 128);
    pl.off_act = align_up(pl.off_tok + (size_t)n * sizeof(float), 128);
    pl.off_alpha = align_up(pl.off_act + (size_t)n * pl.ld_act * 2, 128);
    pl.off_bits = align_up(pl.off_alpha + blocks_alpha * pl.alpha_bytes, 128);
    pl.planes_bytes = chunks_bits * pl.bits_bytes;
    pl.off_partial = align_up(pl.off_bits + pl.planes_bytes, 128);
    pl.total = pl.off_partial + (pl.splits > 1 ? (size_t)pl.splits * n * Mdim * sizeof(float) : 0);
    return pl;
}

struct DecodePlan {
    int m_tiles, num_kb, splits, kb_per_split;
    size_t total;
};

DecodePlan plan_decode(int d_out, int d_in, int n) {
    DecodePlan pl;
    const int sms = sm_count();
    pl.m_tiles = ceil_div(d_out, kBlockM);
    pl.num_kb = ceil_div(d_in, kBlockK);
    int splits = (2 * sms) / pl.m_tiles;  // 72 KiB of shared memory per CTA: several CTAs per SM
    if (splits < 1) splits = 1;
    const int max_splits = (pl.num_kb + 7) / 8;  // at least 8 K blocks per CTA
    if (splits > max_splits) splits = max_splits;
    if (splits > 64) splits = 64;
    pl.kb_per_split = ceil_div(pl.num_kb, splits);
    pl.splits = ceil_div(pl.num_kb, pl.kb_per_split);
    pl.total = pl.splits > 1 ? (size_t)pl.splits * n * d_out * sizeof(float) : 0;
    return pl;
}

template <int MODE>
bcq_status ensure_expand_smem(int q, size_t smem) {
    if (q <= 3) return ensure_dynamic_smem(expand_gemm_kernel<MODE, QM_LUT3>, smem);
    if (q == 4) return ensure_dynamic_smem(expand_gemm_kernel<MODE, QM_LUT4>, smem);
    return ensure_dynamic_smem(expand_gemm_kernel<MODE, QM_GENERIC>, smem);
}

template <int MODE, int QM>
bcq_status launch_expand(const CUtensorMap& tm, const CUtensorMap& tmo, const ExpandParams& p, const ExpandPlan& pl,
                         cudaStream_t stream) {
    auto kern = expand_gemm_kernel<MODE, QM>;
    bcq_status st0 = ensure_dynamic_smem(kern, pl.smem);
    if (st0 != BCQ_OK) return st0;
    const int tiles = pl.m_tiles * pl.n_tiles * pl.splits;
    // persistent, at most one CTA per SM; with more tiles than SMs every CTA gets the same number of
    // tiles (as many as the busiest would get anyway): fewer CTAs pay the prologue, more epilogues
    // overlap the next tile's main loop, and the SMs left over can run other kernels
    const int per_cta = ceil_div(tiles, sm_count());
    const int grid = ceil_div(tiles, per_cta);
    kern<<<grid, kPfThreads, pl.smem, stream>>>(tm, tmo, p);
    bcq::count_launch();
    BCQ_CUDA_TRY(cudaGetLastError());
    return BCQ_OK;
}

template <int MODE>
bcq_status launch_expand_q(const CUtensorMap& tm, const CUtensorMap& tmo, const ExpandParams& p, const ExpandPlan& pl,
                           cudaStream_t stream) {
    if (p.q <= 3) return launch_expand<MODE, QM_LUT3>(tm, tmo, p, pl, stream);
    if (p.q == 4) return launch_expand<MODE, QM_LUT4>(tm, tmo, p, pl, stream);
    return launch_expand<MODE, QM_GENERIC>(tm, tmo, p, pl, stream);
}

// act: bf16 [n][ldact] with Kdim valid columns (X for the forward, dY for dX).
// Writes the selector codes of the planes (q <= 4) in the chunk order of mode `mode`.
bcq_status launch_code_planes(int mode, int d_out, int d_in, int q, const ExpandPlan& pl, const uint32_t* bits,
                              uint32_t* codes, cudaStream_t s) {
    const int pitch = (int)bcq_pitch_words(d_in);
    const int rows_padded = (mode == MODE_FWD) ? pl.m_tiles * 128 : pl.num_kb * 64;
    const int words_padded = (mode == MODE_FWD) ? pl.num_kb * 2 : pl.m_tiles * 4;
    const long long total = (long long)rows_padded * words_padded;
    const unsigned grid = (unsigned)((total + 255) / 256);
    if (q == 4)
        code_planes_kernel<4><<<grid, 256, 0, s>>>(mode, d_out, pitch, q, rows_padded, words_padded, pl.num_kb, bits, codes);
    else
        code_planes_kernel<3><<<grid, 256, 0, s>>>(mode, d_out, pitch, q, rows_padded, words_padded, pl.num_kb, bits, codes);
    bcq::count_launch();
    BCQ_CUDA_TRY(cudaGetLastError());
    return BCQ_OK;
}

// act: bf16 [n][ldact] with Kdim valid columns (X for the forward, dY for dX).  `prepared`: the
// planes as written by bcq_prepare_planes for this mode, or null (then `bits` is regrouped into
// the workspace by this call).
template <int MODE>
bcq_status run_expand(int d_out, int d_in, int q, int g, int n, const void* act, size_t ldact,
                      const uint32_t* bits, const void* prepared, const float* alpha, const float* bias, void* out,
                      size_t ldo, int out_dtype, void* ws, size_t ws_bytes, void* stream) {
    const int Mdim = (MODE == MODE_FWD) ? d_out : d_in;
    const int Kdim = (MODE == MODE_FWD) ? d_in : d_out;
    const ExpandPlan pl = plan_expand(MODE, d_out, d_in, q, g, n);
    // the kernel indexes the regrouped planes and scales with 32-bit word offsets
    if ((pl.planes_bytes >> 2) >= (1ull << 32) || (pl.off_bits - pl.off_alpha) / 4 >= (1ull << 32)) return BCQ_ERR_UNSUPPORTED;
    if (ws == nullptr) return BCQ_ERR_NULL;
    if (ws_bytes < pl.total) return BCQ_ERR_WORKSPACE;
    if (!aligned16(ws)) return BCQ_ERR_ALIGN;
    cudaStream_t s = (cudaStream_t)stream;
    uint8_t* wsb = reinterpret_cast<uint8_t*>(ws);
    WsHeader* hdr = reinterpret_cast<WsHeader*>(wsb);
    float* tok = reinterpret_cast<float*>(wsb + pl.off_tok);
    __half* act16 = reinterpret_cast<__half*>(wsb + pl.off_act);
    const int pitch = (int)bcq_pitch_words(d_in);

    CUtensorMap tm;
    bcq_status st = make_tmap_16bit(&tm, act16, 1, pl.ld_act, n, (size_t)pl.ld_act, pl.TN);
    if (st != BCQ_OK) return st;

    // everything that can fail is done before the first launch: the output tensor map and the
    // shared-memory limits of the kernels this call may run
    const bool fast_epi = (out_dtype == BCQ_BF16 && pl.splits == 1 && aligned16(out) && (ldo * 2) % 16 == 0 &&
                           ldo >= (size_t)Mdim);
    CUtensorMap tmo = tm;
    if (fast_epi) {
        st = make_tmap_out_bf16(&tmo, out, Mdim, n, ldo);
        if (st != BCQ_OK) return st;
    }
    if ((st = ensure_expand_smem<MODE>(q, pl.smem)) != BCQ_OK) return st;

    PrepParams pp;
    pp.n = n; pp.K = Kdim; pp.act_blocks = n;
    pp.ld_in = (long long)ldact; pp.ld_out = pl.ld_act;
    pp.in = reinterpret_cast<const __nv_bfloat16*>(act); pp.out = act16; pp.tok_inv_scale = tok;
    pp.alpha = alpha; pp.alpha_count = (long long)bcq_alpha_count(d_out, d_in, q, g); pp.hdr = hdr;
    long long ablocks = (pp.alpha_count + 256 * 16 - 1) / (256 * 16);
    if (ablocks > kMaxAlphaBlocks) ablocks = kMaxAlphaBlocks;
    if (ablocks < 1) ablocks = 1;
    pp.mode = MODE; pp.d_out = d_out; pp.q = q; pp.G = (int)bcq_num_groups(d_in, g); pp.pitch = pitch;
    pp.num_kb = pl.num_kb;
    pp.amax_blocks = (int)ablocks;
    pp.row_tiles = ceil_div(d_out, 128);
    pp.bits_cblk = ceil_div(pitch, 32);
    pp.alpha_cblk = ceil_div(pp.G, 32);
    const bool coded = q <= 4;  // selector codes (written once, or by the launch below); q > 4: plane words
    pp.bits_blocks = coded ? 0 : q * pp.row_tiles * pp.bits_cblk;
    const int alpha_tr_blocks = q * pp.row_tiles;  // one block per (plane, tile of 128 rows)
    pp.bits = bits;
    pp.alpha_t = reinterpret_cast<float*>(wsb + pl.off_alpha);
    pp.bits_t = reinterpret_cast<uint32_t*>(wsb + pl.off_bits);
    if (coded && prepared == nullptr) {
        if ((st = launch_code_planes(MODE, d_out, d_in, q, pl, bits, pp.bits_t, s)) != BCQ_OK) return st;
    }
    const int tok_blocks = ceil_div(n, kPrepTokensPerBlock);
    pp.act_blocks = tok_blocks;
    const unsigned pgrid = (unsigned)(tok_blocks + ablocks + pp.bits_blocks + alpha_tr_blocks);
    const int nvec = (Kdim + 7) / 8;
    // Rows of up to 1024 elements stay in registers between the two passes over them.  Longer
    // rows are read twice instead (the second time from L2), four loads of a lane at a time:
    // holding them costs so many registers that the blocks resident on an SM are too few to
    // cover the memory latency (measured: 14.8 us against 11.3 us for 4096 rows of 1600).
    if (nvec <= 32 * 4) prepare_kernel<4><<<pgrid, 256, 0, s>>>(pp);
    else prepare_kernel<0><<<pgrid, 256, 0, s>>>(pp);
    bcq::count_launch();
    BCQ_CUDA_TRY(cudaGetLastError());

    ExpandParams p;
    p.d_out = d_out; p.d_in = d_in; p.q = q; p.g = g;
    p.G = (int)bcq_num_groups(d_in, g);
    p.pitch = pitch;
    p.n = n; p.Mdim = Mdim; p.num_kb = pl.num_kb; p.kb_per_split = pl.kb_per_split; p.splits = pl.splits;
    p.m_tiles = pl.m_tiles; p.n_tiles = pl.n_tiles;
    p.tn = pl.TN;
    p.acc_cols = 32;
    while ((int)p.acc_cols < pl.TN) p.acc_cols *= 2;
    p.a_slots = pl.a_slots; p.b_slots = pl.b_slots; p.epi_bufs = pl.epi_bufs; p.chunk_words = pl.bits_bytes / 4;
    p.bits_t = (coded && prepared != nullptr) ? reinterpret_cast<const uint32_t*>(prepared) : pp.bits_t;
    p.alpha_t = pp.alpha_t; p.bias = bias; p.hdr = hdr; p.tok_inv_scale = tok;
    p.out = out; p.ldo = (long long)ldo; p.out_bf16 = (out_dtype == BCQ_BF16);
    p.partial = reinterpret_cast<float*>(wsb + pl.off_partial);
    // bf16 output with an aligned base and pitch and no K split goes out through TMA stores
    p.fast_epi = fast_epi ? 1 : 0;
    // The workers find the last tile's accumulator by barrier parity alone.  They run at most
    // `a_slots` pipeline stages ahead of the tensor core, so the parity is unambiguous only if
    // two tiles are longer than that: then the accumulator's previous use (two tiles back) is
    // certain to be complete when a worker has finished the last tile's stages.
    p.helpers = (p.fast_epi && 2 * pl.num_kb >= pl.a_slots + 2) ? 1 : 0;
    st = launch_expand_q<MODE>(tm, tmo, p, pl, s);
    if (st != BCQ_OK) return st;
    if (pl.splits > 1) {
        const long long total = (long long)n * Mdim;
        splitk_reduce_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(
            n, Mdim, pl.splits, p.partial, bias, out, (long long)ldo, p.out_bf16);
    bcq::count_launch();
        BCQ_CUDA_TRY(cudaGetLastError());
    }
    return BCQ_OK;
}

template <int QM>
bcq_status launch_decode(const CUtensorMap& tm_bits, const DecodeParams& p, const DecodePlan& pl,
                         cudaStream_t s) {
    constexpr size_t smem = (size_t)kDecStages * StageLayout<MODE_FWD, kDecTN, QM>::kStageBytes + 1024 + 512;
    auto kern = decode_kernel<QM>;
    bcq_status st0 = ensure_dynamic_smem(kern, smem);
    if (st0 != BCQ_OK) return st0;
    dim3 grid((unsigned)pl.m_tiles, (unsigned)pl.splits);
    kern<<<grid, kThreads, smem, s>>>(tm_bits, p);
    bcq::count_launch();
    BCQ_CUDA_TRY(cudaGetLastError());
    return BCQ_OK;
}

bcq_status run_decode(int d_out, int d_in, int q, int g, int n, const void* X, size_t ldx,
                      const uint32_t* bits, const float* alpha, const float* bias, void* Y, size_t ldy,
                      int y_dtype, void* ws, size_t ws_bytes, void* stream) {
    const DecodePlan pl = plan_decode(d_out, d_in, n);
    if (pl.total > 0) {
        if (ws == nullptr) return BCQ_ERR_NULL;
        if (ws_bytes < pl.total) return BCQ_ERR_WORKSPACE;
        if (!aligned16(ws)) return BCQ_ERR_ALIGN;
    }
    DecodeParams p;
    p.d_out = d_out; p.d_in = d_in; p.q = q; p.g = g;
    p.G = (int)bcq_num_groups(d_in, g);
    p.pitch = (int)bcq_pitch_words(d_in);
    p.n = n; p.num_kb = pl.num_kb; p.kb_per_split = pl.kb_per_split; p.splits = pl.splits;
    p.alpha = alpha; p.bias = bias;
    p.X = reinterpret_cast<const __nv_bfloat16*>(X); p.ldx = (long long)ldx;
    p.out = Y; p.ldo = (long long)ldy; p.out_bf16 = (y_dtype == BCQ_BF16);
    p.partial = reinterpret_cast<float*>(ws);
    CUtensorMap tm_bits;
    bcq_status st = make_tmap_bits(&tm_bits, bits, d_out, p.pitch, q, 128);
    if (st != BCQ_OK) return st;
    cudaStream_t s = (cudaStream_t)stream;
    if (q <= 3) st = launch_decode<QM_LUT3>(tm_bits, p, pl, s);
    else if (q == 4) st = launch_decode<QM_LUT4>(tm_bits, p, pl, s);
    else st = launch_decode<QM_GENERIC>(tm_bits, p, pl, s);
    if (st != BCQ_OK) return st;
    if (pl.splits > 1) {
        const long long total = (long long)n * d_out;
        splitk_reduce_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(
            n, d_out, pl.splits, p.partial, bias, Y, (long long)ldy, p.out_bf16);
    bcq::count_launch();
        BCQ_CUDA_TRY(cudaGetLastError());
    }
    return BCQ_OK;
}

// Argument checks of the forward and decode entry points (host arithmetic and pointer tests only).
bcq_status check_fwd_args(int decode, int d_out, int d_in, int q, int g, int n, const void* X, size_t ldx,
                          const uint32_t* bits, const float* alpha, const void* Y, size_t ldy, int y_dtype) {
    bcq_status st = check_shape(d_out, d_in, q, g);
    if (st != BCQ_OK) return st;
    if (n < 1 || (decode && n > 16)) return BCQ_ERR_SHAPE;
    if (!bits || !alpha || !Y) return BCQ_ERR_NULL;
    if ((st = check_act(X, ldx, d_in)) != BCQ_OK) return st;
    if (ldy < (size_t)d_out) return BCQ_ERR_SHAPE;
    if (y_dtype != BCQ_F32 && y_dtype != BCQ_BF16) return BCQ_ERR_SHAPE;
    if (!aligned16(bits)) return BCQ_ERR_ALIGN;
    return BCQ_OK;
}

bcq_status fwd_common(int decode, int d_out, int d_in, int q, int g, int n, const void* X, size_t ldx,
                      const uint32_t* bits, const float* alpha, const float* bias, void* Y, size_t ldy,
                      int y_dtype, void* ws, size_t ws_bytes, void* stream) {
    const bcq_status st = check_fwd_args(decode, d_out, d_in, q, g, n, X, ldx, bits, alpha, Y, ldy, y_dtype);
    if (st != BCQ_OK) return st;
    if (decode)
        return run_decode(d_out, d_in, q, g, n, X, ldx, bits, alpha, bias, Y, ldy, y_dtype, ws, ws_bytes, stream);
    return run_expand<MODE_FWD>(d_out, d_in, q, g, n, X, ldx, bits, nullptr, alpha, bias, Y, ldy, y_dtype, ws,
                                ws_bytes, stream);
}

}  // namespace

namespace bcq {
bcq_status expand_timeout_flag(int* flag_out, int reset) {
    int v = 0;
    BCQ_CUDA_TRY(cudaMemcpyFromSymbol(&v, g_timeout_flag, sizeof(int)));
    *flag_out = v;
    if (reset && v != 0) {
        const int zero = 0;
        BCQ_CUDA_TRY(cudaMemcpyToSymbol(g_timeout_flag, &zero, sizeof(int)));
    }
    return BCQ_OK;
}

size_t fwd_workspace_bytes(int d_out, int d_in, int q, int g, int n) {
    return plan_expand(MODE_FWD, d_out, d_in, q, g, n).total;
}
size_t decode_workspace_bytes(int d_out, int d_in, int, int, int n) { return plan_decode(d_out, d_in, n).total; }
size_t bwd_x_workspace_bytes(int d_out, int d_in, int q, int g, int n) {
    return plan_expand(MODE_BWDX, d_out, d_in, q, g, n).total;
}
}  // namespace bcq

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

// ------------------------------------------------------------------------------------------
// decode without a caller-provided workspace
// ------------------------------------------------------------------------------------------

namespace {

// Scratch for the split-K partial sums of bcq_linear_decode_noalloc.  Lives in every CUDA context
// that loads this library.  In host code the symbol is only a handle: the device address comes
// from cudaGetSymbolAddress, once per device.
static __device__ __align__(256) unsigned char g_noalloc_scratch[BCQ_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;

bcq_status noalloc_scratch_address(void** out) {
    static void* address[kMaxDevices] = {};
    static std::mutex lock;
    int dev = -1;
    BCQ_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return BCQ_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> guard(lock);
    if (address[dev] == nullptr) {
        void* p = nullptr;
        BCQ_CUDA_TRY(cudaGetSymbolAddress(&p, g_noalloc_scratch));
        address[dev] = p;
    }
    *out = address[dev];
    return BCQ_OK;
}

}  // namespace

extern "C" bcq_status bcq_linear_decode_noalloc(int d_out, int d_in, int q, int g, int n, const void* X,
                                                size_t ldx, const uint32_t* bits, const float* alpha,
                                                const float* bias, void* Y, size_t ldy, int y_dtype,
                                                void* stream) {
    // Every argument is checked before the scratch symbol is resolved.  (The size check asks the
    // device for its SM count, so it is not free of CUDA calls; without a device the count falls
    // back to a B200's.)  The address found for a device is kept for the life of the process: after
    // cudaDeviceReset it is stale, and the library has to be loaded again.
    bcq_status st = check_fwd_args(1, d_out, d_in, q, g, n, X, ldx, bits, alpha, Y, ldy, y_dtype);
    if (st != BCQ_OK) return st;
    if (bcq::decode_workspace_bytes(d_out, d_in, q, g, n) > (size_t)BCQ_NOALLOC_SCRATCH_BYTES)
        return BCQ_ERR_WORKSPACE;
    void* scratch = nullptr;
    if ((st = noalloc_scratch_address(&scratch)) != BCQ_OK) return st;
    return fwd_common(1, d_out, d_in, q, g, n, X, ldx, bits, alpha, bias, Y, ldy, y_dtype, scratch,
                      (size_t)BCQ_NOALLOC_SCRATCH_BYTES, stream);
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
    return run_expand<MODE_BWDX>(d_out, d_in, q, g, n, dY, lddy, bits, nullptr, alpha, nullptr, dX, lddx, dx_dtype,
                                 ws, ws_bytes, stream);
}

// ------------------------------------------------------------------------------------------
// planes prepared once (B is frozen)
// ------------------------------------------------------------------------------------------

namespace {
bcq_status check_prepared(int op, int d_out, int d_in, int q, int g) {
    bcq_status st = check_shape(d_out, d_in, q, g);
    if (st != BCQ_OK) return st;
    if (op != BCQ_OP_FWD && op != BCQ_OP_BWD_X) return BCQ_ERR_SHAPE;
    if (q > 4) return BCQ_ERR_UNSUPPORTED;
    return BCQ_OK;
}
}  // namespace

extern "C" size_t bcq_prepared_bytes(int op, int d_out, int d_in, int q, int g) {
    if (check_prepared(op, d_out, d_in, q, g) != BCQ_OK) return 0;
    return plan_expand(op == BCQ_OP_FWD ? MODE_FWD : MODE_BWDX, d_out, d_in, q, g, 256).planes_bytes;
}

extern "C" bcq_status bcq_prepare_planes(int op, int d_out, int d_in, int q, int g, const uint32_t* bits,
                                         void* prepared, size_t prepared_bytes, void* stream) {
    bcq_status st = check_prepared(op, d_out, d_in, q, g);
    if (st != BCQ_OK) return st;
    if (!bits || !prepared) return BCQ_ERR_NULL;
    if (!aligned16(bits) || !aligned16(prepared)) return BCQ_ERR_ALIGN;
    const int mode = (op == BCQ_OP_FWD) ? MODE_FWD : MODE_BWDX;
    const ExpandPlan pl = plan_expand(mode, d_out, d_in, q, g, 256);
    if (prepared_bytes < pl.planes_bytes) return BCQ_ERR_WORKSPACE;
    return launch_code_planes(mode, d_out, d_in, q, pl, bits, reinterpret_cast<uint32_t*>(prepared),
                              (cudaStream_t)stream);
}

extern "C" bcq_status bcq_linear_fwd_prepared(int d_out, int d_in, int q, int g, int n, const void* X, size_t ldx,
                                              const void* prepared, const float* alpha, const float* bias,
                                              void* Y, size_t ldy, int y_dtype, void* ws, size_t ws_bytes,
                                              void* stream) {
    bcq_status st = check_prepared(BCQ_OP_FWD, d_out, d_in, q, g);
    if (st != BCQ_OK) return st;
    if (n < 1) return BCQ_ERR_SHAPE;
    if (!prepared || !alpha || !Y) return BCQ_ERR_NULL;
    if ((st = check_act(X, ldx, d_in)) != BCQ_OK) return st;
    if (ldy < (size_t)d_out) return BCQ_ERR_SHAPE;
    if (y_dtype != BCQ_F32 && y_dtype != BCQ_BF16) return BCQ_ERR_SHAPE;
    if (!aligned16(prepared)) return BCQ_ERR_ALIGN;
    return run_expand<MODE_FWD>(d_out, d_in, q, g, n, X, ldx, nullptr, prepared, alpha, bias, Y, ldy, y_dtype, ws,
                                ws_bytes, stream);
}

extern "C" bcq_status bcq_linear_bwd_x_prepared(int d_out, int d_in, int q, int g, int n, const void* dY,
                                                size_t lddy, const void* prepared, const float* alpha, void* dX,
                                                size_t lddx, int dx_dtype, void* ws, size_t ws_bytes, void* stream) {
    bcq_status st = check_prepared(BCQ_OP_BWD_X, d_out, d_in, q, g);
    if (st != BCQ_OK) return st;
    if (n < 1) return BCQ_ERR_SHAPE;
    if (!prepared || !alpha || !dX) return BCQ_ERR_NULL;
    if ((st = check_act(dY, lddy, d_out)) != BCQ_OK) return st;
    if (lddx < (size_t)d_in) return BCQ_ERR_SHAPE;
    if (dx_dtype != BCQ_F32 && dx_dtype != BCQ_BF16) return BCQ_ERR_SHAPE;
    if (!aligned16(prepared)) return BCQ_ERR_ALIGN;
    return run_expand<MODE_BWDX>(d_out, d_in, q, g, n, dY, lddy, nullptr, prepared, alpha, nullptr, dX, lddx,
                                 dx_dtype, ws, ws_bytes, stream);
}
