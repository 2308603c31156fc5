/*
 * bcq_ref.c -- reference ("oracle") implementation of the binary-coding-quantized
 * (BCQ) linear layer of AlphaTuning, in plain C, fp64 arithmetic, host memory only.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It exists so that the CUDA library can
 * be checked against something written directly from the paper.  It shares no code,
 * header, table or helper with the CUDA path, is never called by it, and is deliberately
 * slow and plain: scalar loops, no blocking, no fusion.  OpenMP is used over the outermost
 * independent index only (rows or tokens); every output element is still produced by one
 * sequential loop, so results do not depend on the thread count.
 *
 * Notation follows the paper: W is h_out x h_in (here d_out x d_in), q planes,
 * group size g along d_in, G = ceil(d_in / g) groups per row, plane index i (0-based here),
 * row j, column k, token t.  b_i[j,k] in {-1,+1}; alpha_i[j,c] is shared by the g weights of
 * group c of row j (Section "BCQ Format", Eq. 1; group-wise extension in Appendix
 * "group-wise quantization").
 *
 * Container format (the same bytes the CUDA library reads and writes, but packed and
 * unpacked here by this file's own code):
 *   bits [q][d_out][pitch] uint32, pitch = 4*ceil(d_in/128); bit (k & 31) of word (k >> 5)
 *         is 1  <=>  b = +1; padding bits (k >= d_in) are 0.
 *   alpha[q][d_out][G] float32.
 *
 * Every function below states the passage of the paper it follows.  All of them are pinned
 * by tests that do not go through this file (closed forms, brute force, finite differences,
 * numpy's dense matmul and least squares, hand-computed examples); none is "parity
 * unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define BCQ_REF_MAX_Q 8

/* ---------------------------------------------------------------- sizes ---------- */

/* Row pitch of the bit container in 32-bit words: rows are padded to 128 bits. */
int64_t bcq_ref_pitch_words(int64_t d_in) { return 4 * ((d_in + 127) / 128); }

/* Number of groups per row, G = ceil(d_in / g) (last group may be short). */
int64_t bcq_ref_num_groups(int64_t d_in, int64_t g) { return (d_in + g - 1) / g; }

/* Table 1 accounting of a quantized layer: one bit per (plane, weight) plus one fp32
 * scale per (plane, row, group).  Exact in eighths of a byte, so it is returned in bits. */
int64_t bcq_ref_payload_bits(int64_t d_out, int64_t d_in, int64_t q, int64_t g) {
    return q * d_out * d_in + 32 * q * d_out * bcq_ref_num_groups(d_in, g);
}

/* ---------------------------------------------------------------- bf16 ----------- */

/* A bf16 value is the upper half of an IEEE binary32; widening is exact. */
static double bf16_to_double(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* ---------------------------------------------------------------- format --------- */

static int get_bit(const uint32_t* bits, int64_t pitch, int64_t d_out, int i, int64_t j,
                   int64_t k) {
    const uint32_t* row = bits + ((int64_t)i * d_out + j) * pitch;
    return (int)((row[k >> 5] >> (k & 31)) & 1u);
}

static void set_bit(uint32_t* bits, int64_t pitch, int64_t d_out, int i, int64_t j, int64_t k) {
    uint32_t* row = bits + ((int64_t)i * d_out + j) * pitch;
    row[k >> 5] |= (1u << (k & 31));
}

/* signs[q][d_out][d_in] int8 in {-1,+1}  ->  bits (padding cleared). */
void bcq_ref_pack(int64_t d_out, int64_t d_in, int q, const int8_t* signs, uint32_t* bits) {
    int64_t pitch = bcq_ref_pitch_words(d_in);
    memset(bits, 0, (size_t)q * d_out * pitch * sizeof(uint32_t));
    for (int i = 0; i < q; ++i)
        for (int64_t j = 0; j < d_out; ++j)
            for (int64_t k = 0; k < d_in; ++k)
                if (signs[((int64_t)i * d_out + j) * d_in + k] > 0)
                    set_bit(bits, pitch, d_out, i, j, k);
}

/* bits -> signs[q][d_out][d_in] int8 in {-1,+1}. */
void bcq_ref_unpack(int64_t d_out, int64_t d_in, int q, const uint32_t* bits, int8_t* signs) {
    int64_t pitch = bcq_ref_pitch_words(d_in);
    for (int i = 0; i < q; ++i)
        for (int64_t j = 0; j < d_out; ++j)
            for (int64_t k = 0; k < d_in; ++k)
                signs[((int64_t)i * d_out + j) * d_in + k] =
                    get_bit(bits, pitch, d_out, i, j, k) ? 1 : -1;
}

/* ---------------------------------------------------------------- quantizer ------ */

/* Least-squares scales for fixed signs (Appendix, Eq. ap:4):
 *   [alpha_1..alpha_q] = (B^T B)^{-1} B^T w,  B = [b_1..b_q] in {-1,+1}^{m x q}.
 * Solved by Gaussian elimination with partial pivoting in fp64.  Returns 0 and leaves
 * alpha untouched if a pivot is below 1e-12*m (two planes equal or opposite: the paper
 * assumes invertibility, this keeps the previous scales for that group).  On success each
 * alpha is rounded to fp32 at once and the rounded value is what everything downstream
 * sees. */
static int ls_alpha(int q, int64_t m, const double* w, const int8_t* b /*[q][m]*/,
                    float* alpha /*[q]*/) {
    double A[BCQ_REF_MAX_Q][BCQ_REF_MAX_Q + 1];
    for (int i = 0; i < q; ++i) {
        for (int l = 0; l < q; ++l) {
            int64_t dot = 0;
            for (int64_t k = 0; k < m; ++k) dot += (int64_t)b[i * m + k] * b[l * m + k];
            A[i][l] = (double)dot;
        }
        double c = 0.0;
        for (int64_t k = 0; k < m; ++k) c += (b[i * m + k] > 0) ? w[k] : -w[k];
        A[i][q] = c;
    }
    const double tiny = 1e-12 * (double)m;
    for (int col = 0; col < q; ++col) {
        int piv = col;
        for (int r = col + 1; r < q; ++r)
            if (fabs(A[r][col]) > fabs(A[piv][col])) piv = r;
        if (fabs(A[piv][col]) < tiny) return 0;
        if (piv != col)
            for (int l = 0; l <= q; ++l) {
                double tmp = A[col][l];
                A[col][l] = A[piv][l];
                A[piv][l] = tmp;
            }
        for (int r = col + 1; r < q; ++r) {
            double f = A[r][col] / A[col][col];
            for (int l = col; l <= q; ++l) {
                double prod = f * A[col][l];
                A[r][l] = A[r][l] - prod;
            }
        }
    }
    double x[BCQ_REF_MAX_Q];
    for (int r = q - 1; r >= 0; --r) {
        double s = A[r][q];
        for (int l = r + 1; l < q; ++l) {
            double prod = A[r][l] * x[l];
            s = s - prod;
        }
        x[r] = s / A[r][r];
    }
    for (int i = 0; i < q; ++i) alpha[i] = (float)x[i];
    return 1;
}

/* Quantize one group w[0..m) to q planes.
 *
 * Greedy approximation (Appendix, Eq. ap:1 applied to the residual, Eq. ap:2 and ap:3):
 *   r <- w;  for i = 1..q:  b_i = sign(r) with sign(0) = +1,  alpha_i = r^T b_i / m
 *   (= mean |r|),  r <- r - alpha_i b_i.
 * Alternating method (Appendix, Eq. ap:4 and the paragraph after it): starting from the
 * greedy result, T times [ least-squares alpha for the current signs; then every element
 * takes the nearest of the 2^q levels sum_i +-alpha_i ], and one last least-squares fit so
 * that the returned alpha is optimal for the returned signs.  No early stop.  Among
 * equidistant levels the largest code wins (code bit i set <=> b_i = +1): codes are scanned
 * from 2^q-1 down with a strict '<'.
 *
 * margin_out (optional): the smallest decision margin met, divided by mean|w|:
 * |r[k]| for a greedy sign, distance gap to the runner-up level for a nearest-level choice.
 * A tiny margin marks a group where fp rounding order may legitimately flip a bit. */
static void quantize_group(int q, int64_t m, const double* w, int alt_iters, int8_t* b /*[q][m]*/,
                           float* alpha /*[q]*/, double* sq_err_out, double* margin_out) {
    double* r = (double*)malloc((size_t)m * sizeof(double));
    double mean_abs_w = 0.0;
    for (int64_t k = 0; k < m; ++k) mean_abs_w += fabs(w[k]);
    mean_abs_w /= (double)m;
    double margin = INFINITY;

    for (int64_t k = 0; k < m; ++k) r[k] = w[k];
    for (int i = 0; i < q; ++i) {
        double sum_abs = 0.0;
        for (int64_t k = 0; k < m; ++k) {
            b[i * m + k] = (r[k] >= 0.0) ? 1 : -1;
            sum_abs += fabs(r[k]);
            if (fabs(r[k]) < margin) margin = fabs(r[k]);
        }
        alpha[i] = (float)(sum_abs / (double)m);
        double a = (double)alpha[i];
        for (int64_t k = 0; k < m; ++k) r[k] = (b[i * m + k] > 0) ? r[k] - a : r[k] + a;
    }

    if (alt_iters > 0) {
        const int ncodes = 1 << q;
        double level[1 << BCQ_REF_MAX_Q];
        for (int it = 0; it < alt_iters; ++it) {
            ls_alpha(q, m, w, b, alpha);
            for (int s = 0; s < ncodes; ++s) {
                double L = 0.0;
                for (int i = 0; i < q; ++i)
                    L = ((s >> i) & 1) ? L + (double)alpha[i] : L - (double)alpha[i];
                level[s] = L;
            }
            for (int64_t k = 0; k < m; ++k) {
                int best = ncodes - 1;
                double dbest = fabs(w[k] - level[best]);
                double dsecond = INFINITY;
                for (int s = ncodes - 2; s >= 0; --s) {
                    double d = fabs(w[k] - level[s]);
                    if (d < dbest) {
                        dsecond = dbest;
                        dbest = d;
                        best = s;
                    } else if (d < dsecond) {
                        dsecond = d;
                    }
                }
                if (ncodes > 1 && dsecond - dbest < margin) margin = dsecond - dbest;
                for (int i = 0; i < q; ++i) b[i * m + k] = ((best >> i) & 1) ? 1 : -1;
            }
        }
        ls_alpha(q, m, w, b, alpha);
    }

    if (sq_err_out) {
        double e = 0.0;
        for (int64_t k = 0; k < m; ++k) {
            double wh = 0.0;
            for (int i = 0; i < q; ++i)
                wh = (b[i * m + k] > 0) ? wh + (double)alpha[i] : wh - (double)alpha[i];
            e += (w[k] - wh) * (w[k] - wh);
        }
        *sq_err_out = e;
    }
    if (margin_out) *margin_out = (mean_abs_w > 0.0) ? margin / mean_abs_w : 0.0;
    free(r);
}

/* Quantize a matrix row by row, group by group (Appendix "group-wise quantization": each
 * row is cut into consecutive vectors of g weights, each with its own q scales; g = d_in is
 * the row-wise scheme of Eq. 1).  A short last group uses its own length as n.
 *   W [d_out][ldw] fp32;  bits, alpha: container format above;
 *   sq_err, margin: [d_out][G] or NULL.
 * Returns 0, or -1 on invalid arguments. */
int bcq_ref_quantize(int64_t d_out, int64_t d_in, int q, int64_t g, const float* W, int64_t ldw,
                     int alt_iters, uint32_t* bits, float* alpha, double* sq_err,
                     double* margin) {
    if (q < 1 || q > BCQ_REF_MAX_Q || g < 1 || g > d_in || d_out < 1 || d_in < 1 || alt_iters < 0)
        return -1;
    const int64_t pitch = bcq_ref_pitch_words(d_in);
    const int64_t G = bcq_ref_num_groups(d_in, g);
    memset(bits, 0, (size_t)q * d_out * pitch * sizeof(uint32_t));
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t j = 0; j < d_out; ++j) {
        double* w = (double*)malloc((size_t)g * sizeof(double));
        int8_t* b = (int8_t*)malloc((size_t)q * g);
        for (int64_t c = 0; c < G; ++c) {
            const int64_t k0 = c * g;
            const int64_t m = (k0 + g <= d_in) ? g : d_in - k0;
            float a[BCQ_REF_MAX_Q];
            double e, mg;
            for (int64_t k = 0; k < m; ++k) w[k] = (double)W[j * ldw + k0 + k];
            quantize_group(q, m, w, alt_iters, b, a, &e, &mg);
            for (int i = 0; i < q; ++i) {
                alpha[((int64_t)i * d_out + j) * G + c] = a[i];
                for (int64_t k = 0; k < m; ++k)
                    if (b[i * m + k] > 0) set_bit(bits, pitch, d_out, i, j, k0 + k);
            }
            if (sq_err) sq_err[j * G + c] = e;
            if (margin) margin[j * G + c] = mg;
        }
        free(w);
        free(b);
    }
    return 0;
}

/* W_hat[j,k] = sum_i alpha_i[j, k/g] * b_i[j,k]  (Eq. 1 with the group-wise scales). */
void bcq_ref_dequantize(int64_t d_out, int64_t d_in, int q, int64_t g, const uint32_t* bits,
                        const float* alpha, double* W_hat, int64_t ldw) {
    const int64_t pitch = bcq_ref_pitch_words(d_in);
    const int64_t G = bcq_ref_num_groups(d_in, g);
#pragma omp parallel for
    for (int64_t j = 0; j < d_out; ++j)
        for (int64_t k = 0; k < d_in; ++k) {
            double s = 0.0;
            for (int i = 0; i < q; ++i) {
                double a = (double)alpha[((int64_t)i * d_out + j) * G + k / g];
                s += get_bit(bits, pitch, d_out, i, j, k) ? a : -a;
            }
            W_hat[j * ldw + k] = s;
        }
}

/* ---------------------------------------------------------------- forward -------- */

/* One output of Eq. 2, Y = sum_i (X B_i^T) diag(alpha_i), with the scale taken per group:
 *   Y[t,j] = sum_i sum_c alpha_i[j,c] * ( sum_{k in c} X[t,k] b_i[j,k] )  (+ bias[j]).
 * X holds bf16 bit patterns, widened exactly. */
static double fwd_one(int64_t d_out, int64_t d_in, int q, int64_t g, int64_t pitch, int64_t G,
                      const uint16_t* xrow, const uint32_t* bits, const float* alpha,
                      const float* bias, int64_t j) {
    double y = 0.0;
    for (int i = 0; i < q; ++i)
        for (int64_t c = 0; c < G; ++c) {
            const int64_t k1 = ((c + 1) * g < d_in) ? (c + 1) * g : d_in;
            double s = 0.0;
            for (int64_t k = c * g; k < k1; ++k) {
                double x = bf16_to_double(xrow[k]);
                s += get_bit(bits, pitch, d_out, i, j, k) ? x : -x;
            }
            y += (double)alpha[((int64_t)i * d_out + j) * G + c] * s;
        }
    if (bias) y += (double)bias[j];
    return y;
}

/* Full forward, Y [n][ldy] fp64 (Eq. 2). */
void bcq_ref_fwd(int64_t d_out, int64_t d_in, int q, int64_t g, int64_t n, const uint16_t* X,
                 int64_t ldx, const uint32_t* bits, const float* alpha, const float* bias,
                 double* Y, int64_t ldy) {
    const int64_t pitch = bcq_ref_pitch_words(d_in);
    const int64_t G = bcq_ref_num_groups(d_in, g);
#pragma omp parallel for
    for (int64_t t = 0; t < n; ++t)
        for (int64_t j = 0; j < d_out; ++j)
            Y[t * ldy + j] = fwd_one(d_out, d_in, q, g, pitch, G, X + t * ldx, bits, alpha, bias, j);
}

/* Forward at chosen positions only: out[s] = Y[t_idx[s], j_idx[s]]. */
void bcq_ref_fwd_at(int64_t d_out, int64_t d_in, int q, int64_t g, const uint16_t* X, int64_t ldx,
                    const uint32_t* bits, const float* alpha, const float* bias, int64_t ns,
                    const int64_t* t_idx, const int64_t* j_idx, double* out) {
    const int64_t pitch = bcq_ref_pitch_words(d_in);
    const int64_t G = bcq_ref_num_groups(d_in, g);
#pragma omp parallel for
    for (int64_t s = 0; s < ns; ++s)
        out[s] = fwd_one(d_out, d_in, q, g, pitch, G, X + t_idx[s] * ldx, bits, alpha, bias,
                         j_idx[s]);
}

/* ---------------------------------------------------------------- backward ------- */

static double what_one(int64_t d_out, int q, int64_t g, int64_t pitch, int64_t G,
                       const uint32_t* bits, const float* alpha, int64_t j, int64_t k) {
    double s = 0.0;
    for (int i = 0; i < q; ++i) {
        double a = (double)alpha[((int64_t)i * d_out + j) * G + k / g];
        s += get_bit(bits, pitch, d_out, i, j, k) ? a : -a;
    }
    return s;
}

/* Eq. 3:  dX = dY (sum_i diag(alpha_i) B_i),  dX[t,k] = sum_j dY[t,j] W_hat[j,k].
 * dY holds bf16 bit patterns; dX [n][lddx] fp64. */
void bcq_ref_bwd_x(int64_t d_out, int64_t d_in, int q, int64_t g, int64_t n, const uint16_t* dY,
                   int64_t lddy, const uint32_t* bits, const float* alpha, double* dX,
                   int64_t lddx) {
    double* What = (double*)malloc((size_t)d_out * d_in * sizeof(double));
    bcq_ref_dequantize(d_out, d_in, q, g, bits, alpha, What, d_in);
#pragma omp parallel for
    for (int64_t t = 0; t < n; ++t) {
        double* out = dX + t * lddx;
        for (int64_t k = 0; k < d_in; ++k) out[k] = 0.0;
        for (int64_t j = 0; j < d_out; ++j) {
            const double dy = bf16_to_double(dY[t * lddy + j]);
            const double* wrow = What + j * d_in;
            for (int64_t k = 0; k < d_in; ++k) out[k] += dy * wrow[k];
        }
    }
    free(What);
}

/* Eq. 3 at chosen positions: out[s] = dX[t_idx[s], k_idx[s]]. */
void bcq_ref_bwd_x_at(int64_t d_out, int64_t d_in, int q, int64_t g, const uint16_t* dY,
                      int64_t lddy, const uint32_t* bits, const float* alpha, int64_t ns,
                      const int64_t* t_idx, const int64_t* k_idx, double* out) {
    const int64_t pitch = bcq_ref_pitch_words(d_in);
    const int64_t G = bcq_ref_num_groups(d_in, g);
#pragma omp parallel for
    for (int64_t s = 0; s < ns; ++s) {
        double acc = 0.0;
        for (int64_t j = 0; j < d_out; ++j)
            acc += bf16_to_double(dY[t_idx[s] * lddy + j]) *
                   what_one(d_out, q, g, pitch, G, bits, alpha, j, k_idx[s]);
        out[s] = acc;
    }
}

/* One entry of Eq. 4, read as the chain rule through Eq. 1 and 2 (the printed product
 * (dY)^T X B_i^T 1 is not well-formed; what is meant is the diagonal of (dY^T X) B_i^T):
 *   dalpha_i[j,c] = scale * sum_{k in c} b_i[j,k] * ( sum_t dY[t,j] X[t,k] ).
 * scale = 1 is the gradient; scale = 1/g_L is the paper's stabilised update. */
static double dalpha_one(int64_t d_out, int64_t d_in, int64_t g, int64_t pitch, int64_t n,
                         const uint16_t* dY, int64_t lddy, const uint16_t* X, int64_t ldx,
                         const uint32_t* bits, double scale, int i, int64_t j, int64_t c) {
    const int64_t k1 = ((c + 1) * g < d_in) ? (c + 1) * g : d_in;
    double acc = 0.0;
    for (int64_t k = c * g; k < k1; ++k) {
        double p = 0.0;
        for (int64_t t = 0; t < n; ++t)
            p += bf16_to_double(dY[t * lddy + j]) * bf16_to_double(X[t * ldx + k]);
        acc += get_bit(bits, pitch, d_out, i, j, k) ? p : -p;
    }
    return scale * acc;
}

/* Eq. 4 for every plane in plane_mask; dalpha [q][d_out][G] fp64, entries of planes not in
 * the mask are left untouched. */
void bcq_ref_bwd_alpha(int64_t d_out, int64_t d_in, int q, int64_t g, int64_t n,
                       const uint16_t* dY, int64_t lddy, const uint16_t* X, int64_t ldx,
                       const uint32_t* bits, uint32_t plane_mask, double scale, double* dalpha) {
    const int64_t pitch = bcq_ref_pitch_words(d_in);
    const int64_t G = bcq_ref_num_groups(d_in, g);
#pragma omp parallel for
    for (int64_t j = 0; j < d_out; ++j) {
        /* p[k] = (dY^T X)[j,k] */
        double* p = (double*)calloc((size_t)d_in, sizeof(double));
        for (int64_t t = 0; t < n; ++t) {
            const double dy = bf16_to_double(dY[t * lddy + j]);
            for (int64_t k = 0; k < d_in; ++k) p[k] += dy * bf16_to_double(X[t * ldx + k]);
        }
        for (int i = 0; i < q; ++i) {
            if (!((plane_mask >> i) & 1u)) continue;
            for (int64_t c = 0; c < G; ++c) {
                const int64_t k1 = ((c + 1) * g < d_in) ? (c + 1) * g : d_in;
                double acc = 0.0;
                for (int64_t k = c * g; k < k1; ++k)
                    acc += get_bit(bits, pitch, d_out, i, j, k) ? p[k] : -p[k];
                dalpha[((int64_t)i * d_out + j) * G + c] = scale * acc;
            }
        }
        free(p);
    }
}

/* Eq. 4 at chosen entries: out[s] = dalpha_{i_idx[s]}[j_idx[s], c_idx[s]]. */
void bcq_ref_bwd_alpha_at(int64_t d_out, int64_t d_in, int q, int64_t g, int64_t n,
                          const uint16_t* dY, int64_t lddy, const uint16_t* X, int64_t ldx,
                          const uint32_t* bits, double scale, int64_t ns, const int64_t* i_idx,
                          const int64_t* j_idx, const int64_t* c_idx, double* out) {
    const int64_t pitch = bcq_ref_pitch_words(d_in);
    (void)q;
#pragma omp parallel for
    for (int64_t s = 0; s < ns; ++s)
        out[s] = dalpha_one(d_out, d_in, g, pitch, n, dY, lddy, X, ldx, bits, scale,
                            (int)i_idx[s], j_idx[s], c_idx[s]);
}

/* Number of OpenMP threads the loops above will use (1 when built without OpenMP). */
/* ---------------------------------------------------------------- optimiser -------- */

/* Learning rate of step `step` (0-based) under the linear-decay schedule of Section
 * "Experimental Setup" ("a linear decay learning rate schedule"; Appendix: "linear-decaying
 * learning rate scheduler"), with the optional warm-up of the hyper-parameter ablation table:
 * the rate rises linearly from 0 to lr0 over `warmup` steps, then falls linearly to 0 at step
 * `total`. */
double bcq_ref_lr_linear(double lr0, int64_t step, int64_t warmup, int64_t total) {
    if (step < warmup) return lr0 * (double)step / (double)warmup;
    if (step >= total) return 0.0;
    return lr0 * (double)(total - step) / (double)(total - warmup);
}

/* One AdamW step on the scales (Appendix "Experimental Details": "AdamW optimizer"), i.e. Adam
 * with decoupled weight decay (Loshchilov & Hutter), t = step (1-based):
 *     g      = grad_scale * grad            grad_scale = 1/g_L is the paper's Eq. 4 factor
 *     alpha <- alpha * (1 - lr * wd)
 *     m     <- beta1 m + (1 - beta1) g ;    v <- beta2 v + (1 - beta2) g^2
 *     alpha <- alpha - lr * (m / (1 - beta1^t)) / (sqrt(v / (1 - beta2^t)) + eps)
 * alpha, m, v are stored in fp32 (as the trainable state is); the arithmetic of a step is fp64
 * and each stored value is rounded once. */
void bcq_ref_adamw(int64_t count, float* alpha, const float* grad, float* m, float* v, int64_t step,
                   double lr, double beta1, double beta2, double eps, double wd, double grad_scale) {
    const double bc1 = 1.0 - pow(beta1, (double)step);
    const double bc2 = 1.0 - pow(beta2, (double)step);
    for (int64_t e = 0; e < count; ++e) {
        const double g = grad_scale * (double)grad[e];
        double a = (double)alpha[e] * (1.0 - lr * wd);
        const double mm = beta1 * (double)m[e] + (1.0 - beta1) * g;
        const double vv = beta2 * (double)v[e] + (1.0 - beta2) * g * g;
        a -= lr * (mm / bc1) / (sqrt(vv / bc2) + eps);
        alpha[e] = (float)a;
        m[e] = (float)mm;
        v[e] = (float)vv;
    }
}

#ifdef _OPENMP
#include <omp.h>
int bcq_ref_num_threads(void) { return omp_get_max_threads(); }
#else
int bcq_ref_num_threads(void) { return 1; }
#endif
