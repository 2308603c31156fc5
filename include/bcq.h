/*
 * bcq.h -- C ABI of the B200 (sm_100a) library for AlphaTuning's binary-coding-quantized
 * (BCQ) linear layer.
 *
 * The layer stores a weight matrix W (d_out x d_in; the paper's h_out x h_in) as
 *     W ~= sum_{i=1..q} diag(alpha_i) * B_i ,   B_i in {-1,+1}^{d_out x d_in}        (Eq. 1)
 * with q bit-planes and fp32 scales alpha that are shared by groups of g consecutive weights
 * of a row (Section "BCQ Format"; group-wise extension in the Appendix paragraph
 * "group-wise quantization"; g = d_in is the row-wise scheme of Eq. 1).
 *
 * Conventions common to every call
 *   - All data pointers are DEVICE pointers on the current CUDA device unless a parameter is
 *     documented as host memory.  The caller owns every buffer; the library never allocates or
 *     frees device memory.
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*, NULL = default stream);
 *     no call synchronises.
 *   - The return value is the only error channel.  Arguments are validated on the host before
 *     anything is launched; on an error nothing has been enqueued.
 *   - Kernels never trap.  Every wait inside a kernel is time-limited; if one expires the kernel
 *     records it in a device flag (see bcq_device_timeout_flag) and returns.
 *
 * Container format of a quantized matrix, G = ceil(d_in / g):
 *   bits  : uint32 [q][d_out][pitch],  pitch = bcq_pitch_words(d_in) = 4 * ceil(d_in / 128);
 *           bit (k & 31) of word (k >> 5) of row (i, j) is 1  <=>  b_i[j,k] = +1;
 *           padding bits (k >= d_in) are 0.  Rows are 16-byte aligned.
 *   alpha : float  [q][d_out][G];  alpha[i][j][c] scales weights k in [c*g, min((c+1)*g, d_in)).
 *
 * Supported shapes: 1 <= q <= 8, 1 <= d_out, 1 <= d_in, and either g == d_in or
 * (g % 32 == 0 and 32 <= g <= d_in).  Other (q, g) give BCQ_ERR_UNSUPPORTED.
 * bf16 tensors (X, dY) must be 16-byte aligned with a row pitch that is a multiple of 8
 * elements (BCQ_ERR_ALIGN otherwise).
 */
#ifndef BCQ_H_
#define BCQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    BCQ_OK = 0,
    BCQ_ERR_NULL = -1,          /* a required pointer is NULL */
    BCQ_ERR_SHAPE = -2,         /* a size or pitch is out of range */
    BCQ_ERR_ALIGN = -3,         /* a pointer or pitch breaks the alignment rules above */
    BCQ_ERR_UNSUPPORTED = -4,   /* valid BCQ problem, but outside what the kernels cover */
    BCQ_ERR_WORKSPACE = -5,     /* ws_bytes smaller than bcq_workspace_bytes() */
    BCQ_ERR_CUDA = -6,          /* a CUDA call failed; see bcq_last_cuda_error() */
    BCQ_ERR_DEVICE_TIMEOUT = -7 /* a kernel gave up on a wait (bcq_device_timeout_flag) */
} bcq_status;

typedef enum { BCQ_F32 = 0, BCQ_BF16 = 1 } bcq_dtype;

typedef enum {
    BCQ_OP_QUANTIZE = 0,
    BCQ_OP_FWD = 1,
    BCQ_OP_DECODE = 2,
    BCQ_OP_BWD_X = 3,
    BCQ_OP_BWD_ALPHA = 4,
    BCQ_OP_DECODE_PACKED = 5
} bcq_op;

/* ------------------------------------------------------------------ sizes (host only) */

/* Row pitch of `bits` in 32-bit words: 4 * ceil(d_in / 128).  0 if d_in < 1. */
size_t bcq_pitch_words(int d_in);
/* Bytes of the `bits` buffer: q * d_out * pitch * 4. */
size_t bcq_bits_bytes(int d_out, int d_in, int q);
/* G = ceil(d_in / g).  0 if g < 1. */
size_t bcq_num_groups(int d_in, int g);
/* Number of floats in `alpha`: q * d_out * G. */
size_t bcq_alpha_count(int d_out, int d_in, int q, int g);
/* Size of the quantized layer the way Table 1 counts it, in BITS (one bit per plane and
 * weight, 32 bits per scale): q*d_out*d_in + 32*q*d_out*G. */
size_t bcq_payload_bits(int d_out, int d_in, int q, int g);
/* Bytes of scratch (`ws`) that operation `op` needs for this shape and token count n
 * (n is ignored for BCQ_OP_QUANTIZE).  May be 0.  The scratch holds partial sums between the
 * main kernel and its reduction; its contents are undefined afterwards and it must not be
 * shared by calls that may overlap on the GPU. */
size_t bcq_workspace_bytes(int op, int d_out, int d_in, int q, int g, int n);

/* ------------------------------------------------------------------ quantizer */

/* Post-training BCQ of W, one independent problem per (row, group).
 *
 * alt_iters = 0: Greedy approximation (Appendix, Eq. ap:1-ap:3): r = w; for each plane
 *   b_i = sign(r) with sign(0) = +1, alpha_i = mean|r| over the group, r -= alpha_i b_i.
 * alt_iters = T > 0: Alternating method (Appendix, Eq. ap:4 and the paragraph after it):
 *   starting from the greedy result, T rounds of [least-squares alpha for the current signs,
 *   then every weight moves to the nearest of the 2^q levels sum_i +-alpha_i; among
 *   equidistant levels the one with the largest code sum_i 2^i [b_i = +1] wins], followed by one
 *   last least-squares fit.  A group whose planes make B^T B singular keeps its previous
 *   alpha in that round.
 * Sums, residuals and the q x q solve are carried in fp64; every alpha is rounded to fp32 as
 * soon as it is computed and the rounded value is used from then on.
 *
 *   W      in : float [d_out][ldw], ldw >= d_in
 *   bits   out: container format above (padding bits are written as 0)
 *   alpha  out: container format above
 *   sq_err out: float64 [d_out][G], sum over the group of (w - w_hat)^2; may be NULL
 * Group sizes up to 32768 are supported. */
bcq_status bcq_quantize(int d_out, int d_in, int q, int g, const float* W, size_t ldw,
                        int alt_iters, uint32_t* bits, float* alpha, double* sq_err,
                        void* stream);

/* W_hat[j][k] = sum_i alpha[i][j][k/g] * b_i[j,k]  (Eq. 1), fp32, W_hat: float [d_out][ldw]. */
bcq_status bcq_dequantize(int d_out, int d_in, int q, int g, const uint32_t* bits,
                          const float* alpha, float* W_hat, size_t ldw, void* stream);

/* ------------------------------------------------------------------ linear layer */

/* Forward (Eq. 2), computed from the packed planes without materialising W in memory:
 *     Y[t][j] = sum_i sum_c alpha[i][j][c] * sum_{k in group c} X[t][k] * b_i[j,k]  (+ bias[j])
 *   X    in : bf16 [n][ldx]
 *   bias in : float [d_out] or NULL (the frozen bias of the layer)
 *   Y    out: y_dtype [n][ldy], ldy >= d_out
 *   ws      : scratch of bcq_workspace_bytes(BCQ_OP_FWD, ...) bytes, 16-byte aligned (NULL if 0);
 *             it holds an fp16 copy of X and a regrouped copy of the planes and scales, so it
 *             is about 2*n*d_in + bcq_bits_bytes() + 4*bcq_alpha_count() bytes (the same,
 *             with dY and d_out, for bcq_linear_bwd_x)
 * Arithmetic: the scaled weight sum_i alpha_i b_i is formed in fp32 and rounded once to fp16;
 * the bf16 activations are converted exactly to fp16 after a per-token power-of-two scaling
 * that is undone on output; products are accumulated in fp32 in the tensor core.  The same
 * holds for bcq_linear_decode and bcq_linear_bwd_x. */
bcq_status bcq_linear_fwd(int d_out, int d_in, int q, int g, int n, const void* X, size_t ldx,
                          const uint32_t* bits, const float* alpha, const float* bias, void* Y,
                          size_t ldy, int y_dtype, void* ws, size_t ws_bytes, void* stream);

/* Planes prepared once.  AlphaTuning freezes B after quantization and trains only alpha, so the
 * regrouping of the planes that bcq_linear_fwd / bcq_linear_bwd_x do on every call can be done once
 * per layer: bcq_prepare_planes writes, for op = BCQ_OP_FWD or BCQ_OP_BWD_X, the planes in the
 * chunk order of that kernel with every weight's level index already in the form the expansion
 * consumes (q <= 4; q > 4 gives BCQ_ERR_UNSUPPORTED and keeps using the calls above).  The buffer
 * is bcq_prepared_bytes() bytes (0 if unsupported; about bcq_bits_bytes(), more for q = 1 or 2,
 * which are stored like q = 3), 16-byte aligned, caller-owned, and read-only for the *_prepared
 * calls, which take it in place of `bits` and otherwise behave exactly like bcq_linear_fwd /
 * bcq_linear_bwd_x (same results bit for bit, same workspace sizes).  alpha stays an argument of
 * every call: it changes with every optimiser step. */
size_t bcq_prepared_bytes(int op, int d_out, int d_in, int q, int g);
bcq_status bcq_prepare_planes(int op, int d_out, int d_in, int q, int g, const uint32_t* bits,
                              void* prepared, size_t prepared_bytes, void* stream);
bcq_status bcq_linear_fwd_prepared(int d_out, int d_in, int q, int g, int n, const void* X, size_t ldx,
                                   const void* prepared, const float* alpha, const float* bias, void* Y,
                                   size_t ldy, int y_dtype, void* ws, size_t ws_bytes, void* stream);
bcq_status bcq_linear_bwd_x_prepared(int d_out, int d_in, int q, int g, int n, const void* dY, size_t lddy,
                                     const void* prepared, const float* alpha, void* dX, size_t lddx,
                                     int dx_dtype, void* ws, size_t ws_bytes, void* stream);

/* Same computation for the decode regime, 1 <= n <= 16 tokens, where the cost is streaming
 * the packed planes from memory once (Section "Inference Speed").  Workspace op is
 * BCQ_OP_DECODE.  n > 16 gives BCQ_ERR_SHAPE. */
bcq_status bcq_linear_decode(int d_out, int d_in, int q, int g, int n, const void* X, size_t ldx,
                             const uint32_t* bits, const float* alpha, const float* bias,
                             void* Y, size_t ldy, int y_dtype, void* ws, size_t ws_bytes,
                             void* stream);

/* bcq_linear_decode without a caller-provided workspace.  (The paper has no counterpart; this is
 * a convenience of the library.)
 *
 * Some callers of the decode path cannot hand over scratch memory: code that runs where
 * cudaMalloc is off limits -- inside a region that must not touch the allocator (a latency-critical
 * serving loop, a plugin that is only given its input and output tensors), or a process whose
 * memory was carved up in advance.  For them the partial sums of the split over d_in live in a
 * fixed array inside the library, BCQ_NOALLOC_SCRATCH_BYTES (2 MiB) of device memory that
 * every GPU using the library holds from the moment the library is loaded until the process exits.
 * The call allocates nothing and frees nothing.
 *
 *   - Same arguments and results as bcq_linear_decode, minus ws / ws_bytes.
 *   - If bcq_workspace_bytes(BCQ_OP_DECODE, ...) for the shape exceeds
 *     BCQ_NOALLOC_SCRATCH_BYTES the call returns BCQ_ERR_WORKSPACE and launches nothing (on a
 *     B200 that is roughly n * d_out beyond 128K with a split d_in, e.g. 16 tokens of a
 *     12288-row layer; 8 tokens of it fit).  Such problems need bcq_linear_decode.
 *   - The first call on each device looks up the device address of the array
 *     (cudaGetSymbolAddress) with that device current; make that first call outside any stream
 *     capture.  Later calls on the device only launch kernels.  The address is kept for the
 *     life of the process: after cudaDeviceReset on that device it is stale and the library
 *     must be loaded again.
 *   - All calls on a device share the one array.  It keeps whatever the last call left in it;
 *     every call overwrites the part it reads, so nothing has to be cleared.  Two calls that may
 *     overlap on the GPU (different streams, no dependency) race on it: serialise them. */
#define BCQ_NOALLOC_SCRATCH_BYTES (2u << 20)
bcq_status bcq_linear_decode_noalloc(int d_out, int d_in, int q, int g, int n, const void* X,
                                     size_t ldx, const uint32_t* bits, const float* alpha,
                                     const float* bias, void* Y, size_t ldy, int y_dtype,
                                     void* stream);

/* Decode from a packed copy of the frozen weights.
 *
 * At inference both B and alpha are fixed (Section "Inference Speed": a small-batch layer costs
 * what moving its weights costs), so whatever does not depend on the activations can be done
 * once.  bcq_decode_pack rewrites a quantized matrix (q <= 4) into the order and encoding the
 * decode kernel consumes:
 *   - per weight the index of its level among the 2^q sums +-alpha_1 .. +-alpha_q of its
 *     (row, group), q bits per weight as in `bits`;
 *   - per (row, group) the eight fp16 levels sum_i +-alpha_i (for q = 4 those with b_4 = +1; the
 *     others are their negatives), 16 bytes, multiplied by a power of two per row that brings
 *     q * max|alpha| of the row to [2^13, 2^14) -- the values bcq_linear_decode forms on the fly;
 *   - per row that power of two, and one arrival counter per tile of 128 rows.
 * The pack is bcq_decode_pack_bytes() bytes (0 for an unsupported shape; about the size of bits
 * plus alpha), 128-byte aligned, caller-owned.  q > 4 gives BCQ_ERR_UNSUPPORTED: use
 * bcq_linear_decode.  If alpha changes, pack again. */
size_t bcq_decode_pack_bytes(int d_out, int d_in, int q, int g);
bcq_status bcq_decode_pack(int d_out, int d_in, int q, int g, const uint32_t* bits, const float* alpha,
                           void* pack, size_t pack_bytes, void* stream);

/* Y = X W_hat^T (+ bias) for 1 <= n <= 16 tokens from a pack (Eq. 2; same arithmetic as
 * bcq_linear_decode: fp16 levels, bf16 activations scaled per token by a power of two, fp32
 * accumulation).  One kernel: the 128-row x 128-column pieces of the matrix are dealt evenly to
 * one CTA per SM; where two CTAs share a row tile the partial sums go through `ws`
 * (bcq_workspace_bytes(BCQ_OP_DECODE_PACKED, ...) bytes, may be 0) and are added in a fixed order,
 * so the result is the same in every run.
 * The pack is not const: the call uses its arrival counters and leaves them zero again.  Calls
 * that use the same pack must not overlap on the GPU.  After BCQ_ERR_DEVICE_TIMEOUT (see
 * bcq_device_timeout_flag) write the pack again. */
bcq_status bcq_linear_decode_packed(int d_out, int d_in, int q, int g, int n, const void* X, size_t ldx,
                                    void* pack, const float* bias, void* Y, size_t ldy, int y_dtype,
                                    void* ws, size_t ws_bytes, void* stream);

/* Input gradient (Eq. 3):  dX[t][k] = sum_j dY[t][j] * W_hat[j][k],  W_hat as in Eq. 1.
 *   dY in : bf16 [n][lddy];   dX out: dx_dtype [n][lddx], lddx >= d_in. */
bcq_status bcq_linear_bwd_x(int d_out, int d_in, int q, int g, int n, const void* dY, size_t lddy,
                            const uint32_t* bits, const float* alpha, void* dX, size_t lddx,
                            int dx_dtype, void* ws, size_t ws_bytes, void* stream);

/* Scale gradient (Eq. 4, read as the chain rule through Eq. 1 and Eq. 2):
 *     dalpha[i][j][c] (+)= scale * sum_{k in group c} b_i[j,k] * sum_t dY[t][j] * X[t][k]
 * for every plane i whose bit is set in plane_mask; entries of other planes are not touched.
 * scale = 1 gives the gradient; scale = 1/g gives the paper's stabilised update.  The
 * d_out x d_in product dY^T X only ever exists tile by tile on chip.
 *   accumulate: 0 overwrites dalpha, 1 adds to it.
 *   dalpha out: float [q][d_out][G]. */
bcq_status bcq_linear_bwd_alpha(int d_out, int d_in, int q, int g, int n, const void* dY,
                                size_t lddy, const void* X, size_t ldx, const uint32_t* bits,
                                uint32_t plane_mask, float scale, int accumulate, float* dalpha,
                                void* ws, size_t ws_bytes, void* stream);

/* ------------------------------------------------------------------ the AlphaTuning update */

/* Learning rate of 0-based step `step` under the schedule the paper trains with (Section
 * "Experimental Setup": linear decay; the hyper-parameter ablation also uses a warm-up): linear
 * rise from 0 to lr0 over warmup_steps (0 = none), then linear decay to 0 at total_steps.  Host
 * function. */
float bcq_lr_linear_decay(float lr0, long long step, long long warmup_steps, long long total_steps);

/* One AdamW step (Appendix "Experimental Details": AdamW; decoupled weight decay, bias-corrected
 * moments) on the trained scales of a whole model in one launch.  alpha, dalpha, m, v are flat
 * fp32 device arrays with the same indexing: every linear's alpha[q][d_out][G] one after the
 * other.  The trained elements are `count` elements given by nseg segments -- seg_begin[s] is the
 * first flat index of segment s, seg_prefix[s] the number of trained elements before it
 * (seg_prefix[nseg] = count), both int64 DEVICE arrays; a plane of a linear is one segment, so
 * "alpha_1 of every linear" (what the paper trains) is one segment per linear.  nseg = 0 updates
 * the contiguous range [0, count).  For element e with gradient g = grad_scale * seg_scale[s] *
 * dalpha[e] (seg_scale: float device array or NULL = 1; 1/g_L of Eq. 4 goes here when dalpha was
 * computed with scale 1), t = step (1-based):
 *     m <- beta1 m + (1 - beta1) g;   v <- beta2 v + (1 - beta2) g^2
 *     alpha <- alpha (1 - lr weight_decay) - lr (m / (1 - beta1^t)) / (sqrt(v / (1 - beta2^t)) + eps)
 * in fp32.  Elements outside the segments, and their moments, are not touched. */
bcq_status bcq_alpha_adamw(long long count, int nseg, const long long* seg_begin, const long long* seg_prefix,
                           const float* seg_scale, float* alpha, const float* dalpha, float* m, float* v,
                           long long step, float lr, float beta1, float beta2, float eps, float weight_decay,
                           float grad_scale, void* stream);

/* The scale-only checkpoint (the paper's per-task checkpoint holds nothing but the trained
 * alpha): bcq_alpha_pack gathers the segments' elements of the flat array into the compact array
 * packed[count], in segment order; bcq_alpha_unpack scatters them back.  Layout of a checkpoint =
 * that compact fp32 array; the segments are a function of the model's shapes and the trained
 * planes alone. */
bcq_status bcq_alpha_pack(long long count, int nseg, const long long* seg_begin, const long long* seg_prefix,
                          const float* alpha_flat, float* packed, void* stream);
bcq_status bcq_alpha_unpack(long long count, int nseg, const long long* seg_begin, const long long* seg_prefix,
                            const float* packed, float* alpha_flat, void* stream);

/* ------------------------------------------------------------------ status */

const char* bcq_status_string(int status);
/* cudaError_t value of the last CUDA failure seen by this library on the calling thread. */
int bcq_last_cuda_error(void);
/* Number of GPU kernels this library has launched from the calling thread since it was loaded
 * (a monotonic counter; memsets are not counted).  Lets a caller state how many of this
 * library's kernels ran inside a region it timed. */
unsigned long long bcq_kernel_launches(void);
/* Reads (and with reset != 0 clears) the device-side flag that kernels set when a bounded wait
 * expired.  Synchronises the device.  *flag_out = 0 means no kernel has given up. */
bcq_status bcq_device_timeout_flag(int* flag_out /* host */, int reset);
/* Synchronises the device and reports its state as a status: BCQ_ERR_DEVICE_TIMEOUT if a kernel
 * of this library has given up on a wait since the flag was last cleared (the results of the
 * calls since then are not to be trusted; bcq_device_timeout_flag tells which wait and clears the
 * flag), BCQ_ERR_CUDA if the synchronisation itself failed, BCQ_OK otherwise. */
bcq_status bcq_check_device(void);

#ifdef __cplusplus
}
#endif
#endif /* BCQ_H_ */
