/*
 * libaq -- low-bit block-quantised linear layers for NVIDIA B200 (sm_100a).
 *
 * C ABI.  Every pointer argument says whether it is HOST or DEVICE memory.
 * Citations name passages of "ActQuant: Sub-4-bit Action-Guided Quantization
 * for Vision-Language-Action Models" (the paper).
 *
 * The format (Section 3, "Weight quantization", Eq. 1): a weight matrix W of
 * N rows (output features) by K columns (input features) is cut, along each
 * row, into blocks of 32 consecutive elements; a block has a scale and a zero
 * point and all its elements are coded with the same number of bits n; one
 * matrix has one n (Section 1 / Section 4.1: one bit-width per matrix).  Eq. 1's
 * decode s_b (q_i - z_b) is stored as  scale * q_i + min  (min = -s_b z_b),
 * scale and min in IEEE binary16, q_i in {0 .. 2^n - 1}, n in {2, 3, 4}.
 *
 * Canonical bytes (the container of Appendix D: packed codes, per-block
 * scales and zero points; byte order is this library's choice): blocks in
 * row-major order over (row, block); a block record is
 *     [scale: binary16 LE][min: binary16 LE][codes: 4n bytes]
 * where the codes form one little-endian integer of 32 n bits with code i at
 * bits [n i, n i + n).  N*K*(n+1)/8 bytes in total.
 *
 * Errors: every call returns an aq_status_t; nothing throws, aborts or traps
 * the device.  Arguments are checked on the host before any launch.
 * All launches are asynchronous on the given stream unless stated otherwise.
 * The library runs only on compute capability 10.x devices (AQ_ERR_ARCH).
 */
#ifndef AQ_H_
#define AQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct aq_handle_s* aq_handle_t;   /* opaque; owns its device memory */
typedef void* aq_stream_t;                 /* a cudaStream_t (0 = default stream) */

typedef enum {
    AQ_OK = 0,
    AQ_ERR_INVALID_ARG = 1,   /* null / misaligned pointer, bad size, bad enum */
    AQ_ERR_UNSUPPORTED = 2,   /* bits not in {2,3,4}, block != 32, dtype not allowed here */
    AQ_ERR_ALLOC = 3,         /* device or host allocation failed */
    AQ_ERR_CUDA = 4,          /* a CUDA runtime call failed (see aq_last_cuda_error) */
    AQ_ERR_TIMEOUT = 5,       /* a bounded device-side wait ran out */
    AQ_ERR_ARCH = 6,          /* current device is not sm_100 */
    AQ_ERR_RANGE = 7          /* non-finite weight, or a block's scale/min overflows binary16 */
} aq_status_t;

typedef enum { AQ_F16 = 0, AQ_BF16 = 1, AQ_F32 = 2 } aq_dtype_t;

/* Largest token count M of one aq_linear / aq_stack_forward call. */
#define AQ_MAX_M 4096
/* Token counts up to this run the weight-streaming (decode) kernel. */
#define AQ_DECODE_MAX_M 8

/*
 * aq_pack -- quantise and pack (Eq. 1, the argmin over a uniform codebook:
 * round-to-nearest; the "RTN block quantization" row of the ablation table).
 *   bits   : n in {2,3,4};  block : must be 32
 *   W_dev  : DEVICE, float32, row-major [N][K], 16-byte aligned; read during
 *            the call's stream work, not retained
 *   N, K   : N >= 1; K >= 32 and K % 32 == 0
 *   out    : HOST pointer receiving the new handle
 * Per block, in binary32 with one rounding per operation:
 *   scale = f16((max - min) / (2^n - 1)), min = f16(min),
 *   q = clamp(rint((w - min) / scale), 0, 2^n - 1)   (rint: ties to even),
 *   q = 0 everywhere when scale rounds to 0.
 * A non-finite weight or an overflowing scale/min is recorded in the handle
 * and reported as AQ_ERR_RANGE by aq_info / aq_export.
 */
aq_status_t aq_pack(int bits, int block, const float* W_dev, int64_t N, int64_t K,
                    aq_stream_t stream, aq_handle_t* out);

/*
 * aq_pack_opt -- quantise and pack with optimised block parameters (Section 3.3, "Intra-Tensor Scale
 * Optimization": Eq. 10, the weighted block objective Phi_b with omega = F sqrt(sigma_b^2 + w^2); Eq. 11,
 * the alternation of nearest codes and the closed-form parameters).
 *   arguments as aq_pack, plus
 *   F_dev  : DEVICE, float32, row-major [N][K], 16-byte aligned: the diagonal Fisher scores of Eq. 9, or
 *            NULL for F = 1 (the magnitude-weighted variant of the ablation table)
 *   rounds : alternations of Eq. 11 (0 .. 64; 0 gives aq_pack's result)
 * The paper's decode in Eq. 10 is s q; this container decodes scale * q + min, so the closed-form step solves the
 * weighted least squares for the pair (scale, min).  Start: the round-to-nearest parameters.  A block keeps its
 * round-to-nearest form when the optimised parameters, rounded to binary16, do not lower Phi_b, so no block is
 * worse than aq_pack's under Eq. 10.  Each arithmetic step is one correctly rounded operation in a fixed order:
 * the result is reproducible bit for bit.  Errors as aq_pack.
 */
aq_status_t aq_pack_opt(int bits, int block, const float* W_dev, const float* F_dev, int rounds, int64_t N, int64_t K,
                        aq_stream_t stream, aq_handle_t* out);

/* ---- inter-tensor stage (Section 4.1): HSIC sensitivities and bit allocation ------------------------------
 * The three device calls below share one static device scratch area: issue them on one stream (or otherwise
 * serialised).  None of them allocates memory. */
#define AQ_HSIC_MAX_K 16384

/*
 * aq_rbf_gram -- RBF kernel matrix of K calibration samples (Section 3, "HSIC": [K_A]_ij = k(a_i, a_j) with the
 * Gaussian kernel k(a, a') = exp(-|a - a'|^2 / (2 sigma^2)); the paper prints no bandwidth, sigma is the caller's).
 *   A_dev  : DEVICE, [K][d] row-major, AQ_F16 or AQ_BF16 (activations are kept at half precision), 16-byte
 *            aligned; d % 8 == 0 (pad with zero columns: they do not change a distance)
 *   K      : 2 .. AQ_HSIC_MAX_K samples;  d >= 8 features;  sigma > 0 and finite
 *   G_dev  : DEVICE, float32 [K][ldg], ldg >= K; receives the full symmetric matrix, diagonal exactly 1
 * Squared distances are formed as n_i + n_j - 2 <a_i, a_j> (clamped at 0) from exact products accumulated in
 * binary32 on the tensor cores.  Asynchronous on `stream`; a wait that runs out is reported by aq_check.
 */
aq_status_t aq_rbf_gram(const void* A_dev, aq_dtype_t dtype, int64_t K, int64_t d, float sigma, float* G_dev,
                        int64_t ldg, aq_stream_t stream);

/*
 * aq_hsic -- the empirical criterion of Eq. 2, (K-1)^-2 tr(K_A C K_B C) with C = I - 11^T/K.
 *   KA_dev, KB_dev : DEVICE, float32 [K][ld] symmetric kernel matrices (e.g. from aq_rbf_gram), ld >= K
 *   out_dev        : DEVICE, one binary64 value
 * Evaluated in binary64 in a fixed order (reproducible).  Asynchronous on `stream`.
 */
aq_status_t aq_hsic(const float* KA_dev, const float* KB_dev, int64_t K, int64_t ld, double* out_dev,
                    aq_stream_t stream);

/*
 * aq_sensitivity -- Eq. 5: S = -alpha HSIC(X, Z) + beta HSIC(Z, Y) for one weight matrix, from the kernel
 * matrices of the backbone inputs X, the matrix's outputs Z and the action labels Y.
 *   out3_dev : DEVICE, three binary64 values: S, HSIC(X, Z), HSIC(Z, Y)
 *   alpha, beta >= 0.  Other arguments as aq_hsic.
 */
aq_status_t aq_sensitivity(const float* KX_dev, const float* KZ_dev, const float* KY_dev, int64_t K, int64_t ld,
                           double alpha, double beta, double* out3_dev, aq_stream_t stream);

/*
 * aq_allocate_bits -- the layer-balanced allocation of Eq. 6 by the greedy solver of Section 4.1 (HOST only).
 * Minimises sum_l E_l^2, E_l = sum_{j in layer l} S_j 2^(-2 b_j), subject to the parameter-weighted mean of b_j
 * being <= budget.
 *   S, numel, layer_of : HOST arrays of n entries: sensitivity (Eq. 5), number of weights, layer index (>= 0)
 *   types              : HOST, n_types strictly ascending bit-widths (1..16), e.g. {2, 3, 4}
 *   bits_out           : HOST, n entries;  objective_out : HOST, may be NULL
 * Every matrix starts at types[0]; each step applies, among the upgrades to the next type that keep the budget,
 * the one with the largest (E_l^2 - E~_l^2) / ((b_new - b_old) numel); it stops when none is left or the best
 * one does not lower the objective (ties: lowest index).  AQ_ERR_INVALID_ARG for malformed input,
 * AQ_ERR_RANGE when the budget is below types[0].
 */
aq_status_t aq_allocate_bits(const double* S, const int64_t* numel, const int32_t* layer_of, int64_t n,
                             const int32_t* types, int n_types, double budget, int32_t* bits_out,
                             double* objective_out);

/*
 * Attention of one decoded token over a key/value cache, with rotary position embedding: the step between the
 * projections W_Q, W_K, W_V and W_O of a decoder block (Section 2, "Vision-Language-Action models", names the
 * projections of every transformer block; the operation between them is the textbook scaled-dot-product attention
 * and rotary embedding of the LLaMA-style backbone, which the paper does not restate).  Head dimension 128 only.
 *
 * Caches are DEVICE arrays [n_kv_heads][L_max][128] of `dtype` (AQ_F16 / AQ_BF16), head-major, owned by the caller.
 *
 * aq_rope       rotates, in place, one token's heads x_dev [n_heads][head_dim] (AQ_F16 / AQ_BF16 / AQ_F32; head_dim even):
 *               pair (i, i + head_dim/2) of every head by the angle pos * theta^(-2 i / head_dim).
 * aq_kv_append  cache[h][pos][:] = row[h][:] for keys and values (k_dev, v_dev [n_kv_heads][128]; pos < L_max).
 * aq_attn_decode  out[m][h] = softmax_p(scale * q[m][h] . K[h / G][p]) V[h / G][p] for M new tokens whose keys and
 *               values are the last M of the L cached positions: token m sees positions p <= L - M + m (itself and
 *               everything before it).  G = n_heads / n_kv_heads query heads share a key/value head; G * M <= 16
 *               (with 32 heads of their own: 1 <= M <= 16; AQ_DECODE_MAX_M tokens need G <= 2).  q_dev
 *               [M][n_heads][128] of `dtype`; out_dev [M][n_heads][128] of out_dtype (any of the three); scale <= 0
 *               means 1/sqrt(128).
 *               scratch_dev: DEVICE, 256-byte aligned, aq_attn_scratch_bytes(n_kv_heads) bytes, contents irrelevant
 *               before and after.  Calls on one device must not overlap in time (they share a small static ticket
 *               array besides the scratch): keep them on one stream, or order the streams.
 * Scores and sums are binary32; the softmax weights enter the second product rounded to `dtype`, so against the exact
 * result an output is off by at most about 2^-10 (AQ_F16; 2^-7 for AQ_BF16) of sum_p softmax_p |V[p]|.
 * Errors: AQ_ERR_INVALID_ARG (null / misaligned pointer, M < 1, L not in M..L_max, n_heads not a multiple of
 * n_kv_heads), AQ_ERR_UNSUPPORTED (head_dim != 128, G * M > 16, n_kv_heads > 64, dtype), AQ_ERR_ARCH, AQ_ERR_CUDA.
 */
size_t aq_attn_scratch_bytes(int n_kv_heads);
aq_status_t aq_rope(void* x_dev, int n_heads, int head_dim, int64_t pos, float theta, aq_dtype_t dtype, aq_stream_t stream);
aq_status_t aq_kv_append(void* k_cache_dev, void* v_cache_dev, const void* k_dev, const void* v_dev, int n_kv_heads,
                         int head_dim, int64_t pos, int64_t L_max, aq_dtype_t dtype, aq_stream_t stream);
aq_status_t aq_attn_decode(const void* q_dev, const void* k_cache_dev, const void* v_cache_dev, void* out_dev, int M, int n_heads,
                           int n_kv_heads, int head_dim, int64_t L, int64_t L_max, float scale, aq_dtype_t dtype,
                           aq_dtype_t out_dtype, void* scratch_dev, size_t scratch_bytes, aq_stream_t stream);

/*
 * aq_pack_sb / aq_import_sb / aq_export_sb -- the two-level (super-block) form of the format (Section 3, "Weight
 * quantization": every S consecutive blocks form a super-block with its own scale and zero point that compress the
 * per-block parameters).  The paper prints neither S nor the width of the compressed parameters; this library takes
 * S = 8 blocks (256 weights) and, per super-block, three binary16 values D, Dm, Mn and per block two 6-bit codes
 * u, v in {0 .. 63}:      scale_b = f16(D u_b),      min_b = f16(fma(Dm, v_b, Mn)),
 * Eq. 1's rule one level up (zero point 0 for the scales, Mn for the minima), the decoded block parameters rounded
 * to binary16; codes q as in aq_pack with those parameters.  K % 256 == 0; sblock must be 8.
 * Canonical bytes: super-blocks in row-major order over (row, super-block); a record is
 *     [D][Dm][Mn] (binary16 LE) [12 bytes: a little-endian integer of 96 bits, block b's u at bits [12 b, 12 b + 6),
 *     its v at [12 b + 6, 12 b + 12)] [codes of the 8 blocks, each as in the plain record]
 * i.e. n + 0.5625 bits per weight instead of n + 1 (aq_info's packed_bytes).  Quantiser, in binary32 with one
 * rounding per operation: s_b = (max - min) / (2^n - 1) and mn_b = min per block; D = f16(max_b s_b / 63),
 * u_b = clamp(rint(s_b / D)); Mn = f16(min_b mn_b), Dm = f16(max(0, max_b mn_b - Mn) / 63), v_b = clamp(rint((mn_b -
 * Mn) / Dm)) (codes 0 where a divisor is 0).  On the device the handle keeps the decoded block parameters in the
 * ordinary layout, so aq_dequant, aq_linear and aq_stack_forward take it like any other handle (its device memory is
 * that of a plain handle plus 32 bytes per super-block; the saving is the container's).  aq_export on such a handle
 * gives the plain record form with the decoded parameters.  Errors as aq_pack / aq_import / aq_export.
 */
aq_status_t aq_pack_sb(int bits, int block, int sblock, const float* W_dev, int64_t N, int64_t K, aq_stream_t stream,
                       aq_handle_t* out);
aq_status_t aq_import_sb(int bits, int block, int sblock, int64_t N, int64_t K, const void* canon_host, size_t nbytes,
                         aq_stream_t stream, aq_handle_t* out);
aq_status_t aq_export_sb(aq_handle_t h, void* canon_host, size_t cap, size_t* nbytes);

/*
 * aq_import -- build a handle from canonical bytes (Appendix D container).
 *   canon_host : HOST, nbytes == N*K*(bits+1)/8 bytes in the layout above
 * Synchronises `stream` before returning (the host buffer may be reused).
 */
aq_status_t aq_import(int bits, int block, int64_t N, int64_t K, const void* canon_host,
                      size_t nbytes, aq_stream_t stream, aq_handle_t* out);

/*
 * aq_export -- canonical bytes of a handle (Appendix D container).
 *   canon_host : HOST buffer of capacity cap (may be NULL to query the size)
 *   nbytes     : HOST, receives N*K*(bits+1)/8
 * Synchronises the handle's last stream.  AQ_ERR_RANGE if packing saw a
 * non-finite weight or an overflow (the bytes are still written).
 */
aq_status_t aq_export(aq_handle_t h, void* canon_host, size_t cap, size_t* nbytes);

/*
 * aq_info -- shape and sizes; any out pointer may be NULL.
 *   packed_bytes : N*K*(bits+1)/8, the closed form
 *   device_bytes : bytes the handle holds on the device for the weights
 *                  (the closed form plus padding of N to 16 and K to 256)
 * Synchronises the handle's last stream; AQ_ERR_RANGE as for aq_export.
 */
aq_status_t aq_info(aq_handle_t h, int* bits, int* block, int64_t* N, int64_t* K,
                    size_t* packed_bytes, size_t* device_bytes);

/*
 * aq_dequant -- the whole dequantised matrix (Eq. 1).
 *   out_dev : DEVICE, row-major [N][K] of out_dtype, 16-byte aligned
 * Each element is fmaf(f32(scale), f32(q), f32(min)) rounded once to
 * out_dtype (nearest even); bit-exact with that definition.
 */
aq_status_t aq_dequant(aq_handle_t h, void* out_dev, aq_dtype_t out_dtype, aq_stream_t stream);

/*
 * aq_linear -- y = x W_hat^T on the packed weights (Section 4.3 / Appendix D:
 * each matmul of the converted model runs as one low-bit kernel that
 * dequantises on the fly; activations stay in half precision).
 *   x_dev : DEVICE, row-major [M][K], AQ_F16 or AQ_BF16, 16-byte aligned
 *   y_dev : DEVICE, row-major [M][N], same dtype (AQ_F32 output is accepted
 *           with xy_dtype's input type via aq_linear_f32out)
 *   M     : 1 .. AQ_MAX_M.  M <= AQ_DECODE_MAX_M runs the weight-streaming
 *           kernel, larger M the tensor-core GEMM.
 * Accumulation is binary32.  Error against the exact product, per output, with T = sum_k |x_k w_hat_k|: the
 * weight-streaming kernel multiplies exact codes (about K 2^-24 T); the GEMM rounds each dequantised weight to
 * binary16 before the tensor core, so at most 2^-11 T for either activation type (bfloat16 activations are widened
 * to binary16 first, which is exact inside binary16's range; a token row with a magnitude of 2^15 or more is scaled
 * by a power of two and scaled back after the sum).  Calls on one handle must be ordered on a stream (the handle
 * owns accumulation scratch that concurrent calls would share).  With M > AQ_DECODE_MAX_M the handle allocates
 * further scratch (float32 sums, the widened activations) the first time it sees such a call and again when a
 * later call needs more; calls in between allocate nothing.
 */
aq_status_t aq_linear(aq_handle_t h, const void* x_dev, void* y_dev, int M,
                      aq_dtype_t xy_dtype, aq_stream_t stream);

/* As aq_linear but y_dev is float32 [M][N] holding the unrounded accumulators. */
aq_status_t aq_linear_f32out(aq_handle_t h, const void* x_dev, float* y_dev, int M,
                             aq_dtype_t x_dtype, aq_stream_t stream);

/*
 * aq_linear_noalloc -- aq_linear for M <= AQ_DECODE_MAX_M that reserves no
 * memory.  (No counterpart in the paper: this entry point exists for the
 * library's users, not for the method.)
 *
 * Who needs it: code that runs where device allocation is forbidden or
 * unaffordable -- a control loop with a hard deadline that may not take the
 * allocator's locks or an implicit device synchronisation, a process whose
 * memory budget was fixed at start-up, a plug-in that is handed a stream and
 * told not to touch the allocator.  aq_linear itself allocates nothing per
 * call either, but its accumulation scratch was allocated when the handle was
 * made; here the scratch is a fixed array of AQ_DECODE_MAX_M *
 * AQ_NOALLOC_MAX_N float32 (512 KiB) in the library's device image, which every
 * GPU that loads the library holds until the process exits.
 *
 *   arguments as aq_linear (x_dev, y_dev DEVICE, 16-byte aligned, same dtype)
 *   AQ_ERR_UNSUPPORTED when M > AQ_DECODE_MAX_M or N (rounded up to 16) >
 *   AQ_NOALLOC_MAX_N: the fixed scratch cannot hold the sums.
 * The first call on each device looks up the array's device address (with that
 * device current); make that first call before any stream capture begins.
 * All calls on a device share the one array: it is cleared on the stream at the
 * start of every call, and two calls that overlap on the GPU (different
 * streams, no ordering) race on it and corrupt each other's result.
 * Calls no cudaMalloc/cudaFree and no allocating library routine.
 */
#define AQ_NOALLOC_MAX_N 16384
aq_status_t aq_linear_noalloc(aq_handle_t h, const void* x_dev, void* y_dev, int M,
                              aq_dtype_t xy_dtype, aq_stream_t stream);

/*
 * A program over a list of handles: the linears of a stack of transformer
 * blocks (Section 3: each block holds W_Q, W_K, W_V, W_O, W_gate, W_up,
 * W_down) with the glue between them.  Activations live in float32 buffers
 * [M][width] inside the caller's workspace; the vector a linear consumes is
 * formed from them and rounded to the activation dtype:
 *   AQ_IN_PLAIN    : x = src
 *   AQ_IN_RMSNORM  : x = src / sqrt(mean_k(src^2) + 1e-6)      (no gain)
 *   AQ_IN_SILU_MUL : x = silu(src) * src2,  silu(g) = g / (1 + exp(-g))
 * and the result is dst = W x (AQ_OUT_STORE) or dst = res + W x (AQ_OUT_ADD).
 * Buffer 0 is the program input.  Handles are borrowed, not owned.
 */
typedef enum { AQ_IN_PLAIN = 0, AQ_IN_RMSNORM = 1, AQ_IN_SILU_MUL = 2 } aq_in_op_t;
typedef enum { AQ_OUT_STORE = 0, AQ_OUT_ADD = 1 } aq_out_op_t;

typedef struct {
    aq_handle_t w;      /* the packed matrix, N = width[dst], K = width[src] */
    int32_t src;        /* input buffer index */
    int32_t src2;       /* second input for AQ_IN_SILU_MUL, else ignored */
    int32_t dst;        /* output buffer index (> 0; written by this op only) */
    int32_t res;        /* residual buffer for AQ_OUT_ADD, else ignored */
    int32_t in_op;      /* aq_in_op_t */
    int32_t out_op;     /* aq_out_op_t */
} aq_stack_op_t;

typedef struct {
    int32_t n_ops;
    int32_t n_bufs;
    const aq_stack_op_t* ops;     /* HOST, n_ops entries, in execution order */
    const int64_t* buf_width;     /* HOST, n_bufs entries */
} aq_stack_t;

/* Bytes of workspace aq_stack_forward needs for M tokens (0 on a bad program).  For M <= AQ_DECODE_MAX_M this
 * includes 8 bytes per buffer element for the decode kernel's packed sums. */
size_t aq_stack_workspace_bytes(const aq_stack_t* prog, int M);

/*
 * aq_stack_forward -- run the program (Section 4.3: the deployed forward pass
 * dispatches every quantised matmul to a low-bit kernel).
 *   x0_dev        : DEVICE [M][width[0]] of `dtype` (AQ_F16 / AQ_BF16)
 *   out_dev       : DEVICE [M][width[out_buf]] of `dtype`, the rounded contents
 *                   of buffer out_buf after the last op (may be NULL)
 *   workspace_dev : DEVICE, 256-byte aligned, >= aq_stack_workspace_bytes();
 *                   afterwards buffer b is float32 [M][width[b]] at byte
 *                   offset aq_stack_buffer_offset(prog, M, b): every op's
 *                   input and output stay readable for per-op checks
 * CUDA graphs: the call may be recorded into a graph (stream capture) and
 * replayed.  For M <= AQ_DECODE_MAX_M make one eager call with the same
 * program, M, dtype and workspace on that device first: it builds the device
 * tables of the one-launch kernel, which allocates, and a capture forbids
 * allocation (without that call the capture records the slower form, one
 * launch per linear).  Tables used under a capture stay until a handle of the
 * program is freed.  aq_free of any handle of the program releases them and
 * invalidates every graph recorded with it: destroy those graphs first.
 */
aq_status_t aq_stack_forward(const aq_stack_t* prog, const void* x0_dev, void* out_dev, int out_buf,
                             int M, aq_dtype_t dtype, void* workspace_dev, size_t ws_bytes,
                             aq_stream_t stream);

/*
 * aq_stack_forward_attn -- aq_stack_forward for M <= AQ_DECODE_MAX_M new tokens with attention over a key/value cache
 * between the linears (Section 2: W_Q, W_K, W_V feed the attention whose output W_O reads; the attention itself is
 * the textbook operation, see aq_attn_decode).
 *
 * A buffer of the program that no op writes and that is not buffer 0 is an input filled by somebody else (float32
 * [M][width] in the workspace).  Each aq_stack_attn_t says: after op `after_op` (the last op of a phase; its q, k, v
 * buffers are complete then) rotate q and k for positions pos .. pos + M - 1 (aq_rope's rule), append the rounded k
 * and v to rows pos .. pos + M - 1 of the caches, and write softmax attention of the M tokens over the L = pos + M
 * cached positions (token m sees positions up to pos + m), scale 1/sqrt(128), as float32 into buffer dst_buf, which no
 * op writes and which later ops (W_O) read.  Entries ascend in after_op.  Head dimension 128; (n_heads / n_kv_heads) *
 * M <= 16; widths: q_buf and dst_buf n_heads * 128, k_buf and v_buf n_kv_heads * 128.
 *   attn_scratch_dev : DEVICE, 256-byte aligned, aq_stack_attn_scratch_bytes(n_heads, n_kv_heads, M) bytes (the largest
 *                      over the entries); contents irrelevant
 * The linears between two attention steps run as one launch each of the whole-program decode kernel; a program that
 * kernel cannot take returns AQ_ERR_UNSUPPORTED (the outputs are undefined then).  Other arguments, the workspace and what it
 * holds afterwards as in aq_stack_forward (its rules on CUDA graphs too: one eager call with the same arguments first);
 * calls on one device must not overlap (see aq_attn_decode).
 */
typedef struct {
    int32_t after_op;
    int32_t q_buf, k_buf, v_buf, dst_buf;
    int32_t n_heads, n_kv_heads;
    int32_t pad_;
    void* k_cache_dev;        /* DEVICE [n_kv_heads][L_max][128] of the activation dtype */
    void* v_cache_dev;
    int64_t L_max;
} aq_stack_attn_t;

size_t aq_stack_attn_scratch_bytes(int n_heads, int n_kv_heads, int M);
aq_status_t aq_stack_forward_attn(const aq_stack_t* prog, const aq_stack_attn_t* attn, int n_attn, int64_t pos, float theta,
                                  const void* x0_dev, void* out_dev, int out_buf, int M, aq_dtype_t dtype,
                                  void* workspace_dev, size_t ws_bytes, void* attn_scratch_dev, size_t attn_scratch_bytes,
                                  aq_stream_t stream);

/* Byte offset of buffer b inside the workspace ((size_t)-1 on a bad argument). */
size_t aq_stack_buffer_offset(const aq_stack_t* prog, int M, int b);

/*
 * Byte offset, inside the workspace, of the rounded input vector op `op`
 * consumed: [M][K] of the activation dtype, kept after the call so that each
 * linear can be checked against exactly what it read ((size_t)-1 on a bad
 * argument).  Ops that share an input share the region.
 */
size_t aq_stack_input_offset(const aq_stack_t* prog, int M, int op);

/*
 * aq_check -- synchronises `stream`, then reports whether any kernel of this
 * library gave up on a bounded device-side wait since the last aq_check
 * (AQ_ERR_TIMEOUT; the record is cleared) or the stream saw a CUDA error
 * (AQ_ERR_CUDA).  Outputs of a call that timed out are undefined.
 */
aq_status_t aq_check(aq_stream_t stream);

/*
 * aq_set_wait_limit_ns -- how long a device-side wait of the whole-program decode kernel (for an input another
 * CTA has not finished, for a weight copy) may last before the kernel gives up, raises the status that aq_check
 * reports as AQ_ERR_TIMEOUT, and returns with the context intact.  0 restores the default (two seconds).
 * Applies to launches made after the call.  (Section 4.3's runtime has no counterpart: this is the library's
 * failure detection.)
 */
aq_status_t aq_set_wait_limit_ns(uint64_t ns);

/*
 * aq_debug_decode_hold -- TESTING ONLY.  While on, the tables aq_stack_forward builds for the decode kernel make the
 * first phase that reads another op's output expect one contribution more than will ever arrive, so every CTA's
 * wait for that input runs out (after the limit above) and the time-out path can be exercised on a healthy GPU:
 * nothing traps, faults or spins without bound.  Programs run while it is off are not affected.
 */
void aq_debug_decode_hold(int on);

/* Releases the handle and its device memory (synchronises its last stream). */
void aq_free(aq_handle_t h);

const char* aq_status_string(aq_status_t s);

/* Text of the last CUDA error this thread's libaq call saw ("" if none). */
const char* aq_last_cuda_error(void);

/* Number of CUDA kernels this library has launched in this process so far. */
uint64_t aq_kernel_launches(void);

#ifdef __cplusplus
}
#endif
#endif /* AQ_H_ */
