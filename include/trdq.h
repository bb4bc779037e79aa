/* trdq.h -- C ABI of the time-rotated quantized linear layer for NVIDIA B200 (sm_100a).
 *
 * The library implements the online path of TR-DQ's rotated quantized linear layer
 * (Sec. 3.2, Eq. 10):
 *
 *     F_t(X, W) = G_t(X) . H_t(W),   G_t(X) = (X . Delta_t) . R_t,   H_t(W) = R_t^T . (Delta_t^-1 . W)
 *
 * with the parameter set {R_t, Delta_t} chosen by the current diffusion time-step t
 * ("Time-Rotation"), activations quantized dynamically per token and weights per
 * output channel (Sec. 3.1, Eq. 1-2, used in symmetric signed form: zero-point 0,
 * scale = absmax / qmax, nearest rounding with ties to even).
 *
 * The rotation R_g of a time-step group g is block diagonal (Eq. 8) with blocks of
 * 128 x 128: R_g = diag(d_g) . BlockDiag(H_128) / sqrt(128), H_128 the Sylvester
 * Walsh-Hadamard matrix in natural order and d_g a +-1 vector.  The per-group channel
 * scaling Delta_g (Eq. 4-5; the per-time-step hyper-parameter alpha of Eq. 5 enters
 * through it) multiplies X online and divides W offline, exactly as Eq. 10 is written.
 *
 * Conventions
 *   - Every matrix is row major with the reduction dimension K (= C_in) contiguous:
 *     X [M, K], W [N, K] (the transpose of the paper's C_in x C_out matrix), Y [M, N].
 *   - "dev" pointers are CUDA device pointers, "host" pointers are ordinary host
 *     memory.  bf16 tensors are passed as `const void*` / `void*` to 2-byte elements.
 *   - `stream` is a `cudaStream_t` passed as `void*` (NULL = the legacy default stream).
 *   - All device work is enqueued asynchronously on `stream`; no entry point
 *     synchronises unless its comment says so.  The online calls (trdq_rotate_quantize and
 *     its _asym, _dense and norm-fused forms, trdq_linear and its _cfg, _act, _asym and split-K
 *     forms, trdq_run_layers, trdq_gemm_i32) allocate no memory; trdq_prepare_weights with a
 *     dense-block rotation is the one call that waits for its own work (it frees a scratch buffer).
 *   - The caller owns every tensor it passes.  The library owns only the opaque
 *     trdq_rotation / trdq_weights objects until their _destroy call.  An object belongs to the
 *     device that was current when it was created; calls that use it with another device
 *     current return TRDQ_ERR_MISMATCH.  Entry points may be called from several host threads.
 *   - Errors are reported by return code only; the library never aborts, traps or
 *     prints.  Argument errors are found on the host before anything is launched.
 *     NaN/Inf in X or W give unspecified codes (not checked).
 *   - There is no CPU fallback: without a CUDA device every call that needs one
 *     returns TRDQ_ERR_CUDA.
 *   - Debug runs: with TRDQ_DEBUG=1 in the environment (read once per process) every online call waits
 *     for its own work and returns TRDQ_ERR_CUDA / TRDQ_ERR_TIMEOUT itself if the device reported an
 *     error or a bounded wait expired (the status word is read and cleared), so a problem is pinned to
 *     the call that caused it.  Such a process must not capture those calls into a CUDA graph.
 */
#ifndef TRDQ_H_
#define TRDQ_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define TRDQ_BLOCK 128        /* rotation block size 2^n (Eq. 8), n = 7 */
#define TRDQ_MAX_K 131072     /* keeps |sum_k q*qw| <= K*127*127 below 2^31 */

typedef enum trdq_status {
  TRDQ_OK = 0,
  TRDQ_ERR_NULL = 1,      /* a required pointer is NULL */
  TRDQ_ERR_SHAPE = 2,     /* K % 128 != 0, N % 16 != 0, M < 0, K > TRDQ_MAX_K, block != 128, ld too small */
  TRDQ_ERR_ALIGN = 3,     /* a device pointer or row stride is not 16-byte aligned */
  TRDQ_ERR_TIMESTEP = 4,  /* t outside [t_bounds[0], t_bounds[G]) */
  TRDQ_ERR_GROUP = 5,     /* num_groups < 1, bounds not strictly ascending, sign not +-1, smooth <= 0 */
  TRDQ_ERR_WBITS = 6,     /* wbits is neither 8 nor 4, or the call does not support this weight format */
  TRDQ_ERR_CUDA = 7,      /* a CUDA runtime / driver call failed (no device, launch error, ...) */
  TRDQ_ERR_NOMEM = 8,     /* host or device allocation failed */
  TRDQ_ERR_TIMEOUT = 9,   /* a bounded device-side wait expired (see trdq_device_status) */
  TRDQ_ERR_MISMATCH = 10, /* objects passed together were built for different K / groups, the rotation's kind does not fit the call,
                             or the current device is not the one the object was created on */
  TRDQ_ERR_SCRATCH = 11   /* the problem needs more than the library's built-in scratch area (trdq_linear_splitk_static) */
} trdq_status;

/* Description of the per-group transforms (Time-Rotation, Sec. 3.2).  All arrays are
 * host memory and are copied by trdq_rotation_create. */
typedef struct trdq_rotation_spec {
  int32_t K;                /* C_in; multiple of 128 */
  int32_t block;            /* rotation block size; must be 128 */
  int32_t num_groups;       /* G >= 1 time-step groups */
  const int32_t* t_bounds;  /* host [G+1], strictly ascending; group g covers t_bounds[g] <= t < t_bounds[g+1] */
  const int8_t* signs;      /* host [G][K], each +1 or -1: the diagonal d_g */
  const float* smooth;      /* host [G][K], > 0: Delta_g as multiplied onto X (Eq. 10); NULL = all ones */
} trdq_rotation_spec;

typedef struct trdq_rotation trdq_rotation; /* per-group device tables of one C_in */
typedef struct trdq_weights trdq_weights;   /* H_t(W) of one linear layer, quantized, for all groups */

/* Human-readable name of a status code (static storage, never NULL). */
const char* trdq_status_string(trdq_status s);

/* Builds the per-group tables.  For each group the two fused fp32 vectors
 *   act[j]    = fl32(d[j] * Delta[j] * 2^-3.5)     (applied to X)
 *   weight[j] = fl32(d[j] / Delta[j] * 2^-3.5)     (applied to W)
 * are formed in double precision, rounded once and uploaded (2^-3.5 = 1/sqrt(128) is the
 * Hadamard normalisation).  Synchronous (blocking copies).  `*out` is set only on TRDQ_OK. */
trdq_status trdq_rotation_create(const trdq_rotation_spec* spec, trdq_rotation** out);
trdq_status trdq_rotation_destroy(trdq_rotation* rot);

/* Tables for the FULL balancing transform of Eq. 9 / Eq. 10,
 *     G_t(X) = (X . Delta_t) . R1_t . P_t . R2_t,      H_t(W) = R2_t^T . P_t^T . R1_t^T . (Delta_t^-1 . W):
 * R1 is the rotation described by `spec`, P the zigzag channel permutation given as an index vector
 * ((v P)[j] = v[perm[j]]), and R2 a second block rotation of the same form with its own +-1 vector:
 *   v1 = ((x o act) . BlockDiag(H_128));  v2[j] = fl32(v1[perm[j]] * fl32(d2[j] * 2^-3.5));  v3 = v2 . BlockDiag(H_128)
 * perm: host int32 [G][K], each group a permutation of 0 .. K-1 (TRDQ_ERR_GROUP otherwise); signs2: host
 * int8 [G][K] of +-1, or NULL for all +1.  K <= 16384.  An object created here makes trdq_rotate_quantize,
 * trdq_prepare_weights and everything built on them use the full transform; the GEMM is unchanged. */
trdq_status trdq_rotation_create_full(const trdq_rotation_spec* spec, const int32_t* perm, const int8_t* signs2,
                                      trdq_rotation** out);

/* Zigzag permutation of Sec. 3.2 from per-channel magnitudes (host arrays; K a multiple of 128): channels
 * sorted by magnitude, largest first (ties: lower index first), are dealt to the K/128 blocks in serpentine
 * order -- round r fills slot r of blocks 0 .. B-1 when r is even and of blocks B-1 .. 0 when r is odd --
 * so strong channels are spread evenly over the blocks before the second rotation.  Pure host arithmetic. */
trdq_status trdq_zigzag_permutation(const float* magnitude, int32_t K, int32_t* perm);

/* Time-step -> group (Sec. 3.2: the parameter set is selected by the current time-step).
 * Pure host arithmetic.  TRDQ_ERR_TIMESTEP if t is outside the covered range. */
trdq_status trdq_group_of(const trdq_rotation* rot, int32_t t, int32_t* g);

/* The same lookup on a bare table (host [num_groups+1], strictly ascending), for callers that
 * schedule sampling steps before any device object exists.  Pure host arithmetic. */
trdq_status trdq_find_group(const int32_t* t_bounds, int32_t num_groups, int32_t t, int32_t* g);

/* Offline side of Eq. 10: for every group g, rotate each output channel's row of W with
 * the weight vector of g (H_t(W) = R_t^T Delta_t^-1 W, written on rows of W^T) and quantize
 *   wbits = 8: per output channel, codes int8 [N, K] in [-127, 127], scale fp32 [N] = absmax / 127;
 *   wbits = 4: per (output channel, 128 consecutive k), codes in [-7, 7] packed two per byte
 *              (uint8 [N, K/2], even k in the low nibble, two's complement), scale fp32 [N, K/128] = absmax / 7.
 * W_bf16: dev [N, K] contiguous, 16-byte aligned.  N % 16 == 0.  Allocates the G quantized copies
 * (cudaMalloc) and enqueues the kernels on `stream`; the object may be used on the same stream
 * right away.  `*out` is set only on TRDQ_OK. */
trdq_status trdq_prepare_weights(const trdq_rotation* rot, const void* W_bf16, int32_t N, int32_t wbits,
                                 trdq_weights** out, void* stream);
trdq_status trdq_weights_destroy(trdq_weights* w);

/* Shape and format of a prepared layer (any output pointer may be NULL). */
trdq_status trdq_weights_info(const trdq_weights* w, int32_t* N, int32_t* K, int32_t* wbits, int32_t* num_groups);

/* Device pointers to group g's quantized codes and scales (layouts as in trdq_prepare_weights);
 * the memory stays owned by `w`. */
trdq_status trdq_weights_view(const trdq_weights* w, int32_t g, const void** Wq, const float** scales);

/* Copies group g's codes and scales into caller-owned device buffers of exactly the sizes given
 * in trdq_prepare_weights (device-to-device, asynchronous on `stream`); either may be NULL. */
trdq_status trdq_weights_export(const trdq_weights* w, int32_t g, void* codes_out, float* scales_out, void* stream);

/* Online activation path G_t(X) followed by dynamic per-token quantization (Sec. 3.1 Eq. 1-2,
 * Sec. 3.2: the activation scales are computed online, per token):
 *   v[m, :]   = (x[m, :] o act_g) . BlockDiag(H_128), fp32 butterflies in the order h = 1, 2, ..., 64
 *   scales[m] = absmax_k |v[m, k]| / 127
 *   codes[m,k]= rne(v[m, k] * fl32(127 / absmax))     (all-zero row: scale 0, codes 0)
 * with g the group of time-step t.  X_bf16: dev [M, ldx] (ldx >= K elements, ldx % 8 == 0, base
 * 16-byte aligned); codes: dev int8 [M, K] contiguous, 16-byte aligned; scales: dev fp32 [M].
 * M == 0 is a no-op.  Both CFG halves are simply rows of the same call. */
trdq_status trdq_rotate_quantize(const trdq_rotation* rot, int32_t t, const void* X_bf16, int64_t ldx, int32_t M,
                                 int8_t* codes, float* scales, void* stream);

/* Integer GEMM of Eq. 10 on the codes with the dequantizing epilogue:
 *   wbits = 8:  y[m, n] = bf16( (sum_k q[m,k] * qw_g[n,k]) * sx[m] * sw_g[n] + bias[n] )
 *   wbits = 4:  y[m, n] = bf16( sx[m] * sum_kg sw4_g[n,kg] * (sum_{k in kg} q[m,k] * qw4_g[n,k]) + bias[n] )
 * int8 x int8 (int4) products accumulate exactly in int32 on the tensor cores; the epilogue runs in
 * fp32.  codes: dev int8 [M, K] contiguous, 16-byte aligned; scales: dev fp32 [M]; bias_bf16: dev [N]
 * or NULL; Y_bf16: dev [M, ldy], ldy >= N, ldy % 8 == 0, base 16-byte aligned.  Conditional and
 * unconditional CFG rows stacked in one call share a single read of the weights. */
trdq_status trdq_linear(const trdq_weights* w, int32_t t, const int8_t* codes, const float* scales, int32_t M,
                        const void* bias_bf16, void* Y_bf16, int64_t ldy, void* stream);

/* Same as trdq_linear for two separately stored row segments (the conditional and the
 * unconditional CFG half) of the same time-step, in ONE launch so that each weight tile is
 * fetched once for both.  Segment s has M[s] rows (either may be 0). */
trdq_status trdq_linear_cfg(const trdq_weights* w, int32_t t, const int8_t* const codes[2], const float* const scales[2],
                            const int32_t M[2], const void* bias_bf16, void* const Y_bf16[2], const int64_t ldy[2],
                            void* stream);

/* Split-K form of trdq_linear for problems with few rows and a very long reduction (K >= 8192 and
 * fewer output tiles than half the SMs; shorter reductions are faster in one kernel): the k range of Eq. 10's integer sum is cut into `splits` parts computed by different
 * CTAs, their exact int32 partial sums go to a caller-provided workspace, and a second kernel adds
 * them and applies the epilogue.  Integer addition is associative, so the output is bit-identical to
 * trdq_linear's.  8-bit weights, one row segment.
 * trdq_linear_splitk_workspace reports how many parts the library would use for M rows (1 = split-K does
 * not pay for this shape) and the workspace bytes needed (splits * M * N * 4; 0 when splits == 1).
 * trdq_linear_splitk: workspace is dev memory, 16-byte aligned, of at least that many bytes
 * (TRDQ_ERR_NOMEM if smaller); with splits == 1 it is not touched and the call is trdq_linear.
 * The workspace is written and read on `stream`; concurrent calls must not share it. */
trdq_status trdq_linear_splitk_workspace(const trdq_weights* w, int32_t M, int32_t* splits, uint64_t* bytes);
trdq_status trdq_linear_splitk(const trdq_weights* w, int32_t t, const int8_t* codes, const float* scales, int32_t M,
                               const void* bias_bf16, void* Y_bf16, int64_t ldy, void* workspace, uint64_t workspace_bytes,
                               void* stream);

/* trdq_linear_splitk for callers that cannot provide a workspace because they cannot allocate device
 * memory at this point: an inference server that handed all device memory to its own pool at start-up
 * (a cudaMalloc would simply fail), or a latency-critical loop in which the device-wide synchronisation
 * that cudaMalloc / cudaFree imply is not acceptable.  (The paper has no counterpart; this is a
 * deployment convenience.)  The partial sums go to a fixed array of TRDQ_STATIC_SCRATCH_ELEMS int32
 * (8 MiB) that is part of the library image: every GPU on which the library is used holds it until the
 * process exits.  The call allocates nothing (no cudaMalloc / cudaFree, no allocating library routine);
 * inputs and outputs are the caller's as in trdq_linear.
 *   - TRDQ_ERR_SCRATCH if splits * M * N (splits as reported by trdq_linear_splitk_workspace) exceeds
 *     TRDQ_STATIC_SCRATCH_ELEMS; nothing is launched.  With splits == 1 the scratch is not used and the
 *     call is trdq_linear.
 *   - The first call on a device looks up the array's device address (once per device, with that device
 *     current) and configures the kernels; make that first call during start-up, before any stream capture.
 *   - "Allocates nothing" holds once the library's GEMM code is resident on the device: the array is part of
 *     that code image and the driver reserves its 8 MiB when the image is first used there (any trdq_linear*
 *     call, or trdq_prepare_weights with 8-bit weights, does that).  A server that hands the rest of the
 *     device to its own pool must make one such call first, or the load itself fails with TRDQ_ERR_CUDA.
 *   - All calls share the one array, and it keeps the last call's contents.  That is harmless for
 *     calls that run one after another (every value read is written by the same call first), but two
 *     calls that overlap on the GPU -- different streams, or concurrent host threads -- race on it:
 *     serialise them. */
#define TRDQ_STATIC_SCRATCH_ELEMS (2u * 1024u * 1024u)
trdq_status trdq_linear_splitk_static(const trdq_weights* w, int32_t t, const int8_t* codes, const float* scales, int32_t M,
                                      const void* bias_bf16, void* Y_bf16, int64_t ldy, void* stream);

/* The quantizer of Eq. 1-3 taken literally for the activations (asymmetric, unsigned 8 bit, one zero point per
 * token), after the same block rotation as trdq_rotate_quantize:
 *   s[m] = (max - min) / 255,  z[m] = -rne(min * fl(255 / (max - min))),  q[m,k] = clamp(rne(v * fl(255 / (max - min))) + z[m], 0, 255)
 * (Eq. 3's printed sign of z is read as a typo: with Eq. 1's "+ z" the minimum must map to code 0.)  Dequantized
 * value: s[m] * (q - z[m]).  codes: dev uint8 [M, K]; scales: dev fp32 [M]; zero_points: dev int32 [M].
 * K <= 10240; single rotation only (not with trdq_rotation_create_full).
 * trdq_linear_asym consumes them with 8-bit weights:
 *   y[m,n] = bf16( s[m] * sw[n] * (sum_k q[m,k] * qw[n,k] - z[m] * sum_k qw[n,k]) + bias[n] )
 * the first sum on the tensor cores (unsigned x signed 8 bit), the column sums of the weight codes taken once at
 * trdq_prepare_weights.  K <= 32768 keeps every intermediate inside int32. */
trdq_status trdq_rotate_quantize_asym(const trdq_rotation* rot, int32_t t, const void* X_bf16, int64_t ldx, int32_t M,
                                      uint8_t* codes, float* scales, int32_t* zero_points, void* stream);
trdq_status trdq_linear_asym(const trdq_weights* w, int32_t t, const uint8_t* codes, const float* scales, const int32_t* zero_points,
                             int32_t M, const void* bias_bf16, void* Y_bf16, int64_t ldy, void* stream);

/* trdq_rotate_quantize with the producer of its input folded in: the quantized linears of a transformer block read a
 * LayerNorm output modulated per sample (adaLN),
 *   h[m,k] = (X[m,k] - mean_m) / sqrt(var_m + eps) * (1 + scale[s,k]) + shift[s,k],   s = m / rows_per_sample,
 * mean and biased variance over the K channels of row m.  h is formed in fp32 in registers (never stored, not rounded to
 * bf16) and takes the place of X in Eq. 10's G_t: v = (h o Delta_t) R_t, then the per-token quantizer, codes and scales as
 * in trdq_rotate_quantize.  shift_bf16 / scale_bf16: dev bf16 [ceil(M / rows_per_sample), K], 16-byte aligned, or NULL (zero).
 * Single Hadamard rotation only (TRDQ_ERR_MISMATCH for the full transform or dense blocks); K <= 8192; eps >= 0.
 * The reductions run in a fixed order, so equal inputs give equal codes.  The row statistics are fp32 sums; against an
 * evaluation in double h agrees to about 2^-18 relative to its terms, which moves a code only at a rounding boundary.
 * The paper does not discuss normalisation; this is a fusion on the boundary of its layer. */
trdq_status trdq_norm_rotate_quantize(const trdq_rotation* rot, int32_t t, const void* X_bf16, int64_t ldx, int32_t M,
                                      const void* shift_bf16, const void* scale_bf16, int32_t rows_per_sample, float eps, int8_t* codes,
                                      float* scales, void* stream);

/* trdq_linear with the activation that follows the layer folded into its epilogue, so that the activation costs no
 * pass over memory of its own (the first MLP linear of a transformer block is followed by GELU, and its output is what
 * the next trdq_rotate_quantize reads):
 *   y[m,n] = bf16( act( acc[m,n] * sx[m] * sw[n] + bias[n] ) )
 * act: TRDQ_ACT_NONE (identical to trdq_linear) or TRDQ_ACT_GELU_TANH,
 *   gelu(x) = 0.5 x (1 + tanh( sqrt(2/pi) (x + 0.044715 x^3) )),
 * evaluated in fp32 with a relative error near 1e-6 (well inside the bf16 rounding of the result).  8- and 4-bit weights.
 * The paper does not discuss activations; this is a fusion on the boundary of its layer.  Any other act: TRDQ_ERR_SHAPE. */
#define TRDQ_ACT_NONE 0
#define TRDQ_ACT_GELU_TANH 1
trdq_status trdq_linear_act(const trdq_weights* w, int32_t t, const int8_t* codes, const float* scales, int32_t M, const void* bias_bf16,
                            void* Y_bf16, int64_t ldy, int32_t act, void* stream);

/* Dense block rotations (Sec. 3.2, Eq. 6-8): R = BlockDiag(R_b1 .. R_bK) with dense 128 x 128 orthogonal blocks, one
 * set per time-step group (Eq. 10).  blocks: host fp32 [G][K/128][128][128], R_b[i][j] with i the input channel
 * (v = x R).  smooth: host [G][K] (> 0) or NULL, the multiplier Delta_t of Eq. 10, folded into the rows of each block.
 * The scaled blocks are STORED IN BF16, S_b[i][j] = bf16(Delta[128 b + i] * R_b[i][j]) (nearest, ties to even), because
 * that is the format the tensor cores apply them in; the weight side (trdq_prepare_weights with this object, 8- or 4-bit)
 * multiplies by the exact inverse of the stored S_b, computed on the host in double, so the product
 * G_t(X) . H_t(W) = X W of Eq. 9 is preserved whatever the rounding did:
 *   wr[n, 128 b + j] = fl32( sum_i (S_b^-1)[j][i] * W[n, 128 b + i] )      sums in double, i ascending.
 * TRDQ_ERR_GROUP: bounds not ascending, a non-positive smooth value, a non-finite product or a singular block.
 * The object is accepted by trdq_prepare_weights, trdq_group_of, trdq_rotate_dense_quantize and
 * trdq_rotation_destroy, and by trdq_run_layers through the op's workspace; the Hadamard entry points (trdq_rotate_quantize,
 * _asym, trdq_norm_rotate_quantize) return TRDQ_ERR_MISMATCH. */
trdq_status trdq_rotation_create_dense(int32_t K, int32_t num_groups, const int32_t* t_bounds, const float* blocks, const float* smooth,
                                       trdq_rotation** out);

/* Online side with dense blocks: v[m, 128 b + j] = sum_i X[m, 128 b + i] * S_b[i][j] on the tensor cores (bf16 operands, every
 * product exact, fp32 accumulation), then the per-token quantizer of trdq_rotate_quantize on v (same scale and code
 * definitions).  The row maximum must be known before the first code, so X is read twice; `workspace` (device,
 * 4-byte aligned, at least the size trdq_rotate_dense_workspace reports = 32 * M bytes) holds partial row maxima between
 * the two passes.  It is scratch: no initialisation needed, contents undefined afterwards; two calls that
 * may overlap on the GPU need separate workspaces.  Asynchronous on `stream`; allocates nothing.
 * TRDQ_ERR_MISMATCH if rot was not made by trdq_rotation_create_dense; TRDQ_ERR_NOMEM if the workspace is too small;
 * otherwise the errors of trdq_rotate_quantize.  Because the accumulation order inside the tensor cores is not
 * specified, v agrees with the exactly rounded sum only to a few units of 2^-24 * sum_i |x_i S_ij|; codes can differ by
 * one step from an exactly rounded evaluation where v * 127 / amax falls that close to a rounding boundary. */
trdq_status trdq_rotate_dense_workspace(const trdq_rotation* rot, int32_t M, uint64_t* bytes);
trdq_status trdq_rotate_dense_quantize(const trdq_rotation* rot, int32_t t, const void* X_bf16, int64_t ldx, int32_t M, int8_t* codes,
                                       float* scales, void* workspace, uint64_t workspace_bytes, void* stream);

/* Greedy construction of ONE block (Eq. 6-7), on the host in double; offline calibration, no GPU work.
 * x_calib: host fp32 [rows][128], calibration activations of the block's 128 channels.  gauss: host double
 * [steps][128][128], the random draws of the method (standard normal), passed in so that the result is reproducible.
 * Step k: C swaps column 0 with the column holding the largest |entry| of the current activations; Q_k has the uniform
 * first row 1/sqrt(128) and rows 1..127 from gauss[k-1] made orthonormal by Gram-Schmidt; R^k = C Q_k C (Eq. 6).  The
 * result is R^1 R^2 .. R^n with n the first step that minimises max |X R^1 .. R^n| (Eq. 7), written to R_out [128][128]
 * (fp32) and *n_used (may be NULL).  TRDQ_ERR_GROUP for non-finite inputs or a degenerate draw. */
trdq_status trdq_greedy_rotation_block(const float* x_calib, int32_t rows, int32_t steps, const double* gauss, float* R_out,
                                       int32_t* n_used);

/* One quantized linear layer of a denoising step: rotate + quantize X into the caller's code and
 * scale buffers, then the integer GEMM with its epilogue into Y (shapes as in the two calls above). */
typedef struct trdq_layer_op {
  const trdq_rotation* rot; /* tables for this layer's C_in */
  const trdq_weights* w;    /* prepared weights; w's K must equal rot's K */
  const void* X_bf16;       /* dev [M, ldx] */
  int64_t ldx;
  int32_t M;
  int8_t* codes;            /* dev [M, K] scratch owned by the caller */
  float* scales;            /* dev [M] scratch owned by the caller */
  const void* bias_bf16;    /* dev [N] or NULL */
  void* Y_bf16;             /* dev [M, ldy] */
  int64_t ldy;
  int32_t act;              /* TRDQ_ACT_NONE or TRDQ_ACT_GELU_TANH: activation folded into this layer's epilogue */
  void* workspace;          /* only for a rot made by trdq_rotation_create_dense: scratch of trdq_rotate_dense_quantize */
  uint64_t workspace_bytes; /* at least what trdq_rotate_dense_workspace reports for M; ignored otherwise */
} trdq_layer_op;

/* Runs `count` layer ops in order for time-step t on `stream`: the group switch of the sampling
 * loop (Sec. 3.2: every layer selects its parameter set by the current time-step) without one
 * host round trip per kernel.  Validates every op before launching anything.  TRDQ_ERR_MISMATCH
 * if an op's rot and w disagree in K or in their time-step bounds.  An op whose rot holds dense blocks runs
 * trdq_rotate_dense_quantize with the op's workspace (TRDQ_ERR_NULL / TRDQ_ERR_NOMEM if it is missing or too small).
 * Every op has its own row count M, so a block whose unconditional branch reuses the conditional
 * attention (attention sharing, Sec. 3.3) lists its attention linears with the conditional rows only
 * and its MLP linears with all rows; nothing is computed for the skipped rows. */
trdq_status trdq_run_layers(const trdq_layer_op* ops, int32_t count, int32_t t, void* stream);

/* Raw accumulators of the integer GEMM (wbits = 8 only): acc[m, n] = sum_k q[m,k] * qw_g[n,k],
 * dev int32 [M, ldacc], ldacc >= N, ldacc % 4 == 0.  Exists so that the exact integer result
 * can be checked bit for bit. */
trdq_status trdq_gemm_i32(const trdq_weights* w, int32_t t, const int8_t* codes, int32_t M, int32_t* acc, int64_t ldacc,
                          void* stream);

/* Reads and clears the device-side status word of the current device.  Kernels never spin
 * without bound: a wait on a memory barrier that exceeds its limit sets a bit in this word
 * and the kernel runs to completion with unspecified output.  SYNCHRONISES the device.
 * Returns TRDQ_OK (word was 0), TRDQ_ERR_TIMEOUT, or TRDQ_ERR_CUDA; `*word` (may be NULL)
 * receives the raw bits. */
trdq_status trdq_device_status(uint32_t* word);

/* Reports which kernel a call would run on the current device, for benchmark and profile reports (the paper has no
 * counterpart).  stage 0: trdq_rotate_quantize on M rows of K channels (N, wbits ignored); stage 1: trdq_linear on M rows
 * against [N, K] weights of `wbits` bits.  `name` (host, at least 48 bytes, `name_bytes` its size) receives a
 * NUL-terminated kernel name such as "gemm_w8a8_pair_kernel<256>".  The answer comes from the same functions the
 * launchers use.  TRDQ_ERR_CUDA without a device: the choice depends on its SM count. */
trdq_status trdq_kernel_choice(int32_t stage, int32_t M, int32_t K, int32_t N, int32_t wbits, char* name, int32_t name_bytes);

/* Measurement aid (the paper has no counterpart): runs the tensor pipe by itself.  Every resident CTA pair issues
 * `mmas_per_cluster` (8 ... 2^22) back-to-back tcgen05.mma cta_group::2 kind::i8 of shape 256 x 256 x 32 on constant
 * operands that already sit in shared memory: no loads, no epilogue, nothing is written to global memory.
 * `*clusters` (host) receives the number of CTA pairs launched, so one launch performs
 *     clusters * mmas_per_cluster * 2 * 256 * 256 * 32   integer operations;
 * the caller times the launch on `stream`.  The rate is the ceiling of the INT8 GEMM at the clocks the device runs at.
 * The wait for completion is bounded like every other one (trdq_device_status reports an expiry). */
trdq_status trdq_measure_mma_ceiling(int32_t mmas_per_cluster, int32_t* clusters, void* stream);

/* Exercises the bounded wait on purpose: launches one warp that waits on a memory barrier nothing will ever
 * signal.  The wait expires after 20 ms, sets bit 31 of the status word and the kernel ends normally; the next
 * trdq_device_status returns TRDQ_ERR_TIMEOUT with that bit and clears it, and the device stays fully usable.
 * For checking that a stuck pipeline would be reported instead of hanging the GPU. */
trdq_status trdq_selftest_wait_expiry(void* stream);

/* Library version, major * 100 + minor. */
int32_t trdq_version(void);

#ifdef __cplusplus
}
#endif
#endif /* TRDQ_H_ */
