/*
 * lqlora.h -- C ABI of the B200 (sm_100a) LQ-LoRA linear-layer library.
 *
 * The layer (Sec. 2.1 and Sec. 3.1 of arXiv 2311.12023) keeps a pretrained matrix as a fixed
 * quantized matrix Q plus a trainable rank-r product L1 L2 and computes X (Q + L1 L2).  This
 * library stores matrices the way nn.Linear does, i.e. transposed with respect to the paper:
 *
 *     Q, W : [N = out_features, K = in_features]  row major
 *     L1   : [N, r] bf16        L2 : [r, K] bf16
 *     X    : [M, K] bf16        Y, dY : [M, N] bf16        dX : [M, K] bf16
 *
 *     forward          Y  = X deq(Q)^T + (X L2^T) L1^T
 *     input gradient   dX = dY deq(Q)  + (dY L1) L2
 *
 * Q is produced by the NormalFloat double quantization of Sec. 2.2 / Sec. 3.2 with the
 * configuration tuple c = (b0, b1, b2, B0, B1).
 *
 * General rules
 *   - Every pointer named *_dev or documented as "device" is a CUDA device pointer owned by the
 *     caller; the library never allocates or frees device memory and keeps no state besides
 *     immutable code-book tables in constant memory (uploaded on first use per device).
 *   - `stream` is a cudaStream_t passed as void*.  Calls enqueue work on it and return without
 *     synchronizing, unless stated otherwise.
 *   - Every function returns an lqlora_status (0 = success, negative = error).  Arguments are
 *     validated on the host before anything is launched; on error nothing has been enqueued.
 *     No function throws, aborts or traps.
 *   - Inputs must be finite.
 *   - There is no CPU fallback: without a CUDA device every compute entry point returns
 *     LQLORA_ERR_CUDA.
 *   - One device per process (the usual one-process-per-GPU arrangement): kernel attributes and the SM
 *     count are looked up once, on the device that is current at the first call.
 */
#ifndef LQLORA_H_
#define LQLORA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    LQLORA_OK = 0,
    LQLORA_ERR_INVALID_CONFIG = -1,   /* b0 not in {2,3,4,8}; B0 not a power of two in [16,256];
                                         B1 not a power of two in [16,4096]; b1 not in {2,3,4,8};
                                         b2 not one of LQLORA_B2_*                                  */
    LQLORA_ERR_INVALID_SHAPE = -2,    /* N, K, M <= 0; K % 64 != 0; K % B0 != 0; r % 16 != 0; r > 128 */
    LQLORA_ERR_NULL_POINTER = -3,
    LQLORA_ERR_MISALIGNED = -4,       /* a device pointer is not 16-byte aligned                    */
    LQLORA_ERR_WORKSPACE_TOO_SMALL = -5,
    LQLORA_ERR_CUDA = -6,             /* a CUDA runtime / driver call failed (no device, launch)   */
    LQLORA_ERR_TIMEOUT = -7,          /* a bounded device-side wait expired (see lqlora_workspace_status) */
    LQLORA_ERR_UNSUPPORTED = -8       /* valid arguments that this build has no kernel for          */
} lqlora_status;

/* Configuration tuple c = (b0, b1, b2, B0, B1) of Sec. 3.2 (search space: Table 1). */
enum { LQLORA_B2_FP32 = 32, LQLORA_B2_FP16 = 16, LQLORA_B2_BF16 = -16 };
typedef struct {
    int b0;   /* bits of a NormalFloat code: 2, 3, 4 or 8                         */
    int B0;   /* weights per first-level block (along K): 16, 32, 64, 128, 256    */
    int b1;   /* bits of a quantized block scale: 2, 3, 4 or 8                    */
    int B1;   /* blocks per second-level group (flattened row-major block order)  */
    int b2;   /* format of a second-level scale, cast(v, b2): LQLORA_B2_FP32, _FP16 (IEEE half) or _BF16;
                 the storage formula counts |b2| bits                              */
} lqlora_config;

/*
 * A quantized matrix.  All three arrays are device memory owned by the caller, each 16-byte
 * aligned, of the sizes lqlora_packed_sizes reports.
 *
 *   scale_codes  s^_i in flattened row-major block order (block i covers elements [i*B0, (i+1)*B0) of the
 *                row-major matrix): one byte each for b1 = 8; for b1 < 8 a bit stream of b1 bits each, code i in
 *                bits [i*b1, (i+1)*b1) of the little-endian byte stream (eight codes take b1 bytes)
 *   scale2       v_g = absmax of the block scales of group g, [ceil(nblk / B1)] numbers in the format b2 names
 *                (lqlora_unpack_scales returns both arrays as one byte per code and fp32)
 *   codes        packed b0-bit codes, exactly b0 bits per weight when N % 128 == 0 (rows are
 *                padded to a multiple of 128 otherwise).  Layout ("tile-interleaved bitstream"):
 *                  - the matrix is cut into tiles of 128 rows x 64 columns, stored one after the
 *                    other in row-major tile order; a tile takes 1024*b0 bytes;
 *                  - a tile is four slabs of 32 rows (rows 32q .. 32q+31, q = 0..3), 256*b0 bytes each;
 *                  - inside a slab, the 64 columns form two groups g = 0, 1 of 32 columns; the 32
 *                    codes c[0..31] of (row, g) take b0 32-bit words w = 0..b0-1, each a string of
 *                    eight 4-bit fields (for b0 = 8: four bytes):
 *                      b0 = 4: field i of word w = c[8w+i];
 *                      b0 = 3: low three bits of field i of word w (w < 3) = c[8w+i], top bit = bit w of c[24+i];
 *                      b0 = 2: low two bits of field i of word w = c[16w+i], high two bits = c[16w+8+i];
 *                      b0 = 8: byte i of word w = c[4w+i];
 *                  - word w of (row, g) in tile column kt is the 32-bit word number
 *                    (g*b0 + w)*32 + ((row + 8*g + 16*(kt % 2)) % 32) of the slab (the rows of a word plane
 *                    are rotated per group and per tile column to spread shared-memory banks).
 *                Consecutive 32-bit words of a slab therefore belong to consecutive rows, so a
 *                warp reads or writes a slab with fully coalesced accesses and conflict-free
 *                shared-memory accesses.  Use lqlora_unpack to obtain one code per byte.
 */
typedef struct {
    void* codes;
    uint8_t* scale_codes;
    float* scale2;
    int64_t N, K;
    lqlora_config cfg;
} lqlora_qmatrix;

/* Storage cost in bits per parameter, Eq. (2) of Sec. 3.2: b0 + b1/B0 + b2/(B0*B1).  Pure host
 * arithmetic.  Returns a negative value if cfg is NULL or invalid. */
double lqlora_storage_bits_per_param(const lqlora_config* cfg);

/* Sizes in bytes of the three arrays of an [N, K] quantized matrix and of the scratch that
 * lqlora_encode needs.  Any output pointer may be NULL.  Host only.
 * When N % 128 == 0 the three sizes add up to exactly N*K*Eq.(2)/8 bytes (scale2 rounded up to
 * one fp32 per started group). */
int lqlora_packed_sizes(int64_t N, int64_t K, const lqlora_config* cfg, size_t* code_bytes,
                        size_t* scale_bytes, size_t* scale2_bytes, size_t* encode_workspace_bytes);

/* The NormalFloat code book of Sec. 2.2 for b0 bits: 2^b0 ascending fp32 values in [-1, 1]
 * (2^(b0-1) evenly spaced probabilities on [delta, 1/2], 2^(b0-1)+1 on [1/2, 1-delta],
 * delta = (1/30 + 1/32)/2, Gaussian quantiles divided by the largest).  out_host: host memory,
 * 2^b0 floats.  Host only. */
int lqlora_nf_codebook(int b0, float* out_host);

/*
 * Quantize(A, c) of Sec. 3.2 (Quantize-NF, then Quantize-INT of the block absmax values, then
 * cast to fp32) for A = W_dev, fp32 [N, K] row major, device memory.
 *   s_i  = max |u_j| over block i (B0 consecutive elements along K);
 *   c_j  = argmin_k |q~_k - fl32(u_j / s_i)|, the lower index on a tie; the code of 0 if s_i = 0;
 *   v_g  = max s_i over group g (B1 consecutive blocks; the last group may be short);
 *   s^_i = clamp(round_half_even(fl32(s_i / fl32(v_g / 127))), 0, 127); 0 if v_g = 0.
 * out->N, K, cfg must be filled in and its three arrays allocated by the caller.
 * With b1 < 8 the codes use the 2^(b1-1) - 1 levels of the b1-bit quantizer (127 above becomes that number); the
 * stored second-level scale is cast(v_g, b2), computed after the scale codes (which use the uncast v_g).
 * workspace_dev: device scratch of at least encode_workspace_bytes (block absmax values in fp32, and the unpacked
 * scales before packing when b1 < 8 or b2 is a 16-bit format).
 * Errors: INVALID_CONFIG, INVALID_SHAPE, NULL_POINTER, MISALIGNED, WORKSPACE_TOO_SMALL, CUDA.
 */
int lqlora_encode(const float* W_dev, lqlora_qmatrix* out, void* workspace_dev,
                  size_t workspace_bytes, void* stream);

/* Parity / debug exports (not on the hot path).
 * lqlora_unpack: one code per byte, codes_dev uint8 [N, K] row major (device).
 * lqlora_dequant: the inverse of lqlora_encode, step by step in reverse order (Sec. 3.2):
 *   s~_i = fl32(float(s^_i) * fl32(v_g / 127));  w~_j = fl32(q~[c_j] * s~_i)  -> deq32_dev fp32 [N, K];
 *   deq16_dev = w~ rounded to bf16, nearest-even, [N, K] (the cast for bf16 training, App. A).
 *   Either output may be NULL. */
int lqlora_unpack(const lqlora_qmatrix* q, uint8_t* codes_dev, void* stream);
int lqlora_dequant(const lqlora_qmatrix* q, float* deq32_dev, void* deq16_dev, void* stream);
/* The scales in plain form: scale_codes_dev uint8 [N*K/B0] (one code per byte), scale2_dev fp32 [ngrp] (the value each
 * stored second-level scale decodes to), whatever b1 and b2 are (Sec. 3.2: s^ and cast(v, b2)). */
int lqlora_unpack_scales(const lqlora_qmatrix* q, uint8_t* scale_codes_dev, float* scale2_dev, void* stream);

/* Bytes of device scratch lqlora_linear_fwd / lqlora_linear_bwd_input need for M rows.
 * Returns 0 (and sets *bytes) or an error.  Host only. */
int lqlora_linear_workspace_bytes(int64_t N, int64_t K, const lqlora_config* cfg, int r, int64_t M,
                                  size_t* bytes);

/*
 * Forward of the layer, X (Q + L1 L2) of Sec. 2.1 / Sec. 3.1 in nn.Linear orientation:
 *     Y[M, N] = X[M, K] deq16(Q)^T + bf16(X L2^T) L1^T
 * bf16 operands, fp32 accumulation, bf16 output; Q is dequantized on the fly and never written
 * to global memory.  r = 0 (L1 = L2 = NULL) computes the quantized part alone.
 * All of Q's arrays, L1, L2, X, Y, workspace_dev: device, 16-byte aligned.
 * The first 256 bytes of the workspace hold a status word (see lqlora_workspace_status); the rest
 * is scratch for the rank-r intermediate.  Concurrent calls must use different workspaces.
 * Errors: as lqlora_encode, plus UNSUPPORTED.
 */
int lqlora_linear_fwd(const lqlora_qmatrix* q, const void* L1_dev, const void* L2_dev, int r,
                      const void* X_dev, int64_t M, void* Y_dev, void* workspace_dev,
                      size_t workspace_bytes, void* stream);

/*
 * Input gradient of the same layer (only L1, L2 are trained, Q gets no gradient; Sec. 1, Sec. 2.1):
 *     dX[M, K] = dY[M, N] deq16(Q) + bf16(dY L1) L2
 * Same conventions as lqlora_linear_fwd.
 */
int lqlora_linear_bwd_input(const lqlora_qmatrix* q, const void* L1_dev, const void* L2_dev, int r,
                            const void* dY_dev, int64_t M, void* dX_dev, void* workspace_dev,
                            size_t workspace_bytes, void* stream);

/*
 * The layer with quantized factors (compression setting of Sec. 4.2: after training, L1 and L2 are themselves stored in
 * NF-8, i.e. Quantize with b0 = 8): qL1 is the [N, r] factor and qL2 the [r, K] factor as quantized matrices (any
 * configuration; r a multiple of 64 so that qL1's rows satisfy the K % 64 rule).  Computes what lqlora_linear_fwd /
 * lqlora_linear_bwd_input compute with L1 = deq16(qL1), L2 = deq16(qL2); the factors are dequantized to bf16 inside the
 * workspace (lqlora_linear_qfactors_workspace_bytes).  Errors as for lqlora_linear_fwd.
 */
int lqlora_linear_qfactors_workspace_bytes(int64_t N, int64_t K, const lqlora_config* cfg, int r, int64_t M, size_t* bytes);
int lqlora_linear_fwd_qfactors(const lqlora_qmatrix* q, const lqlora_qmatrix* qL1, const lqlora_qmatrix* qL2, const void* X_dev,
                               int64_t M, void* Y_dev, void* workspace_dev, size_t workspace_bytes, void* stream);
int lqlora_linear_bwd_input_qfactors(const lqlora_qmatrix* q, const lqlora_qmatrix* qL1, const lqlora_qmatrix* qL2,
                                     const void* dY_dev, int64_t M, void* dX_dev, void* workspace_dev, size_t workspace_bytes,
                                     void* stream);

/*
 * Gradients of the low-rank factors (the trained parameters: Sec. 1, Sec. 2.1; layer of Sec. 3.1).  With the layer
 * Y = X deq(Q)^T + (X L2^T) L1^T the chain rule gives
 *     dL1[N, r] = dY^T bf16(X L2^T)          dL2[r, K] = bf16(dY L1)^T X
 * (the rank-r intermediates are rounded to bf16 as in the forward pass and the input gradient; products and sums in
 * fp32 on the tensor cores).  The quantized matrix takes no part.
 *   L1_dev [N, r], L2_dev [r, K], X_dev [M, K], dY_dev [M, N] : bf16, row-major, device, read only
 *   dL1_dev [N, r], dL2_dev [r, K] : fp32, row-major, device, overwritten (not accumulated into)
 *   r : multiple of 16 in [16, 128];  N, K : multiples of 8;  1 <= M <= 2^24
 *   workspace_dev : device scratch of at least lqlora_lora_grads_workspace_bytes(N, K, r, M); it starts with the
 *                   same status word as a linear workspace (lqlora_workspace_status)
 * Asynchronous on `stream`; the library allocates nothing.
 * Errors: INVALID_SHAPE, NULL_POINTER, MISALIGNED (16-byte alignment), WORKSPACE_TOO_SMALL, CUDA.
 */
int lqlora_lora_grads_workspace_bytes(int64_t N, int64_t K, int r, int64_t M, size_t* bytes);
int lqlora_lora_grads(const void* L1_dev, const void* L2_dev, int r, int64_t N, int64_t K, const void* X_dev,
                      const void* dY_dev, int64_t M, float* dL1_dev, float* dL2_dev, void* workspace_dev,
                      size_t workspace_bytes, void* stream);

/*
 * The same gradients from the rank-r intermediates that the other two passes have already computed (the trained layer of
 * Sec. 2.1 runs forward, input gradient and factor gradients on the same X and dY): T = bf16(X L2^T) is what
 * lqlora_linear_fwd leaves in its workspace, T' = bf16(dY L1) what lqlora_linear_bwd_input leaves in its own, each at the
 * byte offset lqlora_linear_intermediate_offset reports for that call's (N, K, cfg, r, M, direction), as [M, r] bf16
 * row-major, valid until that workspace is used again.  X and dY are then read once instead of twice.
 *   T_dev, Tp_dev [M, r] : bf16, device, 16-byte aligned, read only;  the other arguments as for lqlora_lora_grads
 *   workspace_dev : at least 256 bytes (the status word only); it must not be one of the workspaces that hold T or T'
 * Asynchronous on `stream`; the library allocates nothing.  Errors as for lqlora_lora_grads.
 */
int lqlora_linear_intermediate_offset(int64_t N, int64_t K, const lqlora_config* cfg, int r, int64_t M, int backward,
                                      size_t* offset);
int lqlora_lora_grads_from(const void* T_dev, const void* Tp_dev, int r, int64_t N, int64_t K, const void* X_dev,
                           const void* dY_dev, int64_t M, float* dL1_dev, float* dL2_dev, void* workspace_dev,
                           size_t workspace_bytes, void* stream);

/*
 * The low-rank plus quantized decomposition of Sec. 3.1 (Eq. (1)-(2), Algorithm 2), with Factorize of Sec. 3.3
 * (Eq. (4), Algorithm 4), in nn.Linear orientation:  W [N, K] ~ deq(Q) + L1 [N, r] L2 [r, K].
 *     Q <- 0;  repeat  L1, L2 <- Factorize(W - Q, F, r);  Q <- Quantize(W - L1 L2, c);  e_t <- error
 *     until e_t > e_(t-1) or max_steps steps are done.
 * error = || W - (Q + L1 L2) ||_F, or || sqrt(F) o (W - (Q + L1 L2)) ||_F when F is given (Eq. (3)); with F, Factorize
 * takes the SVD of D_row A D_col (D_row, D_col = row / column means of sqrt(F)) and divides the factors by D_row, D_col.
 * Factorize is a randomized SVD (footnote to Eq. (2)): range finder with the caller's test matrix Omega, `power_iters`
 * power iterations, exact SVD of the projected (r + oversample) x K matrix; L1 = U sqrt(S), L2 = sqrt(S) V^T.
 * The iterate before the error rose is returned (Sec. 3.1: the algorithm terminates if the error increases).
 *   W_dev, F_dev (may be NULL) : fp32 [N, K], device, read only
 *   out                        : N, K, cfg filled in and the three arrays allocated by the caller (as for lqlora_encode)
 *   L1_dev [N, r], L2_dev [r, K] : fp32, device, written
 *   omega_dev                  : fp32 [K, r + oversample] standard-normal entries, device (the random numbers of the
 *                                method are an input); 1 <= r <= 128, 0 <= oversample <= 64
 *   errors_host [max_steps], steps_taken : host memory; errors_host[t] = e_(t+1) for the steps that ran (the last one
 *                                is the rejected step when the loop ended on a rise)
 *   workspace_dev              : at least lqlora_lq_workspace_bytes (two fp32 copies of the matrix and the factors)
 * Synchronous: the stopping rule needs the error of every step on the host; the small (r + oversample)^2
 * factorizations run on the host between the launches.  Preparation work, not the layer's hot path.
 * Errors: INVALID_CONFIG, INVALID_SHAPE, NULL_POINTER, MISALIGNED, WORKSPACE_TOO_SMALL, CUDA.
 */
int lqlora_lq_workspace_bytes(int64_t N, int64_t K, const lqlora_config* cfg, int r, int oversample, size_t* bytes);
int lqlora_lq_decompose(const float* W_dev, const float* F_dev, lqlora_qmatrix* out, float* L1_dev, float* L2_dev, int r,
                        int max_steps, const float* omega_dev, int oversample, int power_iters, double* errors_host,
                        int* steps_taken, void* workspace_dev, size_t workspace_bytes, void* stream);
/* y = bf16(x), n elements, device (the trained factors are kept in bf16 by the layer: Sec. 4, App. A). */
int lqlora_to_bf16(const float* x_dev, void* y_dev, int64_t n, void* stream);

/*
 * The budgeted assignment of Sec. 3.2 (Algorithm 3, ILPSolve): errors[i * n_configs + c] = error(A_i, c)^2 and
 * storage[i * n_configs + c] = storage(A_i, c) (Eq. (2) times the matrix size); picks one configuration per matrix so
 * that the summed storage is <= budget and the summed error is minimal.  Exact dynamic programming over the Pareto
 * frontier of (storage, error) prefixes (thinned beyond 32768 points).  Host only.  assignment: [n_matrices];
 * total_error / total_storage may be NULL.  Returns LQLORA_ERR_UNSUPPORTED when no assignment fits the budget.
 */
int lqlora_assign_configs(const double* errors, const double* storage, int n_matrices, int n_configs, double budget,
                          int* assignment, double* total_error, double* total_storage);

/*
 * Forward pass for callers that are not allowed to allocate device memory (no counterpart in the
 * paper: this entry point exists for deployment reasons only).  Typical examples are an inference
 * server whose memory pool was carved up at start-up, or code running inside another framework's
 * stream callback or plug-in hook, where calling cudaMalloc (directly or through a tensor library)
 * is forbidden or would synchronize the device.  The call computes exactly what lqlora_linear_fwd
 * computes, with the same kernels, but takes its scratch from an 8 MiB array that is compiled into
 * the library (lqlora_static_scratch_bytes() returns the size).  The caller passes only the
 * inputs and the output; the function itself never allocates or frees anything.
 *   - A problem whose scratch (lqlora_linear_workspace_bytes) exceeds the array is refused with
 *     LQLORA_ERR_WORKSPACE_TOO_SMALL before anything is enqueued; use lqlora_linear_fwd then.
 *   - Every device that loads the library carries the array until the process ends.
 *   - The first call on a device looks up the array's device address (a one-off set-up step);
 *     make that first call outside any stream capture.
 *   - All calls share the one array.  It still holds the previous call's data when the next call
 *     starts; the one word that has to start at zero (the status word) is cleared on the stream by
 *     each call.  Two calls whose kernels can overlap on the GPU (different streams without ordering
 *     between them) would race on it: order them, or use lqlora_linear_fwd with separate workspaces.
 *   - lqlora_static_scratch_status(stream) is lqlora_workspace_status for this array: it synchronizes
 *     `stream` and returns LQLORA_OK, or LQLORA_ERR_TIMEOUT if a kernel of the last call on the current
 *     device gave up on a bounded wait.  It allocates nothing either.
 * Other arguments, layouts and error codes as for lqlora_linear_fwd.
 */
size_t lqlora_static_scratch_bytes(void);
int lqlora_linear_fwd_static(const lqlora_qmatrix* q, const void* L1_dev, const void* L2_dev, int r,
                             const void* X_dev, int64_t M, void* Y_dev, void* stream);
int lqlora_static_scratch_status(void* stream);

/*
 * Host-buffer variants (end-to-end use: activations arrive from and results return to pinned host
 * memory).  They enqueue, on `stream`: a host-to-device copy of the input into the caller's device
 * staging buffer, the same kernels as the device-pointer entry points (Sec. 2.1, Sec. 3.2 as
 * above), and a device-to-host copy of the result.  Nothing is allocated; the quantized matrix
 * and L1, L2 stay on the device.
 *   X_host / dY_host / W_host : host memory (pinned for asynchronous copies), read only
 *   Y_host / dX_host          : host memory, written when the stream reaches the copy
 *   *_stage_dev               : device scratch of the same size as the matching host buffer
 * Errors as for the device-pointer entry points.
 */
int lqlora_encode_host(const float* W_host, float* W_stage_dev, lqlora_qmatrix* out, void* workspace_dev,
                       size_t workspace_bytes, void* stream);
int lqlora_linear_fwd_host(const lqlora_qmatrix* q, const void* L1_dev, const void* L2_dev, int r,
                           const void* X_host, int64_t M, void* Y_host, void* X_stage_dev, void* Y_stage_dev,
                           void* workspace_dev, size_t workspace_bytes, void* stream);
int lqlora_linear_bwd_input_host(const lqlora_qmatrix* q, const void* L1_dev, const void* L2_dev, int r,
                                 const void* dY_host, int64_t M, void* dX_host, void* dY_stage_dev,
                                 void* dX_stage_dev, void* workspace_dev, size_t workspace_bytes, void* stream);

/* Synchronizes `stream`, reads the status word at the start of a linear workspace and returns it
 * as an lqlora_status: LQLORA_OK, or LQLORA_ERR_TIMEOUT if a kernel gave up on a bounded wait
 * (its output is then undefined).  The word is cleared by every linear call before it launches. */
int lqlora_workspace_status(const void* workspace_dev, void* stream);

/* Self-test of the bounded device-side waits: enqueues a one-CTA kernel that holds a tensor-memory allocation and waits,
 * with the helper and status word the linear kernels use, on an mbarrier armed for bytes that nothing delivers.  After
 * budget_cycles SM clocks (1e3 .. 2e9) the wait is abandoned: the kernel records the time-out in the status word at the
 * head of workspace_dev (at least 256 bytes), frees its tensor memory and returns, so lqlora_workspace_status then
 * reports LQLORA_ERR_TIMEOUT while the context stays usable.  Nothing traps, faults or spins without bound. */
int lqlora_selftest_bounded_wait(void* workspace_dev, int64_t budget_cycles, void* stream);

/* Which kernel lqlora_linear_fwd (backward = 0) or lqlora_linear_bwd_input (backward != 0) dispatches to for M rows:
 *   LQLORA_PATH_PLAIN    plain-FMA fall-back (shapes the vector paths do not take)
 *   LQLORA_PATH_STREAM   weight-streaming kernel for decode-sized inputs (M <= 16)
 *   LQLORA_PATH_TC_ONE   tcgen05 kernel, one CTA per output tile, contraction split over a cluster
 *   LQLORA_PATH_TC_PAIR  tcgen05 kernel, CTA pairs (cta_group::2) on [512, 256] output tiles
 * *splits (may be NULL) receives the number of CTAs that share one output tile's contraction (the cluster size; 1 for
 * CTA pairs and the fall-back).  Returns a negative lqlora_status for invalid arguments.  Host only. */
enum { LQLORA_PATH_PLAIN = 0, LQLORA_PATH_STREAM = 1, LQLORA_PATH_TC_ONE = 2, LQLORA_PATH_TC_PAIR = 3 };
int lqlora_linear_path(int64_t N, int64_t K, const lqlora_config* cfg, int r, int64_t M, int backward, int* splits);

/* lqlora_encode finds the nearest code (Sec. 2.2: c_j = argmin_k |q~_k - u_j / s_i|) with a bin table over [-1, 1]:
 * every bin holds at most one decision threshold (the midpoint of two neighbouring code-book entries), and inputs
 * closer than 1e-6 to a threshold are decided with the exact IEEE quotient.  This returns the smallest distance
 * between a threshold and a bin edge for the b0-bit table; it must exceed that 1e-6 by a wide margin for the
 * fast and the exact route to agree (checked by the host tests).  Negative for an invalid b0.  Host only. */
double lqlora_encode_search_clearance(int b0);

/* Number of kernel launches the library has enqueued since it was loaded (for launch accounting). */
int64_t lqlora_launch_count(void);

const char* lqlora_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* LQLORA_H_ */
