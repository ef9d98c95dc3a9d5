/*
 * bwla.h - C ABI of the BWLA W1AX linear layer for NVIDIA B200 (sm_100a).
 *
 * The layer (assembled from the paper's weight format Eq. 1-4, the Orthogonal-Kronecker
 * Transformation of Sec. 3.1, the PSP residual of Sec. 3.2 and the per-token activation
 * quantisation of Sec. 4.1), per token x_t in R^K:
 *
 *   Y_t   = P1^T * reshape(x_t, n1 x n2) * P2               (OKT applied online, K = n1*n2)
 *   s_t   = max|Y_t| / qmax,  q_t = clamp(rne(Y_t / s_t))    (symmetric INT-b, qmax = 2^(b-1) - 1)
 *   acc   = sum_k sign(W')[n][k] * q_t[k]                    (1-bit weights, exact int32)
 *   out   = bf16( alpha[n] * s_t * acc + U[n,:] . (V x_t) [+ mu[n] * s_t * sum_k q_t[k]] )
 *
 * General rules for every entry point
 *   - All data pointers are DEVICE pointers owned by the caller.  The library never allocates,
 *     frees or keeps them.  `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *   - Calls are asynchronous on `stream`; nothing synchronises the host except bwla_check_status.
 *   - Matrices are row-major.  bf16 data is passed as void* to 16-bit elements.
 *   - Return value: BWLA_OK or a negative error code.  Invalid arguments never launch anything.
 *   - There is no CPU fallback: on a machine without an sm_100 device the compute entry points
 *     return BWLA_ERR_UNSUPPORTED.
 *   - Packed sign format: uint32 words, row-major [N][K/32]; weight k of output row n is bit
 *     (k & 31) of word (k >> 5); bit 1 means +1, bit 0 means -1.  Sign(w) = +1 iff w > 0 (Eq. 3),
 *     so 0, -0.0 and NaN pack as -1.
 */
#ifndef BWLA_H_
#define BWLA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    BWLA_OK = 0,
    BWLA_ERR_INVALID_ARG = -1,     /* NULL pointer, bad dimension, K != n1*n2, K % 32 != 0, bits not in {4,6,8}, ... */
    BWLA_ERR_UNSUPPORTED = -2,     /* no sm_100 device is current */
    BWLA_ERR_WORKSPACE = -3,       /* workspace NULL, misaligned (256 B) or smaller than bwla_workspace_bytes */
    BWLA_ERR_CUDA = -4,            /* a CUDA call failed; see bwla_last_cuda_error */
    BWLA_ERR_DEVICE_TIMEOUT = -5,  /* a bounded device-side wait ran out (only from bwla_check_status) */
    BWLA_ERR_STATIC_SCRATCH = -6   /* bwla_w1ax_linear_static: the problem needs more scratch than the built-in array holds */
};

/* Kernel families the layer can run its contraction on (see bwla_force_path). */
enum {
    BWLA_PATH_AUTO = 0,       /* per-shape choice from measurement: I8 wherever it can run; up to four tokens of a shape
                                 it cannot take go to BITPLANE, the rest to SIMPLE */
    BWLA_PATH_SIMPLE = 1,     /* one-warp-per-output-row CUDA kernel: slow, the on-device cross-check and the path of
                                 shapes the other two do not take */
    BWLA_PATH_BITPLANE = 2,   /* up to four tokens: two's-complement bit-planes of the codes against the packed sign
                                 words with and + popc on the integer pipes; the weights are never expanded */
    BWLA_PATH_I8 = 3          /* sign words expanded to int8 in tensor memory, tcgen05 kind::i8 with int32 accumulators
                                 in tensor memory; needs K % 128 == 0 and r <= 64 */
};

#define BWLA_DTYPE_F32 0
#define BWLA_DTYPE_BF16 1

/*
 * Binarise already rotated/centred weights: packed[n][k>>5] bit (k&31) = (W'[n][k] > 0).   (Eq. 2-3)
 *   w      device, [N][ldw] fp32 (dtype 0) or bf16 (dtype 1), ldw >= K elements
 *   packed device, uint32 [N][K/32], written in full
 *   K must be a positive multiple of 32; N >= 0 (N == 0 is a no-op).
 */
int bwla_pack_signs(const void* w, int dtype, int64_t N, int64_t K, int64_t ldw,
                    uint32_t* packed, void* stream);

/*
 * Final binarisation in the rotated coordinates, offline, once per layer.   (Alg. 2, last step; Eq. 1-3)
 * Every row of W_res = W - M (the weights less the PSP low-rank part) goes through the same map as an activation row,
 * X_n = flatten(P1^T reshape(w_n, n1 x n2) P2); then mu[n] = mean_k X[n][k], alpha[n] = mean_k |X[n][k] - mu[n]|,
 * packed bit (n, k) = (X[n][k] - mu[n] > 0).  The outputs are what bwla_w1ax_linear / bwla_layer_create take.
 *   w_res  device, [N][ldw] fp32 (dtype 0) or bf16 (dtype 1), ldw >= K
 *   P1, P2 device, fp32, 16-byte aligned; n1*n2 == K, K a positive multiple of 32
 *   packed device, uint32 [N][K/32]; alpha, mu device, fp32 [N]; all written in full
 *   workspace: 256-byte aligned device scratch of bwla_binarize_workspace_bytes(K) bytes (0 for an invalid K); the call
 *     clears its status words itself.
 * The rotation runs on the tensor-core kernel (fp32 rows as three bf16 terms, three passes); its error is below 1e-6 of
 * a row's largest rotated magnitude, so a sign can differ from the exact one only where |X - mu| is below that.
 * Factor sizes that kernel does not take (n2 % 8 != 0, n2 > 256, n1 > 192) return BWLA_ERR_UNSUPPORTED.
 * N == 0 is a no-op.  Asynchronous on `stream`; bwla_check_status(workspace, stream) reports a device-side timeout.
 */
size_t bwla_binarize_workspace_bytes(int64_t K);
int bwla_binarize_rows(const void* w_res, int dtype, int64_t N, int64_t K, int64_t ldw, const float* P1, int n1,
                       const float* P2, int n2, uint32_t* packed, float* alpha, float* mu, void* workspace,
                       size_t workspace_bytes, void* stream);

/*
 * Online OKT + per-token symmetric quantisation.   (Sec. 3.1 Kronecker evaluation; Sec. 4.1 per-token)
 *   x_bf16 device, bf16 [M][ldx], ldx >= K
 *   P1     device, fp32 [n1][n1];  P2 device, fp32 [n2][n2];  n1*n2 == K
 *   bits   4, 6 or 8;  qmax = 2^(bits-1) - 1; the most negative code is never produced
 *   codes  device, int8 [M][K];  scales device, fp32 [M]   (both written in full)
 * Arithmetic: fp32 accumulation; s_t = amax / qmax; q = rne(Y * (qmax / amax)); an all-zero row
 * gives s_t = 1 and zero codes.  M == 0 is a no-op.  K must be a multiple of 32, K <= 65536 and
 * 8*K bytes of shared memory must fit one block (K <= 25600 elements).
 */
int bwla_rotate_quant_act(const void* x_bf16, int64_t M, int64_t K, int64_t ldx,
                          const float* P1, int n1, const float* P2, int n2, int bits,
                          int8_t* codes, float* scales, void* stream);

/*
 * Bytes of scratch bwla_w1ax_linear / bwla_w1a_gemm_codes need for this problem (a multiple of 256).
 * Returns 0 for invalid dimensions.
 */
size_t bwla_workspace_bytes(int64_t M, int64_t K, int64_t N, int r, int bits);

/*
 * The whole layer (formula at the top of this file).
 *   packed device uint32 [N][K/32];  alpha device fp32 [N];  mu device fp32 [N] or NULL   (Eq. 4)
 *   U_bf16 device bf16 [N][r], V_bf16 device bf16 [r][K]; both may be NULL iff r == 0      (Sec. 3.2, M = A B)
 *   out_bf16 device bf16 [M][ldo], ldo >= N
 *   workspace device, 256-byte aligned, >= bwla_workspace_bytes(M,K,N,r,bits); contents are scratch, except that
 *     its first 256 bytes must be zero before the first call that uses it.  The first word is a status word that
 *     bounded device-side waits set and that stays set (later calls on this workspace then skip their work) until
 *     bwla_check_status reads and clears it; a few of the following words are arrival counters that every call
 *     leaves at zero.
 *   Two calls that share a workspace must be ordered on one stream.
 *   The kernels are launched with programmatic stream serialisation: the part of a call that depends only on the
 *   layer's constants (streaming the sign words, fetching P1, P2 and V) may overlap the tail of the preceding kernel
 *   of `stream`; x is read and every global store is made only after that kernel has finished, so a call may consume
 *   what the preceding call of the stream produced.
 */
int bwla_w1ax_linear(const void* x_bf16, int64_t M, int64_t K, int64_t ldx,
                     const float* P1, int n1, const float* P2, int n2, int bits,
                     const uint32_t* packed, const float* alpha, const float* mu,
                     const void* U_bf16, const void* V_bf16, int r,
                     void* out_bf16, int64_t N, int64_t ldo,
                     void* workspace, size_t workspace_bytes, void* stream);

/*
 * The whole layer without a workspace argument, for callers that cannot allocate.  (The paper has no counterpart:
 * it describes no kernels and no memory management; this entry point exists for integration only.)
 *
 * Who needs it: code that is handed its input and output tensors and nothing else -- a plug-in or custom-op slot
 * of a host framework, a stage that runs after the framework has frozen its memory pool, a serving process that
 * may not call cudaMalloc once traffic flows.  Such a caller cannot supply the scratch buffer bwla_w1ax_linear
 * wants, so here the scratch is a fixed array of BWLA_STATIC_SCRATCH_BYTES inside the library's device image.
 * Every GPU that loads the library holds that array until the process exits.
 *
 * Arguments, layouts and results are those of bwla_w1ax_linear (same kernels, same arithmetic); the workspace
 * pair is gone.  The call allocates and frees nothing, through CUDA or any other library.
 *   - Limit: bwla_workspace_bytes(M,K,N,r,bits) must not exceed BWLA_STATIC_SCRATCH_BYTES (4 MiB: e.g. 64 tokens
 *     at K = 25600, or 512 tokens at K = 5120).  Larger problems return BWLA_ERR_STATIC_SCRATCH and launch nothing.
 *   - The first call on each device looks up the array's device address (a host-side runtime query).  Make that
 *     first call outside any stream capture.
 *   - All calls on a device share the one array, and it keeps what the last call left in it.  The entry point
 *     clears the status words itself at the start of every call; nothing else needs to start at zero.  Two calls
 *     that may overlap on the GPU (different streams, or the same stream from two host threads without ordering)
 *     race on the array and give wrong results: order them.
 *   - The status word of the built-in array is not exposed: a device-side wait that runs out leaves this call's
 *     outputs invalid and the next call starts clean.  Use bwla_w1ax_linear with bwla_check_status where that
 *     must be observed.
 */
#define BWLA_STATIC_SCRATCH_BYTES (4 * 1024 * 1024)
int bwla_w1ax_linear_static(const void* x_bf16, int64_t M, int64_t K, int64_t ldx,
                            const float* P1, int n1, const float* P2, int n2, int bits,
                            const uint32_t* packed, const float* alpha, const float* mu,
                            const void* U_bf16, const void* V_bf16, int r,
                            void* out_bf16, int64_t N, int64_t ldo, void* stream);

/*
 * ---- Prepared layers ------------------------------------------------------------------------------------------
 * A layer's constants can be put once into the form the kernels read, instead of on every call: the Kronecker
 * factors P1, P2 (Sec. 3.1) split into bf16 terms and laid out as tensor-core operands.  A bwla_layer is a small
 * host object that remembers the layer's device pointers (it copies nothing and owns no device memory: the caller
 * keeps P1 ... V and the `prepared` buffer alive and unchanged until bwla_layer_destroy) and the launch plan.
 * Calls through a prepared layer compute exactly what bwla_w1ax_linear computes.
 *
 *   bwla_layer_prepared_bytes  device bytes `prepared` must have for these sizes (a multiple of 256; never 0 for
 *                              valid sizes)
 *   bwla_layer_create          checks the arguments as bwla_w1ax_linear does, launches the preparation on `stream`
 *                              and returns the handle in *layer (host memory from malloc).  `prepared` must be
 *                              256-byte aligned.
 *   bwla_layer_destroy         frees the host object only.
 */
typedef struct bwla_layer bwla_layer;
size_t bwla_layer_prepared_bytes(int64_t K, int64_t N, int n1, int n2, int r);
int bwla_layer_create(bwla_layer** layer, int64_t K, int64_t N, const float* P1, int n1, const float* P2, int n2,
                      int bits, const uint32_t* packed, const float* alpha, const float* mu,
                      const void* U_bf16, const void* V_bf16, int r,
                      void* prepared, size_t prepared_bytes, void* stream);
void bwla_layer_destroy(bwla_layer* layer);

/*
 * Online OKT + per-token quantiser of a prepared layer (what bwla_rotate_quant_act computes; Sec. 3.1, Sec. 4.1).
 *   codes device int8 [M][K] (natural k order), scales device fp32 [M]
 *   y_f32 device fp32 [M][K] or NULL: receives the rotated activations Y_t before the quantiser
 */
int bwla_layer_rotate_quant(const bwla_layer* layer, const void* x_bf16, int64_t M, int64_t ldx,
                            int8_t* codes, float* scales, float* y_f32, void* stream);

/*
 * Activation quantiser of a prepared layer.  BWLA_ACT_SYMMETRIC (the default): codes in [-qmax, qmax] and one scale per
 * token.  BWLA_ACT_ASYMMETRIC: the paper's stated setting (Sec. 4.1, "per-token asymmetric quantization for
 * activations"): lo = min(0, min y), hi = max(0, max y), scale = (hi - lo) / (2^b - 1), an integer zero point
 * z = rne(-lo / scale), codes u = clamp(rne(y / scale) + z, 0, 2^b - 1); the layer then computes
 *   out = bf16( alpha[n] * s_t * (sum_k sign[n][k] * u_k - z_t * rowsum[n]) + U (V x_t) [+ mu[n] * s_t * sum_k (u_k - z_t)] ),
 * rowsum[n] = sum_k sign[n][k] (prepared once per layer).  Returns BWLA_ERR_UNSUPPORTED for factor sizes only the
 * fallback rotation kernel takes.
 */
enum { BWLA_ACT_SYMMETRIC = 0, BWLA_ACT_ASYMMETRIC = 1 };
int bwla_layer_set_activation_quant(bwla_layer* layer, int mode);

/*
 * The weight-only operating point, W1A16 (Table 1, upper half: binarised weights, 16-bit activations), on a prepared
 * layer: the rotated activation Y = P1^T X P2 (Sec. 3.1) is rounded to bf16 instead of being quantised to integer codes,
 *   out[t][n] = bf16( alpha[n] * sum_k sign[n][k] * bf16(Y[t][k]) + U (V x_t) [+ mu[n] * sum_k bf16(Y[t][k])] ),
 * a bf16 contraction on the tensor cores with fp32 accumulation (partial sums of 128 values of k are added in rounded
 * fp32).  The layer's activation bit width and quantiser mode are not used.
 *   x_bf16 device, bf16 [M][ldx], 16-byte aligned, ldx >= K and a multiple of 8; out_bf16 device, bf16 [M][ldo], ldo >= N
 *   workspace: 256-byte aligned device scratch of bwla_w1a16_workspace_bytes(layer, M) bytes (about 7 bytes per
 *     activation value); its first 256 bytes must be zero before the first call; bwla_check_status reads it.
 * Needs K % 64 == 0, r <= 64 and factor sizes the tensor-core rotation takes, else BWLA_ERR_UNSUPPORTED.  M == 0 is a
 * no-op.  Asynchronous on `stream`.
 */
size_t bwla_w1a16_workspace_bytes(const bwla_layer* layer, int64_t M);
int bwla_layer_w1a16_linear(const bwla_layer* layer, const void* x_bf16, int64_t M, int64_t ldx, void* out_bf16,
                            int64_t ldo, void* workspace, size_t workspace_bytes, void* stream);

/* The asymmetric quantiser alone: codes device uint8 [M][K] (u), scales device fp32 [M], zeros device int32 [M] (z),
 * y_f32 device fp32 [M][K] or NULL. */
int bwla_layer_rotate_quant_asym(const bwla_layer* layer, const void* x_bf16, int64_t M, int64_t ldx,
                                 uint8_t* codes, float* scales, int32_t* zeros, float* y_f32, void* stream);

/*
 * Several layers that read the same activations (q, k, v of an attention block; gate and up of an MLP) in one
 * call: x is rotated and quantised for every layer (each has its own P1, P2) by one launch, and the contractions
 * follow.  All layers must have the same K, n1, n2 and bits; count <= 4.
 *   outs  host array of `count` device pointers, bf16 [M][ldos[i]];  ldos host array, ldos[i] >= N_i
 *   workspace: 256-byte aligned device scratch of bwla_group_workspace_bytes; its first 256 bytes must be zero
 *   before the first call (status words, as for bwla_w1ax_linear; bwla_check_status applies to it)
 */
size_t bwla_group_workspace_bytes(const bwla_layer* const* layers, int count, int64_t M);
int bwla_w1ax_linear_group(const bwla_layer* const* layers, int count, const void* x_bf16, int64_t M, int64_t ldx,
                           void* const* outs, const int64_t* ldos, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Contraction + epilogue from given codes (the part of the layer after the quantiser), so that
 * integer accumulators can be compared for identical codes.
 *   codes device int8 [M][K]; scales device fp32 [M]
 *   x_bf16 (with ldx) is only read for the low-rank branch and may be NULL iff r == 0
 *   out_bf16 may be NULL when only accumulators are wanted
 *   acc_debug device int32 [M][N] or NULL: receives sum_k sign[n][k] * codes[t][k]
 */
int bwla_w1a_gemm_codes(const int8_t* codes, const float* scales, int64_t M, int64_t K, int bits,
                        const uint32_t* packed, const float* alpha, const float* mu,
                        const void* x_bf16, int64_t ldx,
                        const void* U_bf16, const void* V_bf16, int r,
                        void* out_bf16, int64_t N, int64_t ldo, int32_t* acc_debug,
                        void* workspace, size_t workspace_bytes, void* stream);

/*
 * Synchronise `stream`, read the workspace status word and clear it.
 * Returns BWLA_OK, BWLA_ERR_DEVICE_TIMEOUT (a device-side wait gave up; outputs of that call are
 * invalid but the context stays usable) or BWLA_ERR_CUDA.
 */
int bwla_check_status(void* workspace, void* stream);

/*
 * Where bwla_w1ax_linear keeps an intermediate inside its workspace, so that tests can compare the quantiser's
 * output of the fused call itself (Sec. 4.1) and not only that of bwla_rotate_quant_act.  No launch.
 *   which: BWLA_WS_SCALES  fp32 [M]                        per-token scale s_t
 *          BWLA_WS_QSUM    int32 [M][8]                    partial code sums; sum_k q_t[k] is the sum of the eight
 *          BWLA_WS_T       bf16 [3][M][max(64, r)]         T = V x as hi + mid + lo
 *          BWLA_WS_CODES   int8 [M][K]                     codes; on the tensor-core path inside each group of 32
 *                                                          consecutive k, byte 4*j + i holds k = j + 8*i
 *          BWLA_WS_ZEROS   int32 [M]                       asymmetric quantiser only: zero points; codes and zero
 *                                                          points are both kept minus 2^(b-1) so that codes fit int8
 *   offset, bytes: host pointers that receive the section's position and size.
 * Returns BWLA_ERR_INVALID_ARG for invalid dimensions or an unknown section.
 */
enum { BWLA_WS_SCALES = 0, BWLA_WS_QSUM = 1, BWLA_WS_T = 2, BWLA_WS_CODES = 3, BWLA_WS_ZEROS = 4 };
int bwla_workspace_section(int64_t M, int64_t K, int64_t N, int r, int bits, int which, size_t* offset, size_t* bytes);

/* Force every later call of the calling thread onto one kernel family (benchmarking the non-chosen path,
 * cross-checks); the setting is per thread.  Returns BWLA_ERR_INVALID_ARG for an unknown value. */
int bwla_force_path(int path);

/* The same for the kernel that evaluates the online OKT + quantiser: BWLA_ROT_AUTO (per shape), BWLA_ROT_SIMT (the
 * kernel with fp32 FMA tiles, P1/P2 staged in shared memory and warp-shuffle reductions; takes every shape) or
 * BWLA_ROT_UMMA (the tcgen05 kernel; shapes it does not take still go to the other one). */
enum { BWLA_ROT_AUTO = 0, BWLA_ROT_SIMT = 1, BWLA_ROT_UMMA = 2 };
int bwla_force_rotation(int which);

/* The family BWLA_PATH_AUTO resolves to for this problem (no launch). */
int bwla_chosen_path(int64_t M, int64_t K, int64_t N, int r, int bits);

/* Number of kernels the most recent bwla_w1ax_linear / bwla_w1a_gemm_codes / bwla_rotate_quant_act /
 * bwla_pack_signs call on this thread launched. */
int bwla_last_launch_count(void);

/*
 * Per-kernel timing for benchmarks.  While enabled (per calling thread), every kernel the library launches is
 * bracketed by CUDA events recorded on the launching stream and launched without programmatic overlap, so that an
 * event pair times one kernel alone.  bwla_profile_collect waits for them, adds the
 * elapsed milliseconds and launch counts per kernel kind into two caller arrays of 8 entries
 * (0 prologue: rotate + quantise + V x, 2 contraction with its fused epilogue, 4 code preparation, 5 pack_signs;
 * the other entries stay zero)
 * and forgets the events.  Host arrays.  Do not enable during stream capture.
 */
int bwla_profile_enable(int on);
int bwla_profile_collect(float* ms_by_kind, int* launches_by_kind);

/* cudaError_t of the most recent failing CUDA call on this thread (0 if none). */
int bwla_last_cuda_error(void);

/* Static, human-readable name of a status code. */
const char* bwla_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* BWLA_H_ */
