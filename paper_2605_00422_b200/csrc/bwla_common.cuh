// Shared declarations of the CUDA library: status handling, workspace layout, kernel launchers.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <algorithm>

#include "bwla.h"

namespace bwla {

// ---------------------------------------------------------------------------------------------
// per-thread bookkeeping (the library keeps no process-global mutable state)
// ---------------------------------------------------------------------------------------------
extern thread_local int g_last_cuda_error;
extern thread_local int g_launch_count;

inline int cuda_fail(cudaError_t e) {
    g_last_cuda_error = (int)e;
    return BWLA_ERR_CUDA;
}

#define BWLA_CUDA_TRY(expr)                                   \
    do {                                                      \
        cudaError_t e__ = (expr);                             \
        if (e__ != cudaSuccess) return ::bwla::cuda_fail(e__); \
    } while (0)

// Checks the launch that has just been issued and counts it.
inline int after_launch() {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e);
    ++g_launch_count;
    return BWLA_OK;
}

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Number of SMs of the current device (cached per thread and device); 0 if it cannot be queried.
inline int sm_count() {
    static thread_local int cached_dev = -1, cached_n = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return 0; }
    if (dev != cached_dev) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) { cudaGetLastError(); return 0; }
        cached_dev = dev; cached_n = n;
    }
    return cached_n;
}

// ---------------------------------------------------------------------------------------------
// optional per-kernel timing (bwla_profile_enable / bwla_profile_collect): CUDA events recorded on the launching
// stream right around each kernel launch, summed per kernel kind.  Off by default; not usable under stream capture.
// ---------------------------------------------------------------------------------------------
enum ProfKind { kProfRotateQuant = 0, kProfContraction = 2, kProfPrepare = 4,
                kProfPack = 5, kProfKinds = 8 };
// 1 unless per-kernel timing is on: timed kernels are launched fully serialised so that each event pair brackets
// one kernel alone.
unsigned launch_overlap_allowed();
void prof_begin(int kind, cudaStream_t stream);
void prof_end(int kind, cudaStream_t stream);
struct ProfScope {
    int kind; cudaStream_t stream;
    ProfScope(int k, cudaStream_t s) : kind(k), stream(s) { prof_begin(kind, stream); }
    ~ProfScope() { prof_end(kind, stream); }
};

// ---------------------------------------------------------------------------------------------
// workspace layout (byte offsets into the caller's scratch buffer; every section 256-byte aligned)
// ---------------------------------------------------------------------------------------------
constexpr int kStatusBytes = 256;        // word 0: status; words 1..: where a bounded wait gave up
constexpr int kLowrankPad = 64;          // T is kept as bf16 [3][M][64] (T = hi + mid + lo), zero beyond r <= 64

// The code sum of a token is kept as kQsumParts partial sums (one per CTA of the prologue cluster that quantised a slab
// of the token; unused parts are zero): the consumer adds them, the producers need no exchange.
constexpr int kQsumParts = 8;

// With few tokens and a large K the rows of V are read by several blocks that each take a part of K; their partial sums
// of T meet in the workspace and the last block to arrive adds them in a fixed order (counters: status words 4..11).
constexpr int kLrKSplitMax = 8;
constexpr int kLrCounterWord = 4;

__host__ __device__ inline int lowrank_cols(int r) { return r > kLowrankPad ? (r + 1) / 2 * 2 : kLowrankPad; }

// T = V x for many tokens on the tensor cores (lowrank_umma.cu): whether it takes the problem, the bytes of partial sums
// it needs in the workspace (0: none), and the launch for the problems of one group (all share x, M, K; every entry of
// `lowrank` has V, Thl and, where partial sums are needed, lr_part set).
struct OktLowrank;
bool lowrank_umma_supports(int64_t M, int64_t K, int r);
size_t lowrank_umma_part_bytes(int64_t M, int64_t K, int r);
int launch_lowrank_umma(const void* x, int64_t M, int64_t K, int64_t ldx, int n_problems, const OktLowrank* lowrank,
                        uint32_t* status, cudaStream_t stream);

struct Workspace {
    size_t status, scales, zp, qsum, T, lr_part, codes, prep, total;
};

// Room for the prepared Kronecker factors of one call (bf16 terms of P2^T and P1^T for the largest factor sizes the
// tensor-core rotation takes): calls that are handed raw P1, P2 prepare them into the workspace every time.
constexpr size_t kOktPreparedMax = 640 * 1024;

inline Workspace workspace_layout(int64_t M, int64_t K, int64_t N, int r, int bits, bool with_prepared = true) {
    Workspace w{};
    size_t off = 0;
    w.status = off; off += kStatusBytes;
    w.scales = off; off += align_up((size_t)M * 4, 256);
    w.zp = off;     off += align_up((size_t)M * 4, 256);        // per-token zero points (asymmetric activations)
    w.qsum = off;   off += align_up((size_t)M * 4 * kQsumParts, 256);
    const size_t lr_cols = (size_t)lowrank_cols(r);
    w.T = off;      off += align_up((size_t)M * lr_cols * 6, 256);     // bf16 [3][M][cols]
    // partial sums of T: fp32 [KS][16][cols] for the few-token blocks, [tile][part][cols][128] for the tensor-core kernel
    w.lr_part = off; off += r > 0 ? align_up(std::max((size_t)kLrKSplitMax * 16 * lr_cols * 4, lowrank_umma_part_bytes(M, K, r)), 256) : 0;
    w.codes = off;  off += align_up((size_t)M * (size_t)K, 256);
    w.prep = off;   off += with_prepared ? kOktPreparedMax : 0;
    (void)N; (void)bits;
    w.total = off;
    return w;
}

// Argument checks of bwla_w1ax_linear (everything that can be refused without touching the GPU, then the device check).
// BWLA_OK also for the empty problems M == 0 / N == 0, which the caller turns into a no-op.
int validate_linear_call(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, const float* P1, int n1, const float* P2,
                         int n2, int bits, const uint32_t* packed, const float* alpha, const void* U_bf16,
                         const void* V_bf16, int r, const void* out_bf16, int64_t N, int64_t ldo, const void* workspace,
                         size_t workspace_bytes);

// ---------------------------------------------------------------------------------------------
// kernel launchers (each returns a BWLA status; all asynchronous on `stream`)
// ---------------------------------------------------------------------------------------------
int launch_pack_signs(const void* w, int dtype, int64_t N, int64_t K, int64_t ldw, uint32_t* packed,
                      cudaStream_t stream);
// rowsum[n] = sum_k sign(n,k) = 2 * popc(row n) - K
int launch_row_sums(const uint32_t* packed, int64_t N, int64_t K, int32_t* rowsum, cudaStream_t stream);

// One launch: fused rotate + absmax + quantise (skipped when codes == NULL) and T = V x (skipped when r == 0 or
// Thl == NULL).  codes_layout: 0 = natural k order, 1 = interleaved order used by the tensor-core contraction (inside
// each group of 32, position 4*j + i holds k = j + 8*i).  qsum (int32 [M][kQsumParts], partial sums) may be NULL.
// Thl: bf16 [3][M][cols], cols = lowrank_cols(r): T as the sum of three bf16 terms (exact for an fp32 T).
// lr_part / status (both may be NULL): scratch for the partial sums of T and the workspace status words (see kLrKSplitMax).
int launch_prologue(const void* x, int64_t M, int64_t K, int64_t ldx, const float* P1, int n1, const float* P2, int n2,
                    int bits, int8_t* codes, int codes_layout, float* scales, int32_t* qsum, const void* V, int r,
                    void* Thl, float* lr_part, uint32_t* status, cudaStream_t stream);

// ---- tcgen05 version of the rotation + quantiser (okt_umma.cu) ----
// Geometry of the kernel for one pair of Kronecker factor sizes; computed on the host, passed to the kernels by value.
struct OktGeom {
    int n1, n2, K;
    int n1p, n2p;           // n1, n2 rounded up to 16: columns of Z^T / Y^T, contraction depth of the first stage
    int atom2, atom1;       // bytes of one K-atom row (the swizzle span) of operands contracted over b / over a
    int dt_count, dt_rows;  // tiles of the rows d of P2^T (= tensor-memory lanes) and rows per tile (a multiple of 8)
    int cs_count, cs_cols;  // slabs of the rows c of P1^T (= output columns) and columns per slab (a multiple of 16)
    int p2t_bytes, p1t_bytes, x_bytes;      // one tile of P2^T terms, one slab of P1^T terms, one token's X tile
    int p1t_off, x_off, bar_off;            // shared-memory offsets (P2^T tile at 0)
    int tmem_cols, smem_bytes;
};
constexpr int kOktMaxProblems = 4;          // linears that share one x and are rotated by one launch
struct OktProblem {
    const uint8_t* prepared;    // bf16 terms of P2^T tiles and P1^T slabs (launch_prepare_okt)
    int8_t* codes;              // [M][K]
    int codes_layout;           // 0: natural k order; 1: the interleaved order of the tensor-core contraction
    int32_t* zp;                // [M] zero points (asymmetric quantiser), or NULL
    int code_bias;              // added to every stored code and to the stored zero point (see launch_okt)
    float* scales;              // [M]
    int32_t* qsum;              // [M][kQsumParts] or NULL
    float* y_debug;             // [M][K] fp32 rotated activations before the quantiser, or NULL
};
struct OktLowrank { const void* V; int r; void* Thl; float* lr_part; uint32_t* lr_count; };   // V == NULL: no T = V x blocks
// false when the factor sizes are outside what the kernel takes (n2 a multiple of 8 up to 256, n1 up to 192, ...)
bool okt_geometry(int n1, int n2, OktGeom* out);
// false when x cannot be read by tiled TMA loads (16-byte aligned base, row stride a multiple of 8 elements)
bool okt_accepts_x(const void* x, int64_t ldx);
size_t okt_prepared_bytes(const OktGeom& g);
int launch_prepare_okt(const OktGeom& g, const float* P1, const float* P2, void* prepared, cudaStream_t stream);
// One launch for up to kOktMaxProblems linears that read the same x: rotation + quantiser for each, and the T = V x
// blocks of those with a low-rank branch.
// asym == 0: symmetric codes in [-qmax, qmax], qmax = 2^(b-1) - 1.  asym == 1 (Sec. 4.1, per-token asymmetric): with
// u in [0, 2^b - 1] and the integer zero point z of the token, the stored code is u - 2^(b-1) + code_bias and the
// stored zero point z - 2^(b-1) + code_bias; a code minus the zero point times the scale is the value it stands for.
int launch_okt(const OktGeom& g, const void* x, int64_t M, int64_t ldx, int bits, int asym, int n_problems,
               const OktProblem* problems, const OktLowrank* lowrank, uint32_t* status, cudaStream_t stream);

// qsum[t][0] = sum_k codes[t][k] (the other parts zero); optionally rewrites natural-order codes into the interleaved order.
int launch_prepare_codes(const int8_t* codes, int64_t M, int64_t K, int8_t* codes_interleaved, int32_t* qsum,
                         cudaStream_t stream);

struct GemmArgs {
    const int8_t* codes;      // [M][K]; natural order for the simple path
    const float* scales;      // [M]
    const int32_t* qsum;      // [M][kQsumParts] partial sums
    int64_t M, K, N;
    int bits;
    const uint32_t* packed;   // [N][K/32]
    const float* alpha;       // [N]
    const float* mu;          // [N] or NULL
    const int32_t* zp;        // [M] per-token zero points of the codes, or NULL (symmetric codes)
    const int32_t* rowsum;    // [N] sum_k sign(n,k) = 2 * popc(row n) - K; read only when zp is given
    const void* Thl;          // bf16 [3][M][lowrank_cols(r)] or NULL
    const void* U;            // bf16 [N][r] or NULL
    int r;
    void* out;                // bf16 [M][ldo] or NULL
    int64_t ldo;
    int32_t* acc_debug;       // [M][N] or NULL
    uint32_t* status;         // workspace status words
    // Contractions of a group that read the results of the same preceding kernel (the rotation launch): the first one
    // (kDepHead) lets the next kernel of the stream start only once it has itself seen that kernel complete, so the
    // others (kDepSibling) need not wait for their predecessor, a sibling, before they read: they run beside it.
    // kDepChain: the ordinary chain (wait for the predecessor before reading its results).
    int dep_mode;
    int sm_budget;            // SMs this launch should plan for (0: all): siblings share the device
};
enum { kDepChain = 0, kDepHead = 1, kDepSibling = 2 };

// W1A16, the weight-only operating point (gemm_a16.cu): Y (fp32) -> bf16 + per-token sums; the bf16 contraction against
// the packed signs with the fused epilogue.  Thl as for the int8 contractions (NULL when r == 0).
bool a16_supports(int64_t M, int64_t K, int64_t N, int r);
int launch_y_to_bf16(const float* Y, int64_t M, int64_t K, void* yhat, float* ysum, cudaStream_t stream);
int launch_gemm_a16(const void* yhat, const float* ysum, int64_t M, int64_t K, int64_t N, const uint32_t* packed, const float* alpha,
                    const float* mu, const void* U, int r, const void* Thl, void* out, int64_t ldo, uint32_t* status,
                    cudaStream_t stream);

// Final binarisation of weight rows in the rotated coordinates (binarize.cu).
size_t binarize_workspace_bytes(int64_t K);
int launch_binarize(const void* w, int dtype, int64_t N, int64_t K, int64_t ldw, const float* P1, int n1, const float* P2, int n2,
                    uint32_t* packed, float* alpha, float* mu, void* workspace, cudaStream_t stream);

int launch_gemm_simple(const GemmArgs& a, cudaStream_t stream);

// One to four tokens: activation bit-planes against the packed sign words (and + popc), weights never expanded.
// a.codes in natural k order.
bool bitplane_supports(int64_t M, int64_t K, int64_t N, int r, int bits);
int launch_gemm_bitplane(const GemmArgs& a, cudaStream_t stream);

// tcgen05 path with the fused epilogue.  codes_interleaved: int8 [M][K] in the interleaved order.
bool umma_supports(int64_t M, int64_t K, int64_t N, int r, int bits);
int launch_gemm_umma(const GemmArgs& a, const int8_t* codes_interleaved, cudaStream_t stream);
// More than 64 tokens: the same contraction in CTAs that stay on their SM and take tiles of 128 rows x 128 tokens in turn.
bool umma_persistent_supports(int64_t M, int64_t K, int64_t N, int r);
int launch_gemm_umma_persistent(const GemmArgs& a, const int8_t* codes_interleaved, cudaStream_t stream);

}  // namespace bwla
