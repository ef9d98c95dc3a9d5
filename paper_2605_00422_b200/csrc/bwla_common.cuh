// Shared declarations of the CUDA library: status handling, workspace layout, kernel launchers.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "bwla.h"

namespace bwla {

// ---------------------------------------------------------------------------------------------
// per-thread bookkeeping (no global mutable state apart from the forced path)
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

// ---------------------------------------------------------------------------------------------
// optional per-kernel timing (bwla_profile_enable / bwla_profile_collect): CUDA events recorded on the launching
// stream right around each kernel launch, summed per kernel kind.  Off by default; not usable under stream capture.
// ---------------------------------------------------------------------------------------------
enum ProfKind { kProfRotateQuant = 0, kProfLowrankT = 1, kProfContraction = 2, kProfFinalize = 3, kProfPrepare = 4,
                kProfPack = 5, kProfKinds = 8 };
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
constexpr int kBitplaneMaxTokens = 1;    // the bit-plane path keeps M*bits + 1 <= 8 MMA columns
constexpr int kSplitKMaxTokens = 64;     // int32 partial sums in scratch are kept for M up to this

struct Workspace {
    size_t status, scales, qsum, T, codes, planes, acc, total;
};

inline Workspace workspace_layout(int64_t M, int64_t K, int64_t N, int r, int bits) {
    Workspace w{};
    size_t off = 0;
    w.status = off; off += kStatusBytes;
    w.scales = off; off += align_up((size_t)M * 4, 256);
    w.qsum = off;   off += align_up((size_t)M * 4, 256);
    w.T = off;      off += align_up((size_t)M * (size_t)(r > 0 ? r : 1) * 4, 256);
    w.codes = off;  off += align_up((size_t)M * (size_t)K, 256);
    w.planes = off; off += (M <= kBitplaneMaxTokens) ? align_up((size_t)M * 8 * (size_t)(K / 32) * 4, 256) : 0;
    w.acc = off;    off += align_up((size_t)M * (size_t)N * 4, 256);
    (void)bits;
    w.total = off;
    return w;
}

// ---------------------------------------------------------------------------------------------
// kernel launchers (each returns a BWLA status; all asynchronous on `stream`)
// ---------------------------------------------------------------------------------------------
int launch_pack_signs(const void* w, int dtype, int64_t N, int64_t K, int64_t ldw, uint32_t* packed,
                      cudaStream_t stream);

// Fused rotate + absmax + quantise.  codes_layout: 0 = natural k order, 1 = interleaved order used by the
// tensor-core contraction (inside each group of 32, position 4*j + i holds k = j + 8*i).
// qsum (int32 [M]) and planes (uint32 [M][bits+... ]) may be NULL.
int launch_rotate_quant(const void* x, int64_t M, int64_t K, int64_t ldx, const float* P1, int n1,
                        const float* P2, int n2, int bits, int8_t* codes, int codes_layout, float* scales,
                        int32_t* qsum, uint32_t* planes, uint32_t* status, cudaStream_t stream);

// T[t][j] = sum_k V[j][k] * x[t][k], fp32 accumulate.
int launch_lowrank_T(const void* x, int64_t M, int64_t K, int64_t ldx, const void* V, int r, float* T,
                     cudaStream_t stream);

// qsum[t] = sum_k codes[t][k]; optionally rewrites natural-order codes into the interleaved order.
int launch_prepare_codes(const int8_t* codes, int64_t M, int64_t K, int8_t* codes_interleaved, int32_t* qsum,
                         uint32_t* status, cudaStream_t stream);

struct GemmArgs {
    const int8_t* codes;      // [M][K]; natural order for the simple path
    const float* scales;      // [M]
    const int32_t* qsum;      // [M]
    int64_t M, K, N;
    int bits;
    const uint32_t* packed;   // [N][K/32]
    const float* alpha;       // [N]
    const float* mu;          // [N] or NULL
    const float* T;           // [M][r] fp32 or NULL
    const void* U;            // bf16 [N][r] or NULL
    int r;
    void* out;                // bf16 [M][ldo] or NULL
    int64_t ldo;
    int32_t* acc_debug;       // [M][N] or NULL
    uint32_t* status;         // workspace status words
};

int launch_gemm_simple(const GemmArgs& a, cudaStream_t stream);

// tcgen05 path.  codes_interleaved: int8 [M][K] in the interleaved order; raw: int32 [M][N] scratch.
bool umma_supports(int64_t M, int64_t K, int64_t N);
int launch_gemm_umma(const GemmArgs& a, const int8_t* codes_interleaved, int32_t* raw, cudaStream_t stream);

}  // namespace bwla
