// Binary contraction for one to four tokens on activation bit-planes: the packed sign words are never expanded.
//
//   sum_k bit(n,k) * q[t][k] = sum_i w_i * popc(word(n) & plane_i[t]),      q in two's complement on b bits:
//                                                                           w_i = 2^i for i < b-1, w_{b-1} = -2^(b-1)
//   acc[t][n] = sum_k sign(n,k) * q[t][k] = 2 * sum_k bit(n,k) * q[t][k] - sum_k q[t][k]        (sign = 2*bit - 1)
//   out[t][n] = bf16(alpha[n] * s_t * acc + U[n,:] . T[t,:] [+ mu[n] * s_t * sum_k q[t][k]])    (Eq. 4; Sec. 3.2)
//
// Three instructions (and, popc, add) per 32 weights and plane on the ordinary integer pipes: on this part they issue
// at the full rate (the and + popc + add probe of microbench/issue_rates.cu sustains ~1280 weight-planes per clock and
// SM), which for one token of 6-bit codes is about the rate at which HBM delivers the sign bits; the warp-level 1-bit
// tensor-core instruction of the same probe is slower (~790 weight-columns per clock and SM).  With every further
// token the work grows in proportion, so from a few tokens on the tcgen05 kind::i8 kernel is the faster one.
//
// A CTA owns R output rows and all of K.  Before the preceding kernel of the stream has finished it only asks the L2 for
// its rows' sign words; afterwards it builds the bit-planes of the tokens in shared memory (one ballot per plane and 32
// codes), and its warps take work items of 16 rows x 32 sign words in turn: a lane owns one word position, keeps that
// position's planes in registers and runs over the 16 rows (16 independent loads in flight), the 16 sums are reduced
// across the lanes by shuffles and added into the tile's accumulators in shared memory.  The epilogue is one thread
// per output.
#include <cuda_bf16.h>

#include <algorithm>

#include "bwla_common.cuh"
#include "umma_ptx.cuh"

namespace bwla {

using namespace ptx;

constexpr int kBpThreads = 512;
constexpr int kBpItemRows = 16;
constexpr int kBpMaxTokens = 4;

struct BitplaneParams {
    const int8_t* codes;      // [M][K], natural k order
    const float* scales;      // [M]
    const int32_t* qsum;      // [M][kQsumParts]
    const uint32_t* packed;   // [N][K/32]
    const float* alpha; const float* mu;
    const int32_t* zp; const int32_t* rowsum;       // asymmetric codes: per-token zero points, per-row sign sums (or NULL)
    const __nv_bfloat16* U; const __nv_bfloat16* Thl; int r, lr_cols;
    __nv_bfloat16* out; int64_t ldo; int32_t* acc_debug;
    int M, N, K, bits, R;     // R: rows per CTA (a multiple of 16)
};

__device__ __forceinline__ void prefetch_l2(const void* p, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(bytes) : "memory");
}

template <int MT, int B>
__global__ void __launch_bounds__(kBpThreads, MT <= 2 ? 2 : 1) bitplane_w1a_kernel(BitplaneParams p) {
    extern __shared__ __align__(16) uint32_t bp_smem[];
    const int words = p.K >> 5;
    constexpr int b = B;
    constexpr int stride = MT * b + 1 - ((MT * b) & 1);          // odd: lanes read their planes without bank conflicts
    uint32_t* planes = bp_smem;                               // [words][stride]: plane i of token t at t * b + i
    int32_t* tile_acc = reinterpret_cast<int32_t*>(planes + (size_t)words * stride);   // [R][MT]
    float* Ts = reinterpret_cast<float*>(tile_acc + p.R * MT);                          // [MT][lr_cols]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = kBpThreads / 32;
    const int n0 = blockIdx.x * p.R;
    const int rows_here = min(p.R, p.N - n0);

    // ---- before the preceding kernel has finished: ask the L2 for this tile's sign words (they depend on nothing)
    griddep_launch_dependents();
    {
        const uint32_t row_bytes = (uint32_t)(p.K >> 3);
        if ((row_bytes & 15) == 0)
            for (int r = threadIdx.x; r < rows_here; r += kBpThreads)
                prefetch_l2(p.packed + (size_t)(n0 + r) * words, row_bytes);
    }
    for (int i = threadIdx.x; i < p.R * MT; i += kBpThreads) tile_acc[i] = 0;
    griddep_wait();

    // ---- bit-planes of the tokens (two's complement bits of the codes) and T = hi + mid + lo
    for (int item = warp; item < words * MT; item += nwarps) {
        const int g = item / MT, t = item - g * MT;
        const int q = t < p.M ? (int)p.codes[(size_t)t * p.K + 32 * g + lane] : 0;
        uint32_t mine = 0;
        for (int i = 0; i < b; ++i) {
            const uint32_t w = __ballot_sync(0xFFFFFFFFu, (q >> i) & 1);
            if (lane == i) mine = w;
        }
        if (lane < b) planes[(size_t)g * stride + t * b + lane] = mine;
    }
    if (p.r > 0)
        for (int i = threadIdx.x; i < MT * p.lr_cols; i += kBpThreads) {
            const int t = i / p.lr_cols, j = i - t * p.lr_cols;
            float v = 0.f;
            if (t < p.M) {
                const size_t at = (size_t)t * p.lr_cols + j, plane_sz = (size_t)p.M * p.lr_cols;
                v = (__bfloat162float(p.Thl[at]) + __bfloat162float(p.Thl[plane_sz + at])) + __bfloat162float(p.Thl[2 * plane_sz + at]);
            }
            Ts[i] = v;
        }
    __syncthreads();

    // ---- work items: 16 rows x 32 sign words
    const int chunks = (words + 31) >> 5;
    const int row_groups = (rows_here + kBpItemRows - 1) / kBpItemRows;
    for (int item = warp; item < row_groups * chunks; item += nwarps) {
        const int rg = item / chunks, c = item - rg * chunks;
        const int g = 32 * c + lane;                          // this lane's word position
        const bool word_ok = g < words;
        uint32_t pl[MT][B];
#pragma unroll
        for (int t = 0; t < MT; ++t)
#pragma unroll
            for (int i = 0; i < B; ++i) pl[t][i] = word_ok ? planes[(size_t)g * stride + t * b + i] : 0u;
        const int r0 = rg * kBpItemRows;
        uint32_t w[kBpItemRows];
#pragma unroll
        for (int r = 0; r < kBpItemRows; ++r)
            w[r] = (word_ok && r0 + r < rows_here) ? __ldg(p.packed + (size_t)(n0 + r0 + r) * words + g) : 0u;
        int acc[kBpItemRows][MT];
#pragma unroll
        for (int r = 0; r < kBpItemRows; ++r)
#pragma unroll
            for (int t = 0; t < MT; ++t) {
                int s = 0;
#pragma unroll
                for (int i = 0; i < B; ++i) {
                    const int pc = __popc(w[r] & pl[t][i]);
                    s += (i == B - 1) ? -(pc << i) : (pc << i);        // the top plane carries the negative weight
                }
                acc[r][t] = s;
            }
        // sum over the 32 word positions: after step j a lane holds the partial sums of 16 >> j rows
#pragma unroll
        for (int t = 0; t < MT; ++t) {
            int v16[16];
#pragma unroll
            for (int r = 0; r < 16; ++r) v16[r] = acc[r][t];
            // lane bit 4 picks the half of the rows a lane keeps, and so on down to one row per lane pair
#pragma unroll
            for (int step = 0; step < 4; ++step) {
                const int half = 8 >> step;                   // rows kept after this step
                const bool upper = (lane >> (4 - step)) & 1;
#pragma unroll
                for (int r = 0; r < 8; ++r) {
                    if (r < half) {
                        const int keep = upper ? v16[r + half] : v16[r];
                        const int give = upper ? v16[r] : v16[r + half];
                        v16[r] = keep + __shfl_xor_sync(0xFFFFFFFFu, give, 16 >> step);
                    }
                }
            }
            // 16 rows are now spread over lane bits 4..1 (row = bits 4,3,2,1 read as upper choices); bit 0 still to add
            int v = v16[0] + __shfl_xor_sync(0xFFFFFFFFu, v16[0], 1);
            const int row = ((lane >> 4) & 1) * 8 + ((lane >> 3) & 1) * 4 + ((lane >> 2) & 1) * 2 + ((lane >> 1) & 1);
            if ((lane & 1) == 0 && r0 + row < rows_here && v != 0) atomicAdd(&tile_acc[(r0 + row) * MT + t], v);
        }
    }
    __syncthreads();

    // ---- epilogue: one thread per output
    for (int o = threadIdx.x; o < rows_here * MT; o += kBpThreads) {
        const int row = o / MT, t = o - row * MT;
        if (t >= p.M) continue;
        const int n = n0 + row;
        int32_t qs = 0;
        for (int c = 0; c < kQsumParts; ++c) qs += p.qsum[(size_t)t * kQsumParts + c];
        const int32_t zp = p.zp ? p.zp[t] : 0;
        const int32_t acc = 2 * tile_acc[o] - qs - (p.zp ? zp * p.rowsum[n] : 0);
        qs -= p.K * zp;
        if (p.acc_debug) p.acc_debug[(size_t)t * p.N + n] = acc;
        if (p.out) {
            const float sc = p.scales[t];
            float l = 0.f;
            if (p.r > 0) {
                const __nv_bfloat16* u = p.U + (size_t)n * p.r;
                const float* tt = Ts + t * p.lr_cols;
                for (int j = 0; j < p.r; ++j) l = fmaf(__bfloat162float(u[j]), tt[j], l);
            }
            const float mu_sc = p.mu ? __fmul_rn(p.mu[n], sc) : 0.f;
            const float y = fmaf(mu_sc, (float)qs, __fmul_rn(__fmul_rn(p.alpha[n], sc), (float)acc) + l);
            p.out[(size_t)t * p.ldo + n] = __float2bfloat16_rn(y);
        }
    }
}

static size_t bitplane_smem(int MT, int64_t K, int R, int r, int bits) {
    const int stride = MT * bits + 1 - ((MT * bits) & 1);
    return ((size_t)(K / 32) * stride + (size_t)R * MT + (size_t)MT * lowrank_cols(r)) * 4;
}

bool bitplane_supports(int64_t M, int64_t K, int64_t N, int r, int bits) {
    if (M < 1 || M > kBpMaxTokens || N < 1 || K % 32 != 0 || K > 65536 || N >= ((int64_t)1 << 31)) return false;
    const int MT = M <= 1 ? 1 : M <= 2 ? 2 : 4;
    return bitplane_smem(MT, K, 64, r, bits) <= 100 * 1024;
}

template <int MT, int B>
static int launch_bitplane_t(const BitplaneParams& p, int grid, size_t smem, cudaStream_t stream) {
    auto kernel = bitplane_w1a_kernel<MT, B>;
    static thread_local int configured = -1;
    int dev = 0;
    BWLA_CUDA_TRY(cudaGetDevice(&dev));
    if (configured != dev) {
        BWLA_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024));
        configured = dev;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(kBpThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attrs[1];
    attrs[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attrs[0].val.programmaticStreamSerializationAllowed = launch_overlap_allowed();
    cfg.attrs = attrs;
    cfg.numAttrs = 1;
    ProfScope prof(kProfContraction, stream);
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, p);
    if (e != cudaSuccess) { cudaGetLastError(); return cuda_fail(e); }
    return after_launch();
}

// a.codes: int8 [M][K] in natural order
int launch_gemm_bitplane(const GemmArgs& a, cudaStream_t stream) {
    if (a.M == 0 || a.N == 0) return BWLA_OK;
    const int sms = sm_count();
    if (sms <= 0) return BWLA_ERR_CUDA;
    BitplaneParams p{};
    p.codes = a.codes; p.scales = a.scales; p.qsum = a.qsum; p.packed = a.packed; p.alpha = a.alpha; p.mu = a.mu;
    p.zp = a.zp; p.rowsum = a.rowsum;
    p.U = (const __nv_bfloat16*)a.U; p.Thl = (const __nv_bfloat16*)a.Thl; p.r = a.r; p.lr_cols = lowrank_cols(a.r);
    p.out = (__nv_bfloat16*)a.out; p.ldo = a.ldo; p.acc_debug = a.acc_debug;
    p.M = (int)a.M; p.N = (int)a.N; p.K = (int)a.K; p.bits = a.bits;
    // rows per CTA: 64, or 32 or 16 when that is what it takes to give every SM about two CTAs
    p.R = 64;
    while (p.R > 16 && (a.N + p.R - 1) / p.R < 2 * sms) p.R >>= 1;
    const int grid = (int)((a.N + p.R - 1) / p.R);
    const int MT = a.M <= 1 ? 1 : a.M <= 2 ? 2 : 4;
    const size_t smem = bitplane_smem(MT, a.K, p.R, a.r, a.bits);
#define BWLA_BP_CASE(mt, bb) if (MT == mt && a.bits == bb) return launch_bitplane_t<mt, bb>(p, grid, smem, stream)
    BWLA_BP_CASE(1, 4); BWLA_BP_CASE(1, 6); BWLA_BP_CASE(1, 8);
    BWLA_BP_CASE(2, 4); BWLA_BP_CASE(2, 6); BWLA_BP_CASE(2, 8);
    BWLA_BP_CASE(4, 4); BWLA_BP_CASE(4, 6); BWLA_BP_CASE(4, 8);
#undef BWLA_BP_CASE
    return BWLA_ERR_INVALID_ARG;
}

}  // namespace bwla
