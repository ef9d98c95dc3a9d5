// T = V x for many tokens on the tcgen05 tensor cores (PSP low-rank branch, Sec. 3.2: the layer output carries the
// term U (V x) beside the binarised product; this file evaluates the inner factor for a prefill-sized batch).
//
//   T[t][j] = sum_k x[t][k] V[j][k]        x bf16 [M][K], V bf16 [r][K], r <= 64, T fp32 kept as three bf16 terms
//
// Both operands are bf16 already, so every product is exact in fp32 and only the order of the additions matters.  The
// tensor core adds each group of 16 products into its accumulator with truncation; over the thousands of k-steps of a
// large K that bias would reach 1e-4 of the sum.  The accumulator therefore only ever holds 128 values of k: after
// every 128 it is read back and added, with ordinary rounded fp32 additions, into running sums the epilogue warps keep
// in registers, while the next 128 go into the second accumulator.
//
// Work of one CTA: a tile of 128 tokens (the accumulator's lanes) x all 64 columns x one part of K.  With fewer token
// tiles than SMs, K is split into parts; the parts leave their sums in the workspace and a second small kernel adds
// them in the order of the parts and splits the result into the three terms (so the result does not depend on which
// CTA finished last).  Warp 0 copies (TMA: 64 values of k of the x tile and of V per stage), warp 1 issues the MMAs,
// warps 2..5 are the epilogue, one per quarter of the accumulator's lanes.  Every wait is bounded.
#include <cuda_bf16.h>

#include <algorithm>

#include "bwla_common.cuh"
#include "tensor_map.cuh"
#include "umma_ptx.cuh"
#include "umma_wait.cuh"

namespace bwla {

namespace lru {
constexpr int kTok = 128;                 // tokens per tile
constexpr int kCols = 64;                 // columns of T (r padded)
constexpr int kBlockK = 64;               // values of k per stage: one 128-byte swizzle atom of bf16
constexpr int kFlushBlocks = 2;           // stages per accumulator: 128 values of k
constexpr int kStages = 4;
constexpr int kThreads = 192;
constexpr int x_bytes = kTok * kBlockK * 2, v_bytes = kCols * kBlockK * 2, stage_bytes = x_bytes + v_bytes;
constexpr int bars_off = kStages * stage_bytes;
constexpr int smem_bytes = bars_off + 256 + 1024;
constexpr int kTmemCols = 2 * kCols;
constexpr int kMaxParts = 16;             // parts of K per token tile
constexpr int kTargetCtas = 160;          // parts are chosen so that tiles x parts comes near this
}  // namespace lru

struct LrUmmaParams {
    int64_t M;
    int K, ks, tiles, n_problems;
    float* part[kOktMaxProblems];                 // [tile][part][column][lane] fp32 (ks > 1)
    __nv_bfloat16* Thl[kOktMaxProblems];          // [3][M][64]
    uint32_t* status;
};
struct LrMaps { CUtensorMap v[kOktMaxProblems]; };

__device__ __forceinline__ void store_terms(__nv_bfloat16* Thl, int64_t M, int64_t t, int c0, const float (&s)[8]) {
    // three bf16 terms carry all 24 bits of an fp32 value; eight columns = 16 bytes per term
    uint32_t h[4], m[4], l[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float a = s[2 * i], b = s[2 * i + 1];
        const __nv_bfloat16 ha = __float2bfloat16_rn(a), hb = __float2bfloat16_rn(b);
        const float ra = a - __bfloat162float(ha), rb = b - __bfloat162float(hb);
        const __nv_bfloat16 ma = __float2bfloat16_rn(ra), mb = __float2bfloat16_rn(rb);
        const __nv_bfloat16 la = __float2bfloat16_rn(ra - __bfloat162float(ma)), lb = __float2bfloat16_rn(rb - __bfloat162float(mb));
        h[i] = (uint32_t)__bfloat16_as_ushort(ha) | ((uint32_t)__bfloat16_as_ushort(hb) << 16);
        m[i] = (uint32_t)__bfloat16_as_ushort(ma) | ((uint32_t)__bfloat16_as_ushort(mb) << 16);
        l[i] = (uint32_t)__bfloat16_as_ushort(la) | ((uint32_t)__bfloat16_as_ushort(lb) << 16);
    }
    const int64_t at = t * lru::kCols + c0;
    *reinterpret_cast<uint4*>(Thl + at) = make_uint4(h[0], h[1], h[2], h[3]);
    *reinterpret_cast<uint4*>(Thl + M * lru::kCols + at) = make_uint4(m[0], m[1], m[2], m[3]);
    *reinterpret_cast<uint4*>(Thl + 2 * M * lru::kCols + at) = make_uint4(l[0], l[1], l[2], l[3]);
}

__global__ void __launch_bounds__(lru::kThreads, 2)
lowrank_umma_kernel(const __grid_constant__ CUtensorMap x_map, const __grid_constant__ LrMaps maps, const LrUmmaParams p) {
    using namespace lru;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + bars_off);
    uint64_t* full = bars;                    // [kStages]
    uint64_t* empty = full + kStages;         // [kStages]
    uint64_t* acc_full = empty + kStages;     // [2]
    uint64_t* acc_free = acc_full + 2;        // [2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_free + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // blocks that share a token tile and a part of K (one per problem) are neighbours: the x tile is in the L2 for all but one
    const int pi = (int)blockIdx.x % p.n_problems;
    const int rest = (int)blockIdx.x / p.n_problems;
    const int kp = rest % p.ks, tile = rest / p.ks;
    const int nblocks = p.K / kBlockK;
    const int b_lo = (int)((int64_t)nblocks * kp / p.ks), b_hi = (int)((int64_t)nblocks * (kp + 1) / p.ks);
    const int nb = b_hi - b_lo;
    const int units = (nb + kFlushBlocks - 1) / kFlushBlocks;
    const int64_t t0 = (int64_t)tile * kTok;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int i = 0; i < kStages; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&acc_full[i], 1); mbar_init(&acc_free[i], 4); }
        fence_barrier_init();
        fence_proxy_async();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    griddep_launch_dependents();

    if (warp == 0) {
        if (elect_one()) {
            tma_prefetch_desc(&x_map);
            tma_prefetch_desc(&maps.v[pi]);
            griddep_wait();                           // x may be the output of the preceding kernel
            if (p.status && *reinterpret_cast<volatile uint32_t*>(p.status) != 0) *abort_flag = 1;   // the call already failed
            int s = 0; uint32_t ph = 0;
            for (int b = b_lo; b < b_hi && !*abort_flag; ++b) {
                if (!wait_or_abort(&empty[s], ph ^ 1u, abort_flag)) { give_up(p.status, abort_flag, 0x210); break; }
                mbar_expect_tx(&full[s], stage_bytes);
                tma_load_2d(smem + s * stage_bytes, &x_map, b * kBlockK, (int)t0, &full[s]);
                tma_load_2d(smem + s * stage_bytes + x_bytes, &maps.v[pi], b * kBlockK, 0, &full[s]);
                if (++s == kStages) { s = 0; ph ^= 1u; }
            }
            if (*abort_flag) for (int i = 0; i < 500; ++i) __nanosleep(100);   // let copies in flight land
        }
    } else if (warp == 1) {
        if (elect_one()) {
            // D = f32, A = B = bf16, both K-major, M = 128, N = 64
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kCols >> 3) << 17) | ((128u >> 4) << 24);
            int s = 0; uint32_t ph = 0;
            bool ok = true;
            int b = b_lo;
            for (int u = 0; u < units && ok; ++u) {
                const int buf = u & 1;
                if (u >= 2 && !wait_or_abort(&acc_free[buf], (uint32_t)(((u >> 1) - 1) & 1), abort_flag)) { give_up(p.status, abort_flag, 0x220); break; }
                tc_fence_after();
                const uint32_t d_addr = tmem_base + (uint32_t)(buf * kCols);
                for (int i = 0; i < kFlushBlocks && b < b_hi; ++i, ++b) {
                    if (!wait_or_abort(&full[s], ph, abort_flag)) { give_up(p.status, abort_flag, 0x221); ok = false; break; }
                    tc_fence_after();
                    const uint32_t xa = smem_u32(smem + s * stage_bytes), va = xa + x_bytes;
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        mma_f16_ss(d_addr, smem_desc_sw128(xa, 32 * j), smem_desc_sw128(va, 32 * j), idesc, (i | j) ? 1u : 0u);
                    tc_commit(&empty[s]);
                    if (++s == kStages) { s = 0; ph ^= 1u; }
                }
                if (ok) tc_commit(&acc_full[buf]);
            }
        }
    } else {
        const int q = warp & 3;
        const int lane_d = q * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
        float run[kCols];
#pragma unroll
        for (int c = 0; c < kCols; ++c) run[c] = 0.f;
        bool ok = true;
        for (int u = 0; u < units && ok; ++u) {
            const int buf = u & 1;
            if (!warp_wait(&acc_full[buf], (uint32_t)((u >> 1) & 1), abort_flag)) { give_up(p.status, abort_flag, 0x230); ok = false; break; }
            tc_fence_after();
            uint32_t v[4][16];
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld_32x16(tmem_base + lane_addr + (uint32_t)(buf * kCols + 16 * c), v[c]);
            tc_wait_ld();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_free[buf]);
#pragma unroll
            for (int c = 0; c < 4; ++c)
#pragma unroll
                for (int i = 0; i < 16; ++i) run[16 * c + i] += __uint_as_float(v[c][i]);
        }
        griddep_wait();                               // nothing is stored before the preceding kernel has completed
        if (ok) {
            const int64_t t = t0 + lane_d;
            if (p.ks == 1) {
                if (t < p.M) {
#pragma unroll
                    for (int c = 0; c < kCols; c += 8) {
                        const float s8[8] = {run[c], run[c + 1], run[c + 2], run[c + 3], run[c + 4], run[c + 5], run[c + 6], run[c + 7]};
                        store_terms(p.Thl[pi], p.M, t, c, s8);
                    }
                }
            } else {
                float* mine = p.part[pi] + ((size_t)tile * p.ks + kp) * (kCols * kTok) + lane_d;
#pragma unroll
                for (int c = 0; c < kCols; ++c) mine[c * kTok] = run[c];
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// The parts of K of every tile, added in the order of the parts, then split into the three bf16 terms.  One block per
// (problem, tile, group of eight columns); a thread is a token.
__global__ void __launch_bounds__(lru::kTok) lowrank_reduce_kernel(const LrUmmaParams p) {
    using namespace lru;
    griddep_launch_dependents();
    griddep_wait();                                   // the partial sums are the preceding kernel's
    const int pi = (int)blockIdx.x % p.n_problems;
    const int rest = (int)blockIdx.x / p.n_problems;
    const int cg = rest % (kCols / 8), tile = rest / (kCols / 8);
    const int64_t t = (int64_t)tile * kTok + threadIdx.x;
    float s[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    const float* src = p.part[pi] + (size_t)tile * p.ks * (kCols * kTok) + (size_t)(8 * cg) * kTok + threadIdx.x;
    // all loads of four parts are in flight before the first addition (the loop is a chain of L2 latencies otherwise);
    // the additions keep the order of the parts
    for (int k0 = 0; k0 < p.ks; k0 += 4) {
        float v[4][8];
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
#pragma unroll
            for (int c = 0; c < 8; ++c)
                v[kk][c] = k0 + kk < p.ks ? __ldcg(src + (size_t)(k0 + kk) * (kCols * kTok) + c * kTok) : 0.f;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
#pragma unroll
            for (int c = 0; c < 8; ++c) s[c] += v[kk][c];
    }
    if (t < p.M) store_terms(p.Thl[pi], p.M, t, 8 * cg, s);
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
// Parts of K for M tokens: enough CTAs to fill the device while every part keeps at least eight stages.
static int lowrank_umma_parts(int64_t M, int64_t K) {
    const int64_t tiles = (M + lru::kTok - 1) / lru::kTok;
    int64_t ks = std::max<int64_t>(1, lru::kTargetCtas / tiles);
    ks = std::min<int64_t>(ks, lru::kMaxParts);
    ks = std::min<int64_t>(ks, std::max<int64_t>(1, K / (8 * lru::kBlockK)));
    return (int)ks;
}

bool lowrank_umma_supports(int64_t M, int64_t K, int r) {
    return M >= 256 && r > 0 && r <= lru::kCols && lowrank_cols(r) == lru::kCols && K % lru::kBlockK == 0 && K >= lru::kBlockK;
}

size_t lowrank_umma_part_bytes(int64_t M, int64_t K, int r) {
    if (!lowrank_umma_supports(M, K, r)) return 0;
    const int ks = lowrank_umma_parts(M, K);
    if (ks == 1) return 0;
    const int64_t tiles = (M + lru::kTok - 1) / lru::kTok;
    return (size_t)tiles * ks * lru::kCols * lru::kTok * 4;
}

int launch_lowrank_umma(const void* x, int64_t M, int64_t K, int64_t ldx, int n_problems, const OktLowrank* lowrank,
                        uint32_t* status, cudaStream_t stream) {
    using namespace lru;
    if (n_problems < 1 || n_problems > kOktMaxProblems || M >= ((int64_t)1 << 31)) return BWLA_ERR_INVALID_ARG;
    LrUmmaParams p{};
    LrMaps maps{};
    p.M = M; p.K = (int)K; p.ks = lowrank_umma_parts(M, K); p.tiles = (int)((M + kTok - 1) / kTok); p.n_problems = n_problems;
    p.status = status;
    CUtensorMap xm;
    {
        const uint64_t dims[2] = {(uint64_t)K, (uint64_t)M};
        const uint64_t strides[1] = {(uint64_t)ldx * 2};
        const uint32_t box[2] = {kBlockK, kTok};
        int st = make_map(&xm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, x, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
        if (st != BWLA_OK) return st;
    }
    for (int i = 0; i < n_problems; ++i) {
        if (!lowrank[i].V || !lowrank[i].Thl || (p.ks > 1 && !lowrank[i].lr_part)) return BWLA_ERR_INVALID_ARG;
        const uint64_t dims[2] = {(uint64_t)K, (uint64_t)lowrank[i].r};       // rows beyond r read as zero
        const uint64_t strides[1] = {(uint64_t)K * 2};
        const uint32_t box[2] = {kBlockK, kCols};
        int st = make_map(&maps.v[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, lowrank[i].V, dims, strides, box,
                          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
        if (st != BWLA_OK) return st;
        p.part[i] = lowrank[i].lr_part;
        p.Thl[i] = (__nv_bfloat16*)lowrank[i].Thl;
    }
    static thread_local int configured_device = -1;
    int dev = 0;
    BWLA_CUDA_TRY(cudaGetDevice(&dev));
    if (configured_device != dev) {
        BWLA_CUDA_TRY(cudaFuncSetAttribute(lowrank_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes));
        configured_device = dev;
    }
    cudaLaunchAttribute attrs[1];
    attrs[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attrs[0].val.programmaticStreamSerializationAllowed = launch_overlap_allowed();
    {
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3((unsigned)(p.tiles * p.ks * n_problems), 1, 1);
        cfg.blockDim = dim3(kThreads, 1, 1);
        cfg.dynamicSmemBytes = smem_bytes;
        cfg.stream = stream;
        cfg.attrs = attrs;
        cfg.numAttrs = 1;
        ProfScope prof(kProfRotateQuant, stream);
        cudaError_t e = cudaLaunchKernelEx(&cfg, lowrank_umma_kernel, xm, maps, p);
        if (e != cudaSuccess) { cudaGetLastError(); return cuda_fail(e); }
        int st = after_launch();
        if (st != BWLA_OK) return st;
    }
    if (p.ks > 1) {
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3((unsigned)(p.tiles * (kCols / 8) * n_problems), 1, 1);
        cfg.blockDim = dim3(kTok, 1, 1);
        cfg.dynamicSmemBytes = 0;
        cfg.stream = stream;
        cfg.attrs = attrs;
        cfg.numAttrs = 1;
        ProfScope prof(kProfRotateQuant, stream);
        cudaError_t e = cudaLaunchKernelEx(&cfg, lowrank_reduce_kernel, p);
        if (e != cudaSuccess) { cudaGetLastError(); return cuda_fail(e); }
        return after_launch();
    }
    return BWLA_OK;
}

}  // namespace bwla
