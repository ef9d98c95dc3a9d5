// Binary-weight contraction on tcgen05 tensor cores (kind::i8, accumulators in tensor memory).
//
//   D[n][t] = sum_k byte(n,k) * q[t][k],  byte(n,k) = -128 if the sign bit of weight (n,k) is set, else 0
//   acc[t][n] = sum_k sign(n,k) * q[t][k] = -D/64 - sum_k q[t][k]            (sign = 2*bit - 1, exact in int32)
//
// One CTA owns 128 output rows x up to 128 tokens x a slice of K:
//   * a TMA warp streams packed sign words (128 rows x 128 bytes = 1024 weights per row, 128B-swizzled);
//   * a second TMA warp streams the activation codes (tokens x 128 bytes per stage, the canonical K-major
//     128B-swizzled UMMA layout);
//   * four expander warps (one per tensor-memory lane quarter, thread = output row) turn each 32-bit word into eight
//     registers of four int8 with one shift and one mask per register ((w << (7-j)) & 0x80808080) and write them
//     with tcgen05.st into tensor memory, where they are the A operand -- expanded weights never touch shared memory;
//   * one thread issues tcgen05.mma.kind::i8 (M = 128, N = tokens, K = 32) with A from tensor memory and B from
//     shared memory, accumulating int32 in tensor memory;
//   * the expander warps read the accumulator back (tcgen05.ld) and add it to the int32 result with red.global
//     (split-K) or plain stores.
// The shift-and-mask expansion meets the weights of a 32-group in the order k = j + 8*i (register j, byte i), so the
// codes are stored in that interleaved order by the quantiser.
//
// Every wait is bounded: on give-up the CTA records where in the workspace status words, stops issuing work, lets
// in-flight copies land, frees its tensor memory and returns.
#include <cuda_bf16.h>

#include "bwla_common.cuh"
#include "umma_ptx.cuh"

namespace bwla {

using namespace ptx;

constexpr int kRowsPerCta = 128;
constexpr int kUnitK = 1024;             // weights per row in one packed-word stage (128 bytes)
constexpr int kBlockK = 128;             // K per code stage / per tensor-memory A stage
constexpr int kTmemCols = 256;           // per CTA, so that two CTAs share an SM's 512 columns
constexpr int kThreads = 224;            // warp 0: weight TMA, 1: MMA, 2: code TMA, 3..6: expand + epilogue
constexpr uint32_t kWaitLimit = 1u << 20;   // polls per wait before giving up (tens of milliseconds)

struct UmmaParams {
    int M, N, K;
    int total_units, units_per_split;
    int32_t* acc;        // [M][N] raw accumulator D
    int use_atomics;
    uint32_t* status;
};

// Shared-memory and tensor-memory budget of one CTA.
//   weights: WS stages of 128 rows x 128 bytes (one K-unit of 1024 weights per row);
//   codes:   BS stages of 16 KB = SUBS k-blocks of (N_TOK rows x 128 bytes), so that small token tiles still move
//            16 KB per barrier round trip;
//   tensor memory: D in columns [0, DCOLS), then AS stages of 32 columns (one k-block of expanded weights each).
template <int N_TOK, int WS, int BS>
struct UmmaCfg {
    static constexpr int w_bytes = kRowsPerCta * 128;
    static constexpr int sub_bytes = N_TOK * 128;
    static constexpr int SUBS = (128 / N_TOK) < 1 ? 1 : ((128 / N_TOK) > 8 ? 8 : (128 / N_TOK));
    static constexpr int b_bytes = SUBS * sub_bytes;
    static constexpr int DCOLS = N_TOK <= 64 ? 64 : 128;
    static constexpr int AS = (kTmemCols - DCOLS) / 32;
    static constexpr int bars_off = WS * w_bytes + BS * b_bytes;
    static constexpr int n_bars = 2 * WS + 2 * BS + 2 * AS + 1;
    static constexpr int total = bars_off + n_bars * 8 + 64 + 1024;   // + slack for 1024-byte alignment
};

__device__ __forceinline__ void give_up(uint32_t* status, volatile int* abort_flag, uint32_t where) {
    if (status) {
        atomicExch(status, 1u);
        status[1] = where;
        status[2] = blockIdx.x | (blockIdx.y << 16);
    }
    *abort_flag = 1;
}

__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    for (uint32_t i = 0; i < kWaitLimit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (i > 32) __nanosleep(32);
    }
    return false;
}

template <int N_TOK, int WS, int BS>
__global__ void __launch_bounds__(kThreads, 1)
umma_w1a_kernel(const __grid_constant__ CUtensorMap w_map, const __grid_constant__ CUtensorMap b_map, UmmaParams p) {
    extern __shared__ uint8_t smem_raw[];
    using L = UmmaCfg<N_TOK, WS, BS>;
    constexpr int AS = L::AS;
    constexpr int SUBS = L::SUBS;
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* wbuf = smem;
    uint8_t* bbuf = smem + WS * L::w_bytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::bars_off);
    uint64_t* w_full = bars;                 // [WS]
    uint64_t* w_empty = bars + WS;           // [WS]
    uint64_t* b_full = bars + 2 * WS;        // [BS]
    uint64_t* b_empty = b_full + BS;         // [BS]
    uint64_t* a_full = b_empty + BS;         // [AS]
    uint64_t* a_empty = a_full + AS;         // [AS]
    uint64_t* d_full = a_empty + AS;         // [1]
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag_s;
    volatile int* abort_flag = &abort_flag_s;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = blockIdx.x * kRowsPerCta;
    const int t0 = blockIdx.y * N_TOK;
    const int unit_begin = blockIdx.z * p.units_per_split;
    const int unit_end = min(p.total_units, unit_begin + p.units_per_split);

    if (threadIdx.x == 0) {
        // a CTA of this launch that already gave up makes the rest of the grid skip its work
        abort_flag_s = (p.status && *reinterpret_cast<volatile uint32_t*>(p.status) != 0) ? 1 : 0;
        for (int i = 0; i < WS; ++i) { mbar_init(&w_full[i], 1); mbar_init(&w_empty[i], 4); }
        for (int i = 0; i < BS; ++i) { mbar_init(&b_full[i], 1); mbar_init(&b_empty[i], 1); }
        for (int i = 0; i < AS; ++i) { mbar_init(&a_full[i], 4); mbar_init(&a_empty[i], 1); }
        mbar_init(d_full, 1);
        fence_barrier_init();
        fence_proxy_async();
    }
    if (warp == 1) {
        tmem_alloc(&tmem_base_slot, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;

    auto sub_count = [&](int u) { return min(kUnitK / kBlockK, (p.K - u * kUnitK) / kBlockK); };

    if (warp == 0) {
        // ---------------- packed sign words: HBM -> shared memory ----------------
        if (elect_one()) {
            tma_prefetch_desc(&w_map);
            int ws = 0; uint32_t wph = 0;
            for (int u = unit_begin; u < unit_end && !*abort_flag; ++u) {
                if (!wait_or_abort(&w_empty[ws], wph ^ 1, abort_flag)) { give_up(p.status, abort_flag, 0x10); break; }
                mbar_expect_tx(&w_full[ws], L::w_bytes);
                tma_load_2d(wbuf + ws * L::w_bytes, &w_map, u * (kUnitK / 32), n0, &w_full[ws]);
                if (++ws == WS) { ws = 0; wph ^= 1; }
            }
            if (*abort_flag) for (int i = 0; i < 500; ++i) __nanosleep(100);   // let copies in flight land
        }
    } else if (warp == 2) {
        // ---------------- activation codes: L2/HBM -> shared memory ----------------
        if (elect_one()) {
            tma_prefetch_desc(&b_map);
            int bs = 0; uint32_t bph = 0;
            bool ok = true;
            for (int u = unit_begin; u < unit_end && ok && !*abort_flag; ++u) {
                const int ns = sub_count(u);
                for (int s0 = 0; s0 < ns; s0 += SUBS) {
                    const int cnt = min(SUBS, ns - s0);
                    if (!wait_or_abort(&b_empty[bs], bph ^ 1, abort_flag)) { give_up(p.status, abort_flag, 0x20); ok = false; break; }
                    mbar_expect_tx(&b_full[bs], cnt * L::sub_bytes);
                    for (int s = 0; s < cnt; ++s)
                        tma_load_2d(bbuf + bs * L::b_bytes + s * L::sub_bytes, &b_map, (u * 8 + s0 + s) * kBlockK, t0, &b_full[bs]);
                    if (++bs == BS) { bs = 0; bph ^= 1; }
                }
            }
            if (*abort_flag) for (int i = 0; i < 500; ++i) __nanosleep(100);
        }
    } else if (warp == 1) {
        // ---------------- MMA issue ----------------
        if (elect_one()) {
            // instruction descriptor: D = s32, A = s8 (tensor memory, K-major), B = s8 (shared, K-major), M = 128
            const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N_TOK >> 3) << 17) | ((128u >> 4) << 24);
            int as = 0; uint32_t aph = 0; int bs = 0; uint32_t bph = 0; uint32_t first = 1;
            bool ok = true;
            for (int u = unit_begin; u < unit_end && ok; ++u) {
                const int ns = sub_count(u);
                for (int s = 0; s < ns; ++s) {
                    const int sb = s % SUBS;
                    if (sb == 0 && !wait_or_abort(&b_full[bs], bph, abort_flag)) { give_up(p.status, abort_flag, 0x30); ok = false; break; }
                    if (!wait_or_abort(&a_full[as], aph, abort_flag)) { give_up(p.status, abort_flag, 0x31); ok = false; break; }
                    tc_fence_after();
                    const uint32_t b_addr = smem_u32(bbuf + bs * L::b_bytes + sb * L::sub_bytes);
                    const uint32_t a_addr = tmem_base + L::DCOLS + 32 * as;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        mma_i8_ts(tmem_base, a_addr + 8 * i, smem_desc_sw128(b_addr, 32 * i), idesc, first ? 0u : 1u);
                        first = 0;
                    }
                    tc_commit(&a_empty[as]);
                    if (++as == AS) { as = 0; aph ^= 1; }
                    if (sb == SUBS - 1 || s == ns - 1) {
                        tc_commit(&b_empty[bs]);
                        if (++bs == BS) { bs = 0; bph ^= 1; }
                    }
                }
            }
            tc_commit(d_full);
        }
    } else {
        // ---------------- expand sign bits into tensor memory, then drain the accumulator ----------------
        const int q = warp & 3;                       // tensor-memory lane quarter this warp may touch
        const int row = q * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
        int ws = 0; uint32_t wph = 0; int as = 0; uint32_t aph = 0;
        bool ok = true;
        for (int u = unit_begin; u < unit_end && ok; ++u) {
            if (!__all_sync(0xFFFFFFFFu, wait_or_abort(&w_full[ws], wph, abort_flag))) { give_up(p.status, abort_flag, 0x40); ok = false; break; }
            const uint8_t* wrow = wbuf + ws * L::w_bytes + row * 128;
            const int ns = sub_count(u);
            for (int s = 0; s < ns; ++s) {
                const uint4 w4 = *reinterpret_cast<const uint4*>(wrow + ((s ^ (row & 7)) << 4));
                uint32_t v[32];
                const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 8; ++j) v[8 * i + j] = (w[i] << (7 - j)) & 0x80808080u;
                if (!__all_sync(0xFFFFFFFFu, wait_or_abort(&a_empty[as], aph ^ 1, abort_flag))) { give_up(p.status, abort_flag, 0x41); ok = false; break; }
                tc_fence_after();
                tmem_st_32x32(tmem_base + lane_addr + L::DCOLS + 32 * as, v);
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&a_full[as]);
                if (++as == AS) { as = 0; aph ^= 1; }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&w_empty[ws]);
            if (++ws == WS) { ws = 0; wph ^= 1; }
        }
        if (ok && unit_begin < unit_end) {
            if (!__all_sync(0xFFFFFFFFu, wait_or_abort(d_full, 0, abort_flag))) { give_up(p.status, abort_flag, 0x50); ok = false; }
        }
        if (ok && unit_begin < unit_end) {
            tc_fence_after();
            const int n = n0 + row;
#pragma unroll 1
            for (int c = 0; c < N_TOK / 16; ++c) {
                uint32_t v[16];
                tmem_ld_32x16(tmem_base + lane_addr + 16 * c, v);
                tc_wait_ld();
                if (n < p.N) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int t = t0 + 16 * c + j;
                        if (t < p.M) {
                            int32_t* dst = p.acc + (int64_t)t * p.N + n;
                            if (p.use_atomics) atomicAdd(dst, (int32_t)v[j]);
                            else *dst = (int32_t)v[j];
                        }
                    }
                }
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

// -------------------------------------------------------------------------------------------------
// epilogue from the raw int32 accumulator: acc = -D/64 - qsum; out = bf16(alpha * s * acc + U.T + mu * s * qsum)
// -------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) finalize_kernel(GemmArgs a, int32_t* raw) {
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= a.M * a.N) return;
    const int64_t t = idx / a.N, n = idx - t * a.N;
    const int32_t d = raw[idx];
    const int32_t qs = a.qsum[t];
    const int32_t acc = -(d >> 6) - qs;
    if (a.acc_debug) a.acc_debug[idx] = acc;        // may alias raw: same element, read before written
    if (a.out) {
        const float sc = a.scales[t];
        float y = __fmul_rn(__fmul_rn(a.alpha[n], sc), (float)acc);
        if (a.r > 0) {
            const __nv_bfloat16* u = (const __nv_bfloat16*)a.U + n * a.r;
            const float* tr = a.T + t * a.r;
            float l = 0.f;
            for (int j = 0; j < a.r; ++j) l = fmaf(__bfloat162float(u[j]), tr[j], l);
            y += l;
        }
        if (a.mu) y = fmaf(__fmul_rn(a.mu[n], sc), (float)qs, y);
        ((__nv_bfloat16*)a.out)[t * a.ldo + n] = __float2bfloat16_rn(y);
    }
}

// -------------------------------------------------------------------------------------------------
// host side
// -------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

static int make_map_2d(CUtensorMap* map, CUtensorMapDataType dt, const void* base, uint64_t inner, uint64_t outer,
                       uint64_t row_stride_bytes, uint32_t box_inner, uint32_t box_outer, CUtensorMapSwizzle sw,
                       CUtensorMapL2promotion promo) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return BWLA_ERR_CUDA;
    cuuint64_t dims[2] = {inner, outer};
    cuuint64_t strides[1] = {row_stride_bytes};
    cuuint32_t box[2] = {box_inner, box_outer};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                    promo, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { g_last_cuda_error = (int)r; return BWLA_ERR_CUDA; }
    return BWLA_OK;
}

template <int N_TOK, int WS, int BS>
static int launch_umma_t(const CUtensorMap& wm, const CUtensorMap& bm, const UmmaParams& p, dim3 grid, cudaStream_t s) {
    using L = UmmaCfg<N_TOK, WS, BS>;
    constexpr int AS = L::AS;
    constexpr int SUBS = L::SUBS;
    static thread_local int configured = -1;
    int dev = 0;
    BWLA_CUDA_TRY(cudaGetDevice(&dev));
    if (configured != dev) {
        BWLA_CUDA_TRY(cudaFuncSetAttribute(umma_w1a_kernel<N_TOK, WS, BS>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::total));
        configured = dev;
    }
    ProfScope prof(kProfContraction, s);
    umma_w1a_kernel<N_TOK, WS, BS><<<grid, kThreads, L::total, s>>>(wm, bm, p);
    return after_launch();
}

bool umma_supports(int64_t M, int64_t K, int64_t N) {
    return M > 0 && N > 0 && K % 128 == 0 && M * N < (int64_t)1 << 31 && encode_tiled_fn() != nullptr;
}

// codes_interleaved: int8 [M][K] in the interleaved order.  raw: int32 [M][N] scratch (or the caller's acc_debug).
int launch_gemm_umma(const GemmArgs& a, const int8_t* codes_interleaved, int32_t* raw, cudaStream_t stream) {
    const int M = (int)a.M, N = (int)a.N, K = (int)a.K;
    const int n_tok = M <= 16 ? 16 : M <= 32 ? 32 : M <= 64 ? 64 : 128;
    const int row_tiles = (N + kRowsPerCta - 1) / kRowsPerCta;
    const int tok_tiles = (M + n_tok - 1) / n_tok;
    const int units = (K + kUnitK - 1) / kUnitK;
    // split K until there are about two CTAs per SM
    int split = 1;
    const int target = 148 * 2;
    while (split < units && row_tiles * tok_tiles * split < target) ++split;
    int ups = (units + split - 1) / split;
    split = (units + ups - 1) / ups;

    CUtensorMap wm, bm;
    int st = make_map_2d(&wm, CU_TENSOR_MAP_DATA_TYPE_UINT32, a.packed, (uint64_t)K / 32, (uint64_t)N, (uint64_t)K / 8,
                         32, kRowsPerCta, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
    if (st != BWLA_OK) return st;
    st = make_map_2d(&bm, CU_TENSOR_MAP_DATA_TYPE_UINT8, codes_interleaved, (uint64_t)K, (uint64_t)M, (uint64_t)K,
                     kBlockK, (uint32_t)n_tok, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
    if (st != BWLA_OK) return st;

    UmmaParams p{};
    p.M = M; p.N = N; p.K = K; p.total_units = units; p.units_per_split = ups; p.acc = raw;
    p.use_atomics = split > 1; p.status = a.status;
    if (split > 1) BWLA_CUDA_TRY(cudaMemsetAsync(raw, 0, (size_t)M * N * 4, stream));
    dim3 grid((unsigned)row_tiles, (unsigned)tok_tiles, (unsigned)split);
    switch (n_tok) {
        case 16: st = launch_umma_t<16, 3, 3>(wm, bm, p, grid, stream); break;
        case 32: st = launch_umma_t<32, 3, 3>(wm, bm, p, grid, stream); break;
        case 64: st = launch_umma_t<64, 3, 3>(wm, bm, p, grid, stream); break;
        default: st = launch_umma_t<128, 2, 4>(wm, bm, p, grid, stream); break;
    }
    if (st != BWLA_OK) return st;
    const int64_t total = (int64_t)M * N;
    ProfScope prof(kProfFinalize, stream);
    finalize_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(a, raw);
    return after_launch();
}

}  // namespace bwla
