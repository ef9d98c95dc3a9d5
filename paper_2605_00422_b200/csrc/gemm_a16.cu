// The weight-only operating point, W1A16 (Table 1, upper half: binarised weights, 16-bit activations): the rotated
// activation is kept in bf16 instead of being quantised to integer codes, and meets the packed signs on the tcgen05
// tensor cores as a bf16 contraction with fp32 accumulation:
//
//   yhat = bf16(Y)                                      (y_to_bf16_kernel; also sum_k yhat for the row-shift term)
//   out[t][n] = bf16( alpha[n] * sum_k s[n][k] * yhat[t][k] + U[n,:] . T[t,:] + mu[n] * sum_k yhat[t][k] )
//
// Tile of one CTA: 128 tokens (the accumulator's lanes) x 128 weight rows (its columns) x all of K.
//   A operand: yhat, K-major, by TMA (64 values of k = one 128-byte swizzle atom per stage);
//   B operand: the signs of 128 rows expanded to +-1 in bf16 by four warps (each owns one stage and takes every fourth
//              k-block: 64 bits in, eight 128-bit shared-memory stores out per row, swizzled K-major);
//   the tensor core adds each group of 16 products into its accumulator with truncation, so the accumulator only ever
//   holds 512 values of k (32 such additions: a bias of at most 2e-6 of the sum of magnitudes, far below the bf16
//   output): after every 512 it is read back and added, with rounded fp32 additions, into running sums in the epilogue
//   warps' registers while the next 512 go to the second accumulator (as in lowrank_umma.cu);
//   the low-rank term is twelve more MMAs (three bf16 terms of T against the tile's rows of U) into a third accumulator.
// Warp 0 copies, warp 1 allocates tensor memory and issues the MMAs, warps 2..5 expand signs and stage U, warps 6..13
// are the epilogue (two per quarter of the lanes, 64 columns each).  Every wait is bounded (umma_wait.cuh).
#include <cuda_bf16.h>

#include <algorithm>

#include "bwla_common.cuh"
#include "tensor_map.cuh"
#include "umma_ptx.cuh"
#include "umma_wait.cuh"

namespace bwla {

namespace a16 {
constexpr int kTok = 128, kRows = 128, kBlockK = 64, kFlushBlocks = 8;
// The yhat tiles come by TMA and take about a microsecond to land, the sign tiles are made on the SM: the ring of the
// former is deep (what bounds the loop is tiles in flight over that latency), the ring of the latter short.
constexpr int kAStages = 7, kBStages = 4;            // (an expander warp owns one sign stage: kBStages == 4 warps)
constexpr int kExpFirst = 64, kEpiFirst = 192, kThreads = 448;
constexpr int a_bytes = kTok * 128, b_bytes = kRows * 128;
constexpr int b_off = kAStages * a_bytes;
constexpr int u_off = b_off + kBStages * b_bytes;
constexpr int par_off = u_off + kRows * 128;                  // alpha[128], mu[128]
constexpr int bars_off = par_off + 2 * kRows * 4;
constexpr int smem_bytes = bars_off + 256 + 1024;
constexpr int ACC_COL = 0, LR_COL = 2 * kRows, kTmemCols = 512;
static_assert(smem_bytes <= 232448, "shared memory");
}  // namespace a16

struct A16Params {
    int M, N, K, r;
    const uint32_t* packed;
    const float* alpha; const float* mu; const float* ysum;
    const __nv_bfloat16* U;
    __nv_bfloat16* out; int64_t ldo;
    uint32_t* status;
};

// One block per token: Y (fp32) -> bf16, and the sum of the rounded values (fp64 accumulation, one fp32 result).
__global__ void __launch_bounds__(256) y_to_bf16_kernel(const float* __restrict__ Y, int64_t K, __nv_bfloat16* __restrict__ yhat,
                                                       float* __restrict__ ysum) {
    __shared__ double red[8];
    const int64_t t = blockIdx.x;
    double s = 0.0;
    for (int64_t k = threadIdx.x; k < K; k += blockDim.x) {
        const __nv_bfloat16 v = __float2bfloat16_rn(Y[t * K + k]);
        yhat[t * K + k] = v;
        s += (double)__bfloat162float(v);
    }
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        double a = 0.0;
        for (int i = 0; i < (int)(blockDim.x >> 5); ++i) a += red[i];
        ysum[t] = (float)a;
    }
}

// Eight sign bits (bit 1 = +1), given inverted in the low byte of `nbits` -> eight bf16 values +-1, two per word, the
// lower k in the low half.  A pair of inverted bits t = b0 + 2 b1 times (2^15 + 2^30) puts b0 at bit 15 and b1 at bit
// 31 (and copies at bits 16 and 30, masked off): three instructions per word.
__device__ __forceinline__ uint4 expand8(uint32_t nbits) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) w[i] = 0x3F803F80u | ((((nbits >> (2 * i)) & 3u) * 0x40008000u) & 0x80008000u);
    return make_uint4(w[0], w[1], w[2], w[3]);
}

__global__ void __launch_bounds__(a16::kThreads, 1)
a16_gemm_kernel(const __grid_constant__ CUtensorMap y_map, const __grid_constant__ CUtensorMap t_map, const A16Params p) {
    using namespace a16;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* ubuf = smem + u_off;
    float* alpha_s = reinterpret_cast<float*>(smem + par_off);
    float* mu_s = alpha_s + kRows;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + bars_off);
    uint64_t* a_full = bars;                  // [kAStages] yhat tile landed
    uint64_t* a_empty = a_full + kAStages;    // [kAStages] the MMAs that read it have completed
    uint64_t* b_full = a_empty + kAStages;    // [kBStages] signs expanded
    uint64_t* b_empty = b_full + kBStages;    // [kBStages]
    uint64_t* acc_full = b_empty + kBStages;  // [2]
    uint64_t* acc_free = acc_full + 2;        // [2]
    uint64_t* u_full = acc_free + 2;
    uint64_t* t_full = u_full + 1;
    uint64_t* lr_full = t_full + 1;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(lr_full + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = (int)blockIdx.x * kRows, t0 = (int)blockIdx.y * kTok;
    const int nblocks = p.K / kBlockK;
    const int units = (nblocks + kFlushBlocks - 1) / kFlushBlocks;
    const bool lowrank = p.r > 0;

    if (threadIdx.x == 0) {
        *abort_flag = (p.status && *reinterpret_cast<volatile uint32_t*>(p.status) != 0) ? 1 : 0;   // the call already failed
        for (int i = 0; i < kAStages; ++i) { mbar_init(&a_full[i], 1); mbar_init(&a_empty[i], 1); }
        for (int i = 0; i < kBStages; ++i) { mbar_init(&b_full[i], 1); mbar_init(&b_empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&acc_full[i], 1); mbar_init(&acc_free[i], 8); }
        mbar_init(u_full, 4); mbar_init(t_full, 1); mbar_init(lr_full, 1);
        fence_barrier_init();
        fence_proxy_async();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, kTmemCols);
        tmem_relinquish();
    }
    if (threadIdx.x >= kEpiFirst && threadIdx.x < kEpiFirst + kRows) {
        const int i = threadIdx.x - kEpiFirst, n = n0 + i;
        alpha_s[i] = n < p.N ? p.alpha[n] : 0.f;
        mu_s[i] = (p.mu && n < p.N) ? p.mu[n] : 0.f;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---------------- copies: the yhat tile stage by stage, then the three terms of T into the next three slots ----------------
        if (elect_one()) {
            tma_prefetch_desc(&y_map);
            if (lowrank) tma_prefetch_desc(&t_map);
            int s = 0; uint32_t ph = 0;
            bool ok = !*abort_flag;
            for (int b = 0; b < nblocks && ok && !*abort_flag; ++b) {
                if (!wait_or_abort(&a_empty[s], ph ^ 1u, abort_flag)) { give_up(p.status, abort_flag, 0x310); ok = false; break; }
                mbar_expect_tx(&a_full[s], a_bytes);
                tma_load_2d(smem + s * a_bytes, &y_map, b * kBlockK, t0, &a_full[s]);
                if (++s == kAStages) { s = 0; ph ^= 1u; }
            }
            if (lowrank && ok && !*abort_flag) {
                mbar_expect_tx(t_full, 3 * a_bytes);
                for (int h = 0; h < 3 && ok; ++h) {
                    if (!wait_or_abort(&a_empty[s], ph ^ 1u, abort_flag)) { give_up(p.status, abort_flag, 0x311); ok = false; break; }
                    tma_load_3d(smem + s * a_bytes, &t_map, 0, t0, h, t_full);
                    if (++s == kAStages) { s = 0; ph ^= 1u; }
                }
            }
            if (*abort_flag) for (int i = 0; i < 500; ++i) __nanosleep(100);   // let copies in flight land
        }
    } else if (warp == 1) {
        // ---------------- MMA issue ----------------
        if (elect_one()) {
            // D = f32, A = B = bf16, both K-major, M = 128, N = 128
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kRows >> 3) << 17) | ((128u >> 4) << 24);
            const uint64_t desc0 = smem_desc_sw128(0u, 0u);                         // everything but the start address
            const uint32_t desc_hi = (uint32_t)(desc0 >> 32);
            const uint32_t a_lo0 = (uint32_t)desc0 | ((smem_u32(smem) & 0x3FFFFu) >> 4);
            const uint32_t b_lo0 = (uint32_t)desc0 | ((smem_u32(smem + b_off) & 0x3FFFFu) >> 4);
            int sa = 0, sb = 0; uint32_t pha = 0, phb = 0;
            bool ok = !*abort_flag;
            int b = 0;
            for (int u = 0; u < units && ok; ++u) {
                const int buf = u & 1;
                if (u >= 2 && !wait_or_abort(&acc_free[buf], (uint32_t)(((u >> 1) - 1) & 1), abort_flag)) { give_up(p.status, abort_flag, 0x320); ok = false; break; }
                tc_fence_after();
                const uint32_t d_addr = tmem_base + ACC_COL + (uint32_t)(buf * kRows);
                for (int i = 0; i < kFlushBlocks && b < nblocks; ++i, ++b) {
                    if (!wait_or_abort(&a_full[sa], pha, abort_flag)) { give_up(p.status, abort_flag, 0x321); ok = false; break; }
                    if (!wait_or_abort(&b_full[sb], phb, abort_flag)) { give_up(p.status, abort_flag, 0x322); ok = false; break; }
                    tc_fence_after();
                    // (this thread is a chain of dependent scalar instructions: descriptors are a constant high word and a
                    // low word that only takes additions)
                    const uint32_t a_lo = a_lo0 + (uint32_t)sa * (a_bytes >> 4), g_lo = b_lo0 + (uint32_t)sb * (b_bytes >> 4);
                    if (i == 0) mma_f16_ss_words<false>(d_addr, a_lo, desc_hi, g_lo, desc_hi, idesc);
                    else mma_f16_ss_words<true>(d_addr, a_lo, desc_hi, g_lo, desc_hi, idesc);
#pragma unroll
                    for (int j = 1; j < 4; ++j)
                        mma_f16_ss_words<true>(d_addr, a_lo + 2u * j, desc_hi, g_lo + 2u * j, desc_hi, idesc);
                    tc_commit(&a_empty[sa]);
                    tc_commit(&b_empty[sb]);
                    if (++sa == kAStages) { sa = 0; pha ^= 1u; }
                    if (++sb == kBStages) { sb = 0; phb ^= 1u; }
                }
                if (ok) tc_commit(&acc_full[buf]);
            }
            if (ok && lowrank) {
                if (!wait_or_abort(u_full, 0, abort_flag)) { give_up(p.status, abort_flag, 0x323); ok = false; }
                if (ok && !wait_or_abort(t_full, 0, abort_flag)) { give_up(p.status, abort_flag, 0x324); ok = false; }
                if (ok) {
                    tc_fence_after();
                    const uint32_t u_addr = smem_u32(ubuf);
#pragma unroll
                    for (int h = 0; h < 3; ++h) {
                        // (the terms of T sit in the three slots of the yhat ring that follow the last yhat tile)
                        const uint32_t t_addr = smem_u32(smem + sa * a_bytes);
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            mma_f16_ss(tmem_base + LR_COL, smem_desc_sw128(t_addr, 32 * j), smem_desc_sw128(u_addr, 32 * j), idesc,
                                       (h | j) ? 1u : 0u);
                        if (++sa == kAStages) sa = 0;
                    }
                    tc_commit(lr_full);
                }
            }
        }
    } else if (warp < 6) {
        // ---------------- signs of the tile's 128 rows -> +-1 in bf16, K-major, swizzled; then the rows of U ----------------
        // Expander warp w takes the k-blocks w, w + 4, ... and owns sign stage w: what a warp does per block (wait for
        // its stage, 32 stores, the fence that makes them visible to the tensor core's reads, the hand-over) is a serial
        // chain of several hundred cycles whatever its size, so four blocks are in the making at once.  A lane expands
        // the rows lane, lane + 32, lane + 64, lane + 96 of the tile.
        const int w = warp - 2;
        const int row = threadIdx.x - kExpFirst;            // (for the rows of U below)
        const int n = n0 + row;
        const bool valid = n < p.N;
        const uint2* words[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int ni = n0 + lane + 32 * i;
            words[i] = reinterpret_cast<const uint2*>(p.packed + (size_t)(ni < p.N ? ni : 0) * (size_t)(p.K >> 5));
        }
        bool ok = !*abort_flag;
        uint2 nxt[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) nxt[i] = (ok && w < nblocks) ? __ldg(words[i] + w) : make_uint2(0u, 0u);
        uint8_t* const stage = smem + b_off + w * b_bytes;
        for (int b = w; b < nblocks && ok; b += kBStages) {
            uint2 cur[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                cur[i] = make_uint2(~nxt[i].x, ~nxt[i].y);            // inverted once: a set bit now means -1
                if (b + kBStages < nblocks) nxt[i] = __ldg(words[i] + b + kBStages);
            }
            if (!warp_wait(&b_empty[w], (uint32_t)(((b >> 2) & 1) ^ 1), abort_flag)) { give_up(p.status, abort_flag, 0x330); ok = false; break; }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int r = lane + 32 * i;
                uint8_t* dst = stage + r * 128;
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const uint32_t byte = ((c < 4 ? cur[i].x : cur[i].y) >> (8 * (c & 3))) & 0xFFu;
                    *reinterpret_cast<uint4*>(dst + ((c ^ (r & 7)) << 4)) = expand8(byte);
                }
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(&b_full[w]);
        }
        if (ok && lowrank) {
            // this tile's rows of U: 128 rows x 8 chunks of 16 bytes, 128B-swizzled K-major, zero beyond N and r
            const bool vec = (p.r % 8 == 0) && ((reinterpret_cast<uintptr_t>(p.U) & 15) == 0);
#pragma unroll
            for (int ch = 0; ch < 8; ++ch) {
                uint4 v = make_uint4(0u, 0u, 0u, 0u);
                if (valid && ch * 8 < p.r) {
                    const __nv_bfloat16* src = p.U + (int64_t)n * p.r + ch * 8;
                    if (vec) {
                        v = __ldg(reinterpret_cast<const uint4*>(src));
                    } else {
                        uint32_t w[4] = {0u, 0u, 0u, 0u};
                        for (int c = 0; c < 8 && ch * 8 + c < p.r; ++c)
                            w[c >> 1] |= (uint32_t)__bfloat16_as_ushort(src[c]) << (16 * (c & 1));
                        v = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
                *reinterpret_cast<uint4*>(ubuf + row * 128 + ((ch ^ (row & 7)) << 4)) = v;
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(u_full);
        }
    } else {
        // ---------------- epilogue: running sums, then scale, low-rank term, row shift, bf16 ----------------
        const int q = warp & 3;
        const int half = (warp - 6) >> 2;                  // which 64 columns of the tile
        const int lane_d = q * 32 + lane;                  // token of the tile
        const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
        const int64_t t = (int64_t)t0 + lane_d;
        float run[64];
#pragma unroll
        for (int c = 0; c < 64; ++c) run[c] = 0.f;
        bool ok = !*abort_flag;
        for (int u = 0; u < units && ok; ++u) {
            const int buf = u & 1;
            if (!warp_wait(&acc_full[buf], (uint32_t)((u >> 1) & 1), abort_flag)) { give_up(p.status, abort_flag, 0x340); ok = false; break; }
            tc_fence_after();
            // two batches of 32 columns: the loads of a batch are in flight together, the registers stay few
#pragma unroll
            for (int hb = 0; hb < 2; ++hb) {
                uint32_t v[2][16];
#pragma unroll
                for (int c = 0; c < 2; ++c)
                    tmem_ld_32x16(tmem_base + lane_addr + (uint32_t)(ACC_COL + buf * kRows + 64 * half + 32 * hb + 16 * c), v[c]);
                tc_wait_ld();
                if (hb == 1) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&acc_free[buf]);
                }
#pragma unroll
                for (int c = 0; c < 2; ++c)
#pragma unroll
                    for (int i = 0; i < 16; ++i) run[32 * hb + 16 * c + i] += __uint_as_float(v[c][i]);
            }
        }
        if (ok && lowrank && !warp_wait(lr_full, 0, abort_flag)) { give_up(p.status, abort_flag, 0x341); ok = false; }
        if (ok && lowrank) tc_fence_after();
        // (the tensor-memory loads below are warp-wide instructions: every lane of the warp executes them, whether or
        // not its token exists; only the stores look at the token)
        if (ok) {
            const bool live = t < p.M;
            const float ys = live ? p.ysum[t] : 0.f;
            const int c0 = 64 * half;
            __nv_bfloat16* dst = p.out + (live ? t : 0) * p.ldo + n0 + c0;
            const bool vec = ((reinterpret_cast<uintptr_t>(p.out) & 15) == 0) && (p.ldo % 8 == 0) && (n0 + c0 + 64 <= p.N);
#pragma unroll
            for (int c16 = 0; c16 < 4; ++c16) {
                uint32_t l[16];
                if (lowrank) {
                    tmem_ld_32x16(tmem_base + lane_addr + (uint32_t)(LR_COL + c0 + 16 * c16), l);
                    tc_wait_ld();
                } else {
#pragma unroll
                    for (int i = 0; i < 16; ++i) l[i] = 0u;
                }
#pragma unroll
                for (int g8 = 0; g8 < 2; ++g8) {
                    uint32_t w[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int cl = 8 * g8 + 2 * i, c = 16 * c16 + cl;
                        const float y0 = fmaf(mu_s[c0 + c], ys, fmaf(alpha_s[c0 + c], run[c], __uint_as_float(l[cl])));
                        const float y1 = fmaf(mu_s[c0 + c + 1], ys, fmaf(alpha_s[c0 + c + 1], run[c + 1], __uint_as_float(l[cl + 1])));
                        w[i] = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(y0)) |
                               ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(y1)) << 16);
                    }
                    const int cb = 16 * c16 + 8 * g8;
                    if (!live) continue;
                    if (vec) {
                        *reinterpret_cast<uint4*>(dst + cb) = make_uint4(w[0], w[1], w[2], w[3]);
                    } else {
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            if (n0 + c0 + cb + i < p.N)
                                dst[cb + i] = __ushort_as_bfloat16((unsigned short)((w[i >> 1] >> (16 * (i & 1))) & 0xFFFFu));
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

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
bool a16_supports(int64_t M, int64_t K, int64_t N, int r) {
    return M >= 1 && N >= 1 && K % a16::kBlockK == 0 && r >= 0 && r <= kLowrankPad && M < ((int64_t)1 << 31);
}

int launch_y_to_bf16(const float* Y, int64_t M, int64_t K, void* yhat, float* ysum, cudaStream_t stream) {
    ProfScope prof(kProfRotateQuant, stream);
    y_to_bf16_kernel<<<(unsigned)M, 256, 0, stream>>>(Y, K, (__nv_bfloat16*)yhat, ysum);
    return after_launch();
}

int launch_gemm_a16(const void* yhat, const float* ysum, int64_t M, int64_t K, int64_t N, const uint32_t* packed, const float* alpha,
                    const float* mu, const void* U, int r, const void* Thl, void* out, int64_t ldo, uint32_t* status,
                    cudaStream_t stream) {
    using namespace a16;
    CUtensorMap ym, tm;
    {
        const uint64_t dims[2] = {(uint64_t)K, (uint64_t)M};
        const uint64_t strides[1] = {(uint64_t)K * 2};
        const uint32_t box[2] = {kBlockK, kTok};
        int st = make_map(&ym, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, yhat, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
        if (st != BWLA_OK) return st;
    }
    if (r > 0) {
        const uint64_t dims[3] = {(uint64_t)kLowrankPad, (uint64_t)M, 3};
        const uint64_t strides[2] = {(uint64_t)kLowrankPad * 2, (uint64_t)M * kLowrankPad * 2};
        const uint32_t box[3] = {(uint32_t)kLowrankPad, kTok, 1};
        int st = make_map(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, Thl, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
        if (st != BWLA_OK) return st;
    } else {
        tm = ym;   // never dereferenced
    }
    A16Params p{};
    p.M = (int)M; p.N = (int)N; p.K = (int)K; p.r = r; p.packed = packed; p.alpha = alpha; p.mu = mu; p.ysum = ysum;
    p.U = (const __nv_bfloat16*)U; p.out = (__nv_bfloat16*)out; p.ldo = ldo; p.status = status;
    static thread_local int configured = -1;
    int dev = 0;
    BWLA_CUDA_TRY(cudaGetDevice(&dev));
    if (configured != dev) {
        BWLA_CUDA_TRY(cudaFuncSetAttribute(a16_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes));
        configured = dev;
    }
    const dim3 grid((unsigned)((N + kRows - 1) / kRows), (unsigned)((M + kTok - 1) / kTok), 1);
    ProfScope prof(kProfContraction, stream);
    a16_gemm_kernel<<<grid, kThreads, smem_bytes, stream>>>(ym, tm, p);
    return after_launch();
}

}  // namespace bwla
