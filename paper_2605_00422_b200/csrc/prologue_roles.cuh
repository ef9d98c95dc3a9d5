// Pieces of the per-call prologue that more than one kernel uses: the parameter block, warp reductions, the split of an
// fp32 value into three bf16 terms, and the blocks that evaluate the first stage of the PSP low-rank branch,
// T = V x (Sec. 3.2: W x = (W - M) x + A (B x)).
#pragma once

#include <cuda_bf16.h>

#include <algorithm>

#include "bwla_common.cuh"
#include "umma_ptx.cuh"

namespace bwla {

using namespace ptx;

constexpr int kLrMaxWarps = 16;   // blocks have at most 512 threads

struct PrologueParams {
    const __nv_bfloat16* x; int64_t M; int K; int64_t ldx;
    // rotation + quantiser (rot_blocks == 0 skips them)
    const float* P1; int n1; const float* P2; int n2; int bits;
    int8_t* codes; int codes_layout; float* scales; int32_t* qsum;
    int C;              // CTAs per token (cluster size)
    int rot_blocks;     // clusters * C
    int tok_stride;     // number of clusters: a cluster takes tokens t, t + tok_stride, ... (== M unless the clusters stay and loop)
    int rot_first;      // first rotation block: 0, or (clusters that stay) behind the low-rank blocks, which then start first
    int row_gran;       // slab boundaries are multiples of this many rows of X
    int slab_cap;       // floats reserved for one slab
    int ps_cap;         // floats reserved for a staged chunk of P2 / P1
    int ch1, ch2;       // columns of P2 / of P1 staged at a time
    int prefetch;       // 1: all of P2 and this CTA's columns of P1 are fetched at the start, with x
    int p1_cap;         // floats reserved for the prefetched columns of P1
    int tr1, tr2;       // rows per thread in the two contractions
    int split_y;        // 1 (C > 1): each CTA evaluates its rows of Y from all of x, nothing but absmax is exchanged
    int sp_tr, sp_rp;   // split_y: rows per thread tile (4 or 8); slab rows rounded up to it (row stride of P1s and Zt)
    int sp_s;           // split_y: slices the contraction depth is cut into (partial sums are added afterwards); with sp_tc:
                        // parts the columns of P2 are staged in
    int sp_tc;          // split_y: 1: both contractions on the warp-level tensor-core path (split-bf16 operands)
    int sp_zt_off;      // split_y: where Z'^T lives, in floats from the start of shared memory (0: over x, dead by then)
    int sp_rest_off;    // split_y: where P2 starts
    // low-rank
    const __nv_bfloat16* V; int r; int lr_cols; __nv_bfloat16* Thl;   // [3][M][lr_cols]
    int lr_wide;        // low-rank blocks: 0: 2 rows of V x 16 tokens (FMA), 1: 8 x 8 (FMA, many tokens), 2: 8 columns x 16 tokens on the
                        // warp-level tensor-core path (few tokens), 3: all 64 columns x 16 tokens on that path (many tokens)
    int lr_ks;          // lr_wide == 2: blocks that share a tile of T and split K (1: no split)
    float* lr_part;     // [tiles][lr_ks][16 * 8] partial sums of those blocks
    uint32_t* lr_count; // one arrival counter per tile, zero between calls
    int lr_stage;       // 1: a low-rank block copies its rows of V into shared memory before it waits for x
    int late_trigger;   // 1: the next kernel of the stream is let in only when this one is nearly done (see launch_prologue)
};

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
    return v;
}

__device__ __forceinline__ int warp_sum(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// ---------------------------------------------------------------------------------------------
// The two slab contractions on the warp-level tensor-core path (mma.sync m16n8k16, bf16 in, fp32 out).
//
// An fp32 factor is split into three bf16 terms (hi + mid + lo carry all 24 bits); x is bf16 already.  Every k-step of
// 16 starts from a zero accumulator, takes the products of the terms that matter (smallest first) and is then added to
// the running fp32 sum with an ordinary rounded addition: the tensor core only ever sums 16 exact products (48 or 96
// with the terms), so what its internal accumulation does to long sums does not enter.  The error stays at the level
// of the fp32 FMA chain (a CPU model of this scheme with the partial sums rounded toward zero is within 3.4e-7 of the
// token's full scale for K = 25600, the fp32 chain within 5.9e-7; the code window is 1e-6).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void split3(float v, __nv_bfloat16& h, __nv_bfloat16& m, __nv_bfloat16& l) {
    h = __float2bfloat16_rn(v);
    const float r1 = v - __bfloat162float(h);
    m = __float2bfloat16_rn(r1);
    l = __float2bfloat16_rn(r1 - __bfloat162float(m));
}

__device__ __forceinline__ uint32_t pack_bf16(__nv_bfloat16 a, __nv_bfloat16 b) {
    return (uint32_t)__bfloat16_as_ushort(a) | ((uint32_t)__bfloat16_as_ushort(b) << 16);
}

// ---------------------------------------------------------------------------------------------
// T = V x, written as three bf16 terms
// ---------------------------------------------------------------------------------------------
// acc += dot of eight bf16 pairs (two packed 128-bit words)
__device__ __forceinline__ float dot8(float acc, const uint4& v, const uint4& xv) {
    const uint32_t a[4] = {v.x, v.y, v.z, v.w}, b[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        acc = fmaf(__uint_as_float(a[i] << 16), __uint_as_float(b[i] << 16), acc);
        acc = fmaf(__uint_as_float(a[i] & 0xFFFF0000u), __uint_as_float(b[i] & 0xFFFF0000u), acc);
    }
    return acc;
}

// One block reduces R rows of V against T tokens (R x T accumulators per thread, threads stride over K).  Few tokens:
// R = 2, T = 16 (many blocks).  Many tokens: R = T = 8, which reads each operand four times less often from L2.
template <int R, int T>
static __device__ void lowrank_role(const PrologueParams& p, int b, float* smem) {
    const int jblocks = p.lr_cols / R;
    const int jb = b % jblocks;
    const int64_t t0 = (int64_t)(b / jblocks) * T;
    if (t0 >= p.M) return;
    const int j0 = jb * R;
    const int nt = (int)min((int64_t)T, p.M - t0);
    float (*red)[R * T] = reinterpret_cast<float (*)[R * T]>(smem);            // [kLrMaxWarps][R * T]
    const uint4* vs = reinterpret_cast<const uint4*>(smem + kLrMaxWarps * R * T);   // staged rows of V, [R][K / 8]
    float acc[R][T];
#pragma unroll
    for (int j = 0; j < R; ++j)
#pragma unroll
        for (int i = 0; i < T; ++i) acc[j][i] = 0.f;
    const int K = p.K;
    const int nr = min(R, p.r - j0);                          // rows of V this block really has (<= 0: padding only)
    const bool vec = ((reinterpret_cast<uintptr_t>(p.V) | reinterpret_cast<uintptr_t>(p.x)) & 15) == 0 && (p.ldx & 7) == 0 && (K & 7) == 0;
    const bool staged = p.lr_stage && vec && nr > 0;
    if (staged) {
        // V is a constant of the layer: in shared memory before the activations exist
        uint4* dst = reinterpret_cast<uint4*>(smem + kLrMaxWarps * R * T);
        for (int j = 0; j < R; ++j) {
            const uint4* src = reinterpret_cast<const uint4*>(p.V + (int64_t)(j0 + min(j, nr - 1)) * K);
            for (int kc = threadIdx.x; kc < (K >> 3); kc += blockDim.x) dst[j * (K >> 3) + kc] = __ldg(src + kc);
        }
    }
    griddep_launch_dependents();
    griddep_wait();                                           // x may be the output of the preceding kernel
    if (nr > 0) {
        const __nv_bfloat16* vrow[R];
#pragma unroll
        for (int j = 0; j < R; ++j) vrow[j] = p.V + (int64_t)(j0 + min(j, nr - 1)) * K;
        const __nv_bfloat16* xt = p.x + t0 * p.ldx;
        if (vec) {
            for (int kc = threadIdx.x; kc < (K >> 3); kc += blockDim.x) {
                uint4 a[R];
#pragma unroll
                for (int j = 0; j < R; ++j) a[j] = staged ? vs[j * (K >> 3) + kc] : __ldg(reinterpret_cast<const uint4*>(vrow[j]) + kc);
#pragma unroll
                for (int tt = 0; tt < T; ++tt) {
                    if (tt < nt) {
                        const uint4 xv = __ldg(reinterpret_cast<const uint4*>(xt + tt * p.ldx) + kc);
#pragma unroll
                        for (int j = 0; j < R; ++j) acc[j][tt] = dot8(acc[j][tt], a[j], xv);
                    }
                }
            }
        } else {
            for (int k = threadIdx.x; k < K; k += blockDim.x) {
                float a[R];
#pragma unroll
                for (int j = 0; j < R; ++j) a[j] = __bfloat162float(vrow[j][k]);
#pragma unroll
                for (int tt = 0; tt < T; ++tt) {
                    if (tt < nt) {
                        const float xv = __bfloat162float(xt[tt * p.ldx + k]);
#pragma unroll
                        for (int j = 0; j < R; ++j) acc[j][tt] = fmaf(a[j], xv, acc[j][tt]);
                    }
                }
            }
        }
#pragma unroll
        for (int j = 0; j < R; ++j)
            if (j >= nr) {
#pragma unroll
                for (int i = 0; i < T; ++i) acc[j][i] = 0.f;
            }
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int j = 0; j < R; ++j)
#pragma unroll
        for (int i = 0; i < T; ++i) {
            float v = acc[j][i];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
            if (lane == 0) red[warp][j * T + i] = v;
        }
    __syncthreads();
    for (int o = threadIdx.x; o < R * T; o += blockDim.x) {
        const int j = o / T, i = o % T;
        if (i < nt) {
            float s = 0.f;
            for (int w = 0; w < (int)(blockDim.x >> 5); ++w) s += red[w][o];
            // three bf16 terms carry all 24 bits of the fp32 sum
            const __nv_bfloat16 hi = __float2bfloat16_rn(s);
            const float r1 = s - __bfloat162float(hi);
            const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
            const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
            const int64_t at = (t0 + i) * p.lr_cols + j0 + j;
            p.Thl[at] = hi;
            p.Thl[p.M * p.lr_cols + at] = mid;
            p.Thl[2 * p.M * p.lr_cols + at] = lo;
        }
    }
}

// Few tokens: T for a tile of 16 tokens x 8 columns per block on the warp-level tensor-core path
// (mma.sync m16n8k16, bf16 in, fp32 accumulate): far fewer instructions than the FMA version, so these blocks do not
// take issue slots from the rotation blocks they share SMs with.  The warps of the block split K in chunks of 32; a
// lane reads 16 bytes of two token rows and of one row of V per chunk, and the chunk is contracted by two MMAs whose
// k order is permuted the same way for both operands (a sum over k does not care).  Partial tiles are added across
// the warps in shared memory in warp order.
__device__ __forceinline__ void mma_bf16_16x8x16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                 uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

static __device__ void lowrank_mma_role(const PrologueParams& p, int b, float* smem) {
    const int jtiles = p.lr_cols / 8;
    const int KS = p.lr_ks;
    const int j0 = (b % jtiles) * 8;
    const int ks = (b / jtiles) % KS;
    const int64_t t0 = (int64_t)(b / (jtiles * KS)) * 16;
    if (t0 >= p.M) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int g = lane >> 2, tg = lane & 3;
    const int K = p.K;
    griddep_launch_dependents();
    griddep_wait();                                           // x may be the output of the preceding kernel
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    if (j0 < p.r) {
        const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
        const bool row_lo = t0 + g < p.M, row_hi = t0 + g + 8 < p.M, col = j0 + g < p.r;
        const uint4* xlo = reinterpret_cast<const uint4*>(p.x + (t0 + (row_lo ? g : 0)) * p.ldx) + tg;
        const uint4* xhi = reinterpret_cast<const uint4*>(p.x + (t0 + (row_hi ? g + 8 : 0)) * p.ldx) + tg;
        const uint4* vj = reinterpret_cast<const uint4*>(p.V + (int64_t)(j0 + (col ? g : 0)) * K) + tg;
        const int chunks = K >> 5;
        const int c_lo = (int)((int64_t)chunks * ks / KS), c_hi = (int)((int64_t)chunks * (ks + 1) / KS);
        // The tensor core adds each group of 16 products into the accumulator with truncation; over the hundreds of
        // steps of a large K that bias would reach 1e-5 of the sum.  Every four chunks the accumulator is added into a
        // running fp32 sum with an ordinary rounded addition and starts from zero again.
        float run[4] = {0.f, 0.f, 0.f, 0.f};
        int since = 0;
#pragma unroll 4
        for (int c = c_lo + warp; c < c_hi; c += nwarps) {
            const uint4 a = row_lo ? __ldg(xlo + 4 * c) : zero;
            const uint4 h = row_hi ? __ldg(xhi + 4 * c) : zero;
            const uint4 v = col ? __ldg(vj + 4 * c) : zero;
            mma_bf16_16x8x16(acc, a.x, h.x, a.y, h.y, v.x, v.y);
            mma_bf16_16x8x16(acc, a.z, h.z, a.w, h.w, v.z, v.w);
            if (++since == 4) {
                since = 0;
#pragma unroll
                for (int i = 0; i < 4; ++i) { run[i] += acc[i]; acc[i] = 0.f; }
            }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[i] += run[i];
    }
    // acc: (token g, columns 2tg, 2tg+1), (token g+8, same columns)
    float* red = smem;                                        // [nwarps][16 * 8]
    red[warp * 128 + g * 8 + 2 * tg] = acc[0];
    red[warp * 128 + g * 8 + 2 * tg + 1] = acc[1];
    red[warp * 128 + (g + 8) * 8 + 2 * tg] = acc[2];
    red[warp * 128 + (g + 8) * 8 + 2 * tg + 1] = acc[3];
    __syncthreads();
    if (KS > 1) {
        // Several blocks share this tile of T and split K.  Each leaves its partial tile in the workspace; the last one
        // to arrive adds them in the order of the K parts (so the result does not depend on who came last).
        const int tile = (int)(b / (jtiles * KS)) * jtiles + (b % jtiles);
        float* mine = p.lr_part + ((size_t)tile * KS + ks) * 128;
        for (int o = threadIdx.x; o < 128; o += blockDim.x) {
            float s = 0.f;
            for (int w = 0; w < nwarps; ++w) s += red[w * 128 + o];
            mine[o] = s;
        }
        __threadfence();
        __syncthreads();
        __shared__ uint32_t arrived;
        if (threadIdx.x == 0) arrived = atomicAdd(p.lr_count + tile, 1u);
        __syncthreads();
        if (arrived != (uint32_t)(KS - 1)) return;
        __threadfence();
        for (int o = threadIdx.x; o < 128; o += blockDim.x) {
            const int i = o >> 3, j = o & 7;
            float s = 0.f;
            for (int k = 0; k < KS; ++k) s += __ldcg(p.lr_part + ((size_t)tile * KS + k) * 128 + o);
            if (t0 + i < p.M) {
                const __nv_bfloat16 hi = __float2bfloat16_rn(s);
                const float r1 = s - __bfloat162float(hi);
                const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
                const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
                const int64_t at = (t0 + i) * p.lr_cols + j0 + j;
                p.Thl[at] = hi;
                p.Thl[p.M * p.lr_cols + at] = mid;
                p.Thl[2 * p.M * p.lr_cols + at] = lo;
            }
        }
        if (threadIdx.x == 0) p.lr_count[tile] = 0;          // ready for the next call
        return;
    }
    for (int o = threadIdx.x; o < 128; o += blockDim.x) {
        const int i = o >> 3, j = o & 7;
        if (t0 + i < p.M) {
            float s = 0.f;
            for (int w = 0; w < nwarps; ++w) s += red[w * 128 + o];
            // three bf16 terms carry all 24 bits of the fp32 sum
            const __nv_bfloat16 hi = __float2bfloat16_rn(s);
            const float r1 = s - __bfloat162float(hi);
            const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
            const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
            const int64_t at = (t0 + i) * p.lr_cols + j0 + j;
            p.Thl[at] = hi;
            p.Thl[p.M * p.lr_cols + at] = mid;
            p.Thl[2 * p.M * p.lr_cols + at] = lo;
        }
    }
}

// Many tokens: the same on tiles of 16 tokens x all 64 columns, so that x is read once; a lane keeps the eight
// column tiles' accumulators (32 registers) and reads one row of V per column tile and chunk.
static __device__ void lowrank_mma_wide_role(const PrologueParams& p, int b, float* smem) {
    const int64_t t0 = (int64_t)b * 16;
    if (t0 >= p.M) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int g = lane >> 2, tg = lane & 3;
    const int K = p.K;
    const int ntiles = p.lr_cols / 8;                         // <= 8
    griddep_launch_dependents();
    griddep_wait();                                           // x may be the output of the preceding kernel
    float acc[8][4], run[8][4];
#pragma unroll
    for (int nt = 0; nt < 8; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) { acc[nt][i] = 0.f; run[nt][i] = 0.f; }
    int since = 0;
    {
        const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
        const bool row_lo = t0 + g < p.M, row_hi = t0 + g + 8 < p.M;
        const uint4* xlo = reinterpret_cast<const uint4*>(p.x + (t0 + (row_lo ? g : 0)) * p.ldx) + tg;
        const uint4* xhi = reinterpret_cast<const uint4*>(p.x + (t0 + (row_hi ? g + 8 : 0)) * p.ldx) + tg;
        const uint4* vbase = reinterpret_cast<const uint4*>(p.V) + tg;
        const int chunks = K >> 5;
#pragma unroll 2
        for (int c = warp; c < chunks; c += nwarps) {
            const uint4 a = row_lo ? __ldg(xlo + 4 * c) : zero;
            const uint4 h = row_hi ? __ldg(xhi + 4 * c) : zero;
            uint4 v[8];
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                const int j = 8 * nt + g;
                v[nt] = (nt < ntiles && j < p.r) ? __ldg(vbase + (size_t)j * (K >> 3) + 4 * c) : zero;
            }
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                mma_bf16_16x8x16(acc[nt], a.x, h.x, a.y, h.y, v[nt].x, v[nt].y);
                mma_bf16_16x8x16(acc[nt], a.z, h.z, a.w, h.w, v[nt].z, v[nt].w);
            }
            // short in-core sums only (see lowrank_mma_role): every four chunks into a rounded running sum
            if (++since == 4) {
                since = 0;
#pragma unroll
                for (int nt = 0; nt < 8; ++nt)
#pragma unroll
                    for (int i = 0; i < 4; ++i) { run[nt][i] += acc[nt][i]; acc[nt][i] = 0.f; }
            }
        }
#pragma unroll
        for (int nt = 0; nt < 8; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[nt][i] += run[nt][i];
    }
    // partial tiles of the warps, [warp][token 0..15][column 0..63], added in warp order
    float* red = smem;
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
        float* r = red + warp * 1024 + 8 * nt + 2 * tg;
        r[g * 64] = acc[nt][0]; r[g * 64 + 1] = acc[nt][1];
        r[(g + 8) * 64] = acc[nt][2]; r[(g + 8) * 64 + 1] = acc[nt][3];
    }
    __syncthreads();
    for (int o = threadIdx.x; o < 1024; o += blockDim.x) {
        const int i = o >> 6, j = o & 63;
        if (t0 + i < p.M && j < p.lr_cols) {
            float s = 0.f;
            for (int w = 0; w < nwarps; ++w) s += red[w * 1024 + o];
            // three bf16 terms carry all 24 bits of the fp32 sum
            const __nv_bfloat16 hi = __float2bfloat16_rn(s);
            const float r1 = s - __bfloat162float(hi);
            const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
            const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
            const int64_t at = (t0 + i) * p.lr_cols + j;
            p.Thl[at] = hi;
            p.Thl[p.M * p.lr_cols + at] = mid;
            p.Thl[2 * p.M * p.lr_cols + at] = lo;
        }
    }
}

// Host side: chooses the kind of low-rank blocks for the problem in p (x, M, K, ldx, V, r, lr_cols, Thl set), fills the
// lr_* fields and returns the number of blocks; *smem receives the dynamic shared memory one such block needs.
// lr_part / lr_count (either may be NULL): workspace for blocks that share a tile of T and split K.
inline int plan_lowrank(PrologueParams& p, float* lr_part, uint32_t* lr_count, size_t smem_limit, size_t* smem) {
    const int64_t M = p.M;
    const int K = p.K;
    // few tokens: the tensor-core version (needs 16-byte rows); many tokens: tiles that re-read little
    const bool rows16 = ((reinterpret_cast<uintptr_t>(p.x) | reinterpret_cast<uintptr_t>(p.V)) & 15) == 0 && p.ldx % 8 == 0 &&
                        K % 32 == 0 && p.lr_cols % 8 == 0;
    // (the wide tiles read x once but need enough token tiles to fill the device: 16 tokens x 64 columns per block)
    p.lr_wide = rows16 ? ((M >= 1024 && p.lr_cols == 64) ? 3 : 2) : ((M >= 64 && p.lr_cols % 8 == 0) ? 1 : 0);
    int blocks = p.lr_wide == 1 ? (p.lr_cols / 8) * (int)((M + 7) / 8)
               : p.lr_wide == 2 ? (p.lr_cols / 8) * (int)((M + 15) / 16)
               : p.lr_wide == 3 ? (int)((M + 15) / 16) : (p.lr_cols / 2) * (int)((M + 15) / 16);
    // One tile of 16 tokens and a large K: eight blocks would stream all of V (cold: from HBM) through eight SMs and
    // become the longest part of the launch; more blocks take a part of K each.
    p.lr_ks = 1; p.lr_part = lr_part; p.lr_count = lr_count;
    if (p.lr_wide == 2 && M <= 16 && lr_part && lr_count && p.lr_cols / 8 <= 8) {
        const int ksplit = (int)std::min<int64_t>(kLrKSplitMax, (K >> 5) / 100);
        if (ksplit > 1) { p.lr_ks = ksplit; blocks *= ksplit; }
    }
    // shared memory of a low-rank block: per-warp partial sums, and its rows of V when those are staged (few tokens)
    const size_t red_bytes = (size_t)kLrMaxWarps * 4 * (p.lr_wide == 3 ? 1024 : p.lr_wide == 2 ? 128 : 64);
    const size_t stage_bytes = (size_t)2 * (size_t)K * 2;
    p.lr_stage = (p.lr_wide == 0 && red_bytes + stage_bytes <= smem_limit) ? 1 : 0;
    *smem = red_bytes + (p.lr_stage ? stage_bytes : 0);
    return blocks;
}

}  // namespace bwla
