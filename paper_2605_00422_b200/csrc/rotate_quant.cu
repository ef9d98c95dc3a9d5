// The per-call prologue, one launch: online OKT + per-token symmetric quantiser, and the first stage of the PSP
// low-rank branch.
//
//   X = reshape(x_t, n1 x n2) (row-major), Z = X * P2, Y = P1^T * Z, amax = max|Y|,
//   q = clamp(rne(Y * (qmax / amax)), +-qmax), s_t = amax / qmax;          T[t][j] = sum_k V[j][k] * x_t[k]
//
// (Sec. 3.1: R = R1 (x) R2 evaluated as two small contractions on the reshaped vector; Sec. 4.1: per-token
// activation quantisation; Sec. 3.2: W x = (W - M) x + A (B x).)
//
// Rotation blocks.  Many tokens whose constants fit beside X and Z: one CTA per token evaluates Z = X * P2, Y = P1^T * Z
// with register-tiled fp32 FMA loops.  Few tokens: a thread-block cluster of C CTAs owns one token; CTA c owns a slab of
// rows of Y and evaluates the product in the other order, Z' = (P1^T X)[slab], Y[slab] = Z' * P2, which needs all of x (a
// few KB) but nothing from the other CTAs; only the absmax crosses the cluster (distributed shared memory).  Where the
// operands fit, these slab contractions run on the warp-level tensor-core path with fp32 factors split into three bf16
// terms (see tc_stage_a); a P2 too large for that keeps its fp32 form and only the first contraction does.  Many
// tokens of a large K: such clusters stay resident, keep the constants and take tokens in turn.  X, Z and Y never
// touch HBM; codes leave as 128-bit stores; the code sum of a token is left as one partial sum per CTA.
//
// Low-rank blocks (in the same grid): T = V x on the warp-level tensor-core path, tiles of 16 tokens x 8 (or 64)
// columns, written as three bf16 terms (T = hi + mid + lo, all 24 bits of the fp32 sum), the form the tensor-core
// epilogue of the contraction consumes.  (FMA versions remain for rows that are not 16-byte aligned.)
//
// The kernel is launched with programmatic stream serialisation.  The activations may be the output of the
// preceding kernel of the stream, so only the layer's own constants (P1, P2, rows of V) are fetched before that
// kernel has finished; x is read, and everything is stored, after it.
#include <cuda_bf16.h>

#include <algorithm>

#include "bwla_common.cuh"
#include "prologue_roles.cuh"
#include "umma_ptx.cuh"

namespace bwla {

constexpr int kPrologueSmemFloats = 57728;   // dynamic shared memory of a prologue block, in floats (225.5 KB; static use is under 1 KB)


__device__ __forceinline__ void st_cluster_u32(uint32_t addr, uint32_t v) {
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}

__device__ __forceinline__ int slab_begin(int c, int C, int n1, int gran) {
    if (c >= C) return n1;
    return (int)(((int64_t)n1 * c / C) / gran * gran);
}

// Z[0 .. rows)[dc .. dc+cw) = X * P2[:, dc .. dc+cw) for the `rows` rows of X at Xs.  Ps holds that chunk of P2 (row
// stride cw).  Each thread owns TR rows x 4 columns; the sum runs over b in increasing order.
template <int TR>
__device__ __forceinline__ void stage1_chunk(const float* __restrict__ Xs, int rows, int n2, const float* __restrict__ Ps,
                                             int dc, int cw, float* Zf, float* amax = nullptr) {
    const int ct = cw >> 2;
    const int tiles = ((rows + TR - 1) / TR) * ct;
    for (int tile = threadIdx.x; tile < tiles; tile += blockDim.x) {
        const int mt = tile / ct, dl = (tile - mt * ct) << 2;
        const int r0 = mt * TR;
        const float* xr[TR];
#pragma unroll
        for (int i = 0; i < TR; ++i) xr[i] = Xs + min(r0 + i, rows - 1) * n2;
        float acc[TR][4];
#pragma unroll
        for (int i = 0; i < TR; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
        const float* pp = Ps + dl;
#pragma unroll 2
        for (int b = 0; b < n2; b += 4) {
            float4 xa[TR];
#pragma unroll
            for (int i = 0; i < TR; ++i) xa[i] = *reinterpret_cast<const float4*>(xr[i] + b);
#pragma unroll
            for (int bb = 0; bb < 4; ++bb) {
                const float4 pv = *reinterpret_cast<const float4*>(pp + (b + bb) * cw);
#pragma unroll
                for (int i = 0; i < TR; ++i) {
                    const float x = bb == 0 ? xa[i].x : bb == 1 ? xa[i].y : bb == 2 ? xa[i].z : xa[i].w;
                    acc[i][0] = fmaf(x, pv.x, acc[i][0]);
                    acc[i][1] = fmaf(x, pv.y, acc[i][1]);
                    acc[i][2] = fmaf(x, pv.z, acc[i][2]);
                    acc[i][3] = fmaf(x, pv.w, acc[i][3]);
                }
            }
        }
#pragma unroll
        for (int i = 0; i < TR; ++i)
            if (r0 + i < rows) {
                const float4 v = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
                if (amax) *amax = fmaxf(*amax, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
                *reinterpret_cast<float4*>(Zf + (r0 + i) * n2 + dc + dl) = v;
            }
    }
}

// Y[c0 .. c0+cw)[all d] = sum_a P1[a][a_lo + c0 + .] * Z[a][d].  Ps holds P1[:, a_lo+c0 .. a_lo+c0+cw) with row
// stride cwp (cw rounded up to 4, padding zero).  Each thread owns TR output rows x 4 columns.
template <int TR>
__device__ __forceinline__ void stage2_chunk(const float* __restrict__ Zf, int n1, int n2, const float* __restrict__ Ps,
                                             int cwp, int c0, int cw, float* Ys, float& amax) {
    const int dt = n2 >> 2;
    const int tiles = ((cw + TR - 1) / TR) * dt;
    for (int tile = threadIdx.x; tile < tiles; tile += blockDim.x) {
        const int mt = tile / dt, d0 = (tile - mt * dt) << 2;
        const int r0 = mt * TR;
        float acc[TR][4];
#pragma unroll
        for (int i = 0; i < TR; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
        const float* zp = Zf + d0;
        const float* pp = Ps + r0;
#pragma unroll 4
        for (int a = 0; a < n1; ++a) {
            const float4 zv = *reinterpret_cast<const float4*>(zp + a * n2);
            float pa[TR];
            if (TR % 4 == 0) {
#pragma unroll
                for (int i = 0; i < TR; i += 4) {
                    const float4 v = *reinterpret_cast<const float4*>(pp + a * cwp + i);
                    pa[i] = v.x; pa[i + 1] = v.y; pa[i + 2] = v.z; pa[i + 3] = v.w;
                }
            } else {
#pragma unroll
                for (int i = 0; i < TR; ++i) pa[i] = pp[a * cwp + min(i, cw - 1 - r0)];
            }
#pragma unroll
            for (int i = 0; i < TR; ++i) {
                acc[i][0] = fmaf(pa[i], zv.x, acc[i][0]);
                acc[i][1] = fmaf(pa[i], zv.y, acc[i][1]);
                acc[i][2] = fmaf(pa[i], zv.z, acc[i][2]);
                acc[i][3] = fmaf(pa[i], zv.w, acc[i][3]);
            }
        }
#pragma unroll
        for (int i = 0; i < TR; ++i)
            if (r0 + i < cw) {
                *reinterpret_cast<float4*>(Ys + (c0 + r0 + i) * n2 + d0) = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
                amax = fmaxf(amax, fmaxf(fmaxf(fabsf(acc[i][0]), fabsf(acc[i][1])), fmaxf(fabsf(acc[i][2]), fabsf(acc[i][3]))));
            }
    }
}

// ---------------------------------------------------------------------------------------------
// rotation + quantiser
// ---------------------------------------------------------------------------------------------
// Partial sums of C[r][d] = sum_k A[k][r] * B[k][d] for a slab of rp rows (A: [depth][rp], zero beyond the real
// rows) and n2 columns.  A work item is a tile of TR rows x 4 columns over one of S slices of the depth; items are
// dealt to threads with the column index fastest, so a warp reads one run of B and broadcasts A.  The sums over k run
// in increasing order inside a slice.  part: [S][rp][n2].  B is fp32, or bf16 when B_BF16 (the activations).
template <int TR, bool B_BF16>
__device__ __forceinline__ void slab_partial(const float* __restrict__ A, int rp, const void* __restrict__ B, int depth,
                                             int n2, int S, float* __restrict__ part) {
    const int cq = n2 >> 2;
    const int tiles = (rp / TR) * cq;
    const int items = tiles * S;
    for (int item = threadIdx.x; item < items; item += blockDim.x) {
        const int sl = item / tiles, tile = item - sl * tiles;
        const int mt = tile / cq, d0 = (tile - mt * cq) << 2;
        const int k0 = (int)((int64_t)depth * sl / S), k1 = (int)((int64_t)depth * (sl + 1) / S);
        float acc[TR][4];
#pragma unroll
        for (int i = 0; i < TR; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
        // operand pointers advance by addition: index arithmetic inside this loop cost as many issue slots as the FMAs
        const float* ap = A + (size_t)k0 * rp + mt * TR;
        const float* bf = reinterpret_cast<const float*>(B) + (size_t)k0 * n2 + d0;
        const __nv_bfloat16* bh = reinterpret_cast<const __nv_bfloat16*>(B) + (size_t)k0 * n2 + d0;
#pragma unroll 4
        for (int k = k0; k < k1; ++k) {
            float4 bv;
            if (B_BF16) {
                const uint2 w = *reinterpret_cast<const uint2*>(bh);
                bv = make_float4(__uint_as_float(w.x << 16), __uint_as_float(w.x & 0xFFFF0000u),
                                 __uint_as_float(w.y << 16), __uint_as_float(w.y & 0xFFFF0000u));
                bh += n2;
            } else {
                bv = *reinterpret_cast<const float4*>(bf);
                bf += n2;
            }
            float a[TR];
#pragma unroll
            for (int i = 0; i < TR; i += 4) {
                const float4 v = *reinterpret_cast<const float4*>(ap + i);
                a[i] = v.x; a[i + 1] = v.y; a[i + 2] = v.z; a[i + 3] = v.w;
            }
            ap += rp;
#pragma unroll
            for (int i = 0; i < TR; ++i) {
                acc[i][0] = fmaf(a[i], bv.x, acc[i][0]);
                acc[i][1] = fmaf(a[i], bv.y, acc[i][1]);
                acc[i][2] = fmaf(a[i], bv.z, acc[i][2]);
                acc[i][3] = fmaf(a[i], bv.w, acc[i][3]);
            }
        }
        float* dst = part + ((size_t)sl * rp + mt * TR) * n2 + d0;
#pragma unroll
        for (int i = 0; i < TR; ++i)
            *reinterpret_cast<float4*>(dst + (size_t)i * n2) = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
    }
}

// Adds the S partial sums.  TRANSPOSED: the result goes to out[d][r] (row stride rp), the A operand of the next
// contraction; otherwise to out[r][d] (row stride n2), only for the real rows, and the largest magnitude is returned.
template <bool TRANSPOSED>
__device__ __forceinline__ float slab_reduce(const float* __restrict__ part, int rp, int rows, int n2, int S, float* out) {
    float amax = 0.f;
    const int cq = n2 >> 2;
    const int quads = (TRANSPOSED ? rp : rows) * cq;
    for (int o = threadIdx.x; o < quads; o += blockDim.x) {
        const int r = o / cq, d0 = (o - r * cq) << 2;
        float4 v = *reinterpret_cast<const float4*>(part + (size_t)r * n2 + d0);
        for (int sl = 1; sl < S; ++sl) {
            const float4 w = *reinterpret_cast<const float4*>(part + ((size_t)sl * rp + r) * n2 + d0);
            v.x += w.x; v.y += w.y; v.z += w.z; v.w += w.w;
        }
        if (TRANSPOSED) {
            out[(size_t)(d0 + 0) * rp + r] = v.x; out[(size_t)(d0 + 1) * rp + r] = v.y;
            out[(size_t)(d0 + 2) * rp + r] = v.z; out[(size_t)(d0 + 3) * rp + r] = v.w;
        } else {
            *reinterpret_cast<float4*>(out + (size_t)r * n2 + d0) = v;
            amax = fmaxf(amax, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
        }
    }
    return amax;
}

__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// A fragment of a row-major [row][k] bf16 tile (row stride `ld` elements): rows r0 + g, r0 + g + 8; k0 + 2tg, + 8
__device__ __forceinline__ void load_a_frag(uint32_t (&a)[4], const __nv_bfloat16* base, int ld, int r0, int k0, int g, int tg) {
    const __nv_bfloat16* p0 = base + (size_t)(r0 + g) * ld + k0 + 2 * tg;
    a[0] = *reinterpret_cast<const uint32_t*>(p0);
    a[1] = *reinterpret_cast<const uint32_t*>(p0 + 8 * ld);
    a[2] = *reinterpret_cast<const uint32_t*>(p0 + 8);
    a[3] = *reinterpret_cast<const uint32_t*>(p0 + 8 * ld + 8);
}

// Geometry of the tensor-core slab contractions in shared memory (element counts, bf16 unless noted)
struct TcLayout {
    int n1p;      // n1 rounded up to 16 (contraction depth of the first stage)
    int mt;       // 16-row tiles of the slab
    int xs;       // row stride of x [n1p][n2 + 8]
    int ps;       // row stride of the P1^T terms [3][16 mt][n1p + 8]
    int zs;       // row stride of the Z' terms [3][16 mt][n2 + 8]
    int pc;       // columns of P2 resident at a time (n2, or a part of it when all of P2 does not fit)
    int p2s;      // row stride of the P2 terms [3][n2][pc + 8]
};

__host__ __device__ inline TcLayout tc_layout(int n1, int n2, int slab_rows, int p2_chunks) {
    TcLayout L;
    L.pc = n2 / p2_chunks;
    L.p2s = L.pc + 8;
    L.n1p = (n1 + 15) / 16 * 16;
    L.mt = (slab_rows + 15) / 16;
    L.xs = n2 + 8;
    L.ps = L.n1p + 8;
    L.zs = n2 + 8;
    return L;
}
// bytes of x, the P1^T terms, the Z' terms and the P2 terms, in this order; each a multiple of 16
__host__ __device__ inline size_t tc_x_bytes(const TcLayout& L) { return (size_t)L.n1p * L.xs * 2; }
__host__ __device__ inline size_t tc_p1_bytes(const TcLayout& L) { return (size_t)3 * 16 * L.mt * L.ps * 2; }
__host__ __device__ inline size_t tc_z_bytes(const TcLayout& L) { return (size_t)3 * 16 * L.mt * L.zs * 2; }
__host__ __device__ inline size_t tc_p2_bytes(const TcLayout& L, int n2) { return (size_t)3 * n2 * L.p2s * 2; }

// columns [c0, c0 + L.pc) of P2, split into bf16 terms, in the [k][column] order of the source (the B fragments come from
// transposing matrix loads, as for x)
__device__ __forceinline__ void stage_p2_terms(const TcLayout& L, const float* __restrict__ P2, int n2, int c0, __nv_bfloat16* P2T) {
    const int qpr = L.pc >> 2;                  // float4 per row of the chunk
    for (int i = threadIdx.x; i < n2 * qpr; i += blockDim.x) {
        const int b = i / qpr, d = 4 * (i - b * qpr);
        const float4 v = __ldg(reinterpret_cast<const float4*>(P2 + (size_t)b * n2 + c0 + d));
        __nv_bfloat16 h[4], m[4], l[4];
        split3(v.x, h[0], m[0], l[0]); split3(v.y, h[1], m[1], l[1]);
        split3(v.z, h[2], m[2], l[2]); split3(v.w, h[3], m[3], l[3]);
        __nv_bfloat16* dst = P2T + (size_t)b * L.p2s + d;
        *reinterpret_cast<uint2*>(dst) = make_uint2(pack_bf16(h[0], h[1]), pack_bf16(h[2], h[3]));
        *reinterpret_cast<uint2*>(dst + (size_t)n2 * L.p2s) = make_uint2(pack_bf16(m[0], m[1]), pack_bf16(m[2], m[3]));
        *reinterpret_cast<uint2*>(dst + (size_t)2 * n2 * L.p2s) = make_uint2(pack_bf16(l[0], l[1]), pack_bf16(l[2], l[3]));
    }
}

// Z' = (P1^T X)[slab] as three bf16 terms.  The warps take tiles of 16 rows x 8 columns in turn.  The three term
// products of a k-step go to accumulators of their own (independent instructions), then into the running sum.
// With Zf != nullptr the result is written as fp32, transposed ([column][row], row stride 16 mt), for the FMA version
// of the second contraction, instead of as terms.
__device__ __forceinline__ void tc_stage_a(const TcLayout& L, int n2, const __nv_bfloat16* Xp, const __nv_bfloat16* P1T,
                                           __nv_bfloat16* ZT, float* Zf = nullptr) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int g = lane >> 2, tg = lane & 3;
    const int rows16 = 16 * L.mt;
    const int ntiles = n2 >> 3;
    for (int tile = warp; tile < L.mt * ntiles; tile += nwarps) {
        const int m = tile / ntiles, nt = tile - m * ntiles;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 2
        for (int ks = 0; ks < (L.n1p >> 4); ++ks) {
            // x is stored [k][n]: the transposing matrix load gives the B fragment (k pairs for column g)
            uint32_t b0, b1;
            const uint32_t addr = smem_u32(Xp + (size_t)(ks * 16 + (lane & 15)) * L.xs + nt * 8);
            asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0, %1}, [%2];" : "=r"(b0), "=r"(b1) : "r"(addr));
            uint32_t a[3][4];
#pragma unroll
            for (int term = 0; term < 3; ++term)
                load_a_frag(a[term], P1T + (size_t)term * rows16 * L.ps, L.ps, 16 * m, 16 * ks, g, tg);
            float c[3][4];
#pragma unroll
            for (int term = 0; term < 3; ++term) {
#pragma unroll
                for (int i = 0; i < 4; ++i) c[term][i] = 0.f;
                mma_bf16(c[term], a[term], b0, b1);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[i] += (c[2][i] + c[1][i]) + c[0][i];       // lo + mid, then hi
        }
        if (Zf) {
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int r = 16 * m + g + 8 * half;
                Zf[(size_t)(nt * 8 + 2 * tg) * rows16 + r] = acc[2 * half];
                Zf[(size_t)(nt * 8 + 2 * tg + 1) * rows16 + r] = acc[2 * half + 1];
            }
            continue;
        }
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            __nv_bfloat16 h0, m0, l0, h1, m1, l1;
            split3(acc[2 * half], h0, m0, l0);
            split3(acc[2 * half + 1], h1, m1, l1);
            __nv_bfloat16* dst = ZT + (size_t)(16 * m + g + 8 * half) * L.zs + nt * 8 + 2 * tg;
            *reinterpret_cast<uint32_t*>(dst) = pack_bf16(h0, h1);
            *reinterpret_cast<uint32_t*>(dst + (size_t)rows16 * L.zs) = pack_bf16(m0, m1);
            *reinterpret_cast<uint32_t*>(dst + (size_t)2 * rows16 * L.zs) = pack_bf16(l0, l1);
        }
    }
}

// Y[slab] = Z' P2 from the terms of both; the real rows go to Y (fp32, row stride n2); returns the largest magnitude.
// P2T holds columns [c0, c0 + L.pc) of the P2 terms; only those columns of Y are produced.  Of the nine term products
// the six whose weight is at least 2^-16 of the leading one are taken, in two independent chains per k-step.
__device__ __forceinline__ float tc_stage_b(const TcLayout& L, int n2, int rows, int c0, const __nv_bfloat16* ZT,
                                            const __nv_bfloat16* P2T, float* Y) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int g = lane >> 2, tg = lane & 3;
    const int rows16 = 16 * L.mt;
    const int ntiles = L.pc >> 3;
    float amax = 0.f;
    for (int tile = warp; tile < L.mt * ntiles; tile += nwarps) {
        const int m = tile / ntiles, nt = (c0 >> 3) + tile - m * ntiles;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 2
        for (int ks = 0; ks < (n2 >> 4); ++ks) {
            uint32_t b[3][2];                                         // P2 terms hi, mid, lo, stored [k][column] like x
#pragma unroll
            for (int term = 0; term < 3; ++term) {
                const uint32_t addr = smem_u32(P2T + ((size_t)term * n2 + ks * 16 + (lane & 15)) * L.p2s + nt * 8 - c0);
                asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0, %1}, [%2];"
                             : "=r"(b[term][0]), "=r"(b[term][1]) : "r"(addr));
            }
            uint32_t a[3][4];
#pragma unroll
            for (int term = 0; term < 3; ++term)
                load_a_frag(a[term], ZT + (size_t)term * rows16 * L.zs, L.zs, 16 * m, 16 * ks, g, tg);
            float cs[4] = {0.f, 0.f, 0.f, 0.f}, cb[4] = {0.f, 0.f, 0.f, 0.f};
            // small products: mid*mid, lo*hi, hi*lo; large: mid*hi, hi*mid, hi*hi
            mma_bf16(cs, a[1], b[1][0], b[1][1]);
            mma_bf16(cb, a[1], b[0][0], b[0][1]);
            mma_bf16(cs, a[2], b[0][0], b[0][1]);
            mma_bf16(cb, a[0], b[1][0], b[1][1]);
            mma_bf16(cs, a[0], b[2][0], b[2][1]);
            mma_bf16(cb, a[0], b[0][0], b[0][1]);
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[i] += cs[i] + cb[i];
        }
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int r = 16 * m + g + 8 * half;
            if (r < rows) {
                const float v0 = acc[2 * half], v1 = acc[2 * half + 1];
                *reinterpret_cast<float2*>(Y + (size_t)r * n2 + nt * 8 + 2 * tg) = make_float2(v0, v1);
                amax = fmaxf(amax, fmaxf(fabsf(v0), fabsf(v1)));
            }
        }
    }
    return amax;
}

// asynchronous copies global -> shared (no register in between, so all of a thread's copies are in flight at once)
__device__ __forceinline__ void cp_async_16(void* dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_4(void* dst, const void* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
    asm volatile("cp.async.wait_all;" ::: "memory");
}

// x_t[first .. first+len) -> fp32 in shared memory
__device__ __forceinline__ void load_x(const __nv_bfloat16* __restrict__ xt, int len, float* Xs) {
    if ((reinterpret_cast<uintptr_t>(xt) & 15) == 0 && (len & 7) == 0) {
        const uint4* xv = reinterpret_cast<const uint4*>(xt);
        for (int i = threadIdx.x; i < (len >> 3); i += blockDim.x) {
            const uint4 v = __ldg(xv + i);
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
            float f[8];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                f[2 * j] = __uint_as_float(w[j] << 16);
                f[2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
            }
            *reinterpret_cast<float4*>(Xs + 8 * i) = make_float4(f[0], f[1], f[2], f[3]);
            *reinterpret_cast<float4*>(Xs + 8 * i + 4) = make_float4(f[4], f[5], f[6], f[7]);
        }
    } else {
        for (int k = threadIdx.x; k < len; k += blockDim.x) Xs[k] = __bfloat162float(xt[k]);
    }
}

// columns [a_lo, a_lo+rows) of P1 -> shared memory, row stride cwp (padding zero)
__device__ __forceinline__ void load_p1_columns(const float* __restrict__ P1, int n1, int a_lo, int rows, int cwp, float* dst) {
    for (int i = threadIdx.x; i < n1 * cwp; i += blockDim.x) {
        const int a = i / cwp, j = i - a * cwp;
        dst[i] = j < rows ? __ldg(P1 + (size_t)a * n1 + a_lo + j) : 0.f;
    }
}

// Second half of a token: absmax over the block and the cluster, quantisation of this CTA's rows of Y (at Xs), code
// sums, scale.  One cluster barrier per token when C > 1 (every CTA of the cluster calls this for the same tokens).
__device__ __forceinline__ void finish_token(const PrologueParams& p, int64_t t, int C, int rank, const float* Xs, float* slots,
                                             float amax, int rows, int a_lo, float* red_max, int* red_sum_p, bool last) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int qmax = (1 << (p.bits - 1)) - 1;
    const int n2 = p.n2, K = p.K;
    int& red_sum = *red_sum_p;
    // ---- absmax over the block, then over the cluster
    amax = warp_max(amax);
    if (lane == 0) red_max[warp] = amax;
    __syncthreads();
    amax = (lane < nwarps) ? red_max[lane] : 0.f;
    amax = warp_max(amax);
    if (C > 1) {
        if (threadIdx.x < C) st_cluster_u32(map_shared_rank(smem_u32(slots + rank), threadIdx.x), __float_as_uint(amax));
        cluster_arrive_release();
        cluster_wait_acquire();
        float m = (lane < C) ? slots[lane] : 0.f;
        amax = warp_max(m);
        if (!last) {
            // a cluster that goes on to another token: nobody may store the next token's absmax into these slots before
            // every CTA has read this token's
            cluster_arrive_release();
            cluster_wait_acquire();
        }
    }

    float inv, scale;
    if (amax == 0.f) { inv = 0.f; scale = 1.f; }
    else { inv = __fdiv_rn((float)qmax, amax); scale = __fdiv_rn(amax, (float)qmax); }

    if (p.late_trigger && last) griddep_launch_dependents();
    // nothing is stored to global memory before the preceding kernel of the stream has completed
    griddep_wait();

    int local_sum = 0;
    int8_t* ct = p.codes + t * (int64_t)K + (int64_t)a_lo * n2;
    const int words = (rows * n2) >> 5;
    for (int g = threadIdx.x; g < words; g += blockDim.x) {
        const float* y = Xs + 32 * g;
        int q[32];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float4 v = *reinterpret_cast<const float4*>(y + 4 * i);
            const float f[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                int c = __float2int_rn(__fmul_rn(f[j], inv));
                c = max(-qmax, min(qmax, c));
                q[4 * i + j] = c;
                local_sum += c;
            }
        }
        uint32_t w[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            uint32_t v = 0;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int k = p.codes_layout ? (j + 8 * i) : (4 * j + i);
                v |= (uint32_t)(q[k] & 0xFF) << (8 * i);
            }
            w[j] = v;
        }
        uint4* dst = reinterpret_cast<uint4*>(ct + 32 * g);
        dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
        dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
    }
    local_sum = warp_sum(local_sum);
    if (lane == 0 && local_sum != 0) atomicAdd(&red_sum, local_sum);
    __syncthreads();
    // every CTA leaves its own part of the token's code sum; the consumer adds the parts, so no exchange is needed here
    if (threadIdx.x == 0) {
        if (p.qsum) {
            p.qsum[t * kQsumParts + rank] = red_sum;
            if (rank == 0)
                for (int c = C; c < kQsumParts; ++c) p.qsum[t * kQsumParts + c] = 0;
        }
        if (rank == 0) p.scales[t] = scale;
    }
}

__device__ void rotate_role(const PrologueParams& p, float* smem) {
    const int C = p.C;
    const int rank = C > 1 ? (int)cluster_ctarank() : 0;
    const int64_t t = ((int)blockIdx.x - p.rot_first) / C;   // the cluster's first (with few tokens: only) token
    const int n1 = p.n1, n2 = p.n2, K = p.K;
    const int a_lo = slab_begin(rank, C, n1, p.row_gran), a_hi = slab_begin(rank + 1, C, n1, p.row_gran);
    const int rows = a_hi - a_lo;
    float* Xs = smem;                          // this CTA's rows of Y end up here in every mode
    float* slots;                              // [0..7] absmax per rank
    __shared__ float red_max[32];
    __shared__ int red_sum;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int qmax = (1 << (p.bits - 1)) - 1;
    float amax = 0.f;
    if (threadIdx.x == 0) red_sum = 0;

    if (p.split_y && p.sp_tc == 1) {
        // ---- few tokens, tensor-core contractions: this CTA's rows of Y from all of x
        const TcLayout L = tc_layout(n1, n2, p.sp_rp, p.sp_s);
        uint8_t* base = reinterpret_cast<uint8_t*>(smem);
        __nv_bfloat16* Xp = reinterpret_cast<__nv_bfloat16*>(base);                       // x, later this CTA's rows of Y (fp32)
        __nv_bfloat16* P1T = reinterpret_cast<__nv_bfloat16*>(base + tc_x_bytes(L));
        __nv_bfloat16* ZT = reinterpret_cast<__nv_bfloat16*>(base + tc_x_bytes(L) + tc_p1_bytes(L));
        __nv_bfloat16* P2T = reinterpret_cast<__nv_bfloat16*>(base + tc_x_bytes(L) + tc_p1_bytes(L) + tc_z_bytes(L));
        slots = reinterpret_cast<float*>(base + tc_x_bytes(L) + tc_p1_bytes(L) + tc_z_bytes(L) + tc_p2_bytes(L, n2));
        // the layer's constants, split into bf16 terms (the first columns of P2 when not all of it fits)
        stage_p2_terms(L, p.P2, n2, 0, P2T);
        for (int i = threadIdx.x; i < 16 * L.mt * L.n1p; i += blockDim.x) {
            const int r = i / L.n1p, a = i - r * L.n1p;
            const float v = (r < rows && a < n1) ? __ldg(p.P1 + (size_t)a * n1 + a_lo + r) : 0.f;
            __nv_bfloat16 h, m, l;
            split3(v, h, m, l);
            __nv_bfloat16* dst = P1T + (size_t)r * L.ps + a;
            dst[0] = h; dst[(size_t)16 * L.mt * L.ps] = m; dst[(size_t)2 * 16 * L.mt * L.ps] = l;
        }
        cluster_arrive_release();              // "this CTA is running": waited for before the first remote store
        if (!p.late_trigger) griddep_launch_dependents();
        griddep_wait();                        // x may be the output of the preceding kernel
        {
            const __nv_bfloat16* xt = p.x + t * p.ldx;
            const int cpr = n2 >> 3;           // 16-byte chunks per row of X
            if ((reinterpret_cast<uintptr_t>(xt) & 15) == 0) {
                for (int i = threadIdx.x; i < n1 * cpr; i += blockDim.x) {
                    const int a = i / cpr, c = i - a * cpr;
                    *reinterpret_cast<uint4*>(Xp + (size_t)a * L.xs + 8 * c) = __ldg(reinterpret_cast<const uint4*>(xt) + i);
                }
            } else {
                for (int k = threadIdx.x; k < K; k += blockDim.x) Xp[(size_t)(k / n2) * L.xs + k % n2] = xt[k];
            }
            // rows of the depth padding must be finite: 0 * garbage could be NaN
            for (int i = threadIdx.x; i < (L.n1p - n1) * cpr; i += blockDim.x) {
                const int a = n1 + i / cpr, c = i % cpr;
                *reinterpret_cast<uint4*>(Xp + (size_t)a * L.xs + 8 * c) = make_uint4(0u, 0u, 0u, 0u);
            }
        }
        __syncthreads();
        tc_stage_a(L, n2, Xp, P1T, ZT);
        __syncthreads();
        amax = tc_stage_b(L, n2, rows, 0, ZT, P2T, Xs);
        for (int c0 = L.pc; c0 < n2; c0 += L.pc) {
            __syncthreads();                   // every warp is done with the columns in place
            stage_p2_terms(L, p.P2, n2, c0, P2T);
            __syncthreads();
            amax = fmaxf(amax, tc_stage_b(L, n2, rows, c0, ZT, P2T, Xs));
        }
        cluster_wait_acquire();
    } else if (p.split_y && p.sp_tc == 2) {
        // ---- few tokens, large P2: the first contraction on the tensor-core path (its factor, a slab of P1^T, is small),
        //      the second as FMA tiles over fp32 P2 (splitting all of P2 into terms costs more than it saves there)
        const TcLayout L = tc_layout(n1, n2, p.sp_rp, 1);
        const int rp = 16 * L.mt, S = p.sp_s;
        uint8_t* base = reinterpret_cast<uint8_t*>(smem);
        __nv_bfloat16* Xp = reinterpret_cast<__nv_bfloat16*>(base);                       // x | P1^T terms; later the partial
        __nv_bfloat16* P1T = reinterpret_cast<__nv_bfloat16*>(base + tc_x_bytes(L));      // sums and this CTA's rows of Y
        float* part = smem;
        float* Zt = reinterpret_cast<float*>(base + tc_x_bytes(L) + tc_p1_bytes(L));      // Z'^T fp32 [n2][rp]
        float* P2s = Zt + (size_t)n2 * rp;
        slots = P2s + n2 * n2 + 8;
        for (int i = threadIdx.x; i < (n2 * n2) >> 2; i += blockDim.x) cp_async_16(P2s + 4 * i, p.P2 + 4 * i);
        {
            // the slab of P1^T: eight loads in flight per thread (consecutive threads read one row of P1), then the terms
            constexpr int U = 8;
            const int total = rp * L.n1p;
            for (int i0 = threadIdx.x; i0 < total; i0 += U * blockDim.x) {
                float v[U];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int i = i0 + u * blockDim.x;
                    const int a = i / rp, r = i - a * rp;
                    v[u] = (i < total && r < rows && a < n1) ? __ldg(p.P1 + (size_t)a * n1 + a_lo + r) : 0.f;
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int i = i0 + u * blockDim.x;
                    if (i < total) {
                        const int a = i / rp, r = i - a * rp;
                        __nv_bfloat16 h, m, l;
                        split3(v[u], h, m, l);
                        __nv_bfloat16* dst = P1T + (size_t)r * L.ps + a;
                        dst[0] = h; dst[(size_t)rp * L.ps] = m; dst[(size_t)2 * rp * L.ps] = l;
                    }
                }
            }
        }
        cluster_arrive_release();              // "this CTA is running": waited for before the first remote store
        if (!p.late_trigger) griddep_launch_dependents();
        griddep_wait();                        // x may be the output of the preceding kernel
        // The cluster takes tokens t, t + tok_stride, ...: with few tokens exactly one; with many tokens of a large K the
        // clusters stay, and the constants above are fetched and split once per cluster instead of once per token.
        for (int64_t tt = t; tt < p.M; tt += p.tok_stride) {
            if (tt != t) {
                // every thread of the block is past its reads of the previous token's Y (the barriers of finish_token)
                if (threadIdx.x == 0) red_sum = 0;
                amax = 0.f;
            }
            const __nv_bfloat16* xt = p.x + tt * p.ldx;
            const int cpr = n2 >> 3;           // 16-byte chunks per row of X
            if ((reinterpret_cast<uintptr_t>(xt) & 15) == 0) {
                for (int i = threadIdx.x; i < n1 * cpr; i += blockDim.x) {
                    const int a = i / cpr, c = i - a * cpr;
                    *reinterpret_cast<uint4*>(Xp + (size_t)a * L.xs + 8 * c) = __ldg(reinterpret_cast<const uint4*>(xt) + i);
                }
            } else {
                for (int k = threadIdx.x; k < K; k += blockDim.x) Xp[(size_t)(k / n2) * L.xs + k % n2] = xt[k];
            }
            for (int i = threadIdx.x; i < (L.n1p - n1) * cpr; i += blockDim.x) {
                const int a = n1 + i / cpr, c = i % cpr;
                *reinterpret_cast<uint4*>(Xp + (size_t)a * L.xs + 8 * c) = make_uint4(0u, 0u, 0u, 0u);
            }
            __syncthreads();
            tc_stage_a(L, n2, Xp, P1T, nullptr, Zt);
            cp_async_wait_all();               // P2 has been arriving meanwhile; it is first read below
            __syncthreads();                   // x is dead: its place takes the partial sums (and, with one token per
                    // cluster, that of the P1^T terms too)
            slab_partial<8, false>(Zt, rp, P2s, n2, n2, S, part);
            __syncthreads();
            // Y goes where the first slice of the partial sums is: a thread reads its own elements of every slice first
            amax = slab_reduce<false>(part, rp, rows, n2, S, Xs);
            if (tt == t) cluster_wait_acquire();
            finish_token(p, tt, C, rank, Xs, slots, amax, rows, a_lo, red_max, &red_sum, tt + p.tok_stride >= p.M);
        }
        return;
    } else if (p.split_y) {
        // ---- few tokens: this CTA's rows of Y from all of x; nothing but absmax and code sums is exchanged
        const int rp = p.sp_rp, S = p.sp_s;
        __nv_bfloat16* Xh = reinterpret_cast<__nv_bfloat16*>(smem);   // all of x_t as it comes; later this CTA's rows of Y (fp32)
        float* Zt = smem + p.sp_zt_off;        // Z'^T: [n2][rp], Z' = rows [a_lo, a_hi) of P1^T X (written once x is dead)
        float* P2s = smem + p.sp_rest_off;     // all of P2
        float* P1s = P2s + p.ps_cap;           // columns [a_lo, a_hi) of P1: [n1][rp]
        float* part = P1s + p.p1_cap;          // [S][rp][n2] partial sums
        slots = part + S * rp * n2;
        // the layer's constants do not depend on the preceding kernel; asynchronous copies, so that one round trip
        // brings all of them (with a load and a store per loop iteration it was one round trip per iteration)
        for (int i = threadIdx.x; i < (n2 * n2) >> 2; i += blockDim.x) cp_async_16(P2s + 4 * i, p.P2 + 4 * i);
        for (int i = threadIdx.x; i < n1 * rp; i += blockDim.x) {
            const int a = i / rp, j = i - a * rp;
            if (j < rows) cp_async_4(P1s + i, p.P1 + (size_t)a * n1 + a_lo + j);
            else P1s[i] = 0.f;
        }
        cluster_arrive_release();              // "this CTA is running": waited for before the first remote store
        if (!p.late_trigger) griddep_launch_dependents();
        cp_async_wait_all();                   // made visible to the block by the barrier behind the load of x
        griddep_wait();                        // x may be the output of the preceding kernel
        {
            const __nv_bfloat16* xt = p.x + t * p.ldx;
            if ((reinterpret_cast<uintptr_t>(xt) & 15) == 0) {
                for (int i = threadIdx.x; i < (K >> 3); i += blockDim.x)
                    reinterpret_cast<uint4*>(Xh)[i] = __ldg(reinterpret_cast<const uint4*>(xt) + i);
            } else {
                for (int k = threadIdx.x; k < K; k += blockDim.x) Xh[k] = xt[k];
            }
        }
        __syncthreads();
        if (p.sp_tr == 8) slab_partial<8, true>(P1s, rp, Xh, n1, n2, S, part);
        else slab_partial<4, true>(P1s, rp, Xh, n1, n2, S, part);
        __syncthreads();
        slab_reduce<true>(part, rp, rows, n2, S, Zt);
        __syncthreads();
        if (p.sp_tr == 8) slab_partial<8, false>(Zt, rp, P2s, n2, n2, S, part);
        else slab_partial<4, false>(Zt, rp, P2s, n2, n2, S, part);
        __syncthreads();
        amax = slab_reduce<false>(part, rp, rows, n2, S, Xs);
        cluster_wait_acquire();
    } else if ((n2 & 3) == 0) {
        // ---- one CTA per token: Z = X * P2, Y = P1^T * Z, the factors staged chunk by chunk
        float* Zf = smem + p.slab_cap;         // all of Z
        float* Ps = Zf + K;                    // staged chunk of P2, later of P1
        float* P1s = Ps + p.ps_cap;            // all of P1 when it is prefetched
        slots = P1s + p.p1_cap;
        if (p.prefetch) {
            for (int i = threadIdx.x; i < (n2 * n2) >> 2; i += blockDim.x)
                *reinterpret_cast<float4*>(Ps + 4 * i) = __ldg(reinterpret_cast<const float4*>(p.P2) + i);
            load_p1_columns(p.P1, n1, 0, n1, (n1 + 3) & ~3, P1s);
        }
        if (!p.late_trigger) griddep_launch_dependents();
        griddep_wait();                        // x may be the output of the preceding kernel
        load_x(p.x + t * p.ldx, K, Xs);
        for (int dc = 0; dc < n2; dc += p.ch1) {
            const int cw = min(p.ch1, n2 - dc);
            if (!p.prefetch) for (int i = threadIdx.x; i < n2 * (cw >> 2); i += blockDim.x) {
                const int b = i / (cw >> 2), j = (i - b * (cw >> 2)) << 2;
                *reinterpret_cast<float4*>(Ps + b * cw + j) = __ldg(reinterpret_cast<const float4*>(p.P2 + (size_t)b * n2 + dc + j));
            }
            __syncthreads();
            switch (p.tr1) {
                case 8: stage1_chunk<8>(Xs, n1, n2, Ps, dc, cw, Zf); break;
                case 4: stage1_chunk<4>(Xs, n1, n2, Ps, dc, cw, Zf); break;
                case 2: stage1_chunk<2>(Xs, n1, n2, Ps, dc, cw, Zf); break;
                default: stage1_chunk<1>(Xs, n1, n2, Ps, dc, cw, Zf); break;
            }
            __syncthreads();
        }
        // Y overwrites X, which is dead now; one chunk of output rows (columns of P1) at a time
        for (int c0 = 0; c0 < n1; c0 += p.ch2) {
            const int cw = min(p.ch2, n1 - c0), cwp = (cw + 3) & ~3;
            const float* Pc = p.prefetch ? P1s : Ps;
            if (!p.prefetch) load_p1_columns(p.P1, n1, c0, cw, cwp, Ps);
            __syncthreads();
            switch (p.tr2) {
                case 8: stage2_chunk<8>(Zf, n1, n2, Pc, cwp, c0, cw, Xs, amax); break;
                case 4: stage2_chunk<4>(Zf, n1, n2, Pc, cwp, c0, cw, Xs, amax); break;
                case 2: stage2_chunk<2>(Zf, n1, n2, Pc, cwp, c0, cw, Xs, amax); break;
                default: stage2_chunk<1>(Zf, n1, n2, Pc, cwp, c0, cw, Xs, amax); break;
            }
            __syncthreads();
        }
    } else {
        // generic shapes (n2 not a multiple of 4; one CTA per token): one output per thread step
        float* Zf = smem + p.slab_cap;
        slots = Zf + K;
        if (!p.late_trigger) griddep_launch_dependents();
        griddep_wait();
        load_x(p.x + t * p.ldx, K, Xs);
        __syncthreads();
        for (int o = threadIdx.x; o < K; o += blockDim.x) {
            const int a = o / n2, d = o - a * n2;
            float s = 0.f;
            for (int b = 0; b < n2; ++b) s = fmaf(Xs[a * n2 + b], __ldg(p.P2 + b * n2 + d), s);
            Zf[o] = s;
        }
        __syncthreads();
        for (int o = threadIdx.x; o < K; o += blockDim.x) {
            const int c = o / n2, d = o - c * n2;
            float s = 0.f;
            for (int a = 0; a < n1; ++a) s = fmaf(__ldg(p.P1 + a * n1 + c), Zf[a * n2 + d], s);
            Xs[o] = s;
            amax = fmaxf(amax, fabsf(s));
        }
    }
    finish_token(p, t, C, rank, Xs, slots, amax, rows, a_lo, red_max, &red_sum, true);
}

__global__ void prologue_kernel(PrologueParams p) {
    extern __shared__ __align__(16) float smem[];
    const int b = (int)blockIdx.x;
    const int lr = p.rot_first ? b : b - p.rot_blocks;        // index among the low-rank blocks (when not a rotation block)
    if (b >= p.rot_first && b < p.rot_first + p.rot_blocks) rotate_role(p, smem);
    else if (p.lr_wide == 1) lowrank_role<8, 8>(p, lr, smem);
    else if (p.lr_wide == 2) lowrank_mma_role(p, lr, smem);
    else if (p.lr_wide == 3) lowrank_mma_wide_role(p, lr, smem);
    else lowrank_role<2, 16>(p, lr, smem);
}

// How many clusters of `c` prologue blocks (threads, dynamic shared memory) the device holds at once; cached.
__global__ void prologue_kernel(PrologueParams p);
static int clusters_resident(int c, int threads, size_t smem) {
    struct Key { int dev, c, threads; size_t smem; int n; };
    static thread_local Key cache[16];
    static thread_local int used = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    for (int i = 0; i < used; ++i)
        if (cache[i].dev == dev && cache[i].c == c && cache[i].threads == threads && cache[i].smem == smem) return cache[i].n;
    if (cudaFuncSetAttribute(prologue_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPrologueSmemFloats * 4) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)(c * (sm_count() > 0 ? sm_count() : 1)), 1, 1);
    cfg.blockDim = dim3((unsigned)threads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)c; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, prologue_kernel, &cfg) != cudaSuccess) { cudaGetLastError(); n = 0; }
    if (used < 16) cache[used++] = Key{dev, c, threads, smem, n};
    return n;
}

static int gcd_int(int a, int b) { while (b) { int t = a % b; a = b; b = t; } return a; }

int launch_prologue(const void* x, int64_t M, int64_t K, int64_t ldx, const float* P1, int n1, const float* P2, int n2,
                    int bits, int8_t* codes, int codes_layout, float* scales, int32_t* qsum, const void* V, int r,
                    void* Thl, float* lr_part, uint32_t* status, cudaStream_t stream) {
    if (M == 0) return BWLA_OK;
    const bool rotate = codes != nullptr;
    PrologueParams p{};
    p.x = (const __nv_bfloat16*)x; p.M = M; p.K = (int)K; p.ldx = ldx;
    p.P1 = P1; p.n1 = n1; p.P2 = P2; p.n2 = n2; p.bits = bits;
    p.codes = codes; p.codes_layout = codes_layout; p.scales = scales; p.qsum = qsum;
    p.V = (const __nv_bfloat16*)V; p.r = r; p.Thl = (__nv_bfloat16*)Thl;
    p.lr_cols = lowrank_cols(r);

    int C = 1;
    int threads = 256;
    size_t smem = 0;
    if (rotate) {
        const int gran = 32 / gcd_int(n2, 32);
        // clusters that stay and take several tokens must keep the terms of P1^T: the partial sums then take x's place only
        bool keep_p1t = false;
        // lays the block out for clusters of `c` CTAs per token; false if it does not fit
        auto plan = [&](int c) -> bool {
            int cap = 0;
            for (int i = 0; i < c; ++i) {
                const int lo = (int)(((int64_t)n1 * i / c) / gran * gran);
                const int hi = (i + 1 >= c) ? n1 : (int)(((int64_t)n1 * (i + 1) / c) / gran * gran);
                cap = cap > (hi - lo) ? cap : (hi - lo);
            }
            p.C = c; p.rot_blocks = (int)(M * c); p.row_gran = gran; p.slab_cap = (cap * n2 + 3) / 4 * 4;
            p.prefetch = 0; p.p1_cap = 0; p.split_y = 0;
            auto pick = [](int rows, int cols4, int want_tiles) {
                for (int tr = 8; tr > 1; tr >>= 1)
                    if (((rows + tr - 1) / tr) * cols4 >= want_tiles) return tr;
                return 1;
            };
            if (c > 1) {
                // all of x (bf16), this CTA's rows of Z' (transposed), all of P2, this CTA's columns of P1, partial sums
                if ((K & 7) != 0) return false;
                p.split_y = 1;
                p.sp_tc = 0;
                if (n2 % 16 == 0 && (cap + 15) / 16 <= 4 && n2 <= 96) {
                    // both contractions on the warp-level tensor-core path when the split operands fit and P2 is small
                    // (splitting all of a larger P2 into terms costs more than the FMA version of the second contraction:
                    // o_proj, n2 = 128, is 1.6 us faster the mixed way)
                    // P2 whole.  (Staging it in parts of its columns works -- the kernel takes any number of parts -- but
                    // was measured no faster than the FMA version for K = 25600: mma.sync runs at ~6 cycles per
                    // m16n8k16 per SM on this part, and the restaging is exposed.)
                    int chunks = 1;
                    size_t bytes = 0;
                    for (; chunks <= 1; chunks *= 2) {
                        if ((n2 / chunks) % 8 != 0 || n2 % chunks != 0) { chunks = 8; break; }
                        const TcLayout L = tc_layout(n1, n2, cap, chunks);
                        bytes = tc_x_bytes(L) + tc_p1_bytes(L) + tc_z_bytes(L) + tc_p2_bytes(L, n2) + 64;
                        if (bytes <= (size_t)kPrologueSmemFloats * 4) break;
                    }
                    if (chunks <= 1) {
                        p.sp_tc = 1; p.sp_rp = cap; p.sp_tr = 0; p.sp_s = chunks;   // sp_s: parts of P2 in this mode
                        p.ps_cap = 0; p.p1_cap = 0; p.ch1 = n2; p.ch2 = cap; p.tr1 = p.tr2 = 1;
                        // all the warps a block may have: splitting the constants into terms is instruction-bound, and a
                        // block of this kernel cannot share an SM with the contraction CTAs before it in any case
                        threads = 512;
                        smem = bytes;
                        return true;
                    }
                }
                if (n2 % 8 == 0 && (cap + 15) / 16 <= 4) {
                    // P2 too large for its terms: first contraction on the tensor-core path, second as FMA tiles
                    const TcLayout L = tc_layout(n1, n2, cap, 1);
                    const int rp16 = 16 * L.mt;
                    const size_t r0 = tc_x_bytes(L) + tc_p1_bytes(L);
                    const size_t part_room = keep_p1t ? tc_x_bytes(L) : r0;
                    const size_t slice = (size_t)rp16 * n2 * 4;
                    const size_t rest = (size_t)n2 * rp16 * 4 + ((size_t)n2 * n2 + 8) * 4 + 64;
                    if (slice <= part_room && r0 + rest <= (size_t)kPrologueSmemFloats * 4) {
                        const int tiles = (rp16 / 8) * (n2 / 4);
                        int S = 1;
                        while (S < 8 && tiles * S < 512 && n2 / (S * 2) >= 4 && (size_t)(S * 2) * slice <= part_room) S *= 2;
                        p.sp_tc = 2; p.sp_rp = cap; p.sp_tr = 8; p.sp_s = S;
                        p.ps_cap = 0; p.p1_cap = 0; p.ch1 = n2; p.ch2 = cap; p.tr1 = p.tr2 = 8;
                        threads = 512;
                        smem = r0 + rest;
                        return true;
                    }
                }
                // thread tiles of 8 rows unless padding the slab to a multiple of 8 wastes more than 15 %
                p.sp_tr = ((cap + 7) / 8 * 8) * 100 <= cap * 115 ? 8 : 4;
                p.sp_rp = (cap + p.sp_tr - 1) / p.sp_tr * p.sp_tr;
                p.ps_cap = n2 * n2 + 8;
                p.p1_cap = n1 * p.sp_rp + 8;
                p.ch1 = n2; p.ch2 = cap; p.tr1 = p.tr2 = p.sp_tr;
                const int tiles = (p.sp_rp / p.sp_tr) * (n2 / 4);
                // Z'^T is written when x is dead and may take its place; Y is written when Z'^T is dead
                const int64_t zt = (int64_t)n2 * p.sp_rp;
                p.sp_zt_off = zt <= K / 2 ? 0 : (int)(K / 2);
                p.sp_rest_off = (int)(K / 2 + (zt <= K / 2 ? 0 : zt));
                const int64_t fixed = p.sp_rest_off + p.ps_cap + p.p1_cap + 16;
                // cut the depth until there are about 512 work items, at least four steps per slice, while it fits
                int S = 1;
                while (S < 8 && tiles * S < 512 && std::min(n1, n2) / (S * 2) >= 4 &&
                       fixed + (int64_t)(S * 2) * p.sp_rp * n2 <= kPrologueSmemFloats) S *= 2;
                p.sp_s = S;
                const int64_t need = fixed + (int64_t)S * p.sp_rp * n2;
                if (need > kPrologueSmemFloats) return false;
                const int items = tiles * S;
                threads = (items + 31) / 32 * 32;
                threads = threads < 256 ? 256 : (threads > 512 ? 512 : threads);
                smem = (size_t)need * 4;
                return true;
            }
            if ((n2 & 3) == 0) {
                // chunks of P2 (ch1 columns) and of P1 (ch2 columns) that fit beside the X slab and Z
                const int64_t avail = kPrologueSmemFloats - p.slab_cap - K - 16 - 8;
                const int max1 = (int)std::min<int64_t>(n2, avail / n2 / 4 * 4);
                const int max2 = (int)std::min<int64_t>((cap + 3) / 4 * 4, avail / n1 / 4 * 4);
                if (max1 < 4 || max2 < 4) return false;
                // equal chunks rather than full ones and a sliver
                const int nch1 = (n2 + max1 - 1) / max1, nch2 = (cap + max2 - 1) / max2;
                const int ch1 = ((n2 + nch1 - 1) / nch1 + 3) / 4 * 4;
                const int ch2 = std::min(cap, ((cap + nch2 - 1) / nch2 + 3) / 4 * 4);
                p.ch1 = ch1; p.ch2 = ch2;
                p.ps_cap = std::max(n2 * ch1, n1 * ((ch2 + 3) / 4 * 4)) + 8;
                // all of P2 and this CTA's columns of P1 at once, fetched together with x, when both fit
                const int64_t p1_need = (int64_t)n1 * ((cap + 3) / 4 * 4) + 8;
                if (nch1 == 1 && nch2 == 1 && (int64_t)n2 * n2 + 8 + p1_need <= avail) {
                    p.prefetch = 1; p.ps_cap = n2 * n2 + 8; p.p1_cap = (int)p1_need;
                }
                // rows per thread: as many as still leave enough tiles to hide latency
                p.tr1 = pick(cap, ch1 / 4, 256);
                p.tr2 = pick(ch2, n2 / 4, 256);
                const int tiles = std::max(((cap + p.tr1 - 1) / p.tr1) * (ch1 / 4), ((ch2 + p.tr2 - 1) / p.tr2) * (n2 / 4));
                const int rounds = (tiles + 511) / 512;
                threads = ((tiles + rounds - 1) / rounds + 31) / 32 * 32;
                // never fewer than 256: the low-rank blocks of the same launch stride over K with this many threads
                threads = threads < 256 ? 256 : (threads > 512 ? 512 : threads);
            } else {
                p.ps_cap = 0; p.ch1 = p.ch2 = 4; p.tr1 = p.tr2 = 1;
                threads = 256;
            }
            smem = ((size_t)p.slab_cap + (size_t)K + (size_t)p.ps_cap + (size_t)p.p1_cap + 16) * 4;
            return true;
        };
        int64_t clusters = M;                  // clusters of C CTAs; each takes tokens t, t + clusters, ...
        if ((n2 & 3) == 0) {
            const double flops = 2.0 * (double)K * (n1 + n2);
            int cmax = 8;
            while (cmax > 1 && (flops / cmax < 1.5e5 || n1 / cmax < gran)) --cmax;
            // Few tokens: spread one token over several SMs, as long as every token's cluster is resident at once (a
            // second wave of clusters would double the latency).
            bool chosen = false;
            for (int c = cmax; c > 1 && !chosen; --c) {
                if (M * c > sm_count() || !plan(c)) continue;
                if (clusters_resident(c, threads, smem) >= M) { C = c; chosen = true; }
            }
            // Many tokens of a large K: one CTA per token would stage P1 and P2 chunk by chunk for every token.  Clusters
            // that stay, keep the constants and take tokens in turn do that once per cluster; the cluster size that puts
            // the most CTAs on the device wins.  (Only the mode whose first contraction runs on the tensor-core path is
            // fast enough per token to beat one CTA per token.)
            if (!chosen && plan(1) && !p.prefetch) {
                keep_p1t = true;
                int best_ctas = 0;
                for (int c = cmax; c > 1; --c) {
                    if (!plan(c) || p.sp_tc != 2) continue;
                    const int64_t n = std::min<int64_t>(M, clusters_resident(c, threads, smem));
                    if (n * c > best_ctas) { best_ctas = (int)(n * c); C = c; clusters = n; chosen = true; }
                }
                if (!chosen) keep_p1t = false;
            }
            if (!chosen) C = 1;
        }
        if (!plan(C)) return BWLA_ERR_INVALID_ARG;
        p.rot_blocks = (int)(clusters * C);
        p.tok_stride = (int)clusters;
    } else {
        p.C = 1; p.rot_blocks = 0;
    }
    int lr_blocks = 0;
    if (r > 0 && Thl) {
        size_t lr_smem = 0;
        lr_blocks = plan_lowrank(p, lr_part, status ? status + kLrCounterWord : nullptr, kPrologueSmemFloats * 4, &lr_smem);
        smem = std::max(smem, lr_smem);
    }
    // A block with this much shared memory leaves no room on its SM for a block of the next kernel of the stream.  Let
    // in early, that kernel would crowd onto the SMs this one leaves free and stay there; so it is let in late, when
    // the blocks of this one are about to leave.
    p.late_trigger = smem > 110 * 1024 ? 1 : 0;
    // Clusters that stay hold their SMs until the last token: the low-rank blocks go first in block order then, or they
    // would only start when the rotation is over.
    p.rot_first = (rotate && p.tok_stride < M && lr_blocks > 0) ? (lr_blocks + C - 1) / C * C : 0;
    int grid = p.rot_first ? p.rot_first + p.rot_blocks : p.rot_blocks + lr_blocks;
    grid = (grid + C - 1) / C * C;
    if (grid == 0) return BWLA_OK;

    static thread_local int configured_device = -1;
    int dev = 0;
    BWLA_CUDA_TRY(cudaGetDevice(&dev));
    if (configured_device != dev) {
        BWLA_CUDA_TRY(cudaFuncSetAttribute(prologue_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPrologueSmemFloats * 4));
        configured_device = dev;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3((unsigned)threads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attrs[2];
    attrs[0].id = cudaLaunchAttributeClusterDimension;
    attrs[0].val.clusterDim.x = (unsigned)C; attrs[0].val.clusterDim.y = 1; attrs[0].val.clusterDim.z = 1;
    attrs[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attrs[1].val.programmaticStreamSerializationAllowed = launch_overlap_allowed();
    cfg.attrs = attrs;
    cfg.numAttrs = 2;
    ProfScope prof(kProfRotateQuant, stream);
    cudaError_t e = cudaLaunchKernelEx(&cfg, prologue_kernel, p);
    if (e != cudaSuccess) { cudaGetLastError(); return cuda_fail(e); }
    return after_launch();
}

// ---------------------------------------------------------------------------------------------
// qsum and interleaving for codes supplied by the caller
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) prepare_codes_kernel(const int8_t* __restrict__ codes, int64_t M, int K,
                                                            int8_t* __restrict__ inter, int32_t* __restrict__ qsum) {
    __shared__ int red_sum;
    const int64_t t = blockIdx.x;
    if (threadIdx.x == 0) red_sum = 0;
    __syncthreads();
    int local = 0;
    const int words = K >> 5;
    for (int g = threadIdx.x; g < words; g += blockDim.x) {
        const uint4* src = reinterpret_cast<const uint4*>(codes + t * (int64_t)K + 32 * g);
        const uint4 a = src[0], b = src[1];
        const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
        int q[32];
#pragma unroll
        for (int j = 0; j < 8; ++j)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                q[4 * j + i] = (int)(int8_t)((w[j] >> (8 * i)) & 0xFF);
                local += q[4 * j + i];
            }
        if (inter) {
            uint32_t o[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                uint32_t v = 0;
#pragma unroll
                for (int i = 0; i < 4; ++i) v |= (uint32_t)(q[j + 8 * i] & 0xFF) << (8 * i);
                o[j] = v;
            }
            uint4* dst = reinterpret_cast<uint4*>(inter + t * (int64_t)K + 32 * g);
            dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
            dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
        }
    }
    local = warp_sum(local);
    if ((threadIdx.x & 31) == 0 && local != 0) atomicAdd(&red_sum, local);
    __syncthreads();
    if (threadIdx.x < kQsumParts && qsum) qsum[t * kQsumParts + threadIdx.x] = threadIdx.x == 0 ? red_sum : 0;
}

int launch_prepare_codes(const int8_t* codes, int64_t M, int64_t K, int8_t* codes_interleaved, int32_t* qsum,
                         cudaStream_t stream) {
    if (M == 0) return BWLA_OK;
    ProfScope prof(kProfPrepare, stream);
    prepare_codes_kernel<<<(unsigned)M, 256, 0, stream>>>(codes, M, (int)K, codes_interleaved, qsum);
    return after_launch();
}

}  // namespace bwla
