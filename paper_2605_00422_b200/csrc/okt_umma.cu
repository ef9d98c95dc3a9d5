// Online OKT + per-token symmetric quantiser on the tcgen05 tensor cores.
//
//   X = reshape(x_t, n1 x n2) (row-major),  Y = P1^T X P2,  amax = max|Y|,  q = clamp(rne(Y * (qmax / amax)), +-qmax)
//
// (Sec. 3.1: the rotation R = R1 (x) R2 evaluated as two small contractions on the reshaped vector; Sec. 4.1:
// per-token activation quantisation.)  Both contractions run as dense bf16 MMAs with fp32 accumulators in tensor
// memory, and still deliver fp32 accuracy: x is bf16 already, the fp32 factors P1, P2 are kept as three bf16 terms
// (hi + mid + lo carry all 24 bits; they are split once per layer by prepare_okt_kernel), the fp32 intermediate is
// split the same way on the fly, and the term products whose weight is at least 2^-16 of the leading one are summed
// (3 for the first contraction, 6 for the second), the small ones first.
//
// Work of one CTA, per token (the two contractions are chained through tensor memory, nothing goes to shared memory
// in between):
//   stage A   Z^T[d][a] = sum_b P2[b][d] X[a][b]      A = rows d of P2^T (shared memory, K-major, three terms),
//                                                     B = X as it lies in global memory: rows a, K = b (one TMA load
//                                                     per K-atom, rows beyond n1 and columns beyond n2 zero-filled),
//                                                     D = 128 lanes (d) x n1p columns (a), fp32
//   stage B   read Z^T back (tcgen05.ld), split each value into three bf16 terms, write them as the A operand of the
//             second contraction (tcgen05.st; two bf16 per 32-bit column)
//   stage C   Y^T[d][c] = sum_a Z^T[d][a] P1[a][c]    A = the terms of Z^T in tensor memory,
//                                                     B = rows c of P1^T (shared memory, K-major, three terms),
//                                                     D = 128 lanes (d) x columns c (over the columns of stage A's D)
//   stage D   absmax over the CTA (and, where a token is spread over several CTAs, over their cluster through
//             distributed shared memory), then a second read of Y^T: scale, round, clamp, store the codes
// A token whose factors do not fit one CTA is spread over a cluster: up to two tiles of the lanes (n2 > 128) times up
// to four slabs of the output columns c (when the terms of P1^T and P2^T do not fit shared memory together); the CTAs
// of a cluster repeat stage A and share nothing but the absmax.
// Warp 0 moves data (constants once, then one token's X per step), warp 1 allocates tensor memory and issues the
// MMAs, warps 2..13 are the ALU warps of stages B and D (three per tensor-memory lane quarter, taking 16-column chunks
// in turn).  Clusters stay on their SMs and take tokens in turn, so the constants are fetched once per CTA.
//
// The blocks behind the rotation CTAs evaluate T = V x for the PSP low-rank branch (prologue_roles.cuh).
//
// Launched with programmatic stream serialisation: the constants are fetched before the preceding kernel of the stream
// has finished; x is read, and everything is stored, after it.  Every wait is bounded (umma_wait.cuh).
#include <cuda_bf16.h>

#include <algorithm>

#include "bwla_common.cuh"
#include "prologue_roles.cuh"
#include "umma_ptx.cuh"
#include "umma_wait.cuh"
#include "tensor_map.cuh"

namespace bwla {

constexpr int kOktAluPerQuarter = 3;      // ALU warps per tensor-memory lane quarter
constexpr int kOktAluWarps = 4 * kOktAluPerQuarter;
constexpr int kOktAluThreads = 32 * kOktAluWarps;
constexpr int kOktThreads = 64 + kOktAluThreads;   // warp 0: copies; warp 1: MMA issue; then the ALU warps
constexpr int kOktChunksD = 3;            // 16-column chunks of Y^T one ALU warp holds in registers: 128 columns / 16 / 3 warps, rounded up
constexpr int kOktMaxSmem = 231424;       // the 227 KB a block may have, less 1 KB for the static shared memory of the roles
constexpr int kOktBarBytes = 1024;        // barriers and small per-CTA state behind the operand tiles

// Byte offset inside a K-major operand block in the canonical swizzled layout: rows of atom_bytes, the 16-byte chunk
// index XORed with the low bits of (offset >> 7).
__host__ __device__ inline uint32_t okt_swizzle(uint32_t off, int atom_bytes) {
    return off ^ (((off >> 7) & (uint32_t)((atom_bytes >> 4) - 1)) << 4);
}

__host__ __device__ inline int round_up_int(int v, int m) { return (v + m - 1) / m * m; }
// Swizzle span (bytes of one K-atom row) for an operand whose contraction depth is `k` elements, and the depth padded
// to whole atoms.  MMAs on 32-byte atoms were measured about 2.5 times slower than on 64- or 128-byte ones, so the depth
// is padded to the next multiple of 32 elements rather than taking 32-byte atoms, unless k <= 16.
static int pick_atom(int k, int* padded) {
    if (k <= 16) { *padded = 16; return 32; }
    if (k % 64 == 0) { *padded = k; return 128; }
    *padded = round_up_int(k, 32);
    return *padded % 64 == 0 ? 128 : 64;
}

bool okt_geometry(int n1, int n2, OktGeom* out) {
    if (n1 < 1 || n2 < 8 || n2 % 8 != 0 || n2 > 256 || n1 > 192) return false;
    OktGeom g{};
    g.n1 = n1; g.n2 = n2; g.K = n1 * n2;
    g.atom2 = pick_atom(n2, &g.n2p);
    g.atom1 = pick_atom(n1, &g.n1p);
    g.dt_count = n2 > 128 ? 2 : 1;
    g.x_bytes = g.n1p * g.n2p * 2;
    int tc = 32;
    while (tc < (5 * g.n1p + 1) / 2) tc *= 2;
    if (tc > 512) return false;
    g.tmem_cols = tc;
    const int chunks = g.n1p / 16;
    // Two lane tiles: the boundary on a multiple of 32 rows when that fits (a warp's 32 code bytes of a column then fill
    // one whole 32-byte sector), else on a multiple of 8.
    for (int align = (g.dt_count == 2 && n2 % 32 == 0) ? 32 : 8; align >= 8; align = (align == 32 ? 8 : 0))
    for (int cs = 1; cs <= 4; cs *= 2) {
        g.dt_rows = g.dt_count == 1 ? n2 : round_up_int((n2 + 1) / 2, align);
        if (g.dt_count == 2 && g.dt_rows >= n2) continue;
        g.p2t_bytes = 3 * g.dt_rows * g.n2p * 2;
        const int per = (chunks + cs - 1) / cs;
        if (cs > 1 && (cs - 1) * per >= chunks) continue;       // a slab would be empty
        g.cs_count = cs;
        g.cs_cols = per * 16;
        if (g.cs_cols > 16 * kOktAluPerQuarter * kOktChunksD) continue;   // the ALU warps keep their chunks of Y^T in registers
        g.p1t_bytes = 3 * g.cs_cols * g.n1p * 2;
        g.p1t_off = round_up_int(g.p2t_bytes, 1024);
        g.x_off = g.p1t_off + round_up_int(g.p1t_bytes, 1024);
        g.bar_off = g.x_off + round_up_int(g.x_bytes, 1024);
        int total = g.bar_off + kOktBarBytes;
        // the MMAs of stage A read 128 rows of every block of P2^T terms, whatever the tile's row count: what lies
        // behind the last block must still be this CTA's shared memory
        total = std::max(total, g.p2t_bytes + (128 - std::min(128, g.dt_rows)) * g.atom2);
        g.smem_bytes = total + 1024;                              // + slack for 1024-byte alignment
        if (g.smem_bytes <= kOktMaxSmem && g.dt_count * cs <= 8) { *out = g; return true; }
    }
    return false;
}

size_t okt_prepared_bytes(const OktGeom& g) {
    return (size_t)g.dt_count * round_up_int(g.p2t_bytes, 1024) + (size_t)g.cs_count * round_up_int(g.p1t_bytes, 1024);
}

// ---------------------------------------------------------------------------------------------
// once per layer: P1, P2 (fp32) -> the bf16 terms of P2^T tiles and P1^T slabs, in the layout the MMAs read
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) prepare_okt_kernel(OktGeom g, const float* __restrict__ P1, const float* __restrict__ P2,
                                                         uint8_t* __restrict__ prepared) {
    const int p2_region = round_up_int(g.p2t_bytes, 1024), p1_region = round_up_int(g.p1t_bytes, 1024);
    const int64_t p2_elems = (int64_t)g.dt_count * g.dt_rows * g.n2p;       // (tile, row d, column b)
    const int64_t p1_elems = (int64_t)g.cs_count * g.cs_cols * g.n1p;       // (slab, row c, column a)
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < p2_elems + p1_elems; i += (int64_t)gridDim.x * blockDim.x) {
        float v = 0.f;
        uint8_t* region;
        int rows, row, kk, atom, kdim;
        if (i < p2_elems) {
            const int tile = (int)(i / ((int64_t)g.dt_rows * g.n2p));
            const int rem = (int)(i - (int64_t)tile * g.dt_rows * g.n2p);
            row = rem / g.n2p; kk = rem - row * g.n2p;
            const int d = tile * g.dt_rows + row;
            if (d < g.n2 && kk < g.n2) v = P2[(size_t)kk * g.n2 + d];                  // P2^T[d][b]
            region = prepared + (size_t)tile * p2_region;
            rows = g.dt_rows; atom = g.atom2; kdim = g.n2p;
        } else {
            const int64_t i1 = i - p2_elems;
            const int slab = (int)(i1 / ((int64_t)g.cs_cols * g.n1p));
            const int rem = (int)(i1 - (int64_t)slab * g.cs_cols * g.n1p);
            row = rem / g.n1p; kk = rem - row * g.n1p;
            const int c = slab * g.cs_cols + row;
            if (c < g.n1 && kk < g.n1) v = P1[(size_t)kk * g.n1 + c];                  // P1^T[c][a]
            region = prepared + (size_t)g.dt_count * p2_region + (size_t)slab * p1_region;
            rows = g.cs_cols; atom = g.atom1; kdim = g.n1p;
        }
        __nv_bfloat16 t[3];
        split3(v, t[0], t[1], t[2]);
        const int ae = atom >> 1;                                   // elements per K-atom
        const int atoms = kdim / ae;
        const int j = kk / ae, kin = kk - j * ae;
        const uint32_t in_block = okt_swizzle((uint32_t)(row * atom + kin * 2), atom);
#pragma unroll
        for (int h = 0; h < 3; ++h)
            *reinterpret_cast<__nv_bfloat16*>(region + (size_t)(h * atoms + j) * rows * atom + in_block) = t[h];
    }
}

int launch_prepare_okt(const OktGeom& g, const float* P1, const float* P2, void* prepared, cudaStream_t stream) {
    const int64_t elems = (int64_t)g.dt_count * g.dt_rows * g.n2p + (int64_t)g.cs_count * g.cs_cols * g.n1p;
    const int blocks = (int)std::min<int64_t>((elems + 255) / 256, 1024);
    ProfScope prof(kProfPrepare, stream);
    prepare_okt_kernel<<<blocks, 256, 0, stream>>>(g, P1, P2, (uint8_t*)prepared);
    return after_launch();
}

// ---------------------------------------------------------------------------------------------
// per call
// ---------------------------------------------------------------------------------------------
struct OktKernelParams {
    OktGeom g;
    int64_t M;
    int bits, asym;
    int n_problems;
    int clusters_per_problem;       // cluster i of a problem takes tokens i, i + clusters_per_problem, ...
    int rot_first, rot_ctas;        // rotation CTAs are blocks [rot_first, rot_first + rot_ctas)
    OktProblem prob[kOktMaxProblems];
    uint32_t* status;
    // low-rank blocks: problem i owns blocks [lr_begin[i], lr_begin[i + 1]) counted among the non-rotation blocks
    int lr_begin[kOktMaxProblems + 1];
    PrologueParams lr[kOktMaxProblems];
};

// Two fp32 values into their three bf16 terms, two per word (low half: the first value): packed conversions, and the
// bf16 -> fp32 direction is a shift or a mask.
__device__ __forceinline__ uint32_t cvt_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ void split3_pair(float a, float b, uint32_t& h, uint32_t& m, uint32_t& l) {
    h = cvt_bf16x2(a, b);
    const float ra = a - __uint_as_float(h << 16), rb = b - __uint_as_float(h & 0xFFFF0000u);
    m = cvt_bf16x2(ra, rb);
    l = cvt_bf16x2(ra - __uint_as_float(m << 16), rb - __uint_as_float(m & 0xFFFF0000u));
}

// ALU warps only: barrier 1 with an OR over a predicate (a uniform decision for all of them), barrier 2 plain.
__device__ __forceinline__ bool alu_barrier_or(bool pred) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred P, Q;\n\t"
        "setp.ne.b32 P, %1, 0;\n\t"
        "barrier.cta.red.or.pred Q, 1, %2, P;\n\t"
        "selp.u32 %0, 1, 0, Q;\n\t}"
        : "=r"(out) : "r"((uint32_t)pred), "r"(kOktAluThreads) : "memory");
    return out != 0;
}
__device__ __forceinline__ void alu_barrier() { asm volatile("bar.sync 2, %0;" ::"r"(kOktAluThreads) : "memory"); }

__device__ __forceinline__ bool warp_wait_cluster(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    for (uint32_t i = 0; i < kWaitLimit; ++i) {
        const bool done = mbar_try_wait_cluster(bar, parity, kParkNs);
        if (__all_sync(0xFFFFFFFFu, done)) return true;
        if (*abort_flag) return false;
    }
    return false;
}

// One term of a contraction: `atoms` K-atoms of STEPS k-steps (16 elements, 32 bytes = 2 descriptor units) each, both
// operands in shared memory, blocks of blk_a / blk_b descriptor units per K-atom.  `clear` starts the accumulator afresh.
template <int STEPS>
__device__ __forceinline__ void issue_term_ss(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t blk_a, uint32_t b_lo, uint32_t b_hi,
                                              uint32_t blk_b, int atoms, uint32_t idesc, bool clear) {
    if (clear) ptx::mma_f16_ss_words<false>(d_tmem, a_lo, a_hi, b_lo, b_hi, idesc);
    else ptx::mma_f16_ss_words<true>(d_tmem, a_lo, a_hi, b_lo, b_hi, idesc);
#pragma unroll
    for (int s = 1; s < STEPS; ++s) ptx::mma_f16_ss_words<true>(d_tmem, a_lo + 2u * s, a_hi, b_lo + 2u * s, b_hi, idesc);
    for (int at = 1; at < atoms; ++at) {
        a_lo += blk_a; b_lo += blk_b;
#pragma unroll
        for (int s = 0; s < STEPS; ++s) ptx::mma_f16_ss_words<true>(d_tmem, a_lo + 2u * s, a_hi, b_lo + 2u * s, b_hi, idesc);
    }
}
// The same with the A operand in tensor memory: 8 columns (16 bf16) per k-step.
template <int STEPS>
__device__ __forceinline__ void issue_term_ts(uint32_t d_tmem, uint32_t a_col, uint32_t b_lo, uint32_t b_hi, uint32_t blk_b, int atoms,
                                              uint32_t idesc, bool clear) {
    if (clear) ptx::mma_f16_ts_words<false>(d_tmem, a_col, b_lo, b_hi, idesc);
    else ptx::mma_f16_ts_words<true>(d_tmem, a_col, b_lo, b_hi, idesc);
#pragma unroll
    for (int s = 1; s < STEPS; ++s) ptx::mma_f16_ts_words<true>(d_tmem, a_col + 8u * s, b_lo + 2u * s, b_hi, idesc);
    for (int at = 1; at < atoms; ++at) {
        a_col += 8u * STEPS; b_lo += blk_b;
#pragma unroll
        for (int s = 0; s < STEPS; ++s) ptx::mma_f16_ts_words<true>(d_tmem, a_col + 8u * s, b_lo + 2u * s, b_hi, idesc);
    }
}

__global__ void __launch_bounds__(kOktThreads, 1)
okt_umma_kernel(const __grid_constant__ CUtensorMap x_map, const OktKernelParams p) {
    extern __shared__ __align__(16) uint8_t smem_raw[];
    const int b = (int)blockIdx.x;
    if (b < p.rot_first || b >= p.rot_first + p.rot_ctas) {
        // ---------------- T = V x blocks ----------------
        const int lb = b < p.rot_first ? b : b - p.rot_ctas;
        int i = 0;
        while (i + 1 < p.n_problems && lb >= p.lr_begin[i + 1]) ++i;
        if (lb >= p.lr_begin[p.n_problems]) return;
        const PrologueParams& lp = p.lr[i];
        float* fsmem = reinterpret_cast<float*>(smem_raw);
        const int rel = lb - p.lr_begin[i];
        if (lp.lr_wide == 1) lowrank_role<8, 8>(lp, rel, fsmem);
        else if (lp.lr_wide == 2) lowrank_mma_role(lp, rel, fsmem);
        else lowrank_role<2, 16>(lp, rel, fsmem);
        return;
    }

    const OktGeom& g = p.g;
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* p2t = smem;
    uint8_t* p1t = smem + g.p1t_off;
    uint8_t* xs = smem + g.x_off;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + g.bar_off);
    uint64_t* const_full = bars + 0;
    uint64_t* x_full = bars + 1;
    uint64_t* x_empty = bars + 2;
    uint64_t* d1_full = bars + 3;
    uint64_t* a2_full = bars + 4;
    uint64_t* d2_full = bars + 5;
    uint64_t* d_free = bars + 6;
    uint64_t* xbar = bars + 7;                      // [2] absmax of every CTA of the cluster has arrived (by token parity)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 10);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 10) + 1;
    int* red_sum = reinterpret_cast<int*>(bars + 11);
    float* red_max = reinterpret_cast<float*>(bars + 12);        // [16] largest value (symmetric: largest magnitude) per ALU warp
    float* slots = red_max + 16;                                 // [2][8] the same per CTA of the cluster, by token parity
    float* red_min = slots + 16;                                 // [16], [2][8]: smallest value (asymmetric quantiser only)
    float* slots_min = red_min + 16;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int D = g.dt_count * g.cs_count;
    const int rank = D > 1 ? (int)cluster_ctarank() : 0;
    const int dt = rank % g.dt_count, cs = rank / g.dt_count;
    const int cl = (b - p.rot_first) / D;
    const int prob_i = cl / p.clusters_per_problem;
    const int64_t tok0 = cl % p.clusters_per_problem;
    const OktProblem pr = p.prob[prob_i];
    const int d0 = dt * g.dt_rows;
    const int rows = min(g.dt_rows, g.n2 - d0);               // lanes that hold something
    const int c0 = cs * g.cs_cols;
    const int n1p = g.n1p;
    const int ncols = min(g.cs_cols, n1p - c0);               // columns of Y^T this CTA evaluates (a multiple of 16)
    const int ntok = tok0 < p.M ? (int)((p.M - tok0 + p.clusters_per_problem - 1) / p.clusters_per_problem) : 0;

    if (threadIdx.x == 0) {
        // the constants first: their copies run while the rest of the set-up (barriers, tensor memory) completes
        mbar_init(const_full, 1);
        fence_barrier_init();
        fence_proxy_async();
        const int p2_region = (g.p2t_bytes + 1023) / 1024 * 1024, p1_region = (g.p1t_bytes + 1023) / 1024 * 1024;
        const uint8_t* src2 = pr.prepared + (size_t)dt * p2_region;
        const uint8_t* src1 = pr.prepared + (size_t)g.dt_count * p2_region + (size_t)cs * p1_region;
        mbar_expect_tx(const_full, (uint32_t)(g.p2t_bytes + g.p1t_bytes));
        for (int off = 0; off < g.p2t_bytes; off += 16384)
            tma_bulk_g2s(p2t + off, src2 + off, (uint32_t)min(16384, g.p2t_bytes - off), const_full);
        for (int off = 0; off < g.p1t_bytes; off += 16384)
            tma_bulk_g2s(p1t + off, src1 + off, (uint32_t)min(16384, g.p1t_bytes - off), const_full);
        *abort_flag = 0;
        red_sum[0] = 0; red_sum[1] = 0;
        mbar_init(x_full, 1);
        mbar_init(x_empty, 1);
        mbar_init(d1_full, 1);
        mbar_init(a2_full, kOktAluThreads / 32);
        mbar_init(d2_full, 1);
        mbar_init(d_free, kOktAluThreads / 32);
        mbar_init(&xbar[0], (uint32_t)D);
        mbar_init(&xbar[1], (uint32_t)D);
        fence_barrier_init();
        fence_proxy_async();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, (uint32_t)g.tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    if (D > 1) {
        // nobody touches a neighbour's barriers or slots before that neighbour has set them up
        cluster_arrive_release();
        cluster_wait_acquire();
    }
    // the next kernel of the stream may start its own independent preamble now
    griddep_launch_dependents();

    const uint32_t tm_d = tmem_base;                           // fp32 accumulator of both stages, n1p columns
    const uint32_t tm_a2 = tmem_base + (uint32_t)n1p;          // three terms of Z^T, n1p / 2 columns each
    const int atoms2 = (g.n2p * 2) / g.atom2;
    const int atoms1 = (n1p * 2) / g.atom1;

    if (warp == 0) {
        // ---------------- copies: the layer's constants once, then one token's X per step ----------------
        if (elect_one()) {
            tma_prefetch_desc(&x_map);
            griddep_wait();                           // x may be the output of the preceding kernel
            if (p.status && *reinterpret_cast<volatile uint32_t*>(p.status) != 0) *abort_flag = 1;   // the call already failed
            const int ae2 = g.atom2 >> 1;
            for (int it = 0; it < ntok && !*abort_flag; ++it) {
                if (it > 0 && !wait_or_abort(x_empty, (uint32_t)((it - 1) & 1), abort_flag)) { give_up(p.status, abort_flag, 0x60); break; }
                mbar_expect_tx(x_full, (uint32_t)g.x_bytes);
                const int t = (int)(tok0 + (int64_t)it * p.clusters_per_problem);
                for (int j = 0; j < atoms2; ++j)
                    tma_load_3d(xs + (size_t)j * n1p * g.atom2, &x_map, j * ae2, 0, t, x_full);
            }
            if (*abort_flag) for (int i = 0; i < 500; ++i) __nanosleep(100);   // let copies in flight land
        }
    } else if (warp == 1) {
        // ---------------- MMA issue ----------------
        if (elect_one()) {
            // D = f32, A = B = bf16, both K-major, M = 128
            const uint32_t idesc_a = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n1p >> 3) << 17) | ((128u >> 4) << 24);
            const uint32_t idesc_c = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(ncols >> 3) << 17) | ((128u >> 4) << 24);
            // Shared-memory descriptors differ only in their start-address field (16-byte units in the low word): one
            // descriptor per operand is built here, the loops below only add.  This thread is a chain of dependent scalar
            // instructions; everything that can be precomputed is.
            const uint64_t dP2 = smem_desc_kmajor(smem_u32(p2t), g.atom2), dX = smem_desc_kmajor(smem_u32(xs), g.atom2),
                           dP1 = smem_desc_kmajor(smem_u32(p1t), g.atom1);
            const uint32_t blk_a = (uint32_t)(g.dt_rows * g.atom2) >> 4;      // one (term, K-atom) block of P2^T
            const uint32_t blk_x = (uint32_t)(n1p * g.atom2) >> 4;            // one K-atom block of X
            const uint32_t blk_p1 = (uint32_t)(g.cs_cols * g.atom1) >> 4;     // one (term, K-atom) block of P1^T
            const int steps2 = g.atom2 / 32, steps1 = g.atom1 / 32;           // MMAs (K = 16) per K-atom: 1, 2 or 4
            const uint32_t lo_p2 = (uint32_t)dP2, hi_p2 = (uint32_t)(dP2 >> 32), lo_x = (uint32_t)dX, hi_x = (uint32_t)(dX >> 32),
                           lo_p1 = (uint32_t)dP1, hi_p1 = (uint32_t)(dP1 >> 32);
            bool ok = wait_or_abort(const_full, 0, abort_flag);
            if (!ok) give_up(p.status, abort_flag, 0x61);
            for (int it = 0; it < ntok && ok; ++it) {
                const uint32_t ph = (uint32_t)(it & 1);
                if (it > 0 && !wait_or_abort(d_free, ph ^ 1u, abort_flag)) { give_up(p.status, abort_flag, 0x62); break; }
                if (!wait_or_abort(x_full, ph, abort_flag)) { give_up(p.status, abort_flag, 0x63); break; }
                tc_fence_after();
                // stage A: the small terms first, so that the large partial sums meet as few additions as possible
                for (int h = 2; h >= 0; --h) {
                    const uint32_t a_lo = lo_p2 + (uint32_t)(h * atoms2) * blk_a;
                    if (steps2 == 4) issue_term_ss<4>(tm_d, a_lo, hi_p2, blk_a, lo_x, hi_x, blk_x, atoms2, idesc_a, h == 2);
                    else if (steps2 == 2) issue_term_ss<2>(tm_d, a_lo, hi_p2, blk_a, lo_x, hi_x, blk_x, atoms2, idesc_a, h == 2);
                    else issue_term_ss<1>(tm_d, a_lo, hi_p2, blk_a, lo_x, hi_x, blk_x, atoms2, idesc_a, h == 2);
                }
                tc_commit(x_empty);
                tc_commit(d1_full);
                if (!wait_or_abort(a2_full, ph, abort_flag)) { give_up(p.status, abort_flag, 0x64); break; }
                tc_fence_after();
                // stage C: (term of Z^T, term of P1^T), smallest products first
#pragma unroll
                for (int pair = 0; pair < 6; ++pair) {
                    constexpr int hz_of[6] = {2, 0, 1, 1, 0, 0};
                    constexpr int hp_of[6] = {0, 2, 1, 0, 1, 0};
                    const uint32_t a_col = tm_a2 + (uint32_t)(hz_of[pair] * (n1p >> 1));
                    const uint32_t b_lo = lo_p1 + (uint32_t)(hp_of[pair] * atoms1) * blk_p1;
                    if (steps1 == 4) issue_term_ts<4>(tm_d, a_col, b_lo, hi_p1, blk_p1, atoms1, idesc_c, pair == 0);
                    else if (steps1 == 2) issue_term_ts<2>(tm_d, a_col, b_lo, hi_p1, blk_p1, atoms1, idesc_c, pair == 0);
                    else issue_term_ts<1>(tm_d, a_col, b_lo, hi_p1, blk_p1, atoms1, idesc_c, pair == 0);
                }
                tc_commit(d2_full);
            }
        }
    } else {
        // ---------------- ALU warps: stage B and stage D ----------------
        const int q = warp & 3;                        // tensor-memory lane quarter this warp may touch
        const int part = (warp - 2) >> 2;              // which of the warps of that quarter
        const int e = threadIdx.x - 64;                // index among the ALU threads
        const int lane_d = q * 32 + lane;              // lane of the accumulator = row d of this CTA's tile
        const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
        const bool lane_valid = lane_d < rows;
        const bool quarter_valid = q * 32 < rows;      // warp-uniform: a quarter without valid lanes only keeps the protocol
        const int d = d0 + lane_d;
        const int qmax = (1 << (p.bits - 1)) - 1;
        const bool asym = p.asym != 0;
        const int chunks_b = n1p >> 4, chunks_d = ncols >> 4;
        bool failed = false;
        bool dep_waited = false;
        // Stage B of one token: every chunk's read is requested while the one before it is split and written back.
        auto stage_b = [&](uint32_t phb) {
            if (!failed && !warp_wait(d1_full, phb, abort_flag)) { give_up(p.status, abort_flag, 0x70); failed = true; }
            if (failed) return;
            tc_fence_after();
            if (quarter_valid) {
                uint32_t v[16];
                int ch = part;
                if (ch < chunks_b) tmem_ld_32x16(tm_d + lane_addr + 16 * ch, v);
                while (ch < chunks_b) {
                    tc_wait_ld();
                    float f[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) f[i] = __uint_as_float(v[i]);
                    const int nxt = ch + kOktAluPerQuarter;
                    if (nxt < chunks_b) tmem_ld_32x16(tm_d + lane_addr + 16 * nxt, v);
                    uint32_t th[8], tmid[8], tl[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) split3_pair(f[2 * i], f[2 * i + 1], th[i], tmid[i], tl[i]);
                    tmem_st_32x8(tm_a2 + lane_addr + 8 * ch, th);
                    tmem_st_32x8(tm_a2 + lane_addr + (n1p >> 1) + 8 * ch, tmid);
                    tmem_st_32x8(tm_a2 + lane_addr + n1p + 8 * ch, tl);
                    ch = nxt;
                }
                tc_wait_st();
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(a2_full);
        };
        // The ALU warps run one stage ahead of themselves: stage B of token it + 1 sits in the middle of stage D of token
        // it (after its accumulator has gone to registers and its absmax has been sent off), so that the second
        // contraction of the next token, and the exchange of the absmax inside a cluster, run under the rounding and
        // the stores of this one.
        // every CTA of the cluster leaves its own part of the token's code sum; the consumer adds the parts
        auto put_qsum = [&](int64_t tq, int parq) {
            if (pr.qsum) {
                pr.qsum[tq * kQsumParts + rank] = red_sum[parq];
                if (rank == 0)
                    for (int c = D; c < kQsumParts; ++c) pr.qsum[tq * kQsumParts + c] = 0;
            }
            red_sum[parq] = 0;
        };
        // Where element k of a token is stored: at k, or (interleaved layout) inside each group of 32 at byte 4 (k % 8) +
        // (k % 32) / 8.  The codes go straight to global memory, one byte per lane: the 32 lanes of a warp fill one
        // 32-byte sector per column (two halves where n2 is not a multiple of 32).  16 columns on, and 4 columns on,
        // the position inside the group repeats (n2 is a multiple of 8), so four offsets per thread cover every column.
        const bool interleave = pr.codes_layout != 0;
        int off[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int k = (c0 + 16 * part) * g.n2 + d + r * g.n2, kl = k & 31;
            off[r] = (interleave ? ((k & ~31) | ((kl & 7) << 2) | (kl >> 3)) : k) - r * g.n2;
        }
        if (ntok > 0) stage_b(0u);
        for (int it = 0; it < ntok; ++it) {
            const uint32_t ph = (uint32_t)(it & 1);
            const int64_t t = tok0 + (int64_t)it * p.clusters_per_problem;
            // ---- stage D: this warp's chunks of Y^T go to registers (all reads in flight at once) and the accumulator is
            //      handed back at once: the next token's stage A runs under the reduction below
            if (!failed && !warp_wait(d2_full, ph, abort_flag)) { give_up(p.status, abort_flag, 0x71); failed = true; }
            uint32_t yv[kOktChunksD][16];
            if (!failed && quarter_valid) {
                tc_fence_after();
#pragma unroll
                for (int j = 0; j < kOktChunksD; ++j)
                    if (part + j * kOktAluPerQuarter < chunks_d) tmem_ld_32x16(tm_d + lane_addr + 16 * (part + j * kOktAluPerQuarter), yv[j]);
                tc_wait_ld();
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0 && !failed) mbar_arrive(d_free);
            // Columns beyond n1 are exact zeros (the padding rows of P1^T are), which changes neither reduction: the
            // largest magnitude is at least zero and the asymmetric range contains zero by definition.  Lanes beyond the
            // tile's rows hold anything and are masked once, after the loops.
            float amax = 0.f, vmin = 0.f;                       // asymmetric: amax holds the largest value, zero included
            if (!failed && quarter_valid) {
                float m0 = 0.f, m1 = 0.f, l0 = 0.f, l1 = 0.f;  // two chains each
#pragma unroll
                for (int j = 0; j < kOktChunksD; ++j) {
                    if (part + j * kOktAluPerQuarter < chunks_d) {
                        if (!asym) {
#pragma unroll
                            for (int i = 0; i < 16; i += 2) {
                                m0 = fmaxf(m0, fabsf(__uint_as_float(yv[j][i])));
                                m1 = fmaxf(m1, fabsf(__uint_as_float(yv[j][i + 1])));
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < 16; i += 2) {
                                const float a = __uint_as_float(yv[j][i]), c = __uint_as_float(yv[j][i + 1]);
                                m0 = fmaxf(m0, a); m1 = fmaxf(m1, c);
                                l0 = fminf(l0, a); l1 = fminf(l1, c);
                            }
                        }
                    }
                }
                if (lane_valid) { amax = fmaxf(m0, m1); vmin = fminf(l0, l1); }
            }
            // both are non-negative here (NaNs aside), so their bit patterns order like the values: one warp-wide integer
            // reduction each instead of five shuffle steps
            amax = __uint_as_float(__reduce_max_sync(0xFFFFFFFFu, __float_as_uint(fmaxf(amax, 0.f))));
            if (asym) vmin = -__uint_as_float(__reduce_max_sync(0xFFFFFFFFu, __float_as_uint(fmaxf(-vmin, 0.f))));
            if (lane == 0) { red_max[warp - 2] = amax; red_min[warp - 2] = vmin; }
            // one decision for all ALU warps: a warp that gave up must not leave the others alone at a barrier
            if (alu_barrier_or(failed || *abort_flag != 0)) break;
            if (e == 0 && it > 0) put_qsum(t - p.clusters_per_problem, (it - 1) & 1);
            amax = 0.f; vmin = 0.f;
#pragma unroll
            for (int wi = 0; wi < kOktAluWarps; ++wi) { amax = fmaxf(amax, red_max[wi]); vmin = fminf(vmin, red_min[wi]); }
            const int par = it & 1;
            if (D > 1 && e < D) {
                // this CTA's absmax into slot [par][rank] of CTA e, then one arrival on that CTA's barrier
                st_shared_cluster_u32(map_shared_rank(smem_u32(slots + par * 8 + rank), (uint32_t)e), __float_as_uint(amax));
                st_shared_cluster_u32(map_shared_rank(smem_u32(slots_min + par * 8 + rank), (uint32_t)e), __float_as_uint(vmin));
                mbar_arrive_remote(map_shared_rank(smem_u32(&xbar[par]), (uint32_t)e));
            }
            // symmetric: codes in [-qmax, qmax] around zero.  Asymmetric (Sec. 4.1): u = rne(y * inv) + zero in [0, 2^b - 1]
            // with an integer zero point; what is stored is u - 2^(b-1) (+ the caller's bias), so that it fits int8.
            float inv = 0.f, scale = 1.f, zero_f = 0.f, lo_c = -(float)qmax, hi_c = (float)qmax, half_f = 0.f;
            auto set_scales = [&]() {
                if (!asym) {
                    if (amax != 0.f) { inv = __fdiv_rn((float)qmax, amax); scale = __fdiv_rn(amax, (float)qmax); }
                } else {
                    const float levels = (float)((1 << p.bits) - 1);
                    const float range = __fsub_rn(amax, vmin);
                    if (range != 0.f) { inv = __fdiv_rn(levels, range); scale = __fdiv_rn(range, levels); }
                    const float tz = __fmul_rn(-vmin, inv);
                    zero_f = fminf(fmaxf(__fadd_rn(__fadd_rn(tz, 12582912.f), -12582912.f), 0.f), levels);
                    lo_c = 0.f; hi_c = levels; half_f = (float)(1 << (p.bits - 1));
                }
            };
            // (a CTA that owns its token alone has the absmax now: the divisions go in front of stage B, which still
            // waits for the next token's stage A at this point)
            if (D == 1) set_scales();
            if (it + 1 < ntok) stage_b(ph ^ 1u);
            if (D > 1) {
                if (!failed && !warp_wait_cluster(&xbar[par], (uint32_t)((it >> 1) & 1), abort_flag)) { give_up(p.status, abort_flag, 0x72); failed = true; }
                if (!failed) {
                    amax = 0.f; vmin = 0.f;
                    for (int c = 0; c < D; ++c) { amax = fmaxf(amax, slots[par * 8 + c]); vmin = fminf(vmin, slots_min[par * 8 + c]); }
                }
                set_scales();
            }
            const float store_shift = (float)pr.code_bias - half_f;
            // nothing is stored to global memory before the preceding kernel of the stream has completed
            if (!dep_waited) { griddep_wait(); dep_waited = true; }
            // ---- codes.  With B = 1.5 * 2^23 + an even integer, fl(v + B) = B + rne(v) for |v| < 2^22: one addition
            //      rounds to nearest-even (the sum's ulp is 1, and ties go to an even sum, hence to an even rne(v)) and
            //      leaves the integer in the low mantissa bits; no float-to-integer conversions, which are slow
            //      instructions.  Everything added to the rounded product (zero point, shift of the stored code) goes
            //      into B except its parity bit, which is added to the bit pattern.  The clamp acts on the sum (products
            //      beyond the range only come from rounding of the reciprocal and of the zero point).  The stored byte
            //      is the low byte of the pattern, and the patterns themselves are summed for the code sum: every one
            //      is 0x4B400000 + the stored code.
            const int shift_i = (int)(zero_f + store_shift);                 // small integer, exact
            const uint32_t odd = (uint32_t)(shift_i & 1);
            const float bias_even = 12582912.f + (float)(shift_i - (int)odd);
            const float lo_b = 12582912.f + (lo_c + store_shift) - (float)odd, hi_b = 12582912.f + (hi_c + store_shift) - (float)odd;
            uint32_t usum = 0u;
            int counted = 0;
            int8_t* ct = pr.codes + t * (int64_t)g.K;
            if (!failed && quarter_valid) {
#pragma unroll
                for (int j = 0; j < kOktChunksD; ++j) {
                    const int ch = part + j * kOktAluPerQuarter;
                    const int cols_left = g.n1 - (c0 + 16 * ch);             // warp-uniform
                    if (ch < chunks_d && cols_left > 0) {
                        const int k0 = (c0 + 16 * ch) * g.n2 + d;
                        int8_t* const cb = ct + (int64_t)(16 * kOktAluPerQuarter * j) * g.n2;
                        if (cols_left >= 16) {
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                const float sv = fminf(fmaxf(__fadd_rn(__fmul_rn(__uint_as_float(yv[j][i]), inv), bias_even), lo_b), hi_b);
                                const uint32_t w = __float_as_uint(sv) + odd;
                                usum += w;
                                if (lane_valid) cb[off[i & 3] + i * g.n2] = (int8_t)w;
                            }
                            counted += 16;
                        } else {
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                const float sv = fminf(fmaxf(__fadd_rn(__fmul_rn(__uint_as_float(yv[j][i]), inv), bias_even), lo_b), hi_b);
                                const uint32_t w = __float_as_uint(sv) + odd;
                                if (i < cols_left) {
                                    usum += w;
                                    if (lane_valid) cb[off[i & 3] + i * g.n2] = (int8_t)w;
                                }
                            }
                            counted += cols_left;
                        }
                        if (pr.y_debug) {
                            float* yt = pr.y_debug + t * (int64_t)g.K + k0;
#pragma unroll
                            for (int i = 0; i < 16; ++i)
                                if (lane_valid && i < cols_left) yt[i * g.n2] = __uint_as_float(yv[j][i]);
                        }
                    }
                }
            }
            // sum of (stored code - the caller's bias) over this lane's elements, in wrap-around arithmetic; the CTA's sum
            // is collected in red_sum[par] and leaves after the next token's barrier (or the one behind the loop)
            int local_sum = lane_valid ? (int)(usum - (uint32_t)counted * (0x4B400000u + (uint32_t)pr.code_bias)) : 0;
            local_sum = __reduce_add_sync(0xFFFFFFFFu, local_sum);
            if (lane == 0 && local_sum != 0 && !failed) atomicAdd(&red_sum[par], local_sum);
            if (e == 0 && !failed && rank == 0) {
                pr.scales[t] = scale;
                if (pr.zp) pr.zp[t] = shift_i;
            }
        }
        // the last token's code sum
        if (!alu_barrier_or(failed || *abort_flag != 0) && e == 0 && ntok > 0)
            put_qsum(tok0 + (int64_t)(ntok - 1) * p.clusters_per_problem, (ntok - 1) & 1);
    }
    tc_fence_before();
    __syncthreads();
    if (D > 1) {
        // nobody leaves while a neighbour may still store into its shared memory or arrive on its barriers
        cluster_arrive_release();
        cluster_wait_acquire();
    }
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, (uint32_t)g.tmem_cols);
    }
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
bool okt_accepts_x(const void* x, int64_t ldx) {
    return (reinterpret_cast<uintptr_t>(x) & 15) == 0 && ldx % 8 == 0 && encode_tiled_fn() != nullptr;
}

int launch_okt(const OktGeom& g, const void* x, int64_t M, int64_t ldx, int bits, int asym, int n_problems,
               const OktProblem* problems, const OktLowrank* lowrank, uint32_t* status, cudaStream_t stream) {
    if (M == 0 || n_problems == 0) return BWLA_OK;
    if (n_problems > kOktMaxProblems || M >= ((int64_t)1 << 31)) return BWLA_ERR_INVALID_ARG;
    const int sms = sm_count();
    if (sms <= 0) return BWLA_ERR_CUDA;
    OktKernelParams p{};
    p.g = g; p.M = M; p.bits = bits; p.asym = asym; p.n_problems = n_problems; p.status = status;
    const int D = g.dt_count * g.cs_count;
    size_t smem = (size_t)g.smem_bytes;
    int lr_total = 0;
    // Many tokens: T = V x of all problems goes first, as a launch of its own on the tensor cores.  Every kernel of the
    // chain waits for its predecessor before it ends, so the contraction still finds T complete.
    bool lr_done[kOktMaxProblems] = {};
    if (lowrank) {
        OktLowrank batch[kOktMaxProblems];
        int nb = 0;
        for (int i = 0; i < n_problems; ++i)
            if (lowrank[i].V && lowrank[i].r > 0 && lowrank[i].Thl && lowrank_umma_supports(M, g.K, lowrank[i].r) &&
                (reinterpret_cast<uintptr_t>(lowrank[i].V) & 15) == 0 &&
                (lowrank[i].lr_part || lowrank_umma_part_bytes(M, g.K, lowrank[i].r) == 0)) {
                batch[nb++] = lowrank[i];
                lr_done[i] = true;
            }
        if (nb > 0) {
            int st = launch_lowrank_umma(x, M, g.K, ldx, nb, batch, status, stream);
            if (st != BWLA_OK) return st;
        }
    }
    for (int i = 0; i < n_problems; ++i) {
        p.prob[i] = problems[i];
        p.lr_begin[i] = lr_total;
        if (lowrank && !lr_done[i] && lowrank[i].V && lowrank[i].r > 0 && lowrank[i].Thl) {
            PrologueParams& lp = p.lr[i];
            lp.x = (const __nv_bfloat16*)x; lp.M = M; lp.K = g.K; lp.ldx = ldx;
            lp.V = (const __nv_bfloat16*)lowrank[i].V; lp.r = lowrank[i].r; lp.Thl = (__nv_bfloat16*)lowrank[i].Thl;
            lp.lr_cols = lowrank_cols(lowrank[i].r);
            size_t lr_smem = 0;
            const int blocks = plan_lowrank(lp, lowrank[i].lr_part, lowrank[i].lr_count, kOktMaxSmem, &lr_smem);
            if (lp.lr_wide == 3) {
                // Many tokens: the wide tiles (64 columns x 16 tokens per block, 64 accumulators per lane) need more
                // registers than a block of this kernel has; they go first, as a launch of their own.  Every kernel of the
                // chain waits for its predecessor before it ends, so the contraction still finds T complete.
                int st = launch_prologue(x, M, g.K, ldx, nullptr, 0, nullptr, 0, bits, nullptr, 0, nullptr, nullptr, lowrank[i].V,
                                         lowrank[i].r, lowrank[i].Thl, lowrank[i].lr_part,
                                         lowrank[i].lr_count ? lowrank[i].lr_count - kLrCounterWord : nullptr, stream);
                if (st != BWLA_OK) return st;
                lp = PrologueParams{};
            } else {
                lr_total += blocks;
                smem = std::max(smem, lr_smem);
            }
        }
    }
    for (int i = n_problems; i <= kOktMaxProblems; ++i) p.lr_begin[i] = lr_total;
    // One cluster per token while every cluster finds an SM of its own; beyond that the clusters stay and take tokens
    // in turn (the T = V x blocks then go first in block order, or they would only start when the rotation is over).
    const int64_t room = std::max<int64_t>(1, (int64_t)sms / ((int64_t)n_problems * D));
    p.clusters_per_problem = (int)std::min<int64_t>(M, room);
    p.rot_ctas = n_problems * p.clusters_per_problem * D;
    const bool stay = p.clusters_per_problem < M;
    p.rot_first = (stay && lr_total > 0) ? (lr_total + D - 1) / D * D : 0;
    int grid = p.rot_first ? p.rot_first + p.rot_ctas : p.rot_ctas + lr_total;
    grid = (grid + D - 1) / D * D;

    CUtensorMap xm;
    {
        // x as [M][n1][n2]: one box is one K-atom of one token's X, rows beyond n1 and columns beyond n2 read as zero
        const uint64_t dims[3] = {(uint64_t)g.n2, (uint64_t)g.n1, (uint64_t)M};
        const uint64_t strides[2] = {(uint64_t)g.n2 * 2, (uint64_t)ldx * 2};
        const uint32_t box[3] = {(uint32_t)(g.atom2 >> 1), (uint32_t)g.n1p, 1};
        const CUtensorMapSwizzle sw = g.atom2 == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                    : g.atom2 == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
        int st = make_map(&xm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, x, dims, strides, box, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
        if (st != BWLA_OK) return st;
    }

    static thread_local int configured_device = -1;
    int dev = 0;
    BWLA_CUDA_TRY(cudaGetDevice(&dev));
    if (configured_device != dev) {
        BWLA_CUDA_TRY(cudaFuncSetAttribute(okt_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kOktMaxSmem));
        configured_device = dev;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(kOktThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attrs[2];
    attrs[0].id = cudaLaunchAttributeClusterDimension;
    attrs[0].val.clusterDim.x = (unsigned)D; attrs[0].val.clusterDim.y = 1; attrs[0].val.clusterDim.z = 1;
    attrs[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attrs[1].val.programmaticStreamSerializationAllowed = launch_overlap_allowed();
    cfg.attrs = attrs;
    cfg.numAttrs = 2;
    ProfScope prof(kProfRotateQuant, stream);
    cudaError_t e = cudaLaunchKernelEx(&cfg, okt_umma_kernel, xm, p);
    if (e != cudaSuccess) { cudaGetLastError(); return cuda_fail(e); }
    return after_launch();
}

}  // namespace bwla
