// The binary-weight contraction for many tokens: the arithmetic of gemm_umma.cu (sign words expanded into tensor memory
// as the A operand of tcgen05.mma kind::i8, low-rank term as kind::f16 MMAs, fused epilogue) in CTAs that stay on their
// SM and take tiles of 128 output rows x 128 tokens in turn.
//
// One CTA per tile pays its set-up (barriers, tensor memory, the first loads from HBM) and its epilogue (read-back,
// scaling, 32 KB of output) with the tensor core idle: at 128 tokens that was more than the tile's K loop.  Here the
// producers, the expanders and the MMA issuer run on into the next tile while four epilogue warps finish the last one:
//   warp 0        packed sign words by TMA (a unit of 1024 weights x 128 rows per stage), all tiles back to back
//   warp 1        per tile: the tokens' scales / code sums / zero points into shared memory, the codes k-block by k-block
//                 by TMA, then the three bf16 terms of T
//   warp 2        MMA issue: the tile's K loop into the int32 accumulator, then the low-rank MMAs, one commit per tile
//   warps 4..7    epilogue: stage the tile's rows of U, read the accumulators back, scale, write bf16 through shared
//                 memory with 128-bit stores; the accumulator is handed back as soon as it has been read
//   warps 8..23   expansion of sign bits into the tensor-memory operand ring (as in gemm_umma.cu), tile boundaries unseen
// Every wait is bounded (umma_wait.cuh).
#include <cuda_bf16.h>

#include <algorithm>

#include "bwla_common.cuh"
#include "umma_ptx.cuh"
#include "umma_wait.cuh"
#include "tensor_map.cuh"

namespace bwla {

using namespace ptx;

namespace persist {
constexpr int kRows = 128;                // output rows per tile
constexpr int kTok = 128;                 // tokens per tile
constexpr int kUnitK = 1024;              // weights per row in one sign-word stage
constexpr int kBlockK = 128;              // K per code stage and per operand stage
constexpr int WS = 2, BS = 5, AS = 4, EW = 4;
static_assert(AS % EW == 0, "an operand stage must keep one owner among the expander parts");
constexpr int kEpiFirst = 128, kExpFirst = 256;
constexpr int kThreads = kExpFirst + 128 * EW;       // 768
constexpr int w_bytes = kRows * 128, b_bytes = kTok * 128;
constexpr int u_off = WS * w_bytes + BS * b_bytes;
constexpr int t_off = u_off + kRows * 128;
constexpr int o_off = t_off + 3 * b_bytes;           // finished outputs [token][row] bf16
constexpr int bars_off = o_off + kTok * kRows * 2;
constexpr int n_bars = 2 * WS + 2 * BS + 2 * AS + 12;
constexpr int misc_off = bars_off + n_bars * 8;
constexpr int tok_off = misc_off + 16;               // [2][scales, code sums, zero points][kTok]
constexpr int used = tok_off + 2 * 12 * kTok;
constexpr int total = used + 1024;
// tensor memory: two int32 accumulators (tiles alternate, so the MMAs of a tile never wait for the epilogue of the one
// before), one fp32 low-rank accumulator (written at the very end of a tile's MMAs, long after the previous epilogue has
// read it), then the operand ring
constexpr int D_COL = 0, LR_COL = 2 * kTok, A_COL = 3 * kTok, TMEM_COLS = 512;
static_assert(A_COL + 32 * AS <= TMEM_COLS, "tensor memory");
static_assert(total <= 232448, "shared memory");
}  // namespace persist

struct PersistParams {
    int M, N, K;
    int row_tiles, tok_tiles;
    int r;
    const float* scales; const int32_t* qsum; const int32_t* zp;
    const float* alpha; const float* mu; const int32_t* rowsum;
    const __nv_bfloat16* U;
    __nv_bfloat16* out; int64_t ldo;
    int32_t* acc_debug;
    uint32_t* status;
};

__global__ void __launch_bounds__(persist::kThreads, 1)
umma_w1a_persistent_kernel(const __grid_constant__ CUtensorMap w_map, const __grid_constant__ CUtensorMap b_map,
                           const __grid_constant__ CUtensorMap t_map, PersistParams p) {
    using namespace persist;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* wbuf = smem;
    uint8_t* bbuf = smem + WS * w_bytes;
    uint8_t* ubuf = smem + u_off;
    uint8_t* tbuf = smem + t_off;
    __nv_bfloat16* otile = reinterpret_cast<__nv_bfloat16*>(smem + o_off);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + bars_off);
    uint64_t* w_full = bars;                 // [WS]
    uint64_t* w_empty = w_full + WS;
    uint64_t* b_full = w_empty + WS;         // [BS]
    uint64_t* b_empty = b_full + BS;
    uint64_t* a_full = b_empty + BS;         // [AS]
    uint64_t* a_empty = a_full + AS;
    uint64_t* d_full = a_empty + AS;         // the tile's MMAs (low-rank ones included) have completed
    uint64_t* acc_free = d_full + 1;         // the epilogue has read the tile's accumulators
    uint64_t* u_full = acc_free + 1;         // the tile's rows of U are staged
    uint64_t* u_empty = u_full + 1;          // the low-rank MMAs have read them
    uint64_t* t_full = u_empty + 1;
    uint64_t* t_empty = t_full + 1;
    uint64_t* tok_full = t_empty + 1;        // [2] per-token scales ... staged (by tile parity)
    uint64_t* epi_done = tok_full + 2;       // [2] the epilogue is through with them
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + misc_off);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + misc_off + 4);
    auto tok_scale = [&](int buf) { return reinterpret_cast<float*>(smem + tok_off + buf * 12 * kTok); };
    auto tok_qsum = [&](int buf) { return reinterpret_cast<int32_t*>(smem + tok_off + buf * 12 * kTok + 4 * kTok); };
    auto tok_zp = [&](int buf) { return reinterpret_cast<int32_t*>(smem + tok_off + buf * 12 * kTok + 8 * kTok); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tiles = p.row_tiles * p.tok_tiles;
    const int my_tiles = (int)blockIdx.x < tiles ? (tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
    const int units = (p.K + kUnitK - 1) / kUnitK;
    const int kblocks = p.K / kBlockK;
    const bool lowrank = p.r > 0;
    // tile i of this CTA: row tiles fastest, so that the CTAs working at the same time share a token tile's codes in the L2
    auto tile_n0 = [&](int i) { return (((int)blockIdx.x + i * (int)gridDim.x) % p.row_tiles) * kRows; };
    auto tile_t0 = [&](int i) { return (((int)blockIdx.x + i * (int)gridDim.x) / p.row_tiles) * kTok; };

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int i = 0; i < WS; ++i) { mbar_init(&w_full[i], 1); mbar_init(&w_empty[i], 4 * EW); }
        for (int i = 0; i < BS; ++i) { mbar_init(&b_full[i], 1); mbar_init(&b_empty[i], 1); }
        for (int i = 0; i < AS; ++i) { mbar_init(&a_full[i], 4); mbar_init(&a_empty[i], 1); }
        mbar_init(d_full, 1); mbar_init(acc_free, 4);
        mbar_init(u_full, 4); mbar_init(u_empty, 1);
        mbar_init(t_full, 1); mbar_init(t_empty, 1);
        for (int i = 0; i < 2; ++i) { mbar_init(&tok_full[i], 1); mbar_init(&epi_done[i], 4); }
        fence_barrier_init();
        fence_proxy_async();
    }
    if (warp == 2) {
        tmem_alloc(tmem_slot, TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    griddep_launch_dependents();

    if (warp == 0) {
        // ---------------- packed sign words (independent of the preceding kernel) ----------------
        if (elect_one()) {
            tma_prefetch_desc(&w_map);
            const uint64_t stream_once = l2_policy_evict_first();
            int ws = 0; uint32_t wph = 0;
            for (int i = 0; i < my_tiles && !*abort_flag; ++i) {
                const int n0 = tile_n0(i);
                for (int u = 0; u < units && !*abort_flag; ++u) {
                    if (!mbar_test_wait(&w_empty[ws], wph ^ 1)) {
                        griddep_wait();
                        if (!wait_or_abort(&w_empty[ws], wph ^ 1, abort_flag)) { give_up(p.status, abort_flag, 0x110); break; }
                    }
                    mbar_expect_tx(&w_full[ws], w_bytes);
                    tma_load_2d_hint(wbuf + ws * w_bytes, &w_map, u * (kUnitK / 32), n0, &w_full[ws], stream_once);
                    if (++ws == WS) { ws = 0; wph ^= 1; }
                }
            }
            if (*abort_flag) for (int i = 0; i < 500; ++i) __nanosleep(100);
        }
    } else if (warp == 1) {
        // ---------------- per-token scalars, codes and T ----------------
        griddep_wait();
        if (lane == 0) {
            tma_prefetch_desc(&b_map);
            if (lowrank) tma_prefetch_desc(&t_map);
            if (p.status && *reinterpret_cast<volatile uint32_t*>(p.status) != 0) *abort_flag = 1;   // the call already failed
        }
        __syncwarp();
        int bs = 0; uint32_t bph = 0;
        bool ok = true;
        for (int i = 0; i < my_tiles && ok && !*abort_flag; ++i) {
            const int t0 = tile_t0(i), buf = i & 1;
            if (i >= 2 && !warp_wait(&epi_done[buf], (uint32_t)(((i >> 1) - 1) & 1), abort_flag)) { give_up(p.status, abort_flag, 0x120); ok = false; break; }
            for (int j = lane; j < kTok; j += 32) {
                const int t = t0 + j;
                tok_scale(buf)[j] = t < p.M ? p.scales[t] : 0.f;
                int32_t qs = 0;
                if (t < p.M) {
                    const int4* parts = reinterpret_cast<const int4*>(p.qsum + (size_t)t * kQsumParts);
                    const int4 a = parts[0], b = parts[1];
                    qs = a.x + a.y + a.z + a.w + b.x + b.y + b.z + b.w;
                }
                tok_qsum(buf)[j] = qs;
                tok_zp(buf)[j] = (p.zp && t < p.M) ? p.zp[t] : 0;
            }
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(&tok_full[buf]);
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!wait_or_abort(&b_empty[bs], bph ^ 1, abort_flag)) { give_up(p.status, abort_flag, 0x121); ok = false; break; }
                    mbar_expect_tx(&b_full[bs], b_bytes);
                    tma_load_2d(bbuf + bs * b_bytes, &b_map, kb * kBlockK, t0, &b_full[bs]);
                    if (++bs == BS) { bs = 0; bph ^= 1; }
                }
                // T is first needed when the K loop is over; the previous tile's low-rank MMAs have long read theirs
                if (ok && lowrank) {
                    if (i >= 1 && !wait_or_abort(t_empty, (uint32_t)((i - 1) & 1), abort_flag)) { give_up(p.status, abort_flag, 0x122); ok = false; }
                    if (ok) {
                        mbar_expect_tx(t_full, 3 * b_bytes);
                        for (int h = 0; h < 3; ++h) tma_load_3d(tbuf + h * b_bytes, &t_map, 0, t0, h, t_full);
                    }
                }
            }
            ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
        }
        if (lane == 0 && *abort_flag) for (int i = 0; i < 500; ++i) __nanosleep(100);
    } else if (warp == 2) {
        // ---------------- MMA issue ----------------
        if (elect_one()) {
            const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTok >> 3) << 17) | ((128u >> 4) << 24);
            const uint32_t idesc_lr = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTok >> 3) << 17) | ((128u >> 4) << 24);
            const uint32_t a_base = tmem_base + A_COL;
            const uint64_t desc_hi = smem_desc_sw128(0u, 0u);
            const uint32_t b_lo0 = (smem_u32(bbuf) & 0x3FFFFu) >> 4;
            int as = 0; uint32_t aph = 0;
            int bs = 0; uint32_t bph = 0;
            bool ok = true;
            griddep_wait();                           // everything this thread waits for follows the preceding kernel
            for (int i = 0; i < my_tiles && ok; ++i) {
                // accumulator i & 1 was last used by tile i - 2, whose epilogue this thread has seen finish at the end of tile
                // i - 1 (below)
                tc_fence_after();
                const uint32_t d_addr = tmem_base + D_COL + (uint32_t)(i & 1) * kTok;
                uint32_t acc = 0;
                for (int kb = 0; kb < kblocks && ok; ++kb) {
                    if (!wait_or_abort(&b_full[bs], bph, abort_flag)) { give_up(p.status, abort_flag, 0x131); ok = false; break; }
                    if (!wait_or_abort(&a_full[as], aph, abort_flag)) { give_up(p.status, abort_flag, 0x132); ok = false; break; }
                    tc_fence_after();
                    const uint64_t desc = desc_hi | (uint64_t)(b_lo0 + (uint32_t)bs * (b_bytes >> 4));
                    const uint32_t a_addr = a_base + 32 * as;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        mma_i8_ts(d_addr, a_addr + 8 * j, desc + 2 * j, idesc, acc);
                        acc = 1u;
                    }
                    tc_commit(&a_empty[as]);
                    tc_commit(&b_empty[bs]);
                    if (++as == AS) { as = 0; aph ^= 1u; }
                    if (++bs == BS) { bs = 0; bph ^= 1u; }
                }
                // The epilogue of the tile before has had this tile's whole K loop to read its accumulators; it is waited for
                // here, before this tile's MMAs are committed, so that completions of acc_free are seen strictly in order
                // (a parity wait only tells the current phase from the one before it).  It frees the low-rank accumulator
                // for this tile and the int32 accumulator for the next.
                if (ok && i >= 1 && !wait_or_abort(acc_free, (uint32_t)((i - 1) & 1), abort_flag)) { give_up(p.status, abort_flag, 0x130); ok = false; }
                if (ok && lowrank) {
                    if (!wait_or_abort(u_full, (uint32_t)(i & 1), abort_flag)) { give_up(p.status, abort_flag, 0x133); ok = false; }
                    if (ok && !wait_or_abort(t_full, (uint32_t)(i & 1), abort_flag)) { give_up(p.status, abort_flag, 0x134); ok = false; }
                    if (ok) {
                        tc_fence_after();
                        const uint32_t u_addr = smem_u32(ubuf);
#pragma unroll
                        for (int h = 0; h < 3; ++h) {
                            const uint32_t t_addr = smem_u32(tbuf + h * b_bytes);
#pragma unroll
                            for (int j = 0; j < 4; ++j)
                                mma_f16_ss(tmem_base + LR_COL, smem_desc_sw128(u_addr, 32 * j), smem_desc_sw128(t_addr, 32 * j),
                                           idesc_lr, (h | j) ? 1u : 0u);
                        }
                        tc_commit(u_empty);
                        tc_commit(t_empty);
                    }
                }
                tc_commit(d_full);
            }
        }
    } else if (warp >= 4 && warp < 8) {
        // ---------------- epilogue ----------------
        const int q = warp & 3;
        const int e = threadIdx.x - kEpiFirst;        // 0..127: output row of the tile
        const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
        bool ok = true;
        for (int i = 0; i < my_tiles; ++i) {
            const int n0 = tile_n0(i), t0 = tile_t0(i), buf = i & 1;
            const int n = n0 + e;
            const bool valid_row = n < p.N;
            const float alpha_n = valid_row ? __ldg(p.alpha + n) : 0.f;
            const float mu_n = (p.mu && valid_row) ? __ldg(p.mu + n) : 0.f;
            const int32_t rs_n = (p.zp && valid_row) ? __ldg(p.rowsum + n) : 0;
            if (lowrank) {
                // this tile's rows of U: 128 rows x 8 chunks of 16 bytes, 128B-swizzled K-major, zero beyond N and r
                if (ok && i >= 1 && !warp_wait(u_empty, (uint32_t)((i - 1) & 1), abort_flag)) { give_up(p.status, abort_flag, 0x140); ok = false; }
                if (ok) {
                    const bool vec = (p.r % 8 == 0) && ((reinterpret_cast<uintptr_t>(p.U) & 15) == 0);
#pragma unroll
                    for (int it = 0; it < 8; ++it) {
                        const int idx = it * 128 + e;
                        const int ur = idx >> 3, ch = idx & 7;
                        uint4 v = make_uint4(0u, 0u, 0u, 0u);
                        const int un = n0 + ur;
                        if (un < p.N && ch * 8 < p.r) {
                            const __nv_bfloat16* src = p.U + (int64_t)un * p.r + ch * 8;
                            if (vec) {
                                v = __ldg(reinterpret_cast<const uint4*>(src));
                            } else {
                                uint32_t w[4] = {0u, 0u, 0u, 0u};
                                for (int c = 0; c < 8 && ch * 8 + c < p.r; ++c)
                                    w[c >> 1] |= (uint32_t)__bfloat16_as_ushort(src[c]) << (16 * (c & 1));
                                v = make_uint4(w[0], w[1], w[2], w[3]);
                            }
                        }
                        *reinterpret_cast<uint4*>(ubuf + ur * 128 + ((ch ^ (ur & 7)) << 4)) = v;
                    }
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(u_full);
                }
            }
            if (i == 0) griddep_wait();                       // nothing is stored before the preceding kernel has completed
            if (ok && !warp_wait(&tok_full[buf], (uint32_t)((i >> 1) & 1), abort_flag)) { give_up(p.status, abort_flag, 0x141); ok = false; }
            if (ok && !warp_wait(d_full, (uint32_t)(i & 1), abort_flag)) { give_up(p.status, abort_flag, 0x142); ok = false; }
            if (ok) {
                tc_fence_after();
                const float* sc_s = tok_scale(buf);
                const int32_t* qs_s = tok_qsum(buf);
                const int32_t* zp_s = tok_zp(buf);
#pragma unroll 1
                for (int c = 0; c < kTok / 16; ++c) {
                    uint32_t v[16], l[16];
                    tmem_ld_32x16(tmem_base + lane_addr + D_COL + (uint32_t)(i & 1) * kTok + 16 * c, v);
                    if (lowrank) tmem_ld_32x16(tmem_base + lane_addr + LR_COL + 16 * c, l);
                    tc_wait_ld();
                    if (c == kTok / 16 - 1) {
                        // both accumulators are in registers: the next tile's MMAs may start
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(acc_free);
                    }
                    if (t0 + 16 * c >= p.M) continue;            // warp-uniform; nothing of this chunk is stored
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const float sc = sc_s[16 * c + j];
                        const int32_t qs = qs_s[16 * c + j], zp = zp_s[16 * c + j];
                        const int32_t acc = -((int32_t)v[j] >> 6) - qs - zp * rs_n;
                        if (p.acc_debug && valid_row && t0 + 16 * c + j < p.M) p.acc_debug[(int64_t)(t0 + 16 * c + j) * p.N + n] = acc;
                        const float lr = lowrank ? __uint_as_float(l[j]) : 0.f;
                        const float y = fmaf(__fmul_rn(mu_n, sc), (float)(qs - p.K * zp), __fmul_rn(__fmul_rn(alpha_n, sc), (float)acc) + lr);
                        otile[(16 * c + j) * kRows + e] = __float2bfloat16_rn(y);
                    }
                }
            } else if (!*abort_flag) {
                *abort_flag = 1;
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");       // the output tile is complete (all epilogue warps, always)
            if (ok && p.out) {
                // 16 threads move one token's 128 outputs (256 bytes) with 128-bit stores
                const bool vec = ((reinterpret_cast<uintptr_t>(p.out) & 15) == 0) && (p.ldo % 8 == 0) && (n0 + kRows <= p.N);
                for (int tt = e >> 4; tt < kTok && t0 + tt < p.M; tt += 8) {
                    const int c8 = (e & 15) * 8;
                    __nv_bfloat16* dst = p.out + (int64_t)(t0 + tt) * p.ldo + n0 + c8;
                    const uint4 val = *reinterpret_cast<const uint4*>(otile + tt * kRows + c8);
                    if (vec) {
                        *reinterpret_cast<uint4*>(dst) = val;
                    } else {
                        const __nv_bfloat16* sv = reinterpret_cast<const __nv_bfloat16*>(&val);
                        for (int j = 0; j < 8; ++j)
                            if (n0 + c8 + j < p.N) dst[j] = sv[j];
                    }
                }
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");       // the tile buffer may be written again
            if (lane == 0) mbar_arrive(&epi_done[buf]);
        }
    } else if (warp >= 8) {
        // ---------------- expansion of sign bits into the operand ring (tile boundaries do not matter here) ----------------
        const int q = warp & 3;
        const int part = (warp - 8) >> 2;             // which of the EW warps of the lane quarter
        const int row = q * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
        int ws = 0; uint32_t wph = 0;
        int kb_base = 0;                              // k-blocks of this CTA before the current unit: block g lives in stage g % AS
        bool ok = true;
        for (int i = 0; i < my_tiles && ok; ++i) {
            for (int u = 0; u < units && ok; ++u) {
                if (!warp_wait(&w_full[ws], wph, abort_flag)) { give_up(p.status, abort_flag, 0x150); ok = false; break; }
                const uint8_t* wrow = wbuf + ws * w_bytes + row * 128;
                const int ns = min(kUnitK / kBlockK, (p.K - u * kUnitK) / kBlockK);
                // Block g of this CTA (a running count over its tiles) belongs to part g % EW and to stage g % AS.  AS is a
                // multiple of EW, so a stage always has the same owner and the owner is never more than one phase ahead of
                // the stage's consumer: a parity wait cannot tell a phase from the one two before it.  (The last unit of a
                // row may hold fewer than eight blocks, which is why neither follows from the position inside the unit.)
#pragma unroll 1
                for (int s = (part + EW - kb_base % EW) % EW; s < ns && ok; s += EW) {
                    const uint4 w4 = *reinterpret_cast<const uint4*>(wrow + ((s ^ (row & 7)) << 4));
                    uint32_t v[32];
                    const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
                    for (int c = 0; c < 4; ++c)
#pragma unroll
                        for (int j = 0; j < 8; ++j) v[8 * c + j] = (w[c] << (7 - j)) & 0x80808080u;
                    const int as = (kb_base + s) % AS;
                    const uint32_t aph = (uint32_t)(((kb_base + s) / AS) & 1);
                    if (!__all_sync(0xFFFFFFFFu, mbar_test_wait(&a_empty[as], aph ^ 1u))) {
                        griddep_wait();
                        if (!warp_wait(&a_empty[as], aph ^ 1u, abort_flag)) { give_up(p.status, abort_flag, 0x151); ok = false; }
                    }
                    if (ok) {
                        tc_fence_after();
                        tmem_st_32x32(tmem_base + lane_addr + A_COL + 32 * as, v);
                        tc_wait_st();
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&a_full[as]);
                    }
                }
                // the stage is released only after every word of it that this warp needs has gone through the expansion
                __syncwarp();
                if (lane == 0) mbar_arrive(&w_empty[ws]);
                if (++ws == WS) { ws = 0; wph ^= 1u; }
                kb_base += ns;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 2) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

bool umma_persistent_supports(int64_t M, int64_t K, int64_t N, int r) {
    // every k-block of a tile must exist in full (a whole number of 128-weight blocks), and the tile loop pays off with
    // more tiles than SMs
    return M > 64 && K % 128 == 0 && r <= kLowrankPad && N > 0;
}

int launch_gemm_umma_persistent(const GemmArgs& a, const int8_t* codes_interleaved, cudaStream_t stream) {
    using namespace persist;
    const int M = (int)a.M, N = (int)a.N, K = (int)a.K;
    const int sms = sm_count();
    if (sms <= 0) return BWLA_ERR_CUDA;
    CUtensorMap wm, bm, tm;
    {
        const uint64_t dims[2] = {(uint64_t)K / 32, (uint64_t)N};
        const uint64_t strides[1] = {(uint64_t)K / 8};
        const uint32_t box[2] = {32, kRows};
        int st = make_map(&wm, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, a.packed, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
        if (st != BWLA_OK) return st;
    }
    {
        const uint64_t dims[2] = {(uint64_t)K, (uint64_t)M};
        const uint64_t strides[1] = {(uint64_t)K};
        const uint32_t box[2] = {kBlockK, kTok};
        int st = make_map(&bm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, codes_interleaved, dims, strides, box,
                          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
        if (st != BWLA_OK) return st;
    }
    if (a.r > 0) {
        const uint64_t dims[3] = {(uint64_t)kLowrankPad, (uint64_t)M, 3};
        const uint64_t strides[2] = {(uint64_t)kLowrankPad * 2, (uint64_t)M * kLowrankPad * 2};
        const uint32_t box[3] = {(uint32_t)kLowrankPad, kTok, 1};
        int st = make_map(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, a.Thl, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
        if (st != BWLA_OK) return st;
    } else {
        tm = bm;   // never dereferenced
    }
    PersistParams p{};
    p.M = M; p.N = N; p.K = K; p.row_tiles = (N + kRows - 1) / kRows; p.tok_tiles = (M + kTok - 1) / kTok; p.r = a.r;
    p.scales = a.scales; p.qsum = a.qsum; p.zp = a.zp; p.alpha = a.alpha; p.mu = a.mu; p.rowsum = a.rowsum;
    p.U = (const __nv_bfloat16*)a.U; p.out = (__nv_bfloat16*)a.out; p.ldo = a.ldo; p.acc_debug = a.acc_debug; p.status = a.status;
    const int tiles = p.row_tiles * p.tok_tiles;

    static thread_local int configured = -1;
    int dev = 0;
    BWLA_CUDA_TRY(cudaGetDevice(&dev));
    if (configured != dev) {
        BWLA_CUDA_TRY(cudaFuncSetAttribute(umma_w1a_persistent_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, total));
        configured = dev;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)std::min(tiles, sms), 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = total;
    cfg.stream = stream;
    cudaLaunchAttribute attrs[1];
    attrs[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attrs[0].val.programmaticStreamSerializationAllowed = launch_overlap_allowed();
    cfg.attrs = attrs;
    cfg.numAttrs = 1;
    ProfScope prof(kProfContraction, stream);
    cudaError_t e = cudaLaunchKernelEx(&cfg, umma_w1a_persistent_kernel, wm, bm, tm, p);
    if (e != cudaSuccess) { cudaGetLastError(); return cuda_fail(e); }
    return after_launch();
}

}  // namespace bwla
