// Binary-weight contraction on tcgen05 tensor cores with the whole epilogue fused in.
//
//   D[n][t]  = sum_k byte(n,k) * q[t][k],  byte(n,k) = -128 if the sign bit of weight (n,k) is set, else 0
//   acc[t][n] = sum_k sign(n,k) * q[t][k] = -D/64 - sum_k q[t][k]            (sign = 2*bit - 1, exact in int32)
//   D2[n][t] = sum_j U[n][j] * T[t][j]                                        (PSP low-rank term, Sec. 3.2)
//   out[t][n] = bf16(alpha[n] * s_t * acc + D2 [+ mu[n] * s_t * sum_k q[t][k]])   (Eq. 4 on the accumulator)
//
// One CTA owns 128 output rows x up to 64 tokens x a slice of K; the CTAs that share a tile and split K form a
// thread-block cluster and add their partial sums through distributed shared memory, so nothing but the bf16
// result is written to global memory.  Inside a CTA:
//   * warp 0 streams packed sign words by TMA (128 rows x 128 bytes = 1024 weights per row, 128B-swizzled); these
//     loads do not depend on the activations and start before the preceding kernel of the stream has finished
//     (programmatic dependent launch);
//   * warp 1 waits for the preceding kernel, then streams the three bf16 terms of T and the activation codes
//     (tokens x 128 bytes per k-block, the canonical K-major 128B-swizzled UMMA layout);
//   * warps 6.. (EW = 2 or 4 per tensor-memory lane quarter, thread = output row, the warps of a quarter taking
//     k-blocks in turn) stage the U tile in shared memory, then turn each 32-bit sign word into eight registers
//     of four int8 with one shift and one mask per register ((w << (7-j)) & 0x80808080) and write them with
//     tcgen05.st into tensor memory, where they are the A operand: expanded weights never touch shared memory.
//   * NISS threads (one each in warps 2..5) issue tcgen05.mma.kind::i8 (M = 128, N = tokens, K = 32; A from tensor
//     memory, B from shared memory), taking k-blocks round-robin, each into an int32 accumulator of its own in
//     tensor memory: with few tokens an MMA is short and the issue latency of one thread would be the bottleneck.
//     The first of them also issues the kind::f16 MMAs of the low-rank term (A = U tile, B = T as three bf16
//     terms, fp32 accumulator in tensor memory);
//   * the same warps read the accumulators back (tcgen05.ld), reduce across the cluster when K is split, apply the
//     scales, transpose through shared memory and store bf16 with 128-bit stores.
// Few tokens make the K loop a chain of latencies rather than of throughput; the launch then takes either two CTAs per SM
// (8 expander warps and 256 tensor-memory columns each) or, when a K split puts the whole grid on the SMs at once, one
// CTA per SM with 16 expander warps and all 512 columns (a twice as deep operand ring).
// The shift-and-mask expansion meets the weights of a 32-group in the order k = j + 8*i (register j, byte i), so the
// codes are stored in that interleaved order by the quantiser.
//
// Every wait is bounded: on give-up the CTA records where in the workspace status words, stops issuing work, lets
// in-flight copies land, still takes part in the cluster barriers, frees its tensor memory and returns.
#include <cuda_bf16.h>

#include <algorithm>

#include "bwla_common.cuh"
#include "umma_ptx.cuh"
#include "umma_wait.cuh"
#include "tensor_map.cuh"

namespace bwla {

using namespace ptx;

constexpr int kRowsPerCta = 128;
constexpr int kUnitK = 1024;             // weights per row in one packed-word stage (128 bytes)
constexpr int kBlockK = 128;             // K per code sub-block / per tensor-memory A stage
constexpr int kFirstExpander = 192;      // warps 0, 1: TMA; warps 2..5: MMA issue; warps 6..: expand + epilogue
struct UmmaParams {
    int M, N, K;
    int total_units, splits;
    int r;                       // low-rank width, 0..kLowrankPad
    const float* scales;         // [M]
    const int32_t* qsum;         // [M][kQsumParts] partial sums
    const float* alpha;          // [N]
    const float* mu;             // [N] or NULL
    const int32_t* zp;           // [M] zero points of asymmetric codes, or NULL
    const int32_t* rowsum;       // [N] sum_k sign(n,k); read only when zp is given
    const __nv_bfloat16* U;      // [N][r] or NULL
    __nv_bfloat16* out;          // [M][ldo] or NULL
    int64_t ldo;
    int32_t* acc_debug;          // [M][N] or NULL
    int dep_mode;                // kDepChain / kDepHead / kDepSibling (bwla_common.cuh)
    uint32_t* status;
};

// Shared-memory and tensor-memory budget of one CTA.
//   weights: WS stages of 128 rows x 128 bytes (one K-unit of 1024 weights per row);
//   codes:   BS stages of 16 KB = SUBS k-blocks of (N_TOK rows x 128 bytes), so that small token tiles still move
//            16 KB per barrier round trip;
//   U tile:  128 rows x 64 bf16 (128 bytes), zero padded beyond r;  T tiles: 3 x (N_TOK rows x 64 bf16);
//   tensor memory: NISS int32 accumulators of N_TOK columns, the fp32 low-rank accumulator (N_TOK columns), then AS
//   stages of 32 columns (one k-block of expanded weights each).
// The cluster reduction buffers (int32 and fp32, N_TOK x 128 each) and the bf16 output tile reuse the stage memory
// once the K loop is over.
template <int N_TOK, int WS, int BS, int TMEM_COLS, int NISS, int EW>
struct UmmaCfg {
    static constexpr int kExpanders = 128 * EW;                        // EW warps per tensor-memory lane quarter
    static constexpr int kThreads = kFirstExpander + kExpanders;
    static constexpr int w_bytes = kRowsPerCta * 128;
    static constexpr int sub_bytes = N_TOK * 128;
    static constexpr int SUBS = (128 / N_TOK) < 1 ? 1 : ((128 / N_TOK) > 8 ? 8 : (128 / N_TOK));
    static constexpr int b_bytes = SUBS * sub_bytes;
    static constexpr int D2_COL = NISS * N_TOK;
    static constexpr int A_COL = ((NISS + 1) * N_TOK + 31) / 32 * 32;
    static constexpr int AS = ((TMEM_COLS - A_COL) / 32) / EW * EW;   // a multiple of EW: the warps of a quarter take turns
    static constexpr int u_off = WS * w_bytes + BS * b_bytes;
    static constexpr int t_off = u_off + kRowsPerCta * 128;
    static constexpr int bars_off = t_off + 3 * sub_bytes;
    static constexpr int n_bars = 2 * WS + 2 * BS + 2 * AS + 4;
    static constexpr int misc_off = bars_off + n_bars * 8;            // tmem slot, abort flag
    static constexpr int tok_off = misc_off + 16;                      // scales[N_TOK], qsum[N_TOK], zero points[N_TOK]
    static constexpr int used = tok_off + 12 * N_TOK;
    static constexpr int total = used + 1024;                          // + slack for 1024-byte alignment
    static constexpr int red_bytes = 2 * N_TOK * kRowsPerCta * 4;
    static constexpr bool can_split = red_bytes <= u_off;
    static_assert(NISS >= 1 && NISS <= 4, "one to four issuing warps");
    static_assert(EW == 2 || EW == 4, "two or four expander warps per lane quarter");
    static_assert(AS >= 2 * EW, "tensor memory: no room for the expanded-weight ring");
    static_assert(N_TOK * kRowsPerCta * 2 <= u_off, "output tile does not fit the stage memory");
};

// One output value from its two accumulators (mu_sc is zero when the layer has no row shift).  zr = zero point of the
// token x sign sum of the row, kz = K x zero point (both zero for symmetric codes): a code stands for scale * (code -
// zero point), and the zero point's share of the sums is taken out in exact integer arithmetic.
__device__ __forceinline__ float finish_value(int32_t d, float l, float alpha_sc, float mu_sc, int32_t qs, int32_t zr, int32_t kz) {
    const int32_t acc = -(d >> 6) - qs - zr;
    return fmaf(mu_sc, (float)(qs - kz), __fmul_rn(alpha_sc, (float)acc) + l);
}

template <int N_TOK, int WS, int BS, int TMEM_COLS, int NISS, int EW>
__global__ void __launch_bounds__(kFirstExpander + 128 * EW, TMEM_COLS == 256 ? 2 : 1)
umma_w1a_kernel(const __grid_constant__ CUtensorMap w_map, const __grid_constant__ CUtensorMap b_map,
                const __grid_constant__ CUtensorMap t_map, UmmaParams p) {
    extern __shared__ uint8_t smem_raw[];
    using L = UmmaCfg<N_TOK, WS, BS, TMEM_COLS, NISS, EW>;
    constexpr int AS = L::AS;
    constexpr int SUBS = L::SUBS;
    constexpr int kExpanders = L::kExpanders;
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* wbuf = smem;
    uint8_t* bbuf = smem + WS * L::w_bytes;
    uint8_t* ubuf = smem + L::u_off;
    uint8_t* tbuf = smem + L::t_off;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::bars_off);
    uint64_t* w_full = bars;                 // [WS]
    uint64_t* w_empty = bars + WS;           // [WS]
    uint64_t* b_full = bars + 2 * WS;        // [BS]
    uint64_t* b_empty = b_full + BS;         // [BS]
    uint64_t* a_full = b_empty + BS;         // [AS]
    uint64_t* a_empty = a_full + AS;         // [AS]
    uint64_t* d_full = a_empty + AS;         // [1] every issuing thread's MMAs have completed
    uint64_t* u_full = d_full + 1;           // [1] U tile staged by the expander warps
    uint64_t* t_full = u_full + 1;           // [1] the three terms of T landed
    uint64_t* s_full = t_full + 1;           // [1] per-token scales and code sums staged in shared memory
    uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(smem + L::misc_off);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::misc_off + 4);
    float* scale_s = reinterpret_cast<float*>(smem + L::tok_off);
    int32_t* qsum_s = reinterpret_cast<int32_t*>(smem + L::tok_off + 4 * N_TOK);
    int32_t* zp_s = reinterpret_cast<int32_t*>(smem + L::tok_off + 8 * N_TOK);
    // after the K loop the stage memory is free:
    int32_t* red_i = reinterpret_cast<int32_t*>(smem);                                 // [N_TOK][128] partial sums
    float* red_f = reinterpret_cast<float*>(smem + N_TOK * kRowsPerCta * 4);           // [N_TOK][128] low-rank term
    __nv_bfloat16* otile = reinterpret_cast<__nv_bfloat16*>(smem);                     // [N_TOK][128] finished outputs

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = blockIdx.x * kRowsPerCta;
    const int t0 = blockIdx.y * N_TOK;
    const int split = blockIdx.z;                      // == rank in the (1,1,splits) cluster
    const int unit_begin = (int)(((int64_t)split * p.total_units) / p.splits);
    const int unit_end = (int)(((int64_t)(split + 1) * p.total_units) / p.splits);
    const bool lowrank = p.r > 0;
    const bool lowrank_here = lowrank && split == 0;   // the low-rank accumulator lives in the first CTA of a cluster

    auto sub_count = [&](int u) { return min(kUnitK / kBlockK, (p.K - u * kUnitK) / kBlockK); };
    // k-blocks this CTA contracts; every unit but the last of the matrix has eight
    const int my_blocks = (unit_end - unit_begin - 1) * (kUnitK / kBlockK) + sub_count(unit_end - 1);

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int i = 0; i < WS; ++i) { mbar_init(&w_full[i], 1); mbar_init(&w_empty[i], kExpanders / 32); }
        for (int i = 0; i < BS; ++i) { mbar_init(&b_full[i], 1); mbar_init(&b_empty[i], NISS); }
        for (int i = 0; i < AS; ++i) { mbar_init(&a_full[i], 4); mbar_init(&a_empty[i], 1); }
        mbar_init(d_full, NISS);
        mbar_init(u_full, kExpanders / 32);
        mbar_init(t_full, 1);
        mbar_init(s_full, 1);
        fence_barrier_init();
        fence_proxy_async();
    }
    if (warp == 2) {
        tmem_alloc(tmem_base_slot, TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_base_slot;
    // The next kernel of the stream may start its own independent preamble now.  The head of a group of sibling
    // contractions holds this back until it has seen the kernel before it complete (warp 1 below): whoever starts after
    // that may read that kernel's results without waiting for anything.
    const bool dep_wait = p.dep_mode != kDepSibling;   // a sibling's inputs are complete before it starts
    if (p.dep_mode != kDepHead) griddep_launch_dependents();

    if (warp == 0) {
        // ---------------- packed sign words: HBM -> shared memory (independent of the preceding kernel) ----------------
        if (elect_one()) {
            tma_prefetch_desc(&w_map);
            // every sign word is read once per call: it should not push codes, constants and kernel code out of the L2
            const uint64_t stream_once = l2_policy_evict_first();
            int ws = 0; uint32_t wph = 0;
            for (int u = unit_begin; u < unit_end && !*abort_flag; ++u) {
                // A stage that is not free yet is released by the expansion, which in the end waits for the preceding
                // kernel's codes: the bounded wait starts counting once that kernel has finished.
                if (!mbar_test_wait(&w_empty[ws], wph ^ 1)) {
                    if (dep_wait) griddep_wait();
                    if (!wait_or_abort(&w_empty[ws], wph ^ 1, abort_flag)) { give_up(p.status, abort_flag, 0x10); break; }
                }
                mbar_expect_tx(&w_full[ws], L::w_bytes);
                tma_load_2d_hint(wbuf + ws * L::w_bytes, &w_map, u * (kUnitK / 32), n0, &w_full[ws], stream_once);
                if (++ws == WS) { ws = 0; wph ^= 1; }
            }
            if (*abort_flag) for (int i = 0; i < 500; ++i) __nanosleep(100);   // let copies in flight land
        }
    } else if (warp == 1) {
        // ---------------- T and the activation codes: L2 -> shared memory ----------------
        // The first copies leave right behind the dependency: everything that can be done before it is (descriptor
        // prefetch), everything else that follows it (the per-token scalars: warp 5; the look at the status word) comes
        // after them or elsewhere.  The K loop cannot start before the first codes have landed.
        if (lane == 0) {
            tma_prefetch_desc(&b_map);
            if (lowrank_here) tma_prefetch_desc(&t_map);
        }
        if (dep_wait) griddep_wait();             // all of them come from the preceding kernel
        if (p.dep_mode == kDepHead && lane == 0) griddep_launch_dependents();
        if (elect_one()) {
            int bs = 0; uint32_t bph = 0;
            bool ok = true, first = true;
            for (int u = unit_begin; u < unit_end && ok && !*abort_flag; ++u) {
                const int ns = sub_count(u);
                for (int s0 = 0; s0 < ns; s0 += SUBS) {
                    const int cnt = min(SUBS, ns - s0);
                    if (!wait_or_abort(&b_empty[bs], bph ^ 1, abort_flag)) { give_up(p.status, abort_flag, 0x20); ok = false; break; }
                    mbar_expect_tx(&b_full[bs], cnt * L::sub_bytes);
                    for (int s = 0; s < cnt; ++s)
                        tma_load_2d(bbuf + bs * L::b_bytes + s * L::sub_bytes, &b_map, (u * 8 + s0 + s) * kBlockK, t0, &b_full[bs]);
                    if (++bs == BS) { bs = 0; bph ^= 1; }
                    if (first) {
                        first = false;
                        if (lowrank_here) {
                            mbar_expect_tx(t_full, 3 * L::sub_bytes);
                            for (int h = 0; h < 3; ++h) tma_load_3d(tbuf + h * L::sub_bytes, &t_map, 0, t0, h, t_full);
                        }
                        if (p.status && *reinterpret_cast<volatile uint32_t*>(p.status) != 0) *abort_flag = 1;   // the call already failed
                    }
                }
            }
            if (*abort_flag) for (int i = 0; i < 500; ++i) __nanosleep(100);
        }
    } else if (warp < 6) {
        // ---------------- MMA issue: thread `iss` takes k-blocks kb = iss, iss + NISS, ... ----------------
        const int iss = warp - 2;
        static_assert(NISS <= 3, "warp 5 stages the per-token scalars");
        if (warp == 5) {
            // ---------------- per-token scales, code sums and zero points into shared memory ----------------
            if (dep_wait) griddep_wait();             // they come from the preceding kernel (a sibling's are complete)
            for (int i = lane; i < N_TOK; i += 32) {
                const int t = t0 + i;
                scale_s[i] = t < p.M ? p.scales[t] : 0.f;
                int32_t qs = 0;
                if (t < p.M) {
                    const int4* parts = reinterpret_cast<const int4*>(p.qsum + (size_t)t * kQsumParts);
                    const int4 a = parts[0], b = parts[1];
                    qs = a.x + a.y + a.z + a.w + b.x + b.y + b.z + b.w;
                }
                qsum_s[i] = qs;
                zp_s[i] = (p.zp && t < p.M) ? p.zp[t] : 0;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(s_full);
        } else if (iss < NISS && elect_one()) {
            // instruction descriptors: D = s32, A = s8 (tensor memory, K-major), B = s8 (shared, K-major), M = 128;
            // and D = f32, A = B = bf16 (shared, K-major), M = 128
            const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N_TOK >> 3) << 17) | ((128u >> 4) << 24);
            const uint32_t idesc_lr = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N_TOK >> 3) << 17) | ((128u >> 4) << 24);
            bool ok = true;
            if (dep_wait) griddep_wait();             // everything this thread waits for follows the preceding kernel
            if (iss == 0 && lowrank_here) {
                if (!wait_or_abort(u_full, 0, abort_flag)) { give_up(p.status, abort_flag, 0x32); ok = false; }
                if (ok && !wait_or_abort(t_full, 0, abort_flag)) { give_up(p.status, abort_flag, 0x33); ok = false; }
                if (ok) {
                    tc_fence_after();
                    const uint32_t u_addr = smem_u32(ubuf);
#pragma unroll
                    for (int h = 0; h < 3; ++h) {
                        const uint32_t t_addr = smem_u32(tbuf + h * L::sub_bytes);
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            mma_f16_ss(tmem_base + L::D2_COL, smem_desc_sw128(u_addr, 32 * i), smem_desc_sw128(t_addr, 32 * i),
                                       idesc_lr, (h | i) ? 1u : 0u);
                    }
                }
            }
            // This thread runs a long chain of dependent scalar instructions beside warps that keep the schedulers busy, so
            // every instruction here costs several cycles: indices advance by addition (no division), descriptors are
            // built by adding to one precomputed word, and only this thread's own k-blocks are visited.
            // k-block kb of the CTA sits in code stage (kb / SUBS) % BS at sub-block kb % SUBS (all units but the last of
            // the matrix have eight sub-blocks, a multiple of SUBS) and in operand stage kb % AS.
            const uint32_t d_addr = tmem_base + iss * N_TOK;
            const uint32_t a_base = tmem_base + L::A_COL;
            const uint64_t desc_hi = smem_desc_sw128(0u, 0u);                      // everything but the start address
            const uint32_t b_lo0 = (smem_u32(bbuf) & 0x3FFFFu) >> 4;               // start-address field of stage 0, sub-block 0
            int as = iss; uint32_t aph = 0;                                        // NISS <= AS
            uint32_t acc = 0;
            int bs = 0; uint32_t bph = 0;
            for (int kb0 = 0; kb0 < my_blocks && ok; kb0 += SUBS) {
                // every issuing thread sees each code stage filled before it releases it, whether or not one of the
                // stage's k-blocks is its own: its release can then never run a whole ring ahead
                if (!wait_or_abort(&b_full[bs], bph, abort_flag)) { give_up(p.status, abort_flag, 0x30); ok = false; break; }
                const int cnt = min(SUBS, my_blocks - kb0);
                const uint32_t stage_lo = b_lo0 + (uint32_t)bs * (L::b_bytes >> 4);
#pragma unroll
                for (int sb = 0; sb < SUBS; ++sb) {
                    const bool own = (SUBS % NISS == 0) ? (sb % NISS == iss) : ((kb0 + sb) % NISS == iss);
                    if (ok && sb < cnt && own) {
                        if (!wait_or_abort(&a_full[as], aph, abort_flag)) { give_up(p.status, abort_flag, 0x31); ok = false; }
                        if (ok) {
                            tc_fence_after();
                            const uint64_t desc = desc_hi | (uint64_t)(stage_lo + (uint32_t)sb * (L::sub_bytes >> 4));
                            const uint32_t a_addr = a_base + 32 * as;
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                mma_i8_ts(d_addr, a_addr + 8 * i, desc + 2 * i, idesc, acc);   // 32 bytes along K = 2 address units
                                acc = 1u;
                            }
                            tc_commit(&a_empty[as]);
                            as += NISS;
                            if (as >= AS) { as -= AS; aph ^= 1u; }
                        }
                    }
                }
                // this thread is done with the code stage once its MMAs so far have completed
                tc_commit(&b_empty[bs]);
                if (++bs == BS) { bs = 0; bph ^= 1u; }
            }
            tc_commit(d_full);
        }
    } else {
        // ---------------- U tile, expansion of sign bits into tensor memory, then the epilogue ----------------
        const int q = warp & 3;                       // tensor-memory lane quarter this warp may touch
        const int part = (warp - 6) >> 2;             // which of the EW warps of that quarter
        const int row = q * 32 + lane;
        const int e = threadIdx.x - kFirstExpander;   // 0..255 among the expander threads
        const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
        // this row's weight scale and shift do not depend on the preceding kernel: fetched now, used in the epilogue
        float alpha_row = n0 + row < p.N ? __ldg(p.alpha + n0 + row) : 0.f;
        float mu_row = (p.mu && n0 + row < p.N) ? __ldg(p.mu + n0 + row) : 0.f;
        const int32_t rs_row = (p.zp && n0 + row < p.N) ? __ldg(p.rowsum + n0 + row) : 0;
        // pinned in registers: left alone, the compiler re-issues the global loads where the values are used
        asm volatile("" : "+f"(alpha_row), "+f"(mu_row));
        if (lowrank_here) {
            // 128 rows x 8 chunks of 16 bytes, 128B-swizzled K-major; rows beyond N and columns beyond r are zero
            const bool vec = (p.r % 8 == 0) && ((reinterpret_cast<uintptr_t>(p.U) & 15) == 0);
#pragma unroll
            for (int it = 0; it < 1024 / kExpanders; ++it) {
                const int idx = it * kExpanders + e;
                const int ur = idx >> 3, ch = idx & 7;
                uint4 v = make_uint4(0u, 0u, 0u, 0u);
                const int n = n0 + ur;
                if (n < p.N && ch * 8 < p.r) {
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
                *reinterpret_cast<uint4*>(ubuf + ur * 128 + ((ch ^ (ur & 7)) << 4)) = v;
            }
            fence_proxy_async();                      // generic-proxy stores -> visible to the tensor core's reads
            __syncwarp();
            if (lane == 0) mbar_arrive(u_full);
        }
        // This warp expands k-blocks kb = part, part + EW, ... of the CTA (operand stage kb % AS; AS is a multiple of EW and
        // every unit but the last of the matrix has eight k-blocks, also a multiple of EW, so inside each unit the warp
        // takes sub-blocks part, part + EW, ...).  Its registers are left alone until tcgen05.wait::st has returned; the
        // other warps of the quarter fill the store's latency.
        int ws = 0; uint32_t wph = 0;
        int as = part; uint32_t aph = 0;
        bool ok = true;
        for (int u = unit_begin; u < unit_end && ok; ++u) {
            if (!warp_wait(&w_full[ws], wph, abort_flag)) { give_up(p.status, abort_flag, 0x40); ok = false; break; }
            const uint8_t* wrow = wbuf + ws * L::w_bytes + row * 128;
            const int ns = sub_count(u);
            // a rolled loop over this warp's k-blocks of the unit; each block's sign words are loaded just before they are
            // expanded
#pragma unroll 1
            for (int s = part; s < ns && ok; s += EW) {
                const uint4 w4 = *reinterpret_cast<const uint4*>(wrow + ((s ^ (row & 7)) << 4));
                uint32_t v[32];
                const uint32_t w[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int j = 0; j < 8; ++j) v[8 * c + j] = (w[c] << (7 - j)) & 0x80808080u;
                // An operand stage that is still taken frees up only when MMAs have run, and those need the codes of the
                // preceding kernel: the bounded wait starts counting once that kernel has finished.
                if (!__all_sync(0xFFFFFFFFu, mbar_test_wait(&a_empty[as], aph ^ 1u))) {
                    if (dep_wait) griddep_wait();
                    if (!warp_wait(&a_empty[as], aph ^ 1u, abort_flag)) { give_up(p.status, abort_flag, 0x41); ok = false; }
                }
                if (ok) {
                    tc_fence_after();
                    tmem_st_32x32(tmem_base + lane_addr + L::A_COL + 32 * as, v);
                    tc_wait_st();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&a_full[as]);
                    as += EW;
                    if (as >= AS) { as = part; aph ^= 1u; }
                }
            }
            // The stage is released only here, after every word of it that this warp needs has gone through the expansion:
            // an arrive placed earlier let the copy of a later unit overwrite words not yet read.
            __syncwarp();
            if (lane == 0) mbar_arrive(&w_empty[ws]);
            if (++ws == WS) { ws = 0; wph ^= 1u; }
        }
        // the stores of the epilogue come after the preceding kernel (for a sibling: this is the wait every kernel of the
        // chain executes before it ends); the per-token scales and code sums were staged in shared memory by warp 1
        // while the K loop ran
        griddep_wait();
        if (!warp_wait(s_full, 0, abort_flag)) { give_up(p.status, abort_flag, 0x51); ok = false; }
        if (ok) {
            if (!warp_wait(d_full, 0, abort_flag)) { give_up(p.status, abort_flag, 0x50); ok = false; }
        }
        if (ok) {
            tc_fence_after();
            const int n = n0 + row;
            const int nacc = min(NISS, my_blocks);             // accumulators that hold something
            const bool single = p.splits == 1;
            const float alpha_n = alpha_row, mu_n = mu_row;
            int32_t* const dbg = p.acc_debug;
            const int M_ = p.M, N_ = p.N;
            const bool valid_row = n < N_;
            // the warps of a quarter take chunks of 16 tokens in turn
#pragma unroll 1
            for (int c = part; c < N_TOK / 16; c += EW) {
                if (t0 + 16 * c >= p.M) break;                 // warp-uniform
                uint32_t v[16], l[16];
                tmem_ld_32x16(tmem_base + lane_addr + 16 * c, v);
                if (lowrank_here) tmem_ld_32x16(tmem_base + lane_addr + L::D2_COL + 16 * c, l);
                tc_wait_ld();
#pragma unroll
                for (int a = 1; a < NISS; ++a) {
                    if (a < nacc) {
                        uint32_t v2[16];
                        tmem_ld_32x16(tmem_base + lane_addr + a * N_TOK + 16 * c, v2);
                        tc_wait_ld();
#pragma unroll
                        for (int j = 0; j < 16; ++j) v[j] += v2[j];
                    }
                }
                // the chunk's scales and code sums go to registers first: the tile stores below may alias them as far as
                // the compiler knows, and a load behind every store would serialise the loop
                float sc[16]; int32_t qs[16], zp[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) { sc[j] = scale_s[16 * c + j]; qs[j] = qsum_s[16 * c + j]; zp[j] = zp_s[16 * c + j]; }
                // branch-free per element (rows beyond N and tokens beyond M produce values nobody stores):
                // a branch per element costs more than the arithmetic it would skip
                if (dbg && valid_row) {
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        if (t0 + 16 * c + j < M_) dbg[(int64_t)(t0 + 16 * c + j) * N_ + n] = -((int32_t)v[j] >> 6) - qs[j] - zp[j] * rs_row;
                }
                if (single) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const float lr = lowrank_here ? __uint_as_float(l[j]) : 0.f;
                        const float y = finish_value((int32_t)v[j], lr, __fmul_rn(alpha_n, sc[j]), __fmul_rn(mu_n, sc[j]), qs[j],
                                                     zp[j] * rs_row, p.K * zp[j]);
                        otile[(16 * c + j) * kRowsPerCta + row] = __float2bfloat16_rn(y);      // [token][row]
                    }
                } else if (L::can_split) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        red_i[(16 * c + j) * kRowsPerCta + row] = (int32_t)v[j];
                        if (lowrank_here) red_f[(16 * c + j) * kRowsPerCta + row] = __uint_as_float(l[j]);
                    }
                }
            }
        }
        if (p.splits == 1) {
            asm volatile("bar.sync 1, %0;" ::"r"(kExpanders) : "memory");   // the output tile is complete (all expander warps, always)
            if (ok && p.out) {
                // 16 threads move one token's 128 outputs (256 bytes) with 128-bit stores
                const bool vec = ((reinterpret_cast<uintptr_t>(p.out) & 15) == 0) && (p.ldo % 8 == 0) && (n0 + kRowsPerCta <= p.N);
                for (int tt = e >> 4; tt < N_TOK && t0 + tt < p.M; tt += kExpanders / 16) {
                    const int c8 = (e & 15) * 8;
                    __nv_bfloat16* dst = p.out + (int64_t)(t0 + tt) * p.ldo + n0 + c8;
                    const uint4 val = *reinterpret_cast<const uint4*>(otile + tt * kRowsPerCta + c8);
                    if (vec) {
                        *reinterpret_cast<uint4*>(dst) = val;
                    } else {
                        const __nv_bfloat16* sv = reinterpret_cast<const __nv_bfloat16*>(&val);
                        for (int j = 0; j < 8; ++j)
                            if (n0 + c8 + j < p.N) dst[j] = sv[j];
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (p.splits > 1) {
        // every thread of every CTA of the cluster takes part, whether or not its CTA gave up
        cluster_arrive_release();
        cluster_wait_acquire();
        if (L::can_split && warp >= 6 && !*abort_flag) {
            // the tokens of the tile are dealt round-robin to the CTAs of the cluster; a thread sums four consecutive
            // rows of one token over all CTAs with 128-bit distributed-shared-memory loads
            const int e = threadIdx.x - kFirstExpander;
            const int r4 = (e & 31) * 4;
            const int n = n0 + r4;
            for (int ti = e >> 5; ; ti += kExpanders / 32) {
                const int tt = split + ti * p.splits;
                if (tt >= N_TOK || t0 + tt >= p.M) break;
                const uint32_t off_i = smem_u32(&red_i[tt * kRowsPerCta + r4]);
                uint4 part[8];
#pragma unroll
                for (int c = 0; c < 8; ++c)
                    if (c < p.splits) part[c] = ld_shared_cluster_v4(map_shared_rank(off_i, c));
                uint4 lf = make_uint4(0u, 0u, 0u, 0u);
                if (lowrank) lf = ld_shared_cluster_v4(map_shared_rank(smem_u32(&red_f[tt * kRowsPerCta + r4]), 0));
                int32_t d[4] = {0, 0, 0, 0};
#pragma unroll
                for (int c = 0; c < 8; ++c)
                    if (c < p.splits) { d[0] += (int32_t)part[c].x; d[1] += (int32_t)part[c].y; d[2] += (int32_t)part[c].z; d[3] += (int32_t)part[c].w; }
                const float l4[4] = {__uint_as_float(lf.x), __uint_as_float(lf.y), __uint_as_float(lf.z), __uint_as_float(lf.w)};
                __align__(8) __nv_bfloat16 y4[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    float y = 0.f;
                    if (n + j < p.N) {
                        const int32_t zr = p.zp ? zp_s[tt] * p.rowsum[n + j] : 0;
                        y = finish_value(d[j], l4[j], __fmul_rn(p.alpha[n + j], scale_s[tt]),
                                         p.mu ? __fmul_rn(p.mu[n + j], scale_s[tt]) : 0.f, qsum_s[tt], zr, p.K * zp_s[tt]);
                        if (p.acc_debug) p.acc_debug[(int64_t)(t0 + tt) * p.N + n + j] = -(d[j] >> 6) - qsum_s[tt] - zr;
                    }
                    y4[j] = __float2bfloat16_rn(y);
                }
                if (p.out) {
                    __nv_bfloat16* dst = p.out + (int64_t)(t0 + tt) * p.ldo + n;
                    if (((reinterpret_cast<uintptr_t>(dst) & 7) == 0) && n + 3 < p.N) {
                        *reinterpret_cast<uint2*>(dst) = *reinterpret_cast<const uint2*>(y4);
                    } else {
                        for (int j = 0; j < 4; ++j)
                            if (n + j < p.N) dst[j] = y4[j];
                    }
                }
            }
        }
        // nobody leaves while a neighbour may still read its shared memory
        cluster_arrive_release();
        cluster_wait_acquire();
    }
    if (warp == 2) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// -------------------------------------------------------------------------------------------------
// host side
// -------------------------------------------------------------------------------------------------
template <int N_TOK, int WS, int BS, int TMEM_COLS, int NISS, int EW>
static int launch_umma_t(const CUtensorMap& wm, const CUtensorMap& bm, const CUtensorMap& tm, const UmmaParams& p,
                         dim3 grid, cudaStream_t s) {
    using L = UmmaCfg<N_TOK, WS, BS, TMEM_COLS, NISS, EW>;
    auto kernel = umma_w1a_kernel<N_TOK, WS, BS, TMEM_COLS, NISS, EW>;
    static thread_local int configured = -1;
    int dev = 0;
    BWLA_CUDA_TRY(cudaGetDevice(&dev));
    if (configured != dev) {
        BWLA_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, L::total));
        configured = dev;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(L::kThreads, 1, 1);
    cfg.dynamicSmemBytes = L::total;
    cfg.stream = s;
    cudaLaunchAttribute attrs[2];
    attrs[0].id = cudaLaunchAttributeClusterDimension;
    attrs[0].val.clusterDim.x = 1; attrs[0].val.clusterDim.y = 1; attrs[0].val.clusterDim.z = grid.z;
    attrs[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attrs[1].val.programmaticStreamSerializationAllowed = launch_overlap_allowed();
    cfg.attrs = attrs;
    cfg.numAttrs = 2;
    ProfScope prof(kProfContraction, s);
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, wm, bm, tm, p);
    if (e != cudaSuccess) { cudaGetLastError(); return cuda_fail(e); }
    return after_launch();
}

bool umma_supports(int64_t M, int64_t K, int64_t N, int r, int bits) {
    // the tensor core sums -128 * code over the set sign bits: |D| <= 128 * K * qmax must fit the int32 accumulator
    // (asymmetric codes reach -2^(b-1), one step further than the symmetric ones)
    const int64_t qmax = (int64_t)1 << (bits - 1);
    return M > 0 && N > 0 && K % 128 == 0 && 128 * K * qmax < ((int64_t)1 << 31) && r <= kLowrankPad &&
           M * N < (int64_t)1 << 31 && M < (int64_t)1 << 30 && encode_tiled_fn() != nullptr;
}

// How many CTAs share a tile and split K, for the configuration with two CTAs per SM.  Enough to put about one CTA on
// every SM, never more than the units there are, never more than the portable cluster size; powers of two.
static int choose_splits(int tiles, int units, bool can_split, int sms) {
    if (!can_split) return 1;
    int s = 1;
    while (s * 2 <= 8 && s * 2 <= units && tiles * s * 2 <= sms + sms / 4) s *= 2;
    return s;
}

// Few tokens: a CTA's K loop is a chain of latencies, not of throughput, so one CTA per SM with twice the expander warps
// and a twice as deep operand ring (all 512 tensor-memory columns) gets through its k-blocks about 1.7 times as fast
// as one of two CTAs that share an SM.  It is worth it when a K split puts the whole grid on the SMs at once.
// Returns the split for that configuration, or 0 when two CTAs per SM are expected to finish sooner.
static int choose_wide_splits(int tiles, int units, int narrow_splits, int sms) {
    if (tiles > sms) return 0;
    int s = sms / tiles;
    if (s > 8) s = 8;
    if (s > units) s = units;
    if (s < 1) return 0;
    const int blocks = units * (kUnitK / kBlockK);
    const double wide = (double)((blocks + s - 1) / s) / 1.7;
    const double narrow = (double)((blocks + narrow_splits - 1) / narrow_splits) * (tiles * narrow_splits > sms ? 1.2 : 1.0);
    return wide < narrow ? s : 0;
}

// codes_interleaved: int8 [M][K] in the interleaved order.  a.Thl: bf16 [3][M][64], T = hi + mid + lo.
int launch_gemm_umma(const GemmArgs& a, const int8_t* codes_interleaved, cudaStream_t stream) {
    const int M = (int)a.M, N = (int)a.N, K = (int)a.K;
    if (umma_persistent_supports(a.M, a.K, a.N, a.r)) return launch_gemm_umma_persistent(a, codes_interleaved, stream);
    if (M > 64) return BWLA_ERR_UNSUPPORTED;                  // (every such problem this path takes went to the persistent kernel)
    const int n_tok = M <= 16 ? 16 : M <= 32 ? 32 : 64;
    const int row_tiles = (N + kRowsPerCta - 1) / kRowsPerCta;
    const int tok_tiles = (M + n_tok - 1) / n_tok;
    const int units = (K + kUnitK - 1) / kUnitK;
    const int sms = sm_count();
    if (sms <= 0) return BWLA_ERR_CUDA;
    // siblings that run beside one another plan for their share of the SMs
    const int plan_sms = a.sm_budget > 0 ? std::max(std::min(sms, a.sm_budget), row_tiles * tok_tiles) : sms;
    int split = choose_splits(row_tiles * tok_tiles, units, n_tok <= 64, plan_sms);
    const int wide_split = n_tok <= 32 ? choose_wide_splits(row_tiles * tok_tiles, units, split, plan_sms) : 0;
    if (wide_split) split = wide_split;

    CUtensorMap wm, bm, tm;
    {
        const uint64_t dims[2] = {(uint64_t)K / 32, (uint64_t)N};
        const uint64_t strides[1] = {(uint64_t)K / 8};
        const uint32_t box[2] = {32, kRowsPerCta};
        int st = make_map(&wm, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, a.packed, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
        if (st != BWLA_OK) return st;
    }
    {
        const uint64_t dims[2] = {(uint64_t)K, (uint64_t)M};
        const uint64_t strides[1] = {(uint64_t)K};
        const uint32_t box[2] = {kBlockK, (uint32_t)n_tok};
        int st = make_map(&bm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, codes_interleaved, dims, strides, box,
                          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
        if (st != BWLA_OK) return st;
    }
    if (a.r > 0) {
        const uint64_t dims[3] = {(uint64_t)kLowrankPad, (uint64_t)M, 3};
        const uint64_t strides[2] = {(uint64_t)kLowrankPad * 2, (uint64_t)M * kLowrankPad * 2};
        const uint32_t box[3] = {(uint32_t)kLowrankPad, (uint32_t)n_tok, 1};
        int st = make_map(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, a.Thl, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
        if (st != BWLA_OK) return st;
    } else {
        tm = bm;   // never dereferenced
    }

    UmmaParams p{};
    p.M = M; p.N = N; p.K = K; p.total_units = units; p.splits = split; p.r = a.r;
    p.scales = a.scales; p.qsum = a.qsum; p.alpha = a.alpha; p.mu = a.mu; p.zp = a.zp; p.rowsum = a.rowsum; p.U = (const __nv_bfloat16*)a.U;
    p.out = (__nv_bfloat16*)a.out; p.ldo = a.ldo; p.acc_debug = a.acc_debug; p.status = a.status; p.dep_mode = a.dep_mode;

    dim3 grid((unsigned)row_tiles, (unsigned)tok_tiles, (unsigned)split);
    switch (n_tok) {
                case 16: return wide_split ? launch_umma_t<16, 3, 2, 512, 2, 4>(wm, bm, tm, p, grid, stream)
                                   : launch_umma_t<16, 3, 2, 256, 2, 2>(wm, bm, tm, p, grid, stream);
        case 32: return wide_split ? launch_umma_t<32, 3, 2, 512, 2, 4>(wm, bm, tm, p, grid, stream)
                                   : launch_umma_t<32, 3, 2, 256, 2, 2>(wm, bm, tm, p, grid, stream);
        // a grid larger than the SM count would run in two waves with one CTA per SM: two smaller CTAs per SM instead
        case 64: return grid.x * grid.y * grid.z > (unsigned)sms ? launch_umma_t<64, 2, 2, 256, 1, 2>(wm, bm, tm, p, grid, stream)
                                                       : launch_umma_t<64, 4, 3, 512, 2, 4>(wm, bm, tm, p, grid, stream);
    }
    return BWLA_ERR_UNSUPPORTED;
}

}  // namespace bwla
