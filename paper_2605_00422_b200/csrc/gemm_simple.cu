// A one-warp-per-output-row contraction + epilogue in plain CUDA.  Deliberately simple: it is the on-device
// cross-check for the tensor-core path and the path of last resort for shapes that path does not take.
#include <cuda_bf16.h>

#include "bwla_common.cuh"

namespace bwla {

constexpr int kTokTile = 8;

// One warp per output row n and tile of kTokTile tokens; lanes split the K/32 weight words.
__global__ void __launch_bounds__(128) gemm_simple_kernel(GemmArgs a) {
    const int lane = threadIdx.x & 31;
    const int64_t n = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5);
    if (n >= a.N) return;
    const int64_t t0 = (int64_t)blockIdx.y * kTokTile;
    const int nt = (int)min((int64_t)kTokTile, a.M - t0);
    const int words = (int)(a.K >> 5);
    int acc[kTokTile];
#pragma unroll
    for (int i = 0; i < kTokTile; ++i) acc[i] = 0;
    for (int wd = lane; wd < words; wd += 32) {
        const uint32_t w = __ldg(a.packed + n * words + wd);
#pragma unroll
        for (int i = 0; i < kTokTile; ++i) {
            if (i < nt) {
                const int8_t* c = a.codes + (t0 + i) * a.K + 32 * wd;
                int s = 0;
#pragma unroll
                for (int k = 0; k < 32; ++k) s += ((w >> k) & 1u) ? (int)c[k] : -(int)c[k];
                acc[i] += s;
            }
        }
    }
#pragma unroll
    for (int i = 0; i < kTokTile; ++i) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc[i] += __shfl_xor_sync(0xFFFFFFFFu, acc[i], o);
    }
    if (lane < nt) {
        int v = 0;
#pragma unroll
        for (int i = 0; i < kTokTile; ++i) v = (lane == i) ? acc[i] : v;
        const int64_t t = t0 + lane;
        // asymmetric codes: the zero point leaves through the row's sign sum (exact in int32)
        const int32_t zp = a.zp ? a.zp[t] : 0;
        if (a.zp) v -= zp * a.rowsum[n];
        if (a.acc_debug) a.acc_debug[t * a.N + n] = v;
        if (a.out) {
            const float sc = a.scales[t];
            float y = __fmul_rn(__fmul_rn(a.alpha[n], sc), (float)v);
            if (a.r > 0) {
                // PSP term U (V x) (Sec. 3.2) from T kept as three bf16 terms
                const int cols = lowrank_cols(a.r);
                const __nv_bfloat16* u = (const __nv_bfloat16*)a.U + n * a.r;
                const __nv_bfloat16* hi = (const __nv_bfloat16*)a.Thl + t * cols;
                const __nv_bfloat16* mid = hi + a.M * cols;
                const __nv_bfloat16* lo = mid + a.M * cols;
                float l = 0.f;
                for (int j = 0; j < a.r; ++j)
                    l = fmaf(__bfloat162float(u[j]), (__bfloat162float(hi[j]) + __bfloat162float(mid[j])) + __bfloat162float(lo[j]), l);
                y += l;
            }
            if (a.mu) {
                int32_t qs = 0;
                for (int c = 0; c < kQsumParts; ++c) qs += a.qsum[t * kQsumParts + c];
                qs -= (int32_t)a.K * zp;
                y = fmaf(__fmul_rn(a.mu[n], sc), (float)qs, y);
            }
            ((__nv_bfloat16*)a.out)[t * a.ldo + n] = __float2bfloat16_rn(y);
        }
    }
}

int launch_gemm_simple(const GemmArgs& a, cudaStream_t stream) {
    if (a.M == 0 || a.N == 0) return BWLA_OK;
    dim3 grid((unsigned)((a.N + 3) / 4), (unsigned)((a.M + kTokTile - 1) / kTokTile));
    ProfScope prof(kProfContraction, stream);
    gemm_simple_kernel<<<grid, 128, 0, stream>>>(a);
    return after_launch();
}

}  // namespace bwla
