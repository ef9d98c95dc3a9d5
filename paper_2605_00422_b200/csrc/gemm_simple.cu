// Plain CUDA kernels: the first stage of the PSP low-rank branch, T = V x (Sec. 3.2: W x = (W - M) x + A (B x)),
// and a one-warp-per-output-row contraction + epilogue.  The latter is deliberately simple: it is the on-device
// cross-check for the tensor-core paths and the path of last resort for shapes they do not take.
#include <cuda_bf16.h>

#include "bwla_common.cuh"

namespace bwla {

constexpr int kTokTile = 8;

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// grid (r, ceil(M / kTokTile)); each block reduces one row of V against kTokTile activation rows.
__global__ void __launch_bounds__(256) lowrank_T_kernel(const __nv_bfloat16* __restrict__ x, int64_t M, int K,
                                                        int64_t ldx, const __nv_bfloat16* __restrict__ V, int r,
                                                        float* __restrict__ T) {
    const int j = blockIdx.x;
    const int64_t t0 = (int64_t)blockIdx.y * kTokTile;
    const int nt = (int)min((int64_t)kTokTile, M - t0);
    float acc[kTokTile];
#pragma unroll
    for (int i = 0; i < kTokTile; ++i) acc[i] = 0.f;
    const __nv_bfloat16* vrow = V + (int64_t)j * K;
    for (int k = threadIdx.x; k < K; k += blockDim.x) {
        const float v = __bfloat162float(vrow[k]);
#pragma unroll
        for (int i = 0; i < kTokTile; ++i)
            if (i < nt) acc[i] = fmaf(v, __bfloat162float(x[(t0 + i) * ldx + k]), acc[i]);
    }
    __shared__ float red[kTokTile][8];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int i = 0; i < kTokTile; ++i) {
        float v = acc[i];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
        if (lane == 0) red[i][warp] = v;
    }
    __syncthreads();
    if (threadIdx.x < nt) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) s += red[threadIdx.x][w];
        T[(t0 + threadIdx.x) * r + j] = s;
    }
}

int launch_lowrank_T(const void* x, int64_t M, int64_t K, int64_t ldx, const void* V, int r, float* T,
                     cudaStream_t stream) {
    if (M == 0 || r == 0) return BWLA_OK;
    dim3 grid((unsigned)r, (unsigned)((M + kTokTile - 1) / kTokTile));
    ProfScope prof(kProfLowrankT, stream);
    lowrank_T_kernel<<<grid, 256, 0, stream>>>((const __nv_bfloat16*)x, M, (int)K, ldx, (const __nv_bfloat16*)V, r, T);
    return after_launch();
}

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
        if (a.acc_debug) a.acc_debug[t * a.N + n] = v;
        if (a.out) {
            const float sc = a.scales[t];
            float y = __fmul_rn(__fmul_rn(a.alpha[n], sc), (float)v);
            if (a.r > 0) {
                const __nv_bfloat16* u = (const __nv_bfloat16*)a.U + n * a.r;
                float l = 0.f;
                for (int j = 0; j < a.r; ++j) l = fmaf(__bfloat162float(u[j]), a.T[t * a.r + j], l);
                y += l;
            }
            if (a.mu) y = fmaf(__fmul_rn(a.mu[n], sc), (float)a.qsum[t], y);
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
