// Online OKT + per-token symmetric quantiser, fused: one block per token.
//
//   X = reshape(x_t, n1 x n2) (row-major), Z = X * P2, Y = P1^T * Z, amax = max|Y|,
//   q = clamp(rne(Y * (qmax / amax)), +-qmax), s_t = amax / qmax.
//
// (Sec. 3.1: R = R1 (x) R2 evaluated as two small contractions on the reshaped vector; Sec. 4.1: per-token
// activation quantisation.)  X, Z and Y live in shared memory (2*K floats); Y never touches HBM.  The two
// contractions are register-tiled 4x4 fp32 FMA loops; the absmax is a warp-shuffle + shared-memory reduction;
// codes leave as 128-bit stores.
#include <cuda_bf16.h>

#include "bwla_common.cuh"

namespace bwla {

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

// Generic contraction used when n2 is not a multiple of 4 (odd test shapes): one output per thread step.
__device__ void rotate_scalar(const float* __restrict__ X, float* __restrict__ Z, float* __restrict__ Y,
                              const float* __restrict__ P1, int n1, const float* __restrict__ P2, int n2,
                              float& amax) {
    const int K = n1 * n2;
    for (int o = threadIdx.x; o < K; o += blockDim.x) {
        const int a = o / n2, d = o - a * n2;
        float s = 0.f;
        for (int b = 0; b < n2; ++b) s = fmaf(X[a * n2 + b], __ldg(P2 + b * n2 + d), s);
        Z[o] = s;
    }
    __syncthreads();
    for (int o = threadIdx.x; o < K; o += blockDim.x) {
        const int c = o / n2, d = o - c * n2;
        float s = 0.f;
        for (int a = 0; a < n1; ++a) s = fmaf(__ldg(P1 + a * n1 + c), Z[a * n2 + d], s);
        Y[o] = s;
        amax = fmaxf(amax, fabsf(s));
    }
}

// Register-tiled contraction, n2 % 4 == 0: each thread owns 4 rows x 4 columns of the output.
__device__ void rotate_tiled(const float* __restrict__ X, float* __restrict__ Z, float* __restrict__ Y,
                             const float* __restrict__ P1, int n1, const float* __restrict__ P2, int n2,
                             float& amax) {
    const int dt_count = n2 >> 2;
    const int mt_count = (n1 + 3) >> 2;
    const int tiles = dt_count * mt_count;
    // Z = X * P2
    for (int tile = threadIdx.x; tile < tiles; tile += blockDim.x) {
        const int mt = tile / dt_count, d0 = (tile - mt * dt_count) << 2;
        const int a0 = mt << 2;
        const float* xr[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) xr[i] = X + min(a0 + i, n1 - 1) * n2;
        float acc[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
        const float* p = P2 + d0;
#pragma unroll 4
        for (int b = 0; b < n2; ++b) {
            const float4 pv = __ldg(reinterpret_cast<const float4*>(p + (size_t)b * n2));
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float xa = xr[i][b];
                acc[i][0] = fmaf(xa, pv.x, acc[i][0]);
                acc[i][1] = fmaf(xa, pv.y, acc[i][1]);
                acc[i][2] = fmaf(xa, pv.z, acc[i][2]);
                acc[i][3] = fmaf(xa, pv.w, acc[i][3]);
            }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
            if (a0 + i < n1)
                *reinterpret_cast<float4*>(Z + (a0 + i) * n2 + d0) = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
    }
    __syncthreads();
    // Y = P1^T * Z   (Y overwrites X, which is dead now)
    for (int tile = threadIdx.x; tile < tiles; tile += blockDim.x) {
        const int mt = tile / dt_count, d0 = (tile - mt * dt_count) << 2;
        const int c0 = mt << 2;
        int cc[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) cc[i] = min(c0 + i, n1 - 1);
        float acc[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
#pragma unroll 4
        for (int a = 0; a < n1; ++a) {
            const float4 zv = *reinterpret_cast<const float4*>(Z + a * n2 + d0);
            const float* prow = P1 + (size_t)a * n1;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float pa = __ldg(prow + cc[i]);
                acc[i][0] = fmaf(pa, zv.x, acc[i][0]);
                acc[i][1] = fmaf(pa, zv.y, acc[i][1]);
                acc[i][2] = fmaf(pa, zv.z, acc[i][2]);
                acc[i][3] = fmaf(pa, zv.w, acc[i][3]);
            }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
            if (c0 + i < n1) {
                *reinterpret_cast<float4*>(Y + (c0 + i) * n2 + d0) = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
                amax = fmaxf(amax, fmaxf(fmaxf(fabsf(acc[i][0]), fabsf(acc[i][1])), fmaxf(fabsf(acc[i][2]), fabsf(acc[i][3]))));
            }
    }
}

// codes_layout 0: byte p of a 32-group holds k = p.  1: byte 4*j + i holds k = j + 8*i (j < 8, i < 4), the
// order in which the tensor-core contraction meets the weights after its shift-and-mask expansion.
__global__ void rotate_quant_kernel(const __nv_bfloat16* __restrict__ x, int64_t M, int K, int64_t ldx,
                                    const float* __restrict__ P1, int n1, const float* __restrict__ P2, int n2,
                                    int bits, int8_t* __restrict__ codes, int codes_layout,
                                    float* __restrict__ scales, int32_t* __restrict__ qsum,
                                    uint32_t* __restrict__ planes, uint32_t* __restrict__ status) {
    if (status && blockIdx.x == 0 && threadIdx.x == 0) status[0] = 0;   // this call's status starts clean
    extern __shared__ __align__(16) float smem[];
    float* bufX = smem;        // X, later Y
    float* bufZ = smem + K;    // Z
    __shared__ float red_max[32];
    __shared__ int red_sum;
    const int qmax = (1 << (bits - 1)) - 1;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;

    for (int64_t t = blockIdx.x; t < M; t += gridDim.x) {
        const __nv_bfloat16* xt = x + t * ldx;
        if ((reinterpret_cast<uintptr_t>(xt) & 15) == 0) {
            const uint4* xv = reinterpret_cast<const uint4*>(xt);
            for (int i = threadIdx.x; i < (K >> 3); i += blockDim.x) {
                const uint4 v = __ldg(xv + i);
                const uint32_t w[4] = {v.x, v.y, v.z, v.w};
                float f[8];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    f[2 * j] = __uint_as_float(w[j] << 16);
                    f[2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
                }
                *reinterpret_cast<float4*>(bufX + 8 * i) = make_float4(f[0], f[1], f[2], f[3]);
                *reinterpret_cast<float4*>(bufX + 8 * i + 4) = make_float4(f[4], f[5], f[6], f[7]);
            }
        } else {
            for (int k = threadIdx.x; k < K; k += blockDim.x) bufX[k] = __bfloat162float(xt[k]);
        }
        if (threadIdx.x == 0) red_sum = 0;
        __syncthreads();

        float amax = 0.f;
        if ((n2 & 3) == 0) rotate_tiled(bufX, bufZ, bufX, P1, n1, P2, n2, amax);
        else {
            // the scalar variant may not alias: Y goes to bufX only after Z is complete (it syncs inside)
            rotate_scalar(bufX, bufZ, bufX, P1, n1, P2, n2, amax);
        }
        amax = warp_max(amax);
        if (lane == 0) red_max[warp] = amax;
        __syncthreads();
        amax = (lane < nwarps) ? red_max[lane] : 0.f;
        amax = warp_max(amax);

        float inv, scale;
        if (amax == 0.f) { inv = 0.f; scale = 1.f; }
        else { inv = __fdiv_rn((float)qmax, amax); scale = __fdiv_rn(amax, (float)qmax); }

        int local_sum = 0;
        int8_t* ct = codes + t * (int64_t)K;
        const int words = K >> 5;
        for (int g = threadIdx.x; g < words; g += blockDim.x) {
            const float* y = bufX + 32 * g;
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
                    const int k = codes_layout ? (j + 8 * i) : (4 * j + i);
                    v |= (uint32_t)(q[k] & 0xFF) << (8 * i);
                }
                w[j] = v;
            }
            uint4* dst = reinterpret_cast<uint4*>(ct + 32 * g);
            dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
            dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
            if (planes) {
                // plane i of u = q + qmax, LSB-first like the weight words; plane index `bits` is all ones
                uint32_t* pt = planes + (t * 8) * (int64_t)words;
                for (int i = 0; i < bits; ++i) {
                    uint32_t pw = 0;
#pragma unroll
                    for (int k = 0; k < 32; ++k) pw |= (uint32_t)(((q[k] + qmax) >> i) & 1) << k;
                    pt[(int64_t)i * words + g] = pw;
                }
                for (int i = bits; i < 8; ++i) pt[(int64_t)i * words + g] = (i == bits) ? 0xFFFFFFFFu : 0u;
            }
        }
        local_sum = warp_sum(local_sum);
        if (lane == 0 && local_sum != 0) atomicAdd(&red_sum, local_sum);
        __syncthreads();
        if (threadIdx.x == 0) {
            scales[t] = scale;
            if (qsum) qsum[t] = red_sum;
        }
        __syncthreads();
    }
}

int launch_rotate_quant(const void* x, int64_t M, int64_t K, int64_t ldx, const float* P1, int n1,
                        const float* P2, int n2, int bits, int8_t* codes, int codes_layout, float* scales,
                        int32_t* qsum, uint32_t* planes, uint32_t* status, cudaStream_t stream) {
    if (M == 0) return BWLA_OK;
    const size_t smem = (size_t)K * 8;
    static thread_local int configured_device = -1;
    int dev = 0;
    BWLA_CUDA_TRY(cudaGetDevice(&dev));
    if (configured_device != dev) {
        BWLA_CUDA_TRY(cudaFuncSetAttribute(rotate_quant_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 25600 * 8));
        configured_device = dev;
    }
    const int threads = (K >= 8192) ? 512 : 256;
    const unsigned grid = (unsigned)(M < 148 * 64 ? M : 148 * 64);
    ProfScope prof(kProfRotateQuant, stream);
    rotate_quant_kernel<<<grid, threads, smem, stream>>>((const __nv_bfloat16*)x, M, (int)K, ldx, P1, n1, P2, n2, bits,
                                                         codes, codes_layout, scales, qsum, planes, status);
    return after_launch();
}

// ---------------------------------------------------------------------------------------------
// qsum and interleaving for codes supplied by the caller
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) prepare_codes_kernel(const int8_t* __restrict__ codes, int64_t M, int K,
                                                            int8_t* __restrict__ inter, int32_t* __restrict__ qsum,
                                                            uint32_t* __restrict__ status) {
    if (status && blockIdx.x == 0 && threadIdx.x == 0) status[0] = 0;   // this call's status starts clean
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
    if (threadIdx.x == 0 && qsum) qsum[t] = red_sum;
}

int launch_prepare_codes(const int8_t* codes, int64_t M, int64_t K, int8_t* codes_interleaved, int32_t* qsum,
                         uint32_t* status, cudaStream_t stream) {
    if (M == 0) return BWLA_OK;
    ProfScope prof(kProfPrepare, stream);
    prepare_codes_kernel<<<(unsigned)M, 256, 0, stream>>>(codes, M, (int)K, codes_interleaved, qsum, status);
    return after_launch();
}

}  // namespace bwla
