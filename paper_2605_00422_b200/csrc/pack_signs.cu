// Binarisation of rotated/centred weights into packed sign words (Eq. 2-3: Sign(w) = +1 iff w > 0).
#include <cuda_bf16.h>

#include "bwla_common.cuh"

namespace bwla {

template <typename T>
__device__ __forceinline__ bool is_positive(T v);
template <>
__device__ __forceinline__ bool is_positive<float>(float v) { return v > 0.0f; }
template <>
__device__ __forceinline__ bool is_positive<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v) > 0.0f; }

// One warp produces one 32-bit word per step: lane l looks at weight 32*word + l, the ballot is the word
// (LSB-first).  Loads are coalesced (128 B per warp for fp32, 64 B for bf16).
template <typename T>
__global__ void __launch_bounds__(256) pack_signs_kernel(const T* __restrict__ w, int64_t N, int64_t words,
                                                         int64_t ldw, uint32_t* __restrict__ packed) {
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int64_t total = N * words;
    for (int64_t i = warp; i < total; i += nwarps) {
        const int64_t n = i / words, wd = i - n * words;
        const bool pos = is_positive<T>(w[n * ldw + wd * 32 + lane]);
        const uint32_t word = __ballot_sync(0xFFFFFFFFu, pos);
        if (lane == 0) packed[i] = word;
    }
}

// One warp per row: the number of +1 weights minus the number of -1 weights.
__global__ void __launch_bounds__(256) row_sums_kernel(const uint32_t* __restrict__ packed, int64_t N, int64_t words,
                                                       int32_t* __restrict__ rowsum) {
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= N) return;
    int ones = 0;
    for (int64_t w = lane; w < words; w += 32) ones += __popc(packed[row * words + w]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ones += __shfl_xor_sync(0xFFFFFFFFu, ones, o);
    if (lane == 0) rowsum[row] = 2 * ones - (int32_t)(words * 32);
}

int launch_row_sums(const uint32_t* packed, int64_t N, int64_t K, int32_t* rowsum, cudaStream_t stream) {
    if (N == 0) return BWLA_OK;
    ProfScope prof(kProfPack, stream);
    row_sums_kernel<<<(unsigned)((N + 7) / 8), 256, 0, stream>>>(packed, N, K / 32, rowsum);
    return after_launch();
}

int launch_pack_signs(const void* w, int dtype, int64_t N, int64_t K, int64_t ldw, uint32_t* packed,
                      cudaStream_t stream) {
    const int64_t words = K / 32;
    const int64_t total = N * words;
    if (total == 0) return BWLA_OK;
    const int warps_per_block = 8;
    int64_t blocks = (total + warps_per_block - 1) / warps_per_block;
    const int64_t cap = (int64_t)(sm_count() > 0 ? sm_count() : 128) * 16;   // the kernel strides over the rest
    if (blocks > cap) blocks = cap;
    ProfScope prof(kProfPack, stream);
    if (dtype == BWLA_DTYPE_F32)
        pack_signs_kernel<float><<<(unsigned)blocks, 256, 0, stream>>>((const float*)w, N, words, ldw, packed);
    else
        pack_signs_kernel<__nv_bfloat16><<<(unsigned)blocks, 256, 0, stream>>>((const __nv_bfloat16*)w, N, words,
                                                                             ldw, packed);
    return after_launch();
}

}  // namespace bwla
