// Final binarisation in the rotated coordinates (Alg. 2, last step, with Eq. 1-3), offline, once per layer:
//
//   X = W_res (P1 (x) P2)      every row of W_res = W - M goes through the same map as an activation row
//   mu_n = mean_k X_nk,  alpha_n = mean_k |X_nk - mu_n|,  bit_nk = (X_nk - mu_n > 0)
//
// The rotation is the tensor-core kernel of okt_umma.cu, which takes bf16 rows and hands out fp32.  An fp32 row is the
// exact sum of three bf16 terms and the rotation is linear, so fp32 rows are rotated as three passes over their terms
// and the outputs added (small terms first).  The statistics are accumulated in fp64, one block per row.
#include <cuda_bf16.h>

#include "bwla_common.cuh"
#include "prologue_roles.cuh"

namespace bwla {

// fp32 [rows][K] (row stride ldw) -> its three bf16 terms, each [rows][K] dense
__global__ void __launch_bounds__(256) split_rows_kernel(const float* __restrict__ w, int64_t rows, int64_t K, int64_t ldw,
                                                        __nv_bfloat16* __restrict__ t0, __nv_bfloat16* __restrict__ t1,
                                                        __nv_bfloat16* __restrict__ t2) {
    const int64_t total = rows * K;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / K, k = i - r * K;
        __nv_bfloat16 h, m, l;
        split3(w[r * ldw + k], h, m, l);
        t0[i] = h; t1[i] = m; t2[i] = l;
    }
}

// bf16 [rows][K] with an arbitrary row stride -> dense copy (only when the caller's rows cannot be read in place)
__global__ void __launch_bounds__(256) copy_rows_kernel(const __nv_bfloat16* __restrict__ w, int64_t rows, int64_t K, int64_t ldw,
                                                       __nv_bfloat16* __restrict__ out) {
    const int64_t total = rows * K;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / K, k = i - r * K;
        out[i] = w[r * ldw + k];
    }
}

__device__ __forceinline__ double block_sum(double v, double* red) {
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
    __syncthreads();                                  // red may still be read from the call before
    if (lane == 0) red[warp] = v;
    __syncthreads();
    double s = 0.0;
    for (int i = 0; i < nw; ++i) s += red[i];         // the same order in every thread
    return s;
}

// One block per row.  y0, y1, y2: fp32 [rows][K] outputs of the rotation passes (y1, y2 NULL for bf16 input), added
// small terms first.
__global__ void __launch_bounds__(256) binarize_stats_kernel(const float* __restrict__ y0, const float* __restrict__ y1,
                                                            const float* __restrict__ y2, int64_t K, float* __restrict__ mu,
                                                            float* __restrict__ alpha, uint32_t* __restrict__ packed) {
    __shared__ double red[8];
    const int64_t row = blockIdx.x;
    const float* a = y0 + row * K;
    const float* b = y1 ? y1 + row * K : nullptr;
    const float* c = y2 ? y2 + row * K : nullptr;
    auto value = [&](int64_t k) { return b ? (c[k] + b[k]) + a[k] : a[k]; };
    double s = 0.0;
    for (int64_t k = threadIdx.x; k < K; k += blockDim.x) s += (double)value(k);
    const double mean = block_sum(s, red) / (double)K;
    double d = 0.0;
    for (int64_t k = threadIdx.x; k < K; k += blockDim.x) {     // a warp covers one 32-bit word per step
        const double x = (double)value(k) - mean;
        d += fabs(x);
        const uint32_t word = __ballot_sync(0xFFFFFFFFu, x > 0.0);
        if ((threadIdx.x & 31) == 0) packed[row * (K >> 5) + (k >> 5)] = word;
    }
    const double dev = block_sum(d, red) / (double)K;
    if (threadIdx.x == 0) { mu[row] = (float)mean; alpha[row] = (float)dev; }
}

constexpr int kBinarizeRows = 256;     // rows per pass

struct BinarizeLayout { size_t status, prep, terms, y, codes, scales, total; };
static BinarizeLayout binarize_layout(int64_t K) {
    BinarizeLayout l{};
    size_t off = 0;
    l.status = off; off += kStatusBytes;
    l.prep = off;   off += kOktPreparedMax;
    l.terms = off;  off += align_up((size_t)3 * kBinarizeRows * (size_t)K * 2, 256);
    l.y = off;      off += align_up((size_t)3 * kBinarizeRows * (size_t)K * 4, 256);
    l.codes = off;  off += align_up((size_t)kBinarizeRows * (size_t)K, 256);
    l.scales = off; off += align_up((size_t)kBinarizeRows * 4, 256);
    l.total = off;
    return l;
}

size_t binarize_workspace_bytes(int64_t K) { return binarize_layout(K).total; }

int launch_binarize(const void* w, int dtype, int64_t N, int64_t K, int64_t ldw, const float* P1, int n1, const float* P2, int n2,
                    uint32_t* packed, float* alpha, float* mu, void* workspace, cudaStream_t stream) {
    OktGeom geom;
    if (!okt_geometry(n1, n2, &geom) || okt_prepared_bytes(geom) > kOktPreparedMax) return BWLA_ERR_UNSUPPORTED;
    const BinarizeLayout l = binarize_layout(K);
    char* base = (char*)workspace;
    uint32_t* status = (uint32_t*)(base + l.status);
    BWLA_CUDA_TRY(cudaMemsetAsync(status, 0, kStatusBytes, stream));
    int st = launch_prepare_okt(geom, P1, P2, base + l.prep, stream);
    if (st != BWLA_OK) return st;
    const int n_terms = dtype == 0 ? 3 : 1;
    const size_t term_elems = (size_t)kBinarizeRows * (size_t)K;
    __nv_bfloat16* terms = (__nv_bfloat16*)(base + l.terms);
    float* y = (float*)(base + l.y);
    for (int64_t r0 = 0; r0 < N; r0 += kBinarizeRows) {
        const int64_t rows = std::min<int64_t>(kBinarizeRows, N - r0);
        const void* src[3] = {nullptr, nullptr, nullptr};
        int64_t ld = K;
        const int blocks = (int)std::min<int64_t>((rows * K + 255) / 256, 2048);
        if (dtype == 0) {
            split_rows_kernel<<<blocks, 256, 0, stream>>>((const float*)w + r0 * ldw, rows, K, ldw, terms, terms + term_elems,
                                                        terms + 2 * term_elems);
            st = after_launch();
            if (st != BWLA_OK) return st;
            for (int h = 0; h < 3; ++h) src[h] = terms + h * term_elems;
        } else {
            const __nv_bfloat16* rows_in = (const __nv_bfloat16*)w + r0 * ldw;
            if (okt_accepts_x(rows_in, ldw)) { src[0] = rows_in; ld = ldw; }
            else {
                copy_rows_kernel<<<blocks, 256, 0, stream>>>(rows_in, rows, K, ldw, terms);
                st = after_launch();
                if (st != BWLA_OK) return st;
                src[0] = terms;
            }
        }
        for (int h = 0; h < n_terms; ++h) {
            OktProblem pr{(const uint8_t*)(base + l.prep), (int8_t*)(base + l.codes), 0, nullptr, 0, (float*)(base + l.scales), nullptr,
                          y + h * term_elems};
            st = launch_okt(geom, src[h], rows, h == 0 ? ld : K, 8, 0, 1, &pr, nullptr, status, stream);
            if (st != BWLA_OK) return st;
        }
        binarize_stats_kernel<<<(unsigned)rows, 256, 0, stream>>>(y, n_terms == 3 ? y + term_elems : nullptr,
                                                                 n_terms == 3 ? y + 2 * term_elems : nullptr, K, mu + r0, alpha + r0,
                                                                 packed + r0 * (K >> 5));
        st = after_launch();
        if (st != BWLA_OK) return st;
    }
    return BWLA_OK;
}

}  // namespace bwla
