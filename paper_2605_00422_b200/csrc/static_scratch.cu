// bwla_w1ax_linear_static: the whole layer for callers that cannot hand the library a scratch buffer.
//
// bwla_w1ax_linear keeps its intermediates (int8 codes, per-token scales and code sums, the low-rank vector T) in a
// workspace that the caller allocates.  Some callers have no allocator to ask: code that runs between the
// allocation phases of a host framework, a plug-in that was handed only its input and output tensors, a process
// whose memory pool is frozen once serving starts.  For them the same two kernels run here with the workspace
// carved out of a fixed array that lives in the library's own device image.  Nothing is allocated or freed, by
// CUDA or by any library, on any call.
#include <mutex>

#include "bwla_common.cuh"

namespace bwla {

// The built-in scratch.  Every GPU that loads the library holds these 4 MiB until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[BWLA_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
static std::mutex g_static_mutex;
static void* g_static_ptr[kMaxDevices];      // device address of g_static_scratch on each device, once looked up

// In host code the array's name is only a handle for the runtime, not an address a kernel could use: the device
// address has to be asked for, once per device, with that device current.
static int static_scratch_address(void** out) {
    int dev = 0;
    BWLA_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return BWLA_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        void* p = nullptr;
        BWLA_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
        if (!p || (reinterpret_cast<uintptr_t>(p) & 255)) return BWLA_ERR_WORKSPACE;
        g_static_ptr[dev] = p;
    }
    *out = g_static_ptr[dev];
    return BWLA_OK;
}

}  // namespace bwla

using namespace bwla;

extern "C" int bwla_w1ax_linear_static(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, const float* P1, int n1,
                                       const float* P2, int n2, int bits, const uint32_t* packed, const float* alpha,
                                       const float* mu, const void* U_bf16, const void* V_bf16, int r, void* out_bf16,
                                       int64_t N, int64_t ldo, void* stream) {
    // sizes and arguments first: a call that is going to be refused puts nothing on the stream
    const size_t need = bwla_workspace_bytes(M, K, N, r, bits);
    if (need == 0) return BWLA_ERR_INVALID_ARG;
    if (need > (size_t)BWLA_STATIC_SCRATCH_BYTES) return BWLA_ERR_STATIC_SCRATCH;
    // (the scratch pointer is not known yet; any aligned non-null value passes the workspace check)
    int st = validate_linear_call(x_bf16, M, K, ldx, P1, n1, P2, n2, bits, packed, alpha, U_bf16, V_bf16, r, out_bf16, N, ldo,
                                  reinterpret_cast<const void*>((uintptr_t)256), BWLA_STATIC_SCRATCH_BYTES);
    if (st != BWLA_OK) return st;
    if (M == 0 || N == 0) return BWLA_OK;
    void* scratch = nullptr;
    st = static_scratch_address(&scratch);
    if (st != BWLA_OK) return st;
    // The array keeps what the previous call left.  Only the status words have to start at zero (a stale failure
    // flag would make this call skip its work); everything else is written before it is read.
    BWLA_CUDA_TRY(cudaMemsetAsync(scratch, 0, kStatusBytes, (cudaStream_t)stream));
    return bwla_w1ax_linear(x_bf16, M, K, ldx, P1, n1, P2, n2, bits, packed, alpha, mu, U_bf16, V_bf16, r, out_bf16, N,
                            ldo, scratch, BWLA_STATIC_SCRATCH_BYTES, stream);
}
