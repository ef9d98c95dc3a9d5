// Rate probes for the tcgen05 instructions the kernels are built on: how many cycles one SM needs per tcgen05.mma of the
// shapes in use (kind::i8 with the A operand in tensor memory: the binary contraction; kind::f16 from shared memory and
// from tensor memory: the rotation and the low-rank products), issued back to back by one thread, on every SM at once.
// Operands are zero-filled shared memory and whatever tensor memory holds; results are discarded.  Reported per shape:
// cycles per MMA until the last one has completed, cycles per MMA the issuing thread needs for the issue loop alone, and
// the device-wide rate that corresponds to the first figure.
// Build: python -m paper_2605_00422_b200.build --microbench      Run: paper_2605_00422_b200/microbench/umma_rates
#include <cstdio>
#include <cuda_runtime.h>
#include <stdint.h>

#include "umma_ptx.cuh"
#include "umma_wait.cuh"

using namespace bwla;
using namespace bwla::ptx;

constexpr int kABytes = 128 * 128, kBBytes = 256 * 128;
constexpr int kSmem = kABytes + kBBytes + 64 + 1024;

__device__ __forceinline__ void mma_i8_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// KIND 0: i8, A in tensor memory; 1: i8, A in shared memory; 2: f16 (bf16 operands), shared; 3: f16, A in tensor memory;
// 4: i8, A in shared memory, M = 64
template <int KIND>
__global__ void __launch_bounds__(128, 1) probe(int n_cols, int count, long long* issue_cycles, long long* total_cycles,
                                                uint32_t* status) {
    extern __shared__ uint8_t raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* bar = reinterpret_cast<uint64_t*>(smem + kABytes + kBBytes);
    uint32_t* slot = reinterpret_cast<uint32_t*>(bar + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(slot + 1);
    for (int i = threadIdx.x; i < (kABytes + kBBytes) / 16; i += blockDim.x) reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
    if (threadIdx.x == 0) {
        *abort_flag = 0;
        mbar_init(bar, 1);
        fence_barrier_init();
    }
    fence_proxy_async();
    if (threadIdx.x < 32) {
        tmem_alloc(slot, 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *slot;
    if (threadIdx.x == 0) {
        const uint32_t fmt = (KIND < 2 || KIND == 4) ? (2u << 4) : (1u << 4);           // D = s32 / f32
        const uint32_t m_rows = KIND == 4 ? 64u : 128u;
        const uint32_t idesc = fmt | (1u << 7) | (1u << 10) | ((uint32_t)(n_cols >> 3) << 17) | ((m_rows >> 4) << 24);
        const uint32_t a_addr = smem_u32(smem), b_addr = a_addr + kABytes;
        const long long t0 = clock64();
        for (int i = 0; i < count; ++i) {
            const uint32_t j = (uint32_t)i & 3u;
            const uint64_t db = smem_desc_sw128(b_addr, 32 * j);
            if (KIND == 0) mma_i8_ts(tmem_base, tmem_base + 256 + 8 * j, db, idesc, i ? 1u : 0u);
            else if (KIND == 1 || KIND == 4) mma_i8_ss(tmem_base, smem_desc_sw128(a_addr, 32 * j), db, idesc, i ? 1u : 0u);
            else if (KIND == 2) mma_f16_ss(tmem_base, smem_desc_sw128(a_addr, 32 * j), db, idesc, i ? 1u : 0u);
            else mma_f16_ts(tmem_base, tmem_base + 256 + 8 * j, db, idesc, i ? 1u : 0u);
        }
        const long long t1 = clock64();
        tc_commit(bar);
        if (!wait_or_abort(bar, 0, abort_flag)) give_up(status, abort_flag, 0x900);
        const long long t2 = clock64();
        issue_cycles[blockIdx.x] = t1 - t0;
        total_cycles[blockIdx.x] = t2 - t0;
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x < 32) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

template <int KIND>
static int run(const char* name, int m_rows, int k_per_mma, const int* ns, int n_ns, int sms, double ghz, long long* d_issue, long long* d_total,
               uint32_t* d_status) {
    cudaFuncSetAttribute(probe<KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    const int count = 4096;
    long long* h = new long long[2 * sms];
    for (int q = 0; q < n_ns; ++q) {
        const int n = ns[q];
        for (int rep = 0; rep < 2; ++rep) {          // the second run is the one reported
            probe<KIND><<<sms, 128, kSmem>>>(n, count, d_issue, d_total, d_status);
            if (cudaDeviceSynchronize() != cudaSuccess) { printf("%s: launch failed: %s\n", name, cudaGetErrorString(cudaGetLastError())); return 1; }
        }
        uint32_t st = 0;
        cudaMemcpy(&st, d_status, 4, cudaMemcpyDeviceToHost);
        if (st) { printf("%s N=%d: a wait ran out\n", name, n); return 1; }
        cudaMemcpy(h, d_issue, sizeof(long long) * sms, cudaMemcpyDeviceToHost);
        cudaMemcpy(h + sms, d_total, sizeof(long long) * sms, cudaMemcpyDeviceToHost);
        double issue = 0, total = 0;
        for (int i = 0; i < sms; ++i) { issue += (double)h[i]; total += (double)h[sms + i]; }
        issue /= (double)sms * count; total /= (double)sms * count;
        const double ops = 2.0 * m_rows * n * k_per_mma;
        printf("| %s | %d | %.1f | %.1f | %.0f |\n", name, n, total, issue, ops * sms * ghz / total / 1e3);
    }
    delete[] h;
    return 0;
}

int main() {
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, 0) != cudaSuccess) { printf("no device\n"); return 1; }
    const int sms = prop.multiProcessorCount;
    int khz = 0;
    cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, 0);
    const double ghz = khz / 1e6;
    long long *d_issue, *d_total; uint32_t* d_status;
    cudaMalloc(&d_issue, sizeof(long long) * sms);
    cudaMalloc(&d_total, sizeof(long long) * sms);
    cudaMalloc(&d_status, 256);
    cudaMemset(d_status, 0, 256);
    printf("%s, %d SMs, %.3f GHz (attribute clock), 4096 MMAs (M = 128 unless stated) per SM, all SMs at once\n", prop.name, sms, ghz);
    printf("| instruction | N | cycles per MMA (complete) | cycles per MMA (issue loop) | device Tera-op/s at that rate |\n|---|---|---|---|---|\n");
    const int n_i8[] = {16, 32, 64, 128, 256};
    const int n_f16[] = {16, 64, 80, 128, 160, 256};
    int rc = 0;
    rc |= run<0>("kind::i8, K = 32, A in tensor memory", 128, 32, n_i8, 5, sms, ghz, d_issue, d_total, d_status);
    rc |= run<1>("kind::i8, K = 32, A in shared memory", 128, 32, n_i8, 5, sms, ghz, d_issue, d_total, d_status);
    rc |= run<2>("kind::f16 (bf16), K = 16, A in shared memory", 128, 16, n_f16, 6, sms, ghz, d_issue, d_total, d_status);
    rc |= run<3>("kind::f16 (bf16), K = 16, A in tensor memory", 128, 16, n_f16, 6, sms, ghz, d_issue, d_total, d_status);
    const int n_m64[] = {64, 128, 256};
    rc |= run<4>("kind::i8, K = 32, A in shared memory, M = 64", 64, 32, n_m64, 3, sms, ghz, d_issue, d_total, d_status);
    return rc;
}
