// Instruction-rate probes that decide between the two formulations of the binary contraction at small token counts:
//   * activation bit-planes against packed weight bits on the warp-level 1-bit tensor-core instruction
//     (mma.sync.m16n8k256 .b1 .and.popc: 16 rows x 256 weights x 8 plane columns per instruction), and
//   * the same with plain ALU instructions (lop3 + popc + iadd per 32 weights and plane).
// Each probe runs `iters` dependent-free instructions per warp on every SM with 1..32 warps per SM and reports
// cycles per warp-instruction per SM and the weights (x columns) per clock per SM that rate sustains.
// Build: python -m paper_2605_00422_b200.build --microbench      Run: paper_2605_00422_b200/microbench/issue_rates
#include <cstdio>
#include <cuda_runtime.h>
#include <stdint.h>

__device__ __forceinline__ void mma_b1(int (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k256.row.col.s32.b1.b1.s32.and.popc {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// kind 0: b1 MMA (4 independent accumulators per warp); kind 1: popc chain (and + popc + add, 8 independent chains)
template <int KIND>
__global__ void probe(int iters, uint32_t seed, long long* cycles, int* sink) {
    const uint32_t x = seed * (threadIdx.x + 1);
    long long t0 = 0, t1 = 0;
    if (KIND == 0) {
        int c[4][4] = {};
        uint32_t a[4] = {x, x * 3u, x * 5u, x * 7u};
        __syncthreads();
        t0 = clock64();
        for (int i = 0; i < iters; ++i) {
#pragma unroll
            for (int j = 0; j < 4; ++j) mma_b1(c[j], a, x + j, x ^ (uint32_t)j);
        }
        t1 = clock64();
        int s = 0;
        for (int j = 0; j < 4; ++j) s += c[j][0] + c[j][1] + c[j][2] + c[j][3];
        if (s == 0x7fffffff) *sink = s;
    } else {
        uint32_t acc[8] = {};
        uint32_t w = x;
        __syncthreads();
        t0 = clock64();
        for (int i = 0; i < iters; ++i) {
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[j] += __popc(w & (x + j + i));
        }
        t1 = clock64();
        uint32_t s = 0;
        for (int j = 0; j < 8; ++j) s += acc[j];
        if (s == 0x7fffffffu) *sink = (int)s;
    }
    if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

int main() {
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, 0) != cudaSuccess) { printf("no device\n"); return 1; }
    const int sms = prop.multiProcessorCount;
    long long* d_cycles; int* d_sink;
    cudaMalloc(&d_cycles, sizeof(long long) * sms);
    cudaMalloc(&d_sink, sizeof(int));
    long long* h = new long long[sms];
    printf("device %s, %d SMs\n", prop.name, sms);
    printf("%-28s %6s %14s %22s\n", "probe", "warps", "cycles/instr/SM", "weights x cols /clk/SM");
    const int iters = 4096;
    for (int kind = 0; kind < 2; ++kind) {
        for (int warps = 1; warps <= 32; warps *= 2) {
            for (int rep = 0; rep < 2; ++rep) {   // the first run warms the clocks and the instruction cache
                if (kind == 0) probe<0><<<sms, 32 * warps>>>(iters, 12345u, d_cycles, d_sink);
                else probe<1><<<sms, 32 * warps>>>(iters, 12345u, d_cycles, d_sink);
                cudaDeviceSynchronize();
            }
            cudaMemcpy(h, d_cycles, sizeof(long long) * sms, cudaMemcpyDeviceToHost);
            double mean = 0;
            for (int i = 0; i < sms; ++i) mean += (double)h[i];
            mean /= sms;
            const double instr = (double)iters * (kind == 0 ? 4 : 8) * warps;          // warp-instructions per SM
            const double cyc = mean / instr;
            // one b1 MMA: 16 rows x 256 weights against 8 columns; one popc: 32 lanes x 32 weights against 1 column
            const double work = kind == 0 ? 16.0 * 256.0 * 8.0 : 32.0 * 32.0;
            printf("%-28s %6d %14.2f %22.1f\n", kind == 0 ? "mma.sync b1 m16n8k256" : "and + popc + add", warps, cyc, work / cyc);
        }
    }
    if (cudaGetLastError() != cudaSuccess) { printf("CUDA error\n"); return 1; }
    return 0;
}
