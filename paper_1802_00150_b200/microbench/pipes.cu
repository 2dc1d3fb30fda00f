// Microbenchmark: issue rates per SM of the candidate inner operations of the binary product on sm_100a:
// POPC, LOP3, mma.sync b1 (AND.POPC / XOR.POPC, m16n8k256), mma.sync s8 (m16n8k32).  One CTA of 1024 threads per SM,
// independent accumulator chains per thread, SM clocks from clock64.
#include <cstdio>
#include <cstdlib>
#include <cuda_runtime.h>
#define CK(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { printf("CUDA error %s at %d\n", cudaGetErrorString(e_), __LINE__); exit(1); } } while (0)
constexpr int ITERS = 4096;

__global__ void __launch_bounds__(1024, 1) k_popc(unsigned* out, long long* clk, unsigned seed)
{
    unsigned a0 = seed + threadIdx.x, a1 = a0 * 3, a2 = a0 * 5, a3 = a0 * 7, s0 = 0, s1 = 0, s2 = 0, s3 = 0;
    __syncthreads();
    long long t0 = clock64();
#pragma unroll 1
    for (int i = 0; i < ITERS; ++i) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            s0 += __popc(a0 ^ s3); s1 += __popc(a1 ^ s0); s2 += __popc(a2 ^ s1); s3 += __popc(a3 ^ s2);
        }
    }
    long long t1 = clock64();
    out[blockIdx.x * 1024 + threadIdx.x] = s0 + s1 + s2 + s3;
    if (threadIdx.x == 0) clk[blockIdx.x] = t1 - t0;
}
// 16 popc + 16 xor(lop3) + 16 add per inner iteration per thread

__global__ void __launch_bounds__(1024, 1) k_lop3(unsigned* out, long long* clk, unsigned seed)
{
    unsigned a0 = seed + threadIdx.x, a1 = a0 * 3, a2 = a0 * 5, a3 = a0 * 7, b = seed * 11, c = seed * 13;
    __syncthreads();
    long long t0 = clock64();
#pragma unroll 1
    for (int i = 0; i < ITERS; ++i) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(a0) : "r"(b), "r"(c));
            asm volatile("lop3.b32 %0, %0, %1, %2, 0xE8;" : "+r"(a1) : "r"(b), "r"(c));
            asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(a2) : "r"(b), "r"(c));
            asm volatile("lop3.b32 %0, %0, %1, %2, 0xE8;" : "+r"(a3) : "r"(b), "r"(c));
        }
    }
    long long t1 = clock64();
    out[blockIdx.x * 1024 + threadIdx.x] = a0 + a1 + a2 + a3;
    if (threadIdx.x == 0) clk[blockIdx.x] = t1 - t0;
}

template <int OP>   // 0: b1 and.popc, 1: b1 xor.popc, 2: s8
__global__ void __launch_bounds__(1024, 1) k_mma(unsigned* out, long long* clk, unsigned seed)
{
    unsigned a[4] = {seed, seed * 3, seed * 5, seed * 7}, b[2] = {seed * 11, seed * 13};
    int c0[4] = {0, 0, 0, 0}, c1[4] = {0, 0, 0, 0};
    __syncthreads();
    long long t0 = clock64();
#pragma unroll 1
    for (int i = 0; i < ITERS; ++i) {
        if (OP == 0) {
            asm volatile("mma.sync.aligned.m16n8k256.row.col.s32.b1.b1.s32.and.popc {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                         : "+r"(c0[0]), "+r"(c0[1]), "+r"(c0[2]), "+r"(c0[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
            asm volatile("mma.sync.aligned.m16n8k256.row.col.s32.b1.b1.s32.and.popc {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                         : "+r"(c1[0]), "+r"(c1[1]), "+r"(c1[2]), "+r"(c1[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
        } else if (OP == 1) {
            asm volatile("mma.sync.aligned.m16n8k256.row.col.s32.b1.b1.s32.xor.popc {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                         : "+r"(c0[0]), "+r"(c0[1]), "+r"(c0[2]), "+r"(c0[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
            asm volatile("mma.sync.aligned.m16n8k256.row.col.s32.b1.b1.s32.xor.popc {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                         : "+r"(c1[0]), "+r"(c1[1]), "+r"(c1[2]), "+r"(c1[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
        } else {
            asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                         : "+r"(c0[0]), "+r"(c0[1]), "+r"(c0[2]), "+r"(c0[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
            asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                         : "+r"(c1[0]), "+r"(c1[1]), "+r"(c1[2]), "+r"(c1[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
        }
    }
    long long t1 = clock64();
    out[blockIdx.x * 1024 + threadIdx.x] = c0[0] + c0[1] + c0[2] + c0[3] + c1[0] + c1[1] + c1[2] + c1[3];
    if (threadIdx.x == 0) clk[blockIdx.x] = t1 - t0;
}

int main()
{
    int sms = 0; CK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0));
    unsigned* out; CK(cudaMalloc(&out, sms * 1024 * 4)); long long* clk; CK(cudaMalloc(&clk, sms * 8));
    long long* h = (long long*)malloc(sms * 8);
    auto report = [&](const char* name, double ops_per_thread_iter, const char* unit) {
        CK(cudaDeviceSynchronize()); CK(cudaMemcpy(h, clk, sms * 8, cudaMemcpyDeviceToHost));
        double worst = 0; for (int i = 0; i < sms; ++i) worst = h[i] > worst ? h[i] : worst;
        printf("%-28s %8.1f %s per clock per SM (%.0f clocks for %d iterations, 1024 threads)\n", name,
               ops_per_thread_iter * ITERS * 1024 / worst, unit, worst, ITERS);
    };
    for (int rep = 0; rep < 2; ++rep) {
        k_popc<<<sms, 1024>>>(out, clk, 12345u); report("POPC (+ XOR + ADD each)", 16, "popc");
        k_lop3<<<sms, 1024>>>(out, clk, 12345u); report("LOP3", 16, "lop3");
        k_mma<0><<<sms, 1024>>>(out, clk, 12345u); report("mma.sync b1 AND.POPC k256", 2.0 * 16 * 8 * 256 / 32, "bit-MAC");
        k_mma<1><<<sms, 1024>>>(out, clk, 12345u); report("mma.sync b1 XOR.POPC k256", 2.0 * 16 * 8 * 256 / 32, "bit-MAC");
        k_mma<2><<<sms, 1024>>>(out, clk, 12345u); report("mma.sync s8 k32", 2.0 * 16 * 8 * 32 / 32, "MAC");
    }
    return 0;
}
