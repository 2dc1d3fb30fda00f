// Microbenchmark: rate of 128-bit shared-memory stores in the access pattern of the operand expansion of the
// tensor-core product (thread r owns the 128-byte row r; its eight 16-byte pieces go to the swizzled positions
// j xor (r mod 8)), for several CTA sizes, with and without the proxy fence that follows a pipeline step.  One CTA per SM;
// bytes per clock per SM from clock64.
#include <cstdio>
#include <cstdlib>
#include <cuda_runtime.h>
#define CK(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { printf("CUDA error %s at %d\n", cudaGetErrorString(e_), __LINE__); exit(1); } } while (0)
constexpr int ITERS = 2048;

__device__ __forceinline__ void st_v4(unsigned addr, unsigned a, unsigned b, unsigned c, unsigned d)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" :: "r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

template <int MODE>     // 0: stores, 1: stores + proxy fence per 8 stores
__global__ void __launch_bounds__(1024, 1) k_rows(unsigned* out, long long* clk, unsigned seed)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    const unsigned r = threadIdx.x;
    const unsigned base = (unsigned)__cvta_generic_to_shared(smem) + r * 128;
    unsigned off[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) off[j] = (unsigned)((j ^ (r & 7)) << 4);
    unsigned v = seed + r;
    __syncthreads();
    long long t0 = clock64();
#pragma unroll 1
    for (int i = 0; i < ITERS; ++i) {
#pragma unroll
        for (int j = 0; j < 8; ++j) st_v4(base + off[j], v + j, v ^ i, v + i, v);
        if (MODE == 1) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    long long t1 = clock64();
    __syncthreads();
    out[blockIdx.x * 1024 + threadIdx.x] = *reinterpret_cast<unsigned*>(smem + r * 128);
    if (threadIdx.x == 0) clk[blockIdx.x] = t1 - t0;
}

template <int MODE>
static void run(const char* name, int threads, int sms, unsigned* out, long long* clk)
{
    CK(cudaFuncSetAttribute(k_rows<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, 1024 * 128));
    for (int rep = 0; rep < 2; ++rep) k_rows<MODE><<<sms, threads, 1024 * 128>>>(out, clk, 12345u);
    CK(cudaDeviceSynchronize());
    long long* h = (long long*)malloc(sizeof(long long) * sms);
    CK(cudaMemcpy(h, clk, sizeof(long long) * sms, cudaMemcpyDeviceToHost));
    long long worst = 0;
    for (int i = 0; i < sms; ++i) if (h[i] > worst) worst = h[i];
    free(h);
    const double bytes = (double)threads * 128.0 * ITERS;
    printf("%-34s %4d threads: %6.1f bytes per clock per SM (%.1f clocks per warp-wide 128-bit access)\n", name, threads,
           bytes / (double)worst, (double)worst / ((double)(threads / 32) * 8.0 * ITERS));
}

int main()
{
    int dev = 0, sms = 0;
    CK(cudaGetDevice(&dev));
    CK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    unsigned* out; long long* clk;
    CK(cudaMalloc(&out, sizeof(unsigned) * 1024 * sms));
    CK(cudaMalloc(&clk, sizeof(long long) * sms));
    const int sizes[4] = {128, 320, 640, 1024};
    for (int s = 0; s < 4; ++s) run<0>("st.shared.v4, swizzled rows", sizes[s], sms, out, clk);
    for (int s = 0; s < 4; ++s) run<1>("the same + fence.proxy.async / 8", sizes[s], sms, out, clk);
    CK(cudaFree(out)); CK(cudaFree(clk));
    return 0;
}
