// Microbenchmark: what an exchange of small tagged words between co-resident CTAs through L2 costs on this GPU
// (the h exchange of the batch-1 recurrent kernel with no compute around it).
//   1. ping-pong between CTA 0 and every other CTA (one thread each): round trip in SM clocks;
//   2. all-to-all: every CTA publishes `upc` 64-bit words {payload, round tag} and polls all words of all CTAs;
//      period per round as a function of the number of CTAs, the word layout (packed / one 128-byte line per producer)
//      and the number of copies of the buffer (a CTA polls copy blockIdx % copies).
// Every wait is bounded; a wait that runs out sets an error word and the CTA leaves.
#include <cstdio>
#include <cstdlib>
#include <cuda_runtime.h>
#include <vector>
#include <algorithm>
#define CK(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { printf("CUDA error %s at %d\n", cudaGetErrorString(e_), __LINE__); exit(1); } } while (0)

__device__ __forceinline__ unsigned long long ldr(const unsigned long long* p) { unsigned long long v; asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory"); return v; }
__device__ __forceinline__ void str(unsigned long long* p, unsigned long long v) { asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" :: "l"(p), "l"(v) : "memory"); }

constexpr unsigned LIMIT = 1u << 16;
constexpr int NT = 256, WPT = 4;

__global__ void __launch_bounds__(32, 1) pingpong(unsigned long long* w, int partner, int rounds, long long* out, unsigned* err)
{
    extern __shared__ unsigned char pad[];             // large request: one CTA per SM
    if (threadIdx.x != 0 || (blockIdx.x != 0 && (int)blockIdx.x != partner)) return;
    const bool first = blockIdx.x == 0;
    const long long t0 = clock64();
    for (int t = 1; t <= rounds; ++t) {
        unsigned spins = 0;
        if (first) {
            str(w, (unsigned long long)t);
            while (ldr(w + 32) != (unsigned long long)t) if (++spins > LIMIT) { atomicExch(err, 1u); return; }
        } else {
            while (ldr(w) != (unsigned long long)t) if (++spins > LIMIT) { atomicExch(err, 1u); return; }
            str(w + 32, (unsigned long long)t);
        }
    }
    if (first) out[partner] = (clock64() - t0) / rounds;
}

struct P { unsigned long long* hx; int H, upc, copies, rounds, stride; long long* out; unsigned* err; };

// every CTA publishes its own upc words (`stride` words apart per producer) and waits for everybody's: nobody can be more
// than one round ahead of the slowest CTA, so two buffers alternating by round parity are enough
__global__ void __launch_bounds__(NT, 1) all_to_all(P p)
{
    extern __shared__ unsigned char pad[];
    const int tid = threadIdx.x;
    const int my_copy = blockIdx.x % p.copies;
    const size_t copy_words = (size_t)gridDim.x * p.stride;
    const long long t0 = clock64();
    for (int t = 1; t <= p.rounds; ++t) {
        const unsigned long long word = ((unsigned long long)t << 32) | 7u;
        for (int m = tid; m < p.upc * p.copies; m += NT) {
            const int ul = m % p.upc, cp = m / p.upc;
            if ((int)blockIdx.x * p.upc + ul < p.H)
                str(p.hx + ((size_t)(t & 1) * p.copies + cp) * copy_words + (size_t)blockIdx.x * p.stride + ul, word);
        }
        const unsigned long long* src = p.hx + ((size_t)(t & 1) * p.copies + my_copy) * copy_words;
        const unsigned long long* addr[WPT];
        unsigned pending = 0;
#pragma unroll
        for (int j = 0; j < WPT; ++j) {
            const int u = j * NT + tid;
            addr[j] = src + (size_t)(u / p.upc) * p.stride + (u % p.upc);
            if (u < p.H) pending |= 1u << j;
        }
        unsigned spins = 0;
        while (pending) {
#pragma unroll
            for (int j = 0; j < WPT; ++j)
                if (((pending >> j) & 1u) && (unsigned)(ldr(addr[j]) >> 32) == (unsigned)t) pending &= ~(1u << j);
            if (++spins > LIMIT) break;
        }
        if (__syncthreads_or(pending != 0)) { if (tid == 0) atomicExch(p.err, 1u); return; }
    }
    if (tid == 0) p.out[blockIdx.x] = (clock64() - t0) / p.rounds;
}

int main()
{
    int sms = 0; CK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0));
    unsigned long long* buf; CK(cudaMalloc(&buf, 16 << 20));
    long long* out; CK(cudaMalloc(&out, 8 * 1024)); unsigned* err; CK(cudaMalloc(&err, 4096)); CK(cudaMemset(err, 0, 4096));
    std::vector<long long> h(1024);
    const size_t big = 120 * 1024;                      // one CTA per SM
    const int rounds = 2000;
    CK(cudaFuncSetAttribute(pingpong, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)big));
    CK(cudaFuncSetAttribute(all_to_all, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)big));

    for (int p = 1; p < sms; ++p) {
        CK(cudaMemset(buf, 0, 4096));
        void* args[] = {&buf, &p, (void*)&rounds, &out, &err};
        CK(cudaLaunchCooperativeKernel((void*)pingpong, dim3(sms), dim3(32), args, big, 0));
        CK(cudaDeviceSynchronize());
    }
    CK(cudaMemcpy(h.data(), out, sms * 8, cudaMemcpyDeviceToHost));
    {
        std::vector<long long> v(h.begin() + 1, h.begin() + sms); std::sort(v.begin(), v.end());
        printf("ping-pong round trip, CTA 0 <-> CTA p, SM clocks: min %lld  quartile %lld  median %lld  quartile %lld  max %lld\n",
               v[0], v[v.size() / 4], v[v.size() / 2], v[3 * v.size() / 4], v.back());
    }
    auto run = [&](int G, int upc, int copies, int stride) {
        CK(cudaMemset(buf, 0, 16 << 20));
        P p{buf, G * upc, upc, copies, rounds, stride, out, err};
        if (p.H > NT * WPT) return;
        void* args[] = {&p};
        CK(cudaLaunchCooperativeKernel((void*)all_to_all, dim3(G), dim3(NT), args, big, 0));
        CK(cudaDeviceSynchronize());
        CK(cudaMemcpy(h.data(), out, G * 8, cudaMemcpyDeviceToHost));
        unsigned e; CK(cudaMemcpy(&e, err, 4, cudaMemcpyDeviceToHost));
        long long mx = 0; for (int i = 0; i < G; ++i) mx = std::max(mx, h[i]);
        printf("all-to-all: %3d CTAs x %d words, %2d copies, %2d words between producers -> %5lld clocks per round%s\n", G, upc, copies, stride, mx, e ? " (a wait ran out)" : "");
    };
    const int upc = 6;                                  // words per producer (148 x 6 = 888 words in all)
    for (int G : {2, 8, 32, 64, sms}) { run(G, upc, 1, upc); run(G, upc, 8, upc); }
    for (int copies : {1, 4, 8}) run(sms, upc, copies, 16);
    run(sms, 1, 1, 1); run(sms, 1, 1, 16);
    return 0;
}
