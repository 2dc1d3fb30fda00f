// Microbenchmark: pace of tcgen05.mma.kind::i8 (M = 128, K = 32, both operands in shared memory, 128-byte swizzle, K-major)
// as the product kernel issues it: one thread issues `count` MMAs into one accumulator (or two in turn), commits, and
// waits for the commit.  SM clocks per MMA as a function of N, with and without a second accumulator.  One CTA per SM
// on every SM, so that the figure holds with the whole GPU busy.  Operands are zeros (the pace does not depend on data).
#include <cstdio>
#include <cstdlib>
#include <cstdint>
#include <cuda_runtime.h>
#define CK(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { printf("CUDA error %s at %d\n", cudaGetErrorString(e_), __LINE__); exit(1); } } while (0)

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr)
{
    return (uint64_t)((addr >> 4) & 0x3fffu) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t done;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}"
                 : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done != 0;
}

struct P { int n_mma, count, two_acc; long long* clk; unsigned* err; };

__global__ void __launch_bounds__(128, 1) mma_rate(P p)
{
    extern __shared__ __align__(1024) unsigned char smem[];      // A: 128 rows x 128 bytes, B: 256 rows x 128 bytes, zeros
    __shared__ uint64_t bar;
    __shared__ uint32_t tmem_slot;
    const int tid = threadIdx.x, warp = tid >> 5;
    for (int i = tid; i < (128 + 256) * 128 / 16; i += 128) reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(&bar)), "r"(1u) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_u32(&tmem_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_slot;
    bool ok = true;
    if (tid == 0) {
        const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.n_mma >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
        const uint64_t adesc = smem_desc(smem_u32(smem)), bdesc = smem_desc(smem_u32(smem) + 128 * 128);
        const long long t0 = clock64();
        // four MMAs per iteration (the four K slices of a swizzled row), descriptors rebuilt from their low words inside one
        // block, as the product kernel does it: a dozen instructions of the issuing thread per four MMAs
        const uint32_t a_lo = (uint32_t)adesc, b_lo = (uint32_t)bdesc, hi = (uint32_t)(adesc >> 32);
        for (int i = 0; i < p.count; i += 4) {
            const uint32_t acc = tmem_base + ((p.two_acc && (i & 4)) ? 256u : 0u);
            const uint32_t first = i >= (p.two_acc ? 8 : 4) ? 1u : 0u;
            asm volatile(
                "{\n\t.reg .pred p, q;\n\t.reg .b64 da, db;\n\t.reg .b32 al, bl;\n\t"
                "setp.ne.b32 p, %5, 0;\n\tsetp.eq.b32 q, %5, %5;\n\t"
                "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
                "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %4, p;\n\t"
                "add.u32 al, %1, 2;\n\tadd.u32 bl, %2, 2;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t"
                "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %4, q;\n\t"
                "add.u32 al, %1, 4;\n\tadd.u32 bl, %2, 4;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t"
                "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %4, q;\n\t"
                "add.u32 al, %1, 6;\n\tadd.u32 bl, %2, 6;\n\tmov.b64 da, {al, %3};\n\tmov.b64 db, {bl, %3};\n\t"
                "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %4, q;\n\t}"
                :: "r"(acc), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(first) : "memory");
        }
        const long long t1 = clock64();
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(smem_u32(&bar)) : "memory");
        ok = false;
        for (unsigned i = 0; i < (1u << 22); ++i) if (mbar_try_wait(smem_u32(&bar), 0)) { ok = true; break; }
        const long long t2 = clock64();
        p.clk[blockIdx.x * 2] = t1 - t0;
        p.clk[blockIdx.x * 2 + 1] = t2 - t0;
        if (!ok) atomicExch(p.err, 1u);
    }
    __syncthreads();
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_base), "r"(512u) : "memory");
}

int main()
{
    int sms = 0; CK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0));
    long long* clk; CK(cudaMalloc(&clk, sms * 16)); unsigned* err; CK(cudaMalloc(&err, 4)); CK(cudaMemset(err, 0, 4));
    const size_t smem = (128 + 256) * 128 + 1024;
    CK(cudaFuncSetAttribute(mma_rate, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    long long* h = (long long*)malloc(sms * 16);
    for (int two = 0; two < 2; ++two)
        for (int n : {48, 96, 192, 256}) {
            P p{n, 512, two, clk, err};
            for (int rep = 0; rep < 2; ++rep) { mma_rate<<<sms, 128, smem>>>(p); CK(cudaDeviceSynchronize()); }
            CK(cudaMemcpy(h, clk, sms * 16, cudaMemcpyDeviceToHost));
            unsigned e; CK(cudaMemcpy(&e, err, 4, cudaMemcpyDeviceToHost));
            long long issue = 0, done = 0; for (int i = 0; i < sms; ++i) { issue = h[2 * i] > issue ? h[2 * i] : issue; done = h[2 * i + 1] > done ? h[2 * i + 1] : done; }
            printf("M 128 x N %3d x K 32, %s: %6.1f clocks per MMA until the commit arrives (issue alone %5.1f); ideal at 8192 MAC/clk: %5.1f%s\n",
                   n, two ? "two accumulators in turn" : "one accumulator         ", done / 512.0, issue / 512.0, 128.0 * n * 32 / 8192, e ? "  (a wait ran out)" : "");
        }
    return 0;
}
