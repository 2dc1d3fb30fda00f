// Microbenchmark: how tcgen05.mma (kind::i8, M 128 x N 192 x K 32, both operands in shared memory) and 128-bit
// shared-memory stores share the shared-memory port.  One thread issues MMAs back to back over a fixed operand tile
// while `st_threads` other threads stream stores in the access pattern of the operand expansion (own 128-byte row,
// eight swizzled 16-byte pieces per round) into another region, until the MMAs have completed.  Reported: clocks per
// MMA and store bytes per clock, each alone and together.  One CTA per SM on every SM; every wait is bounded.
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

constexpr int N_MMA = 192;
constexpr int OPERAND_BYTES = (128 + 256) * 128;        // A: 128 rows, B: up to 256 rows of 128 bytes
constexpr int MAX_ROUNDS = 1 << 16;

struct P { int mma_count, st_threads, fence; long long* clk; unsigned long long* rounds; unsigned* err; };

__global__ void __launch_bounds__(1024, 1) mma_with_stores(P p)
{
    extern __shared__ __align__(1024) unsigned char smem[];      // operands (zeros), then one 128-byte row per storing thread
    __shared__ uint64_t bar;
    __shared__ uint32_t tmem_slot;
    __shared__ volatile int mma_done;
    const int tid = threadIdx.x, warp = tid >> 5, nthreads = blockDim.x;
    for (int i = tid; i < OPERAND_BYTES / 16; i += nthreads) reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
    if (tid == 0) {
        mma_done = 0;
        asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(&bar)), "r"(1u) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_u32(&tmem_slot)), "r"(256u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_slot;
    if (tid == 0) {
        const long long t0 = clock64();
        bool ok = true;
        if (p.mma_count > 0) {
            const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N_MMA >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
            const uint64_t adesc = smem_desc(smem_u32(smem)), bdesc = smem_desc(smem_u32(smem) + 128 * 128);
            const uint32_t a_lo = (uint32_t)adesc, b_lo = (uint32_t)bdesc, hi = (uint32_t)(adesc >> 32);
            for (int i = 0; i < p.mma_count; i += 4) {
                const uint32_t first = i >= 4 ? 1u : 0u;
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
                    :: "r"(tmem_base), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(first) : "memory");
            }
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(smem_u32(&bar)) : "memory");
            ok = false;
            for (unsigned i = 0; i < (1u << 22); ++i) if (mbar_try_wait(smem_u32(&bar), 0)) { ok = true; break; }
        } else {
            while (clock64() - t0 < 200000) { }                 // stores alone: a fixed window
        }
        p.clk[blockIdx.x] = clock64() - t0;
        mma_done = 1;
        if (!ok) atomicExch(p.err, 1u);
    } else if (tid >= 32 && tid < 32 + p.st_threads) {
        const unsigned r = (unsigned)(tid - 32);
        const unsigned base = smem_u32(smem) + OPERAND_BYTES + r * 128;
        unsigned off[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) off[j] = (unsigned)((j ^ (r & 7)) << 4);
        unsigned v = 0x22222222u + r;
        int rounds = 0;
        while (rounds < MAX_ROUNDS && !mma_done) {
#pragma unroll
            for (int j = 0; j < 8; ++j)
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" :: "r"(base + off[j]), "r"(v + j), "r"(v ^ rounds), "r"(v), "r"(v + rounds) : "memory");
            if (p.fence) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            ++rounds;
        }
        if (r == 0) p.rounds[blockIdx.x] = (unsigned long long)rounds;
    }
    __syncthreads();
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_base), "r"(256u) : "memory");
}

int main()
{
    int sms = 0; CK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0));
    long long* clk; CK(cudaMalloc(&clk, sms * 8));
    unsigned long long* rounds; CK(cudaMalloc(&rounds, sms * 8));
    unsigned* err; CK(cudaMalloc(&err, 4)); CK(cudaMemset(err, 0, 4));
    const size_t smem = OPERAND_BYTES + 960 * 128;
    CK(cudaFuncSetAttribute(mma_with_stores, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    long long* hc = (long long*)malloc(sms * 8);
    unsigned long long* hr = (unsigned long long*)malloc(sms * 8);
    const int mma_count = 2048;
    for (int fence = 0; fence < 2; ++fence)
        for (int st : {0, 320, 640, 960})
            for (int with_mma = 0; with_mma < 2; ++with_mma) {
                if (!with_mma && st == 0) continue;
                if (fence && st == 0) continue;
                P p{with_mma ? mma_count : 0, st, fence, clk, rounds, err};
                CK(cudaMemset(rounds, 0, sms * 8));
                for (int rep = 0; rep < 2; ++rep) { mma_with_stores<<<sms, 32 + (st > 0 ? st : 0), smem>>>(p); CK(cudaDeviceSynchronize()); }
                CK(cudaMemcpy(hc, clk, sms * 8, cudaMemcpyDeviceToHost));
                CK(cudaMemcpy(hr, rounds, sms * 8, cudaMemcpyDeviceToHost));
                unsigned e; CK(cudaMemcpy(&e, err, 4, cudaMemcpyDeviceToHost));
                double c = 0, r = 0;
                for (int i = 0; i < sms; ++i) { c += (double)hc[i]; r += (double)hr[i]; }
                c /= sms; r /= sms;
                printf("%-14s %3d storing threads%s: ", with_mma ? "MMAs N 192 +" : "no MMAs,", st, fence ? " (+ proxy fence per round)" : "");
                if (with_mma) printf("%6.1f clocks per MMA (alone: 96.6 ideal); ", c / mma_count);
                if (st > 0) printf("stores %6.1f bytes per clock per SM", r * st * 128.0 / c);
                printf("%s\n", e ? "  (a wait ran out)" : "");
            }
    return 0;
}
