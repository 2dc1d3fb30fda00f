// Microbenchmark: how tcgen05.mma (kind::i8, M 128 x N 192 x K 32, both operands in shared memory), 128-bit
// shared-memory stores and the global loads that feed them share the SM's memory pipeline.  One thread issues MMAs back
// to back over a fixed operand tile while `st_threads` other threads do what the expander threads of the product kernel
// do, round after round, until the MMAs have completed: (optionally) load 32 bytes of their own packed row from global
// memory (rows 1 KB apart, L2-resident; as two 16-byte loads or one 256-bit load; 1, 2 or 4 rounds ahead), expand them
// to 4-bit operands with shifts and masks, store the eight 16-byte pieces of their 128-byte shared-memory row at the
// swizzled positions, proxy fence.  Reported: clocks per MMA and store bytes per clock, alone and together.  One CTA per
// SM on every SM; every wait is bounded.
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

// mode bits: 1 proxy fence per round, 2 expansion arithmetic, 4 global loads, 16 two rounds ahead, 64 four rounds ahead,
// 32 one 256-bit load instead of two 128-bit ones
struct P { const uint4* gsrc; int mma_count, st_threads, fence; long long* clk; unsigned long long* rounds; unsigned* err; };

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
        int rounds = 0;
        const uint4* gsrc = p.gsrc + (size_t)(blockIdx.x * 1024 + r) * 64;
        auto expand_store = [&](const uint4& a, const uint4& b) {
            const unsigned w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const unsigned y0 = ((w[j] << 3) & 0x88888888u) | 0x22222222u;
                const unsigned y1 = ((w[j] << 2) & 0x88888888u) | 0x22222222u;
                const unsigned y2 = ((w[j] << 1) & 0x88888888u) | 0x22222222u;
                const unsigned y3 = (w[j] & 0x88888888u) | 0x22222222u;
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" :: "r"(base + off[j]), "r"(y0), "r"(y1), "r"(y2), "r"(y3) : "memory");
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        };
        auto load2 = [&](int step, uint4& a, uint4& b) {
            const uint4* q = gsrc + ((2 * step) & 63);
            if (p.fence & 32) {
                asm volatile("ld.global.cg.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                             : "=r"(a.x), "=r"(a.y), "=r"(a.z), "=r"(a.w), "=r"(b.x), "=r"(b.y), "=r"(b.z), "=r"(b.w) : "l"(q) : "memory");
            } else { a = __ldcg(q); b = __ldcg(q + 1); }
        };
        if (p.fence & 16) {
            // two rounds ahead without register moves: two register sets in turn
            uint4 a0, b0, a1, b1;
            load2(0, a0, b0); load2(1, a1, b1);
            while (rounds < MAX_ROUNDS && !mma_done) {
                { const uint4 a = a0, b = b0; load2(rounds + 2, a0, b0); expand_store(a, b); }
                { const uint4 a = a1, b = b1; load2(rounds + 3, a1, b1); expand_store(a, b); }
                rounds += 2;
            }
        } else if (p.fence & 64) {
            // four rounds ahead
            uint4 a0, b0, a1, b1, a2, b2, a3, b3;
            load2(0, a0, b0); load2(1, a1, b1); load2(2, a2, b2); load2(3, a3, b3);
            while (rounds < MAX_ROUNDS && !mma_done) {
                { const uint4 a = a0, b = b0; load2(rounds + 4, a0, b0); expand_store(a, b); }
                { const uint4 a = a1, b = b1; load2(rounds + 5, a1, b1); expand_store(a, b); }
                { const uint4 a = a2, b = b2; load2(rounds + 6, a2, b2); expand_store(a, b); }
                { const uint4 a = a3, b = b3; load2(rounds + 7, a3, b3); expand_store(a, b); }
                rounds += 4;
            }
        } else if (!(p.fence & 2)) {
            // stores of changing register values only
            const unsigned v = 0x22222222u + r;
            while (rounds < MAX_ROUNDS && !mma_done) {
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" :: "r"(base + off[j]), "r"(v + j), "r"(v ^ rounds), "r"(v), "r"(v + rounds) : "memory");
                if (p.fence & 1) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                ++rounds;
            }
        } else {
            uint4 cur, cur2;
            load2(0, cur, cur2);
            while (rounds < MAX_ROUNDS && !mma_done) {
                uint4 a = cur, b = cur2;
                if (p.fence & 4) load2(rounds + 1, cur, cur2);
                else { a.x += rounds; b.y ^= rounds; }
                expand_store(a, b);
                ++rounds;
            }
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
    uint4* gsrc; CK(cudaMalloc(&gsrc, (size_t)sms * 1024 * 64 * 16)); CK(cudaMemset(gsrc, 0x5a, (size_t)sms * 1024 * 64 * 16));
    struct Mode { int bits; const char* name; };
    const Mode modes[] = {{0, "stores"}, {1, "stores + fence"}, {3, "expansion + fence, no loads"},
                          {7, "2 x 16-byte loads, 1 round ahead"}, {7 + 32, "1 x 32-byte load, 1 round ahead"},
                          {7 + 16, "2 x 16-byte loads, 2 rounds ahead"}, {7 + 16 + 32, "1 x 32-byte load, 2 rounds ahead"},
                          {7 + 64, "2 x 16-byte loads, 4 rounds ahead"}, {7 + 64 + 32, "1 x 32-byte load, 4 rounds ahead"}};
    {
        P p{gsrc, mma_count, 0, 0, clk, rounds, err};
        for (int rep = 0; rep < 2; ++rep) { mma_with_stores<<<sms, 32, smem>>>(p); CK(cudaDeviceSynchronize()); }
        CK(cudaMemcpy(hc, clk, sms * 8, cudaMemcpyDeviceToHost));
        double c = 0;
        for (int i = 0; i < sms; ++i) c += (double)hc[i];
        printf("MMAs N 192 alone: %6.1f clocks per MMA\n", c / sms / mma_count);
    }
    for (const Mode& mode : modes)
        for (int st : {320, 640, 960})
            for (int with_mma = 0; with_mma < 2; ++with_mma) {
                const int fence = mode.bits;
                P p{gsrc, with_mma ? mma_count : 0, st, fence, clk, rounds, err};
                CK(cudaMemset(rounds, 0, sms * 8));
                for (int rep = 0; rep < 2; ++rep) { mma_with_stores<<<sms, 32 + (st > 0 ? st : 0), smem>>>(p); CK(cudaDeviceSynchronize()); }
                CK(cudaMemcpy(hc, clk, sms * 8, cudaMemcpyDeviceToHost));
                CK(cudaMemcpy(hr, rounds, sms * 8, cudaMemcpyDeviceToHost));
                unsigned e; CK(cudaMemcpy(&e, err, 4, cudaMemcpyDeviceToHost));
                double c = 0, r = 0;
                for (int i = 0; i < sms; ++i) { c += (double)hc[i]; r += (double)hr[i]; }
                c /= sms; r /= sms;
                printf("%-36s %3d threads, %-13s ", mode.name, st, with_mma ? "beside MMAs:" : "no MMAs:");
                if (with_mma) printf("%6.1f clocks per MMA; ", c / mma_count);
                if (st > 0) printf("stores %6.1f bytes per clock per SM", r * st * 128.0 / c);
                printf("%s\n", e ? "  (a wait ran out)" : "");
            }
    return 0;
}
