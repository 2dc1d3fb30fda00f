// Batched binary matrix product on the 5th-generation tensor cores (tcgen05.mma kind::i8, accumulators
// in tensor memory), in the stacked form of Fig. 3, right: the k_w planes of the weight rows of a tile are
// the M rows of one integer matrix product, the k_a planes of the activation vectors its N columns, the
// packed bit positions its K dimension; the k_w x k_a partials of every (row, vector) pair are folded
// with the row-wise coefficients afterwards (Sec. 4), and for the cells the gate arithmetic of Eq. 6 /
// the GRU follows in the same kernel.
//
// The planes stay bit-packed in global memory.  A CTA expands the bits of its tile into signed bytes in
// shared memory: bit 1 -> -64, bit 0 -> +64 on both operands, so a byte product is 4096 * (+-1 * +-1) and a
// 32-bit accumulator holds 4096 * (dot of the +-1 vectors); pad positions (0 in both operands) add one
// each and are subtracted again.  Expanding costs one shift and one logic operation per four bytes:
// output register s of a 32-bit word keeps bits s, s + 8, s + 16, s + 24 in its four bytes, i.e. the K
// positions inside a word are permuted, identically for both operands, which a dot product does not see.
//
// Shared-memory operand layout: K-major, no swizzle, 8-row x 16-byte core matrices, stored as
// [16-byte K chunk][group of 8 rows][row][16 bytes]; one MMA instruction consumes K = 32 bytes = the two
// chunks of one packed word.  Expansion of K stage s + 1 (all threads, generic-proxy stores, then a
// proxy fence) overlaps the asynchronous MMAs of stage s; an mbarrier per buffer, signalled by
// tcgen05.commit, says when a buffer may be overwritten.  Every wait is bounded: when one runs out the CTA
// records the failure in a status word, skips its stores, frees its tensor memory and returns.
#include "amq_common.cuh"

namespace amq {

namespace {

constexpr int TC_THREADS = 256;
constexpr int TILE_M = 128;                 // stacked weight plane-rows per CTA (= TMEM lanes)
constexpr int STAGE_WORDS = 8;              // packed words of K per pipeline stage (256 bit positions)
constexpr int A_LBO = TILE_M / 8 * 128;     // bytes between 16-byte K chunks of the A tile
constexpr int A_STAGE_BYTES = STAGE_WORDS * 2 * A_LBO;
constexpr unsigned WAIT_LIMIT = 1u << 22;   // polls of an mbarrier before giving up

__device__ uint32_t g_tc_status;            // nonzero after a bounded wait ran out (sticky until read)

struct TcParams {
    GemmArgs a;
    int gates;      // 1 plain, 4 LSTM, 3 GRU
    int units;      // plain: m; cells: H
    int UT;         // units per tile
    int TB;         // batch entries per tile (multiple of 16)
    int nseg;       // 1, or 2 for the GRU (columns [0,I) and [I,n))
    int wpr;
    int n_mma;      // TB * k_a: N of the MMA, multiple of 16, <= 256
    int tmem_cols;  // power of two >= nseg * n_mma
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done != 0;
}

// bounded wait; false when it ran out
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    for (unsigned i = 0; i < WAIT_LIMIT; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}

// K-major, no swizzle: start address, leading (K chunk) byte offset, stride (8-row group) byte offset
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo)
{
    return (uint64_t)((addr >> 4) & 0x3fffu) | ((uint64_t)((lbo >> 4) & 0x3fffu) << 16) |
           ((uint64_t)((sbo >> 4) & 0x3fffu) << 32) | (1ull << 46);
}

__device__ __forceinline__ void mma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        :: "r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

__device__ __forceinline__ void mma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, int (&v)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
}

// 128 packed bits of one plane-row -> 128 signed bytes (-64 for bit 1, +64 for bit 0), written as eight
// 16-byte K chunks `lbo` bytes apart starting at `dst`
__device__ __forceinline__ void expand_store(const uint4& v, unsigned char* dst, int lbo)
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        uint32_t y[8];
#pragma unroll
        for (int s = 0; s < 8; ++s) y[s] = ((w[q] << (7 - s)) & 0x80808080u) ^ 0x40404040u;
        *reinterpret_cast<uint4*>(dst + (2 * q) * lbo) = make_uint4(y[0], y[1], y[2], y[3]);
        *reinterpret_cast<uint4*>(dst + (2 * q + 1) * lbo) = make_uint4(y[4], y[5], y[6], y[7]);
    }
}

__device__ __forceinline__ float logistic(float v) { return 1.0f / (1.0f + __expf(-v)); }

template <int KA>
__global__ void __launch_bounds__(TC_THREADS, 1)
bgemm_tc_kernel(TcParams p)
{
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    const GemmArgs& a = p.a;
    const int k_w = a.k_w;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int TM = p.UT * p.gates;                  // weight rows of the tile
    const int TMp = TM * k_w;                       // plane-rows in use (<= 128)
    const int n_mma = p.n_mma;
    const int b_lbo = n_mma * 16;                   // bytes between K chunks of the B tile
    const int stage_bytes = A_STAGE_BYTES + STAGE_WORDS * 2 * b_lbo;
    const int u0 = blockIdx.x * p.UT, b0 = blockIdx.y * p.TB;

    unsigned char* stage_base = smem_raw;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_raw + 2 * stage_bytes);      // [2] buffer-free barriers
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2);

    if (tid == 0) {
        mbar_init(smem_u32(&bars[0]), 1);
        mbar_init(smem_u32(&bars[1]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     :: "r"(smem_u32(tmem_slot)), "r"((uint32_t)p.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    // ---- expansion roles: per stage a thread expands one 128-bit chunk of an A row and two of a B row ----
    const int a_row = tid & (TILE_M - 1), a_half = tid >> 7;        // A: row, which of the two chunks of the stage
    const uint32_t* a_src = nullptr;
    if (a_row < TMp) {
        const int l = a_row / k_w, i = a_row - l * k_w;
        const int u = u0 + l / p.gates, gate = l % p.gates;
        if (u < p.units) a_src = a.Wcodes + (((size_t)gate * p.units + u) * k_w + i) * p.wpr;
    }
    const uint32_t* b_src = nullptr;                                // B: row tid (stacked activation plane)
    if (tid < n_mma) {
        const int b = b0 + tid / KA, j = tid % KA;
        if (b < a.batch) b_src = a.xcodes + ((size_t)b * KA + j) * p.wpr;
    }
    const int a_off = (a_row >> 3) * 128 + (a_row & 7) * 16;
    const int b_off = (tid >> 3) * 128 + (tid & 7) * 16;

    const int CH = p.wpr >> 2;                                      // 128-bit chunks along K
    const int stages = (CH + 1) >> 1;
    const int split_word = (p.nseg == 2) ? (a.I >> 5) : p.wpr;      // first word of the second column segment
    const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n_mma >> 3) << 17) | ((uint32_t)(TILE_M >> 4) << 24);

    auto load_a = [&](int s) -> uint4 {
        const int c = 2 * s + a_half;
        return (a_src && c < CH) ? __ldg(reinterpret_cast<const uint4*>(a_src) + c) : make_uint4(0, 0, 0, 0);
    };
    auto load_b = [&](int s, int h) -> uint4 {
        const int c = 2 * s + h;
        return (b_src && c < CH) ? __ldg(reinterpret_cast<const uint4*>(b_src) + c) : make_uint4(0, 0, 0, 0);
    };

    uint4 va = load_a(0), vb0 = load_b(0, 0), vb1 = load_b(0, 1);
    bool ok = true;
    for (int s = 0; s < stages; ++s) {
        const int buf = s & 1;
        unsigned char* sa = stage_base + buf * stage_bytes;
        unsigned char* sb = sa + A_STAGE_BYTES;
        // the MMAs that read this buffer two stages ago must have completed
        if (s >= 2) ok = mbar_wait(smem_u32(&bars[buf]), (uint32_t)(((s >> 1) + 1) & 1));
        if (__syncthreads_or(!ok)) { ok = false; break; }          // uniform: every thread leaves the loop

        const uint4 ca = va, cb0 = vb0, cb1 = vb1;
        if (s + 1 < stages) { va = load_a(s + 1); vb0 = load_b(s + 1, 0); vb1 = load_b(s + 1, 1); }
        expand_store(ca, sa + a_off + (a_half * 8) * A_LBO, A_LBO);
        if (tid < n_mma) {
            expand_store(cb0, sb + b_off, b_lbo);
            expand_store(cb1, sb + b_off + 8 * b_lbo, b_lbo);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // generic-proxy stores -> async proxy
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        if (tid == 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t sa_addr = smem_u32(sa), sb_addr = smem_u32(sb);
            for (int q = 0; q < STAGE_WORDS; ++q) {
                const int word = s * STAGE_WORDS + q;
                if (word >= p.wpr) break;
                const int seg = word >= split_word ? 1 : 0;
                const uint32_t accumulate = (word != 0 && word != split_word) ? 1u : 0u;
                mma_i8(tmem_base + seg * n_mma,
                       smem_desc(sa_addr + q * 2 * A_LBO, A_LBO, 128),
                       smem_desc(sb_addr + q * 2 * b_lbo, b_lbo, 128), idesc, accumulate);
            }
            mma_commit(smem_u32(&bars[buf]));
        }
    }
    // all MMAs done: the commit of the last stage covers every earlier one
    if (ok) {
        const int last = stages - 1;
        ok = mbar_wait(smem_u32(&bars[last & 1]), (uint32_t)((last >> 1) & 1));
    }
    if (__syncthreads_or(!ok)) {
        // give the tensor core time to drain what was issued, then release tensor memory and leave
        if (tid == 0) atomicExch(&g_tc_status, 1u);
        __nanosleep(1000000);
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        if (warp == 0)
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_base), "r"((uint32_t)p.tmem_cols) : "memory");
        return;
    }
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");

    // ---- epilogue 1: tensor memory -> registers -> partial products in shared memory ----
    // thread = plane-row (lane of tensor memory); warps 0-3 take the lower half of the batch entries of the
    // tile, warps 4-7 the upper half, 16 entries (16 * KA columns) at a time
    float* Yt = reinterpret_cast<float*>(smem_raw);                 // [nseg][128][TB + 1], reuses the stage buffers
    const int ldy = p.TB + 1;
    const int pr = (warp & 3) * 32 + lane;
    const int pad = p.wpr * 32 - a.n;                               // pad positions, all in the last segment
    {
        const int l = pr / k_w, i = pr - l * k_w;
        const int u = u0 + l / p.gates, gate = l % p.gates;
        const bool row_ok = pr < TMp && u < p.units;
        const size_t row = (size_t)gate * p.units + u;
        const float alpha = (row_ok && a.epilogue != EPI_DOTS) ? __ldg(a.Walpha + row * k_w + i) : 0.0f;
        const int groups = p.TB >> 4, half = (groups + 1) >> 1;
        const int g_lo = (warp < 4) ? 0 : half, g_hi = (warp < 4) ? half : groups;
        for (int seg = 0; seg < p.nseg; ++seg) {
            const int corr = (seg == p.nseg - 1) ? pad : 0;
            const int len = (p.nseg == 2) ? (seg == 0 ? a.I : a.n - a.I) : a.n;
            (void)len;
            for (int g = g_lo; g < g_hi; ++g) {
                int acc[KA][16];
#pragma unroll
                for (int c = 0; c < KA; ++c)
                    tmem_ld16(tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(seg * n_mma + (g * KA + c) * 16), acc[c]);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                    const int bb = g * 16 + e, b = b0 + bb;
                    float y = 0.0f;
#pragma unroll
                    for (int j = 0; j < KA; ++j) {
                        const int col = e * KA + j;                  // compile-time position inside the group
                        const int D = (acc[col >> 4][col & 15] >> 12) - corr;
                        if (a.epilogue == EPI_DOTS) {
                            if (row_ok && b < a.batch)
                                a.D[(((size_t)b * a.m + row) * k_w + i) * KA + j] = D;
                        } else {
                            const float be = (b < a.batch) ? __ldg(a.xbeta + (size_t)b * KA + j) : 0.0f;
                            y += be * (float)D;
                        }
                    }
                    if (a.epilogue != EPI_DOTS) Yt[((size_t)seg * TILE_M + pr) * ldy + bb] = alpha * y;
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_base), "r"((uint32_t)p.tmem_cols) : "memory");
    if (a.epilogue == EPI_DOTS) return;

    // ---- epilogue 2: sum the k_w planes of each weight row, bias, gates ----
    const int TB = p.TB;
    auto pre = [&](int seg, int l, int bb) -> float {
        float s = 0.0f;
        for (int i = 0; i < k_w; ++i) s += Yt[((size_t)seg * TILE_M + l * k_w + i) * ldy + bb];
        return s;
    };
    if (a.epilogue == EPI_Y) {
        for (int idx = tid; idx < TM * TB; idx += TC_THREADS) {
            const int bb = idx / TM, l = idx - bb * TM;              // consecutive threads -> consecutive rows
            const int row = u0 + l, b = b0 + bb;
            if (row < a.m && b < a.batch)
                a.y[(size_t)b * a.ldy + row] = pre(0, l, bb) + (a.bias ? __ldg(a.bias + row) : 0.0f);
        }
    } else if (a.epilogue == EPI_LSTM) {
        const int H = a.H;
        for (int idx = tid; idx < p.UT * TB; idx += TC_THREADS) {
            const int bb = idx / p.UT, ul = idx - bb * p.UT;
            const int u = u0 + ul, b = b0 + bb;
            if (u < H && b < a.batch) {
                float g4[4];
#pragma unroll
                for (int g = 0; g < 4; ++g) g4[g] = pre(0, ul * 4 + g, bb) + (a.bias ? __ldg(a.bias + g * H + u) : 0.0f);
                const float ig = logistic(g4[0]), fg = logistic(g4[1]), og = logistic(g4[2]);
                const float gg = tanhf(g4[3]);
                const size_t o = (size_t)b * H + u;
                const float c = fg * a.c_in[o] + ig * gg;
                a.c_out[o] = c;
                a.h_out[o] = og * tanhf(c);
            }
        }
    } else {    // EPI_GRU
        const int H = a.H;
        for (int idx = tid; idx < p.UT * TB; idx += TC_THREADS) {
            const int bb = idx / p.UT, ul = idx - bb * p.UT;
            const int u = u0 + ul, b = b0 + bb;
            if (u < H && b < a.batch) {
                float px[3], ph[3];
#pragma unroll
                for (int g = 0; g < 3; ++g) { px[g] = pre(0, ul * 3 + g, bb); ph[g] = pre(1, ul * 3 + g, bb); }
                const float br = a.bias ? __ldg(a.bias + u) : 0.0f, bz = a.bias ? __ldg(a.bias + H + u) : 0.0f;
                const float bnx = a.bias ? __ldg(a.bias + 2 * H + u) : 0.0f;
                const float bnh = a.bias ? __ldg(a.bias + 3 * H + u) : 0.0f;
                const float rg = logistic(px[0] + ph[0] + br);
                const float zg = logistic(px[1] + ph[1] + bz);
                const float cand = tanhf(px[2] + bnx + rg * (ph[2] + bnh));
                const size_t o = (size_t)b * H + u;
                a.h_out[o] = (1.0f - zg) * cand + zg * a.h_in[o];
            }
        }
    }
}

struct TcPlan {
    TcParams p;
    dim3 grid;
    size_t smem;
};

bool plan(const GemmArgs& a, TcPlan* out)
{
    TcParams p{};
    p.a = a;
    p.wpr = words_per_row(a.n);
    p.nseg = 1;
    if (a.epilogue == EPI_LSTM) { p.gates = 4; p.units = a.H; }
    else if (a.epilogue == EPI_GRU) {
        p.gates = 3; p.units = a.H; p.nseg = 2;
        if (a.I % 32 != 0 || a.I == 0) return false;        // the column split must fall on a word boundary
    } else { p.gates = 1; p.units = a.m; }
    p.UT = TILE_M / (p.gates * a.k_w);
    if (p.UT < 1) return false;
    // batch entries per tile: multiples of 16, N = TB * k_a <= 256 (and both accumulators of the GRU in 512 columns)
    int tb_max = (256 / a.k_a) / 16 * 16;
    if (tb_max > 128) tb_max = 128;
    const int tiles = (a.batch + tb_max - 1) / tb_max;
    p.TB = ((a.batch + tiles - 1) / tiles + 15) / 16 * 16;
    p.n_mma = p.TB * a.k_a;
    int cols = 32;
    while (cols < p.nseg * p.n_mma) cols <<= 1;
    if (cols > 512) return false;
    p.tmem_cols = cols;
    const size_t stage = (size_t)A_STAGE_BYTES + (size_t)STAGE_WORDS * 2 * p.n_mma * 16;
    if ((size_t)p.nseg * TILE_M * (p.TB + 1) * 4 > 2 * stage) return false;
    out->p = p;
    out->smem = 2 * stage + 64;
    out->grid = dim3((unsigned)((p.units + p.UT - 1) / p.UT), (unsigned)((a.batch + p.TB - 1) / p.TB));
    return out->grid.y <= 65535u && out->smem <= 227 * 1024;
}

template <int KA>
amq_status launch_ka(const TcPlan& pl, cudaStream_t st)
{
    auto kernel = bgemm_tc_kernel<KA>;
    AMQ_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem));
    kernel<<<pl.grid, TC_THREADS, pl.smem, st>>>(pl.p);
    AMQ_LAUNCH_CHECK();
    return AMQ_OK;
}

}  // namespace

bool gemm_tc_supported(const GemmArgs& a)
{
    TcPlan pl;
    return a.batch >= 16 && plan(a, &pl);
}

amq_status launch_binary_gemm_tc(const GemmArgs& a, cudaStream_t st)
{
    TcPlan pl;
    if (!plan(a, &pl)) return AMQ_ERR_UNSUPPORTED;
    switch (a.k_a) {
        case 1: return launch_ka<1>(pl, st);
        case 2: return launch_ka<2>(pl, st);
        case 3: return launch_ka<3>(pl, st);
        case 4: return launch_ka<4>(pl, st);
    }
    return AMQ_ERR_UNSUPPORTED;
}

amq_status read_tc_status(cudaStream_t st, uint32_t* out)
{
    AMQ_CUDA_TRY(cudaStreamSynchronize(st));
    AMQ_CUDA_TRY(cudaMemcpyFromSymbol(out, g_tc_status, sizeof(uint32_t)));
    if (*out) {
        const uint32_t zero = 0;
        AMQ_CUDA_TRY(cudaMemcpyToSymbol(g_tc_status, &zero, sizeof(uint32_t)));
    }
    return AMQ_OK;
}

}  // namespace amq
