// Batch-1 binary matrix-vector product on packed planes (Sec. 4, Fig. 3 left; XOR + bit count,
// Appendix A): y[r] = sum_i alpha[r][i] * sum_j beta[j] * (n - 2 popcount(W_i[r] xor x_j)) + bias[r].
//
// The product streams the packed weight planes from HBM exactly once and is bound by that stream, so
// the kernel is organised around the loads: a segment of SEG lanes owns one weight row (all k_w planes),
// lane c of the segment reads the 128-bit chunks c, c + SEG of every plane, and several rows per lane are
// requested before any is consumed, which keeps enough bytes in flight to cover the DRAM latency.  The k_a
// activation planes are loop invariant for a lane (it always works on the same columns) and live in
// registers.
//
// Bit counting is the second ceiling right behind the memory one (one POPC per weight word and
// activation plane issues at a quarter of the logic rate), so pairs of XOR-ed words first go through a
// carry-save adder on whole words (two LOP3) and only the carries and the final sums are counted.
//
// Fused form (the operation Table 6 times: on-line quantization of the activation vector, then the product, in ONE
// launch): every CTA quantizes the fp32 vector itself (Algorithm 2 with the CTA as the group, the same device code as
// the recurrent kernel; redundant across CTAs, which costs a microsecond of latency and no memory traffic worth
// naming) into shared memory and takes its activation planes from there; its first weight rows are already in flight
// meanwhile.  For vectors of up to 2048 elements.
#include "amq_common.cuh"
#include "amq_quantize_device.cuh"

namespace amq {

namespace {

struct GemvParams {
    const uint4* W;             // [m][k_w][CH] 128-bit chunks
    const float* Walpha;        // [m][k_w]
    const uint4* x;             // [k_a][CH]
    const float* xbeta;         // [k_a]
    const float* bias;          // [m] or null
    float* y;                   // EPI_Y
    int32_t* D;                 // EPI_DOTS: [m][k_w][k_a]
    int m, n, CH;
    int epilogue;
    bool overlap;               // host side only: launch as a programmatic dependent of the preceding kernel
    // fused form: the fp32 vector, alternating cycles, and where CTA 0 leaves the planes and coefficients (or null)
    const float* xf;
    int T;
    uint32_t* xcodes_out;
    float* xbeta_out;
};

constexpr int FQ_EPT = 8;       // fused form: 256 threads x 8 consecutive elements each
constexpr int FQ_MAX_CH = 16;   // = 2048 bit positions
#ifndef FQ_CTAS_PER_SM
#define FQ_CTAS_PER_SM 1
#endif

// differing bits of (w xor x) over the four words of a chunk, accumulated carry-save:
// `ones` carries the bit-wise sums, the return value counts the carries (weight 2)
__device__ __forceinline__ int csa_chunk(const uint4& w, const uint4& x, uint32_t& ones)
{
    const uint32_t t0 = w.x ^ x.x, t1 = w.y ^ x.y, t2 = w.z ^ x.z, t3 = w.w ^ x.w;
    const uint32_t c0 = (ones & t0) | (ones & t1) | (t0 & t1);        // majority -> one LOP3
    ones ^= t0 ^ t1;
    const uint32_t c1 = (ones & t2) | (ones & t3) | (t2 & t3);
    ones ^= t2 ^ t3;
    return __popc(c0) + __popc(c1);
}

// sum over the SEG lanes of a segment (exact integers): one warp-wide reduction instruction when the
// segment is the warp, a shuffle butterfly otherwise
template <int SEG>
__device__ __forceinline__ int segment_sum(int v)
{
    if (SEG == 32) return __reduce_add_sync(0xffffffffu, v);
#pragma unroll
    for (int off = SEG >> 1; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    return v;
}

// SEG_LOG2: lanes per row = 1 << SEG_LOG2.  EXACT: every plane has exactly CPT * SEG chunks, so every lane
// always has work and all load offsets are compile-time constants.
//
// A warp works on blocks of 32 consecutive rows.  One pass of the inner loop covers R * (32 / SEG) of them;
// its loads are issued one pass ahead of the bit counting (register double buffer), so the memory pipe
// never drains while a warp computes.  After the segment sums every lane of a segment holds the totals of
// that segment's row; lane `sub` of segment `seg` keeps the ones of row sub * (32 / SEG) + seg, and when
// the block is complete all 32 lanes fold coefficients and bias and store 32 consecutive outputs at once.
template <int KW, int KA, int CPT, int R, int SEG_LOG2, bool EXACT, bool FQ>
__global__ void __launch_bounds__(256)
bgemv_kernel(GemvParams p)
{
    __shared__ __align__(16) uint4 sX[FQ ? KA : 1][FQ ? FQ_MAX_CH : 1];
    __shared__ QuantScratch<KA, FQ ? 8 : 1> q_scratch;
    if (!FQ) grid_dependency_wait();     // the activation planes may come from the preceding kernel of the stream
    const int lane = threadIdx.x & 31;
    constexpr int SEG = 1 << SEG_LOG2;
    constexpr int spw = 32 >> SEG_LOG2;            // rows per load instruction of the warp
    constexpr int PASSES = SEG / R;                // passes per block of 32 rows
    static_assert(SEG % R == 0, "rows per pass must divide the block");
    const int sub = lane & (SEG - 1), seg = lane >> SEG_LOG2;
    const int CH = EXACT ? CPT * SEG : p.CH;
    const size_t row_chunks = (size_t)KW * CH;

    bool has[CPT];
#pragma unroll
    for (int c = 0; c < CPT; ++c) has[c] = EXACT || (sub + c * SEG < CH);
    uint4 xr[KA][CPT];          // activation planes of this lane's columns, and their coefficients (filled below)
    float beta[KA];

    const long long blocks = ((long long)p.m + 31) >> 5;
    const long long warp_global = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const long long total_warps = (long long)gridDim.x * (blockDim.x >> 5);
    const long long last_row = (long long)p.m - 1;

    // loads of one pass: rows block * 32 + (pass * R + r) * spw + seg, clamped into the matrix
    auto load_pass = [&](uint4 (&w)[R][KW][CPT], long long block, int pass) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
            long long row = block * 32 + (pass * R + r) * spw + seg;
            row = row < last_row ? row : last_row;
            const uint4* src = p.W + (size_t)row * row_chunks + sub;
#pragma unroll
            for (int i = 0; i < KW; ++i)
#pragma unroll
                for (int c = 0; c < CPT; ++c) {
                    if (EXACT) w[r][i][c] = __ldcs(src + (i * CPT + c) * SEG);
                    else w[r][i][c] = has[c] ? __ldcs(src + (size_t)i * CH + c * SEG) : make_uint4(0, 0, 0, 0);
                }
        }
    };

    int mine[KW][KA];           // totals of this lane's row of the current block
#pragma unroll
    for (int i = 0; i < KW; ++i)
#pragma unroll
        for (int j = 0; j < KA; ++j) mine[i][j] = 0;

    // the passes of all blocks, in order, are dealt out to the warps in equal contiguous shares (a share
    // may begin and end inside a block; each warp then finishes only the rows of the passes it ran)
    const long long total = blocks * PASSES;
    const long long share = total / total_warps, extra = total % total_warps;
    long long g = warp_global * share + (warp_global < extra ? warp_global : extra);
    const long long g_end = g + share + (warp_global < extra ? 1 : 0);
    int first_pass = (int)(g % PASSES);          // first pass this warp ran in the current block

    auto step = [&](uint4 (&cur)[R][KW][CPT], uint4 (&nxt)[R][KW][CPT]) {
        const long long block = g / PASSES;
        const int pass = (int)(g - block * PASSES);
        if (g + 1 < g_end) {
            const long long nblock = (g + 1) / PASSES;
            load_pass(nxt, nblock, (int)(g + 1 - nblock * PASSES));
        }
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const bool keep = sub == pass * R + r;
#pragma unroll
            for (int i = 0; i < KW; ++i)
#pragma unroll
                for (int j = 0; j < KA; ++j) {
                    uint32_t ones = 0;
                    int carries = 0;
#pragma unroll
                    for (int c = 0; c < CPT; ++c) carries += csa_chunk(cur[r][i][c], xr[j][c], ones);
                    // lanes without a chunk hold w = x = 0 and contribute nothing
                    const int sum = segment_sum<SEG>(2 * carries + __popc(ones));
                    if (keep) mine[i][j] = sum;
                }
        }
        if (pass == PASSES - 1 || g + 1 == g_end) {
            const long long row = block * 32 + sub * spw + seg;       // this lane's row of the block
            const int my_pass = sub / R;
            if (row < p.m && my_pass >= first_pass && my_pass <= pass) {
                if (p.epilogue == EPI_DOTS) {
                    int32_t* out = p.D + (size_t)row * KW * KA;
#pragma unroll
                    for (int i = 0; i < KW; ++i)
#pragma unroll
                        for (int j = 0; j < KA; ++j) out[i * KA + j] = p.n - 2 * mine[i][j];
                } else {
                    float yv = 0.0f;
#pragma unroll
                    for (int i = 0; i < KW; ++i) {
                        const float al = __ldg(p.Walpha + (size_t)row * KW + i);
#pragma unroll
                        for (int j = 0; j < KA; ++j) yv += al * beta[j] * (float)(p.n - 2 * mine[i][j]);
                    }
                    p.y[row] = yv + (p.bias ? __ldg(p.bias + row) : 0.0f);
                }
            }
            first_pass = 0;
        }
        ++g;
    };

    uint4 wa[R][KW][CPT], wb[R][KW][CPT];
    if (g < g_end) load_pass(wa, g / PASSES, (int)(g % PASSES));     // weights are constant: in flight before anything else

    if constexpr (FQ) {
        // on-line quantization of the vector by this CTA: thread t owns the 8 consecutive elements 8 t .. 8 t + 7, so
        // the sign bits the quantizer leaves in a register are byte t of the packed plane
        quant_scratch_init(q_scratch);
        grid_dependency_wait();                            // the vector may come from the preceding kernel of the stream
        const int tid = threadIdx.x, e0 = tid * FQ_EPT;
        float w[FQ_EPT];
        uint32_t valid = 0;
#pragma unroll
        for (int j = 0; j < FQ_EPT; ++j) {
            const bool ok = e0 + j < p.n;
            w[j] = ok ? __ldcg(p.xf + e0 + j) : 0.0f;
            valid |= (ok ? 1u : 0u) << j;
        }
        uint32_t bits[KA];
        quantize_group<KA, FQ_EPT, 8>(w, valid, p.n, quant_padding_consecutive(p.n, FQ_EPT), p.T, beta, bits, q_scratch);
        if (e0 < CH * 128) {
#pragma unroll
            for (int j = 0; j < KA; ++j) reinterpret_cast<uint8_t*>(&sX[j][0])[tid] = (uint8_t)bits[j];
        }
        __syncthreads();
#pragma unroll
        for (int c = 0; c < CPT; ++c)
#pragma unroll
            for (int j = 0; j < KA; ++j) xr[j][c] = has[c] ? sX[j][sub + c * SEG] : make_uint4(0, 0, 0, 0);
        if (blockIdx.x == 0 && p.xcodes_out) {             // the planes and coefficients, for whoever needs them next
            for (int q = tid; q < KA * CH * 4; q += blockDim.x) {
                const int j = q / (CH * 4), wq = q - j * CH * 4;
                p.xcodes_out[q] = reinterpret_cast<const uint32_t*>(&sX[j][0])[wq];
            }
            if (tid < KA && p.xbeta_out) {
                float b = beta[0];
#pragma unroll
                for (int j = 1; j < KA; ++j) b = (tid == j) ? beta[j] : b;
                p.xbeta_out[tid] = b;
            }
        }
    } else {
#pragma unroll
        for (int c = 0; c < CPT; ++c)
#pragma unroll
            for (int j = 0; j < KA; ++j)
                xr[j][c] = has[c] ? p.x[(size_t)j * CH + sub + c * SEG] : make_uint4(0, 0, 0, 0);   // ordinary load, L1-cached
#pragma unroll
        for (int j = 0; j < KA; ++j) beta[j] = (p.epilogue == EPI_Y) ? p.xbeta[j] : 0.0f;
    }

    while (g < g_end) {
        step(wa, wb);
        if (!(g < g_end)) break;
        step(wb, wa);
    }
}

template <int KW, int KA, int CPT, int SEG_LOG2, bool FQ>
amq_status launch_cfg(const GemvParams& p, cudaStream_t st)
{
    constexpr int SEG = 1 << SEG_LOG2;
    constexpr int R0 = (8 / (KW * CPT)) > 0 ? (8 / (KW * CPT)) : 1;     // about eight 128-bit loads per lane and pass
    constexpr int R = R0 < SEG ? R0 : SEG;
    const bool exact = p.CH == CPT * SEG;
    auto kernel = exact ? bgemv_kernel<KW, KA, CPT, R, SEG_LOG2, true, FQ> : bgemv_kernel<KW, KA, CPT, R, SEG_LOG2, false, FQ>;
    static thread_local int cached_dev = -1, cached_grid[2] = {0, 0}, cached_sms = 0;
    int dev = 0;
    AMQ_CUDA_TRY(cudaGetDevice(&dev));
    if (dev != cached_dev) {
        int sms = 0;
        AMQ_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        for (int e = 0; e < 2; ++e) {
            int per_sm = 0;
            if (e) AMQ_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, bgemv_kernel<KW, KA, CPT, R, SEG_LOG2, true, FQ>, 256, 0));
            else AMQ_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, bgemv_kernel<KW, KA, CPT, R, SEG_LOG2, false, FQ>, 256, 0));
            cached_grid[e] = sms * (per_sm > 0 ? per_sm : 1);
        }
        cached_dev = dev;
        cached_sms = sms;
    }
    constexpr int PASSES = SEG / R;
    const long long passes = ((long long)p.m + 31) / 32 * PASSES;
    const long long need = (passes + 7) / 8;                            // small matrices: one pass per warp, spread over the SMs
    // fused form: every CTA repeats the quantization, so no more than FQ_CTAS_PER_SM of them share an SM's issue slots
    const int limit = FQ ? (cached_sms * FQ_CTAS_PER_SM < cached_grid[exact ? 1 : 0] ? cached_sms * FQ_CTAS_PER_SM : cached_grid[exact ? 1 : 0])
                         : cached_grid[exact ? 1 : 0];
    const int grid = (int)(need < limit ? need : limit);
    AMQ_CUDA_TRY(launch_kernel(kernel, dim3((unsigned)grid), dim3(256), 0, st, p.overlap, p));
    AMQ_LAUNCH_CHECK();
    return AMQ_OK;
}

// chunks per plane -> lanes per row: 2 (up to 256 columns), 8, 16, 32 with one chunk per lane, 32 with two
template <int KW, int KA>
amq_status launch_cpt(const GemvParams& p, cudaStream_t st)
{
    if (p.xf) {                 // fused form: up to 16 chunks
        if (p.CH <= 2) return launch_cfg<KW, KA, 1, 1, true>(p, st);
        if (p.CH <= 8) return launch_cfg<KW, KA, 1, 3, true>(p, st);
        if (p.CH <= FQ_MAX_CH) return launch_cfg<KW, KA, 1, 4, true>(p, st);
        return AMQ_ERR_UNSUPPORTED;
    }
    if (p.CH <= 2) return launch_cfg<KW, KA, 1, 1, false>(p, st);
    if (p.CH <= 8) return launch_cfg<KW, KA, 1, 3, false>(p, st);
    if (p.CH <= 16) return launch_cfg<KW, KA, 1, 4, false>(p, st);
    if (p.CH <= 32) return launch_cfg<KW, KA, 1, 5, false>(p, st);
    return launch_cfg<KW, KA, 2, 5, false>(p, st);
}

template <int KW>
amq_status launch_ka(const GemvParams& p, int k_a, cudaStream_t st)
{
    switch (k_a) {
        case 1: return launch_cpt<KW, 1>(p, st);
        case 2: return launch_cpt<KW, 2>(p, st);
        case 3: return launch_cpt<KW, 3>(p, st);
        case 4: return launch_cpt<KW, 4>(p, st);
    }
    return AMQ_ERR_UNSUPPORTED;
}

amq_status launch_kw(const GemvParams& p, int k_w, int k_a, cudaStream_t st)
{
    switch (k_w) {
        case 1: return launch_ka<1>(p, k_a, st);
        case 2: return launch_ka<2>(p, k_a, st);
        case 3: return launch_ka<3>(p, k_a, st);
        case 4: return launch_ka<4>(p, k_a, st);
    }
    return AMQ_ERR_UNSUPPORTED;
}

}  // namespace

bool gemv_supported(const GemmArgs& a)
{
    return a.batch == 1 && (a.epilogue == EPI_Y || a.epilogue == EPI_DOTS) && words_per_row(a.n) / 4 <= 64;
}

amq_status launch_binary_gemv(const GemmArgs& a, cudaStream_t st)
{
    if (!gemv_supported(a)) return AMQ_ERR_UNSUPPORTED;
    GemvParams p;
    p.W = reinterpret_cast<const uint4*>(a.Wcodes);
    p.Walpha = a.Walpha;
    p.x = reinterpret_cast<const uint4*>(a.xcodes);
    p.xbeta = a.xbeta;
    p.bias = a.bias;
    p.y = a.y;
    p.D = a.D;
    p.m = a.m; p.n = a.n; p.CH = words_per_row(a.n) / 4;
    p.epilogue = a.epilogue;
    p.overlap = a.overlap_with_previous;
    p.xf = nullptr; p.T = 0; p.xcodes_out = nullptr; p.xbeta_out = nullptr;
    return launch_kw(p, a.k_w, a.k_a, st);
}

bool quantized_gemv_supported(int n) { return n >= 1 && words_per_row(n) / 4 <= FQ_MAX_CH; }

amq_status launch_quantized_gemv(const uint32_t* Wcodes, const float* Walpha, int m, int n, int k_w, const float* x, int k_a, int T,
                                 const float* bias, float* y, uint32_t* xcodes_out, float* xbeta_out, cudaStream_t st,
                                 bool overlap_with_previous)
{
    if (!quantized_gemv_supported(n)) return AMQ_ERR_UNSUPPORTED;
    GemvParams p;
    p.W = reinterpret_cast<const uint4*>(Wcodes);
    p.Walpha = Walpha;
    p.x = nullptr; p.xbeta = nullptr;
    p.bias = bias;
    p.y = y; p.D = nullptr;
    p.m = m; p.n = n; p.CH = words_per_row(n) / 4;
    p.epilogue = EPI_Y;
    p.overlap = overlap_with_previous;
    p.xf = x; p.T = T; p.xcodes_out = xcodes_out; p.xbeta_out = xbeta_out;
    return launch_kw(p, k_w, k_a, st);
}

}  // namespace amq

extern "C" amq_status amq_quantized_gemv(const uint32_t* Wcodes, const float* Walpha, int m, int n, int k_w,
                                         const float* x, int k_a, int T, const float* bias, float* y,
                                         uint32_t* xcodes_out, float* xbeta_out, void* stream)
{
    if (m < 0 || n < 1) return AMQ_ERR_INVALID_ARG;
    if (!amq::valid_k(k_w) || !amq::valid_k(k_a) || T < 0 || !amq::quantized_gemv_supported(n)) return AMQ_ERR_UNSUPPORTED;
    if (m == 0) return AMQ_OK;
    if (!Wcodes || !Walpha || !x || !y) return AMQ_ERR_INVALID_ARG;
    if (!amq::aligned16(Wcodes) || (xcodes_out && !amq::aligned16(xcodes_out))) return AMQ_ERR_ALIGNMENT;
    return amq::launch_quantized_gemv(Wcodes, Walpha, m, n, k_w, x, k_a, T, bias, y, xcodes_out, xbeta_out,
                                      (cudaStream_t)stream, false);
}
