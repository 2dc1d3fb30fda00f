// Binary matrix product on the integer pipe: XOR + bit count on packed planes (Appendix A), in the
// stacked ("concatenated codes") form of Fig. 3, right: the k_w planes of every weight row and the k_a
// planes of every activation vector are treated as rows / columns of one 1-bit matrix product, and the
// k_w x k_a partials of each (row, vector) pair are folded with the row-wise coefficients afterwards.
//
// One kernel serves all bit counts (k_w, k_a are run-time values: the stacked form makes the inner
// loop independent of them) and four epilogues: raw integer partials, y = sum alpha beta D + bias, and
// the fused LSTM (Eq. 6) and GRU gate arithmetic.  For the cells a tile holds all gate rows of its
// hidden units, so the state update needs no second pass over global memory.
#include "amq_common.cuh"

namespace amq {

namespace {

constexpr int KC = 32;        // packed words per K chunk (1024 bits)
constexpr int LDS = KC + 1;   // padded smem row stride

struct PopcParams {
    GemmArgs a;
    int gates;      // 1 plain, 4 LSTM, 3 GRU
    int units;      // plain: m; cells: H
    int UT;         // units per tile
    int TB;         // batch entries per tile
    int nseg;       // 1, or 2 for the GRU (columns [0,I) and [I,n))
    int wpr;
};

__device__ __forceinline__ uint32_t range_mask(int q, int lo, int hi)
{
    const int first = q * 32;
    if (first + 32 <= lo || first >= hi) return 0u;
    uint32_t mask = 0xffffffffu;
    if (lo > first) mask &= 0xffffffffu << (lo - first);
    if (hi < first + 32) mask &= 0xffffffffu >> (first + 32 - hi);
    return mask;
}

__device__ __forceinline__ float logistic(float v) { return 1.0f / (1.0f + __expf(-v)); }

__global__ void __launch_bounds__(512)
bgemm_popc_kernel(PopcParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const GemmArgs& a = p.a;
    const int k_w = a.k_w, k_a = a.k_a;
    const int TM = p.UT * p.gates, TMp = TM * k_w, TNp = p.TB * k_a;
    const int TX = TNp / 4, TY = TMp / 4;

    // smem: [ A tile | B tile ] reused as the integer tile P, then two float tiles Y[seg][TM][TB]
    const int ab_words = (TMp + TNp) * LDS, p_words = TMp * TNp;
    uint32_t* As = reinterpret_cast<uint32_t*>(smem_raw);
    uint32_t* Bs = As + TMp * LDS;
    int* Pt = reinterpret_cast<int*>(smem_raw);
    float* Yt = reinterpret_cast<float*>(smem_raw) + (ab_words > p_words ? ab_words : p_words);

    const int tid = threadIdx.x, nthreads = blockDim.x;
    const int ty = tid / TX, tx = tid % TX;
    const bool computes = ty < TY;
    const int u0 = blockIdx.x * p.UT, b0 = blockIdx.y * p.TB;

    for (int seg = 0; seg < p.nseg; ++seg) {
        const int lo = (p.nseg == 2 && seg == 1) ? a.I : 0;
        const int hi = (p.nseg == 2 && seg == 0) ? a.I : a.n;
        int acc[4][4];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[r][c] = 0;

        for (int q0 = lo / 32; q0 * 32 < hi; q0 += KC) {
            for (int idx = tid; idx < TMp * KC; idx += nthreads) {
                const int pr = idx / KC, kk = idx % KC, q = q0 + kk;
                const int l = pr / k_w, i = pr % k_w;
                const int u = u0 + l / p.gates, gate = l % p.gates;
                uint32_t word = 0;
                if (u < p.units && q < p.wpr) {
                    const uint32_t mask = range_mask(q, lo, hi);
                    if (mask) {
                        const size_t row = (size_t)gate * p.units + u;
                        word = __ldg(a.Wcodes + (row * k_w + i) * p.wpr + q) & mask;
                    }
                }
                As[pr * LDS + kk] = word;
            }
            for (int idx = tid; idx < TNp * KC; idx += nthreads) {
                const int pc = idx / KC, kk = idx % KC, q = q0 + kk;
                const int b = b0 + pc / k_a, j = pc % k_a;
                uint32_t word = 0;
                if (b < a.batch && q < p.wpr) {
                    const uint32_t mask = range_mask(q, lo, hi);
                    if (mask) word = __ldg(a.xcodes + ((size_t)b * k_a + j) * p.wpr + q) & mask;
                }
                Bs[pc * LDS + kk] = word;
            }
            __syncthreads();
            if (computes) {
#pragma unroll 8
                for (int kk = 0; kk < KC; ++kk) {
                    uint32_t av[4], bv[4];
#pragma unroll
                    for (int r = 0; r < 4; ++r) av[r] = As[(ty * 4 + r) * LDS + kk];
#pragma unroll
                    for (int c = 0; c < 4; ++c) bv[c] = Bs[(tx * 4 + c) * LDS + kk];
#pragma unroll
                    for (int r = 0; r < 4; ++r)
#pragma unroll
                        for (int c = 0; c < 4; ++c) acc[r][c] += __popc(av[r] ^ bv[c]);
                }
            }
            __syncthreads();
        }

        // integer tile: P[plane row][plane column] = differing bits over the segment
        if (computes) {
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int c = 0; c < 4; ++c) Pt[(ty * 4 + r) * TNp + tx * 4 + c] = acc[r][c];
        }
        __syncthreads();

        // fold the k_w x k_a partials of each (row, vector) pair: D = len - 2 P
        const int len = hi - lo;
        for (int idx = tid; idx < TM * p.TB; idx += nthreads) {
            const int l = idx / p.TB, bb = idx % p.TB;
            const int u = u0 + l / p.gates, gate = l % p.gates, b = b0 + bb;
            float y = 0.0f;
            if (u < p.units && b < a.batch) {
                const size_t row = (size_t)gate * p.units + u;
                if (a.epilogue == EPI_DOTS) {
                    int32_t* out = a.D + (((size_t)b * a.m + row) * k_w) * k_a;
                    for (int i = 0; i < k_w; ++i)
                        for (int j = 0; j < k_a; ++j)
                            out[i * k_a + j] = len - 2 * Pt[(l * k_w + i) * TNp + bb * k_a + j];
                } else {
                    for (int i = 0; i < k_w; ++i) {
                        const float al = __ldg(a.Walpha + row * k_w + i);
                        for (int j = 0; j < k_a; ++j) {
                            const float be = __ldg(a.xbeta + (size_t)b * k_a + j);
                            y += al * be * (float)(len - 2 * Pt[(l * k_w + i) * TNp + bb * k_a + j]);
                        }
                    }
                }
            }
            Yt[(seg * TM + l) * p.TB + bb] = y;
        }
        __syncthreads();
    }

    if (a.epilogue == EPI_Y) {
        for (int idx = tid; idx < TM * p.TB; idx += nthreads) {
            const int l = idx / p.TB, bb = idx % p.TB;
            const int row = u0 + l, b = b0 + bb;
            if (row < a.m && b < a.batch)
                a.y[(size_t)b * a.ldy + row] = Yt[l * p.TB + bb] + (a.bias ? __ldg(a.bias + row) : 0.0f);
        }
    } else if (a.epilogue == EPI_LSTM) {
        const int H = a.H;
        for (int idx = tid; idx < p.UT * p.TB; idx += nthreads) {
            const int ul = idx / p.TB, bb = idx % p.TB;
            const int u = u0 + ul, b = b0 + bb;
            if (u < H && b < a.batch) {
                float pre[4];
#pragma unroll
                for (int g = 0; g < 4; ++g)
                    pre[g] = Yt[(ul * 4 + g) * p.TB + bb] + (a.bias ? __ldg(a.bias + g * H + u) : 0.0f) +
                             (a.addend ? __ldg(a.addend + (size_t)b * a.ld_addend + g * H + u) : 0.0f);
                const float ig = logistic(pre[0]), fg = logistic(pre[1]), og = logistic(pre[2]);
                const float gg = tanhf(pre[3]);
                const size_t o = (size_t)b * H + u;
                const float c = fg * a.c_in[o] + ig * gg;
                a.c_out[o] = c;
                a.h_out[o] = og * tanhf(c);
            }
        }
    } else if (a.epilogue == EPI_GRU) {
        const int H = a.H;
        for (int idx = tid; idx < p.UT * p.TB; idx += nthreads) {
            const int ul = idx / p.TB, bb = idx % p.TB;
            const int u = u0 + ul, b = b0 + bb;
            if (u < H && b < a.batch) {
                float px[3], ph[3];
#pragma unroll
                for (int g = 0; g < 3; ++g) {
                    px[g] = Yt[(0 * TM + ul * 3 + g) * p.TB + bb];
                    ph[g] = Yt[(1 * TM + ul * 3 + g) * p.TB + bb];
                }
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

}  // namespace

amq_status launch_binary_gemm(const GemmArgs& a, cudaStream_t st)
{
    if (gemv_supported(a)) return launch_binary_gemv(a, st);
    if (gemm_tc_supported(a)) return launch_binary_gemm_tc(a, st);
    PopcParams p;
    p.a = a;
    p.wpr = words_per_row(a.n);
    p.nseg = 1;
    if (a.epilogue == EPI_LSTM) { p.gates = 4; p.units = a.H; p.UT = 8; }
    else if (a.epilogue == EPI_GRU) { p.gates = 3; p.units = a.H; p.UT = 8; p.nseg = 2; }
    else { p.gates = 1; p.units = a.m; p.UT = 32; }
    p.TB = a.batch <= 4 ? 4 : 16;
    const int TM = p.UT * p.gates, TMp = TM * a.k_w, TNp = p.TB * a.k_a;
    int threads = (TMp / 4) * (TNp / 4);
    threads = 32 * ((threads + 31) / 32);
    if (threads < 64) threads = 64;
    const int ab_words = (TMp + TNp) * LDS, p_words = TMp * TNp;
    const size_t smem = (size_t)(ab_words > p_words ? ab_words : p_words) * 4 + (size_t)2 * TM * p.TB * 4;
    dim3 grid((unsigned)((p.units + p.UT - 1) / p.UT), (unsigned)((a.batch + p.TB - 1) / p.TB));
    if (grid.y > 65535u) return AMQ_ERR_UNSUPPORTED;
    bgemm_popc_kernel<<<grid, threads, smem, st>>>(p);
    AMQ_LAUNCH_CHECK();
    return AMQ_OK;
}

}  // namespace amq

extern "C" {

amq_status amq_binary_dots(const uint32_t* Wcodes, int m, int n, int k_w,
                           const uint32_t* xcodes, int batch, int k_a, int32_t* D, void* stream)
{
    if (!Wcodes || !xcodes || !D || m < 0 || batch < 0 || n < 1) return AMQ_ERR_INVALID_ARG;
    if (!amq::valid_k(k_w) || !amq::valid_k(k_a)) return AMQ_ERR_UNSUPPORTED;
    if (!amq::aligned16(Wcodes) || !amq::aligned16(xcodes)) return AMQ_ERR_ALIGNMENT;
    if (m == 0 || batch == 0) return AMQ_OK;
    amq::GemmArgs a{};
    a.Wcodes = Wcodes; a.m = m; a.n = n; a.k_w = k_w;
    a.xcodes = xcodes; a.batch = batch; a.k_a = k_a;
    a.epilogue = amq::EPI_DOTS; a.D = D;
    return amq::launch_binary_gemm(a, (cudaStream_t)stream);
}

amq_status amq_binary_gemm(const uint32_t* Wcodes, const float* Walpha, int m, int n, int k_w,
                           const uint32_t* xcodes, const float* xbeta, int batch, int k_a,
                           const float* bias, float* y, int ldy, void* stream)
{
    if (!Wcodes || !Walpha || !xcodes || !xbeta || !y || m < 0 || batch < 0 || n < 1 || ldy < m)
        return AMQ_ERR_INVALID_ARG;
    if (!amq::valid_k(k_w) || !amq::valid_k(k_a)) return AMQ_ERR_UNSUPPORTED;
    if (!amq::aligned16(Wcodes) || !amq::aligned16(xcodes)) return AMQ_ERR_ALIGNMENT;
    if (m == 0 || batch == 0) return AMQ_OK;
    amq::GemmArgs a{};
    a.Wcodes = Wcodes; a.Walpha = Walpha; a.m = m; a.n = n; a.k_w = k_w;
    a.xcodes = xcodes; a.xbeta = xbeta; a.batch = batch; a.k_a = k_a;
    a.bias = bias; a.epilogue = amq::EPI_Y; a.y = y; a.ldy = ldy;
    return amq::launch_binary_gemm(a, (cudaStream_t)stream);
}

amq_status amq_device_status(void* stream)
{
    uint32_t word = 0;
    amq_status s = amq::read_tc_status((cudaStream_t)stream, &word);
    if (s != AMQ_OK) return s;
    return word == 0 ? AMQ_OK : AMQ_ERR_TIMEOUT;
}

}  // extern "C"
