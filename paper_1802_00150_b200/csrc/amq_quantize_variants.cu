// Variants of the row quantizer, for the comparison of Sec. 2 / Tables 1-2 and for the other reading of the
// order of Algorithm 2's half steps: refined greedy (after every greedy bit all coefficients so far are
// re-solved by Eq. 5; codes are never revisited) and a final coefficient refit on the last codes.  Written
// for generality, not speed: one warp per row, elements 32 q + lane, every pass re-reads the row (it stays in
// L1/L2), the sign planes live in shared memory in the packed layout (a warp ballot IS word q of a plane).
#include "amq_common.cuh"
#include "amq_quantize_device.cuh"

namespace amq {
namespace {

constexpr int VAR_WARPS = 4;
constexpr int VAR_MAX_WORDS = AMQ_MAX_N / 32;     // words of a plane without the padding to 128 bits

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    return v;
}

// solve_refit of the production quantizer on the first KK coefficients of alpha[]
template <int KK>
__device__ __forceinline__ void solve_first(const float* c, const int* gram, int n, float* alpha)
{
    float cc[KK], aa[KK];
    int gg[KK > 1 ? KK * (KK - 1) / 2 : 1];
#pragma unroll
    for (int i = 0; i < KK; ++i) { cc[i] = c[i]; aa[i] = alpha[i]; }
#pragma unroll
    for (int q = 0; q < (KK > 1 ? KK * (KK - 1) / 2 : 1); ++q) gg[q] = gram[q];
    if (solve_refit<KK>(cc, gg, n, aa)) {
#pragma unroll
        for (int i = 0; i < KK; ++i) alpha[i] = aa[i];
    }
}

// Eq. 5 on the first kk planes: G = B^T B from popcounts (exact integers, upper triangle in row-major order),
// c = B^T w, then the solve of the production quantizer (a singular system leaves alpha untouched).  Every lane
// runs the same solve.
__device__ void refit(const float* __restrict__ x, int n, int kk, const uint32_t (*planes)[VAR_MAX_WORDS], int lane, float* alpha)
{
    const int Q = (n + 31) >> 5;
    float c[AMQ_MAX_K];
    int gram[AMQ_MAX_K * (AMQ_MAX_K - 1) / 2];
    int g = 0;
    for (int i = 0; i < kk; ++i) {
        for (int j = i + 1; j < kk; ++j) {
            int diff = 0;
            for (int q = lane; q < Q; q += 32) {
                const uint32_t mask = (32 * q + 32 <= n) ? 0xffffffffu : ((1u << (n - 32 * q)) - 1u);
                diff += __popc((planes[i][q] ^ planes[j][q]) & mask);
            }
            gram[g++] = n - 2 * __reduce_add_sync(0xffffffffu, diff);
        }
        float ci = 0.0f;
        for (int q = 0; q < Q; ++q) {
            const int t = 32 * q + lane;
            const float w = t < n ? x[t] : 0.0f;
            ci += ((planes[i][q] >> lane) & 1u) ? w : -w;
        }
        c[i] = warp_sum(ci);
    }
    switch (kk) {
        case 1: solve_first<1>(c, gram, n, alpha); break;
        case 2: solve_first<2>(c, gram, n, alpha); break;
        case 3: solve_first<3>(c, gram, n, alpha); break;
        case 4: solve_first<4>(c, gram, n, alpha); break;
    }
}

__global__ void __launch_bounds__(VAR_WARPS * 32)
quantize_variant_kernel(const float* __restrict__ x, int rows, int n, int ldx, int k, int T, int method, int final_refit,
                        uint32_t* __restrict__ codes, float* __restrict__ coeffs)
{
    __shared__ uint32_t s_planes[VAR_WARPS][AMQ_MAX_K][VAR_MAX_WORDS];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int row = blockIdx.x * VAR_WARPS + warp;
    if (row >= rows) return;
    uint32_t (*planes)[VAR_MAX_WORDS] = s_planes[warp];
    const float* xr = x + (size_t)row * ldx;
    const int Q = (n + 31) >> 5, wpr = 4 * ((n + 127) >> 7);
    float alpha[AMQ_MAX_K] = {0.0f, 0.0f, 0.0f, 0.0f};

    // greedy bits (Eq. 3-4); the refined method re-solves the coefficients after each of them
    for (int j = 0; j < k; ++j) {
        float part = 0.0f;
        for (int q = 0; q < Q; ++q) {
            const int t = 32 * q + lane;
            const bool valid = t < n;
            float r = valid ? xr[t] + 0.0f : 0.0f;
            for (int i = 0; i < j; ++i) r -= ((planes[i][q] >> lane) & 1u) ? alpha[i] : -alpha[i];
            part += valid ? fabsf(r) : 0.0f;
            const uint32_t word = __ballot_sync(0xffffffffu, valid && r >= 0.0f);
            if (lane == 0) planes[j][q] = word;
        }
        __syncwarp();
        alpha[j] = warp_sum(part) / (float)n;
        if (method == 1) refit(xr, n, j + 1, planes, lane, alpha);
    }
    // alternating cycles of Algorithm 2
    if (method == 0) {
        const int M = 1 << k;
        for (int it = 0; it < T; ++it) {
            refit(xr, n, k, planes, lane, alpha);
            // all levels in ascending order, ties by code; plane i is bit k - 1 - i of the code
            float v[1 << AMQ_MAX_K];
            int code[1 << AMQ_MAX_K];
            for (int c = 0; c < M; ++c) {
                float s = 0.0f;
                for (int i = 0; i < k; ++i) s += ((c >> (k - 1 - i)) & 1) ? alpha[i] : -alpha[i];
                int pos = c;
                while (pos > 0 && v[pos - 1] > s) { v[pos] = v[pos - 1]; code[pos] = code[pos - 1]; --pos; }
                v[pos] = s; code[pos] = c;
            }
            __syncwarp();
            for (int q = 0; q < Q; ++q) {
                const int t = 32 * q + lane;
                const bool valid = t < n;
                const float w = valid ? xr[t] : 0.0f;
                int lo = 0, hi = M;
                while (hi - lo > 1) {                                  // Algorithm 1: upper half on >=
                    const int mid = (lo + hi) >> 1;
                    if (w >= 0.5f * (v[mid - 1] + v[mid])) lo = mid; else hi = mid;
                }
                const int c = code[lo];
                for (int i = 0; i < k; ++i) {
                    const uint32_t word = __ballot_sync(0xffffffffu, valid && ((c >> (k - 1 - i)) & 1));
                    if (lane == 0) planes[i][q] = word;
                }
            }
            __syncwarp();
        }
    }
    if (final_refit) refit(xr, n, k, planes, lane, alpha);

    for (int i = 0; i < k; ++i)
        for (int q = lane; q < wpr; q += 32) codes[((size_t)row * k + i) * wpr + q] = q < Q ? planes[i][q] : 0u;
    if (lane < k) coeffs[(size_t)row * k + lane] = alpha[lane];
}

}  // namespace
}  // namespace amq

extern "C" amq_status amq_quantize_variant(const float* x, int rows, int n, int ldx, int k, int T, int method, int final_refit,
                                           uint32_t* codes, float* coeffs, void* stream)
{
    if (rows < 0 || n < 1 || ldx < n) return AMQ_ERR_INVALID_ARG;
    if (!amq::valid_k(k) || T < 0 || n > AMQ_MAX_N || (method != AMQ_METHOD_ALTERNATING && method != AMQ_METHOD_REFINED_GREEDY))
        return AMQ_ERR_UNSUPPORTED;
    if (rows == 0) return AMQ_OK;
    if (!x || !codes || !coeffs) return AMQ_ERR_INVALID_ARG;
    if (!amq::aligned16(codes)) return AMQ_ERR_ALIGNMENT;
    if (method == AMQ_METHOD_ALTERNATING && !final_refit)       // Algorithm 2 as printed: the production kernels
        return amq_quantize(x, rows, n, ldx, k, T, codes, coeffs, stream);
    amq::quantize_variant_kernel<<<(unsigned)((rows + amq::VAR_WARPS - 1) / amq::VAR_WARPS), amq::VAR_WARPS * 32, 0,
                                   (cudaStream_t)stream>>>(x, rows, n, ldx, k, T, method, final_refit, codes, coeffs);
    AMQ_LAUNCH_CHECK();
    return AMQ_OK;
}
