// Row-wise alternating multi-bit quantizer (Algorithm 2): greedy initialisation (Eq. 3-4), then T
// cycles of { least-squares refit of the coefficients (Eq. 5); sorted level table; binary-search-tree
// code assignment (Algorithm 1) }, one thread group per row, the row held in registers.
//
// Data-parallel form of Algorithm 1 ("maintaining a mask vector ... operate BST for all entries
// simultaneously", Sec. 3): the 2^k - 1 midpoints of the ascending level table are non-decreasing, so
// the leaf the tree descent reaches is the number of midpoints that are <= w; every element counts them
// with branch-free compares and looks its sign pattern up in a 64-bit packed code table.
#include "amq_common.cuh"

namespace amq {

namespace {

struct RowSource {
    const float* src0; int ld0; int n0;
    const float* src1; int ld1;
};

__device__ __forceinline__ float load_elem(const RowSource& s, int row, int t)
{
    return (t < s.n0) ? __ldg(s.src0 + (size_t)row * s.ld0 + t) : __ldg(s.src1 + (size_t)row * s.ld1 + (t - s.n0));
}

// Sum of V doubles over the thread group, every thread receives the totals.  Fixed order: butterfly inside
// a warp, then warps in index order, so results are reproducible run to run.
template <int V, bool MULTI>
__device__ __forceinline__ void group_sum(double (&v)[V], double* red /* [warps][V], MULTI only */)
{
#pragma unroll
    for (int i = 0; i < V; ++i) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) v[i] += __shfl_xor_sync(0xffffffffu, v[i], off);
    }
    if (MULTI) {
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, warps = blockDim.x >> 5;
        __syncthreads();                       // previous use of `red` is over
        if (lane == 0) {
#pragma unroll
            for (int i = 0; i < V; ++i) red[warp * V + i] = v[i];
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < V; ++i) {
            double s = 0.0;
            for (int w = 0; w < warps; ++w) s += red[w * V + i];
            v[i] = s;
        }
    }
}

// Solve the K x K system G a = c by Gaussian elimination with partial pivoting (fp64).  Returns false,
// leaving `a` untouched, when a pivot is below 1e-9 * n (the refit is then skipped).
template <int K>
__device__ __forceinline__ bool solve_refit(double (&G)[K][K + 1], int n, double (&a)[K])
{
    const double tiny = 1e-9 * (double)n;
#pragma unroll
    for (int col = 0; col < K; ++col) {
        // bring the largest |entry| of the column to the pivot row by conditional swaps (static indices
        // only, so G stays in registers); the first maximum wins, as in a plain search
#pragma unroll
        for (int row = col + 1; row < K; ++row) {
            if (fabs(G[row][col]) > fabs(G[col][col])) {
#pragma unroll
                for (int j = 0; j <= K; ++j) { double t = G[col][j]; G[col][j] = G[row][j]; G[row][j] = t; }
            }
        }
        const double p = G[col][col];
        if (!(fabs(p) >= tiny) || p == 0.0) return false;
#pragma unroll
        for (int row = col + 1; row < K; ++row) {
            const double f = G[row][col] / p;
#pragma unroll
            for (int j = col; j <= K; ++j) G[row][j] -= f * G[col][j];
        }
    }
    double sol[K];
#pragma unroll
    for (int i = K - 1; i >= 0; --i) {
        double s = G[i][K];
#pragma unroll
        for (int j = i + 1; j < K; ++j) s -= G[i][j] * sol[j];
        sol[i] = s / G[i][i];
    }
#pragma unroll
    for (int i = 0; i < K; ++i) a[i] = sol[i];
    return true;
}

// K bits, EPT elements per thread.  MULTI: one row per CTA (blockDim.x threads); else one row per warp.
template <int K, int EPT, bool MULTI>
__global__ void __launch_bounds__(256)
quantize_kernel(RowSource src, int rows, int n, int T, uint32_t* __restrict__ codes, float* __restrict__ coeffs)
{
    constexpr int M = 1 << K;
    constexpr int V = K + K * (K - 1) / 2;
    __shared__ double red[MULTI ? 8 * V : 1];
    __shared__ float s_level[MULTI ? 1 : 8][M];
    __shared__ int s_code[MULTI ? 1 : 8][M];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int G = MULTI ? blockDim.x : 32;
    const int g = MULTI ? threadIdx.x : lane;
    const int slot = MULTI ? 0 : warp;
    const int row = MULTI ? blockIdx.x : blockIdx.x * (blockDim.x >> 5) + warp;
    if (row >= rows) return;          // whole group leaves together (row is uniform across the group)

    float w[EPT];
    uint32_t valid = 0;
#pragma unroll
    for (int j = 0; j < EPT; ++j) {
        const int t = j * G + g;
        const bool ok = t < n;
        w[j] = ok ? load_elem(src, row, t) : 0.0f;
        valid |= (ok ? 1u : 0u) << j;
    }
    const int nvalid = __popc(valid);

    // ---- greedy initialisation, Eq. 3-4 ----
    float alpha[K];
    uint32_t bits[K];
    {
        float r[EPT];
#pragma unroll
        for (int j = 0; j < EPT; ++j) r[j] = w[j];
#pragma unroll
        for (int i = 0; i < K; ++i) {
            float part = 0.0f;
#pragma unroll
            for (int j = 0; j < EPT; ++j) part += fabsf(r[j]);
            double tot[1] = {(double)part};
            group_sum<1, MULTI>(tot, red);
            const float a = (float)(tot[0] / (double)n);
            alpha[i] = a;
            uint32_t b = 0;
#pragma unroll
            for (int j = 0; j < EPT; ++j) {
                const bool pos = r[j] >= 0.0f;
                b |= (pos ? 1u : 0u) << j;
                r[j] = ((valid >> j) & 1u) ? (pos ? r[j] - a : r[j] + a) : 0.0f;
            }
            bits[i] = b & valid;
        }
    }

    // ---- T alternating cycles ----
    for (int it = 0; it < T; ++it) {
        // least-squares refit, Eq. 5: G = B^T B (integers), c = B^T w
        double red_v[V];
#pragma unroll
        for (int i = 0; i < K; ++i) {
            float part = 0.0f;
#pragma unroll
            for (int j = 0; j < EPT; ++j) part += ((bits[i] >> j) & 1u) ? w[j] : -w[j];
            red_v[i] = (double)part;
        }
        {
            int q = K;
#pragma unroll
            for (int i = 0; i < K; ++i)
#pragma unroll
                for (int j = i + 1; j < K; ++j)
                    red_v[q++] = (double)(nvalid - 2 * __popc((bits[i] ^ bits[j]) & valid));
        }
        group_sum<V, MULTI>(red_v, red);
        double Gm[K][K + 1];
        {
            int q = K;
#pragma unroll
            for (int i = 0; i < K; ++i) {
                Gm[i][i] = (double)n;
                Gm[i][K] = red_v[i];
#pragma unroll
                for (int j = i + 1; j < K; ++j) { Gm[i][j] = red_v[q]; Gm[j][i] = red_v[q]; ++q; }
            }
        }
        double sol[K];
#pragma unroll
        for (int i = 0; i < K; ++i) sol[i] = (double)alpha[i];
        solve_refit<K>(Gm, n, sol);
#pragma unroll
        for (int i = 0; i < K; ++i) alpha[i] = (float)sol[i];

        // level table in ascending order by (value, code index); plane 0 is the most significant code bit
        if (MULTI) __syncthreads(); else __syncwarp();
        if (g < M) {
            float mine = 0.0f;
#pragma unroll
            for (int i = 0; i < K; ++i) mine += ((g >> (K - 1 - i)) & 1) ? alpha[i] : -alpha[i];
            int rank = 0;
#pragma unroll
            for (int c = 0; c < M; ++c) {
                float v = 0.0f;
#pragma unroll
                for (int i = 0; i < K; ++i) v += ((c >> (K - 1 - i)) & 1) ? alpha[i] : -alpha[i];
                rank += (v < mine || (v == mine && c < g)) ? 1 : 0;
            }
            s_level[slot][rank] = mine;
            s_code[slot][rank] = g;
        }
        if (MULTI) __syncthreads(); else __syncwarp();
        float thr[M - 1];
        unsigned long long table = 0ull;
#pragma unroll
        for (int p = 0; p < M - 1; ++p) thr[p] = (s_level[slot][p] + s_level[slot][p + 1]) * 0.5f;
#pragma unroll
        for (int p = 0; p < M; ++p) table |= (unsigned long long)s_code[slot][p] << (4 * p);

        // Algorithm 1 for every element: leaf = number of midpoints <= w
#pragma unroll
        for (int i = 0; i < K; ++i) bits[i] = 0;
#pragma unroll
        for (int j = 0; j < EPT; ++j) {
            int pos = 0;
#pragma unroll
            for (int p = 0; p < M - 1; ++p) pos += (w[j] >= thr[p]) ? 1 : 0;
            const uint32_t code = (uint32_t)(table >> (4 * pos)) & 15u;
#pragma unroll
            for (int i = 0; i < K; ++i) bits[i] |= ((code >> (K - 1 - i)) & 1u) << j;
        }
#pragma unroll
        for (int i = 0; i < K; ++i) bits[i] &= valid;
    }

    // ---- pack: word (j * G/32 + warp-in-group) of plane i = ballot over the warp of bit j ----
    const int wpr = 4 * ((n + 127) / 128);
    const int wig = MULTI ? warp : 0;       // warp index inside the group
    const int gw = G >> 5;                  // warps per group
    uint32_t* out = codes + (size_t)row * K * wpr;
#pragma unroll
    for (int i = 0; i < K; ++i) {
        uint32_t mine = 0;
#pragma unroll
        for (int j = 0; j < EPT; ++j) {
            const uint32_t word = __ballot_sync(0xffffffffu, (bits[i] >> j) & 1u);
            if (lane == j) mine = word;
        }
        if (lane < EPT) {
            const int q = lane * gw + wig;
            if (q < wpr) out[i * wpr + q] = mine;
        }
    }
    if (g < K) {
        float a = alpha[0];
#pragma unroll
        for (int i = 1; i < K; ++i) a = (g == i) ? alpha[i] : a;
        coeffs[(size_t)row * K + g] = a;
    }
}

template <int K, int EPT, bool MULTI>
amq_status run(const RowSource& src, int rows, int n, int T, uint32_t* codes, float* coeffs, int threads,
               cudaStream_t st)
{
    const int rows_per_cta = MULTI ? 1 : threads / 32;
    const unsigned grid = (unsigned)((rows + rows_per_cta - 1) / rows_per_cta);
    quantize_kernel<K, EPT, MULTI><<<grid, threads, 0, st>>>(src, rows, n, T, codes, coeffs);
    AMQ_LAUNCH_CHECK();
    return AMQ_OK;
}

template <int K>
amq_status dispatch(const RowSource& src, int rows, int n, int T, uint32_t* codes, float* coeffs, cudaStream_t st)
{
    const int n128 = 128 * ((n + 127) / 128);
    const bool bulk = rows >= 1024;
    if (bulk && n128 <= 256) return run<K, 8, false>(src, rows, n, T, codes, coeffs, 128, st);
    if (bulk && n128 <= 1024) return run<K, 32, false>(src, rows, n, T, codes, coeffs, 128, st);
    if (bulk || n128 > 2048) {
        const int threads = 32 * ((n128 / 32 + 31) / 32);      // 32 elements per thread
        return run<K, 32, true>(src, rows, n, T, codes, coeffs, threads, st);
    }
    const int threads = 32 * ((n128 / 8 + 31) / 32);           // 8 elements per thread, up to 256 threads
    return run<K, 8, true>(src, rows, n, T, codes, coeffs, threads, st);
}

}  // namespace

amq_status launch_quantize(const float* src0, int ld0, int n0, const float* src1, int ld1, int n1,
                           int rows, int k, int T, uint32_t* codes, float* coeffs, cudaStream_t st)
{
    RowSource src{src0, ld0, n0, src1, ld1};
    const int n = n0 + n1;
    switch (k) {
        case 1: return dispatch<1>(src, rows, n, T, codes, coeffs, st);
        case 2: return dispatch<2>(src, rows, n, T, codes, coeffs, st);
        case 3: return dispatch<3>(src, rows, n, T, codes, coeffs, st);
        case 4: return dispatch<4>(src, rows, n, T, codes, coeffs, st);
    }
    return AMQ_ERR_UNSUPPORTED;
}

}  // namespace amq

extern "C" amq_status amq_quantize(const float* x, int rows, int n, int ldx, int k, int T,
                                   uint32_t* codes, float* coeffs, void* stream)
{
    if (rows < 0 || n < 1 || ldx < n) return AMQ_ERR_INVALID_ARG;
    if (!amq::valid_k(k) || T < 0 || n > AMQ_MAX_N) return AMQ_ERR_UNSUPPORTED;
    if (rows == 0) return AMQ_OK;       // nothing to do; pointers of empty buffers may be NULL
    if (!x || !codes || !coeffs) return AMQ_ERR_INVALID_ARG;
    if (!amq::aligned16(codes)) return AMQ_ERR_ALIGNMENT;
    return amq::launch_quantize(x, ldx, n, nullptr, 0, 0, rows, k, T, codes, coeffs, (cudaStream_t)stream);
}
