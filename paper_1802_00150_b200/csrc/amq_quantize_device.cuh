// Device-side body of the alternating multi-bit quantizer (Algorithm 2), shared by the stand-alone
// row quantizer kernel and by the persistent recurrent kernel, which quantizes [x ; h] in place.
//
// A "group" of threads owns one vector; thread g of a group of G threads holds elements j*G + g,
// j < EPT, in registers.  Data-parallel form of Algorithm 1 ("maintaining a mask vector ... operate BST
// for all entries simultaneously", Sec. 3): the 2^k - 1 midpoints of the ascending level table are
// non-decreasing, so the leaf the tree descent reaches is the number of midpoints that are <= w; every
// element counts them with branch-free compares and looks its sign pattern up in a packed code table.
//
// Arithmetic: sums over the vector are fp32 (per thread, then a fixed butterfly / warp order, so results
// are reproducible run to run); the Gram matrix B^T B is exact integer arithmetic; the k x k solve is
// fp64; levels, midpoints and comparisons are fp32.
//
// When the group is a whole CTA, the per-vector scalar work (cross-warp totals, the k x k solve, the
// sorted level table) is done once by warp 0 and handed to the other warps through shared memory, rather
// than repeated by every warp: in the persistent kernel the quantizer sits on the latency path of each
// timestep, and issue slots, not arithmetic, are what it runs out of.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace amq {

constexpr int QUANT_MAX_WARPS = 16;

template <int K>
struct QuantOut {                       // what the leader warp publishes after a reduction
    float alpha[K];
    float thr[(1 << K) - 1];
    unsigned long long table;
};

// Shared-memory scratch of one group (a warp, or a CTA of up to 16 warps).
template <int K>
struct QuantScratch {
    static constexpr int V = 1 + K + K * (K - 1) / 2;
    static constexpr int STRIDE = V + (V & 1);
    float red[2][QUANT_MAX_WARPS][STRIDE];   // per-warp partial sums, double-buffered by reduction parity
    QuantOut<K> out[2];
    float level[1 << K];
    int code[1 << K];
};

// Totals over the group of VF floats and VI ints (ints are carried exactly).  Returns true in the threads
// that hold the totals afterwards: every thread when the group is one warp; the threads of warp 0 when the
// group is the CTA (MULTI).  In the MULTI case the caller must publish what the others need and
// __syncthreads() before they read it.
template <int VF, int VI, int K, bool MULTI>
__device__ __forceinline__ bool group_totals(float (&f)[VF], int (&iv)[VI > 0 ? VI : 1], QuantScratch<K>& sc, int parity)
{
#pragma unroll
    for (int i = 0; i < VF; ++i) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) f[i] += __shfl_xor_sync(0xffffffffu, f[i], off);
    }
#pragma unroll
    for (int i = 0; i < VI; ++i) iv[i] = __reduce_add_sync(0xffffffffu, iv[i]);
    if (!MULTI) return true;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, warps = blockDim.x >> 5;
    if (lane == 0) {
        float* mine = sc.red[parity][warp];
#pragma unroll
        for (int i = 0; i < VF; ++i) mine[i] = f[i];
#pragma unroll
        for (int i = 0; i < VI; ++i) mine[VF + i] = __int_as_float(iv[i]);
    }
    __syncthreads();
    if (warp != 0) return false;
    // warp 0: lane l holds the partials of warp l; sum over lanes in a fixed butterfly
    const bool have = lane < warps;
    const float* src = sc.red[parity][have ? lane : 0];
#pragma unroll
    for (int i = 0; i < VF; ++i) {
        float v = have ? src[i] : 0.0f;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
        f[i] = v;
    }
#pragma unroll
    for (int i = 0; i < VI; ++i) iv[i] = __reduce_add_sync(0xffffffffu, have ? __float_as_int(src[VF + i]) : 0);
    return true;
}

// Least-squares solve of Eq. 5, G a = c with G = B^T B (G_ii = n, integer off-diagonals in gram[], row
// major upper triangle) in fp64.  Leaves `a` untouched and returns false when a pivot of Gaussian
// elimination with partial pivoting falls below 1e-9 * n (reading for a singular system: skip the refit).
template <int K>
__device__ __forceinline__ bool solve_refit(const float (&c)[K], const int (&gram)[K > 1 ? K * (K - 1) / 2 : 1], int n,
                                            float (&a)[K])
{
    if (K == 1) {
        if (n <= 0) return false;
        a[0] = c[0] / (float)n;
        return true;
    }
    if (K == 2) {
        // pivots of the elimination are n and (n^2 - g^2) / n: the second is below 1e-9 n only when the
        // integer n^2 - g^2 is zero (n <= 8192), i.e. b_1 = +-b_2
        const int g = gram[0];
        const int det = n * n - g * g;                       // |.| <= 2^26: exact in int and in double
        if (det == 0) return false;
        const double dd = (double)det;
        double r = (double)__frcp_rn((float)det);            // fp32 seed, one Newton step in fp64
        r = r * (2.0 - dd * r);
        r = r * (2.0 - dd * r);
        const double c0 = (double)c[0], c1 = (double)c[1], dn = (double)n, dg = (double)g;
        a[0] = (float)((dn * c0 - dg * c1) * r);
        a[1] = (float)((dn * c1 - dg * c0) * r);
        return true;
    }
    double G[K][K + 1];
    {
        int q = 0;
#pragma unroll
        for (int i = 0; i < K; ++i) {
            G[i][i] = (double)n;
            G[i][K] = (double)c[i];
#pragma unroll
            for (int j = i + 1; j < K; ++j) { G[i][j] = (double)gram[q]; G[j][i] = (double)gram[q]; ++q; }
        }
    }
    const double tiny = 1e-9 * (double)n;
    double rp[K];
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
        rp[col] = 1.0 / p;
#pragma unroll
        for (int row = col + 1; row < K; ++row) {
            const double fct = G[row][col] * rp[col];
#pragma unroll
            for (int j = col; j <= K; ++j) G[row][j] -= fct * G[col][j];
        }
    }
    double sol[K];
#pragma unroll
    for (int i = K - 1; i >= 0; --i) {
        double s = G[i][K];
#pragma unroll
        for (int j = i + 1; j < K; ++j) s -= G[i][j] * sol[j];
        sol[i] = s * rp[i];
    }
#pragma unroll
    for (int i = 0; i < K; ++i) a[i] = (float)sol[i];
    return true;
}

// Ascending level table of the 2^K values sum_i +-alpha_i, ordered by (value, code index), plane 0 the most
// significant code bit.  Produces the 2^K - 1 midpoints and the codes packed 4 bits per table position.
// Executed by one full warp (K >= 3 uses its lanes and __syncwarp).
template <int K>
__device__ __forceinline__ void level_table(const float (&alpha)[K], int lane, float (&thr)[(1 << K) - 1],
                                            unsigned long long& table, QuantScratch<K>& sc)
{
    constexpr int M = 1 << K;
    if (K == 1) {
        // levels -a, +a (or swapped when a < 0); the midpoint is 0 either way
        thr[0] = (-alpha[0] + alpha[0]) * 0.5f;
        table = (alpha[0] < 0.0f) ? 0x01ull : 0x10ull;
        return;
    }
    if (K == 2) {
        float v[4];
        int c[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            float s = 0.0f;
            s += (q & 2) ? alpha[0] : -alpha[0];
            s += (q & 1) ? alpha[1] : -alpha[1];
            v[q] = s; c[q] = q;
        }
#define AMQ_CSWAP(x, y)                                                                   \
        if (v[x] > v[y] || (v[x] == v[y] && c[x] > c[y])) {                               \
            const float tv = v[x]; v[x] = v[y]; v[y] = tv;                                \
            const int tc = c[x]; c[x] = c[y]; c[y] = tc;                                  \
        }
        AMQ_CSWAP(0, 1) AMQ_CSWAP(2, 3) AMQ_CSWAP(0, 2) AMQ_CSWAP(1, 3) AMQ_CSWAP(1, 2)
#undef AMQ_CSWAP
#pragma unroll
        for (int p = 0; p < 3; ++p) thr[p] = (v[p] + v[p + 1]) * 0.5f;
        table = (unsigned long long)(c[0] | (c[1] << 4) | (c[2] << 8) | (c[3] << 12));
        return;
    }
    // K >= 3: lane c < 2^K ranks its own level among all, through shared memory
    __syncwarp();
    if (lane < M) {
        float mine = 0.0f;
#pragma unroll
        for (int i = 0; i < K; ++i) mine += ((lane >> (K - 1 - i)) & 1) ? alpha[i] : -alpha[i];
        int rank = 0;
#pragma unroll
        for (int c = 0; c < M; ++c) {
            float v = 0.0f;
#pragma unroll
            for (int i = 0; i < K; ++i) v += ((c >> (K - 1 - i)) & 1) ? alpha[i] : -alpha[i];
            rank += (v < mine || (v == mine && c < lane)) ? 1 : 0;
        }
        sc.level[rank] = mine;
        sc.code[rank] = lane;
    }
    __syncwarp();
    table = 0ull;
#pragma unroll
    for (int p = 0; p < M - 1; ++p) thr[p] = (sc.level[p] + sc.level[p + 1]) * 0.5f;
#pragma unroll
    for (int p = 0; p < M; ++p) table |= (unsigned long long)sc.code[p] << (4 * p);
}

// Quantize the vector held in w[] (elements with their bit clear in `valid` are padding and must be 0).
// On return alpha[i] are the coefficients and bit j of bits[i] is the sign (1 = +1) of element j of this
// thread in plane i.
//
// The greedy step needs k dependent reductions (each coefficient is the mean |residue| left by the
// previous one, Eq. 3-4); the sign plane of the last greedy bit does not depend on its own coefficient,
// so that last reduction travels together with the sums of the first refit (Eq. 5): k + T - 1 group
// reductions in all for T >= 1, with the values Algorithm 2 prescribes.
template <int K, int EPT, bool MULTI>
__device__ __forceinline__ void quantize_group(const float (&w)[EPT], uint32_t valid, int n, int T,
                                               float (&alpha)[K], uint32_t (&bits)[K], QuantScratch<K>& sc)
{
    constexpr int M = 1 << K;
    constexpr int NG = K * (K - 1) / 2;
    const int lane = threadIdx.x & 31;
    const int nvalid = __popc(valid);
    const float inv_n = 1.0f / (float)n;
    int parity = 0;

    // ---- greedy initialisation, Eq. 3-4 ----
    float last_abs = 0.0f;
    {
        float r[EPT];
#pragma unroll
        for (int j = 0; j < EPT; ++j) r[j] = w[j];
#pragma unroll
        for (int i = 0; i < K; ++i) {
            float part = 0.0f;
            uint32_t b = 0;
#pragma unroll
            for (int j = 0; j < EPT; ++j) {
                part += fabsf(r[j]);
                if (r[j] >= 0.0f) b |= 1u << j;
            }
            bits[i] = b & valid;
            if (i == K - 1 && T > 0) { last_abs = part; alpha[i] = 0.0f; break; }
            float tot[1] = {part};
            int none[1] = {0};
            const bool leader = group_totals<1, 0, K, MULTI>(tot, none, sc, parity);
            float a = tot[0] * inv_n;
            if (MULTI) {
                if (leader && lane == 0) sc.out[parity].alpha[0] = a;
                __syncthreads();
                a = sc.out[parity].alpha[0];
            }
            parity ^= 1;
            alpha[i] = a;
#pragma unroll
            for (int j = 0; j < EPT; ++j)
                r[j] = ((valid >> j) & 1u) ? (((b >> j) & 1u) ? r[j] - a : r[j] + a) : 0.0f;
        }
    }

    // ---- T alternating cycles ----
    for (int it = 0; it < T; ++it) {
        // least-squares refit, Eq. 5: G = B^T B (exact integers), c = B^T w
        float fsum[1 + K];
        int gram[NG > 0 ? NG : 1];
        fsum[0] = last_abs;
#pragma unroll
        for (int i = 0; i < K; ++i) {
            float part = 0.0f;
#pragma unroll
            for (int j = 0; j < EPT; ++j)
                part += __uint_as_float(__float_as_uint(w[j]) ^ ((~(bits[i] >> j) & 1u) << 31));   // +-w
            fsum[1 + i] = part;
        }
        {
            int q = 0;
#pragma unroll
            for (int i = 0; i < K; ++i)
#pragma unroll
                for (int j = i + 1; j < K; ++j)
                    gram[q++] = nvalid - 2 * __popc((bits[i] ^ bits[j]) & valid);
            if (NG == 0) gram[0] = 0;
        }
        const bool leader = group_totals<1 + K, NG, K, MULTI>(fsum, gram, sc, parity);
        float thr[M - 1];
        unsigned long long table = 0ull;
        if (leader) {
            if (it == 0) alpha[K - 1] = fsum[0] * inv_n;          // the last greedy coefficient
            float c[K];
#pragma unroll
            for (int i = 0; i < K; ++i) c[i] = fsum[1 + i];
            solve_refit<K>(c, gram, n, alpha);
            level_table<K>(alpha, lane, thr, table, sc);
            if (MULTI && lane == 0) {
                QuantOut<K>& o = sc.out[parity];
#pragma unroll
                for (int i = 0; i < K; ++i) o.alpha[i] = alpha[i];
#pragma unroll
                for (int p = 0; p < M - 1; ++p) o.thr[p] = thr[p];
                o.table = table;
            }
        }
        if (MULTI) {
            __syncthreads();
            const QuantOut<K>& o = sc.out[parity];
#pragma unroll
            for (int i = 0; i < K; ++i) alpha[i] = o.alpha[i];
#pragma unroll
            for (int p = 0; p < M - 1; ++p) thr[p] = o.thr[p];
            table = o.table;
        }
        parity ^= 1;
        last_abs = 0.0f;

        // Algorithm 1 for every element: leaf = number of midpoints <= w
        const uint32_t table_lo = (uint32_t)table;
#pragma unroll
        for (int i = 0; i < K; ++i) bits[i] = 0;
#pragma unroll
        for (int j = 0; j < EPT; ++j) {
            int pos = 0;
#pragma unroll
            for (int p = 0; p < M - 1; ++p) pos += (w[j] >= thr[p]) ? 1 : 0;
            const uint32_t code = (K <= 3) ? (table_lo >> (4 * pos)) : (uint32_t)(table >> (4 * pos));
#pragma unroll
            for (int i = 0; i < K; ++i) bits[i] |= ((code >> (K - 1 - i)) & 1u) << j;
        }
#pragma unroll
        for (int i = 0; i < K; ++i) bits[i] &= valid;
    }
}

// Pack the sign bits of a group into words: word (j * G/32 + warp-in-group) of plane i is the ballot
// over the warp of bit j.  `out` points at the k planes of the vector (global or shared memory).
template <int K, int EPT>
__device__ __forceinline__ void pack_group(const uint32_t (&bits)[K], int lane, int warp_in_group,
                                           int warps_per_group, int wpr, uint32_t* out)
{
#pragma unroll
    for (int i = 0; i < K; ++i) {
        uint32_t mine = 0;
#pragma unroll
        for (int j = 0; j < EPT; ++j) {
            const uint32_t word = __ballot_sync(0xffffffffu, (bits[i] >> j) & 1u);
            if (lane == j) mine = word;
        }
        if (lane < EPT) {
            const int q = lane * warps_per_group + warp_in_group;
            if (q < wpr) out[i * wpr + q] = mine;
        }
    }
}

}  // namespace amq
