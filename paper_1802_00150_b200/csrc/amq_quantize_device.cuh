// Device-side body of the alternating multi-bit quantizer (Algorithm 2), shared by the stand-alone
// row quantizer kernel and by the persistent recurrent kernel, which quantizes [x ; h] in place.
//
// A "group" of threads owns one vector; every thread holds EPT of its elements in registers (which ones is
// the caller's choice).  Data-parallel form of Algorithm 1 ("maintaining a mask vector ... operate BST for
// all entries simultaneously", Sec. 3): every element descends the tree over the 2^k - 1 midpoints of the
// ascending level table with k compares and predicated selects of the next midpoint (no branches), and the
// leaf index looks the sign pattern up in one small bit table per plane.
//
// Instruction economy of the inner loops (they decide the throughput of bulk quantization): inputs are
// canonicalised (-0.0 -> +0.0), after which "r >= 0" is exactly "sign bit clear" for every residue the
// greedy step can produce, so a sign plane is gathered with one funnel shift per element, a residue is
// updated as r - copysign(alpha, r) with one logic operation and one add, and +-w for the refit sums is one
// logic operation; the refit sums of a cycle are accumulated in the same pass that assigns the codes.
// Elements past the end of the vector are zeros that take part in every loop unmasked: their bits are
// cleared at the end, they add nothing to B^T w, the Gram matrix is counted on masked words, and their known
// contribution to the greedy |r| sums (all of them follow the trajectory of a zero element) is subtracted.
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
    uint32_t plane[K];                  // bit p of plane[i]: sign (1 = +1) of plane i at sorted level p
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

// Per-plane bit tables of the sorted code table: bit p of plane[i] = sign (1 = +1) of plane i at level p.
template <int K>
__device__ __forceinline__ void planes_from_table(unsigned long long table, uint32_t (&plane)[K])
{
#pragma unroll
    for (int i = 0; i < K; ++i) plane[i] = 0u;
#pragma unroll
    for (int p = 0; p < (1 << K); ++p) {
        const uint32_t code = (uint32_t)(table >> (4 * p)) & 15u;
#pragma unroll
        for (int i = 0; i < K; ++i) plane[i] |= ((code >> (K - 1 - i)) & 1u) << p;
    }
}

// Algorithm 1 for one element: index of the leaf (sorted level) the descent over the midpoints reaches.
// The midpoints are non-decreasing; ">=" goes to the upper half.
template <int K>
__device__ __forceinline__ int bst_leaf(float x, const float (&thr)[(1 << K) - 1])
{
    if (K == 1) return (x >= thr[0]) ? 1 : 0;
    if (K == 2) {
        const bool c1 = x >= thr[1];
        const bool c2 = x >= (c1 ? thr[2] : thr[0]);
        return (c1 ? 2 : 0) + (c2 ? 1 : 0);
    }
    if (K == 3) {
        const bool c1 = x >= thr[3];
        const bool c2 = x >= (c1 ? thr[5] : thr[1]);
        const float hi = c2 ? thr[6] : thr[4], lo = c2 ? thr[2] : thr[0];
        const bool c3 = x >= (c1 ? hi : lo);
        return (c1 ? 4 : 0) + (c2 ? 2 : 0) + (c3 ? 1 : 0);
    }
    const bool c1 = x >= thr[7];
    const bool c2 = x >= (c1 ? thr[11] : thr[3]);
    const float hi3 = c2 ? thr[13] : thr[9], lo3 = c2 ? thr[5] : thr[1];
    const bool c3 = x >= (c1 ? hi3 : lo3);
    const float q3 = c3 ? thr[14] : thr[12], q2 = c3 ? thr[10] : thr[8];
    const float q1 = c3 ? thr[6] : thr[4], q0 = c3 ? thr[2] : thr[0];
    const float hi4 = c2 ? q3 : q2, lo4 = c2 ? q1 : q0;
    const bool c4 = x >= (c1 ? hi4 : lo4);
    return (c1 ? 8 : 0) + (c2 ? 4 : 0) + (c3 ? 2 : 0) + (c4 ? 1 : 0);
}

// Quantize the vector held in w[] (positions past the end of the vector must hold 0 and have their bit
// clear in `valid`; `padding` is their number over the whole group).  On return alpha[i] are the
// coefficients and bit j of bits[i] is the sign (1 = +1) of element j of this thread in plane i.
//
// The greedy step needs k dependent reductions (each coefficient is the mean |residue| left by the
// previous one, Eq. 3-4); the sign plane of the last greedy bit does not depend on its own coefficient,
// so that last reduction travels together with the sums of the first refit (Eq. 5): k + T - 1 group
// reductions in all for T >= 1, with the values Algorithm 2 prescribes.
template <int K, int EPT, bool MULTI>
__device__ __forceinline__ void quantize_group(const float (&w_in)[EPT], uint32_t valid, int n, int T,
                                               float (&alpha)[K], uint32_t (&bits)[K], QuantScratch<K>& sc)
{
    constexpr int M = 1 << K;
    constexpr int NG = K * (K - 1) / 2;
    constexpr uint32_t SIGN = 0x80000000u;
    const int lane = threadIdx.x & 31;
    const int nvalid = __popc(valid);
    const float inv_n = 1.0f / (float)n;
    const float padding = (float)((MULTI ? (int)blockDim.x : 32) * EPT - n);     // zero elements past the end
    int parity = 0;

    float w[EPT];
#pragma unroll
    for (int j = 0; j < EPT; ++j) w[j] = w_in[j] + 0.0f;          // -0.0 -> +0.0: from here on "x >= 0" is "sign bit clear"

    // ---- greedy initialisation, Eq. 3-4 (and, for T > 0, B^T w of the first refit in the same pass) ----
    float last_abs = 0.0f, csum[K];
    float rho = 0.0f;                                             // residue of a zero element (the padding)
    {
        float r[EPT];
#pragma unroll
        for (int j = 0; j < EPT; ++j) r[j] = w[j];
#pragma unroll
        for (int i = 0; i < K; ++i) {
            float part = 0.0f, cs = 0.0f;
            uint32_t neg = 0;
#pragma unroll
            for (int j = EPT - 1; j >= 0; --j) {
                const uint32_t rb = __float_as_uint(r[j]);
                part += fabsf(r[j]);
                neg = __funnelshift_l(rb, neg, 1);                // sign bit of r[j] enters at bit 0
                cs += __uint_as_float(__float_as_uint(w[j]) ^ (rb & SIGN));        // b_i * w
            }
            bits[i] = ~neg & valid;
            csum[i] = cs;
            if (i == K - 1 && T > 0) { last_abs = part; alpha[i] = 0.0f; break; }
            float tot[1] = {part};
            int none[1] = {0};
            const bool leader = group_totals<1, 0, K, MULTI>(tot, none, sc, parity);
            float a = (tot[0] - padding * fabsf(rho)) * inv_n;
            if (MULTI) {
                if (leader && lane == 0) sc.out[parity].alpha[0] = a;
                __syncthreads();
                a = sc.out[parity].alpha[0];
            }
            parity ^= 1;
            alpha[i] = a;
            const uint32_t ab = __float_as_uint(a);               // a >= 0
            rho -= __uint_as_float(ab | (__float_as_uint(rho) & SIGN));
#pragma unroll
            for (int j = 0; j < EPT; ++j)
                r[j] -= __uint_as_float(ab | (__float_as_uint(r[j]) & SIGN));      // r - copysign(a, r)
        }
    }

    // ---- T alternating cycles ----
    for (int it = 0; it < T; ++it) {
        // least-squares refit, Eq. 5: G = B^T B (exact integers), c = B^T w (summed while the codes were assigned)
        float fsum[1 + K];
        int gram[NG > 0 ? NG : 1];
        fsum[0] = last_abs;
#pragma unroll
        for (int i = 0; i < K; ++i) fsum[1 + i] = csum[i];
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
        uint32_t plane[K];
        if (leader) {
            if (it == 0) alpha[K - 1] = (fsum[0] - padding * fabsf(rho)) * inv_n;   // the last greedy coefficient
            float c[K];
#pragma unroll
            for (int i = 0; i < K; ++i) c[i] = fsum[1 + i];
            solve_refit<K>(c, gram, n, alpha);
            unsigned long long table = 0ull;
            level_table<K>(alpha, lane, thr, table, sc);
            planes_from_table<K>(table, plane);
            if (MULTI && lane == 0) {
                QuantOut<K>& o = sc.out[parity];
#pragma unroll
                for (int i = 0; i < K; ++i) { o.alpha[i] = alpha[i]; o.plane[i] = plane[i]; }
#pragma unroll
                for (int p = 0; p < M - 1; ++p) o.thr[p] = thr[p];
            }
        }
        if (MULTI) {
            __syncthreads();
            const QuantOut<K>& o = sc.out[parity];
#pragma unroll
            for (int i = 0; i < K; ++i) { alpha[i] = o.alpha[i]; plane[i] = o.plane[i]; }
#pragma unroll
            for (int p = 0; p < M - 1; ++p) thr[p] = o.thr[p];
        }
        parity ^= 1;
        last_abs = 0.0f;

        // Algorithm 1 for every element; the sums B^T w of the next refit are taken in the same pass
        const bool more = it + 1 < T;
        uint32_t pos_bits[K];
#pragma unroll
        for (int i = 0; i < K; ++i) { pos_bits[i] = 0u; csum[i] = 0.0f; }
#pragma unroll
        for (int j = EPT - 1; j >= 0; --j) {
            const int sh = 31 - bst_leaf<K>(w[j], thr);
#pragma unroll
            for (int i = 0; i < K; ++i) {
                const uint32_t y = plane[i] << sh;                 // sign of plane i at this leaf, in the top bit
                pos_bits[i] = __funnelshift_l(y, pos_bits[i], 1);
                if (more) csum[i] += __uint_as_float(__float_as_uint(w[j]) ^ (~y & SIGN));
            }
        }
#pragma unroll
        for (int i = 0; i < K; ++i) bits[i] = pos_bits[i] & valid;
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
