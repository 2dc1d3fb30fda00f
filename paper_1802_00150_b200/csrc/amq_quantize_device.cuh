// Device-side body of the alternating multi-bit quantizer (Algorithm 2), shared by the stand-alone
// row quantizer kernel and by the persistent recurrent kernel, which quantizes [x ; h] in place.
//
// A "group" of threads owns one vector; every thread holds EPT of its elements in registers (which ones is
// the caller's choice).  Algorithm 1 is evaluated in its data-parallel form (the remark on operating on all
// entries at once, Sec. 3): every element descends the tree over the 2^k - 1 midpoints of the ascending level
// table with k compares and predicated selects of the next midpoint (no branches), and the leaf index looks
// the sign pattern up in one small bit table per plane.
//
// Instruction economy of the inner loops (they decide the throughput of bulk quantization): inputs are
// canonicalised (-0.0 -> +0.0), after which "r >= 0" is exactly "sign bit clear" for every residue the
// greedy step can produce, so a sign plane is gathered with one funnel shift per element, a residue is
// updated as r - copysign(alpha, r) with one logic operation and one add, and +-w for the refit sums is one
// logic operation; the refit sums of a cycle are accumulated in the same pass that assigns the codes.
// Elements past the end of the vector are zeros that take part in every loop unmasked: their bits are
// cleared at the end, they add nothing to B^T w, the Gram matrix is counted on masked words, and their known
// contribution to the greedy |r| sums (all of them follow the trajectory of a zero element) is subtracted.
// Threads that hold no element of the vector at all leave their |r| sums out instead, so that what is
// subtracted stays a few elements' worth whatever the size of the group (the subtraction of a large known
// sum from a rounded one would cost accuracy on short vectors).
//
// Arithmetic: sums over the vector are fp32 (per thread, then a fixed butterfly over the warp, then the
// per-warp partials in a fixed tree, so results are reproducible run to run); the Gram matrix B^T B is exact
// integer arithmetic; the k x k solve is fp64 for k >= 3 (k = 3: through the exact integer adjugate) and error-compensated fp32 for k = 2 (the products
// n c_i and g c_j are split exactly with fused multiply-adds, so cancellation costs nothing); levels,
// midpoints and comparisons are fp32.
//
// When the group is a whole CTA, a reduction costs ONE barrier: lane 0 of every warp leaves the warp's
// partial sums in shared memory, and after the barrier every thread adds up all partials itself and
// repeats the per-vector scalar work (solve, sorted level table) redundantly.  In the recurrent kernels the
// quantizer sits on the latency path of each timestep, and a second barrier plus a round trip through
// shared memory for "one warp computes, all read" costs more than the repeated arithmetic.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace amq {

constexpr int QUANT_MAX_WARPS = 16;

// Shared-memory scratch of one group of NW warps (NW = 1: a single warp, which needs the level scratch only).
template <int K, int NW>
struct __align__(16) QuantScratch {
    static constexpr int V = 1 + K + K * (K - 1) / 2;
    static constexpr int SLOTS = NW > 1 ? ((NW + 3) / 4) * 4 : 4;
    float red[2][V][SLOTS];             // [reduction parity][value][warp]: per-warp partial sums
    float level[NW][1 << K];            // per-warp scratch of the level sort (k >= 3)
    int code[NW][1 << K];
};

// To be called once by every thread of a CTA-wide group before its first quantize_group (no barrier needed
// afterwards): partial-sum slots of warps that do not exist are read as zeros by every reduction.
template <int K, int NW>
__device__ __forceinline__ void quant_scratch_init(QuantScratch<K, NW>& sc)
{
    constexpr int V = QuantScratch<K, NW>::V, SLOTS = QuantScratch<K, NW>::SLOTS;
    const int warps = blockDim.x >> 5;
    float* flat = &sc.red[0][0][0];
    for (int idx = threadIdx.x; idx < 2 * V * SLOTS; idx += blockDim.x)
        if ((idx % SLOTS) >= warps) flat[idx] = 0.0f;
}

// Totals over the group of VF floats and VI ints (ints are carried exactly); every thread of the group holds
// them afterwards.  NW > 1: the group is the CTA and the call contains exactly one CTA barrier; when `flag`
// is given, that barrier also ORs *flag over the CTA (every thread gets the result).
template <int VF, int VI, int K, int NW>
__device__ __forceinline__ void group_totals(float (&f)[VF], int (&iv)[VI > 0 ? VI : 1], QuantScratch<K, NW>& sc,
                                             int parity, int* flag = nullptr)
{
#pragma unroll
    for (int i = 0; i < VF; ++i) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) f[i] += __shfl_xor_sync(0xffffffffu, f[i], off);
    }
#pragma unroll
    for (int i = 0; i < VI; ++i) iv[i] = __reduce_add_sync(0xffffffffu, iv[i]);
    if (NW == 1) return;
    constexpr int SLOTS = QuantScratch<K, NW>::SLOTS;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) {
#pragma unroll
        for (int i = 0; i < VF; ++i) sc.red[parity][i][warp] = f[i];
#pragma unroll
        for (int i = 0; i < VI; ++i) sc.red[parity][VF + i][warp] = __int_as_float(iv[i]);
    }
    if (flag) *flag = __syncthreads_or(*flag);
    else __syncthreads();
    // every thread: the partials of all warps, added in a fixed tree (slots of absent warps hold zeros)
#pragma unroll
    for (int i = 0; i < VF; ++i) {
        float tot = 0.0f;
#pragma unroll
        for (int q = 0; q < SLOTS / 4; ++q) {
            const float4 v = *reinterpret_cast<const float4*>(&sc.red[parity][i][4 * q]);
            const float s = (v.x + v.y) + (v.z + v.w);
            tot = (q == 0) ? s : tot + s;
        }
        f[i] = tot;
    }
#pragma unroll
    for (int i = 0; i < VI; ++i) {
        int tot = 0;
#pragma unroll
        for (int q = 0; q < SLOTS / 4; ++q) {
            const int4 v = *reinterpret_cast<const int4*>(&sc.red[parity][VF + i][4 * q]);
            tot += (v.x + v.y) + (v.z + v.w);
        }
        iv[i] = tot;
    }
}

// Least-squares solve of Eq. 5, G a = c with G = B^T B (G_ii = n, integer off-diagonals in gram[], row
// major upper triangle).  Leaves `a` untouched and returns false when a pivot of Gaussian elimination with
// partial pivoting falls below 1e-9 * n (reading for a singular system: skip the refit).  k = 2 and k = 3 solve
// through the exact integer adjugate (same rule, evaluated on exact quantities); k = 4 eliminates in fp64.
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
        // integer n^2 - g^2 is zero (n <= 8192), i.e. b_1 = +-b_2.  Cramer's rule on the exact integers; each
        // numerator n c_i - g c_j is formed without cancellation error: t = fl(g c_j), e = g c_j - t exactly
        // (fused multiply-add), fl(n c_i - t) rounds once relative to the RESULT, then e is taken off.
        const int g = gram[0];
        const int det = n * n - g * g;                       // |.| <= 2^26: exact in int
        if (det == 0) return false;
        const float fn = (float)n, fg = (float)g;            // exact (<= 8192)
        const float rdet = __fdividef(1.0f, (float)det);     // |det| <= 2^26: in range of the fast reciprocal
        const float t0 = fg * c[1], e0 = fmaf(fg, c[1], -t0);
        const float t1 = fg * c[0], e1 = fmaf(fg, c[0], -t1);
        a[0] = (fmaf(fn, c[0], -t0) - e0) * rdet;
        a[1] = (fmaf(fn, c[1], -t1) - e1) * rdet;
        return true;
    }
    if (K == 3) {
        // Adjugate of the Gram matrix: its entries and the determinant are integers below 2^53, exact in fp64, so the only
        // roundings are those of the three-term sums and of the division, and the dependent chain is a third of the
        // elimination's (the solve is per-vector scalar work that every warp repeats; on the batched cells' on-line
        // quantizer it was a visible part of a timestep).  The singularity rule is the elimination's, evaluated on the same
        // exact quantities: its second pivot is max(|n^2 - g01^2|, |n g12 - g01 g02|) / n and its third
        // |det| / (n x second pivot), whichever row the pivoting takes.
        const double n_ = (double)n, g01 = (double)gram[0], g02 = (double)gram[1], g12 = (double)gram[2];
        const double A00 = n_ * n_ - g12 * g12, A01 = g02 * g12 - g01 * n_, A02 = g01 * g12 - g02 * n_;
        const double A11 = n_ * n_ - g02 * g02, A12 = g01 * g02 - g12 * n_, A22 = n_ * n_ - g01 * g01;
        const double det = n_ * A00 + g01 * A01 + g02 * A02;
        const double tiny = 1e-9 * n_;
        const double pivot2n = fmax(fabs(A22), fabs(A12));          // n x the second pivot
        if (!(pivot2n >= tiny * n_) || !(fabs(det) >= tiny * pivot2n)) return false;
        const double rd = 1.0 / det;
        const double c0 = (double)c[0], c1 = (double)c[1], c2 = (double)c[2];
        a[0] = (float)((A00 * c0 + A01 * c1 + A02 * c2) * rd);
        a[1] = (float)((A01 * c0 + A11 * c1 + A12 * c2) * rd);
        a[2] = (float)((A02 * c0 + A12 * c1 + A22 * c2) * rd);
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

// Ascending level table of the 2^K values sum_i +-alpha_i, ordered by (value, code index), plane 0 the most
// significant code bit.  Produces the 2^K - 1 midpoints and, per plane, the signs along the table (bit p of
// plane[i]: sign, 1 = +1, of plane i at sorted level p).
// Executed by one full warp (K >= 3 uses its lanes, __syncwarp and the warp's own scratch rows).
template <int K>
__device__ __forceinline__ void level_table(const float (&alpha)[K], int lane, float (&thr)[(1 << K) - 1],
                                            uint32_t (&plane)[K], float* sc_level, int* sc_code)
{
    constexpr int M = 1 << K;
    unsigned long long table = 0ull;          // codes packed 4 bits per table position (K != 2)
    if (K == 1) {
        // levels -a, +a (or swapped when a < 0); the midpoint is 0 either way
        thr[0] = (-alpha[0] + alpha[0]) * 0.5f;
        table = (alpha[0] < 0.0f) ? 0x01ull : 0x10ull;
        planes_from_table<K>(table, plane);
        return;
    }
    if (K == 2) {
        // The four levels +-a +-b in closed form.  With A = |a|, B = |b| the ascending values are
        // -(A+B), -|A-B|, +|A-B|, A+B, so the midpoints are -(fl(A+B) + |fl(A-B)|)/2, 0 and its negative
        // (exactly what sorting the four rounded sums gives).  In terms of the magnitudes the sign patterns
        // come in the order (-,-) (-,+) (+,-) (+,+) when A > B and (-,-) (+,-) (-,+) (+,+) when A < B; a
        // negative coefficient flips its own bit of every code.  Equal values are ordered by code index:
        // A == B ties the two middle levels (the first order is the ascending one unless a < 0); a coefficient
        // that is zero, or vanishes against the other in fp32, ties the outer pairs, and its bit then ascends.
        const float a = alpha[0], b = alpha[1];
        const float A = fabsf(a), B = fabsf(b);
        const float d = A - B;
        const float t0 = -0.5f * ((A + B) + fabsf(d));
        thr[0] = t0; thr[1] = 0.0f; thr[2] = -t0;
        bool sa = a < 0.0f, sb = b < 0.0f;
        const bool first = d > 0.0f || (d == 0.0f && !sa);
        if ((A + B) == fabsf(d)) {            // the smaller coefficient vanishes in the sums: its sign orders nothing
            if (first) sb = false; else sa = false;
        }
        plane[0] = (first ? 0xCu : 0xAu) ^ (sa ? 0xFu : 0u);      // bit p: sign of plane 0 at level p
        plane[K - 1] = (first ? 0xAu : 0xCu) ^ (sb ? 0xFu : 0u);
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
        sc_level[rank] = mine;
        sc_code[rank] = lane;
    }
    __syncwarp();
#pragma unroll
    for (int p = 0; p < M - 1; ++p) thr[p] = (sc_level[p] + sc_level[p + 1]) * 0.5f;
    // bit p of plane[i] = sign of plane i in the code at sorted position p: lane p holds that code, one ballot per plane
    // (the same masks as planes_from_table builds from the packed table, in a tenth of the instructions)
    const int code = lane < M ? sc_code[lane] : 0;
#pragma unroll
    for (int i = 0; i < K; ++i) plane[i] = __ballot_sync(0xffffffffu, ((code >> (K - 1 - i)) & 1) != 0);
    (void)table;
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

// Elements past the end of the vector inside the threads that do hold some of it, for the two ownership patterns in
// use: thread g owns the EPT consecutive elements from g * EPT; lane l of a warp owns the elements j * 32 + l.
__host__ __device__ inline int quant_padding_consecutive(int n, int ept) { return (n + ept - 1) / ept * ept - n; }
__host__ __device__ inline int quant_padding_strided32(int n, int ept) { return (n >= 32 ? 32 : n) * ept - n; }

// Quantize the vector held in w[] (positions past the end of the vector must hold 0 and have their bit
// clear in `valid`; `pad_elems` = how many such positions lie in threads whose `valid` is not zero).  NW = 1: the group is the calling warp; NW > 1: the group is the whole CTA of up to NW
// warps (quant_scratch_init must have run).  On return alpha[i] are the coefficients and bit j of bits[i] is
// the sign (1 = +1) of element j of this thread in plane i.
//
// The greedy step needs k dependent reductions (each coefficient is the mean |residue| left by the
// previous one, Eq. 3-4); the sign plane of the last greedy bit does not depend on its own coefficient,
// so that last reduction travels together with the sums of the first refit (Eq. 5): k + T - 1 group
// reductions in all for T >= 1, with the values Algorithm 2 prescribes; each is one CTA barrier when the
// group is the CTA.  `flag` (CTA groups only, may be NULL): ORed over the CTA by the first of those barriers,
// so a caller can fold a "some thread gave up waiting for its input" vote into it; `parity` (CTA groups
// only): which half of the double-buffered partial-sum scratch the first reduction uses, updated on return,
// so that consecutive calls keep alternating.
template <int K, int EPT, int NW>
__device__ __forceinline__ void quantize_group(const float (&w_in)[EPT], uint32_t valid, int n, int pad_elems, int T,
                                               float (&alpha)[K], uint32_t (&bits)[K], QuantScratch<K, NW>& sc,
                                               int* flag = nullptr, int* parity_io = nullptr)
{
    constexpr int M = 1 << K;
    constexpr int NG = K * (K - 1) / 2;
    constexpr uint32_t SIGN = 0x80000000u;
    const int lane = threadIdx.x & 31;
    const int slot = NW > 1 ? (int)(threadIdx.x >> 5) : 0;
    const int nvalid = __popc(valid);
    const float inv_n = 1.0f / (float)n;
    const float padding = (float)pad_elems;                      // zero elements past the end that are summed along
    const bool holds_some = valid != 0;
    int parity = parity_io ? *parity_io : 0;

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
            part = holds_some ? part : 0.0f;
            if (i == K - 1 && T > 0) { last_abs = part; alpha[i] = 0.0f; break; }
            float tot[1] = {part};
            int none[1] = {0};
            group_totals<1, 0, K, NW>(tot, none, sc, parity, flag);
            flag = nullptr;
            parity ^= 1;
            const float a = (tot[0] - padding * fabsf(rho)) * inv_n;
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
        group_totals<1 + K, NG, K, NW>(fsum, gram, sc, parity, flag);
        flag = nullptr;
        parity ^= 1;
        float thr[M - 1];
        uint32_t plane[K];
        {
            if (it == 0) alpha[K - 1] = (fsum[0] - padding * fabsf(rho)) * inv_n;   // the last greedy coefficient
            float c[K];
#pragma unroll
            for (int i = 0; i < K; ++i) c[i] = fsum[1 + i];
            solve_refit<K>(c, gram, n, alpha);
            level_table<K>(alpha, lane, thr, plane, sc.level[slot], sc.code[slot]);
        }
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
    if (parity_io) *parity_io = parity;
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
