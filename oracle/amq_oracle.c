/*
 * CPU oracle for alternating multi-bit quantization and the binary matrix product.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, double-precision statement of what the
 * method computes.  It is imported by the tests, by the smoke check and by the CPU-baseline leg of
 * the benchmark, and by nothing else.  It shares no code, header, table or helper with the CUDA
 * library, and the CUDA library never calls it.
 *
 * Every function follows one passage of the paper ("Alternating Multi-bit Quantization for
 * Recurrent Neural Networks"), cited at the function.  There is no blocking, fusion or reordering
 * beyond what that passage states.
 *
 * Conventions fixed here where the paper is silent (each is a stated reading, not the paper's text):
 *   - sign(0) = +1 (and -0.0 counts as >= 0), matching Algorithm 1's ">=" that sends ties upward.
 *   - A code index c in [0, 2^k) stands for the sign pattern s_i(c) = +1 if bit (k-i) of c is set,
 *     i = 1..k (plane 1 is the most significant bit).
 *   - The level table is sorted ascending by (value, code index).
 *   - A least-squares refit whose k x k system has a pivot below 1e-9 * n (Gaussian elimination with
 *     partial pivoting) is skipped: the coefficients keep their previous values.
 *   - Bit packing: bit j of 32-bit word q holds element 32q + j, 1 <-> +1; a packed row has
 *     4 * ceil(n / 128) words; pad bits are 0.
 *
 * Parity pins (tests/test_oracle_*.py): closed form for k = 1; Fig. 1 thresholds for k = 2;
 * exhaustive search over all code assignments; a library least-squares solve; monotone objective;
 * float dot of the +-1 vectors; dense double-precision product of the reconstructed operands;
 * textbook LSTM/GRU step.  The GRU equations are not in the paper (it only names the cell), so the
 * GRU step is "parity unpinned" by the paper: it is pinned only to the equations stated at
 * amq_oracle_gru_step.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define AMQ_ORACLE_MAX_K 8

static double sgn(double x) { return (x >= 0.0) ? 1.0 : -1.0; }

/* ---------------------------------------------------------------------------------------------
 * Greedy approximation, Eq. 3-4: r_0 = w; alpha_i = ||r_{i-1}||_1 / n; b_i = sign(r_{i-1});
 * r_i = r_{i-1} - alpha_i b_i.   b is k x n (+1/-1), alpha has k entries.
 * ------------------------------------------------------------------------------------------- */
void amq_oracle_greedy(const double* w, int n, int k, double* alpha, int8_t* b)
{
    double* r = (double*)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
    for (int t = 0; t < n; ++t) r[t] = w[t];
    for (int i = 0; i < k; ++i) {
        double l1 = 0.0;
        for (int t = 0; t < n; ++t) l1 += fabs(r[t]);
        alpha[i] = (n > 0) ? l1 / (double)n : 0.0;
        for (int t = 0; t < n; ++t) {
            double s = sgn(r[t]);
            b[(size_t)i * n + t] = (int8_t)s;
            r[t] -= alpha[i] * s;
        }
    }
    free(r);
}

/* ---------------------------------------------------------------------------------------------
 * Least-squares coefficient refit, Eq. 5: alpha = (B^T B)^{-1} B^T w with B = [b_1 .. b_k].
 * Returns 1 and overwrites alpha if the system was solved, 0 (alpha untouched) if a pivot fell
 * below 1e-9 * n  (reading for a singular Gram matrix: the paper is silent).
 * ------------------------------------------------------------------------------------------- */
int amq_oracle_ls_refit(const double* w, int n, int k, const int8_t* b, double* alpha)
{
    double G[AMQ_ORACLE_MAX_K][AMQ_ORACLE_MAX_K + 1];
    for (int i = 0; i < k; ++i) {
        for (int j = 0; j < k; ++j) {
            double s = 0.0;
            for (int t = 0; t < n; ++t) s += (double)b[(size_t)i * n + t] * (double)b[(size_t)j * n + t];
            G[i][j] = s;
        }
        double c = 0.0;
        for (int t = 0; t < n; ++t) c += (double)b[(size_t)i * n + t] * w[t];
        G[i][k] = c;
    }
    const double tiny = 1e-9 * (double)n;
    for (int col = 0; col < k; ++col) {
        int piv = col;
        for (int row = col + 1; row < k; ++row)
            if (fabs(G[row][col]) > fabs(G[piv][col])) piv = row;
        if (!(fabs(G[piv][col]) >= tiny) || fabs(G[piv][col]) == 0.0) return 0;
        if (piv != col)
            for (int j = 0; j <= k; ++j) { double tmp = G[col][j]; G[col][j] = G[piv][j]; G[piv][j] = tmp; }
        for (int row = col + 1; row < k; ++row) {
            double f = G[row][col] / G[col][col];
            for (int j = col; j <= k; ++j) G[row][j] -= f * G[col][j];
        }
    }
    double sol[AMQ_ORACLE_MAX_K];
    for (int i = k - 1; i >= 0; --i) {
        double s = G[i][k];
        for (int j = i + 1; j < k; ++j) s -= G[i][j] * sol[j];
        sol[i] = s / G[i][i];
    }
    for (int i = 0; i < k; ++i) alpha[i] = sol[i];
    return 1;
}

/* ---------------------------------------------------------------------------------------------
 * Level table (Algorithm 2, the step that lists every feasible code value in ascending order):
 * v_c = sum_i s_i(c) alpha_i for all 2^k codes, sorted ascending by (value, code index).
 * v and code have 2^k entries.
 * ------------------------------------------------------------------------------------------- */
void amq_oracle_levels(const double* alpha, int k, double* v, int* code)
{
    int m = 1 << k;
    for (int c = 0; c < m; ++c) {
        double s = 0.0;
        for (int i = 0; i < k; ++i) s += ((c >> (k - 1 - i)) & 1) ? alpha[i] : -alpha[i];
        v[c] = s;
        code[c] = c;
    }
    /* insertion sort: stable, so equal values stay in code order */
    for (int a = 1; a < m; ++a) {
        double va = v[a]; int ca = code[a]; int p = a - 1;
        while (p >= 0 && v[p] > va) { v[p + 1] = v[p]; code[p + 1] = code[p]; --p; }
        v[p + 1] = va; code[p + 1] = ca;
    }
}

/* ---------------------------------------------------------------------------------------------
 * Algorithm 1 (binary search tree over the ascending table v of 2^k levels), for one entry w: k
 * levels of descent.  A node owns a window of table positions [first, first + 2 * half); the entry
 * moves into the upper half of the window exactly when it is at least the midpoint between the
 * largest level of the lower half and the smallest level of the upper half (so an entry on a
 * midpoint goes up).  After k levels the window is one position: the level assigned to w.
 * ------------------------------------------------------------------------------------------- */
static int bst_position(double w, const double* v, int k)
{
    int first = 0;
    for (int half = (1 << k) >> 1; half >= 1; half >>= 1) {
        double boundary = 0.5 * (v[first + half - 1] + v[first + half]);
        if (w >= boundary) first += half;
    }
    return first;
}

/* Code update of Algorithm 2 via Algorithm 1, for every entry, coefficients fixed. */
void amq_oracle_bst(const double* w, int n, int k, const double* alpha, int8_t* b)
{
    double v[1 << AMQ_ORACLE_MAX_K];
    int code[1 << AMQ_ORACLE_MAX_K];
    amq_oracle_levels(alpha, k, v, code);
    for (int t = 0; t < n; ++t) {
        int c = code[bst_position(w[t], v, k)];
        for (int i = 0; i < k; ++i) b[(size_t)i * n + t] = ((c >> (k - 1 - i)) & 1) ? 1 : -1;
    }
}

/* Objective of Eq. 2: || w - sum_i alpha_i b_i ||^2. */
double amq_oracle_objective(const double* w, int n, int k, const double* alpha, const int8_t* b)
{
    double s = 0.0;
    for (int t = 0; t < n; ++t) {
        double q = 0.0;
        for (int i = 0; i < k; ++i) q += alpha[i] * (double)b[(size_t)i * n + t];
        s += (w[t] - q) * (w[t] - q);
    }
    return s;
}

/* ---------------------------------------------------------------------------------------------
 * Algorithm 2: greedy initialisation, then T times { refit alpha (Eq. 5); build v; update b by
 * Algorithm 1 }.  Returned alpha is from the last refit, b from the last code update, the order the
 * algorithm prints.  trace (may be NULL) receives 1 + 2T objective values: after the greedy step and
 * after every half step.
 * ------------------------------------------------------------------------------------------- */
void amq_oracle_quantize(const double* w, int n, int k, int T, double* alpha, int8_t* b, double* trace)
{
    amq_oracle_greedy(w, n, k, alpha, b);
    if (trace) trace[0] = amq_oracle_objective(w, n, k, alpha, b);
    for (int it = 0; it < T; ++it) {
        amq_oracle_ls_refit(w, n, k, b, alpha);
        if (trace) trace[1 + 2 * it] = amq_oracle_objective(w, n, k, alpha, b);
        amq_oracle_bst(w, n, k, alpha, b);
        if (trace) trace[2 + 2 * it] = amq_oracle_objective(w, n, k, alpha, b);
    }
}

/* Refined greedy approximation (comparison method of Sec. 2(d)): after each greedy bit j, refit
 * alpha_1..alpha_j by Eq. 5; codes are never revisited.  Kept only for the ordering check
 * error(alternating) <= error(refined) <= error(greedy). */
void amq_oracle_refined_greedy(const double* w, int n, int k, double* alpha, int8_t* b)
{
    double* r = (double*)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
    for (int t = 0; t < n; ++t) r[t] = w[t];
    for (int j = 0; j < k; ++j) {
        double l1 = 0.0;
        for (int t = 0; t < n; ++t) l1 += fabs(r[t]);
        alpha[j] = (n > 0) ? l1 / (double)n : 0.0;
        for (int t = 0; t < n; ++t) b[(size_t)j * n + t] = (int8_t)sgn(r[t]);
        amq_oracle_ls_refit(w, n, j + 1, b, alpha);
        for (int t = 0; t < n; ++t) {
            double q = 0.0;
            for (int i = 0; i <= j; ++i) q += alpha[i] * (double)b[(size_t)i * n + t];
            r[t] = w[t] - q;
        }
    }
    free(r);
}

/* Variants of the quantizer (Sec. 2-3), for the comparison of Tables 1-2 and for the other reading of the
 * order of the two half steps:
 *   method 0: Algorithm 2 (greedy start, T alternating cycles); method 1: refined greedy (T ignored);
 *   final_refit != 0: one more coefficient refit (Eq. 5) on the final codes, so that the returned alpha is
 *   optimal for the returned b (Algorithm 2 as printed ends on the code update instead). */
void amq_oracle_quantize_variant(const double* w, int n, int k, int T, int method, int final_refit,
                                 double* alpha, int8_t* b)
{
    if (method == 1) amq_oracle_refined_greedy(w, n, k, alpha, b);
    else amq_oracle_quantize(w, n, k, T, alpha, b, NULL);
    if (final_refit) amq_oracle_ls_refit(w, n, k, b, alpha);
}

void amq_oracle_quantize_rows_variant(const double* x, int rows, int n, int ldx, int k, int T, int method,
                                      int final_refit, uint32_t* codes, double* coeffs)
{
    int wpr = 4 * ((n + 127) / 128);
    int8_t* b = (int8_t*)malloc((size_t)k * (size_t)(n > 0 ? n : 1));
    for (int r = 0; r < rows; ++r) {
        amq_oracle_quantize_variant(x + (size_t)r * ldx, n, k, T, method, final_refit, coeffs + (size_t)r * k, b);
        for (int i = 0; i < k; ++i) {
            uint32_t* words = codes + ((size_t)r * k + i) * wpr;
            for (int q = 0; q < wpr; ++q) words[q] = 0u;
            for (int t = 0; t < n; ++t)
                if (b[(size_t)i * n + t] > 0) words[t >> 5] |= 1u << (t & 31);
        }
    }
    free(b);
}

/* ---------------------------------------------------------------------------------------------
 * Bit packing of one +-1 plane (storage for the XNOR / bitcount product of Appendix A).
 * ------------------------------------------------------------------------------------------- */
int amq_oracle_words_per_row(int n) { return 4 * ((n + 127) / 128); }

void amq_oracle_pack_plane(const int8_t* b, int n, uint32_t* words)
{
    int wpr = amq_oracle_words_per_row(n);
    for (int q = 0; q < wpr; ++q) words[q] = 0u;
    for (int t = 0; t < n; ++t)
        if (b[t] > 0) words[t / 32] |= (1u << (t % 32));
}

void amq_oracle_unpack_plane(const uint32_t* words, int n, int8_t* b)
{
    for (int t = 0; t < n; ++t) b[t] = ((words[t / 32] >> (t % 32)) & 1u) ? 1 : -1;
}

static int popcount32(uint32_t x)
{
    int c = 0;
    while (x) { x &= x - 1u; ++c; }
    return c;
}

/* +-1 dot product as the paper's kernel computes it (Appendix A): XNOR then bit count, i.e.
 * n - 2 * popcount(a xor b) over bits [lo, hi) of the packed planes. */
int32_t amq_oracle_dot_xnor_range(const uint32_t* a, const uint32_t* b, int lo, int hi)
{
    int32_t diff = 0;
    for (int q = lo / 32; q * 32 < hi; ++q) {
        uint32_t x = a[q] ^ b[q];
        int first = q * 32;
        uint32_t mask = 0xFFFFFFFFu;
        if (lo > first) mask &= 0xFFFFFFFFu << (lo - first);
        if (hi < first + 32) mask &= 0xFFFFFFFFu >> (first + 32 - hi);
        diff += popcount32(x & mask);
    }
    return (int32_t)(hi - lo) - 2 * diff;
}

int32_t amq_oracle_dot_xnor(const uint32_t* a, const uint32_t* b, int n)
{
    return amq_oracle_dot_xnor_range(a, b, 0, n);
}

/* The same dot product from its definition: sum_t a_t b_t on the unpacked +-1 vectors. */
double amq_oracle_dot_pm1(const int8_t* a, const int8_t* b, int n)
{
    double s = 0.0;
    for (int t = 0; t < n; ++t) s += (double)a[t] * (double)b[t];
    return s;
}

/* ---------------------------------------------------------------------------------------------
 * Row-wise quantization of a matrix ("row by row", Sec. 4): each of the `rows` rows of x (row
 * stride ldx) gets its own k coefficients and k packed planes.
 *   codes  [row][plane][wpr] uint32,  coeffs [row][k] double.
 * ------------------------------------------------------------------------------------------- */
void amq_oracle_quantize_rows(const double* x, int rows, int n, int ldx, int k, int T,
                              uint32_t* codes, double* coeffs)
{
    int wpr = amq_oracle_words_per_row(n);
    int8_t* b = (int8_t*)malloc((size_t)k * (size_t)(n > 0 ? n : 1));
    for (int r = 0; r < rows; ++r) {
        amq_oracle_quantize(x + (size_t)r * ldx, n, k, T, coeffs + (size_t)r * k, b, NULL);
        for (int i = 0; i < k; ++i)
            amq_oracle_pack_plane(b + (size_t)i * n, n, codes + ((size_t)r * k + i) * wpr);
    }
    free(b);
}

/* ---------------------------------------------------------------------------------------------
 * Integer partials of the quantized product (Sec. 4 and Fig. 3):
 *   D[bt][r][i][j] = B_i[r,:] . x_j[bt]  = n - 2 popcount(xor), over columns [lo, hi).
 * Wcodes [m][k_w][wpr], xcodes [batch][k_a][wpr].
 * ------------------------------------------------------------------------------------------- */
void amq_oracle_binary_dots_range(const uint32_t* Wcodes, int m, int n, int k_w,
                                  const uint32_t* xcodes, int batch, int k_a,
                                  int lo, int hi, int32_t* D)
{
    int wpr = amq_oracle_words_per_row(n);
    for (int bt = 0; bt < batch; ++bt)
        for (int r = 0; r < m; ++r)
            for (int i = 0; i < k_w; ++i)
                for (int j = 0; j < k_a; ++j)
                    D[(((size_t)bt * m + r) * k_w + i) * k_a + j] = amq_oracle_dot_xnor_range(
                        Wcodes + ((size_t)r * k_w + i) * wpr, xcodes + ((size_t)bt * k_a + j) * wpr, lo, hi);
}

void amq_oracle_binary_dots(const uint32_t* Wcodes, int m, int n, int k_w,
                            const uint32_t* xcodes, int batch, int k_a, int32_t* D)
{
    amq_oracle_binary_dots_range(Wcodes, m, n, k_w, xcodes, batch, k_a, 0, n, D);
}

/* Quantized product (Sec. 4): y[bt][r] = sum_i sum_j alpha_{r,i} beta_{bt,j} (B_i[r,:] . x_j[bt]) + bias[r],
 * restricted to columns [lo, hi) of the operands.  bias may be NULL. */
void amq_oracle_binary_gemm_range(const uint32_t* Wcodes, const double* Walpha, int m, int n, int k_w,
                                  const uint32_t* xcodes, const double* xbeta, int batch, int k_a,
                                  const double* bias, int lo, int hi, double* y)
{
    int wpr = amq_oracle_words_per_row(n);
    for (int bt = 0; bt < batch; ++bt)
        for (int r = 0; r < m; ++r) {
            double s = 0.0;
            for (int i = 0; i < k_w; ++i)
                for (int j = 0; j < k_a; ++j) {
                    int32_t d = amq_oracle_dot_xnor_range(Wcodes + ((size_t)r * k_w + i) * wpr,
                                                          xcodes + ((size_t)bt * k_a + j) * wpr, lo, hi);
                    s += Walpha[(size_t)r * k_w + i] * xbeta[(size_t)bt * k_a + j] * (double)d;
                }
            y[(size_t)bt * m + r] = s + (bias ? bias[r] : 0.0);
        }
}

void amq_oracle_binary_gemm(const uint32_t* Wcodes, const double* Walpha, int m, int n, int k_w,
                            const uint32_t* xcodes, const double* xbeta, int batch, int k_a,
                            const double* bias, double* y)
{
    amq_oracle_binary_gemm_range(Wcodes, Walpha, m, n, k_w, xcodes, xbeta, batch, k_a, bias, 0, n, y);
}

static double logistic(double x) { return 1.0 / (1.0 + exp(-x)); }

/* ---------------------------------------------------------------------------------------------
 * One quantized LSTM step, Eq. 6, for `batch` independent sequences.
 *   W: stacked gate matrix, 4H rows in the order i, f, o, g, n = I + H columns (the input part first),
 *      given as packed codes + per-row coefficients (quantized offline, row by row).
 *   z = [x ; h] is quantized on-line with k_a bits and T cycles (one group over the whole vector:
 *      a reading; the paper quantizes h_t and takes x_t from a quantized embedding row).
 *   i, f, o use the logistic function and g uses tanh (reading of "sigma represents the activation
 *      function"); one bias vector of 4H (b_i + b_h summed), may be NULL.
 *   c' = f * c + i * g ;  h' = o * tanh(c').
 * x [batch][I], h/c [batch][H] double.
 * ------------------------------------------------------------------------------------------- */
void amq_oracle_lstm_step(const uint32_t* Wcodes, const double* Walpha, const double* bias,
                          int I, int H, int k_w, const double* x, const double* h_in, const double* c_in,
                          int batch, int k_a, int T, double* h_out, double* c_out)
{
    int n = I + H, m = 4 * H, wpr = amq_oracle_words_per_row(n);
    double* z = (double*)malloc(sizeof(double) * (size_t)n);
    double* p = (double*)malloc(sizeof(double) * (size_t)m);
    uint32_t* zc = (uint32_t*)malloc(sizeof(uint32_t) * (size_t)k_a * wpr);
    double beta[AMQ_ORACLE_MAX_K];
    for (int bt = 0; bt < batch; ++bt) {
        for (int t = 0; t < I; ++t) z[t] = x[(size_t)bt * I + t];
        for (int t = 0; t < H; ++t) z[I + t] = h_in[(size_t)bt * H + t];
        amq_oracle_quantize_rows(z, 1, n, n, k_a, T, zc, beta);
        amq_oracle_binary_gemm(Wcodes, Walpha, m, n, k_w, zc, beta, 1, k_a, bias, p);
        for (int u = 0; u < H; ++u) {
            double ig = logistic(p[u]), fg = logistic(p[H + u]), og = logistic(p[2 * H + u]);
            double gg = tanh(p[3 * H + u]);
            double c = fg * c_in[(size_t)bt * H + u] + ig * gg;
            c_out[(size_t)bt * H + u] = c;
            h_out[(size_t)bt * H + u] = og * tanh(c);
        }
    }
    free(z); free(p); free(zc);
}

/* ---------------------------------------------------------------------------------------------
 * One quantized LSTM step in the form the paper states it (Eq. 6 and the text after it): two weight
 * matrices W_i (4H x I) and W_h (4H x H), each quantized row by row on its own; x_t is a row of the
 * quantized embedding W_e and is used as it is (Sec. 4), so it arrives as k_e packed planes with
 * coefficients; only h_{t-1} is quantized on-line (k_a bits, T cycles).
 *   p = W_i_hat x_hat + W_h_hat h_hat + bias;  i, f, o = logistic(p), g = tanh(p) (gate order i, f, o, g);
 *   c' = f * c + i * g;  h' = o * tanh(c').
 * xcodes [batch][k_e][wpr(I)], xbeta [batch][k_e]; h/c [batch][H] double; bias 4H or NULL.
 * ------------------------------------------------------------------------------------------- */
void amq_oracle_lstm_step_paper(const uint32_t* Wi_codes, const double* Wi_alpha,
                                const uint32_t* Wh_codes, const double* Wh_alpha, const double* bias,
                                int I, int H, int k_w, const uint32_t* xcodes, const double* xbeta, int k_e,
                                const double* h_in, const double* c_in, int batch, int k_a, int T,
                                double* h_out, double* c_out)
{
    int m = 4 * H, wpr_i = amq_oracle_words_per_row(I), wpr_h = amq_oracle_words_per_row(H);
    double* pi = (double*)malloc(sizeof(double) * (size_t)m);
    double* ph = (double*)malloc(sizeof(double) * (size_t)m);
    uint32_t* hc = (uint32_t*)malloc(sizeof(uint32_t) * (size_t)k_a * wpr_h);
    double beta[AMQ_ORACLE_MAX_K];
    for (int bt = 0; bt < batch; ++bt) {
        amq_oracle_quantize_rows(h_in + (size_t)bt * H, 1, H, H, k_a, T, hc, beta);
        amq_oracle_binary_gemm(Wi_codes, Wi_alpha, m, I, k_w, xcodes + (size_t)bt * k_e * wpr_i,
                               xbeta + (size_t)bt * k_e, 1, k_e, NULL, pi);
        amq_oracle_binary_gemm(Wh_codes, Wh_alpha, m, H, k_w, hc, beta, 1, k_a, NULL, ph);
        for (int u = 0; u < H; ++u) {
            double p4[4];
            for (int g = 0; g < 4; ++g) p4[g] = pi[g * H + u] + ph[g * H + u] + (bias ? bias[g * H + u] : 0.0);
            double ig = logistic(p4[0]), fg = logistic(p4[1]), og = logistic(p4[2]), gg = tanh(p4[3]);
            double c = fg * c_in[(size_t)bt * H + u] + ig * gg;
            c_out[(size_t)bt * H + u] = c;
            h_out[(size_t)bt * H + u] = og * tanh(c);
        }
    }
    free(pi); free(ph); free(hc);
}

/* ---------------------------------------------------------------------------------------------
 * One quantized GRU step.  The paper names the GRU but prints no equations; this is the common
 * "linear before reset" form (a stated reading, not the paper's text):
 *   W: 3H rows in the order r, z, n; p = W_hat z_hat with z_hat the quantized [x ; h];
 *   for the n rows the product is split at column I:  p_n^x over [0, I),  p_n^h over [I, I+H);
 *   r = logistic(p_r + b_r);  z = logistic(p_z + b_z);
 *   cand = tanh(p_n^x + b_nx + r * (p_n^h + b_nh));  h' = (1 - z) * cand + z * h.
 * bias has 4H entries [b_r; b_z; b_nx; b_nh] or is NULL.
 * ------------------------------------------------------------------------------------------- */
void amq_oracle_gru_step(const uint32_t* Wcodes, const double* Walpha, const double* bias,
                         int I, int H, int k_w, const double* x, const double* h_in,
                         int batch, int k_a, int T, double* h_out)
{
    int n = I + H, m = 3 * H, wpr = amq_oracle_words_per_row(n);
    double* z = (double*)malloc(sizeof(double) * (size_t)n);
    double* px = (double*)malloc(sizeof(double) * (size_t)m);
    double* ph = (double*)malloc(sizeof(double) * (size_t)m);
    uint32_t* zc = (uint32_t*)malloc(sizeof(uint32_t) * (size_t)k_a * wpr);
    double beta[AMQ_ORACLE_MAX_K];
    for (int bt = 0; bt < batch; ++bt) {
        for (int t = 0; t < I; ++t) z[t] = x[(size_t)bt * I + t];
        for (int t = 0; t < H; ++t) z[I + t] = h_in[(size_t)bt * H + t];
        amq_oracle_quantize_rows(z, 1, n, n, k_a, T, zc, beta);
        amq_oracle_binary_gemm_range(Wcodes, Walpha, m, n, k_w, zc, beta, 1, k_a, NULL, 0, I, px);
        amq_oracle_binary_gemm_range(Wcodes, Walpha, m, n, k_w, zc, beta, 1, k_a, NULL, I, n, ph);
        for (int u = 0; u < H; ++u) {
            double br = bias ? bias[u] : 0.0, bz = bias ? bias[H + u] : 0.0;
            double bnx = bias ? bias[2 * H + u] : 0.0, bnh = bias ? bias[3 * H + u] : 0.0;
            double rg = logistic(px[u] + ph[u] + br);
            double zg = logistic(px[H + u] + ph[H + u] + bz);
            double cand = tanh(px[2 * H + u] + bnx + rg * (ph[2 * H + u] + bnh));
            h_out[(size_t)bt * H + u] = (1.0 - zg) * cand + zg * h_in[(size_t)bt * H + u];
        }
    }
    free(z); free(px); free(ph); free(zc);
}

/* ---------------------------------------------------------------------------------------------
 * One quantized GRU step in the original form of the GRU the paper cites (Cho et al., 2014): the reset gate
 * multiplies the previous state BEFORE the candidate's product, so the step quantizes two vectors on-line:
 *   z1 = [x ; h]:      r = logistic(W_r z1_hat + b_r),  z = logistic(W_z z1_hat + b_z);
 *   z2 = [x ; r * h]:  cand = tanh(W_n z2_hat + b_n);   h' = (1 - z) * cand + z * h.
 * W: 3H rows in the order r, z, n over n = I + H columns; bias has 3H entries [b_r; b_z; b_n] or is NULL.
 * ------------------------------------------------------------------------------------------- */
void amq_oracle_gru_step_original(const uint32_t* Wcodes, const double* Walpha, const double* bias,
                                  int I, int H, int k_w, const double* x, const double* h_in,
                                  int batch, int k_a, int T, double* h_out)
{
    int n = I + H, wpr = amq_oracle_words_per_row(n);
    double* z = (double*)malloc(sizeof(double) * (size_t)n);
    double* p = (double*)malloc(sizeof(double) * (size_t)3 * H);
    double* pn = (double*)malloc(sizeof(double) * (size_t)H);
    uint32_t* zc = (uint32_t*)malloc(sizeof(uint32_t) * (size_t)k_a * wpr);
    double beta[AMQ_ORACLE_MAX_K];
    for (int bt = 0; bt < batch; ++bt) {
        const double* h = h_in + (size_t)bt * H;
        for (int t = 0; t < I; ++t) z[t] = x[(size_t)bt * I + t];
        for (int t = 0; t < H; ++t) z[I + t] = h[t];
        amq_oracle_quantize_rows(z, 1, n, n, k_a, T, zc, beta);
        amq_oracle_binary_gemm(Wcodes, Walpha, 2 * H, n, k_w, zc, beta, 1, k_a, bias, p);      /* rows r, z */
        for (int u = 0; u < H; ++u) z[I + u] = logistic(p[u]) * h[u];                          /* r * h */
        amq_oracle_quantize_rows(z, 1, n, n, k_a, T, zc, beta);
        amq_oracle_binary_gemm(Wcodes + (size_t)2 * H * k_w * wpr, Walpha + (size_t)2 * H * k_w, H, n, k_w,
                               zc, beta, 1, k_a, bias ? bias + 2 * H : NULL, pn);               /* rows n */
        for (int u = 0; u < H; ++u) {
            double zg = logistic(p[H + u]);
            h_out[(size_t)bt * H + u] = (1.0 - zg) * tanh(pn[u]) + zg * h[u];
        }
    }
    free(z); free(p); free(pn); free(zc);
}

/* ---------------------------------------------------------------------------------------------
 * Output layer of Eq. 6: y = softmax(W_s h + b_s), stated here on given logits: log-probabilities
 * logp[t] = z[t] - max - log(sum_u exp(z[u] - max)) and the index of the largest logit (the first
 * one among equal maxima).  Plain definition, fp64.
 * ------------------------------------------------------------------------------------------- */
void amq_oracle_log_softmax_argmax(const double* z, int rows, int n, double* logp, int32_t* arg)
{
    for (int r = 0; r < rows; ++r) {
        const double* zr = z + (size_t)r * n;
        double mx = zr[0];
        int am = 0;
        for (int t = 1; t < n; ++t) if (zr[t] > mx) { mx = zr[t]; am = t; }
        double sum = 0.0;
        for (int t = 0; t < n; ++t) sum += exp(zr[t] - mx);
        double lse = mx + log(sum);
        for (int t = 0; t < n; ++t) logp[(size_t)r * n + t] = zr[t] - lse;
        arg[r] = am;
    }
}

/* Sequences: `steps` applications of the step above, from (h0, c0); x_seq is [steps][batch][I].
 * h_seq (may be NULL) receives every h_t as [steps][batch][H]. */
void amq_oracle_lstm_sequence(const uint32_t* Wcodes, const double* Walpha, const double* bias,
                              int I, int H, int k_w, const double* x_seq, int steps,
                              const double* h0, const double* c0, int batch, int k_a, int T,
                              double* h_seq, double* h_last, double* c_last)
{
    size_t sz = (size_t)batch * H;
    double* h = (double*)malloc(sizeof(double) * sz * 2);
    double* c = (double*)malloc(sizeof(double) * sz * 2);
    memcpy(h, h0, sizeof(double) * sz);
    memcpy(c, c0, sizeof(double) * sz);
    for (int s = 0; s < steps; ++s) {
        amq_oracle_lstm_step(Wcodes, Walpha, bias, I, H, k_w, x_seq + (size_t)s * batch * I, h, c,
                             batch, k_a, T, h + sz, c + sz);
        memcpy(h, h + sz, sizeof(double) * sz);
        memcpy(c, c + sz, sizeof(double) * sz);
        if (h_seq) memcpy(h_seq + (size_t)s * sz, h, sizeof(double) * sz);
    }
    memcpy(h_last, h, sizeof(double) * sz);
    memcpy(c_last, c, sizeof(double) * sz);
    free(h); free(c);
}

void amq_oracle_gru_sequence(const uint32_t* Wcodes, const double* Walpha, const double* bias,
                             int I, int H, int k_w, const double* x_seq, int steps,
                             const double* h0, int batch, int k_a, int T,
                             double* h_seq, double* h_last)
{
    size_t sz = (size_t)batch * H;
    double* h = (double*)malloc(sizeof(double) * sz * 2);
    memcpy(h, h0, sizeof(double) * sz);
    for (int s = 0; s < steps; ++s) {
        amq_oracle_gru_step(Wcodes, Walpha, bias, I, H, k_w, x_seq + (size_t)s * batch * I, h,
                            batch, k_a, T, h + sz);
        memcpy(h, h + sz, sizeof(double) * sz);
        if (h_seq) memcpy(h_seq + (size_t)s * sz, h, sizeof(double) * sz);
    }
    memcpy(h_last, h, sizeof(double) * sz);
    free(h);
}

/* ---------------------------------------------------------------------------------------------
 * Operation-count model of Sec. 3 (quantizer) and Sec. 4 (product).
 *   quantizer: 2 T k^2 n binary + 2 (T + 1) k n non-binary operations;
 *   product (T = 2): 2 k_w k_h m n + 4 k_h^2 n binary, 6 k_h n + 2 k_w k_h m non-binary;
 *   gamma = 2 m n / (binary / 32 + non-binary).  The printed "4 k_n^2 n" is read as 4 k_h^2 n.
 * ------------------------------------------------------------------------------------------- */
void amq_oracle_quantizer_ops(int n, int k, int T, double* binary_ops, double* nonbinary_ops)
{
    *binary_ops = 2.0 * T * k * k * n;
    *nonbinary_ops = 2.0 * (T + 1) * k * n;
}

double amq_oracle_gamma(int m, int n, int k_w, int k_h)
{
    double bin = 2.0 * k_w * k_h * (double)m * n + 4.0 * k_h * k_h * n;
    double non = 6.0 * k_h * n + 2.0 * k_w * k_h * (double)m;
    return 2.0 * (double)m * n / (bin / 32.0 + non);
}
