/*
 * amq.h -- C ABI of the B200 (sm_100a) library for alternating multi-bit quantization:
 * row-wise quantizer, bit-plane packing, binary (XNOR / bit-count) matrix product, and quantized
 * LSTM / GRU steps with the gate arithmetic fused behind the product.
 *
 * Paper: "Alternating Multi-bit Quantization for Recurrent Neural Networks".  Each entry point cites
 * the passage that defines what it computes.
 *
 * General rules
 *   - Unless an argument is documented as HOST, every pointer is a DEVICE pointer owned by the caller
 *     and valid on the device that is current when the call is made.  The library keeps no pointer
 *     after the work it enqueued has finished.  It allocates no device memory: calls that need scratch
 *     take a caller-provided workspace whose size comes from the matching *_workspace_bytes function.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls only enqueue work
 *     and return; they do not synchronise, except the *_host variants, which return after their
 *     results are in host memory.
 *   - Return value: AMQ_OK or a negative amq_status.  Invalid arguments are detected on the host before
 *     anything is launched; nothing traps or aborts.  Faults that can only be seen on the device
 *     (a bounded wait that ran out) are written to a status word at the start of the workspace and are
 *     read with amq_workspace_status.
 *   - Layouts are row-major.  1 <= k <= 4 for every bit count; n >= 1.
 *
 * Packed codes ("k planes of 32-bit words"):
 *   a length-n vector quantized to k bits is stored as k bit-planes, plane i (i = 0..k-1, the paper's
 *   b_{i+1}) in wpr = amq_words_per_row(n) = 4 * ceil(n / 128) consecutive uint32 words; bit j of word q
 *   holds element 32q + j; bit 1 means +1, bit 0 means -1; bits at positions >= n are 0.
 *   A matrix of `rows` vectors is codes[row][plane][wpr] with coefficients coeffs[row][k] (fp32).
 *   Code buffers must be 16-byte aligned (they are read with 128-bit loads).
 */
#ifndef AMQ_H
#define AMQ_H

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define AMQ_API __attribute__((visibility("default")))
#else
#define AMQ_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef int amq_status;
enum {
    AMQ_OK = 0,
    AMQ_ERR_INVALID_ARG = -1,   /* NULL where data is required, non-positive size, ld too small, aliasing */
    AMQ_ERR_UNSUPPORTED = -2,   /* k outside 1..4, T < 0, n beyond AMQ_MAX_N, batch beyond a kernel's limit */
    AMQ_ERR_ALIGNMENT = -3,     /* a code or workspace pointer is not 16-byte aligned */
    AMQ_ERR_WORKSPACE = -4,     /* workspace NULL or smaller than *_workspace_bytes */
    AMQ_ERR_CUDA = -5,          /* a CUDA runtime call failed; see amq_last_cuda_error */
    AMQ_ERR_TIMEOUT = -6        /* a bounded device-side wait ran out (reported by amq_workspace_status) */
};

#define AMQ_MAX_K 4
#define AMQ_MAX_N 8192          /* longest vector the row quantizer accepts */

/* Text for a status code (static storage, never NULL). */
AMQ_API const char* amq_status_string(amq_status s);
/* cudaError_t (as int) of the most recent failing CUDA call made by this library on this thread; 0 if none. */
AMQ_API int amq_last_cuda_error(void);

/* Number of kernels this library has enqueued so far in this process (all threads, all streams). */
AMQ_API unsigned long long amq_kernel_launches(void);

/* 4 * ceil(n / 128): 32-bit words per packed plane. */
AMQ_API int amq_words_per_row(int n);
/* rows * k * amq_words_per_row(n) * 4: bytes of a packed code buffer. */
AMQ_API size_t amq_codes_bytes(int rows, int n, int k);

/*
 * Row-wise alternating multi-bit quantization (Algorithm 2, with the greedy initialisation of Eq. 3-4,
 * the least-squares refit of Eq. 5 and the binary-search-tree code assignment of Algorithm 1).
 * Each of the `rows` rows of x is quantized on its own ("row by row", Sec. 4); the same call quantizes
 * weights offline and activations on-line.
 *   x       [rows][ldx] fp32, ldx >= n (elements).
 *   k, T    bits and alternating cycles (T >= 0; T = 0 returns the greedy solution).
 *   codes   [rows][k][wpr] uint32 out;  coeffs [rows][k] fp32 out.
 * Readings where the paper is silent: sign(0) = +1; the level table is sorted by (value, code index)
 * with plane 0 the most significant code bit; a refit whose k x k system has a pivot below 1e-9 * n
 * (Gaussian elimination with partial pivoting, in double) is skipped and keeps the previous coefficients.
 * Sums over a row are accumulated in fp32 (per thread, then across threads in a fixed order, so results repeat
 * bit for bit); B^T B is exact integer arithmetic; the k x k solve is fp64 for k >= 3 (k = 3: adjugate of the exact integers) and error-compensated fp32 for
 * k = 2; levels, thresholds and comparisons are fp32.
 */
AMQ_API amq_status amq_quantize(const float* x, int rows, int n, int ldx, int k, int T,
                        uint32_t* codes, float* coeffs, void* stream);

/*
 * Variants of the row quantizer (the comparison of Sec. 2 and Tables 1-2; the other reading of the order of
 * Algorithm 2's half steps).  Arguments, layouts and errors as amq_quantize, plus
 *   method:      AMQ_METHOD_ALTERNATING (Algorithm 2: greedy start, T cycles) or AMQ_METHOD_REFINED_GREEDY (after every
 *                greedy bit all coefficients so far are re-solved by Eq. 5; T is ignored); anything else: AMQ_ERR_UNSUPPORTED;
 *   final_refit: nonzero = one more coefficient refit (Eq. 5) on the final codes (Algorithm 2 as printed ends on the
 *                code update, so its coefficients are those of the refit BEFORE the last code update).
 * (AMQ_METHOD_ALTERNATING, 0) is amq_quantize itself; the other combinations run a general, slower kernel.
 */
#define AMQ_METHOD_ALTERNATING 0
#define AMQ_METHOD_REFINED_GREEDY 1
AMQ_API amq_status amq_quantize_variant(const float* x, int rows, int n, int ldx, int k, int T, int method, int final_refit,
                                uint32_t* codes, float* coeffs, void* stream);

/*
 * Pack sign planes given as floats into the bit layout above (storage for the XNOR / bit-count
 * product, Appendix A).  planes [rows][k][n] fp32, value >= 0 -> bit 1.  codes [rows][k][wpr] out.
 */
AMQ_API amq_status amq_pack(const float* planes, int rows, int n, int k, uint32_t* codes, void* stream);

/* Reconstruction of Eq. 2: xhat[row][t] = sum_i coeffs[row][i] * (+1 or -1).  xhat [rows][n] fp32 out. */
AMQ_API amq_status amq_unpack(const uint32_t* codes, const float* coeffs, int rows, int n, int k,
                      float* xhat, void* stream);

/*
 * Integer partials of the quantized product (Sec. 4, Fig. 3; XNOR then bit count, Appendix A):
 *   D[b][r][i][j] = B_i[r,:] . x_j[b] = n - 2 * popcount(Wcodes[r][i] xor xcodes[b][j]),   int32.
 * Wcodes [m][k_w][wpr], xcodes [batch][k_a][wpr], D [batch][m][k_w][k_a] out.  Exact.
 */
AMQ_API amq_status amq_binary_dots(const uint32_t* Wcodes, int m, int n, int k_w,
                           const uint32_t* xcodes, int batch, int k_a, int32_t* D, void* stream);

/*
 * Quantized matrix product (Sec. 4: binary product first, then the row-wise coefficients; the stacked
 * form of Fig. 3, right, for batch > 1):
 *   y[b][r] = sum_i sum_j Walpha[r][i] * xbeta[b][j] * D[b][r][i][j] + bias[r].
 * Walpha [m][k_w], xbeta [batch][k_a], bias [m] or NULL, y [batch][ldy] fp32 out, ldy >= m.
 * The integer partials are exact; the combination is fp32.
 * Wcodes and xcodes must be 16-byte aligned (AMQ_ERR_ALIGNMENT otherwise).  From 16 vectors on the product runs on
 * the tensor cores; its kernels fetch 32 bytes of a packed row at a time where the row starts on a 32-byte boundary
 * (a 32-byte aligned base with an even number of 128-element chunks per row, as torch allocations give for
 * n a multiple of 256) and fall back to 16-byte loads elsewhere: same results, about a fifth slower on large
 * products.
 */
AMQ_API amq_status amq_binary_gemm(const uint32_t* Wcodes, const float* Walpha, int m, int n, int k_w,
                           const uint32_t* xcodes, const float* xbeta, int batch, int k_a,
                           const float* bias, float* y, int ldy, void* stream);

/*
 * The operation Table 6 (Appendix A) times, in one launch: on-line quantization of ONE activation vector (Sec. 4: the
 * hidden state is quantized during inference) followed by the binary matrix-vector product with row-wise quantized
 * weights,
 *   (beta, x_j) = Algorithm 2 on x with k_a bits and T cycles;  y[r] = sum_i sum_j Walpha[r][i] beta[j] D[r][i][j] + bias[r].
 * x [n] DEVICE fp32, n <= 2048 (longer vectors: amq_quantize, then amq_binary_gemm; AMQ_ERR_UNSUPPORTED here);
 * Wcodes [m][k_w][wpr], Walpha [m][k_w], bias [m] or NULL, y [m] fp32 out.  xcodes_out [k_a][wpr] (16-byte aligned) and
 * xbeta_out [k_a], each may be NULL: the planes and coefficients of the quantized vector, for a caller that needs them
 * again (a recurrent product on the same state).  Every CTA of the product quantizes the vector for itself; the
 * arithmetic and the readings of amq_quantize apply (a different but equally fixed summation order, so codes of
 * elements on a decision boundary may differ from amq_quantize's; results repeat bit for bit from run to run).
 */
AMQ_API amq_status amq_quantized_gemv(const uint32_t* Wcodes, const float* Walpha, int m, int n, int k_w,
                              const float* x, int k_a, int T, const float* bias, float* y,
                              uint32_t* xcodes_out, float* xbeta_out, void* stream);

/*
 * Synchronises `stream`, then reads and clears the library's device-side status word of the current
 * device: AMQ_OK, or AMQ_ERR_TIMEOUT if a bounded wait inside a product kernel ran out since the last
 * read (the outputs of that call are then undefined).  Covers amq_binary_dots, amq_binary_gemm and the
 * product inside the cell calls (amq_lstm_step_static included); the sequence kernels report through
 * amq_workspace_status as well.  The word belongs to the device, not to a stream: a failure on any stream of the
 * device is reported to whoever reads next (the read is one atomic swap enqueued on `stream`), and two host threads
 * reading at the same time must be serialised by the caller.
 */
AMQ_API amq_status amq_device_status(void* stream);

/* Scratch for the cell calls below (steps and sequences), in bytes; 0 on invalid arguments. */
AMQ_API size_t amq_cell_workspace_bytes(int I, int H, int batch, int k_a);
/* Additional device staging needed by the *_host variants (x_seq, states and results), in bytes. */
AMQ_API size_t amq_cell_host_staging_bytes(int I, int H, int batch, int steps);

/*
 * One quantized LSTM step (Eq. 6) for `batch` independent sequences.
 *   W: the stacked gate matrix, 4H rows in the order i, f, o, g (the order Eq. 6 prints), I + H columns
 *      (input part first), quantized offline row by row: Wcodes [4H][k_w][wpr(I+H)], Walpha [4H][k_w].
 *   z = [x ; h_in] is quantized on-line as one vector with k_a bits and T cycles, then
 *   p = W_hat z_hat + bias;  i, f, o = logistic(p);  g = tanh(p);  c_out = f*c_in + i*g;  h_out = o*tanh(c_out).
 *   bias [4H] (b_i + b_h of Eq. 6 summed) or NULL.  x [batch][I]; h_in, c_in, h_out, c_out [batch][H] fp32.
 *   h_out must not alias h_in; c_out may alias c_in.
 */
AMQ_API amq_status amq_lstm_step(const uint32_t* Wcodes, const float* Walpha, const float* bias,
                         int I, int H, int k_w,
                         const float* x, const float* h_in, const float* c_in, int batch, int k_a, int T,
                         float* h_out, float* c_out,
                         void* workspace, size_t workspace_bytes, void* stream);

/*
 * amq_lstm_step for callers that cannot allocate device memory (no counterpart in the paper: this is a
 * packaging variant of the step above, computing the same thing).  It is meant for code that runs where
 * cudaMalloc is off limits: inside another application's fixed memory budget, in a loop that must not
 * enter the driver's allocator once it is running, or after all device memory has been handed out.
 * The scratch that amq_lstm_step takes as `workspace` (packed codes and coefficients of the quantized
 * [x ; h_in]) is a fixed array of AMQ_STATIC_SCRATCH_BYTES inside the library image; every GPU that loads
 * the library holds that much until the process exits.  The call allocates and frees nothing.
 *   - Arguments as for amq_lstm_step, without the workspace.  A problem whose scratch
 *     (amq_lstm_step_static_scratch_bytes) exceeds AMQ_STATIC_SCRATCH_BYTES is rejected with
 *     AMQ_ERR_WORKSPACE before anything is launched.
 *   - Every call looks up the array's device address for the device that is current at the call (`stream`
 *     must belong to that device).  The first call on a device also makes the runtime load the library's
 *     module there: make that first call outside any stream capture.
 *   - All calls on a device share the one array, which keeps whatever the last call left.  Each call
 *     rewrites the part it reads in full before reading it, so nothing needs clearing; but two calls
 *     whose work overlaps on the GPU (different streams, no ordering) race on it: order them.
 *   - Always runs the two-kernel chain (row quantizer, then product with the gate epilogue), for every
 *     batch size.
 */
#define AMQ_STATIC_SCRATCH_BYTES (1 << 20)
AMQ_API size_t amq_lstm_step_static_scratch_bytes(int I, int H, int batch, int k_a);
AMQ_API amq_status amq_lstm_step_static(const uint32_t* Wcodes, const float* Walpha, const float* bias,
                                int I, int H, int k_w,
                                const float* x, const float* h_in, const float* c_in, int batch, int k_a, int T,
                                float* h_out, float* c_out, void* stream);

/*
 * One quantized GRU step.  The paper names the GRU (Sec. 1, Sec. 5) without printing its equations;
 * this library computes the "linear before reset" form:
 *   W: 3H rows in the order r, z, n;  p = W_hat z_hat with z_hat the quantized [x ; h_in];
 *   for the n rows the product is kept in two column segments, p_nx over [0, I) and p_nh over [I, I+H);
 *   r = logistic(p_r + b_r);  z = logistic(p_z + b_z);  cand = tanh(p_nx + b_nx + r * (p_nh + b_nh));
 *   h_out = (1 - z) * cand + z * h_in.
 *   bias [4H] = [b_r ; b_z ; b_nx ; b_nh] or NULL.  h_out must not alias h_in.
 */
AMQ_API amq_status amq_gru_step(const uint32_t* Wcodes, const float* Walpha, const float* bias,
                        int I, int H, int k_w,
                        const float* x, const float* h_in, int batch, int k_a, int T,
                        float* h_out,
                        void* workspace, size_t workspace_bytes, void* stream);

/*
 * `steps` consecutive steps without returning to the host (step t+1 consumes h_t, so a sequence is one
 * dependency chain: Sec. 1).  x_seq [steps][batch][I]; h0, c0 [batch][H];
 * h_seq [steps][batch][H] out or NULL; h_last, c_last [batch][H] out.  Outputs must not alias inputs.
 */
AMQ_API amq_status amq_lstm_sequence(const uint32_t* Wcodes, const float* Walpha, const float* bias,
                             int I, int H, int k_w,
                             const float* x_seq, int steps, const float* h0, const float* c0,
                             int batch, int k_a, int T,
                             float* h_seq, float* h_last, float* c_last,
                             void* workspace, size_t workspace_bytes, void* stream);

AMQ_API amq_status amq_gru_sequence(const uint32_t* Wcodes, const float* Walpha, const float* bias,
                            int I, int H, int k_w,
                            const float* x_seq, int steps, const float* h0,
                            int batch, int k_a, int T,
                            float* h_seq, float* h_last,
                            void* workspace, size_t workspace_bytes, void* stream);

/*
 * GRU step in the original form of the GRU the paper cites (Cho et al., 2014; the paper prints no GRU equations):
 *   z1 = [x ; h] quantized on-line:      r = logistic(W_r z1_hat + b_r),  z = logistic(W_z z1_hat + b_z);
 *   z2 = [x ; r * h] quantized on-line:  cand = tanh(W_n z2_hat + b_n);   h' = (1 - z) * cand + z * h.
 * Wcodes / Walpha as for amq_gru_step (3H rows r, z, n over I + H columns); bias [3H] = [b_r; b_z; b_n] or NULL;
 * x [batch][I], h_in / h_out [batch][H] DEVICE fp32, h_out != h_in; workspace: DEVICE,
 * amq_gru_original_workspace_bytes(...) bytes, 16-byte aligned.  Two quantizations and two products per step
 * (amq_gru_step, which applies r after the product, needs one of each).  Errors as amq_gru_step.
 */
AMQ_API size_t amq_gru_original_workspace_bytes(int I, int H, int batch, int k_a);
AMQ_API amq_status amq_gru_step_original(const uint32_t* Wcodes, const float* Walpha, const float* bias, int I, int H, int k_w,
                                 const float* x, const float* h_in, int batch, int k_a, int T, float* h_out,
                                 void* workspace, size_t workspace_bytes, void* stream);

/*
 * The LSTM in the form the paper states it (Eq. 6 and the paragraph after it): separate matrices W_i (4H x I)
 * and W_h (4H x H), each quantized row by row; x_t is a row of the quantized embedding matrix and needs no
 * further quantization; only h_{t-1} is quantized on-line.
 *
 * amq_embedding_rows: x_t = W_e^T y*_{t-1} for one-hot tokens = gather of rows of the quantized W_e.
 *   We_codes [vocab][k][wpr(n)], We_alpha [vocab][k]; tokens [count] int32 (ids outside [0, vocab) are clamped);
 *   xcodes [count][k][wpr(n)], xbeta [count][k] out.
 */
AMQ_API amq_status amq_embedding_rows(const uint32_t* We_codes, const float* We_alpha, int vocab, int n, int k,
                              const int32_t* tokens, int count, uint32_t* xcodes, float* xbeta, void* stream);

/* Scratch of the two calls below, in bytes (steps = 1 for the step call); 0 on invalid arguments. */
AMQ_API size_t amq_lstm_paper_workspace_bytes(int H, int batch, int steps, int k_a);

/*
 * One step:  p = W_i_hat x_hat + W_h_hat h_hat + bias, gates as in amq_lstm_step (order i, f, o, g).
 *   Wi_codes [4H][k_w][wpr(I)], Wi_alpha [4H][k_w]; Wh_codes [4H][k_w][wpr(H)], Wh_alpha [4H][k_w]; bias [4H] or NULL.
 *   xcodes [batch][k_e][wpr(I)], xbeta [batch][k_e]: the inputs, already quantized (k_e bits).
 *   h_in is quantized on-line with k_a bits and T cycles.  h_out must not alias h_in; c_out may alias c_in.
 */
AMQ_API amq_status amq_lstm_step_paper(const uint32_t* Wi_codes, const float* Wi_alpha,
                               const uint32_t* Wh_codes, const float* Wh_alpha, const float* bias,
                               int I, int H, int k_w,
                               const uint32_t* xcodes, const float* xbeta, int k_e,
                               const float* h_in, const float* c_in, int batch, int k_a, int T,
                               float* h_out, float* c_out,
                               void* workspace, size_t workspace_bytes, void* stream);

/*
 * `steps` consecutive steps.  xcodes_seq [steps][batch][k_e][wpr(I)], xbeta_seq [steps][batch][k_e].
 * The input projections W_i x_t + bias of all timesteps do not depend on the state and are computed by one
 * batched binary product before the time loop; each timestep then quantizes h and multiplies by W_h only.
 * h_seq [steps][batch][H] out or NULL; h_last, c_last [batch][H] out; outputs must not alias inputs.
 */
AMQ_API amq_status amq_lstm_sequence_paper(const uint32_t* Wi_codes, const float* Wi_alpha,
                                   const uint32_t* Wh_codes, const float* Wh_alpha, const float* bias,
                                   int I, int H, int k_w,
                                   const uint32_t* xcodes_seq, const float* xbeta_seq, int k_e, int steps,
                                   const float* h0, const float* c0, int batch, int k_a, int T,
                                   float* h_seq, float* h_last, float* c_last,
                                   void* workspace, size_t workspace_bytes, void* stream);

/*
 * Output layer of Eq. 6, y_t = softmax(W_s h_t + b_s), on logits produced by amq_binary_gemm:
 *   logp[r][t] = logits[r][t] - log(sum_u exp(logits[r][u]))   (computed with the row maximum subtracted),
 *   argmax[r]  = index of the largest logit of row r (the smallest index among equal maxima).
 * logits [rows][ld] fp32, ld >= n; logp [rows][ldp] fp32 out or NULL; argmax [rows] int32 out or NULL.
 * argmax may be the `tokens` buffer of the next amq_embedding_rows call (greedy decoding without a host round trip).
 */
AMQ_API amq_status amq_log_softmax_argmax(const float* logits, int rows, int n, int ld,
                                  float* logp, int ldp, int32_t* argmax, void* stream);

/*
 * Greedy decoding with the language model of Eq. 6, one sequence, enqueued as one chain on `stream` (six or seven kernel
 * launches per token, no host round trip).  For t = 0 .. steps-1:
 *   x_t = row tokens[t] of the quantized embedding (We_codes [vocab][k_e][wpr(I)], We_alpha [vocab][k_e]);
 *   (h, c) <- LSTM step in the paper's own form (W_i [4H x I], W_h [4H x H], k_w bits, bias [4H] or NULL; h quantized
 *   on-line with k_a bits and T alternating rounds);
 *   logits = W_s h_hat + bias_s (Ws_codes [vocab][k_s][wpr(H)], Ws_alpha [vocab][k_s], bias_s [vocab] or NULL);
 *   logp[t][.] = log-softmax(logits) when logp is given; tokens[t + 1] = arg-max (first index among equal maxima).
 * tokens: DEVICE int32 [steps + 1], tokens[0] set by the caller (ids outside [0, vocab) are clamped); h, c: DEVICE
 * fp32 [H], start state in, state after the last step out; logp: DEVICE fp32 [steps][vocab] or NULL; workspace: DEVICE,
 * amq_lm_decode_workspace_bytes(...) bytes, 16-byte aligned, owned by the caller, contents undefined between calls.
 * Errors as for the calls it is made of; nothing is enqueued after the first failing launch.
 */
AMQ_API size_t amq_lm_decode_workspace_bytes(int vocab, int I, int H, int k_e, int k_a);
AMQ_API amq_status amq_lm_greedy_decode(const uint32_t* We_codes, const float* We_alpha, int vocab, int I, int k_e,
                                const uint32_t* Wi_codes, const float* Wi_alpha,
                                const uint32_t* Wh_codes, const float* Wh_alpha, const float* bias, int H, int k_w,
                                const uint32_t* Ws_codes, const float* Ws_alpha, const float* bias_s, int k_s,
                                int k_a, int T, int32_t* tokens, int steps, float* h, float* c, float* logp,
                                void* workspace, size_t workspace_bytes, void* stream);

/*
 * The sequence calls with HOST activations and results: x_seq, h0, c0 are read from host memory
 * (pinned memory makes the copies asynchronous) into `staging`, the sequence runs, and h_last / c_last
 * (and h_seq when not NULL) are copied back to host memory; the call returns after the stream has
 * drained.  Weights, bias, workspace and staging (amq_cell_host_staging_bytes) stay DEVICE pointers.
 * Inputs of 4 MiB and more of a batched sequence are copied in up to eight chunks of timesteps on a stream that
 * the call creates and destroys, so that the copy of later timesteps runs beside the kernels of earlier ones;
 * the results do not depend on it.
 */
AMQ_API amq_status amq_lstm_sequence_host(const uint32_t* Wcodes, const float* Walpha, const float* bias,
                                  int I, int H, int k_w,
                                  const float* x_seq_host, int steps, const float* h0_host, const float* c0_host,
                                  int batch, int k_a, int T,
                                  float* h_seq_host, float* h_last_host, float* c_last_host,
                                  void* workspace, size_t workspace_bytes,
                                  void* staging, size_t staging_bytes, void* stream);

AMQ_API amq_status amq_gru_sequence_host(const uint32_t* Wcodes, const float* Walpha, const float* bias,
                                 int I, int H, int k_w,
                                 const float* x_seq_host, int steps, const float* h0_host,
                                 int batch, int k_a, int T,
                                 float* h_seq_host, float* h_last_host,
                                 void* workspace, size_t workspace_bytes,
                                 void* staging, size_t staging_bytes, void* stream);

/*
 * Test aid for the give-up path of the batch-1 sequence kernel (the paper has no counterpart).  Same arguments as
 * amq_lstm_sequence with batch = 1 and steps >= 2, plus `poll_limit` (1 .. 65536): the kernel runs with that many
 * polls as the limit of every wait for the other CTAs' h values and expects step tags that no CTA ever publishes.
 * Step 0 (which waits for nothing) runs normally; in step 1 every wait runs out, every CTA records the failure in
 * the workspace status word and returns, and the outputs are left unwritten.  The call returns AMQ_OK when the launch
 * was enqueued; amq_workspace_status then returns AMQ_ERR_TIMEOUT, and the next cell call on the workspace clears it.
 * Nothing faults or hangs: the waits are the ordinary bounded ones with a smaller bound.  AMQ_ERR_UNSUPPORTED when the
 * problem is not one the batch-1 sequence kernel takes.
 */
AMQ_API amq_status amq_selftest_sequence_give_up(const uint32_t* Wcodes, const float* Walpha, const float* bias,
                                         int I, int H, int k_w,
                                         const float* x_seq, int steps, const float* h0, const float* c0,
                                         int k_a, int T, float* h_last, float* c_last,
                                         void* workspace, size_t workspace_bytes, unsigned poll_limit, void* stream);

/*
 * Synchronises `stream`, then reads the status word at the start of a cell workspace: AMQ_OK, or
 * AMQ_ERR_TIMEOUT if a bounded device-side wait gave up during a call that used this workspace.
 * The word is cleared by the next cell call.
 */
AMQ_API amq_status amq_workspace_status(const void* workspace, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* AMQ_H */
