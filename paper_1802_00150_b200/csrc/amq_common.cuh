// Shared host/device helpers of the CUDA library (status handling, sizes, small device utilities).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "amq.h"

namespace amq {

// Last failing CUDA call of this thread (read through amq_last_cuda_error).
extern thread_local int g_last_cuda_error;

inline amq_status cuda_fail(cudaError_t e)
{
    g_last_cuda_error = (int)e;
    return AMQ_ERR_CUDA;
}

#define AMQ_CUDA_TRY(expr)                                    \
    do {                                                      \
        cudaError_t amq_e_ = (expr);                          \
        if (amq_e_ != cudaSuccess) return ::amq::cuda_fail(amq_e_); \
    } while (0)

// Kernels enqueued by this library (read through amq_kernel_launches).
extern unsigned long long g_kernel_launches;

#define AMQ_LAUNCH_CHECK()                               \
    do {                                                 \
        __atomic_fetch_add(&::amq::g_kernel_launches, 1ull, __ATOMIC_RELAXED); \
        AMQ_CUDA_TRY(cudaGetLastError());                \
    } while (0)

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool valid_k(int k) { return k >= 1 && k <= AMQ_MAX_K; }
inline int words_per_row(int n) { return 4 * ((n + 127) / 128); }
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Copies of the h exchange buffer of the persistent batch-1 kernel: every producer writes each copy, a CTA polls
// copy blockIdx.x % copies, which spreads the polling over that many times more L2 lines.
constexpr int PERSISTENT_EXCHANGE_COPIES = 8;
// words per copy: H rounded up to whole 128-byte lines, so every copy starts on a line
inline size_t persistent_exchange_stride(int H) { return ((size_t)H + 15) / 16 * 16; }

// Layout of a cell workspace: [status block][exchange words][z codes][z coefficients][h ping][h pong][c].
struct CellWorkspace {
    uint32_t* status;   // 64 words: [0] status, [1..] barrier counters
    uint32_t* zcodes;   // [batch][k_a][wpr]
    float* zbeta;       // [batch][k_a]
    float* h[2];        // [batch][H] each
    float* c;           // [batch][H]
    unsigned long long* hx;   // [2][copies][H] exchange words {fp32 bits, step tag} of the persistent kernel
    size_t hx_bytes;
    size_t bytes;
};

inline CellWorkspace carve_cell_workspace(void* base, int I, int H, int batch, int k_a)
{
    CellWorkspace w;
    char* p = static_cast<char*>(base);
    size_t off = 0;
    w.status = reinterpret_cast<uint32_t*>(p + off);            off += 256;
    // the exchange words directly behind the status words: one memset clears both before a sequence
    w.hx = reinterpret_cast<unsigned long long*>(p + off);
    w.hx_bytes = batch == 1 ? round_up((size_t)2 * PERSISTENT_EXCHANGE_COPIES * persistent_exchange_stride(H) * 8, 256) : 0;   // batch 1 only
    off += w.hx_bytes;
    w.zcodes = reinterpret_cast<uint32_t*>(p + off);            off += round_up((size_t)batch * k_a * words_per_row(I + H) * 4, 256);
    w.zbeta = reinterpret_cast<float*>(p + off);                off += round_up((size_t)batch * k_a * 4, 256);
    w.h[0] = reinterpret_cast<float*>(p + off);                 off += round_up((size_t)batch * H * 4, 256);
    w.h[1] = reinterpret_cast<float*>(p + off);                 off += round_up((size_t)batch * H * 4, 256);
    w.c = reinterpret_cast<float*>(p + off);                    off += round_up((size_t)batch * H * 4, 256);
    w.bytes = off;
    return w;
}

// ---- launchers implemented in the .cu files (device pointers, already validated) -----------------------

// Quantize `rows` vectors; element t of row r is src0[r*ld0 + t] for t < n0, else src1[r*ld1 + t - n0].
amq_status launch_quantize(const float* src0, int ld0, int n0, const float* src1, int ld1, int n1,
                           int rows, int k, int T, uint32_t* codes, float* coeffs, cudaStream_t st,
                           bool overlap_with_previous = false);

enum Epilogue { EPI_DOTS = 0, EPI_Y = 1, EPI_LSTM = 2, EPI_GRU = 3 };

struct GemmArgs {
    const uint32_t* Wcodes; const float* Walpha; int m, n, k_w;
    const uint32_t* xcodes; const float* xbeta; int batch, k_a;
    const float* bias;
    int epilogue;
    // EPI_DOTS
    int32_t* D;
    // EPI_Y
    float* y; int ldy;
    // EPI_LSTM / EPI_GRU
    int I, H;
    const float* h_in; const float* c_in; float* h_out; float* c_out;
    // EPI_LSTM only: optional pre-activations computed elsewhere (e.g. W_i x), added before the gates;
    // addend[b * ld_addend + gate * H + unit]
    const float* addend; int ld_addend;
    // the launch may start while the previous kernel of the stream (the on-line quantizer that produces xcodes / xbeta)
    // still runs: the kernel sets itself up, fetches weights, and waits for that kernel before it reads anything else
    bool overlap_with_previous;
};

// programmatic dependent launch (sm_90+): a kernel launched with the programmatic-serialization attribute may have its
// CTAs scheduled as the CTAs of the preceding kernel of the stream exit; `grid_dependency_wait` returns once that kernel
// has completed and its writes are visible (at once when the launch was an ordinary one).  No kernel here signals
// earlier than its exit: measured, early signals only made the waiting CTAs take SM resources sooner.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Launch `kernel`, as a programmatic dependent of the preceding kernel of the stream when `overlap` is set (the kernel
// must then execute grid_dependency_wait() before it reads or writes anything another kernel of the chain touches,
// and read such data with ordinary loads, not through the read-only path).
template <typename... Params, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool overlap,
                                 Args... args)
{
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr; cfg.numAttrs = overlap ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<Params>(args)...);
}

amq_status launch_binary_gemm(const GemmArgs& a, cudaStream_t st);
// whether the tensor-core kernel takes the problem with all its CTAs resident at once (then the quantizer of the next
// timestep is launched as its programmatic dependent: its CTAs move in as the product's CTAs exit)
bool gemm_tc_single_wave(const GemmArgs& a);

// Batch-1 streaming kernel (EPI_DOTS / EPI_Y): whether it covers a problem, and its launch.
// gates of Eq. 6 for one sequence from pre-activations pre[4H] (+ addend[4H] when given), rows i, f, o, g
amq_status launch_lstm_gates(const float* pre, const float* addend, const float* c_in, float* h_out, float* c_out, int H,
                             cudaStream_t st, bool overlap_with_previous = false);
// gather of rows of a quantized embedding / log-softmax and arg-max of rows of logits (validated arguments)
amq_status launch_embedding_rows(const uint32_t* We_codes, const float* We_alpha, int vocab, int n, int k, const int32_t* tokens,
                                 int count, uint32_t* xcodes, float* xbeta, cudaStream_t st, bool overlap_with_previous);
amq_status launch_log_softmax_argmax(const float* logits, int rows, int n, int ld, float* logp, int ldp, int32_t* argmax,
                                     cudaStream_t st, bool overlap_with_previous);
bool gemv_supported(const GemmArgs& a);
amq_status launch_binary_gemv(const GemmArgs& a, cudaStream_t st);
// Fused form for one vector of up to 2048 elements: on-line quantization (k_a bits, T cycles) inside the product kernel;
// xcodes_out [k_a][wpr] / xbeta_out [k_a] (may be null) receive the planes and coefficients.
bool quantized_gemv_supported(int n);
amq_status launch_quantized_gemv(const uint32_t* Wcodes, const float* Walpha, int m, int n, int k_w, const float* x, int k_a, int T,
                                 const float* bias, float* y, uint32_t* xcodes_out, float* xbeta_out, cudaStream_t st,
                                 bool overlap_with_previous);

// Tensor-core kernel (tcgen05, batch >= 16): whether it covers a problem, its launch, and its status word
// (nonzero after a bounded device-side wait ran out; cleared by the read).
bool gemm_tc_supported(const GemmArgs& a);
amq_status launch_binary_gemm_tc(const GemmArgs& a, cudaStream_t st);
amq_status read_tc_status(cudaStream_t st, uint32_t* out);

// Persistent batch-1 recurrent kernel: whether it covers a problem (sizes, shared memory), and its launch.
bool persistent_supported(int I, int H, int batch, int k_w, int k_a, bool gru, int* grid_out, int* upc_out,
                          size_t* smem_out);
amq_status launch_rnn_persistent(const uint32_t* Wcodes, const float* Walpha, const float* bias,
                                 int I, int H, int k_w, int k_a, int T, bool gru,
                                 const float* x_seq, int steps, const float* h0, const float* c0,
                                 float* h_seq, float* h_last, float* c_last,
                                 unsigned long long* hx, uint32_t* status, cudaStream_t st,
                                 unsigned poll_limit = 0, unsigned tag_bias = 0);

}  // namespace amq
