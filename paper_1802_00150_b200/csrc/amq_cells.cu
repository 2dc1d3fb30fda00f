// Quantized LSTM / GRU steps and sequences (Eq. 6; on-line quantization of the activation, Sec. 4):
// each step is the row quantizer on z = [x ; h] followed by the binary product with the fused gate
// epilogue.  No step returns to the host; a sequence is enqueued as one chain on the caller's stream.
#include "amq_common.cuh"

namespace amq {

namespace {

struct CellCall {
    const uint32_t* Wcodes; const float* Walpha; const float* bias;
    int I, H, k_w, batch, k_a, T;
    bool gru;
};

amq_status validate(const CellCall& c, const void* workspace, size_t workspace_bytes)
{
    if (!c.Wcodes || !c.Walpha || c.I < 0 || c.H < 1 || c.batch < 0) return AMQ_ERR_INVALID_ARG;
    if (!valid_k(c.k_w) || !valid_k(c.k_a) || c.T < 0 || c.I + c.H > AMQ_MAX_N) return AMQ_ERR_UNSUPPORTED;
    if (!aligned16(c.Wcodes)) return AMQ_ERR_ALIGNMENT;
    if (!workspace || workspace_bytes < amq_cell_workspace_bytes(c.I, c.H, c.batch, c.k_a)) return AMQ_ERR_WORKSPACE;
    if (!aligned16(workspace)) return AMQ_ERR_ALIGNMENT;
    return AMQ_OK;
}

bool use_persistent(const CellCall& c)
{
    int grid, upc;
    size_t smem;
    return persistent_supported(c.I, c.H, c.batch, c.k_w, c.k_a, c.gru, &grid, &upc, &smem);
}

amq_status enqueue_persistent(const CellCall& c, const CellWorkspace& ws, const float* x_seq, int steps,
                              const float* h0, const float* c0, float* h_seq, float* h_last, float* c_last,
                              cudaStream_t st, unsigned poll_limit = 0, unsigned tag_bias = 0)
{
    // the caller has cleared the status words and, for more than one step, the exchange words behind them (stale
    // step tags must not match; a single step polls nothing)
    return launch_rnn_persistent(c.Wcodes, c.Walpha, c.bias, c.I, c.H, c.k_w, c.k_a, c.T, c.gru, x_seq, steps,
                                 h0, c0, h_seq, h_last, c_last, ws.hx, ws.status, st, poll_limit, tag_bias);
}

// (inputs come from the preceding kernels of the stream: ordinary loads after the wait, no read-only path)
__global__ void lstm_gates_kernel(const float* pre, const float* addend, const float* c_in, float* h_out, float* c_out, int H)
{
    grid_dependency_wait();
    const int u = blockIdx.x * blockDim.x + threadIdx.x;
    if (u >= H) return;
    float g4[4];
#pragma unroll
    for (int g = 0; g < 4; ++g) g4[g] = __ldcg(pre + g * H + u) + (addend ? __ldcg(addend + g * H + u) : 0.0f);
    const float ig = 1.0f / (1.0f + __expf(-g4[0])), fg = 1.0f / (1.0f + __expf(-g4[1])), og = 1.0f / (1.0f + __expf(-g4[2]));
    const float c = fg * __ldcg(c_in + u) + ig * tanhf(g4[3]);
    c_out[u] = c;
    h_out[u] = og * tanhf(c);
}

// quantize z = [x ; h_in] into the workspace, then product + gates
amq_status enqueue_step(const CellCall& c, const CellWorkspace& ws, const float* x, const float* h_in,
                        const float* c_in, float* h_out, float* c_out, cudaStream_t st)
{
    GemmArgs a{};
    a.Wcodes = c.Wcodes; a.Walpha = c.Walpha; a.m = (c.gru ? 3 : 4) * c.H; a.n = c.I + c.H; a.k_w = c.k_w;
    a.xcodes = ws.zcodes; a.xbeta = ws.zbeta; a.batch = c.batch; a.k_a = c.k_a;
    a.bias = c.bias;
    if (use_persistent(c))      // batch 1: one launch of the weight-stationary kernel, a sequence of one step
        return enqueue_persistent(c, ws, x, 1, h_in, c_in, nullptr, h_out, c_out, st);
    a.epilogue = c.gru ? EPI_GRU : EPI_LSTM;
    a.I = c.I; a.H = c.H; a.h_in = h_in; a.c_in = c_in; a.h_out = h_out; a.c_out = c_out;
    // the quantizer may be scheduled while the product of the previous timestep still runs (it waits for it first
    // thing) when that product runs as a single wave
    amq_status s = launch_quantize(x, c.I, c.I, h_in, c.H, c.H, c.batch, c.k_a, c.T, ws.zcodes, ws.zbeta, st,
                                   gemm_tc_single_wave(a));
    if (s != AMQ_OK) return s;
    a.overlap_with_previous = true;             // the quantizer above is the previous kernel of the stream
    return launch_binary_gemm(a, st);
}

// `chunk_ready` (may be NULL): events after which the inputs of steps [q * steps_per_chunk, (q + 1) * steps_per_chunk) are
// in place; the stream waits for event q before the first kernel of that chunk (batched chains only).
amq_status enqueue_sequence(const CellCall& c, const CellWorkspace& ws, const float* x_seq, int steps,
                            const float* h0, const float* c0, float* h_seq, float* h_last, float* c_last,
                            cudaStream_t st, const cudaEvent_t* chunk_ready = nullptr, int steps_per_chunk = 0)
{
    const size_t state_bytes = (size_t)c.batch * c.H * sizeof(float);
    const bool persistent = steps > 0 && use_persistent(c);
    AMQ_CUDA_TRY(cudaMemsetAsync(ws.status, 0, 256 + ((persistent && steps > 1) ? ws.hx_bytes : 0), st));
    if (persistent)
        return enqueue_persistent(c, ws, x_seq, steps, h0, c0, h_seq, h_last, c_last, st);
    if (!c.gru) AMQ_CUDA_TRY(cudaMemcpyAsync(ws.c, c0, state_bytes, cudaMemcpyDeviceToDevice, st));
    const float* h_prev = h0;
    for (int s = 0; s < steps; ++s) {
        float* h_next = h_seq ? h_seq + (size_t)s * c.batch * c.H : ws.h[s & 1];
        const float* x = x_seq + (size_t)s * c.batch * c.I;
        if (chunk_ready && s % steps_per_chunk == 0) AMQ_CUDA_TRY(cudaStreamWaitEvent(st, chunk_ready[s / steps_per_chunk], 0));
        amq_status r = enqueue_step(c, ws, x, h_prev, ws.c, h_next, ws.c, st);
        if (r != AMQ_OK) return r;
        h_prev = h_next;
    }
    AMQ_CUDA_TRY(cudaMemcpyAsync(h_last, h_prev, state_bytes, cudaMemcpyDeviceToDevice, st));
    if (!c.gru) AMQ_CUDA_TRY(cudaMemcpyAsync(c_last, ws.c, state_bytes, cudaMemcpyDeviceToDevice, st));
    return AMQ_OK;
}

amq_status sequence_entry(const CellCall& c, const float* x_seq, int steps, const float* h0, const float* c0,
                          float* h_seq, float* h_last, float* c_last,
                          void* workspace, size_t workspace_bytes, cudaStream_t st)
{
    amq_status s = validate(c, workspace, workspace_bytes);
    if (s != AMQ_OK) return s;
    if (steps < 0 || !h0 || !h_last || (!c.gru && (!c0 || !c_last)) || (steps > 0 && c.I > 0 && !x_seq))
        return AMQ_ERR_INVALID_ARG;
    if (h_last == h0 || (!c.gru && c_last == c0)) return AMQ_ERR_INVALID_ARG;
    if (c.batch == 0) return AMQ_OK;
    CellWorkspace ws = carve_cell_workspace(workspace, c.I, c.H, c.batch, c.k_a);
    return enqueue_sequence(c, ws, x_seq, steps, h0, c0, h_seq, h_last, c_last, st);
}

struct HostStaging {
    float* x_seq; float* h0; float* c0; float* h_seq; float* h_last; float* c_last;
    size_t bytes;
};

HostStaging carve_staging(void* base, int I, int H, int batch, int steps)
{
    HostStaging s;
    char* p = static_cast<char*>(base);
    size_t off = 0;
    const size_t state = round_up((size_t)batch * H * 4, 256);
    s.x_seq = reinterpret_cast<float*>(p + off);  off += round_up((size_t)steps * batch * I * 4, 256);
    s.h0 = reinterpret_cast<float*>(p + off);     off += state;
    s.c0 = reinterpret_cast<float*>(p + off);     off += state;
    s.h_seq = reinterpret_cast<float*>(p + off);  off += round_up((size_t)steps * batch * H * 4, 256);
    s.h_last = reinterpret_cast<float*>(p + off); off += state;
    s.c_last = reinterpret_cast<float*>(p + off); off += state;
    s.bytes = off;
    return s;
}

amq_status sequence_host_entry(const CellCall& c, const float* x_seq_host, int steps, const float* h0_host,
                               const float* c0_host, float* h_seq_host, float* h_last_host, float* c_last_host,
                               void* workspace, size_t workspace_bytes, void* staging, size_t staging_bytes,
                               cudaStream_t st)
{
    amq_status s = validate(c, workspace, workspace_bytes);
    if (s != AMQ_OK) return s;
    if (steps < 0 || !h0_host || !h_last_host || (!c.gru && (!c0_host || !c_last_host)) ||
        (steps > 0 && c.I > 0 && !x_seq_host))
        return AMQ_ERR_INVALID_ARG;
    if (!staging || staging_bytes < amq_cell_host_staging_bytes(c.I, c.H, c.batch, steps)) return AMQ_ERR_WORKSPACE;
    if (!aligned16(staging)) return AMQ_ERR_ALIGNMENT;
    if (c.batch == 0) return AMQ_OK;
    CellWorkspace ws = carve_cell_workspace(workspace, c.I, c.H, c.batch, c.k_a);
    HostStaging hs = carve_staging(staging, c.I, c.H, c.batch, steps);
    const size_t state_bytes = (size_t)c.batch * c.H * sizeof(float);
    const size_t x_bytes = (size_t)steps * c.batch * c.I * sizeof(float);
    // Large inputs of a batched chain travel in chunks of timesteps on a stream of their own, so that the copy of the later
    // timesteps runs beside the kernels of the earlier ones (C4: 73 MB of inputs against 1.7 ms of kernels); the chain waits
    // for a chunk's event before its first step.  The copy stream and the events live for the duration of the call.
    constexpr int MAX_CHUNKS = 8;
    const bool chunked = x_bytes >= ((size_t)4 << 20) && steps >= 2 && !(steps > 0 && use_persistent(c));
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t ready[MAX_CHUNKS + 1] = {};
    int nchunks = 0, steps_per_chunk = 0;
    auto release = [&]() {
        for (int q = 0; q <= MAX_CHUNKS; ++q) if (ready[q]) cudaEventDestroy(ready[q]);
        if (copy_stream) cudaStreamDestroy(copy_stream);
    };
    // the small copies of the initial state go first: host-to-device copies are served in the order they were submitted,
    // whatever their stream, and the chain's first kernel needs them
    cudaError_t e = cudaMemcpyAsync(hs.h0, h0_host, state_bytes, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && !c.gru) e = cudaMemcpyAsync(hs.c0, c0_host, state_bytes, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return AMQ_ERR_CUDA;
    if (chunked) {
        steps_per_chunk = (steps + MAX_CHUNKS - 1) / MAX_CHUNKS;
        nchunks = (steps + steps_per_chunk - 1) / steps_per_chunk;
        e = cudaStreamCreateWithFlags(&copy_stream, cudaStreamNonBlocking);
        for (int q = 0; q <= nchunks && e == cudaSuccess; ++q) e = cudaEventCreateWithFlags(&ready[q], cudaEventDisableTiming);
        // the copy stream starts after what the caller's stream holds so far (the staging buffer may still be in use there)
        if (e == cudaSuccess) e = cudaEventRecord(ready[nchunks], st);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(copy_stream, ready[nchunks], 0);
        const size_t step_bytes = (size_t)c.batch * c.I * sizeof(float);
        for (int q = 0; q < nchunks && e == cudaSuccess; ++q) {
            const int s0 = q * steps_per_chunk, s1 = (s0 + steps_per_chunk < steps) ? s0 + steps_per_chunk : steps;
            e = cudaMemcpyAsync(reinterpret_cast<char*>(hs.x_seq) + s0 * step_bytes,
                                reinterpret_cast<const char*>(x_seq_host) + s0 * step_bytes, (size_t)(s1 - s0) * step_bytes,
                                cudaMemcpyHostToDevice, copy_stream);
            if (e == cudaSuccess) e = cudaEventRecord(ready[q], copy_stream);
        }
        if (e != cudaSuccess) { cudaStreamSynchronize(copy_stream); release(); return AMQ_ERR_CUDA; }
    } else if (x_bytes) {
        AMQ_CUDA_TRY(cudaMemcpyAsync(hs.x_seq, x_seq_host, x_bytes, cudaMemcpyHostToDevice, st));
    }
    s = enqueue_sequence(c, ws, hs.x_seq, steps, hs.h0, hs.c0, h_seq_host ? hs.h_seq : nullptr, hs.h_last, hs.c_last, st,
                         chunked ? ready : nullptr, steps_per_chunk);
    if (chunked) {
        // the events and the stream may go once both streams have drained
        cudaStreamSynchronize(copy_stream);
        if (s != AMQ_OK) cudaStreamSynchronize(st);
    }
    if (s != AMQ_OK) { release(); return s; }
    struct Releaser { decltype(release)& r; ~Releaser() { r(); } } releaser{release};
    if (h_seq_host && steps > 0)
        AMQ_CUDA_TRY(cudaMemcpyAsync(h_seq_host, hs.h_seq, (size_t)steps * state_bytes, cudaMemcpyDeviceToHost, st));
    AMQ_CUDA_TRY(cudaMemcpyAsync(h_last_host, hs.h_last, state_bytes, cudaMemcpyDeviceToHost, st));
    if (!c.gru) AMQ_CUDA_TRY(cudaMemcpyAsync(c_last_host, hs.c_last, state_bytes, cudaMemcpyDeviceToHost, st));
    AMQ_CUDA_TRY(cudaStreamSynchronize(st));
    return AMQ_OK;
}

}  // namespace

amq_status launch_lstm_gates(const float* pre, const float* addend, const float* c_in, float* h_out, float* c_out, int H,
                             cudaStream_t st, bool overlap_with_previous)
{
    AMQ_CUDA_TRY(launch_kernel(lstm_gates_kernel, dim3((unsigned)((H + 255) / 256)), dim3(256), 0, st, overlap_with_previous,
                               pre, addend, c_in, h_out, c_out, H));
    AMQ_LAUNCH_CHECK();
    return AMQ_OK;
}

}  // namespace amq

extern "C" {

size_t amq_cell_workspace_bytes(int I, int H, int batch, int k_a)
{
    if (I < 0 || H < 1 || batch < 0 || !amq::valid_k(k_a)) return 0;
    return amq::carve_cell_workspace(nullptr, I, H, batch, k_a).bytes;
}

size_t amq_cell_host_staging_bytes(int I, int H, int batch, int steps)
{
    if (I < 0 || H < 1 || batch < 0 || steps < 0) return 0;
    return amq::carve_staging(nullptr, I, H, batch, steps).bytes;
}

amq_status amq_lstm_step(const uint32_t* Wcodes, const float* Walpha, const float* bias, int I, int H, int k_w,
                         const float* x, const float* h_in, const float* c_in, int batch, int k_a, int T,
                         float* h_out, float* c_out, void* workspace, size_t workspace_bytes, void* stream)
{
    amq::CellCall c{Wcodes, Walpha, bias, I, H, k_w, batch, k_a, T, false};
    amq_status s = amq::validate(c, workspace, workspace_bytes);
    if (s != AMQ_OK) return s;
    if (!h_in || !c_in || !h_out || !c_out || (I > 0 && !x) || h_out == h_in) return AMQ_ERR_INVALID_ARG;
    if (batch == 0) return AMQ_OK;
    amq::CellWorkspace ws = amq::carve_cell_workspace(workspace, I, H, batch, k_a);
    AMQ_CUDA_TRY(cudaMemsetAsync(ws.status, 0, 256, (cudaStream_t)stream));
    return amq::enqueue_step(c, ws, x, h_in, c_in, h_out, c_out, (cudaStream_t)stream);
}

amq_status amq_gru_step(const uint32_t* Wcodes, const float* Walpha, const float* bias, int I, int H, int k_w,
                        const float* x, const float* h_in, int batch, int k_a, int T,
                        float* h_out, void* workspace, size_t workspace_bytes, void* stream)
{
    amq::CellCall c{Wcodes, Walpha, bias, I, H, k_w, batch, k_a, T, true};
    amq_status s = amq::validate(c, workspace, workspace_bytes);
    if (s != AMQ_OK) return s;
    if (!h_in || !h_out || (I > 0 && !x) || h_out == h_in) return AMQ_ERR_INVALID_ARG;
    if (batch == 0) return AMQ_OK;
    amq::CellWorkspace ws = amq::carve_cell_workspace(workspace, I, H, batch, k_a);
    AMQ_CUDA_TRY(cudaMemsetAsync(ws.status, 0, 256, (cudaStream_t)stream));
    return amq::enqueue_step(c, ws, x, h_in, nullptr, h_out, nullptr, (cudaStream_t)stream);
}

amq_status amq_lstm_sequence(const uint32_t* Wcodes, const float* Walpha, const float* bias, int I, int H, int k_w,
                             const float* x_seq, int steps, const float* h0, const float* c0,
                             int batch, int k_a, int T, float* h_seq, float* h_last, float* c_last,
                             void* workspace, size_t workspace_bytes, void* stream)
{
    amq::CellCall c{Wcodes, Walpha, bias, I, H, k_w, batch, k_a, T, false};
    return amq::sequence_entry(c, x_seq, steps, h0, c0, h_seq, h_last, c_last, workspace, workspace_bytes,
                               (cudaStream_t)stream);
}

amq_status amq_gru_sequence(const uint32_t* Wcodes, const float* Walpha, const float* bias, int I, int H, int k_w,
                            const float* x_seq, int steps, const float* h0, int batch, int k_a, int T,
                            float* h_seq, float* h_last, void* workspace, size_t workspace_bytes, void* stream)
{
    amq::CellCall c{Wcodes, Walpha, bias, I, H, k_w, batch, k_a, T, true};
    return amq::sequence_entry(c, x_seq, steps, h0, nullptr, h_seq, h_last, nullptr, workspace, workspace_bytes,
                               (cudaStream_t)stream);
}

amq_status amq_lstm_sequence_host(const uint32_t* Wcodes, const float* Walpha, const float* bias,
                                  int I, int H, int k_w, const float* x_seq_host, int steps,
                                  const float* h0_host, const float* c0_host, int batch, int k_a, int T,
                                  float* h_seq_host, float* h_last_host, float* c_last_host,
                                  void* workspace, size_t workspace_bytes, void* staging, size_t staging_bytes,
                                  void* stream)
{
    amq::CellCall c{Wcodes, Walpha, bias, I, H, k_w, batch, k_a, T, false};
    return amq::sequence_host_entry(c, x_seq_host, steps, h0_host, c0_host, h_seq_host, h_last_host, c_last_host,
                                    workspace, workspace_bytes, staging, staging_bytes, (cudaStream_t)stream);
}

amq_status amq_gru_sequence_host(const uint32_t* Wcodes, const float* Walpha, const float* bias,
                                 int I, int H, int k_w, const float* x_seq_host, int steps,
                                 const float* h0_host, int batch, int k_a, int T,
                                 float* h_seq_host, float* h_last_host,
                                 void* workspace, size_t workspace_bytes, void* staging, size_t staging_bytes,
                                 void* stream)
{
    amq::CellCall c{Wcodes, Walpha, bias, I, H, k_w, batch, k_a, T, true};
    return amq::sequence_host_entry(c, x_seq_host, steps, h0_host, nullptr, h_seq_host, h_last_host, nullptr,
                                    workspace, workspace_bytes, staging, staging_bytes, (cudaStream_t)stream);
}

amq_status amq_selftest_sequence_give_up(const uint32_t* Wcodes, const float* Walpha, const float* bias,
                                         int I, int H, int k_w,
                                         const float* x_seq, int steps, const float* h0, const float* c0,
                                         int k_a, int T, float* h_last, float* c_last,
                                         void* workspace, size_t workspace_bytes, unsigned poll_limit, void* stream)
{
    amq::CellCall c{Wcodes, Walpha, bias, I, H, k_w, 1, k_a, T, false};
    amq_status s = amq::validate(c, workspace, workspace_bytes);
    if (s != AMQ_OK) return s;
    if (steps < 2 || !h0 || !c0 || !h_last || !c_last || (I > 0 && !x_seq) || h_last == h0 || c_last == c0)
        return AMQ_ERR_INVALID_ARG;
    if (poll_limit < 1 || poll_limit > 65536) return AMQ_ERR_INVALID_ARG;
    if (!amq::use_persistent(c)) return AMQ_ERR_UNSUPPORTED;
    amq::CellWorkspace ws = amq::carve_cell_workspace(workspace, I, H, 1, k_a);
    AMQ_CUDA_TRY(cudaMemsetAsync(ws.status, 0, 256 + ws.hx_bytes, (cudaStream_t)stream));
    // expected tags are offset by 2^30: the tags the CTAs publish (1 .. steps) never match
    return amq::enqueue_persistent(c, ws, x_seq, steps, h0, c0, nullptr, h_last, c_last, (cudaStream_t)stream,
                                   poll_limit, 1u << 30);
}

amq_status amq_workspace_status(const void* workspace, void* stream)
{
    if (!workspace) return AMQ_ERR_INVALID_ARG;
    AMQ_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    uint32_t word = 0;
    AMQ_CUDA_TRY(cudaMemcpy(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost));
    return word == 0 ? AMQ_OK : AMQ_ERR_TIMEOUT;
}

}  // extern "C"
