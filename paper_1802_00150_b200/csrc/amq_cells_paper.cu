// Quantized LSTM in the form the paper states it (Eq. 6 and the paragraph after it): two weight matrices
// W_i (4H x I) and W_h (4H x H), each quantized row by row on its own; the input x_t is a row of the quantized
// embedding matrix and is used as it is, without a second quantization (it arrives as packed planes + coefficients, see
// amq_embedding_rows); only h_{t-1} is quantized on-line.
//
// Because x_t does not depend on the recurrent state, the input projections W_i x_t + b of ALL timesteps of
// a sequence are one batched binary product (steps * batch vectors) done before the time loop; a timestep
// is then the on-line quantizer on h (H columns instead of I + H) and the product with W_h, whose epilogue
// adds the precomputed projection and applies the gates.
#include "amq_common.cuh"

namespace amq {

namespace {

struct PaperWorkspace {
    uint32_t* hcodes;   // [batch][k_a][wpr(H)]
    float* hbeta;       // [batch][k_a]
    float* proj;        // [steps][batch][4H]  W_i x_t + bias
    float* h[2];        // [batch][H] ping / pong
    float* c;           // [batch][H]
    float* gates;       // [4H] pre-activations of a single sequence (batch 1)
    size_t bytes;
};

PaperWorkspace carve(void* base, int H, int batch, int steps, int k_a)
{
    PaperWorkspace w;
    char* p = static_cast<char*>(base);
    size_t off = 0;
    w.hcodes = reinterpret_cast<uint32_t*>(p + off); off += round_up((size_t)batch * k_a * words_per_row(H) * 4, 256);
    w.hbeta = reinterpret_cast<float*>(p + off);     off += round_up((size_t)batch * k_a * 4, 256);
    w.proj = reinterpret_cast<float*>(p + off);      off += round_up((size_t)steps * batch * 4 * H * 4, 256);
    w.h[0] = reinterpret_cast<float*>(p + off);      off += round_up((size_t)batch * H * 4, 256);
    w.h[1] = reinterpret_cast<float*>(p + off);      off += round_up((size_t)batch * H * 4, 256);
    w.c = reinterpret_cast<float*>(p + off);         off += round_up((size_t)batch * H * 4, 256);
    w.gates = reinterpret_cast<float*>(p + off);     off += round_up((size_t)4 * H * 4, 256);
    w.bytes = off;
    return w;
}

struct PaperCall {
    const uint32_t* Wi_codes; const float* Wi_alpha; const uint32_t* Wh_codes; const float* Wh_alpha; const float* bias;
    int I, H, k_w, k_e, batch, k_a, T;
};

amq_status validate(const PaperCall& c, int steps, const void* workspace, size_t workspace_bytes)
{
    if (!c.Wi_codes || !c.Wi_alpha || !c.Wh_codes || !c.Wh_alpha || c.I < 1 || c.H < 1 || c.batch < 0 || steps < 0)
        return AMQ_ERR_INVALID_ARG;
    if (!valid_k(c.k_w) || !valid_k(c.k_e) || !valid_k(c.k_a) || c.T < 0 || c.H > AMQ_MAX_N) return AMQ_ERR_UNSUPPORTED;
    if ((long long)steps * c.batch > 0x7fffffffll / 4) return AMQ_ERR_UNSUPPORTED;
    if (!aligned16(c.Wi_codes) || !aligned16(c.Wh_codes)) return AMQ_ERR_ALIGNMENT;
    if (!workspace || workspace_bytes < amq_lstm_paper_workspace_bytes(c.H, c.batch, steps, c.k_a)) return AMQ_ERR_WORKSPACE;
    if (!aligned16(workspace)) return AMQ_ERR_ALIGNMENT;
    return AMQ_OK;
}

// W_i x + bias for `vectors` pre-quantized inputs -> proj [vectors][4H]
amq_status input_projection(const PaperCall& c, const uint32_t* xcodes, const float* xbeta, int vectors, float* proj,
                            cudaStream_t st)
{
    GemmArgs a{};
    a.Wcodes = c.Wi_codes; a.Walpha = c.Wi_alpha; a.m = 4 * c.H; a.n = c.I; a.k_w = c.k_w;
    a.xcodes = xcodes; a.xbeta = xbeta; a.batch = vectors; a.k_a = c.k_e;
    a.bias = c.bias; a.epilogue = EPI_Y; a.y = proj; a.ldy = 4 * c.H;
    return launch_binary_gemm(a, st);
}

// quantize h_in on-line, then W_h h_hat + proj -> gates -> (h_out, c_out)
amq_status recurrent_part(const PaperCall& c, const PaperWorkspace& ws, const float* proj, const float* h_in,
                          const float* c_in, float* h_out, float* c_out, cudaStream_t st)
{
    GemmArgs a{};
    a.Wcodes = c.Wh_codes; a.Walpha = c.Wh_alpha; a.m = 4 * c.H; a.n = c.H; a.k_w = c.k_w;
    a.xcodes = ws.hcodes; a.xbeta = ws.hbeta; a.batch = c.batch; a.k_a = c.k_a;
    a.bias = nullptr;
    a.epilogue = EPI_LSTM; a.H = c.H;
    // in a sequence the kernel before this quantizer is the recurrent product of the previous timestep: when that
    // runs as a single wave the quantizer may be scheduled behind it early (it waits for it first thing)
    // (with one sequence every kernel of the step is short and waits for its predecessor first thing: all overlapped)
    if (c.batch == 1 && quantized_gemv_supported(c.H) && c.k_a <= 2) {
        // one sequence, a state of up to 2048 elements: the quantizer runs inside the matrix-vector kernel (one launch
        // for both; the same bits as the two launches below), then the small gate kernel
        amq_status s1 = launch_quantized_gemv(c.Wh_codes, c.Wh_alpha, 4 * c.H, c.H, c.k_w, h_in, c.k_a, c.T, nullptr, ws.gates,
                                              nullptr, nullptr, st, true);
        if (s1 != AMQ_OK) return s1;
        return launch_lstm_gates(ws.gates, proj, c_in, h_out, c_out, c.H, st, true);
    }
    amq_status s = launch_quantize(h_in, c.H, c.H, nullptr, 0, 0, c.batch, c.k_a, c.T, ws.hcodes, ws.hbeta, st,
                                   c.batch == 1 || gemm_tc_single_wave(a));
    if (s != AMQ_OK) return s;
    if (c.batch == 1) {
        // one sequence: the bandwidth-bound matrix-vector kernel writes the pre-activations, a small kernel applies the gates
        a.epilogue = EPI_Y; a.y = ws.gates; a.ldy = 4 * c.H;
        if (gemv_supported(a)) {
            a.overlap_with_previous = true;
            s = launch_binary_gemv(a, st);
            if (s != AMQ_OK) return s;
            return launch_lstm_gates(ws.gates, proj, c_in, h_out, c_out, c.H, st, true);
        }
    }
    a.y = nullptr; a.ldy = 0;
    a.epilogue = EPI_LSTM;
    a.overlap_with_previous = true;             // the quantizer above is the previous kernel of the stream
    a.I = 0; a.H = c.H; a.h_in = h_in; a.c_in = c_in; a.h_out = h_out; a.c_out = c_out;
    a.addend = proj; a.ld_addend = 4 * c.H;
    return launch_binary_gemm(a, st);
}

}  // namespace
}  // namespace amq

extern "C" {

size_t amq_lstm_paper_workspace_bytes(int H, int batch, int steps, int k_a)
{
    if (H < 1 || batch < 0 || steps < 0 || !amq::valid_k(k_a)) return 0;
    return amq::carve(nullptr, H, batch, steps > 0 ? steps : 1, k_a).bytes;
}

amq_status amq_lstm_step_paper(const uint32_t* Wi_codes, const float* Wi_alpha, const uint32_t* Wh_codes, const float* Wh_alpha,
                               const float* bias, int I, int H, int k_w,
                               const uint32_t* xcodes, const float* xbeta, int k_e,
                               const float* h_in, const float* c_in, int batch, int k_a, int T,
                               float* h_out, float* c_out, void* workspace, size_t workspace_bytes, void* stream)
{
    amq::PaperCall c{Wi_codes, Wi_alpha, Wh_codes, Wh_alpha, bias, I, H, k_w, k_e, batch, k_a, T};
    amq_status s = amq::validate(c, 1, workspace, workspace_bytes);
    if (s != AMQ_OK) return s;
    if (batch == 0) return AMQ_OK;
    if (!xcodes || !xbeta || !h_in || !c_in || !h_out || !c_out || h_out == h_in) return AMQ_ERR_INVALID_ARG;
    if (!amq::aligned16(xcodes)) return AMQ_ERR_ALIGNMENT;
    amq::PaperWorkspace ws = amq::carve(workspace, H, batch, 1, k_a);
    cudaStream_t st = (cudaStream_t)stream;
    s = amq::input_projection(c, xcodes, xbeta, batch, ws.proj, st);
    if (s != AMQ_OK) return s;
    return amq::recurrent_part(c, ws, ws.proj, h_in, c_in, h_out, c_out, st);
}

amq_status amq_lstm_sequence_paper(const uint32_t* Wi_codes, const float* Wi_alpha, const uint32_t* Wh_codes, const float* Wh_alpha,
                                   const float* bias, int I, int H, int k_w,
                                   const uint32_t* xcodes_seq, const float* xbeta_seq, int k_e, int steps,
                                   const float* h0, const float* c0, int batch, int k_a, int T,
                                   float* h_seq, float* h_last, float* c_last,
                                   void* workspace, size_t workspace_bytes, void* stream)
{
    amq::PaperCall c{Wi_codes, Wi_alpha, Wh_codes, Wh_alpha, bias, I, H, k_w, k_e, batch, k_a, T};
    amq_status s = amq::validate(c, steps, workspace, workspace_bytes);
    if (s != AMQ_OK) return s;
    if (batch == 0) return AMQ_OK;
    if (!h0 || !c0 || !h_last || !c_last || h_last == h0 || c_last == c0 || (steps > 0 && (!xcodes_seq || !xbeta_seq)))
        return AMQ_ERR_INVALID_ARG;
    if (steps > 0 && !amq::aligned16(xcodes_seq)) return AMQ_ERR_ALIGNMENT;
    amq::PaperWorkspace ws = amq::carve(workspace, H, batch, steps > 0 ? steps : 1, k_a);
    cudaStream_t st = (cudaStream_t)stream;
    const size_t state_bytes = (size_t)batch * H * sizeof(float);
    // the input projections of all timesteps at once: they do not depend on the recurrent state
    if (steps > 0) {
        s = amq::input_projection(c, xcodes_seq, xbeta_seq, steps * batch, ws.proj, st);
        if (s != AMQ_OK) return s;
    }
    AMQ_CUDA_TRY(cudaMemcpyAsync(ws.c, c0, state_bytes, cudaMemcpyDeviceToDevice, st));
    const float* h_prev = h0;
    for (int t = 0; t < steps; ++t) {
        float* h_next = h_seq ? h_seq + (size_t)t * batch * H : ws.h[t & 1];
        s = amq::recurrent_part(c, ws, ws.proj + (size_t)t * batch * 4 * H, h_prev, ws.c, h_next, ws.c, st);
        if (s != AMQ_OK) return s;
        h_prev = h_next;
    }
    AMQ_CUDA_TRY(cudaMemcpyAsync(h_last, h_prev, state_bytes, cudaMemcpyDeviceToDevice, st));
    AMQ_CUDA_TRY(cudaMemcpyAsync(c_last, ws.c, state_bytes, cudaMemcpyDeviceToDevice, st));
    return AMQ_OK;
}

}  // extern "C"
