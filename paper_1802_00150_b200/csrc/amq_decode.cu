// Greedy decoding with the quantized language model of Eq. 6 (one sequence, the arg-max token fed back), enqueued
// as one chain on the caller's stream: per token the embedding row (pre-quantized, needs no further quantization),
// the input projection W_i x + b, the recurrent product W_h h_hat on the on-line quantized state, the gates, the
// quantizer on the new state (its planes serve the output layer now and the recurrence of the next token), the
// output product W_s h_hat + b_s and log-softmax / arg-max.  Six launches per token (the quantizer on the new state
// runs inside the output product's kernel when the state has at most 2048 elements and at most 2 bits, else seven), no
// host round trip.
#include "amq_common.cuh"

namespace amq {
namespace {

struct DecodeWorkspace {
    uint32_t* xcodes;   // [k_e][wpr(I)]
    float* xbeta;       // [k_e]
    uint32_t* hcodes;   // [k_a][wpr(H)]
    float* hbeta;       // [k_a]
    float* proj;        // [4H]
    float* pre;         // [4H]
    float* logits;      // [vocab]
    size_t bytes;
};

DecodeWorkspace carve(void* base, int vocab, int I, int H, int k_e, int k_a)
{
    DecodeWorkspace w;
    char* p = static_cast<char*>(base);
    size_t off = 0;
    w.xcodes = reinterpret_cast<uint32_t*>(p + off); off += round_up((size_t)k_e * words_per_row(I) * 4, 256);
    w.xbeta = reinterpret_cast<float*>(p + off);     off += 256;
    w.hcodes = reinterpret_cast<uint32_t*>(p + off); off += round_up((size_t)k_a * words_per_row(H) * 4, 256);
    w.hbeta = reinterpret_cast<float*>(p + off);     off += 256;
    w.proj = reinterpret_cast<float*>(p + off);      off += round_up((size_t)4 * H * 4, 256);
    w.pre = reinterpret_cast<float*>(p + off);       off += round_up((size_t)4 * H * 4, 256);
    w.logits = reinterpret_cast<float*>(p + off);    off += round_up((size_t)vocab * 4, 256);
    w.bytes = off;
    return w;
}

}  // namespace
}  // namespace amq

extern "C" {

size_t amq_lm_decode_workspace_bytes(int vocab, int I, int H, int k_e, int k_a)
{
    if (vocab < 1 || I < 1 || H < 1 || !amq::valid_k(k_e) || !amq::valid_k(k_a)) return 0;
    return amq::carve(nullptr, vocab, I, H, k_e, k_a).bytes;
}

amq_status amq_lm_greedy_decode(const uint32_t* We_codes, const float* We_alpha, int vocab, int I, int k_e,
                                const uint32_t* Wi_codes, const float* Wi_alpha, const uint32_t* Wh_codes, const float* Wh_alpha,
                                const float* bias, int H, int k_w,
                                const uint32_t* Ws_codes, const float* Ws_alpha, const float* bias_s, int k_s,
                                int k_a, int T, int32_t* tokens, int steps, float* h, float* c, float* logp,
                                void* workspace, size_t workspace_bytes, void* stream)
{
    if (!We_codes || !We_alpha || !Wi_codes || !Wi_alpha || !Wh_codes || !Wh_alpha || !Ws_codes || !Ws_alpha || vocab < 1 ||
        I < 1 || H < 1 || steps < 0)
        return AMQ_ERR_INVALID_ARG;
    if (!amq::valid_k(k_e) || !amq::valid_k(k_w) || !amq::valid_k(k_s) || !amq::valid_k(k_a) || T < 0 || I > AMQ_MAX_N ||
        H > AMQ_MAX_N)
        return AMQ_ERR_UNSUPPORTED;
    if (!workspace || workspace_bytes < amq_lm_decode_workspace_bytes(vocab, I, H, k_e, k_a)) return AMQ_ERR_WORKSPACE;
    if (!amq::aligned16(workspace) || !amq::aligned16(We_codes) || !amq::aligned16(Wi_codes) || !amq::aligned16(Wh_codes) ||
        !amq::aligned16(Ws_codes))
        return AMQ_ERR_ALIGNMENT;
    if (steps == 0) return AMQ_OK;
    if (!tokens || !h || !c) return AMQ_ERR_INVALID_ARG;
    const amq::DecodeWorkspace ws = amq::carve(workspace, vocab, I, H, k_e, k_a);
    cudaStream_t st = (cudaStream_t)stream;
    // every launch after the first is a programmatic dependent of its predecessor (each kernel waits for it first
    // thing), which takes most of the gaps between these short kernels out of the chain
    auto product = [&](const uint32_t* Wc, const float* Wa, int m, int n, int kw, const uint32_t* xc, const float* xb, int ka,
                       const float* b, float* y) {
        amq::GemmArgs a{};
        a.Wcodes = Wc; a.Walpha = Wa; a.m = m; a.n = n; a.k_w = kw;
        a.xcodes = xc; a.xbeta = xb; a.batch = 1; a.k_a = ka;
        a.bias = b; a.epilogue = amq::EPI_Y; a.y = y; a.ldy = m;
        a.overlap_with_previous = true;
        return amq::launch_binary_gemm(a, st);
    };
    amq_status s = amq::launch_quantize(h, H, H, nullptr, 0, 0, 1, k_a, T, ws.hcodes, ws.hbeta, st, false);   // h_hat of the start state
    for (int t = 0; t < steps && s == AMQ_OK; ++t) {
        s = amq::launch_embedding_rows(We_codes, We_alpha, vocab, I, k_e, tokens + t, 1, ws.xcodes, ws.xbeta, st, true);
        if (s != AMQ_OK) break;
        s = product(Wi_codes, Wi_alpha, 4 * H, I, k_w, ws.xcodes, ws.xbeta, k_e, bias, ws.proj);
        if (s != AMQ_OK) break;
        s = product(Wh_codes, Wh_alpha, 4 * H, H, k_w, ws.hcodes, ws.hbeta, k_a, nullptr, ws.pre);
        if (s != AMQ_OK) break;
        s = amq::launch_lstm_gates(ws.pre, ws.proj, c, h, c, H, st, true);                  // state updated in place
        if (s != AMQ_OK) break;
        if (amq::quantized_gemv_supported(H) && k_a <= 2) {       // (with more planes the repeated k x k solves cost more than a launch)
            // the quantizer on the new state runs inside the output product's kernel, which also leaves the planes and
            // coefficients for the recurrent product of the next token
            s = amq::launch_quantized_gemv(Ws_codes, Ws_alpha, vocab, H, k_s, h, k_a, T, bias_s, ws.logits, ws.hcodes, ws.hbeta,
                                           st, true);
        } else {
            s = amq::launch_quantize(h, H, H, nullptr, 0, 0, 1, k_a, T, ws.hcodes, ws.hbeta, st, true);
            if (s != AMQ_OK) break;
            s = product(Ws_codes, Ws_alpha, vocab, H, k_s, ws.hcodes, ws.hbeta, k_a, bias_s, ws.logits);
        }
        if (s != AMQ_OK) break;
        s = amq::launch_log_softmax_argmax(ws.logits, 1, vocab, vocab, logp ? logp + (size_t)t * vocab : nullptr, vocab,
                                           tokens + t + 1, st, true);
    }
    return s;
}

}  // extern "C"
