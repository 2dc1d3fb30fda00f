// GRU step in the original form of the GRU the paper cites (Cho et al., 2014): the reset gate multiplies the
// previous state before the candidate's product, so a step quantizes two vectors on-line:
//   z1 = [x ; h]:      r = logistic(W_r z1_hat + b_r),  z = logistic(W_z z1_hat + b_z);
//   z2 = [x ; r * h]:  cand = tanh(W_n z2_hat + b_n);   h' = (1 - z) * cand + z * h.
// Six launches on the caller's stream: quantizer, product with the r and z rows, reset kernel, quantizer, product
// with the n rows, blend kernel.  (The default GRU of this library applies r after the product and needs one
// quantization and one product per step.)
#include "amq_common.cuh"

namespace amq {
namespace {

struct GruOrigWorkspace {
    uint32_t* zcodes;   // [batch][k_a][wpr(I + H)]
    float* zbeta;       // [batch][k_a]
    float* prz;         // [batch][2H] pre-activations of r and z (bias included)
    float* rh;          // [batch][H]  r * h
    float* pn;          // [batch][H]  pre-activation of the candidate (bias included)
    size_t bytes;
};

GruOrigWorkspace carve(void* base, int I, int H, int batch, int k_a)
{
    GruOrigWorkspace w;
    char* p = static_cast<char*>(base);
    size_t off = 0;
    w.zcodes = reinterpret_cast<uint32_t*>(p + off); off += round_up((size_t)batch * k_a * words_per_row(I + H) * 4, 256);
    w.zbeta = reinterpret_cast<float*>(p + off);     off += round_up((size_t)batch * k_a * 4, 256);
    w.prz = reinterpret_cast<float*>(p + off);       off += round_up((size_t)batch * 2 * H * 4, 256);
    w.rh = reinterpret_cast<float*>(p + off);        off += round_up((size_t)batch * H * 4, 256);
    w.pn = reinterpret_cast<float*>(p + off);        off += round_up((size_t)batch * H * 4, 256);
    w.bytes = off;
    return w;
}

// (both elementwise kernels read what the preceding kernels of the stream wrote: ordinary loads after the wait)
__global__ void gru_reset_kernel(const float* prz, const float* h, float* rh, int H, long long total)
{
    grid_dependency_wait();
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const long long b = idx / H;
    const int u = (int)(idx - b * H);
    rh[idx] = __ldcg(h + idx) / (1.0f + __expf(-__ldcg(prz + b * 2 * H + u)));
}

__global__ void gru_blend_kernel(const float* prz, const float* pn, const float* h, float* h_out, int H, long long total)
{
    grid_dependency_wait();
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const long long b = idx / H;
    const int u = (int)(idx - b * H);
    const float zg = 1.0f / (1.0f + __expf(-__ldcg(prz + b * 2 * H + H + u)));
    h_out[idx] = (1.0f - zg) * tanhf(__ldcg(pn + idx)) + zg * __ldcg(h + idx);
}

}  // namespace
}  // namespace amq

extern "C" {

size_t amq_gru_original_workspace_bytes(int I, int H, int batch, int k_a)
{
    if (I < 0 || H < 1 || batch < 0 || !amq::valid_k(k_a)) return 0;
    return amq::carve(nullptr, I, H, batch, k_a).bytes;
}

amq_status amq_gru_step_original(const uint32_t* Wcodes, const float* Walpha, const float* bias, int I, int H, int k_w,
                                 const float* x, const float* h_in, int batch, int k_a, int T, float* h_out,
                                 void* workspace, size_t workspace_bytes, void* stream)
{
    if (!Wcodes || !Walpha || I < 0 || H < 1 || batch < 0) return AMQ_ERR_INVALID_ARG;
    if (!amq::valid_k(k_w) || !amq::valid_k(k_a) || T < 0 || I + H > AMQ_MAX_N) return AMQ_ERR_UNSUPPORTED;
    if (!amq::aligned16(Wcodes)) return AMQ_ERR_ALIGNMENT;
    if (!workspace || workspace_bytes < amq_gru_original_workspace_bytes(I, H, batch, k_a)) return AMQ_ERR_WORKSPACE;
    if (!amq::aligned16(workspace)) return AMQ_ERR_ALIGNMENT;
    if (batch == 0) return AMQ_OK;
    if (!h_in || !h_out || (I > 0 && !x) || h_out == h_in) return AMQ_ERR_INVALID_ARG;
    const amq::GruOrigWorkspace ws = amq::carve(workspace, I, H, batch, k_a);
    cudaStream_t st = (cudaStream_t)stream;
    const int n = I + H, wpr = amq::words_per_row(n);
    const long long total = (long long)batch * H;
    const unsigned blocks = (unsigned)((total + 255) / 256);

    // every kernel of the step waits for its predecessor first thing and is launched as its programmatic dependent
    auto product = [&](const uint32_t* Wc, const float* Wa, int m, const float* b, float* y) {
        amq::GemmArgs a{};
        a.Wcodes = Wc; a.Walpha = Wa; a.m = m; a.n = n; a.k_w = k_w;
        a.xcodes = ws.zcodes; a.xbeta = ws.zbeta; a.batch = batch; a.k_a = k_a;
        a.bias = b; a.epilogue = amq::EPI_Y; a.y = y; a.ldy = m;
        a.overlap_with_previous = true;
        return amq::launch_binary_gemm(a, st);
    };
    amq_status s = amq::launch_quantize(x, I, I, h_in, H, H, batch, k_a, T, ws.zcodes, ws.zbeta, st, true);
    if (s != AMQ_OK) return s;
    s = product(Wcodes, Walpha, 2 * H, bias, ws.prz);
    if (s != AMQ_OK) return s;
    AMQ_CUDA_TRY(amq::launch_kernel(amq::gru_reset_kernel, dim3(blocks), dim3(256), 0, st, true, ws.prz, h_in, ws.rh, H, total));
    AMQ_LAUNCH_CHECK();
    s = amq::launch_quantize(x, I, I, ws.rh, H, H, batch, k_a, T, ws.zcodes, ws.zbeta, st, true);
    if (s != AMQ_OK) return s;
    s = product(Wcodes + (size_t)2 * H * k_w * wpr, Walpha + (size_t)2 * H * k_w, H, bias ? bias + 2 * H : nullptr, ws.pn);
    if (s != AMQ_OK) return s;
    AMQ_CUDA_TRY(amq::launch_kernel(amq::gru_blend_kernel, dim3(blocks), dim3(256), 0, st, true, ws.prz, ws.pn, h_in, h_out, H, total));
    AMQ_LAUNCH_CHECK();
    return AMQ_OK;
}

}  // extern "C"
