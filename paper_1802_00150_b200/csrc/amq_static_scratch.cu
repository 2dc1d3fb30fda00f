// amq_lstm_step_static: the quantized LSTM step for callers that cannot allocate device memory.
//
// Some hosts of this library never get to call cudaMalloc: a plug-in running inside another
// application's allocator budget, a real-time inference loop that must not touch the driver's heap once
// it has started, a process whose memory pool was handed out in full before this library was loaded.
// amq_lstm_step needs a caller-provided workspace for the packed codes and coefficients of the on-line
// quantized activation; this variant keeps that scratch in a fixed array that is part of the library
// image, so the caller passes only inputs and outputs.
//
// The array lives in the data segment of every device that loads the library (AMQ_STATIC_SCRATCH_BYTES per
// GPU, until the process exits).  In host code the array's name is only a host-side handle, not a device
// address, so the address is looked up with cudaGetSymbolAddress (for the device that is current at the
// call) and handed to the kernels as an ordinary pointer.  The lookup is repeated on every call: once the
// module is loaded it is a table lookup, and an address remembered from an earlier call would be stale after
// the application reset the device or tore its context down.
#include "amq_common.cuh"

namespace amq {

namespace {

static __device__ __align__(256) unsigned char g_static_scratch[AMQ_STATIC_SCRATCH_BYTES];

// Device address of the scratch array on the current device.
amq_status static_scratch(unsigned char** out)
{
    void* p = nullptr;
    AMQ_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
    if (!p) return AMQ_ERR_CUDA;
    *out = static_cast<unsigned char*>(p);
    return AMQ_OK;
}

// Scratch layout: [activation codes: batch * k_a * wpr words][activation coefficients: batch * k_a floats]
size_t codes_bytes(int I, int H, int batch, int k_a)
{
    return round_up((size_t)batch * k_a * words_per_row(I + H) * 4, 256);
}

}  // namespace
}  // namespace amq

extern "C" {

size_t amq_lstm_step_static_scratch_bytes(int I, int H, int batch, int k_a)
{
    if (I < 0 || H < 1 || batch < 0 || !amq::valid_k(k_a)) return 0;
    return amq::codes_bytes(I, H, batch, k_a) + amq::round_up((size_t)batch * k_a * 4, 256);
}

amq_status amq_lstm_step_static(const uint32_t* Wcodes, const float* Walpha, const float* bias,
                                int I, int H, int k_w,
                                const float* x, const float* h_in, const float* c_in, int batch, int k_a, int T,
                                float* h_out, float* c_out, void* stream)
{
    if (!Wcodes || !Walpha || I < 0 || H < 1 || batch < 0) return AMQ_ERR_INVALID_ARG;
    if (!amq::valid_k(k_w) || !amq::valid_k(k_a) || T < 0 || I + H > AMQ_MAX_N) return AMQ_ERR_UNSUPPORTED;
    if (!amq::aligned16(Wcodes)) return AMQ_ERR_ALIGNMENT;
    if (amq_lstm_step_static_scratch_bytes(I, H, batch, k_a) > (size_t)AMQ_STATIC_SCRATCH_BYTES)
        return AMQ_ERR_WORKSPACE;               // the problem does not fit the built-in scratch
    if (!h_in || !c_in || !h_out || !c_out || (I > 0 && !x) || h_out == h_in) return AMQ_ERR_INVALID_ARG;
    if (batch == 0) return AMQ_OK;

    unsigned char* scratch = nullptr;
    amq_status s = amq::static_scratch(&scratch);
    if (s != AMQ_OK) return s;
    uint32_t* zcodes = reinterpret_cast<uint32_t*>(scratch);
    float* zbeta = reinterpret_cast<float*>(scratch + amq::codes_bytes(I, H, batch, k_a));
    cudaStream_t st = (cudaStream_t)stream;

    // Both regions are written in full by the quantizer before the product reads them (every word of
    // every plane, pad bits included), so nothing left by an earlier call can leak into this one.
    s = amq::launch_quantize(x, I, I, h_in, H, H, batch, k_a, T, zcodes, zbeta, st);
    if (s != AMQ_OK) return s;
    amq::GemmArgs a{};
    a.Wcodes = Wcodes; a.Walpha = Walpha; a.m = 4 * H; a.n = I + H; a.k_w = k_w;
    a.xcodes = zcodes; a.xbeta = zbeta; a.batch = batch; a.k_a = k_a;
    a.bias = bias; a.epilogue = amq::EPI_LSTM;
    a.I = I; a.H = H; a.h_in = h_in; a.c_in = c_in; a.h_out = h_out; a.c_out = c_out;
    return amq::launch_binary_gemm(a, st);
}

}  // extern "C"
