// Bit-plane packing and reconstruction, plus the small host-side entry points of the C ABI.
#include "amq_common.cuh"

namespace amq {

thread_local int g_last_cuda_error = 0;
unsigned long long g_kernel_launches = 0;

namespace {

// One warp per packed word: lane j tests element 32q + j of its plane; the ballot is the word.
__global__ void pack_kernel(const float* __restrict__ planes, size_t vectors /* rows*k */, int n, int wpr,
                            uint32_t* __restrict__ codes)
{
    const size_t warp = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= vectors * (size_t)wpr) return;
    const size_t vec = warp / wpr;
    const int q = (int)(warp % wpr);
    const int t = q * 32 + lane;
    const bool bit = (t < n) && (planes[vec * (size_t)n + t] >= 0.0f);
    const uint32_t word = __ballot_sync(0xffffffffu, bit);
    if (lane == 0) codes[vec * (size_t)wpr + q] = word;
}

// One thread per element: xhat = sum_i coeff_i * (+1 / -1), Eq. 2.
__global__ void unpack_kernel(const uint32_t* __restrict__ codes, const float* __restrict__ coeffs,
                              size_t rows, int n, int k, int wpr, float* __restrict__ xhat)
{
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= rows * (size_t)n) return;
    const size_t row = idx / n;
    const int t = (int)(idx % n);
    float s = 0.0f;
    for (int i = 0; i < k; ++i) {
        const uint32_t word = codes[(row * k + i) * (size_t)wpr + (t >> 5)];
        const float a = coeffs[row * k + i];
        s += ((word >> (t & 31)) & 1u) ? a : -a;
    }
    xhat[idx] = s;
}

// One thread per 128-bit chunk of the gathered rows: out row c <- table row tokens[c] (codes), and the row's
// coefficients by the first k threads of the row.
__global__ void embedding_rows_kernel(const uint4* __restrict__ codes, const float* __restrict__ coeffs, int vocab,
                                      const int32_t* tokens, size_t count, int k, int chunks /* k * wpr / 4 */,
                                      uint4* __restrict__ out_codes, float* __restrict__ out_coeffs)
{
    grid_dependency_wait();             // the token ids may come from the preceding kernel (greedy decoding)
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= count * (size_t)chunks) return;
    const size_t row = idx / chunks;
    const int c = (int)(idx - row * chunks);
    int tok = __ldcg(tokens + row);
    tok = tok < 0 ? 0 : (tok >= vocab ? vocab - 1 : tok);          // out-of-range ids are clamped, never dereferenced
    out_codes[idx] = __ldg(codes + (size_t)tok * chunks + c);
    if (c < k) out_coeffs[row * k + c] = __ldg(coeffs + (size_t)tok * k + c);
}

}  // namespace

amq_status launch_embedding_rows(const uint32_t* We_codes, const float* We_alpha, int vocab, int n, int k, const int32_t* tokens,
                                 int count, uint32_t* xcodes, float* xbeta, cudaStream_t st, bool overlap_with_previous)
{
    const int chunks = k * words_per_row(n) / 4;
    const size_t total = (size_t)count * chunks;
    const size_t blocks = (total + 255) / 256;
    if (blocks > 0x7fffffffull) return AMQ_ERR_UNSUPPORTED;
    AMQ_CUDA_TRY(launch_kernel(embedding_rows_kernel, dim3((unsigned)blocks), dim3(256), 0, st, overlap_with_previous,
                               reinterpret_cast<const uint4*>(We_codes), We_alpha, vocab, tokens, (size_t)count, k, chunks,
                               reinterpret_cast<uint4*>(xcodes), xbeta));
    AMQ_LAUNCH_CHECK();
    return AMQ_OK;
}

}  // namespace amq

extern "C" {

const char* amq_status_string(amq_status s)
{
    switch (s) {
        case AMQ_OK: return "ok";
        case AMQ_ERR_INVALID_ARG: return "invalid argument";
        case AMQ_ERR_UNSUPPORTED: return "unsupported size or bit count";
        case AMQ_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
        case AMQ_ERR_WORKSPACE: return "workspace missing or too small";
        case AMQ_ERR_CUDA: return "CUDA runtime error";
        case AMQ_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

int amq_last_cuda_error(void) { return amq::g_last_cuda_error; }

unsigned long long amq_kernel_launches(void) { return __atomic_load_n(&amq::g_kernel_launches, __ATOMIC_RELAXED); }

int amq_words_per_row(int n) { return n < 1 ? 0 : amq::words_per_row(n); }

size_t amq_codes_bytes(int rows, int n, int k)
{
    if (rows < 0 || n < 1 || k < 1) return 0;
    return (size_t)rows * (size_t)k * (size_t)amq::words_per_row(n) * 4u;
}

amq_status amq_pack(const float* planes, int rows, int n, int k, uint32_t* codes, void* stream)
{
    if (!planes || !codes || rows < 0 || n < 1) return AMQ_ERR_INVALID_ARG;
    if (!amq::valid_k(k)) return AMQ_ERR_UNSUPPORTED;
    if (!amq::aligned16(codes)) return AMQ_ERR_ALIGNMENT;
    if (rows == 0) return AMQ_OK;
    const int wpr = amq::words_per_row(n);
    const size_t warps = (size_t)rows * k * wpr;
    const size_t blocks = (warps * 32 + 255) / 256;
    if (blocks > 0x7fffffffull) return AMQ_ERR_UNSUPPORTED;
    amq::pack_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(planes, (size_t)rows * k, n, wpr, codes);
    AMQ_LAUNCH_CHECK();
    return AMQ_OK;
}

amq_status amq_embedding_rows(const uint32_t* We_codes, const float* We_alpha, int vocab, int n, int k,
                              const int32_t* tokens, int count, uint32_t* xcodes, float* xbeta, void* stream)
{
    if (count < 0 || vocab < 1 || n < 1) return AMQ_ERR_INVALID_ARG;
    if (!amq::valid_k(k)) return AMQ_ERR_UNSUPPORTED;
    if (count == 0) return AMQ_OK;
    if (!We_codes || !We_alpha || !tokens || !xcodes || !xbeta) return AMQ_ERR_INVALID_ARG;
    if (!amq::aligned16(We_codes) || !amq::aligned16(xcodes)) return AMQ_ERR_ALIGNMENT;
    return amq::launch_embedding_rows(We_codes, We_alpha, vocab, n, k, tokens, count, xcodes, xbeta, (cudaStream_t)stream, false);
}

amq_status amq_unpack(const uint32_t* codes, const float* coeffs, int rows, int n, int k,
                      float* xhat, void* stream)
{
    if (!codes || !coeffs || !xhat || rows < 0 || n < 1) return AMQ_ERR_INVALID_ARG;
    if (!amq::valid_k(k)) return AMQ_ERR_UNSUPPORTED;
    if (!amq::aligned16(codes)) return AMQ_ERR_ALIGNMENT;
    if (rows == 0) return AMQ_OK;
    const size_t total = (size_t)rows * n;
    const size_t blocks = (total + 255) / 256;
    if (blocks > 0x7fffffffull) return AMQ_ERR_UNSUPPORTED;
    amq::unpack_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(codes, coeffs, (size_t)rows, n, k,
                                                                          amq::words_per_row(n), xhat);
    AMQ_LAUNCH_CHECK();
    return AMQ_OK;
}

}  // extern "C"
