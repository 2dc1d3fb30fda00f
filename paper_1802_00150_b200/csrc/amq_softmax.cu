// Output layer of Eq. 6, y = softmax(W_s h + b_s), on logits the binary product has produced: log-probabilities
// and the arg-max token, one CTA per row of logits (a vocabulary of tens of thousands fits three passes over
// L2-resident data: maximum, sum of exponentials, write).
#include "amq_common.cuh"

namespace amq {

namespace {

constexpr int SM_THREADS = 1024;

// (value, index) maximum; among equal values the smaller index wins
__device__ __forceinline__ void max_combine(float& v, int& i, float ov, int oi)
{
    if (ov > v || (ov == v && oi < i)) { v = ov; i = oi; }
}

__global__ void __launch_bounds__(SM_THREADS)
log_softmax_argmax_kernel(const float* __restrict__ logits, int n, int ld, float* __restrict__ logp, int ldp,
                          int32_t* __restrict__ arg)
{
    __shared__ float s_val[32];
    __shared__ int s_idx[32];
    __shared__ float s_sum[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float* z = logits + (size_t)blockIdx.x * ld;

    // pass 1: maximum and its first index
    float mv = -INFINITY;
    int mi = 0x7fffffff;
    for (int t = tid; t < n; t += SM_THREADS) max_combine(mv, mi, __ldg(z + t), t);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1)
        max_combine(mv, mi, __shfl_xor_sync(0xffffffffu, mv, off), __shfl_xor_sync(0xffffffffu, mi, off));
    if (lane == 0) { s_val[warp] = mv; s_idx[warp] = mi; }
    __syncthreads();
    mv = s_val[lane]; mi = s_idx[lane];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1)
        max_combine(mv, mi, __shfl_xor_sync(0xffffffffu, mv, off), __shfl_xor_sync(0xffffffffu, mi, off));

    // pass 2: sum of exp(z - max), fixed order (thread-strided, then butterflies)
    float sum = 0.0f;
    for (int t = tid; t < n; t += SM_THREADS) sum += __expf(__ldg(z + t) - mv);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
    if (lane == 0) s_sum[warp] = sum;
    __syncthreads();
    sum = s_sum[lane];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
    const float lse = mv + logf(sum);

    if (logp) {
        float* out = logp + (size_t)blockIdx.x * ldp;
        for (int t = tid; t < n; t += SM_THREADS) out[t] = __ldg(z + t) - lse;
    }
    if (arg && tid == 0) arg[blockIdx.x] = mi;
}

}  // namespace
}  // namespace amq

extern "C" amq_status amq_log_softmax_argmax(const float* logits, int rows, int n, int ld,
                                             float* logp, int ldp, int32_t* argmax, void* stream)
{
    if (rows < 0 || n < 1 || ld < n || (logp && ldp < n)) return AMQ_ERR_INVALID_ARG;
    if (rows == 0) return AMQ_OK;
    if (!logits || (!logp && !argmax)) return AMQ_ERR_INVALID_ARG;
    amq::log_softmax_argmax_kernel<<<(unsigned)rows, amq::SM_THREADS, 0, (cudaStream_t)stream>>>(logits, n, ld, logp, ldp, argmax);
    AMQ_LAUNCH_CHECK();
    return AMQ_OK;
}
