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

// (value, index) maximum over the CTA; every thread returns the result
__device__ __forceinline__ void block_max(float& mv, int& mi, float* s_val, int* s_idx)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1)
        max_combine(mv, mi, __shfl_xor_sync(0xffffffffu, mv, off), __shfl_xor_sync(0xffffffffu, mi, off));
    if (lane == 0) { s_val[warp] = mv; s_idx[warp] = mi; }
    __syncthreads();
    mv = s_val[lane]; mi = s_idx[lane];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1)
        max_combine(mv, mi, __shfl_xor_sync(0xffffffffu, mv, off), __shfl_xor_sync(0xffffffffu, mi, off));
}

__device__ __forceinline__ float block_sum(float sum, float* s_sum)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
    if (lane == 0) s_sum[warp] = sum;
    __syncthreads();
    sum = s_sum[lane];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
    return sum;
}

// Rows of up to SM_THREADS * 4 * VEC floats whose start is 16-byte aligned: the row is read once, as float4, and
// stays in registers for the three steps (maximum, sum of exponentials, write).
constexpr int VEC = 12;

__global__ void __launch_bounds__(SM_THREADS)
log_softmax_argmax_resident_kernel(const float* logits, int n, int ld, float* __restrict__ logp, int ldp,
                                   int32_t* __restrict__ arg)
{
    grid_dependency_wait();             // the logits come from the preceding kernel of the stream
    __shared__ float s_val[32];
    __shared__ int s_idx[32];
    __shared__ float s_sum[32];
    const int tid = threadIdx.x;
    const float* z = logits + (size_t)blockIdx.x * ld;
    const int n4 = n >> 2;                                          // whole float4 groups; the tail is handled by scalars
    float4 v[VEC];
#pragma unroll
    for (int q = 0; q < VEC; ++q) {
        const int t4 = tid + q * SM_THREADS;
        v[q] = t4 < n4 ? __ldcg(reinterpret_cast<const float4*>(z) + t4) : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
    }
    const int tail = n4 * 4 + tid;                                  // at most three tail elements, one per thread
    const float vt = tail < n ? __ldcg(z + tail) : -INFINITY;

    float mv = vt;
    int mi = tail < n ? tail : 0x7fffffff;
#pragma unroll
    for (int q = 0; q < VEC; ++q) {
        const int base = (tid + q * SM_THREADS) * 4;
        max_combine(mv, mi, v[q].x, base); max_combine(mv, mi, v[q].y, base + 1);
        max_combine(mv, mi, v[q].z, base + 2); max_combine(mv, mi, v[q].w, base + 3);
    }
    block_max(mv, mi, s_val, s_idx);

    float sum = tail < n ? __expf(vt - mv) : 0.0f;
#pragma unroll
    for (int q = 0; q < VEC; ++q)                                    // exp(-inf) = 0 for the positions past the end
        sum += (__expf(v[q].x - mv) + __expf(v[q].y - mv)) + (__expf(v[q].z - mv) + __expf(v[q].w - mv));
    sum = block_sum(sum, s_sum);
    const float lse = mv + logf(sum);

    if (logp) {
        float* out = logp + (size_t)blockIdx.x * ldp;
        if ((ldp & 3) == 0 && (reinterpret_cast<uintptr_t>(logp) & 15) == 0) {
#pragma unroll
            for (int q = 0; q < VEC; ++q) {
                const int t4 = tid + q * SM_THREADS;
                if (t4 < n4) reinterpret_cast<float4*>(out)[t4] = make_float4(v[q].x - lse, v[q].y - lse, v[q].z - lse, v[q].w - lse);
            }
        } else {
#pragma unroll
            for (int q = 0; q < VEC; ++q) {
                const int t4 = tid + q * SM_THREADS;
                if (t4 < n4) { out[4 * t4] = v[q].x - lse; out[4 * t4 + 1] = v[q].y - lse; out[4 * t4 + 2] = v[q].z - lse; out[4 * t4 + 3] = v[q].w - lse; }
            }
        }
        if (tail < n) out[tail] = vt - lse;
    }
    if (arg && tid == 0) arg[blockIdx.x] = mi;
}

__global__ void __launch_bounds__(SM_THREADS)
log_softmax_argmax_kernel(const float* logits, int n, int ld, float* __restrict__ logp, int ldp,
                          int32_t* __restrict__ arg)
{
    grid_dependency_wait();             // the logits come from the preceding kernel of the stream
    __shared__ float s_val[32];
    __shared__ int s_idx[32];
    __shared__ float s_sum[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float* z = logits + (size_t)blockIdx.x * ld;

    // pass 1: maximum and its first index
    float mv = -INFINITY;
    int mi = 0x7fffffff;
    for (int t = tid; t < n; t += SM_THREADS) max_combine(mv, mi, __ldcg(z + t), t);
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
    for (int t = tid; t < n; t += SM_THREADS) sum += __expf(__ldcg(z + t) - mv);
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
        for (int t = tid; t < n; t += SM_THREADS) out[t] = __ldcg(z + t) - lse;
    }
    if (arg && tid == 0) arg[blockIdx.x] = mi;
}

}  // namespace

amq_status launch_log_softmax_argmax(const float* logits, int rows, int n, int ld, float* logp, int ldp, int32_t* argmax,
                                     cudaStream_t st, bool overlap_with_previous)
{
    const bool resident = n <= SM_THREADS * 4 * VEC && (ld & 3) == 0 && (reinterpret_cast<uintptr_t>(logits) & 15) == 0;
    AMQ_CUDA_TRY(launch_kernel(resident ? log_softmax_argmax_resident_kernel : log_softmax_argmax_kernel, dim3((unsigned)rows),
                               dim3(SM_THREADS), 0, st, overlap_with_previous, logits, n, ld, logp, ldp, argmax));
    AMQ_LAUNCH_CHECK();
    return AMQ_OK;
}

}  // namespace amq

extern "C" amq_status amq_log_softmax_argmax(const float* logits, int rows, int n, int ld,
                                             float* logp, int ldp, int32_t* argmax, void* stream)
{
    if (rows < 0 || n < 1 || ld < n || (logp && ldp < n)) return AMQ_ERR_INVALID_ARG;
    if (rows == 0) return AMQ_OK;
    if (!logits || (!logp && !argmax)) return AMQ_ERR_INVALID_ARG;
    return amq::launch_log_softmax_argmax(logits, rows, n, ld, logp, ldp, argmax, (cudaStream_t)stream, false);
}
