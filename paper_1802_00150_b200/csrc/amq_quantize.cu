// Row-wise alternating multi-bit quantizer (Algorithm 2) as a stand-alone kernel: one thread group per
// row, the row held in registers, used for weights (bulk, offline) and for batches of activations.
#include "amq_common.cuh"
#include "amq_quantize_device.cuh"

namespace amq {

namespace {

struct RowSource {
    const float* src0; int ld0; int n0;
    const float* src1; int ld1;
    bool overlap_with_previous;     // host side only: launch as a programmatic dependent of the preceding kernel
};

__device__ __forceinline__ float load_elem(const RowSource& s, int row, int t)
{
    // ordinary L2-cached loads: with an overlapped launch the state may still be written while this kernel is alive
    return (t < s.n0) ? __ldcg(s.src0 + (size_t)row * s.ld0 + t) : __ldcg(s.src1 + (size_t)row * s.ld1 + (t - s.n0));
}

// Bulk variant, one row of up to 1024 elements per warp: lane l holds the 32 CONSECUTIVE elements 32 l ..
// 32 l + 31 (eight 128-bit loads), so the sign word the quantizer leaves in a lane IS packed word l of the
// plane and goes straight to memory, 128 contiguous bytes per warp and plane, with no ballot transposition.
// Requires a single 16-byte-aligned source with a row stride that is a multiple of 4 elements.
template <int K>
__global__ void __launch_bounds__(128)
quantize_rows_consecutive_kernel(const float* __restrict__ x, int ldx, int rows, int n, int T,
                                 uint32_t* __restrict__ codes, float* __restrict__ coeffs)
{
    __shared__ QuantScratch<K, 1> scratch[4];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int row = blockIdx.x * (blockDim.x >> 5) + warp;
    if (row >= rows) return;
    const float* src = x + (size_t)row * ldx + lane * 32;
    float w[32];
    uint32_t valid = 0;
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        const int t = lane * 32 + q * 4;
        float4 v = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        if (t + 3 < n) {
            v = __ldcs(reinterpret_cast<const float4*>(src) + q);
            valid |= 0xFu << (q * 4);
        } else {
            if (t < n) { v.x = __ldcs(src + q * 4); valid |= 1u << (q * 4); }
            if (t + 1 < n) { v.y = __ldcs(src + q * 4 + 1); valid |= 2u << (q * 4); }
            if (t + 2 < n) { v.z = __ldcs(src + q * 4 + 2); valid |= 4u << (q * 4); }
        }
        w[q * 4] = v.x; w[q * 4 + 1] = v.y; w[q * 4 + 2] = v.z; w[q * 4 + 3] = v.w;
    }
    float alpha[K];
    uint32_t bits[K];
    quantize_group<K, 32, 1>(w, valid, n, quant_padding_consecutive(n, 32), T, alpha, bits, scratch[warp]);
    const int wpr = 4 * ((n + 127) / 128);
    if (lane < wpr) {
#pragma unroll
        for (int i = 0; i < K; ++i) codes[((size_t)row * K + i) * wpr + lane] = bits[i];
    }
    if (lane < K) {
        float a = alpha[0];
#pragma unroll
        for (int i = 1; i < K; ++i) a = (lane == i) ? alpha[i] : a;
        coeffs[(size_t)row * K + lane] = a;
    }
}

// K bits, EPT elements per thread.
// MULTI: one row per CTA; thread g owns the EPT CONSECUTIVE elements g * EPT .. g * EPT + EPT - 1 (EPT = 8 with 256
// threads, or 32), so the sign bits the quantizer leaves in a register are a byte (a word) of the packed plane and are
// stored as such, without a ballot transposition.  The fused matrix-vector kernel quantizes a vector with the same
// ownership, thread count and summation order, so both leave the same bits.
// Otherwise one row per warp, lane l owning the elements j * 32 + l.
template <int K, int EPT, bool MULTI>
__global__ void __launch_bounds__(256)
quantize_kernel(RowSource src, int rows, int n, int T, uint32_t* __restrict__ codes, float* __restrict__ coeffs)
{
    constexpr int NW = MULTI ? 8 : 1;
    __shared__ QuantScratch<K, NW> scratch[MULTI ? 1 : 4];
    if (MULTI) quant_scratch_init(scratch[0]);
    grid_dependency_wait();             // launched early behind a product kernel: its state output must be complete

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = MULTI ? threadIdx.x : lane;
    const int row = MULTI ? blockIdx.x : blockIdx.x * (blockDim.x >> 5) + warp;
    if (row >= rows) return;          // whole group leaves together (row is uniform across the group)

    float w[EPT];
    uint32_t valid = 0;
    if (MULTI) {
        const int t0 = g * EPT;
        // whole 16-byte pieces of one source where the addresses allow, single elements otherwise
#pragma unroll
        for (int q = 0; q < EPT / 4; ++q) {
            const int t = t0 + 4 * q;
            const float* p = (t < src.n0) ? src.src0 + (size_t)row * src.ld0 + t : src.src1 + (size_t)row * src.ld1 + (t - src.n0);
            const bool one_piece = t + 3 < n && (t + 3 < src.n0 || t >= src.n0) && (reinterpret_cast<uintptr_t>(p) & 15u) == 0;
            if (one_piece) {
                const float4 v = __ldcg(reinterpret_cast<const float4*>(p));
                w[4 * q] = v.x; w[4 * q + 1] = v.y; w[4 * q + 2] = v.z; w[4 * q + 3] = v.w;
                valid |= 0xFu << (4 * q);
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const bool ok = t + e < n;
                    w[4 * q + e] = ok ? load_elem(src, row, t + e) : 0.0f;
                    valid |= (ok ? 1u : 0u) << (4 * q + e);
                }
            }
        }
    } else {
#pragma unroll
        for (int j = 0; j < EPT; ++j) {
            const int t = j * 32 + g;
            const bool ok = t < n;
            w[j] = ok ? load_elem(src, row, t) : 0.0f;
            valid |= (ok ? 1u : 0u) << j;
        }
    }

    float alpha[K];
    uint32_t bits[K];
    quantize_group<K, EPT, NW>(w, valid, n, MULTI ? quant_padding_consecutive(n, EPT) : quant_padding_strided32(n, EPT), T,
                               alpha, bits, scratch[MULTI ? 0 : warp]);

    const int wpr = 4 * ((n + 127) / 128);
    if (MULTI) {
        if (g * EPT < wpr * 32) {       // this thread's bits lie inside the plane (zeros past the end of the vector)
#pragma unroll
            for (int i = 0; i < K; ++i) {
                uint32_t* plane = codes + ((size_t)row * K + i) * wpr;
                if (EPT == 8) reinterpret_cast<uint8_t*>(plane)[g] = (uint8_t)bits[i];
                else plane[g] = bits[i];
            }
        }
    } else {
        pack_group<K, EPT>(bits, lane, 0, 1, wpr, codes + (size_t)row * K * wpr);
    }
    if (g < K) {
        float a = alpha[0];
#pragma unroll
        for (int i = 1; i < K; ++i) a = (g == i) ? alpha[i] : a;
        coeffs[(size_t)row * K + g] = a;
    }
}

template <int K, int EPT, bool MULTI>
amq_status run(const RowSource& src, int rows, int n, int T, uint32_t* codes, float* coeffs, int threads,
               cudaStream_t st)
{
    const int rows_per_cta = MULTI ? 1 : threads / 32;
    const unsigned grid = (unsigned)((rows + rows_per_cta - 1) / rows_per_cta);
    if (src.overlap_with_previous) {
        // may be scheduled while the preceding kernel of the stream still runs; the kernel waits for it first thing
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3(grid); cfg.blockDim = dim3((unsigned)threads); cfg.dynamicSmemBytes = 0; cfg.stream = st;
        cudaLaunchAttribute attr{};
        attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr.val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = &attr; cfg.numAttrs = 1;
        AMQ_CUDA_TRY(cudaLaunchKernelEx(&cfg, quantize_kernel<K, EPT, MULTI>, src, rows, n, T, codes, coeffs));
        AMQ_LAUNCH_CHECK();
        return AMQ_OK;
    }
    quantize_kernel<K, EPT, MULTI><<<grid, threads, 0, st>>>(src, rows, n, T, codes, coeffs);
    AMQ_LAUNCH_CHECK();
    return AMQ_OK;
}

template <int K>
amq_status dispatch(const RowSource& src, int rows, int n, int T, uint32_t* codes, float* coeffs, cudaStream_t st)
{
    const int n128 = 128 * ((n + 127) / 128);
    const bool bulk = rows >= 1024;
    if (bulk && n128 > 256 && n128 <= 1024 && src.n0 == n && (src.ld0 & 3) == 0 &&
        (reinterpret_cast<uintptr_t>(src.src0) & 15u) == 0) {
        quantize_rows_consecutive_kernel<K><<<(unsigned)((rows + 3) / 4), 128, 0, st>>>(src.src0, src.ld0, rows, n, T, codes, coeffs);
        AMQ_LAUNCH_CHECK();
        return AMQ_OK;
    }
    if (bulk && n128 <= 256) return run<K, 8, false>(src, rows, n, T, codes, coeffs, 128, st);
    if (bulk && n128 <= 1024) return run<K, 32, false>(src, rows, n, T, codes, coeffs, 128, st);
    if (bulk || n128 > 2048) {
        const int threads = 32 * ((n128 / 32 + 31) / 32);      // 32 elements per thread
        return run<K, 32, true>(src, rows, n, T, codes, coeffs, threads, st);
    }
    return run<K, 8, true>(src, rows, n, T, codes, coeffs, 256, st);     // 8 elements per thread, always 256 threads
}

}  // namespace

amq_status launch_quantize(const float* src0, int ld0, int n0, const float* src1, int ld1, int n1,
                           int rows, int k, int T, uint32_t* codes, float* coeffs, cudaStream_t st, bool overlap_with_previous)
{
    RowSource src{src0, ld0, n0, src1, ld1, overlap_with_previous};
    const int n = n0 + n1;
    switch (k) {
        case 1: return dispatch<1>(src, rows, n, T, codes, coeffs, st);
        case 2: return dispatch<2>(src, rows, n, T, codes, coeffs, st);
        case 3: return dispatch<3>(src, rows, n, T, codes, coeffs, st);
        case 4: return dispatch<4>(src, rows, n, T, codes, coeffs, st);
    }
    return AMQ_ERR_UNSUPPORTED;
}

}  // namespace amq

extern "C" amq_status amq_quantize(const float* x, int rows, int n, int ldx, int k, int T,
                                   uint32_t* codes, float* coeffs, void* stream)
{
    if (rows < 0 || n < 1 || ldx < n) return AMQ_ERR_INVALID_ARG;
    if (!amq::valid_k(k) || T < 0 || n > AMQ_MAX_N) return AMQ_ERR_UNSUPPORTED;
    if (rows == 0) return AMQ_OK;       // nothing to do; pointers of empty buffers may be NULL
    if (!x || !codes || !coeffs) return AMQ_ERR_INVALID_ARG;
    if (!amq::aligned16(codes)) return AMQ_ERR_ALIGNMENT;
    return amq::launch_quantize(x, ldx, n, nullptr, 0, 0, rows, k, T, codes, coeffs, (cudaStream_t)stream);
}
