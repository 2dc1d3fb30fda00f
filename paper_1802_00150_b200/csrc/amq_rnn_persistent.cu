// Persistent, weight-stationary kernel for a batch-1 quantized LSTM / GRU sequence (Eq. 6 repeated over
// time; "RNNs can only be executed sequentially", Sec. 1).
//
// The hidden units are split over the CTAs of one co-resident (cooperative) grid; every CTA keeps the
// packed planes of its own gate rows in shared memory for the whole sequence.  A timestep is, in every
// CTA: gather z = [x_t ; h_{t-1}], quantize it on-line (Algorithm 2, all CTAs redundantly, so that one
// exchange per step is enough), XOR + bit-count its planes against the resident rows (Appendix A), fold
// the partials with the row-wise coefficients (Sec. 4), apply the gates and publish the new h slice.
//
// Exchange of h between CTAs: each value travels as one 64-bit word {fp32 bits, step tag}, written with
// a single relaxed gpu-scope store and polled with relaxed gpu-scope loads; a consumer accepts a word
// when its tag equals the step it is gathering for, so value and "ready" flag arrive together and no
// separate barrier, fence or atomic counter is on the critical path.  Two buffers alternate by step
// parity: a CTA can only run one step ahead of the slowest one (it needs every slice of the previous
// step), so a buffer is never overwritten while someone still reads it.  Every poll is bounded; when
// it runs out the CTA records AMQ_ERR_TIMEOUT in the workspace status word and leaves.
#include "amq_common.cuh"
#include "amq_quantize_device.cuh"

namespace amq {

namespace {

constexpr int NT = 512;                  // threads per CTA
constexpr unsigned POLL_LIMIT = 1u << 20;

struct PersistArgs {
    const uint32_t* Wcodes; const float* Walpha; const float* bias;
    int I, H, k_w, T, steps;
    const float* x_seq; const float* h0; const float* c0;
    float* h_seq; float* h_last; float* c_last;
    unsigned long long* hx;              // [2][H] exchange words
    uint32_t* status;
    int upc;                             // hidden units per CTA
    int wpr;
};

__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long* p)
{
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ void st_relaxed_u64(unsigned long long* p, unsigned long long v)
{
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" :: "l"(p), "l"(v) : "memory");
}

// gate nonlinearities from one fast exponential each (absolute error ~1e-7, far inside the output tolerance)
__device__ __forceinline__ float logistic(float v) { return __fdividef(1.0f, 1.0f + __expf(-v)); }
__device__ __forceinline__ float fast_tanh(float v) { return 1.0f - __fdividef(2.0f, 1.0f + __expf(2.0f * v)); }

__device__ __forceinline__ int popc4(uint4 a, uint4 b)
{
    return __popc(a.x ^ b.x) + __popc(a.y ^ b.y) + __popc(a.z ^ b.z) + __popc(a.w ^ b.w);
}

// Lanes per plane-row in the product phase: the largest power of two that still gives every plane-row of
// the CTA its own segment in one pass, at most one lane per 128-bit chunk, at most a warp.
__host__ __device__ inline int product_segment(int PR, int CH)
{
    int cap = 1;
    while (cap < CH && cap < 32) cap <<= 1;
    int seg = 1;
    while (seg * 2 <= cap && seg * 2 * PR <= NT) seg <<= 1;
    return seg;
}

// Row stride of the resident planes in 16-byte units: segments narrower than a quarter-warp are skewed so
// that the 8 lanes served together by one 128-bit shared-memory phase fall into distinct banks.
__host__ __device__ inline int product_row_stride(int CH, int SEG)
{
    return SEG >= 8 ? CH : CH + (((SEG - CH) % 8) + 8) % 8;
}

#ifdef AMQ_PHASE_TIMING
#define AMQ_PHASE(i) do { const long long now_ = clock64(); ph[i] += now_ - tp; tp = now_; } while (0)
#else
#define AMQ_PHASE(i) do { } while (0)
#endif

template <int KA, int EPT, bool GRU>
__global__ void __launch_bounds__(NT, 1)
rnn_persistent_kernel(PersistArgs a)
{
    constexpr int GATES = GRU ? 3 : 4;
    constexpr int PARTS = GRU ? 2 : 1;    // GRU keeps the product in two column segments, [0,I) and [I,n)
    extern __shared__ __align__(16) unsigned char smem_raw[];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = a.I + a.H, wpr = a.wpr, CH = wpr >> 2, k_w = a.k_w;
    const int upc = a.upc, rows = upc * GATES, PR = rows * k_w;
    const int u0 = blockIdx.x * upc;

    // product role: segments of SEG lanes share a plane-row; lane c of a segment owns chunks c, c + SEG, ..
    const int SEG = product_segment(PR, CH), RS = product_row_stride(CH, SEG);
    const int NSEG = NT / SEG, seg = tid / SEG, chunk = tid % SEG;
    const int pr_iters = (PR + NSEG - 1) / NSEG;

    // ---- shared memory carve-up ----
    uint4* sW = reinterpret_cast<uint4*>(smem_raw);                              // [PR][RS]
    uint4* sZ = sW + (size_t)PR * RS;                                            // [KA][CH]
    int* sP = reinterpret_cast<int*>(sZ + KA * CH);                              // [PARTS][PR][KA]
    float* sAlpha = reinterpret_cast<float*>(sP + PARTS * PR * KA);              // [PR]
    float* sBias = sAlpha + PR;                                                  // [upc][4]
    QuantScratch<KA>* scratch = reinterpret_cast<QuantScratch<KA>*>(
        (reinterpret_cast<uintptr_t>(sBias + upc * 4) + 15) & ~uintptr_t(15));

    // ---- resident weights: local plane-row pr = (ul * GATES + gate) * k_w + i ----
    {
        uint32_t* sWw = reinterpret_cast<uint32_t*>(sW);
        for (int idx = tid; idx < PR * wpr; idx += NT) {
            const int pr = idx / wpr, q = idx - pr * wpr;
            const int lr = pr / k_w, i = pr - lr * k_w;
            const int ul = lr / GATES, gate = lr - ul * GATES;
            const int u = u0 + ul;
            sWw[(size_t)pr * RS * 4 + q] =
                (u < a.H) ? __ldg(a.Wcodes + (((size_t)gate * a.H + u) * k_w + i) * wpr + q) : 0u;
        }
        for (int pr = tid; pr < PR; pr += NT) {
            const int lr = pr / k_w, i = pr - lr * k_w;
            const int ul = lr / GATES, gate = lr - ul * GATES;
            const int u = u0 + ul;
            sAlpha[pr] = (u < a.H) ? __ldg(a.Walpha + ((size_t)gate * a.H + u) * k_w + i) : 0.0f;
        }
        for (int idx = tid; idx < upc * 4; idx += NT) {
            const int ul = idx >> 2, s = idx & 3, u = u0 + ul;
            sBias[idx] = (a.bias && u < a.H) ? __ldg(a.bias + (size_t)s * a.H + u) : 0.0f;
        }
    }

    // epilogue role: thread e = ul * 4 + gate slot (slot 3 idle for the GRU), kept inside aligned quads
    const int ep_ul = tid >> 2, ep_gate = tid & 3;
    const int ep_warps = (upc * 4 + 31) >> 5;
    const bool ep_valid = ep_ul < upc && ep_gate < GATES && (u0 + ep_ul) < a.H;
    const bool ep_leader = ep_valid && ep_gate == 0;
    float c_state = 0.0f, h_state = 0.0f;
    if (ep_leader) {
        h_state = __ldg(a.h0 + u0 + ep_ul);
        if (!GRU) c_state = __ldg(a.c0 + u0 + ep_ul);
    }
    __syncthreads();

#ifdef AMQ_PHASE_TIMING
    long long ph[5] = {0, 0, 0, 0, 0};
    long long tp = clock64();
#endif

    for (int t = 0; t < a.steps; ++t) {
        // ---- 1. gather z = [x_t ; h_{t-1}] (element j * NT + tid) ----
        float w[EPT];
        uint32_t valid = 0, pending = 0;
        const float* x = a.x_seq + (size_t)t * a.I;
        const unsigned long long* hx = a.hx + (size_t)(t & 1) * a.H;
#pragma unroll
        for (int j = 0; j < EPT; ++j) {
            const int e = j * NT + tid;
            w[j] = 0.0f;
            if (e < a.I) { w[j] = __ldg(x + e); valid |= 1u << j; }
            else if (e < n) {
                valid |= 1u << j;
                if (t == 0) w[j] = __ldg(a.h0 + (e - a.I)); else pending |= 1u << j;
            }
        }
        unsigned spins = 0;
        while (pending) {
#pragma unroll
            for (int j = 0; j < EPT; ++j) {
                if ((pending >> j) & 1u) {
                    const unsigned long long v = ld_relaxed_u64(hx + (j * NT + tid - a.I));
                    if ((unsigned)(v >> 32) == (unsigned)t) {
                        w[j] = __uint_as_float((unsigned)v);
                        pending &= ~(1u << j);
                    }
                }
            }
            if (++spins > POLL_LIMIT) break;
        }
        if (__syncthreads_or(pending != 0)) {          // some producer never arrived: give up, all together
            if (tid == 0) atomicExch(a.status, 1u);
            return;
        }
        AMQ_PHASE(0);

        // ---- 2. on-line quantization of z (Algorithm 2), planes packed into shared memory ----
        float beta[KA];
        uint32_t bits[KA];
        quantize_group<KA, EPT, true>(w, valid, n, a.T, beta, bits, *scratch);
        AMQ_PHASE(1);
        pack_group<KA, EPT>(bits, lane, warp, NT / 32, wpr, reinterpret_cast<uint32_t*>(sZ));
        __syncthreads();
        AMQ_PHASE(2);

        // ---- 3. binary product: P[pr][j] = popcount(W plane-row pr XOR z plane j) ----
        for (int it = 0; it < pr_iters; ++it) {
            const int pr = it * NSEG + seg;
            int acc[PARTS][KA];
#pragma unroll
            for (int pt = 0; pt < PARTS; ++pt)
#pragma unroll
                for (int j = 0; j < KA; ++j) acc[pt][j] = 0;
            if (pr < PR) {
                for (int c = chunk; c < CH; c += SEG) {
                    const uint4 wv = sW[(size_t)pr * RS + c];
                    const bool in_x = c * 128 < a.I;          // GRU only; the host requires I % 128 == 0
#pragma unroll
                    for (int j = 0; j < KA; ++j) {
                        const int v = popc4(wv, sZ[j * CH + c]);
                        if (GRU) { acc[0][j] += in_x ? v : 0; acc[PARTS - 1][j] += in_x ? 0 : v; }
                        else acc[0][j] += v;
                    }
                }
            }
            for (int off = SEG >> 1; off > 0; off >>= 1) {
#pragma unroll
                for (int pt = 0; pt < PARTS; ++pt)
#pragma unroll
                    for (int j = 0; j < KA; ++j) acc[pt][j] += __shfl_xor_sync(0xffffffffu, acc[pt][j], off);
            }
            if (chunk == 0 && pr < PR) {
#pragma unroll
                for (int pt = 0; pt < PARTS; ++pt)
#pragma unroll
                    for (int j = 0; j < KA; ++j) sP[(pt * PR + pr) * KA + j] = acc[pt][j];
            }
        }
        __syncthreads();
        AMQ_PHASE(3);

        // ---- 4. coefficients, gates, state update; the leader of each unit publishes h ----
        if (warp < ep_warps) {
            float y[PARTS];
#pragma unroll
            for (int pt = 0; pt < PARTS; ++pt) y[pt] = 0.0f;
            if (ep_valid) {
                const int lr = ep_ul * GATES + ep_gate;
#pragma unroll
                for (int pt = 0; pt < PARTS; ++pt) {
                    const int len = GRU ? (pt == 0 ? a.I : a.H) : n;
                    for (int i = 0; i < k_w; ++i) {
                        const float al = sAlpha[lr * k_w + i];
#pragma unroll
                        for (int j = 0; j < KA; ++j)
                            y[pt] += al * beta[j] * (float)(len - 2 * sP[(pt * PR + lr * k_w + i) * KA + j]);
                    }
                }
            }
            const int quad = lane & ~3;
            float h_new;
            if (!GRU) {
                const float pre = y[0] + sBias[(ep_ul < upc ? ep_ul : 0) * 4 + ep_gate];
                const float act = (ep_gate == 3) ? fast_tanh(pre) : logistic(pre);
                const float ig = __shfl_sync(0xffffffffu, act, quad + 0);
                const float fg = __shfl_sync(0xffffffffu, act, quad + 1);
                const float og = __shfl_sync(0xffffffffu, act, quad + 2);
                const float gg = __shfl_sync(0xffffffffu, act, quad + 3);
                c_state = fg * c_state + ig * gg;
                h_new = og * fast_tanh(c_state);
            } else {
                const float* b4 = sBias + (ep_ul < upc ? ep_ul : 0) * 4;
                const float yx = y[0], yh = y[PARTS - 1];
                const float gate_rz = logistic(yx + yh + b4[ep_gate & 1]);        // meaningful for slots 0, 1
                const float rg = __shfl_sync(0xffffffffu, gate_rz, quad + 0);
                const float zg = __shfl_sync(0xffffffffu, gate_rz, quad + 1);
                const float cand_own = fast_tanh(yx + b4[2] + rg * (yh + b4[3]));  // meaningful for slot 2
                const float cand = __shfl_sync(0xffffffffu, cand_own, quad + 2);
                h_new = (1.0f - zg) * cand + zg * h_state;
            }
            if (ep_leader) {
                h_state = h_new;
                const int u = u0 + ep_ul;
                const unsigned long long word =
                    ((unsigned long long)(unsigned)(t + 1) << 32) | (unsigned long long)__float_as_uint(h_new);
                st_relaxed_u64(a.hx + (size_t)((t + 1) & 1) * a.H + u, word);
                if (a.h_seq) a.h_seq[(size_t)t * a.H + u] = h_new;
            }
        }
        AMQ_PHASE(4);
    }
#ifdef AMQ_PHASE_TIMING
    if (tid == 0 && (blockIdx.x == 0 || blockIdx.x == gridDim.x - 1)) {
        for (int i = 0; i < 5; ++i)
            a.status[8 + (blockIdx.x ? 8 : 0) + i] = (uint32_t)(ph[i] / (a.steps > 0 ? a.steps : 1));
    }
#endif

    if (ep_leader) {
        a.h_last[u0 + ep_ul] = h_state;
        if (!GRU) a.c_last[u0 + ep_ul] = c_state;
    }
}

size_t persistent_smem_bytes(int upc, int gates, int k_w, int k_a, int wpr)
{
    const size_t PR = (size_t)upc * gates * k_w, CH = wpr / 4;
    const size_t RS = product_row_stride((int)CH, product_segment((int)PR, (int)CH));
    size_t b = PR * RS * 16 + (size_t)k_a * CH * 16 + (gates == 3 ? 2 : 1) * PR * k_a * 4 + PR * 4 + (size_t)upc * 16;
    return b + 16 + sizeof(QuantScratch<AMQ_MAX_K>);       // alignment slack + quantizer scratch
}

int device_sm_count()
{
    static thread_local int cached_dev = -1, cached_sms = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (dev != cached_dev) {
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        cached_dev = dev; cached_sms = sms;
    }
    return cached_sms;
}

template <int KA, int EPT, bool GRU>
amq_status launch(const PersistArgs& a, int grid, size_t smem, cudaStream_t st)
{
    auto kernel = rnn_persistent_kernel<KA, EPT, GRU>;
    AMQ_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    PersistArgs args = a;
    void* params[] = {&args};
    if (a.steps <= 1) {
        // a single step never waits for another CTA (step 0 reads h0): a plain launch is enough and cheaper
        kernel<<<dim3((unsigned)grid), dim3(NT), smem, st>>>(args);
        AMQ_LAUNCH_CHECK();
        return AMQ_OK;
    }
    AMQ_CUDA_TRY(cudaLaunchCooperativeKernel((void*)kernel, dim3((unsigned)grid), dim3(NT), params, smem, st));
    __atomic_fetch_add(&g_kernel_launches, 1ull, __ATOMIC_RELAXED);
    return AMQ_OK;
}

template <int KA, bool GRU>
amq_status launch_ept(const PersistArgs& a, int n, int grid, size_t smem, cudaStream_t st)
{
    if (n <= NT * 4) return launch<KA, 4, GRU>(a, grid, smem, st);
    return launch<KA, 8, GRU>(a, grid, smem, st);
}

}  // namespace

bool persistent_supported(int I, int H, int batch, int k_w, int k_a, bool gru, int* grid_out, int* upc_out,
                          size_t* smem_out)
{
    const int n = I + H;
    if (batch != 1 || n > NT * 8) return false;
    if (gru && (I % 128) != 0) return false;
    const int sms = device_sm_count();
    if (sms <= 0) return false;
    const int wpr = words_per_row(n);
    if (wpr / 4 > 32) return false;
    const int upc = (H + sms - 1) / sms;
    if (upc * 4 > NT) return false;
    const int grid = (H + upc - 1) / upc;
    const size_t smem = persistent_smem_bytes(upc, gru ? 3 : 4, k_w, k_a, wpr);
    if (smem > 200 * 1024) return false;
    *grid_out = grid; *upc_out = upc; *smem_out = smem;
    return true;
}

amq_status launch_rnn_persistent(const uint32_t* Wcodes, const float* Walpha, const float* bias,
                                 int I, int H, int k_w, int k_a, int T, bool gru,
                                 const float* x_seq, int steps, const float* h0, const float* c0,
                                 float* h_seq, float* h_last, float* c_last,
                                 unsigned long long* hx, uint32_t* status, cudaStream_t st)
{
    int grid = 0, upc = 0;
    size_t smem = 0;
    if (!persistent_supported(I, H, 1, k_w, k_a, gru, &grid, &upc, &smem)) return AMQ_ERR_UNSUPPORTED;
    PersistArgs a{Wcodes, Walpha, bias, I, H, k_w, T, steps, x_seq, h0, c0, h_seq, h_last, c_last, hx, status,
                  upc, words_per_row(I + H)};
    const int n = I + H;
    if (gru) {
        switch (k_a) {
            case 1: return launch_ept<1, true>(a, n, grid, smem, st);
            case 2: return launch_ept<2, true>(a, n, grid, smem, st);
            case 3: return launch_ept<3, true>(a, n, grid, smem, st);
            case 4: return launch_ept<4, true>(a, n, grid, smem, st);
        }
    } else {
        switch (k_a) {
            case 1: return launch_ept<1, false>(a, n, grid, smem, st);
            case 2: return launch_ept<2, false>(a, n, grid, smem, st);
            case 3: return launch_ept<3, false>(a, n, grid, smem, st);
            case 4: return launch_ept<4, false>(a, n, grid, smem, st);
        }
    }
    return AMQ_ERR_UNSUPPORTED;
}

}  // namespace amq
