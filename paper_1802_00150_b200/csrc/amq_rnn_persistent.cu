// Persistent, weight-stationary kernel for a batch-1 quantized LSTM / GRU sequence (Eq. 6 repeated over
// time; timestep t + 1 consumes h_t, Sec. 1, so a sequence is one dependency chain).
//
// The hidden units are split over the CTAs of one co-resident (cooperative) grid; every CTA keeps the
// packed planes of its own gate rows in shared memory for the whole sequence.  A timestep is, in every
// CTA: gather z = [x_t ; h_{t-1}], quantize it on-line (Algorithm 2, all CTAs redundantly, so that one
// exchange per step is enough; one CTA barrier per reduction), pack the planes (one more barrier), then
// one warp per hidden unit XORs and bit-counts the planes against the unit's resident rows (Appendix A),
// folds the partials with the row-wise coefficients (Sec. 4), applies the gates and publishes the new h
// value, all inside the warp with shuffles; the other warps are already gathering for the next step.
//
// Exchange of h between CTAs: each value travels as one 64-bit word {fp32 bits, step tag}, written with
// a single relaxed gpu-scope store and polled with relaxed gpu-scope loads; a consumer accepts a word
// when its tag equals the step it is gathering for, so value and "ready" flag arrive together and no
// separate barrier, fence or atomic counter is on the critical path.  Every producer writes its word to
// several copies of the exchange buffer and a CTA polls the copy blockIdx.x % copies: all CTAs polling the
// same few cache lines queue up at the L2 slices that hold them, and the queueing, not the distance, was
// most of the exchange latency.  Two buffers alternate by step parity: a CTA can only run one step ahead
// of the slowest one (it needs every slice of the previous step), so a buffer is never overwritten while
// someone still reads it.  Every poll is bounded; when it runs out the CTA records AMQ_ERR_TIMEOUT in the
// workspace status word and leaves (the vote is folded into the first barrier of the quantizer).
#include "amq_common.cuh"
#include "amq_quantize_device.cuh"

namespace amq {

namespace {

constexpr unsigned POLL_LIMIT = 1u << 20;

struct PersistArgs {
    const uint32_t* Wcodes; const float* Walpha; const float* bias;
    int I, H, k_w, T, steps;
    const float* x_seq; const float* h0; const float* c0;
    float* h_seq; float* h_last; float* c_last;
    unsigned long long* hx;              // [2][copies][hx_stride] exchange words
    size_t hx_stride;                    // H rounded up to whole 128-byte lines
    int vec_ok;                          // I % EPT == 0, H even, x_seq 16-byte aligned: vector loads, no thread straddles x | h
    uint32_t* status;
    int upc;                             // hidden units per CTA
    int wpr;
    int copies;                          // copies of the exchange buffer (1..32)
    unsigned poll_limit;                 // iterations after which a gather gives up
    unsigned tag_bias;                   // added to the tag a gather expects (0; nonzero only in the self-test of the
                                         // give-up path, where no word can ever match)
};

__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long* p)
{
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

// two adjacent exchange words with one 16-byte load (each word is validated on its own by its tag)
__device__ __forceinline__ ulonglong2 ld_relaxed_v2_u64(const unsigned long long* p)
{
    ulonglong2 v;
    asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(v.x), "=l"(v.y) : "l"(p) : "memory");
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

// Lanes per plane-row in the product phase: a warp holds all plane-rows of one hidden unit (gates x k_w <= 16),
// each owned by a segment of SEG lanes (a power of two).
__host__ __device__ inline int product_segment(int rows_per_unit)
{
    return rows_per_unit <= 4 ? 8 : (rows_per_unit <= 8 ? 4 : 2);
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

template <int KA, int EPT, bool GRU, int NT>
__global__ void __launch_bounds__(NT, 1)
rnn_persistent_kernel(PersistArgs a)
{
    constexpr int NW = NT / 32;
    constexpr int GATES = GRU ? 3 : 4;
    constexpr int PARTS = GRU ? 2 : 1;    // GRU keeps the product in two column segments, [0,I) and [I,n)
    static_assert(EPT == 8 || EPT == 16, "a thread's sign bits are stored as one byte or one half-word");
    extern __shared__ __align__(16) unsigned char smem_raw[];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = a.I + a.H, wpr = a.wpr, CH = wpr >> 2, k_w = a.k_w;
    const int upc = a.upc, RPU = GATES * k_w, PR = upc * RPU;
    const int u0 = blockIdx.x * upc;

    // product role: lane = (plane-row within the unit) * SEG + chunk; lane c of a segment owns chunks c, c + SEG, ..
    const int SEG = product_segment(RPU), RS = product_row_stride(CH, SEG);
    const int my_row = lane / SEG, chunk = lane % SEG;
    const bool row_active = my_row < RPU;
    const int my_gate = row_active ? my_row / k_w : 0;

    // ---- shared memory carve-up ----
    uint4* sW = reinterpret_cast<uint4*>(smem_raw);                              // [PR][RS]
    uint4* sZ = sW + (size_t)PR * RS;                                            // [KA][CH]
    float* sAlpha = reinterpret_cast<float*>(sZ + KA * CH);                      // [PR]
    float* sBias = sAlpha + PR;                                                  // [upc][4]
    float* sH = sBias + upc * 4;                                                 // [upc] h of the unit
    float* sC = sH + upc;                                                        // [upc] c of the unit (LSTM)
    QuantScratch<KA, NW>* scratch = reinterpret_cast<QuantScratch<KA, NW>*>(
        (reinterpret_cast<uintptr_t>(sC + upc) + 15) & ~uintptr_t(15));

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
        for (int ul = tid; ul < upc; ul += NT) {
            const int u = u0 + ul;
            sH[ul] = (u < a.H) ? __ldg(a.h0 + u) : 0.0f;
            sC[ul] = (!GRU && u < a.H) ? __ldg(a.c0 + u) : 0.0f;
        }
        for (int q = tid; q < KA * wpr; q += NT) reinterpret_cast<uint32_t*>(sZ)[q] = 0u;   // plane words no thread owns
        quant_scratch_init(*scratch);
    }
    __syncthreads();

    // ---- element ownership: thread tid holds the EPT consecutive elements e0 .. e0 + EPT - 1 of z, so the sign bits
    // the quantizer leaves in a register ARE a byte (half-word) of the packed plane ----
    const int e0 = tid * EPT;
    uint32_t valid = 0, hmask = 0;
#pragma unroll
    for (int j = 0; j < EPT; ++j) {
        if (e0 + j < n) valid |= 1u << j;
        if (e0 + j >= a.I && e0 + j < n) hmask |= 1u << j;
    }
    const bool vec = a.vec_ok != 0;                    // no thread straddles x and h, 16-byte loads are aligned
    const int copies = a.copies;
    const size_t hs = a.hx_stride;
    const int my_copy = (int)(blockIdx.x % (unsigned)copies);
    int parity = 0;

#ifdef AMQ_PHASE_TIMING
    long long ph[4] = {0, 0, 0, 0};
    long long tp = clock64();
#endif

    for (int t = 0; t < a.steps; ++t) {
        // ---- 1. gather z = [x_t ; h_{t-1}] ----
        float w[EPT];
#pragma unroll
        for (int j = 0; j < EPT; ++j) w[j] = 0.0f;
        uint32_t pending = 0;
        const float* x = a.x_seq + (size_t)t * a.I;
        const unsigned long long* hx = a.hx + ((size_t)(t & 1) * copies + my_copy) * hs;
        const unsigned want = (unsigned)t + a.tag_bias;
        if (vec && e0 < a.I) {
#pragma unroll
            for (int q = 0; q < EPT / 4; ++q) {
                const float4 v = __ldg(reinterpret_cast<const float4*>(x + e0) + q);
                w[4 * q] = v.x; w[4 * q + 1] = v.y; w[4 * q + 2] = v.z; w[4 * q + 3] = v.w;
            }
        } else if (t == 0 || !vec) {
#pragma unroll
            for (int j = 0; j < EPT; ++j) {
                const int e = e0 + j;
                if (e < a.I) w[j] = __ldg(x + e);
                else if (e < n) { if (t == 0) w[j] = __ldg(a.h0 + (e - a.I)); else pending |= 1u << j; }
            }
        } else {
            pending = hmask;
        }
        unsigned spins = 0;
        if (vec) {
            // words come in aligned pairs (H is even and so is every thread's first index)
            while (pending) {
#pragma unroll
                for (int q = 0; q < EPT / 2; ++q) {
                    if ((pending >> (2 * q)) & 3u) {
                        const ulonglong2 v = ld_relaxed_v2_u64(hx + (e0 - a.I) + 2 * q);
                        if ((unsigned)(v.x >> 32) == want) { w[2 * q] = __uint_as_float((unsigned)v.x); pending &= ~(1u << (2 * q)); }
                        if ((unsigned)(v.y >> 32) == want) { w[2 * q + 1] = __uint_as_float((unsigned)v.y); pending &= ~(2u << (2 * q)); }
                    }
                }
                if (++spins > a.poll_limit) break;
            }
        } else {
            while (pending) {
#pragma unroll
                for (int j = 0; j < EPT; ++j) {
                    if ((pending >> j) & 1u) {
                        const unsigned long long v = ld_relaxed_u64(hx + (e0 + j - a.I));
                        if ((unsigned)(v >> 32) == want) {
                            w[j] = __uint_as_float((unsigned)v);
                            pending &= ~(1u << j);
                        }
                    }
                }
                if (++spins > a.poll_limit) break;
            }
        }
        int gave_up = pending != 0;                    // some producer never arrived
        AMQ_PHASE(0);

        // ---- 2. on-line quantization of z (Algorithm 2); its first barrier also takes the give-up vote ----
        float beta[KA];
        uint32_t bits[KA];
        quantize_group<KA, EPT, NW>(w, valid, n, quant_padding_consecutive(n, EPT), a.T, beta, bits, *scratch, &gave_up, &parity);
        if (gave_up) {                                 // uniform over the CTA: leave together
            if (tid == 0) atomicExch(a.status, 1u);
            return;
        }
        AMQ_PHASE(1);
        if (e0 < wpr * 32) {                           // this thread's bits lie inside the plane
#pragma unroll
            for (int i = 0; i < KA; ++i) {
                if (EPT == 8) reinterpret_cast<uint8_t*>(sZ)[(size_t)i * wpr * 4 + tid] = (uint8_t)bits[i];
                else reinterpret_cast<uint16_t*>(sZ)[(size_t)i * wpr * 2 + tid] = (uint16_t)bits[i];
            }
        }
        __syncthreads();
        AMQ_PHASE(2);

        // ---- 3. one warp per hidden unit: binary product, coefficients, gates, state update, publish ----
        float beta_sum = 0.0f;
#pragma unroll
        for (int j = 0; j < KA; ++j) beta_sum += beta[j];
        for (int ul = warp; ul < upc; ul += NW) {
            const int u = u0 + ul;
            if (u >= a.H) break;
            int acc[PARTS][KA];
#pragma unroll
            for (int pt = 0; pt < PARTS; ++pt)
#pragma unroll
                for (int j = 0; j < KA; ++j) acc[pt][j] = 0;
            const float al = row_active ? sAlpha[ul * RPU + my_row] : 0.0f;
            const float* b4 = sBias + ul * 4;
            const float bias_own = b4[my_gate];
            const float state_old = GRU ? sH[ul] : sC[ul];
            if (row_active) {
                const uint4* wrow = sW + (size_t)(ul * RPU + my_row) * RS;
#pragma unroll 4
                for (int c = chunk; c < CH; c += SEG) {
                    const uint4 wv = wrow[c];
                    const bool in_x = c * 128 < a.I;          // GRU only; the host requires I % 128 == 0
#pragma unroll
                    for (int j = 0; j < KA; ++j) {
                        const int v = popc4(wv, sZ[j * CH + c]);
                        if (GRU) { acc[0][j] += in_x ? v : 0; acc[PARTS - 1][j] += in_x ? 0 : v; }
                        else acc[0][j] += v;
                    }
                }
            }
            // this lane's share of its plane-row's dot products, weighted by the activation coefficients: the column
            // count enters once per row (lane 0 of the segment); then the segment's lanes are added up
            float yrow[PARTS];
#pragma unroll
            for (int pt = 0; pt < PARTS; ++pt) {
                const int len = GRU ? (pt == 0 ? a.I : a.H) : n;
                float s = (chunk == 0) ? (float)len * beta_sum : 0.0f;
#pragma unroll
                for (int j = 0; j < KA; ++j) s -= beta[j] * (float)(2 * acc[pt][j]);
                yrow[pt] = al * s;
            }
            for (int off = SEG >> 1; off > 0; off >>= 1) {
#pragma unroll
                for (int pt = 0; pt < PARTS; ++pt) yrow[pt] += __shfl_xor_sync(0xffffffffu, yrow[pt], off);
            }
            // the k_w planes of this lane's gate, added in plane order
            float y[PARTS];
#pragma unroll
            for (int pt = 0; pt < PARTS; ++pt) y[pt] = 0.0f;
            for (int i = 0; i < k_w; ++i) {
                const int src = (my_gate * k_w + i) * SEG;
#pragma unroll
                for (int pt = 0; pt < PARTS; ++pt) y[pt] += __shfl_sync(0xffffffffu, yrow[pt], src);
            }
            const int gate_stride = k_w * SEG;             // first lane of gate g: g * gate_stride
            float h_new, c_new = 0.0f;
            if (!GRU) {
                // logistic for i, f, o; tanh(v) = 2 logistic(2 v) - 1 for g: one exponential either way
                const float sc = (my_gate == 3) ? 2.0f : 1.0f;
                const float act = sc * logistic(sc * (y[0] + bias_own)) - (sc - 1.0f);
                const float ig = __shfl_sync(0xffffffffu, act, 0);
                const float fg = __shfl_sync(0xffffffffu, act, gate_stride);
                const float og = __shfl_sync(0xffffffffu, act, 2 * gate_stride);
                const float gg = __shfl_sync(0xffffffffu, act, 3 * gate_stride);
                c_new = fg * state_old + ig * gg;
                h_new = og * fast_tanh(c_new);
            } else {
                const float yx = y[0], yh = y[PARTS - 1];
                const float gate_rz = logistic(yx + yh + b4[my_gate & 1]);        // meaningful for gates 0, 1
                const float rg = __shfl_sync(0xffffffffu, gate_rz, 0);
                const float zg = __shfl_sync(0xffffffffu, gate_rz, gate_stride);
                const float cand_own = fast_tanh(yx + b4[2] + rg * (yh + b4[3]));  // meaningful for gate 2
                const float cand = __shfl_sync(0xffffffffu, cand_own, 2 * gate_stride);
                h_new = (1.0f - zg) * cand + zg * state_old;
            }
            // every lane holds the unit's new state; lane r < copies publishes copy r
            if (lane < copies) {
                const unsigned long long word =
                    ((unsigned long long)(unsigned)(t + 1) << 32) | (unsigned long long)__float_as_uint(h_new);
                st_relaxed_u64(a.hx + ((size_t)((t + 1) & 1) * copies + lane) * hs + u, word);
            }
            __syncwarp();                                  // all lanes have read the old state
            if (lane == 0) {
                sH[ul] = h_new;
                if (!GRU) sC[ul] = c_new;
                if (a.h_seq) a.h_seq[(size_t)t * a.H + u] = h_new;
            }
        }
        AMQ_PHASE(3);
    }
#ifdef AMQ_PHASE_TIMING
    if (tid == 0 && (blockIdx.x == 0 || blockIdx.x == gridDim.x - 1)) {
        for (int i = 0; i < 4; ++i)
            a.status[8 + (blockIdx.x ? 8 : 0) + i] = (uint32_t)(ph[i] / (a.steps > 0 ? a.steps : 1));
    }
#endif

    __syncthreads();
    for (int ul = tid; ul < upc; ul += NT) {
        const int u = u0 + ul;
        if (u < a.H) {
            a.h_last[u] = sH[ul];
            if (!GRU) a.c_last[u] = sC[ul];
        }
    }
}

template <int NW>
size_t persistent_smem_bytes(int upc, int gates, int k_w, int wpr)
{
    const size_t PR = (size_t)upc * gates * k_w, CH = wpr / 4;
    const size_t RS = product_row_stride((int)CH, product_segment(gates * k_w));
    const size_t b = PR * RS * 16 + (size_t)AMQ_MAX_K * CH * 16 + PR * 4 + (size_t)upc * 16 + (size_t)upc * 8;
    return b + 16 + sizeof(QuantScratch<AMQ_MAX_K, NW>);   // alignment slack + quantizer scratch
}

int device_sm_count()
{
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    return sms;
}

constexpr int NT_SMALL = 128;            // threads per CTA for vectors of up to 1024 elements (8 per thread)
constexpr int NT_LARGE = 256;            // up to 2048 (8 per thread) and 4096 (16 per thread)

template <int KA, int EPT, bool GRU, int NT>
amq_status launch(const PersistArgs& a, int grid, size_t smem, cudaStream_t st)
{
    auto kernel = rnn_persistent_kernel<KA, EPT, GRU, NT>;
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
    PersistArgs b = a;
    const int ept = n <= NT_LARGE * 8 ? 8 : 16;
    b.vec_ok = (a.I % ept) == 0 && (a.H % 2) == 0 && (reinterpret_cast<uintptr_t>(a.x_seq) & 15u) == 0;
    if (n <= NT_SMALL * 8) return launch<KA, 8, GRU, NT_SMALL>(b, grid, smem, st);
    if (n <= NT_LARGE * 8) return launch<KA, 8, GRU, NT_LARGE>(b, grid, smem, st);
    return launch<KA, 16, GRU, NT_LARGE>(b, grid, smem, st);
}

}  // namespace

bool persistent_supported(int I, int H, int batch, int k_w, int k_a, bool gru, int* grid_out, int* upc_out,
                          size_t* smem_out)
{
    const int n = I + H;
    if (batch != 1 || n > NT_LARGE * 16) return false;
    if (gru && (I % 128) != 0) return false;
    const int sms = device_sm_count();
    if (sms <= 0) return false;
    const int wpr = words_per_row(n);
    const int upc = (H + sms - 1) / sms;
    const int grid = (H + upc - 1) / upc;
    const size_t smem = persistent_smem_bytes<NT_LARGE / 32>(upc, gru ? 3 : 4, k_w, wpr);
    (void)k_a;
    if (smem > 200 * 1024) return false;
    *grid_out = grid; *upc_out = upc; *smem_out = smem;
    return true;
}

amq_status launch_rnn_persistent(const uint32_t* Wcodes, const float* Walpha, const float* bias,
                                 int I, int H, int k_w, int k_a, int T, bool gru,
                                 const float* x_seq, int steps, const float* h0, const float* c0,
                                 float* h_seq, float* h_last, float* c_last,
                                 unsigned long long* hx, uint32_t* status, cudaStream_t st,
                                 unsigned poll_limit, unsigned tag_bias)
{
    int grid = 0, upc = 0;
    size_t smem = 0;
    if (!persistent_supported(I, H, 1, k_w, k_a, gru, &grid, &upc, &smem)) return AMQ_ERR_UNSUPPORTED;
    PersistArgs a{Wcodes, Walpha, bias, I, H, k_w, T, steps, x_seq, h0, c0, h_seq, h_last, c_last, hx,
                  persistent_exchange_stride(H), 0, status,
                  upc, words_per_row(I + H), PERSISTENT_EXCHANGE_COPIES, poll_limit ? poll_limit : POLL_LIMIT, tag_bias};
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
