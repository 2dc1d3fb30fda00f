// Batched binary matrix product on the 5th-generation tensor cores (tcgen05.mma kind::i8 or kind::mxf4,
// accumulators in tensor memory), in the stacked form of Fig. 3, right: the k_w planes of the weight rows of a tile are
// the M rows of one integer matrix product, the k_a planes of the activation vectors its N columns, the
// packed bit positions its K dimension; the k_w x k_a partials of every (row, vector) pair are folded
// with the row-wise coefficients afterwards (Sec. 4), and for the cells the gate arithmetic of Eq. 6 /
// the GRU follows in the same kernel.
//
// The planes stay bit-packed in global memory.  A CTA expands the bits of its tile into signed bytes in
// shared memory: bit 1 -> -64, bit 0 -> +64 on both operands, so a byte product is 4096 * (+-1 * +-1) and a
// 32-bit accumulator holds 4096 * (dot of the +-1 vectors); pad positions (0 in both operands) add one
// each and are subtracted again.  Expanding costs one shift (issued as a multiplication, on the FMA pipe)
// and one three-input logic operation per four bytes: output register s of a 32-bit word keeps bits s,
// s + 8, s + 16, s + 24 in its four bytes, i.e. the K positions inside a word are permuted, identically for
// both operands, which a dot product does not see.  What bounds the main loop is the shared-memory port, which
// the expansion stores (128 operand bytes per row and stage) share with the operand reads of the MMAs
// (an M 128 x N 256 x K 32 instruction reads 12 KB), not the arithmetic.
//
// Where tensor memory has 16 columns left beside the accumulators, the operands are 4-bit instead (kind::mxf4, block
// scaled): bit 1 -> the E2M1 nibble 0xA (-1.0), bit 0 -> 0x2 (+1.0), one shift-and-mask per eight nibbles; the block
// scales (one E8M0 byte per 32 elements, read from tensor memory) are all 2^0, the accumulators fp32, exact for sums
// of +-1 up to 2^24 terms.  The same 128 bytes of a row then hold 256 bit positions: half the shared-memory traffic
// and half the MMA time per bit position.  Not possible where the accumulators fill all 512 columns (two M tiles at
// N = 256).
//
// Shared-memory operand layout: K-major with the 128-byte swizzle: a pipeline stage holds 128 bytes of K per
// operand row, rows are 128 bytes apart, groups of 8 rows 1024 bytes apart, and the 16-byte chunk j of row r
// sits at chunk position j xor (r mod 8).  One MMA instruction consumes K = 32 bytes = the two chunks of one
// packed word; its descriptor start address advances by 32 bytes per word inside the swizzled row.
//
// Roles: expander threads, one per operand row (plane-rows of the weight tile, then rows of the activation
// tile), turn packed words into operand bytes, stage by stage (128 bit positions of K per stage, three or
// four stages in flight); where the thread budget allows, two such groups take the stages in turn, so that
// the serial latency of one stage (wait, expand, proxy fence, arrive) is overlapped; one more warp issues
// the MMAs.  A "full" mbarrier per stage is signalled by every expander thread of the group (generic-proxy
// stores, proxy fence, arrive), an "empty" one by tcgen05.commit when the MMAs that read the stage have
// completed.  A CTA may own two M tiles that share one expanded activation tile, which halves the
// expansion work per MMA.  Every wait is bounded: when one runs out the CTA records the failure in a status
// word, skips its stores, frees its tensor memory and returns.
//
// Two kernels share these pieces: bgemm_tc_kernel (one tile, or pair of M tiles, per CTA; all warps run the
// epilogue after the last MMA) and bgemm_tc_persistent_kernel (one CTA per SM walks over tiles; accumulators
// double-buffered in tensor memory, dedicated epilogue warps, so that the epilogue of a tile overlaps the main
// loop of the next).  Both may be launched as programmatic dependents of the kernel that produces the
// activation planes: they set themselves up and fetch weight rows, then wait for it.
#include "amq_common.cuh"

namespace amq {

namespace {

constexpr int MAX_THREADS = 1024;           // expander threads (one or two per operand row) plus the warp that issues the MMAs
constexpr int TILE_M = 128;                 // stacked weight plane-rows per M tile (= TMEM lanes)
constexpr int STAGE_WORDS = 4;              // packed words of K per pipeline stage (128 bit positions)
constexpr int MAX_STAGES = 4;
constexpr unsigned WAIT_LIMIT = 1u << 20;   // attempts on an mbarrier before giving up

__device__ uint32_t g_tc_status;            // nonzero after a bounded wait ran out (sticky until read)
__device__ uint32_t g_tc_status_taken;      // what the last read found

struct TcParams {
    GemmArgs a;
    int gates;      // 1 plain, 4 LSTM, 3 GRU
    int units;      // plain: m; cells: H
    int UT;         // units per M tile
    int MT;         // M tiles per CTA (1 or 2)
    int TB;         // batch entries per tile (multiple of 16)
    int nseg;       // 1, or 2 for the GRU (columns [0,I) and [I,n))
    int wpr;
    int n_mma;      // TB * k_a: N of the MMA, multiple of 16, <= 256
    int tmem_cols;  // power of two >= MT * nseg * n_mma
    int nstages;    // pipeline depth
    int expanders;  // operand rows of a stage, MT * 128 + n_mma, rounded up to whole warps
    int groups;     // expander groups (1 or 2) that take the pipeline steps in turn, `expanders` threads each
    // persistent form only: a CTA walks over tiles blockIdx.x, blockIdx.x + gridDim.x, ..
    int ntiles;     // tiles of the problem = mgroups * (tiles along the batch)
    int mgroups;    // groups of MT M tiles
    int nbuf;       // accumulator buffers in tensor memory (2: the epilogue of a tile overlaps the MMAs of the next)
    int epi_warps;  // warps that only run epilogues (4 or 8)
    int yt_bytes;   // shared memory of the epilogue's staging array
    // run-time copies of compile-time constants: the shifts of the expansion as multipliers (so that they
    // issue on the FMA pipe) and its two byte masks (so that one LOP3 takes both from registers)
    uint32_t mul[8];
    uint32_t mask_sign, mask_half;
    // 4-bit operand form (kind::mxf4: bits expanded to E2M1 nibbles +-1, unit block scales, fp32 accumulators): a pipeline
    // stage then holds 256 bit positions per row in the same 128 bytes, i.e. half the shared-memory traffic and half the
    // MMA time per bit position.  Used when the 16 tensor-memory columns of the scale factors fit beside the accumulators.
    int fp4;
    int sf_col;     // first tensor-memory column of the scale factors (all bytes 0x7F = 2^0)
    int steps;      // pipeline steps per tile: chunks of 128 bit positions, or pairs of them
    int pad;        // bit positions per row that are zero in both operands (they add +1 each to every dot product)
    // persistent form, 4-bit operands: the weight operand of a pipeline step expanded into tensor memory (32 columns per
    // stage, thread = plane-row = lane) instead of shared memory: its stores and the MMA's reads of it leave the
    // load/store unit and the shared-memory port to the activation operand
    int a_tmem;
    int a_col;      // first tensor-memory column of the weight-operand stages
};

// Row stride (floats) of the epilogue's staging array y[plane-row][entry].  The plain product stores and reads it in
// 128-bit pieces (four entries at a time: the epilogue's shared-memory instructions queue behind the expansion's in the
// load/store unit, so their number counts), which wants a stride of 4 (mod 8) words for conflict-free quarter-warps; the cells
// read it entry by entry with unit-strided rows and keep the odd stride.
__host__ __device__ __forceinline__ int staging_stride(int TB, int epilogue) { return epilogue == EPI_Y ? TB + 4 : TB + 1; }

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done != 0;
}

// bounded wait of the single MMA-issuing thread; false when it ran out
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    for (unsigned i = 0; i < WAIT_LIMIT; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}

// the same for the many expander threads: between attempts the thread sleeps, so that waiters do not take
// issue slots from the warps that have work
__device__ __forceinline__ bool mbar_wait_relaxed(uint32_t bar, uint32_t parity)
{
    if (mbar_try_wait(bar, parity)) return true;
    for (unsigned i = 0; i < WAIT_LIMIT; ++i) {
        __nanosleep(40);
        if (mbar_try_wait(bar, parity)) return true;
    }
    return false;
}

// the same, giving up early once another role of the CTA has recorded a failure
__device__ __forceinline__ bool mbar_wait_relaxed(uint32_t bar, uint32_t parity, volatile int* failed)
{
    if (mbar_try_wait(bar, parity)) return true;
    for (unsigned i = 0; i < WAIT_LIMIT && !*failed; ++i) {
        __nanosleep(40);
        if (mbar_try_wait(bar, parity)) return true;
    }
    return false;
}

// barrier 1 joins the epilogue warps only (barrier 0 is the CTA-wide one)
__device__ __forceinline__ void epi_bar(int nthreads)
{
    asm volatile("bar.sync 1, %0;" :: "r"(nthreads) : "memory");
}

// the same with an OR over a per-thread flag, so that all of them take the same way out
__device__ __forceinline__ bool epi_bar_or(int nthreads, bool flag)
{
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %1, 0;\n\t"
        "bar.red.or.pred q, 1, %2, p;\n\t"
        "selp.b32 %0, 1, 0, q;\n\t}"
        : "=r"(out) : "r"((uint32_t)flag), "r"(nthreads) : "memory");
    return out != 0;
}

// K-major, 128-byte swizzle: start address (the tile base is 1024-byte aligned), leading byte offset unused (1),
// stride byte offset = 1024 bytes between groups of 8 rows, descriptor version 1, layout type 2
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr)
{
    return (uint64_t)((addr >> 4) & 0x3fffu) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}

__device__ __forceinline__ void mma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        :: "r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

// The four MMAs of one pipeline stage (K = 4 x 32 bytes of the same swizzled rows) into one accumulator, as one block:
// the two descriptors are rebuilt from their low words (the high words are the same constant for both operands; the
// start-address field advances by 32 bytes = 2 units per MMA and cannot carry out of its 14 bits below 256 KiB), so the
// single issuing thread spends a dozen instructions per stage instead of several per MMA: its pace, not the tensor
// pipe's, was what a stage cost.  `acc_first`: whether the first of the four accumulates (the other three always do).
__device__ __forceinline__ void mma_i8_stage(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc,
                                             uint32_t acc_first)
{
    asm volatile(
        "{\n\t"
        ".reg .pred p, q;\n\t"
        ".reg .b64 da, db;\n\t"
        ".reg .b32 al, bl;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "setp.eq.b32 q, %5, %5;\n\t"
        "mov.b64 da, {%1, %3};\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %4, p;\n\t"
        "add.u32 al, %1, 2;\n\t"
        "add.u32 bl, %2, 2;\n\t"
        "mov.b64 da, {al, %3};\n\t"
        "mov.b64 db, {bl, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %4, q;\n\t"
        "add.u32 al, %1, 4;\n\t"
        "add.u32 bl, %2, 4;\n\t"
        "mov.b64 da, {al, %3};\n\t"
        "mov.b64 db, {bl, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %4, q;\n\t"
        "add.u32 al, %1, 6;\n\t"
        "add.u32 bl, %2, 6;\n\t"
        "mov.b64 da, {al, %3};\n\t"
        "mov.b64 db, {bl, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %4, q;\n\t"
        "}"
        :: "r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(acc_first) : "memory");
}

__device__ __forceinline__ void mma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld8(uint32_t taddr, int (&v)[8])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
        : "r"(taddr) : "memory");
}

__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t x, uint32_t y, uint32_t z, uint32_t w)
{
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" :: "r"(addr), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}

// (x & a) ^ b in one three-input logic instruction
__device__ __forceinline__ uint32_t and_xor(uint32_t x, uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0x6A;" : "=r"(d) : "r"(x), "r"(a), "r"(b));
    return d;
}

// exact conversion of a small integer (|v| < 2^22) on the FMA pipe instead of the conversion unit
__device__ __forceinline__ float small_int_to_float(int v)
{
    return __int_as_float(v + 0x4B400000) - 12582912.0f;
}

// Loads of what the preceding kernel of the stream may have produced (activation planes, their coefficients, added
// pre-activations) are ordinary L2-cached loads (__ldcg), not read-only-path loads: with an overlapped launch this
// kernel is alive while those bytes are still being written, and a read-only load may be moved above the wait.

__device__ __forceinline__ uint4 load_row_chunk(const uint4* p, bool weight_row)
{
    return weight_row ? __ldg(p) : __ldcg(p);       // weights are constant; activation planes: see above
}

// Two consecutive chunks of a packed row (32 bytes, 32-byte aligned) in one 256-bit load.  A warp-wide load of 16 bytes from
// 32 different rows costs the load/store unit about as much as one of 32 bytes (measured: the shared-memory stores of the
// expansion, which queue behind the loads, ran at 34 bytes per clock per SM beside two 16-byte loads per row and step, at
// 53-67 beside one 32-byte load), so the 4-bit form, whose pipeline step consumes 32 bytes per row, loads them at once.
__device__ __forceinline__ void load_row_chunk_pair(const uint4* p, bool weight_row, uint4& lo, uint4& hi)
{
    if (weight_row)
        asm volatile("ld.global.nc.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                     : "=r"(lo.x), "=r"(lo.y), "=r"(lo.z), "=r"(lo.w), "=r"(hi.x), "=r"(hi.y), "=r"(hi.z), "=r"(hi.w) : "l"(p));
    else
        asm volatile("ld.global.cg.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                     : "=r"(lo.x), "=r"(lo.y), "=r"(lo.z), "=r"(lo.w), "=r"(hi.x), "=r"(hi.y), "=r"(hi.z), "=r"(hi.w) : "l"(p) : "memory");
}

// one 128-bit chunk of a packed row -> its 128 operand bytes (eight 16-byte pieces at the swizzled offsets `off`)
__device__ __forceinline__ void expand_chunk(uint32_t base, const uint32_t (&off)[8], const uint4& v, const uint32_t (&mul)[7],
                                             uint32_t m_sign, uint32_t m_half)
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        uint32_t y[8];
#pragma unroll
        for (int s = 0; s < 7; ++s) y[s] = and_xor(w[q] * mul[s], m_sign, m_half);     // w << (7 - s)
        y[7] = and_xor(w[q], m_sign, m_half);
        st_shared_v4(base + off[2 * q], y[0], y[1], y[2], y[3]);
        st_shared_v4(base + off[2 * q + 1], y[4], y[5], y[6], y[7]);
    }
}

// 4-bit form: one 128-bit chunk of a packed row -> its 128 nibbles (64 bytes: four 16-byte pieces at the swizzled offsets
// off[0..3]).  Bit 1 -> 0xA (-1.0 in E2M1), bit 0 -> 0x2 (+1.0).  Output word s of a packed word keeps its bits s, s + 4, ..,
// s + 28 in its eight nibbles: the K positions inside a word are permuted, identically for both operands.
__device__ __forceinline__ void expand_chunk_fp4(uint32_t base, const uint32_t* off, const uint4& v)
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const uint32_t y0 = ((w[q] << 3) & 0x88888888u) | 0x22222222u;
        const uint32_t y1 = ((w[q] << 2) & 0x88888888u) | 0x22222222u;
        const uint32_t y2 = ((w[q] << 1) & 0x88888888u) | 0x22222222u;
        const uint32_t y3 = (w[q] & 0x88888888u) | 0x22222222u;
        st_shared_v4(base + off[q], y0, y1, y2, y3);
    }
}

// The four MMAs of one pipeline stage in the 4-bit form (K = 4 x 64 nibbles = the same 4 x 32 bytes of the swizzled rows),
// block scales of 32 elements read from tensor memory (all ones), fp32 accumulators.
__device__ __forceinline__ void mma_mxf4_stage(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc,
                                               uint32_t acc_first, uint32_t sf_tmem)
{
    asm volatile(
        "{\n\t"
        ".reg .pred p, q;\n\t"
        ".reg .b64 da, db;\n\t"
        ".reg .b32 al, bl;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "setp.eq.b32 q, %5, %5;\n\t"
        "mov.b64 da, {%1, %3};\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.block32 [%0], da, db, %4, [%6], [%6], p;\n\t"
        "add.u32 al, %1, 2;\n\t"
        "add.u32 bl, %2, 2;\n\t"
        "mov.b64 da, {al, %3};\n\t"
        "mov.b64 db, {bl, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.block32 [%0], da, db, %4, [%6], [%6], q;\n\t"
        "add.u32 al, %1, 4;\n\t"
        "add.u32 bl, %2, 4;\n\t"
        "mov.b64 da, {al, %3};\n\t"
        "mov.b64 db, {bl, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.block32 [%0], da, db, %4, [%6], [%6], q;\n\t"
        "add.u32 al, %1, 6;\n\t"
        "add.u32 bl, %2, 6;\n\t"
        "mov.b64 da, {al, %3};\n\t"
        "mov.b64 db, {bl, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.block32 [%0], da, db, %4, [%6], [%6], q;\n\t"
        "}"
        :: "r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(acc_first), "r"(sf_tmem) : "memory");
}

// The same with the weight operand in tensor memory (lanes 0..127, 8 columns = 64 nibbles per MMA).
__device__ __forceinline__ void mma_mxf4_stage_ta(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc,
                                                  uint32_t acc_first, uint32_t sf_tmem)
{
    asm volatile(
        "{\n\t"
        ".reg .pred p, q;\n\t"
        ".reg .b64 db;\n\t"
        ".reg .b32 al, bl;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "setp.eq.b32 q, %5, %5;\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.block32 [%0], [%1], db, %4, [%6], [%6], p;\n\t"
        "add.u32 al, %1, 8;\n\t"
        "add.u32 bl, %2, 2;\n\t"
        "mov.b64 db, {bl, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.block32 [%0], [al], db, %4, [%6], [%6], q;\n\t"
        "add.u32 al, %1, 16;\n\t"
        "add.u32 bl, %2, 4;\n\t"
        "mov.b64 db, {bl, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.block32 [%0], [al], db, %4, [%6], [%6], q;\n\t"
        "add.u32 al, %1, 24;\n\t"
        "add.u32 bl, %2, 6;\n\t"
        "mov.b64 db, {bl, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.block32 [%0], [al], db, %4, [%6], [%6], q;\n\t"
        "}"
        :: "r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(acc_first), "r"(sf_tmem) : "memory");
}

// 4-bit form, weight operand in tensor memory: one 128-bit chunk of a packed row -> 16 columns of the thread's lane, in
// the word order of the shared-memory row (word 4 q + s keeps bits s, s + 4, .. of packed word q).  Warp-collective.
__device__ __forceinline__ void expand_chunk_fp4_tmem(uint32_t taddr, const uint4& v)
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint32_t y[16];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        y[4 * q + 0] = ((w[q] << 3) & 0x88888888u) | 0x22222222u;
        y[4 * q + 1] = ((w[q] << 2) & 0x88888888u) | 0x22222222u;
        y[4 * q + 2] = ((w[q] << 1) & 0x88888888u) | 0x22222222u;
        y[4 * q + 3] = (w[q] & 0x88888888u) | 0x22222222u;
    }
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        :: "r"(taddr), "r"(y[0]), "r"(y[1]), "r"(y[2]), "r"(y[3]), "r"(y[4]), "r"(y[5]), "r"(y[6]), "r"(y[7]),
           "r"(y[8]), "r"(y[9]), "r"(y[10]), "r"(y[11]), "r"(y[12]), "r"(y[13]), "r"(y[14]), "r"(y[15]) : "memory");
}

// Scale factors of the 4-bit form: 16 tensor-memory columns, every byte 0x7F (2^0 in E8M0), written by four warps (one per
// lane quarter); both operands' scale addresses point at this region, whose every byte is the same.
__device__ __forceinline__ void write_unit_scales(uint32_t tmem_base, int sf_col, int warp)
{
    const uint32_t t = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)sf_col;
    const uint32_t one = 0x7F7F7F7Fu;
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1};"
        :: "r"(t), "r"(one) : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}

// an accumulator as the epilogue reads it from tensor memory -> the exact integer dot product (pad positions included)
__device__ __forceinline__ float acc_to_float(int acc, bool fp4)
{
    return fp4 ? __int_as_float(acc) : small_int_to_float(acc >> 12);
}

__device__ __forceinline__ float logistic(float v) { return 1.0f / (1.0f + __expf(-v)); }

// x / d for x >= 0 and the small divisors that occur in the row bookkeeping (bits per weight 1..4; gates 1, 3, 4): inside the
// switch the divisor is a constant, so each case is a shift or one multiplication instead of the generic division sequence
// (every expander thread runs several of these before its first load; they were a visible part of a CTA's start-up time)
__device__ __forceinline__ int div_small(int x, int d)
{
    switch (d) {
        case 1: return x;
        case 2: return x >> 1;
        case 3: return x / 3;
        case 4: return x >> 2;
        default: return x / d;
    }
}

// Epilogue, first half: tensor memory -> registers -> partial products y[plane-row][batch entry] in shared memory
// (EPI_DOTS: the integer partials straight to global memory).  A thread is a plane-row (lane of tensor memory, lane
// quarter `quarter` = warp index mod 4); the work items (M tile, column segment, 8 batch entries = 8 * KA columns)
// are dealt out to `nslots` groups of four warps (group s takes entries 8 s, 8 (s + nslots), .. of every M tile
// and segment).  Reads of the accumulators are complete on return.
template <int KA>
__device__ __forceinline__ void epilogue_tmem_to_smem(const TcParams& p, uint32_t tmem_acc, int u0, int b0, int quarter, int lane,
                                                      int slot, int nslots, const float* sAlpha, const float* sBeta,
                                                      const float* sBcorr, float* Yt)
{
    const GemmArgs& a = p.a;
    const int k_w = a.k_w, n_mma = p.n_mma, ldy = staging_stride(p.TB, a.epilogue);
    const int TMp = p.UT * p.gates * k_w;
    const int pr = quarter * 32 + lane;
    const int groups = p.TB >> 3;
    const uint32_t tlane = tmem_acc + ((uint32_t)(quarter * 32) << 16);
    if (a.epilogue == EPI_DOTS) {
        const int pad = p.pad;
        const bool fp4 = p.fp4 != 0;
        const int l = div_small(pr, k_w), i = pr - l * k_w;
        const int lg = div_small(l, p.gates), gate = l - lg * p.gates;
        for (int mt = 0; mt < p.MT; ++mt)                           // (one column segment in this epilogue)
        for (int g = slot; g < groups; g += nslots) {
            const int u = u0 + mt * p.UT + lg;
            const bool row_ok = pr < TMp && u < p.units;
            const size_t row = (size_t)gate * p.units + u;
            int acc[KA][8];
#pragma unroll
            for (int c = 0; c < KA; ++c) tmem_ld8(tlane + (uint32_t)(mt * n_mma + g * KA * 8 + c * 8), acc[c]);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
            for (int col = 0; col < 8 * KA; ++col) {
                const int b = b0 + g * 8 + col / KA;
                if (row_ok && b < a.batch)
                    a.D[(((size_t)b * a.m + row) * k_w + i) * KA + col % KA] =
                        (fp4 ? (int)__int_as_float(acc[col / 8][col % 8]) : (acc[col / 8][col % 8] >> 12)) - pad;
            }
        }
        return;
    }
    // loops without divisions: the per-item overhead is spread over only 8 * KA accumulators per thread.  This half of the
    // epilogue is a chain of latencies, not of issue slots (about three instructions per accumulator); reading two items
    // from tensor memory before folding the first was measured and lost (registers: the kernel's 1024-thread bound leaves
    // 64, the second item spilled: C5 product 151 us against 120 us), and so was fetching the coefficients ahead of the
    // tensor-memory wait (122 us)
    const bool fp4 = p.fp4 != 0;
    for (int mt = 0; mt < p.MT; ++mt)
    for (int seg = 0; seg < p.nseg; ++seg)
    for (int g = slot; g < groups; g += nslots) {
        const int ms = mt * p.nseg + seg;
        int acc[KA][8];
#pragma unroll
        for (int c = 0; c < KA; ++c) tmem_ld8(tlane + (uint32_t)(ms * n_mma + g * KA * 8 + c * 8), acc[c]);
        // y = alpha_i * sum_j beta_j * D_j with D_j = accumulator / 4096 - pad; the pad correction is taken once per
        // batch entry (sBcorr = -pad * sum_j beta_j), in the last column segment
        const float alpha = sAlpha[mt * TILE_M + pr];
        const bool last = seg == p.nseg - 1;
        float* yrow = Yt + ((size_t)ms * TILE_M + pr) * ldy + g * 8;
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            // coefficients of four entries: 4 * KA consecutive floats, 16-byte aligned
            float4 b4[KA];
#pragma unroll
            for (int q = 0; q < KA; ++q) b4[q] = reinterpret_cast<const float4*>(sBeta + (g * 8 + half * 4) * KA)[q];
            const float4 c4 = *reinterpret_cast<const float4*>(sBcorr + g * 8 + half * 4);
            const float corr4[4] = {c4.x, c4.y, c4.z, c4.w};
            float y4[4];
#pragma unroll
            for (int e4 = 0; e4 < 4; ++e4) {
                float y = last ? corr4[e4] : 0.0f;
#pragma unroll
                for (int j = 0; j < KA; ++j) {
                    const int bi = e4 * KA + j;                     // index among the 4 * KA coefficients
                    const float4 t = b4[bi >> 2];
                    const float beta = (bi & 3) == 0 ? t.x : (bi & 3) == 1 ? t.y : (bi & 3) == 2 ? t.z : t.w;
                    const int col = (half * 4 + e4) * KA + j;
                    y += beta * acc_to_float(acc[col / 8][col % 8], fp4);
                }
                y4[e4] = alpha * y;
            }
            if (a.epilogue == EPI_Y) {
                *reinterpret_cast<float4*>(yrow + half * 4) = make_float4(y4[0], y4[1], y4[2], y4[3]);
            } else {
#pragma unroll
                for (int e4 = 0; e4 < 4; ++e4) yrow[half * 4 + e4] = y4[e4];
            }
        }
    }
}

// Epilogue, second half: sum the k_w planes of each weight row, bias, gates; `nthreads` threads numbered `tid`.
__device__ __forceinline__ void epilogue_smem_to_global(const TcParams& p, const float* Yt, int u0, int b0, int tid, int nthreads)
{
    // thread -> (row or unit, every `bstep`-th batch entry): one division per thread, none per output
    const GemmArgs& a = p.a;
    const int k_w = a.k_w, TB = p.TB, MT = p.MT, ldy = staging_stride(p.TB, a.epilogue);
    const int TM = p.UT * p.gates;
    const int per_tile = (a.epilogue == EPI_Y) ? TM : p.UT;         // rows (plain) or units (cells) of an M tile
    const int items = MT * per_tile;
    const int lanes_b = nthreads / items;                           // threads sharing one row / unit (0: fewer threads than items)
    const int bsub = lanes_b > 0 ? tid / items : 0;
    const int bstep = lanes_b > 0 ? lanes_b : 1;
    const int istep = lanes_b > 0 ? items : nthreads;
    if (lanes_b > 0 && bsub >= lanes_b) return;
    for (int item = lanes_b > 0 ? tid - bsub * items : tid; item < items; item += istep) {
        const int mt = item / per_tile, li = item - mt * per_tile;
        if (a.epilogue == EPI_Y) {
            const int row = u0 + item;
            if (row >= a.m) continue;
            const float bias = a.bias ? __ldg(a.bias + row) : 0.0f;
            const float* y0 = Yt + ((size_t)(mt * p.nseg) * TILE_M + li * k_w) * ldy;
            const int bend = (a.batch - b0 < TB) ? a.batch - b0 : TB;
            // four consecutive entries per item: one 128-bit load per plane, four stores (rows of y are entries)
            float* out = a.y + (size_t)b0 * a.ldy + row;
            for (int b4 = 4 * bsub; b4 < bend; b4 += 4 * bstep) {
                float4 s = *reinterpret_cast<const float4*>(y0 + b4);
                if (k_w > 1) { const float4 v = *reinterpret_cast<const float4*>(y0 + ldy + b4); s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w; }
                if (k_w > 2) { const float4 v = *reinterpret_cast<const float4*>(y0 + 2 * ldy + b4); s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w; }
                if (k_w > 3) { const float4 v = *reinterpret_cast<const float4*>(y0 + 3 * ldy + b4); s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w; }
                out[(size_t)b4 * a.ldy] = bias + s.x;
                if (b4 + 1 < bend) out[(size_t)(b4 + 1) * a.ldy] = bias + s.y;
                if (b4 + 2 < bend) out[(size_t)(b4 + 2) * a.ldy] = bias + s.z;
                if (b4 + 3 < bend) out[(size_t)(b4 + 3) * a.ldy] = bias + s.w;
            }
        } else if (a.epilogue == EPI_LSTM) {
            const int H = a.H, u = u0 + item;
            if (u >= H) continue;
            float bias4[4];
#pragma unroll
            for (int g = 0; g < 4; ++g) bias4[g] = a.bias ? __ldg(a.bias + g * H + u) : 0.0f;
            const float* y0 = Yt + ((size_t)(mt * p.nseg) * TILE_M + li * 4 * k_w) * ldy;
            for (int bb = bsub; bb < TB && b0 + bb < a.batch; bb += bstep) {
                float g4[4];
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    float s = bias4[g];
                    if (a.addend) s += __ldcg(a.addend + (size_t)(b0 + bb) * a.ld_addend + g * H + u);
                    for (int i = 0; i < k_w; ++i) s += y0[(g * k_w + i) * ldy + bb];
                    g4[g] = s;
                }
                const float ig = logistic(g4[0]), fg = logistic(g4[1]), og = logistic(g4[2]);
                const float gg = tanhf(g4[3]);
                const size_t o = (size_t)(b0 + bb) * H + u;
                const float c = fg * a.c_in[o] + ig * gg;
                a.c_out[o] = c;
                a.h_out[o] = og * tanhf(c);
            }
        } else {    // EPI_GRU
            const int H = a.H, u = u0 + item;
            if (u >= H) continue;
            const float br = a.bias ? __ldg(a.bias + u) : 0.0f, bz = a.bias ? __ldg(a.bias + H + u) : 0.0f;
            const float bnx = a.bias ? __ldg(a.bias + 2 * H + u) : 0.0f;
            const float bnh = a.bias ? __ldg(a.bias + 3 * H + u) : 0.0f;
            const float* yx = Yt + ((size_t)(mt * 2 + 0) * TILE_M + li * 3 * k_w) * ldy;
            const float* yh = Yt + ((size_t)(mt * 2 + 1) * TILE_M + li * 3 * k_w) * ldy;
            for (int bb = bsub; bb < TB && b0 + bb < a.batch; bb += bstep) {
                float px[3], ph[3];
#pragma unroll
                for (int g = 0; g < 3; ++g) {
                    float sx = 0.0f, sh = 0.0f;
                    for (int i = 0; i < k_w; ++i) { sx += yx[(g * k_w + i) * ldy + bb]; sh += yh[(g * k_w + i) * ldy + bb]; }
                    px[g] = sx; ph[g] = sh;
                }
                const float rg = logistic(px[0] + ph[0] + br);
                const float zg = logistic(px[1] + ph[1] + bz);
                const float cand = tanhf(px[2] + bnx + rg * (ph[2] + bnh));
                const size_t o = (size_t)(b0 + bb) * H + u;
                a.h_out[o] = (1.0f - zg) * cand + zg * a.h_in[o];
            }
        }
    }
}

template <int KA, bool FP4>
__global__ void __launch_bounds__(MAX_THREADS, 1)
bgemm_tc_kernel(TcParams p)
{
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    const GemmArgs& a = p.a;
    const int k_w = a.k_w;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int TM = p.UT * p.gates;                  // weight rows of an M tile
    const int TMp = TM * k_w;                       // plane-rows in use per M tile (<= 128)
    const int MT = p.MT, S = p.nstages, G = p.groups;
    const int EXP = p.expanders;                    // operand rows rounded up to whole warps
    const int mma_warp = (G * EXP) >> 5, nthreads = G * EXP + 32;
    const int n_mma = p.n_mma;
    const bool a_tmem = FP4 && p.a_tmem != 0;       // weight operand in tensor memory (one M tile): the stages hold the activation rows
    const int a_stage_bytes = a_tmem ? 0 : MT * TILE_M * 128;       // 128 bytes of K per row and stage
    const int stage_bytes = a_stage_bytes + n_mma * 128;
    const int u0 = blockIdx.x * p.UT * MT, b0 = blockIdx.y * p.TB;

    unsigned char* stage_base = smem_raw;
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem_raw + (size_t)S * stage_bytes);   // [S]
    uint64_t* empty_bar = full_bar + MAX_STAGES;                                            // [S]
    uint64_t* done_bar = empty_bar + MAX_STAGES;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(done_bar + 1);
    volatile int* failed = reinterpret_cast<volatile int*>(tmem_slot + 1);
    float* sAlpha = reinterpret_cast<float*>(tmem_slot + 6);        // [MT][128] coefficient of each weight plane-row (16-byte aligned)
    float* sBeta = sAlpha + 2 * TILE_M;                             // [TB][KA]  coefficients of the activation tile
    float* sBcorr = sBeta + 256;                                    // [TB]      -pad * their sum per batch entry

    const int CH = p.wpr >> 2;                                      // 128-bit chunks along K
    constexpr bool fp4 = FP4;                                       // 4-bit operand form (p.fp4)
    const int STEPS = p.steps;                                      // pipeline steps: chunks, or pairs of chunks (4-bit form)
    const int step_words = fp4 ? 2 * STAGE_WORDS : STAGE_WORDS;     // packed words of K per pipeline step
    const int split_word = (p.nseg == 2) ? (a.I >> 5) : p.wpr;      // first word of the second column segment
    // ---- expanders, before the CTA's set-up barrier: G groups of EXP threads take the steps in turn; inside a group thread r
    //      owns operand row r (A plane-rows first, then the B rows).  The row bookkeeping and the first loads come first, so
    //      that their latency runs beside the barrier initialisation and the tensor-memory allocation ----
    const bool expander = warp < mma_warp;
    const int grp = (tid >= EXP ? 1 : 0) + (tid >= 2 * EXP ? 1 : 0) + (tid >= 3 * EXP ? 1 : 0), r_all = tid - grp * EXP;   // G <= 4
    const uint4* src = nullptr;
    uint32_t dst0 = 0;                                              // shared address of the row in stage 0
    const float* coef_src = nullptr;                                // the row's coefficient, staged for the epilogue
    float* coef_dst = nullptr;
    const float* corr_src = nullptr;                                // first of the KA coefficients of a batch entry
    const bool weight_row = r_all < MT * TILE_M;
    const uint4 zero = make_uint4(0, 0, 0, 0);
    // A group's unit of work is a pair of 128-bit chunks of its rows (chunks 2 q and 2 q + 1; one past the end of the row is
    // zeros): one pipeline step in the 4-bit form, two consecutive ones otherwise.  Where the row is 32-byte aligned the
    // pair comes in one load.
    auto load_pair = [&](int q, uint4& lo, uint4& hi) {
        const int c0 = 2 * q;
        if (src && c0 + 1 < CH && (reinterpret_cast<uintptr_t>(src) & 31) == 0) {
            load_row_chunk_pair(src + c0, weight_row, lo, hi);
            return;
        }
        lo = (src && c0 < CH) ? load_row_chunk(src + c0, weight_row) : zero;
        hi = (src && c0 + 1 < CH) ? load_row_chunk(src + c0 + 1, weight_row) : zero;
    };
    uint4 cur = zero, cur2 = zero, nxt = zero, nxt2 = zero;
    if (expander) {
        if (weight_row) {
            // with the operand in tensor memory a warp can only write the lane quarter (warp mod 4): the four weight warps
            // of a group (consecutive warps) take the row blocks in that order
            const int mt = r_all >> 7, r = a_tmem ? ((warp & 3) << 5) | lane : r_all & (TILE_M - 1);
            size_t prow = 0;                                        // plane-row index in Wcodes / Walpha
            if (r < TMp) {
                const int l = div_small(r, k_w), i = r - l * k_w;
                const int lg = div_small(l, p.gates), gate = l - lg * p.gates;
                const int u = u0 + mt * p.UT + lg;
                if (u < p.units) {
                    prow = ((size_t)gate * p.units + u) * k_w + i;
                    src = reinterpret_cast<const uint4*>(a.Wcodes + prow * p.wpr);
                }
            }
            dst0 = smem_u32(stage_base) + r_all * 128;
            if (grp == 0) {
                coef_dst = sAlpha + mt * TILE_M + r;
                if (src && a.epilogue != EPI_DOTS) coef_src = a.Walpha + prow;
            }
        } else {
            const int r = r_all - MT * TILE_M;
            const int b = b0 + r / KA, j = r % KA;
            const bool valid = r < n_mma && b < a.batch;
            if (valid) src = reinterpret_cast<const uint4*>(a.xcodes + ((size_t)b * KA + j) * p.wpr);
            dst0 = smem_u32(stage_base) + a_stage_bytes + r * 128;
            if (grp == 0 && r < n_mma) {
                coef_dst = sBeta + r;
                if (valid && a.epilogue != EPI_DOTS) coef_src = a.xbeta + (size_t)b * KA + j;
                if (j == 0) corr_src = coef_src;
            }
        }
        // weight rows are fetched at once (no kernel of a chain writes them); everything the preceding kernel of the
        // stream may have written (the activation planes and their coefficients, the state) is read after the wait
        if (!weight_row) grid_dependency_wait();
        load_pair(grp, cur, cur2);                                  // own pairs: grp, grp + G, ..
        load_pair(grp + G, nxt, nxt2);
    }

    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(smem_u32(&full_bar[s]), (uint32_t)EXP);
            mbar_init(smem_u32(&empty_bar[s]), 1);
        }
        mbar_init(smem_u32(done_bar), 1);
        *failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == mma_warp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     :: "r"(smem_u32(tmem_slot)), "r"((uint32_t)p.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    if (fp4 && warp < 4) write_unit_scales(tmem_base, p.sf_col, warp);      // (expander warps; ordered before the MMAs by their arrivals)

    if (expander) {
        if (weight_row) grid_dependency_wait();
        const bool writes = r_all < MT * TILE_M + n_mma;            // threads past the last row only arrive
        uint32_t off[8];                                            // swizzled position of chunk j: j xor (row mod 8)
#pragma unroll
        for (int j = 0; j < 8; ++j) off[j] = (uint32_t)((j ^ (r_all & 7)) << 4);
        uint32_t mul[7];
#pragma unroll
        for (int s = 0; s < 7; ++s) mul[s] = p.mul[s];
        const uint32_t m_sign = p.mask_sign, m_half = p.mask_half;  // 0x80808080, 0x40404040
        // coefficients for the epilogue: the loads are issued now, after the first operand loads, and their values are
        // stored only after this thread's first pipeline step, so that no thread waits for them before it has work out
        float coef_val = 0.0f, corr_sum = 0.0f;
        const bool has_corr = coef_dst && r_all >= MT * TILE_M && (r_all - MT * TILE_M) % KA == 0;
        if (coef_dst && coef_src) coef_val = __ldcg(coef_src);
        if (has_corr && corr_src) {
#pragma unroll
            for (int jj = 0; jj < KA; ++jj) corr_sum += __ldcg(corr_src + jj);
        }
        bool coef_pending = coef_dst != nullptr;
        const int PAIRS = (CH + 1) >> 1;
        int buf = fp4 ? grp : 2 * grp;                              // stage buffer of the pair's first pipeline step
        uint32_t empty_parity = 1;                                  // parity that means "never used" on the first lap
        auto advance = [&](int d) {
            buf += d;
            while (buf >= S) { buf -= S; empty_parity ^= 1u; }
        };
        advance(0);
        bool go_on = true;
        // one pipeline step: the MMAs that read this buffer one lap ago must have completed; expand; hand over
        auto step = [&](const uint4& lo, const uint4& hi) {
            bool free_now = mbar_wait_relaxed(smem_u32(&empty_bar[buf]), empty_parity);
            // (the tensor-memory stores below are warp-collective: a weight warp gives up as a whole or not at all)
            if (a_tmem && weight_row) free_now = __all_sync(0xffffffffu, free_now);
            if (!free_now) { *failed = 1; go_on = false; return; }
            if (a_tmem && weight_row) {
                const uint32_t taddr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(p.a_col + buf * 32);
                expand_chunk_fp4_tmem(taddr, lo);
                expand_chunk_fp4_tmem(taddr + 16, hi);
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            } else {
                if (writes) {
                    if (fp4) {
                        expand_chunk_fp4(dst0 + (uint32_t)(buf * stage_bytes), off, lo);
                        expand_chunk_fp4(dst0 + (uint32_t)(buf * stage_bytes), off + 4, hi);
                    } else {
                        expand_chunk(dst0 + (uint32_t)(buf * stage_bytes), off, lo, mul, m_sign, m_half);
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");    // generic-proxy stores -> async proxy
            }
            asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(smem_u32(&full_bar[buf])) : "memory");
        };
        for (int q = grp; q < PAIRS && go_on; q += G) {
            const uint4 v = cur, v2 = cur2;
            cur = nxt; cur2 = nxt2;
            load_pair(q + 2 * G, nxt, nxt2);
            step(v, v2);
            if (!go_on) break;
            if (coef_pending) {
                *coef_dst = coef_val;
                if (has_corr) sBcorr[(r_all - MT * TILE_M) / KA] = -(float)p.pad * corr_sum;
                coef_pending = false;
            }
            if (fp4) {
                advance(G);
            } else {
                advance(1);
                if (2 * q + 1 < CH) step(v2, v2);
                advance(2 * G - 1);
            }
        }
        if (coef_pending) {                                         // (a group without a step of its own)
            *coef_dst = coef_val;
            if (has_corr) sBcorr[(r_all - MT * TILE_M) / KA] = -(float)p.pad * corr_sum;
        }
    } else if (lane == 0) {
        // ---- MMA issuer ----
        // instruction descriptor: int8 (s32 accumulators, signed 8-bit operands), or block-scaled E2M1 (operand format 1,
        // scale format E8M0); N >> 3 at bit 17, M >> 4 at bit 24, both operands K-major
        const uint32_t idesc = fp4 ? ((1u << 7) | (1u << 10) | ((uint32_t)(n_mma >> 3) << 17) | (1u << 23) | ((uint32_t)(TILE_M >> 4) << 24))
                                   : ((2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n_mma >> 3) << 17) | ((uint32_t)(TILE_M >> 4) << 24));
        const uint64_t desc_base = smem_desc(smem_u32(stage_base)); // descriptor of stage 0, tile 0, word 0
        const uint32_t sf_tmem = tmem_base + (uint32_t)p.sf_col;
        int buf = 0;
        uint32_t full_parity = 0;
        for (int c = 0; c < STEPS; ++c) {
            if (!mbar_wait(smem_u32(&full_bar[buf]), full_parity)) { *failed = 1; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            // descriptors of the stage: start addresses are below 256 KiB, so adding to the low word never carries
            const uint64_t adesc0 = desc_base + (uint64_t)((buf * stage_bytes) >> 4);
            const uint64_t bdesc0 = adesc0 + (uint64_t)(a_stage_bytes >> 4);
            const int word0 = c * step_words;
            if (fp4 || word0 >= split_word || word0 + step_words <= split_word) {
                // the whole stage lies in one column segment (always in the 4-bit form; else unless a GRU's input width is
                // not a multiple of 128)
                const int seg = word0 >= split_word ? 1 : 0;
                const uint32_t acc_first = (word0 != 0 && word0 != split_word) ? 1u : 0u;
                const uint32_t hi = (uint32_t)(desc_base >> 32);
                if (a_tmem) {
                    mma_mxf4_stage_ta(tmem_base + seg * n_mma, tmem_base + (uint32_t)(p.a_col + buf * 32), (uint32_t)bdesc0, hi, idesc,
                                      acc_first, sf_tmem);
                } else if (fp4) {
                    mma_mxf4_stage(tmem_base + seg * n_mma, (uint32_t)adesc0, (uint32_t)bdesc0, hi, idesc, acc_first, sf_tmem);
                    if (MT == 2)
                        mma_mxf4_stage(tmem_base + (p.nseg + seg) * n_mma, (uint32_t)adesc0 + (TILE_M * 128 >> 4), (uint32_t)bdesc0, hi,
                                       idesc, acc_first, sf_tmem);
                } else {
                    mma_i8_stage(tmem_base + seg * n_mma, (uint32_t)adesc0, (uint32_t)bdesc0, hi, idesc, acc_first);
                    if (MT == 2)
                        mma_i8_stage(tmem_base + (p.nseg + seg) * n_mma, (uint32_t)adesc0 + (TILE_M * 128 >> 4), (uint32_t)bdesc0, hi,
                                     idesc, acc_first);
                }
            } else {
#pragma unroll
                for (int qq = 0; qq < STAGE_WORDS; ++qq) {
                    const int word = word0 + qq;
                    const int seg = word >= split_word ? 1 : 0;
                    const uint32_t accumulate = (word != 0 && word != split_word) ? 1u : 0u;
                    mma_i8(tmem_base + seg * n_mma, adesc0 + 2 * qq, bdesc0 + 2 * qq, idesc, accumulate);
                    if (MT == 2)
                        mma_i8(tmem_base + (p.nseg + seg) * n_mma, adesc0 + (TILE_M * 128 >> 4) + 2 * qq, bdesc0 + 2 * qq, idesc, accumulate);
                }
            }
            mma_commit(smem_u32(&empty_bar[buf]));
            if (++buf == S) { buf = 0; full_parity ^= 1u; }
        }
        if (!*failed) mma_commit(smem_u32(done_bar));               // covers every MMA issued above
    }
    __syncwarp();

    // all MMAs done?
    bool ok = !*failed;
    if (ok) ok = mbar_wait_relaxed(smem_u32(done_bar), 0);
    if (__syncthreads_or(!ok)) {
        // give the tensor core time to drain what was issued, then release tensor memory and leave
        if (tid == 0) atomicExch(&g_tc_status, 1u);
        __nanosleep(1000000);
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        if (warp == mma_warp)
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_base), "r"((uint32_t)p.tmem_cols) : "memory");
        return;
    }
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");

    // ---- epilogue: tensor memory -> partial products in shared memory (reusing the stage buffers) -> results ----
    float* Yt = reinterpret_cast<float*>(smem_raw);                 // [MT][nseg][128][staging_stride]
    const int epi_slots = mma_warp >> 2;                            // whole groups of four warps among the expanders
    if (warp < 4 * epi_slots)
        epilogue_tmem_to_smem<KA>(p, tmem_base, u0, b0, warp & 3, lane, warp >> 2, epi_slots, sAlpha, sBeta, sBcorr, Yt);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == mma_warp)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_base), "r"((uint32_t)p.tmem_cols) : "memory");
    if (a.epilogue == EPI_DOTS) return;

    epilogue_smem_to_global(p, Yt, u0, b0, tid, nthreads);
}

// The persistent form of the kernel, for problems of more tiles than the GPU has SMs: one CTA per SM walks over
// tiles t = blockIdx.x, blockIdx.x + gridDim.x, ..  The accumulators are double-buffered in tensor memory and
// dedicated warps run the epilogue, so that the epilogue of a tile (arithmetic and global stores) overlaps the
// expansion and the MMAs of the next one (bound by shared-memory traffic).  The stage pipeline runs on across
// tiles; "accumulator full" barriers are signalled by tcgen05.commit after the last MMA of a tile,
// "accumulator empty" ones by the epilogue warps after their last read of tensor memory.
template <int KA, bool FP4>
__global__ void __launch_bounds__(MAX_THREADS, 1)
bgemm_tc_persistent_kernel(TcParams p)
{
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    const GemmArgs& a = p.a;
    const int k_w = a.k_w;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int TMp = p.UT * p.gates * k_w;           // plane-rows in use per M tile (<= 128)
    const int MT = p.MT, S = p.nstages, G = p.groups, EXP = p.expanders;
    const int mma_warp = (G * EXP) >> 5, epi_warp0 = mma_warp + 1, EW = p.epi_warps;
    const int n_mma = p.n_mma;
    const bool a_tmem = FP4 && p.a_tmem != 0;       // weight operand in tensor memory: the stages hold the activation rows only
    const int a_stage_bytes = a_tmem ? 0 : MT * TILE_M * 128;
    const int stage_bytes = a_stage_bytes + n_mma * 128;
    const int acc_cols = MT * p.nseg * n_mma;       // columns of one accumulator buffer
    const int CH = p.wpr >> 2;                      // 128-bit chunks along K
    constexpr bool fp4 = FP4;                       // 4-bit operand form (p.fp4)
    const int STEPS = p.steps;                      // pipeline steps per tile: chunks, or pairs of chunks (4-bit form)
    const int step_words = fp4 ? 2 * STAGE_WORDS : STAGE_WORDS;
    const int split_word = (p.nseg == 2) ? (a.I >> 5) : p.wpr;
    const int ntiles = p.ntiles, MG = p.mgroups, tile_step = (int)gridDim.x;

    unsigned char* stage_base = smem_raw;
    float* Yt = reinterpret_cast<float*>(smem_raw + (size_t)S * stage_bytes);               // [MT][nseg][128][staging_stride]
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem_raw + (size_t)S * stage_bytes + p.yt_bytes);   // [S]
    uint64_t* empty_bar = full_bar + MAX_STAGES;                                            // [S]
    uint64_t* tfull_bar = empty_bar + MAX_STAGES;                                           // [2] accumulator buffer complete
    uint64_t* tempty_bar = tfull_bar + 2;                                                   // [2] accumulator buffer read out
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty_bar + 2);
    volatile int* failed = reinterpret_cast<volatile int*>(tmem_slot + 1);
    float* sAlpha = reinterpret_cast<float*>(tmem_slot + 4);        // [MT][128]
    float* sBeta = sAlpha + 2 * TILE_M;                             // [TB][KA]
    float* sBcorr = sBeta + 256;                                    // [TB]

    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(smem_u32(&full_bar[s]), (uint32_t)EXP);
            mbar_init(smem_u32(&empty_bar[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&tfull_bar[b]), 1);
            mbar_init(smem_u32(&tempty_bar[b]), (uint32_t)EW);      // one arrival per epilogue warp
        }
        *failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == mma_warp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     :: "r"(smem_u32(tmem_slot)), "r"((uint32_t)p.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    if (fp4 && warp < 4) write_unit_scales(tmem_base, p.sf_col, warp);      // (expander warps; ordered before the MMAs by their arrivals)

    if (warp < mma_warp) {
        // ---- expanders: thread r of a group owns operand row r of every tile; the groups take the steps of the
        //      CTA's whole sequence (tiles x steps per tile) in turn ----
        const int grp = (tid >= EXP ? 1 : 0) + (tid >= 2 * EXP ? 1 : 0) + (tid >= 3 * EXP ? 1 : 0), r_all = tid - grp * EXP;   // G <= 4
        const bool is_a = r_all < MT * TILE_M;
        int unit_off = 0, gate = 0, plane = 0, entry = 0;
        bool valid;
        uint32_t dst0;
        if (is_a) {
            const int mt = r_all >> 7, r = r_all & (TILE_M - 1);
            const int l = div_small(r, k_w), lg = div_small(l, p.gates);
            valid = r < TMp;
            plane = r - l * k_w; unit_off = mt * p.UT + lg; gate = l - lg * p.gates;
            dst0 = smem_u32(stage_base) + r_all * 128;
        } else {
            const int r = r_all - MT * TILE_M;
            valid = r < n_mma;
            entry = r / KA; plane = r % KA;
            dst0 = smem_u32(stage_base) + a_stage_bytes + r * 128;
        }
        const bool writes = r_all < MT * TILE_M + n_mma;            // threads past the last row only arrive
        // packed row of this thread in tile `tile` (null: beyond the matrix, the batch or the CTA's last tile)
        auto row_of = [&](int tile) -> const uint4* {
            if (!valid || tile >= ntiles) return nullptr;
            const int bt = tile / MG, mg = tile - bt * MG;
            if (is_a) {
                const int u = mg * p.UT * MT + unit_off;
                return u < p.units ? reinterpret_cast<const uint4*>(a.Wcodes + (((size_t)gate * p.units + u) * k_w + plane) * p.wpr)
                                   : nullptr;
            }
            const int b = bt * p.TB + entry;
            return b < a.batch ? reinterpret_cast<const uint4*>(a.xcodes + ((size_t)b * KA + plane) * p.wpr) : nullptr;
        };
        uint32_t off[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) off[j] = (uint32_t)((j ^ (r_all & 7)) << 4);
        uint32_t mul[7];
#pragma unroll
        for (int s = 0; s < 7; ++s) mul[s] = p.mul[s];
        const uint32_t m_sign = p.mask_sign, m_half = p.mask_half;
        const uint4 zero = make_uint4(0, 0, 0, 0);

        // load cursor: runs two of the group's steps ahead of the expansion, across tile boundaries
        int pf_tile = (int)blockIdx.x, pf_c = grp;
        const uint4* pf_src = row_of(pf_tile);
        // chunk(s) of the cursor's step: one, or a pair in the 4-bit form (a chunk past the end of the row is zeros)
        auto pf_load = [&](uint4& lo, uint4& hi) {
            while (pf_c >= STEPS) { pf_c -= STEPS; pf_tile += tile_step; pf_src = row_of(pf_tile); }
            const int c0 = fp4 ? 2 * pf_c : pf_c;
            if (fp4 && pf_src && c0 + 1 < CH && (reinterpret_cast<uintptr_t>(pf_src) & 31) == 0) {
                load_row_chunk_pair(pf_src + c0, is_a, lo, hi);
            } else {
                lo = pf_src ? load_row_chunk(pf_src + c0, is_a) : zero;
                hi = (fp4 && pf_src && c0 + 1 < CH) ? load_row_chunk(pf_src + c0 + 1, is_a) : zero;
            }
            pf_c += G;
        };
        const int my_tiles = (ntiles - (int)blockIdx.x + tile_step - 1) / tile_step;
        const int total = my_tiles * STEPS;
        if (!is_a) grid_dependency_wait();                          // activation planes come from the preceding kernel
        uint4 cur, cur2, nxt, nxt2;
        pf_load(cur, cur2);
        pf_load(nxt, nxt2);
        if (is_a) grid_dependency_wait();
        int buf = grp;                                              // G <= S
        uint32_t empty_parity = 1;
        for (int q = grp; q < total; q += G) {
            const uint4 v = cur, v2 = cur2;
            cur = nxt; cur2 = nxt2;
            pf_load(nxt, nxt2);
            bool free_now = mbar_wait_relaxed(smem_u32(&empty_bar[buf]), empty_parity, failed);
            // (the tensor-memory stores below are warp-collective: a weight warp gives up as a whole or not at all)
            if (a_tmem && is_a) free_now = __all_sync(0xffffffffu, free_now);
            if (!free_now) { *failed = 1; break; }
            if (a_tmem && is_a) {
                // whole warps of weight rows: lane = plane-row mod 32, lane quarter = warp (the tile's 128 rows are warps 0..3)
                const uint32_t taddr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(p.a_col + buf * 32);
                expand_chunk_fp4_tmem(taddr, v);
                expand_chunk_fp4_tmem(taddr + 16, v2);
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            } else {
                if (writes) {
                    if (fp4) {
                        expand_chunk_fp4(dst0 + (uint32_t)(buf * stage_bytes), off, v);
                        expand_chunk_fp4(dst0 + (uint32_t)(buf * stage_bytes), off + 4, v2);
                    } else {
                        expand_chunk(dst0 + (uint32_t)(buf * stage_bytes), off, v, mul, m_sign, m_half);
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            }
            asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(smem_u32(&full_bar[buf])) : "memory");
            buf += G;
            if (buf >= S) { buf -= S; empty_parity ^= 1u; }
        }
    } else if (warp == mma_warp) {
        if (lane == 0) {
            // ---- MMA issuer ----
            const uint32_t idesc = fp4 ? ((1u << 7) | (1u << 10) | ((uint32_t)(n_mma >> 3) << 17) | (1u << 23) | ((uint32_t)(TILE_M >> 4) << 24))
                                       : ((2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n_mma >> 3) << 17) | ((uint32_t)(TILE_M >> 4) << 24));
            const uint64_t desc_base = smem_desc(smem_u32(stage_base));
            const uint32_t sf_tmem = tmem_base + (uint32_t)p.sf_col;
            int buf = 0;
            uint32_t full_parity = 0;
            bool ok = true;
            int it = 0;
            for (int tile = (int)blockIdx.x; tile < ntiles && ok; tile += tile_step, ++it) {
                const int ab = (p.nbuf == 2) ? (it & 1) : 0;
                const uint32_t use = (p.nbuf == 2) ? (uint32_t)(it >> 1) : (uint32_t)it;    // earlier uses of this buffer
                // the epilogue of the tile that used this buffer last must have read it out
                if (!mbar_wait(smem_u32(&tempty_bar[ab]), (use & 1u) ^ 1u)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t acc = tmem_base + (uint32_t)(ab * acc_cols);
                for (int c = 0; c < STEPS; ++c) {
                    if (!mbar_wait(smem_u32(&full_bar[buf]), full_parity)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint64_t adesc0 = desc_base + (uint64_t)((buf * stage_bytes) >> 4);
                    const uint64_t bdesc0 = adesc0 + (uint64_t)(a_stage_bytes >> 4);
                    const int word0 = c * step_words;
                    if (fp4 || word0 >= split_word || word0 + step_words <= split_word) {
                        const int seg = word0 >= split_word ? 1 : 0;
                        const uint32_t acc_first = (word0 != 0 && word0 != split_word) ? 1u : 0u;
                        const uint32_t hi = (uint32_t)(desc_base >> 32);
                        if (a_tmem) {
                            mma_mxf4_stage_ta(acc + seg * n_mma, tmem_base + (uint32_t)(p.a_col + buf * 32), (uint32_t)bdesc0, hi, idesc,
                                              acc_first, sf_tmem);
                        } else if (fp4) {
                            mma_mxf4_stage(acc + seg * n_mma, (uint32_t)adesc0, (uint32_t)bdesc0, hi, idesc, acc_first, sf_tmem);
                            if (MT == 2)
                                mma_mxf4_stage(acc + (p.nseg + seg) * n_mma, (uint32_t)adesc0 + (TILE_M * 128 >> 4), (uint32_t)bdesc0, hi,
                                               idesc, acc_first, sf_tmem);
                        } else {
                            mma_i8_stage(acc + seg * n_mma, (uint32_t)adesc0, (uint32_t)bdesc0, hi, idesc, acc_first);
                            if (MT == 2)
                                mma_i8_stage(acc + (p.nseg + seg) * n_mma, (uint32_t)adesc0 + (TILE_M * 128 >> 4), (uint32_t)bdesc0, hi, idesc,
                                             acc_first);
                        }
                    } else {
#pragma unroll
                        for (int qq = 0; qq < STAGE_WORDS; ++qq) {
                            const int word = word0 + qq;
                            const int seg = word >= split_word ? 1 : 0;
                            const uint32_t accumulate = (word != 0 && word != split_word) ? 1u : 0u;
                            mma_i8(acc + seg * n_mma, adesc0 + 2 * qq, bdesc0 + 2 * qq, idesc, accumulate);
                            if (MT == 2)
                                mma_i8(acc + (p.nseg + seg) * n_mma, adesc0 + (TILE_M * 128 >> 4) + 2 * qq, bdesc0 + 2 * qq, idesc, accumulate);
                        }
                    }
                    mma_commit(smem_u32(&empty_bar[buf]));
                    if (++buf == S) { buf = 0; full_parity ^= 1u; }
                }
                if (ok) mma_commit(smem_u32(&tfull_bar[ab]));       // covers every MMA of the tile
            }
            if (!ok) *failed = 1;
        }
    } else {
        // ---- epilogue warps ----
        const int tid_e = tid - epi_warp0 * 32, nth_e = EW * 32;
        const int quarter = warp & 3, slot = (warp - epi_warp0) >> 2, nslots = EW >> 2;
        grid_dependency_wait();                                     // coefficients and state come from preceding kernels
        // Coefficients of a tile, staged in shared memory for the first half of the epilogue: alpha per plane-row, beta
        // per (entry, plane), -pad * sum_j beta_j per entry.  The global loads for the next tile are issued before the
        // second half of the epilogue of this one and their values stored after it, so that their latency is off the
        // tile-to-tile chain of the epilogue warps (at most one plane-row and two activation columns per thread:
        // one M tile per CTA, N <= 256, at least 128 epilogue threads).
        float c_alpha = 0.0f, c_beta[2] = {0.0f, 0.0f}, c_corr[2] = {0.0f, 0.0f};
        auto coef_load = [&](int tile) {
            const int bt = tile / MG, mg = tile - bt * MG;
            const int u0 = mg * p.UT * MT, b0 = bt * p.TB;
            c_alpha = 0.0f;
            if (tid_e < MT * TILE_M) {
                const int mt = tid_e >> 7, r = tid_e & (TILE_M - 1);
                const int l = div_small(r, k_w), i = r - l * k_w;
                const int lg = div_small(l, p.gates);
                const int u = u0 + mt * p.UT + lg, gate = l - lg * p.gates;
                if (r < TMp && u < p.units) c_alpha = __ldg(a.Walpha + ((size_t)gate * p.units + u) * k_w + i);
            }
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const int idx = tid_e + k * nth_e;
                c_beta[k] = 0.0f; c_corr[k] = 0.0f;
                if (idx < n_mma) {
                    const int e = idx / KA, j = idx - e * KA, b = b0 + e;
                    if (b < a.batch) {
                        c_beta[k] = __ldcg(a.xbeta + (size_t)b * KA + j);
                        if (j == 0) {
                            float sum = 0.0f;
                            for (int jj = 0; jj < KA; ++jj) sum += __ldcg(a.xbeta + (size_t)b * KA + jj);
                            c_corr[k] = -(float)p.pad * sum;
                        }
                    }
                }
            }
        };
        auto coef_store = [&]() {
            if (tid_e < MT * TILE_M) sAlpha[tid_e] = c_alpha;
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const int idx = tid_e + k * nth_e;
                if (idx < n_mma) {
                    sBeta[idx] = c_beta[k];
                    if (idx % KA == 0) sBcorr[idx / KA] = c_corr[k];
                }
            }
        };
        if (a.epilogue != EPI_DOTS && (int)blockIdx.x < ntiles) { coef_load((int)blockIdx.x); coef_store(); }
        int it = 0;
        for (int tile = (int)blockIdx.x; tile < ntiles; tile += tile_step, ++it) {
            const int ab = (p.nbuf == 2) ? (it & 1) : 0;
            const uint32_t use = (p.nbuf == 2) ? (uint32_t)(it >> 1) : (uint32_t)it;
            const int bt = tile / MG, mg = tile - bt * MG;
            const int u0 = mg * p.UT * MT, b0 = bt * p.TB;
            const bool ok = mbar_wait_relaxed(smem_u32(&tfull_bar[ab]), use & 1u, failed);
            __syncwarp();
            // one barrier: the coefficients are visible, every thread has left the previous tile's second half
            // (the staging array is free), and all threads agree on whether to go on
            if (epi_bar_or(nth_e, !ok || *failed)) { if (!ok) *failed = 1; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            epilogue_tmem_to_smem<KA>(p, tmem_base + (uint32_t)(ab * acc_cols), u0, b0, quarter, lane, slot, nslots,
                                      sAlpha, sBeta, sBcorr, Yt);
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0)
                asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(smem_u32(&tempty_bar[ab])) : "memory");
            if (a.epilogue == EPI_DOTS) continue;
            __syncwarp();
            epi_bar(nth_e);                                         // the staging array is complete, the coefficients are read
            const bool more = tile + tile_step < ntiles;
            if (more) coef_load(tile + tile_step);
            epilogue_smem_to_global(p, Yt, u0, b0, tid_e, nth_e);
            if (more) coef_store();                                 // (visible to the others after the next tile's barrier)
            __syncwarp();
        }
    }
    __syncwarp();
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    const bool bad = __syncthreads_or(*failed != 0);
    if (bad) {
        // give the tensor core time to drain what was issued before tensor memory is released
        if (tid == 0) atomicExch(&g_tc_status, 1u);
        __nanosleep(1000000);
        __syncthreads();
    }
    if (warp == mma_warp)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_base), "r"((uint32_t)p.tmem_cols) : "memory");
}

struct TcPlan {
    TcParams p;
    dim3 grid;
    size_t smem;
    int threads;
    bool persistent;
};

// SMs of the current device (asked every time: an attribute query costs well under a microsecond and the answer
// belongs to the device that is current now, not to the one that was current at the first call)
int sm_count()
{
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0)
        return v;
    return 1;
}

// The persistent form: one M tile per CTA step, dedicated epilogue warps, two accumulator buffers when they fit tensor
// memory.  Possible when there are more tiles than SMs (otherwise nothing could overlap).
bool plan_persistent(const TcParams& base, int mtiles, int btiles, TcPlan* out)
{
    TcParams p = base;
    p.MT = 1;
    p.mgroups = mtiles;
    const int sms = sm_count();
    if (mtiles > 0x7fffffff / btiles) return false;
    p.ntiles = mtiles * btiles;
    if (p.ntiles <= sms) return false;
    const int acc_cols = p.nseg * p.n_mma;
    if (acc_cols > 512) return false;
    // two accumulator buffers when they fit (the epilogue of a tile then overlaps the MMAs of the next); with one (the
    // GRU's two column segments at N = 192) the MMAs of the next tile wait for the epilogue, but its stages are expanded
    // meanwhile and the CTA pays its set-up once: still ahead of three waves of the plain form (measured)
    p.nbuf = (2 * acc_cols > 512) ? 1 : 2;
    // 4-bit operands where the scale factors' 16 tensor-memory columns fit beside the accumulator buffers and a GRU's
    // column split falls on a pipeline step (256 bit positions)
    const int CH = p.wpr >> 2;
    const bool split_ok = p.nseg == 1 || p.a.I % 256 == 0;
    // (the 4-bit form with one buffer beats int8 operands with two: C5 product 123 us against 175 us)
    if (p.nbuf == 2 && split_ok && 2 * acc_cols + 16 > 512 && acc_cols + 16 <= 512) p.nbuf = 1;
    p.fp4 = (p.nbuf * acc_cols + 16 <= 512 && split_ok) ? 1 : 0;
    p.sf_col = p.nbuf * acc_cols;
    p.steps = p.fp4 ? (CH + 1) / 2 : CH;
    p.pad = p.wpr * 32 - p.a.n + ((p.fp4 && (CH & 1)) ? 128 : 0);
    // the weight operand of the 4-bit form goes to tensor memory when at least three stages of 32 columns fit beside the
    // accumulators and the scale factors
    const int a_stages = p.fp4 ? (512 - (p.nbuf * acc_cols + 16)) / 32 : 0;
    p.a_tmem = a_stages >= 3 ? 1 : 0;
    p.a_col = p.sf_col + 16;
    const size_t stage = (size_t)128 * ((p.a_tmem ? 0 : TILE_M) + p.n_mma);
    p.yt_bytes = (int)(((size_t)p.nseg * TILE_M * staging_stride(p.TB, p.a.epilogue) * 4 + 15) / 16 * 16);
    const size_t fixed = (size_t)p.yt_bytes + (2 * MAX_STAGES + 4) * 8 + 16 + (2 * TILE_M + 256 + 128) * 4;
    int S = (int)((225 * 1024 - fixed) / stage);
    if (S > MAX_STAGES) S = MAX_STAGES;
    if (p.a_tmem && S > a_stages) S = a_stages;
    if (S < 2) return false;
    p.nstages = S;
    int cols = 32;
    while (cols < p.nbuf * acc_cols + (p.fp4 ? 16 : 0) + (p.a_tmem ? 32 * S : 0)) cols <<= 1;
    p.tmem_cols = cols;
    p.expanders = (TILE_M + p.n_mma + 31) / 32 * 32;
    // one expander group; eight epilogue warps, or up to sixteen where the MMAs of the next tile have to wait for the
    // epilogue (one accumulator buffer; measured: C4 timestep 53.7 -> 50.3 us, nothing gained with two buffers)
    p.groups = 1;
    p.epi_warps = (p.nbuf == 1) ? 16 : 8;
    while (p.epi_warps > 4 && p.groups * p.expanders + 32 + 32 * p.epi_warps > MAX_THREADS) p.epi_warps -= 4;
    if (p.groups * p.expanders + 32 + 32 * p.epi_warps > MAX_THREADS) return false;
    out->p = p;
    out->smem = S * stage + fixed;
    out->grid = dim3((unsigned)sms);
    out->threads = p.groups * p.expanders + 32 + 32 * p.epi_warps;
    out->persistent = true;
    return out->smem <= 227 * 1024;
}

bool plan(const GemmArgs& a, TcPlan* out)
{
    TcParams p{};
    p.a = a;
    p.wpr = words_per_row(a.n);
    p.nseg = 1;
    if (a.epilogue == EPI_LSTM) { p.gates = 4; p.units = a.H; }
    else if (a.epilogue == EPI_GRU) {
        p.gates = 3; p.units = a.H; p.nseg = 2;
        if (a.I % 32 != 0 || a.I == 0) return false;        // the column split must fall on a word boundary
    } else { p.gates = 1; p.units = a.m; }
    p.UT = TILE_M / (p.gates * a.k_w);
    if (p.UT < 1) return false;
    // batch entries per tile: multiples of 16, N = TB * k_a <= 256
    int tb_max = (256 / a.k_a) / 16 * 16;
    if (tb_max > 128) tb_max = 128;
    const int ntiles = (a.batch + tb_max - 1) / tb_max;
    p.TB = ((a.batch + ntiles - 1) / ntiles + 15) / 16 * 16;
    p.n_mma = p.TB * a.k_a;
    // two M tiles per CTA when their accumulators fit tensor memory and enough CTAs remain to fill the GPU
    const int mtiles = (p.units + p.UT - 1) / p.UT;
    const int btiles = (a.batch + p.TB - 1) / p.TB;
    for (int sft = 0; sft < 8; ++sft) p.mul[sft] = 1u << (7 - sft);
    p.mask_sign = 0x80808080u;
    p.mask_half = 0x40404040u;
    p.MT = (2 * p.nseg * p.n_mma <= 512 && (long long)(mtiles / 2) * btiles >= 2 * sm_count()) ? 2 : 1;
    // with one M tile per CTA and more tiles than SMs, the persistent form hides the epilogues; with two M tiles
    // per CTA the plain form's lower shared-memory traffic per MMA counts for more (measured), unless their accumulators
    // leave no room for the scale factors of the 4-bit form and one M tile per CTA does (C5: 142 us plain with int8
    // operands, 123 us persistent with 4-bit ones)
    const bool two_tiles_4bit = 2 * p.nseg * p.n_mma + 16 <= 512 && (p.nseg == 1 || a.I % 256 == 0);
    if ((p.MT == 1 || !two_tiles_4bit) && plan_persistent(p, mtiles, btiles, out) && (p.MT == 1 || out->p.fp4)) return true;
    // 4-bit operands where the scale factors' 16 tensor-memory columns fit beside the accumulators and a GRU's column
    // split falls on a pipeline step (256 bit positions)
    const int acc_cols = p.MT * p.nseg * p.n_mma;
    const int CH = p.wpr >> 2;
    p.fp4 = (acc_cols + 16 <= 512 && (p.nseg == 1 || a.I % 256 == 0)) ? 1 : 0;
    p.sf_col = acc_cols;
    p.steps = p.fp4 ? (CH + 1) / 2 : CH;
    p.pad = p.wpr * 32 - a.n + ((p.fp4 && (CH & 1)) ? 128 : 0);
    // with one M tile per CTA the weight operand of the 4-bit form goes to tensor memory when at least three stages of 32
    // columns fit beside the accumulators and the scale factors (and the epilogue's staging array still fits the stages)
    const int a_stages = (p.fp4 && p.MT == 1) ? (512 - (acc_cols + 16)) / 32 : 0;
    const size_t epi = (size_t)p.MT * p.nseg * TILE_M * staging_stride(p.TB, a.epilogue) * 4;
    p.a_tmem = (a_stages >= 3 && epi <= (size_t)(a_stages < MAX_STAGES ? a_stages : MAX_STAGES) * 128 * p.n_mma) ? 1 : 0;
    p.a_col = p.sf_col + 16;
    const size_t stage = (size_t)128 * ((p.a_tmem ? 0 : p.MT * TILE_M) + p.n_mma);
    int S = (int)((220 * 1024) / stage);
    if (S > MAX_STAGES) S = MAX_STAGES;
    if (p.a_tmem && S > a_stages) S = a_stages;
    if (S < 2) return false;
    if (epi > S * stage) return false;
    p.nstages = S;
    int cols = 32;
    while (cols < acc_cols + (p.fp4 ? 16 : 0) + (p.a_tmem ? 32 * S : 0)) cols <<= 1;
    if (cols > 512) return false;
    p.tmem_cols = cols;
    p.expanders = (p.MT * TILE_M + p.n_mma + 31) / 32 * 32;
    p.groups = (2 * p.expanders + 32 <= MAX_THREADS) ? 2 : 1;
    out->p = p;
    out->smem = S * stage + (2 * MAX_STAGES + 1) * 8 + 24 + (2 * TILE_M + 256 + 128) * 4;   // stages, barriers, slot, coefficients
    out->grid = dim3((unsigned)((mtiles + p.MT - 1) / p.MT), (unsigned)btiles);
    out->threads = p.groups * p.expanders + 32;
    out->persistent = false;
    return out->grid.y <= 65535u && out->smem <= 227 * 1024;
}

template <int KA>
amq_status launch_ka(const TcPlan& pl, cudaStream_t st)
{
    auto kernel = pl.persistent ? (pl.p.fp4 ? bgemm_tc_persistent_kernel<KA, true> : bgemm_tc_persistent_kernel<KA, false>)
                                : (pl.p.fp4 ? bgemm_tc_kernel<KA, true> : bgemm_tc_kernel<KA, false>);
    AMQ_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem));
    if (pl.p.a.overlap_with_previous) {
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = pl.grid; cfg.blockDim = dim3((unsigned)pl.threads); cfg.dynamicSmemBytes = pl.smem; cfg.stream = st;
        cudaLaunchAttribute attr{};
        attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr.val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = &attr; cfg.numAttrs = 1;
        AMQ_CUDA_TRY(cudaLaunchKernelEx(&cfg, kernel, pl.p));
        AMQ_LAUNCH_CHECK();
        return AMQ_OK;
    }
    kernel<<<pl.grid, pl.threads, pl.smem, st>>>(pl.p);
    AMQ_LAUNCH_CHECK();
    return AMQ_OK;
}

}  // namespace

bool gemm_tc_supported(const GemmArgs& a)
{
    // from 16 vectors on always; for 2..15 vectors (one padded tile of 16) when the weight matrix is large
    // enough that the CUDA-core kernel's tile loop costs more than this kernel's fixed ~10 us
    TcPlan pl;
    const bool big = (long long)a.m * a.k_w * words_per_row(a.n) >= (1ll << 17);
    return (a.batch >= 16 || (a.batch >= 2 && big)) && plan(a, &pl);
}

bool gemm_tc_single_wave(const GemmArgs& a)
{
    TcPlan pl;
    if (!gemm_tc_supported(a) || !plan(a, &pl)) return false;
    return pl.persistent || (long long)pl.grid.x * pl.grid.y <= sm_count();
}

amq_status launch_binary_gemm_tc(const GemmArgs& a, cudaStream_t st)
{
    TcPlan pl;
    if (!plan(a, &pl)) return AMQ_ERR_UNSUPPORTED;
    switch (a.k_a) {
        case 1: return launch_ka<1>(pl, st);
        case 2: return launch_ka<2>(pl, st);
        case 3: return launch_ka<3>(pl, st);
        case 4: return launch_ka<4>(pl, st);
    }
    return AMQ_ERR_UNSUPPORTED;
}

// one thread swaps the status word for zero and leaves the old value in the second word: read and clear are a single
// atomic step, so a failure recorded by a kernel of another stream in between is neither lost nor reported twice
__global__ void take_tc_status_kernel()
{
    g_tc_status_taken = atomicExch(&g_tc_status, 0u);
}

amq_status read_tc_status(cudaStream_t st, uint32_t* out)
{
    take_tc_status_kernel<<<1, 1, 0, st>>>();
    AMQ_LAUNCH_CHECK();
    AMQ_CUDA_TRY(cudaStreamSynchronize(st));
    AMQ_CUDA_TRY(cudaMemcpyFromSymbol(out, g_tc_status_taken, sizeof(uint32_t)));
    return AMQ_OK;
}

}  // namespace amq
