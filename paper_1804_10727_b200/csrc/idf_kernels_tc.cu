// Tensor-core path of the dense Δ-row update (Eq. 4 for a whole row of events at once) with the
// row finalisation (Eq. 2-3) as its epilogue, for bf16 (fp32 state) and int8 (int32 state) nets.
//
// One CTA owns a tile of 128 (stream, x) positions times Ntile output channels of one conv layer
// and walks the block's input rows in order.  While it does so the layer's ring rows for that tile
// live in tensor memory: every ring row is a TMEM accumulator of Ntile columns, and input row r adds
// its contribution to the accumulator of every output row it reaches, one tcgen05.mma per kernel tap
// (ky, kx) and 32-byte K step:   C_o[m, n] += sum_ci  Δ_r[m shifted by kx, ci] * W[ky][kx][n][ci].
//   - the CTA's weight slice (all taps, Ntile channels) is fetched once by TMA and stays in shared
//     memory (weight-stationary);
//   - Δ-rows stream through a ring of shared-memory stages, one TMA box per (input row, kx, K block);
//     the kx shift and the zero padding in x come from the box's start coordinate (out-of-range
//     coordinates read zeros);
//   - an accumulator starts from what its row has so far: zero, or, for a row begun by an earlier
//     block, the partial sums that block left in the ring in global memory (copied in at the start
//     of the launch);
//   - when an input row was the last one an output row was waiting for, the epilogue warps read that
//     accumulator, add the bias, apply f, round or requantise, and write the row for the next layer;
//     rows still open at the end of the block go back to the ring in global memory.
// Warp roles: warp 0 = TMA producer and row scheduler, warp 1 = TMEM owner and MMA issuer,
// warps 2.. = epilogue groups of four warps (one warp per TMEM lane quarter) that take output rows in turn.
// Every wait is bounded; on expiry the kernel records IDF_ERR_TIMEOUT in the status word and leaves.
#include "../../include/idf.h"
#include "idf_internal.h"

#include <cuda.h>
#include <cstdlib>
#include <mutex>

namespace idf {

namespace {

constexpr int MAX_GROUPS = 3;                // epilogue groups (four warps each) taking output rows in turn
constexpr int TC_THREADS = 64 + 128 * MAX_GROUPS;
constexpr int ROWQ = 64;                     // row-schedule queue: two chunks of 32 rows
constexpr uint32_t WAIT_LIMIT = 1u << 22;
constexpr size_t SMEM_LIMIT = 232448;        // 227 KB per CTA

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Non-blocking look at a barrier phase (the result may be consumed much later: the round trip to the
// barrier then overlaps whatever is issued in between).
__device__ __forceinline__ uint32_t mbar_test(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
// Bounded wait: false if the limit ran out or another role has given up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag)
{
    for (uint32_t i = 0; i < WAIT_LIMIT; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 31u) == 31u) {
            if (*abort_flag) return false;
            __nanosleep(32);
        }
    }
    *abort_flag = 1;
    return false;
}
// The same for roles that are not on the critical path (producer waiting for a free stage, epilogue
// waiting for a finished row): sleep between polls, so the polling warp leaves the issue slots of its
// scheduler to the MMA-issuing warp that shares it.
__device__ __forceinline__ bool mbar_wait_relaxed(uint32_t bar, uint32_t parity, volatile int* abort_flag)
{
    for (uint32_t i = 0; i < WAIT_LIMIT; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        __nanosleep(200);
        if ((i & 15u) == 15u && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2, int c3)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}

// true in exactly one lane of a converged warp
__device__ __forceinline__ bool elect_one()
{
    uint32_t pred;
    asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
    return pred != 0;
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

template <int DT>
__device__ __forceinline__ void umma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    if (DT == 1) {
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
    } else {
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
    }
}
// All K steps of one shared-memory tile pair in one go (always accumulating): the descriptors move
// 32 bytes (2 units of 16 B) per step inside the swizzled row.
template <int DT, int KSTEPS>
__device__ __forceinline__ void umma_tile(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc)
{
#define IDF_MMA_KIND(kind)                                                                              \
    if (KSTEPS == 1)                                                                                    \
        asm volatile("{\n\t.reg .pred p;\n\tsetp.eq.b32 p, 0, 0;\n\t"                                   \
                     "tcgen05.mma.cta_group::1.kind::" kind " [%0], %1, %2, %3, p;\n\t}"                 \
                     ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc));                     \
    else if (KSTEPS == 2)                                                                               \
        asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 a1, b1;\n\tsetp.eq.b32 p, 0, 0;\n\t"              \
                     "add.s64 a1, %1, 2;\n\tadd.s64 b1, %2, 2;\n\t"                                     \
                     "tcgen05.mma.cta_group::1.kind::" kind " [%0], %1, %2, %3, p;\n\t"                  \
                     "tcgen05.mma.cta_group::1.kind::" kind " [%0], a1, b1, %3, p;\n\t}"                 \
                     ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc));                     \
    else                                                                                                \
        asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 a1, b1, a2, b2, a3, b3;\n\tsetp.eq.b32 p, 0, 0;\n\t" \
                     "add.s64 a1, %1, 2;\n\tadd.s64 b1, %2, 2;\n\tadd.s64 a2, %1, 4;\n\tadd.s64 b2, %2, 4;\n\t" \
                     "add.s64 a3, %1, 6;\n\tadd.s64 b3, %2, 6;\n\t"                                     \
                     "tcgen05.mma.cta_group::1.kind::" kind " [%0], %1, %2, %3, p;\n\t"                  \
                     "tcgen05.mma.cta_group::1.kind::" kind " [%0], a1, b1, %3, p;\n\t"                  \
                     "tcgen05.mma.cta_group::1.kind::" kind " [%0], a2, b2, %3, p;\n\t"                  \
                     "tcgen05.mma.cta_group::1.kind::" kind " [%0], a3, b3, %3, p;\n\t}"                 \
                     ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc));
    if (DT == 1) { IDF_MMA_KIND("f16") } else { IDF_MMA_KIND("i8") }
#undef IDF_MMA_KIND
}
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void tmem_st16_zero(uint32_t taddr)
{
    const uint32_t z = 0;
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1};"
        ::"r"(taddr), "r"(z) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Position of tap row ky inside a stacked weight tile.  The Kh blocks of Ntile rows are ordered so
// that the taps one input row uses (ky = ph, ph+stride, ...) sit next to each other with ky
// descending: their output rows ascend, and so do the ring slots (TMEM columns) they accumulate
// into, which lets one MMA of N = (taps)*Ntile serve several ring rows at once.
__host__ __device__ __forceinline__ int weight_block(int ky, int Kh, int stride)
{
    const int ph = ky % stride;
    int off = 0;
    for (int p = 0; p < ph; ++p) off += (Kh - p + stride - 1) / stride;
    const int cnt = (Kh - ph + stride - 1) / stride;
    return off + cnt - 1 - ky / stride;
}

// shared-memory matrix descriptor, K-major operand in the canonical swizzled layout:
// rows of `swb` bytes, 8-row groups `8*swb` bytes apart
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr, uint32_t swb)
{
    const uint64_t layout = swb == 128 ? 2 : (swb == 64 ? 4 : 6);
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;                           // leading-dimension offset: unused for swizzled K-major
    d |= (uint64_t)((8u * swb) >> 4) << 32;           // stride-dimension offset between 8-row groups
    d |= (uint64_t)1 << 46;                           // descriptor version of this architecture
    d |= layout << 61;
    return d;
}


// TMEM loads of W consecutive accumulator columns of this thread's lane
template <int W>
__device__ __forceinline__ void tmem_ld(uint32_t taddr, uint32_t (&v)[W])
{
    if (W == 16) {
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
            : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
              "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
            : "r"(taddr) : "memory");
    } else {
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
            "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
            : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
              "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
              "=r"(v[16 % W]), "=r"(v[17 % W]), "=r"(v[18 % W]), "=r"(v[19 % W]), "=r"(v[20 % W]), "=r"(v[21 % W]),
              "=r"(v[22 % W]), "=r"(v[23 % W]), "=r"(v[24 % W]), "=r"(v[25 % W]), "=r"(v[26 % W]), "=r"(v[27 % W]),
              "=r"(v[28 % W]), "=r"(v[29 % W]), "=r"(v[30 % W]), "=r"(v[31 % W])
            : "r"(taddr) : "memory");
    }
}
// (the registers of a tcgen05.ld are valid after this wait: several loads may be in flight before it)
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
template <int W>
__device__ __forceinline__ void tmem_st_zero(uint32_t taddr)
{
    const uint32_t z = 0;
    if (W == 16)
        asm volatile(
            "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1};"
            ::"r"(taddr), "r"(z) : "memory");
    else
        asm volatile(
            "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, "
            "%1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1};"
            ::"r"(taddr), "r"(z) : "memory");
}


// 16 words of this thread's lane into 16 consecutive columns
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
          "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]) : "memory");
}

// Where an emitted row goes first: a shared-memory tile [tile row][panel of pwb bytes], written in
// the swizzle the output tensor map expects, from which one thread sends it out with a TMA store.
struct StageSink {
    uint32_t row_base;     // shared address of this thread's tile row in panel 0
    uint32_t panel_bytes;  // bytes of one panel (staged rows * pwb)
    uint32_t pwb_log2;     // log2(panel row bytes)
    uint32_t phase;        // swizzle phase of this row (XORed into the 16-byte chunk index)
};
__device__ __forceinline__ void stage_store16(const StageSink& k, uint32_t col_byte, int4 v)
{
    const uint32_t panel = col_byte >> k.pwb_log2;
    const uint32_t within = col_byte & ((1u << k.pwb_log2) - 1u);
    const uint32_t addr = k.row_base + panel * k.panel_bytes + ((((within >> 4) ^ k.phase)) << 4);
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ int4 stage_load16(const StageSink& k, uint32_t col_byte)
{
    const uint32_t panel = col_byte >> k.pwb_log2;
    const uint32_t within = col_byte & ((1u << k.pwb_log2) - 1u);
    const uint32_t addr = k.row_base + panel * k.panel_bytes + ((((within >> 4) ^ k.phase)) << 4);
    int4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
// element-wise maximum of two 32-bit words holding OP = 0: two bf16, 1: one fp32, 2: four int8
template <int OP>
__device__ __forceinline__ uint32_t word_max(uint32_t x, uint32_t y)
{
    if (OP == 0) { uint32_t r; asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(x), "r"(y)); return r; }
    if (OP == 1) return __float_as_uint(fmaxf(__uint_as_float(x), __uint_as_float(y)));
    return __vmaxs4(x, y);
}
// 2x2 max-pooling folded into the emission of a conv layer's rows.  A thread owns one (stream, x)
// position; its x neighbour is the next lane.  The x-pooled first row of a pair waits in the group's
// staging tile (or, across launches, in the pool layer's state in global memory) until the second
// row arrives; the pooled row then leaves through the TMA store.
struct PoolCtx {
    int on;            // pooling is folded into this launch
    int writer;        // this thread holds the pooled value of an in-tile position (even x)
    int second;        // the row at hand is the second of its pair
    int from_state;    // ... and the first one was emitted by an earlier launch
    int to_state;      // the row at hand is a first row whose partner comes with a later launch
    int drop;          // a first row at the end of input: never completed, nothing is kept
    StageSink sink;    // pooled tile (half the positions)
    unsigned char* state;   // this thread's pooled position in the pool layer's state, at the CTA's first channel
};
template <int NW, int OP>
__device__ __forceinline__ void deliver(uint32_t (&ow)[NW], const StageSink& sink, uint32_t col_byte, const PoolCtx& pc, bool state_ok)
{
    if (!pc.on) {
#pragma unroll
        for (int j4 = 0; j4 < NW / 4; ++j4)
            stage_store16(sink, col_byte + 16u * j4, make_int4((int)ow[4 * j4], (int)ow[4 * j4 + 1], (int)ow[4 * j4 + 2], (int)ow[4 * j4 + 3]));
        return;
    }
#pragma unroll
    for (int j = 0; j < NW; ++j) ow[j] = word_max<OP>(ow[j], __shfl_xor_sync(0xffffffffu, ow[j], 1));
    if (!pc.writer || pc.drop) return;
#pragma unroll
    for (int j4 = 0; j4 < NW / 4; ++j4) {
        int4 v = make_int4((int)ow[4 * j4], (int)ow[4 * j4 + 1], (int)ow[4 * j4 + 2], (int)ow[4 * j4 + 3]);
        if (pc.second) {
            int4 h = make_int4(0, 0, 0, 0);
            if (!pc.from_state) h = stage_load16(pc.sink, col_byte + 16u * j4);
            else if (state_ok) h = *(const int4*)(pc.state + col_byte + 16u * j4);
            v.x = (int)word_max<OP>((uint32_t)v.x, (uint32_t)h.x); v.y = (int)word_max<OP>((uint32_t)v.y, (uint32_t)h.y);
            v.z = (int)word_max<OP>((uint32_t)v.z, (uint32_t)h.z); v.w = (int)word_max<OP>((uint32_t)v.w, (uint32_t)h.w);
        }
        if (pc.to_state) { if (state_ok) *(int4*)(pc.state + col_byte + 16u * j4) = v; }
        else stage_store16(pc.sink, col_byte + 16u * j4, v);
    }
}
__device__ __forceinline__ void tma_store_4d(const CUtensorMap* tm, uint32_t src, int c0, int c1, int c2, int c3)
{
    asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
                 ::"l"(tm), "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void named_bar_sync(int id, int count)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
// barrier among `count` threads that also tells everyone whether all of them passed `pred`
__device__ __forceinline__ bool named_bar_and(int id, int count, bool pred)
{
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 p, %3, 0;\n\t"
        "bar.red.and.pred q, %1, %2, p;\n\tselp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r) : "r"(id), "r"(count), "r"((uint32_t)pred) : "memory");
    return r != 0;
}

// Row finalisation of W accumulator columns of one (stream, x) position: add what earlier blocks
// left in the ring, then either park the sum in the ring (row still open) or emit f(c + b) in the
// layer's output type.
// Ring rows in global memory are read and written 32 bytes per thread and instruction: a thread's run of channels
// is its own, so narrower accesses would touch every 32-byte sector of the run twice.
__device__ __forceinline__ void ld_global_v8(const void* p, uint32_t (&v)[8])
{
    asm volatile("ld.global.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]) : "l"(p));
}
__device__ __forceinline__ void st_global_v8(void* p, const uint32_t (&v)[8])
{
    asm volatile("st.global.v8.b32 [%8], {%0, %1, %2, %3, %4, %5, %6, %7};"
                 :: "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "l"(p) : "memory");
}

template <int DT, int W, typename TS>
__device__ __forceinline__ void finalise_chunk(const uint32_t (&v)[W], bool emit, TS* rp,
                                               const TS* bias_c, const StageSink& sink, uint32_t col_byte, int out_elem,
                                               int relu, int shift, const PoolCtx& pc, bool state_ok)
{
    TS acc[W];
#pragma unroll
    for (int j = 0; j < W; ++j) acc[j] = DT == 1 ? (TS)__uint_as_float(v[j]) : (TS)(int)v[j];
    if (!emit) {
#pragma unroll
        for (int j8 = 0; j8 < W / 8; ++j8) {
            uint32_t t[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) t[j] = DT == 1 ? __float_as_uint((float)acc[8 * j8 + j]) : (uint32_t)(int)acc[8 * j8 + j];
            st_global_v8(rp + 8 * j8, t);
        }
        return;
    }
    if (DT == 1) {
        float f[W];
#pragma unroll
        for (int j = 0; j < W; ++j) f[j] = (float)acc[j];
        if (bias_c) {
#pragma unroll
            for (int j4 = 0; j4 < W / 4; ++j4) {
                const float4 b4 = ((const float4*)bias_c)[j4];
                f[4 * j4] += b4.x; f[4 * j4 + 1] += b4.y; f[4 * j4 + 2] += b4.z; f[4 * j4 + 3] += b4.w;
            }
        }
        if (out_elem == E_BF16) {
            // two values per instruction: round to nearest even, with the ReLU folded into the conversion
            uint32_t pk[W / 2];
            if (relu) {
#pragma unroll
                for (int j = 0; j < W / 2; ++j)
                    asm("cvt.rn.relu.bf16x2.f32 %0, %1, %2;" : "=r"(pk[j]) : "f"(f[2 * j + 1]), "f"(f[2 * j]));
            } else {
#pragma unroll
                for (int j = 0; j < W / 2; ++j)
                    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(pk[j]) : "f"(f[2 * j + 1]), "f"(f[2 * j]));
            }
            deliver<W / 2, 0>(pk, sink, col_byte, pc, state_ok);
        } else {
            if (relu) {
#pragma unroll
                for (int j = 0; j < W; ++j) f[j] = fmaxf(f[j], 0.f);
            }
            uint32_t fw[W];
#pragma unroll
            for (int j = 0; j < W; ++j) fw[j] = __float_as_uint(f[j]);
            deliver<W, 1>(fw, sink, col_byte, pc, state_ok);
        }
    } else {
        const int lo = relu ? 0 : -127;
        uint32_t pk[W / 4];
#pragma unroll
        for (int j = 0; j < W / 4; ++j) pk[j] = 0;
#pragma unroll
        for (int j = 0; j < W; ++j) {
            int t = (int)acc[j] + (bias_c ? (int)bias_c[j] : 0);
            if (relu && t < 0) t = 0;
            if (shift > 0) t = (t + (1 << (shift - 1))) >> shift;
            t = t < lo ? lo : (t > 127 ? 127 : t);
            pk[j >> 2] |= ((uint32_t)t & 0xffu) << (8 * (j & 3));
        }
        deliver<W / 4, 2>(pk, sink, col_byte, pc, state_ok);
    }
}

struct TcArgs {
    const void* bias;
    void* ring;
    const void* ring_in;         // where the rows begun by earlier blocks are read: the ring, or a copy of it made before a
                                 // launch whose row chunks run in CTAs of their own (one parks rows while another still reads)
    void* out;
    unsigned int* status;
    long long out_row_stride, out_stream_stride, out_row_base;
    long long o_begin;           // absolute index of the first visited output row
    int r0_positive;             // input rows arrived before this block (r0 > 0)
    int n_rows;                  // input rows in this block
    int n_orows;                 // visited output rows: o_begin + [0, n_orows)
    int done_rel;                // rows with relative index < done_rel are emitted, the others go back to the ring
    int sched_rel;               // rows below it are completed by an input row of this block; rows in [sched_rel, done_rel)
                                 // wait only for bottom padding and are completed by the block's last row (end of input)
    int base_ty;                 // r0 + pad - o_begin*stride: input row ri reaches relative output row
                                 // (base_ty + ri - ky) / stride through tap ky when that is a whole number >= 0
    int S, Wout, Cout, Kh, Kw, stride, pad_x, relu, shift, ring_rows, out_elem;
    int BX, BXP, BS, n_xt, Ntile, n_nt, KB, n_kb, swb, nslot, nstage, tmem_cols;
    int shift_mode;              // 1: one box per (row, K block) holds the kx halo, taps address it at row offsets
    int sx;                      // x stride of the conv (1, or more when every kx tap has a box of its own: the tensor map then
                                 // walks the input row in steps of sx, so a box still holds BXP consecutive OUTPUT positions)
    int n_chunks, chunk_rows, chunk_shift;   // the block's output rows are cut into n_chunks runs of chunk_rows rows (the first one
                                 // chunk_shift shorter), one CTA each: see the kernel's prologue
    int a_stage_bytes;
    int n_box, a_box_pitch;      // TMA boxes per stage (one per kx tap when the taps cannot share a haloed box) and their distance in bytes
    int out_esize, out_pwb, out_panels, out_stage_bytes;   // emitted rows: staging panels of out_pwb-byte rows
    int out_stage_rows;          // rows of one staging panel: 128, or 64 when only pooled rows are staged
    int out_groups;              // epilogue groups at work, each with its own staging tile(s)
    int out_bufs;                // staging tiles per group (1 or 2, used in turn)
    int out_row_dim;             // position of the row coordinate in the output tensor map (2 or 3)
    int out_row_first;           // tensor-map row index of relative output row 0
    // 2x2 max-pooling folded into the emission (the output tensor map then describes the pooled rows)
    int pool;                    // 1: emit pooled rows
    int pool_keep;               // 1: a trailing first row of a pair waits in pool_state for a later launch; 0: end of input, it is dropped
    void* pool_state;            // [S][Wout/2][Cout] in the output type: x-pooled first row of an open pair
    long long pool_row_base;     // pooled row p goes to tensor-map row p - pool_row_base
    // small pieces of o_begin, so that the row loop needs no 64-bit arithmetic
    int o_begin_par;             // o_begin & 1
    int o_begin_half_mod;        // (o_begin >> 1) mod out_groups
    int ring_slot0;              // o_begin mod ring_rows
    int pool_row_first;          // (o_begin >> 1) - pool_row_base: tensor-map row of the pair that holds o_begin
    long long ring_elems, pool_state_bytes;   // extents of ring (state words) and pool_state (bytes): range-checked build
    unsigned int smem_bytes;     // dynamic shared memory of the launch (range-checked build)
};

template <int DT> struct Acc;
template <> struct Acc<1> { typedef float S; };
template <> struct Acc<2> { typedef int S; };

// KX3: the common case of 128-byte rows with three kx taps read row-shifted from one haloed box, known at compile time
// (the MMA warp's loop is what the kernel's speed hangs on: every constant it sees helps)
template <int DT, int KSTEPS, int KX3>
__global__ void __launch_bounds__(TC_THREADS, 1)
conv_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW,
               const __grid_constant__ CUtensorMap tmO, const TcArgs a)
{
    typedef typename Acc<DT>::S TS;
    extern __shared__ unsigned char smem_raw[];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    __shared__ int s_issued;
    __shared__ __align__(16) uint32_t s_rowq[ROWQ][16];                // per input row: what the MMA thread must do

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next kernel may start its own prologue
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int taps = a.Kh * a.Kw;
    const uint32_t w_tile_bytes = (uint32_t)a.Ntile * a.swb;
    const uint32_t a_stage_bytes = (uint32_t)a.a_stage_bytes;
    const uint32_t a_box_bytes = (uint32_t)a.BXP * a.BS * a.swb;
    // (rows of 128 bytes always share one haloed box: for that instantiation the compiler sees the constant)
    const int n_box = KSTEPS == 4 ? 1 : a.n_box;

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sW = base;
    const uint32_t sA = (sW + (uint32_t)taps * a.n_kb * w_tile_bytes + 1023u) & ~1023u;
    const uint32_t sOut = sA + (uint32_t)a.nstage * a_stage_bytes;               // one staging tile per epilogue group
    const uint32_t bars = sOut + (uint32_t)(a.out_groups * a.out_bufs) * (uint32_t)a.out_stage_bytes;
    const uint32_t bar_full = bars;
    const uint32_t bar_empty = bar_full + 8u * a.nstage;
    const uint32_t bar_w = bar_empty + 8u * a.nstage;
    const uint32_t bar_ready = bar_w + 8u * taps;
    const uint32_t bar_free = bar_ready + 8u * a.nslot;

    const int nt = blockIdx.x % a.n_nt;
    const int mt_all = blockIdx.x / a.n_nt;
    const int n_mt_all = a.n_xt * ((a.S + a.BS - 1) / a.BS);
    const int mt = mt_all % n_mt_all;
    // Row chunks.  When a layer has few (position, channel) tiles, the block's output rows are cut into runs and
    // every run gets CTAs of its own: a run needs only the input rows its output rows reach, which it reads again
    // at its edges instead of taking partial sums from its neighbour.  Inside a chunk everything is as in a block
    // that starts at the chunk's first output row: taps into rows of other chunks drop out, only the first chunk
    // takes up the ring, only the last one parks rows in it.
    const int chunk = mt_all / n_mt_all;
    const int c_oa = chunk == 0 ? 0 : chunk * a.chunk_rows - a.chunk_shift;                       // first relative output row
    const int c_ob = chunk == a.n_chunks - 1 ? a.n_orows : (chunk + 1) * a.chunk_rows - a.chunk_shift;
    int c_ra = c_oa * a.stride - a.base_ty;                                                        // first input row that reaches it
    if (c_ra < 0) c_ra = 0;
    int c_rb = (c_ob - 1) * a.stride - a.base_ty + a.Kh;                                           // one past the last
    if (c_rb > a.n_rows || chunk == a.n_chunks - 1) c_rb = a.n_rows;
    const int c_base_ty = a.base_ty + c_ra - c_oa * a.stride;
    const int c_n_orows = c_ob - c_oa;
    const int c_done_rel = min(max(a.done_rel - c_oa, 0), c_n_orows);
    const int c_sched_rel = min(max(a.sched_rel - c_oa, 0), c_n_orows);
    const bool c_r0_positive = a.r0_positive && chunk == 0;
    const int xt = mt % a.n_xt, stile = mt / a.n_xt;
    const int x0 = xt * a.BX, s0 = stile * a.BS, n0 = nt * a.Ntile;

    if (threadIdx.x == 0) {
        s_abort = 0;
        s_issued = 0;
        if (!IDF_OK_AT(a.status, (bar_free - smem_u32(smem_raw)) + 8u * a.nslot - 1, a.smem_bytes)) s_abort = 1;
        // The weights come first: they do not depend on earlier kernels of the stream (their fetch overlaps the
        // previous kernel's tail under programmatic dependent launch), and a launch that brings a single row has
        // little else to hide their latency behind.  One copy per K block carries all taps of the CTA's channel
        // slice (the parameters are stored tap by tap in the order the stacked tiles want, see tc_pack_weights).
        mbar_init(bar_w, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_expect_tx(bar_w, (uint32_t)(taps * a.n_kb) * w_tile_bytes);
        for (int kb = 0; kb < a.n_kb; ++kb)
            tma_load_3d(sW + (uint32_t)(kb * taps) * w_tile_bytes, &tmW, bar_w, kb * a.KB, n0, 0);
        for (int i = 0; i < a.nstage; ++i) { mbar_init(bar_full + 8u * i, 1); mbar_init(bar_empty + 8u * i, 1); }
        for (int i = 0; i < a.nslot; ++i) { mbar_init(bar_ready + 8u * i, 1); mbar_init(bar_free + 8u * i, 4); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)), "r"((uint32_t)a.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // everything below reads or writes buffers that earlier kernels of the stream produce or consume
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const uint32_t tmem_base = s_tmem_base;
    volatile int* abort_flag = &s_abort;
    const int n_rows = c_rb - c_ra;

    if (warp == 0) {
        // ------------------------------ TMA producer + row scheduler ---------------------------
        // One thread issues every MMA and the tensor pipe runs only a couple of instructions ahead
        // of it, so that thread must do as little else as possible.  This thread, which mostly waits
        // for free stages, therefore also works out for every input row which accumulators it feeds
        // and leaves the answer in a small queue next to the data (published by the stage's barrier).
        // With t0 = base_ty + ri the taps of input row ri are ky = ph, ph+s, ... (ph = t0 mod s), and
        // tap ky = ph + j*s reaches relative output row hi - j (hi = t0 div s).
        // The 32 lanes work out the schedule of 32 rows at a time (one row each, closed form), then
        // lane 0 issues those rows' copies.
        const uint32_t idesc0 = (DT == 1 ? ((1u << 4) | (1u << 7) | (1u << 10)) : ((2u << 4) | (1u << 7) | (1u << 10))) |
                                ((128u >> 4) << 24);
        const int max_rows = 256 / a.Ntile;              // ring rows one instruction can cover (N <= 256)
        const int s = a.stride, nslot = a.nslot;
        int stage = 0, t = 0;
        uint32_t phase = 0;
        bool ok = true;
        for (int r_chunk = 0; r_chunk < n_rows && ok; r_chunk += 32) {
            {
                const int ri = r_chunk + lane;
                if (ri < n_rows) {
                    uint32_t* q = s_rowq[ri & (ROWQ - 1)];
                    const int t0 = c_base_ty + ri;
                    const int hi = t0 / s, ph = t0 - hi * s;
                    const int slot_hi = hi % nslot, u_hi = hi / nslot;
                    // a new output row starts when ph == 0: its slot's previous row must have been read out
                    const bool fresh = (ri > 0 && ph == 0 && hi >= nslot && hi < c_n_orows);
                    q[0] = fresh ? bar_free + 8u * (uint32_t)slot_hi : 0u;
                    q[1] = (uint32_t)(u_hi & 1);
                    // the row completed by input row ri is (t0 - (Kh-1)) / s when that is a whole number >= 0
                    const int tf = t0 - (a.Kh - 1);
                    const int of = tf >= 0 ? tf / s : -1;
                    q[3] = (tf >= 0 && of * s == tf && of < c_sched_rel) ? bar_ready + 8u * (uint32_t)(of % nslot) : 0u;
                    // taps ky = ph, ph+s, ... < Kh; those that would reach rows above the map drop out
                    const int cnt = (a.Kh - ph + s - 1) / s;
                    int n_t = cnt;
                    if (n_t > hi + 1) n_t = hi + 1;
                    int sl = (slot_hi - (n_t - 1)) % nslot;
                    if (sl < 0) sl += nslot;
                    int poff = 0;
                    for (int p = 0; p < ph; ++p) poff += (a.Kh - p + s - 1) / s;
                    uint32_t blk = (uint32_t)(poff + cnt - n_t);
                    // ... and so do those that reach rows beyond this chunk (the highest rows = the first taps)
                    if (hi > c_n_orows - 1) n_t -= hi - (c_n_orows - 1);
                    // segments: runs of rows whose slots are consecutive TMEM column blocks (N <= 256 each)
                    int n_seg = 0;
                    for (int rem = n_t; rem > 0 && n_seg < 4; ++n_seg) {
                        int len = rem;
                        if (len > nslot - sl) len = nslot - sl;
                        if (len > max_rows) len = max_rows;
                        q[4 + 3 * n_seg] = tmem_base + (uint32_t)(sl * a.Ntile);
                        q[5 + 3 * n_seg] = (blk * w_tile_bytes) >> 4;
                        q[6 + 3 * n_seg] = idesc0 | ((uint32_t)((len * a.Ntile) >> 3) << 17);
                        rem -= len; blk += (uint32_t)len; sl += len;
                        if (sl == nslot) sl = 0;
                    }
                    q[2] = (uint32_t)n_seg;
                }
            }
            __syncwarp();
            if (lane == 0) {
                const int r_end = r_chunk + 32 < n_rows ? r_chunk + 32 : n_rows;
                for (int ri = r_chunk; ri < r_end && ok; ++ri) {
                    // A row that starts a new output row needs that row's slot read out and cleared.  Waiting
                    // here, before the row's first copy, means the MMA thread learns it from the copy's
                    // barrier and has one barrier less to look at.
                    const uint32_t* qr = s_rowq[ri & (ROWQ - 1)];
                    if (qr[0] && !mbar_wait(qr[0], qr[1], abort_flag)) { ok = false; break; }
                    // one stage per (row, K block): the haloed box all kx taps share, or one box per kx tap side by side
                    for (int kb = 0; kb < a.n_kb; ++kb) {
                        if (!mbar_wait(bar_empty + 8u * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
                        if (!IDF_OK_AT(a.status, (sA - smem_u32(smem_raw)) + (uint32_t)stage * a_stage_bytes + (uint32_t)(n_box - 1) * a.a_box_pitch + a_box_bytes - 1,
                                       bars - smem_u32(smem_raw))) { ok = false; break; }
                        mbar_expect_tx(bar_full + 8u * stage, (uint32_t)n_box * a_box_bytes);
                        for (int xl = 0; xl < n_box; ++xl)
                            tma_load_4d(sA + (uint32_t)stage * a_stage_bytes + (uint32_t)xl * a.a_box_pitch, &tmA, bar_full + 8u * stage,
                                        kb * a.KB, x0 * a.sx - a.pad_x + xl, s0, c_ra + ri);
                        ++t;
                        if (++stage == a.nstage) { stage = 0; phase ^= 1u; }
                    }
                }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        }
        if (lane == 0) s_issued = t;     // copies in flight, for the clean-up after a failed wait
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ---------------------------------------------
        // The whole warp runs this loop in step (every value in it is the same in all lanes) and one
        // elected lane issues the tensor-core instructions.  The tensor pipe runs only a few instructions
        // behind the issuing lane, so every cycle spent here on anything but issuing is a cycle the pipe
        // idles.  Hence: the barrier of the NEXT tile is looked at (non-blocking) before the current
        // tile's MMAs are issued and the answer is read after them, the next row's schedule entry is
        // fetched the same way, and the wait for a free accumulator slot is the producer's (a tile of a
        // row only arrives once its slot is free).
        {
            const uint64_t desc_hi = make_smem_desc(0, a.swb);
            const int n_kx = KX3 ? 3 : (a.shift_mode ? a.Kw : n_box);   // kx taps of a stage: row-shifted reads of one box, or one box each
            const int nslot = a.nslot;
            const uint32_t kx_bytes = (KSTEPS == 4 || a.shift_mode) ? (uint32_t)a.swb >> 4 : (uint32_t)a.a_box_pitch >> 4;
            // weight tiles in shared memory: [K block][kx][stacked ky block]
            const uint32_t wtile_kx = ((uint32_t)a.Kh * w_tile_bytes) >> 4;              // descriptor units per kx
            const uint32_t wtile_kb = ((uint32_t)taps * w_tile_bytes) >> 4;
            const uint32_t a_stage_units = a_stage_bytes >> 4;
            const int nstage = a.nstage, n_kb = a.n_kb;
            bool ok = true;
            // every slot this launch uses has been cleared once (a short launch visits fewer rows than there are slots)
            for (int slot = 0; slot < (c_n_orows < nslot ? c_n_orows : nslot) && ok; ++slot)
                ok = mbar_wait(bar_free + 8u * slot, 0, abort_flag);
            ok = ok && mbar_wait(bar_w, 0, abort_flag);          // the CTA's weight slice has landed
            const uint64_t adesc_base = desc_hi | (uint64_t)((sA & 0x3FFFFu) >> 4);
            const uint64_t bdesc_base = desc_hi | (uint64_t)((sW & 0x3FFFFu) >> 4);
            const int n_st = n_kb;                               // tiles (stages) per input row
            const bool issuer = elect_one();                     // the lane that issues (the warp stays converged)
            ok = ok && mbar_wait(bar_full, 0, abort_flag);       // first tile of the first row
            tc_fence_after();
            uint4 hdr = make_uint4(0, 0, 0, 0), sa = hdr, sb = hdr, sc = hdr;
            if (ok) {
                const uint4* q = (const uint4*)s_rowq[0];
                hdr = q[0]; sa = q[1]; sb = q[2]; sc = q[3];
            }
            // The loop runs over tiles (input row, kx box, K block), software-pipelined by hand: everything the NEXT
            // tile needs (stage, barrier, descriptors, and on a row's last tile the next row's schedule entry) is worked
            // out between the first and the last MMA group of the CURRENT tile, while the pipe is busy, so that between
            // the last MMA of one tile and the first MMA of the next there is only the commit and a handful of moves.
            // tap kx reads the same tile kxi rows further down: the swizzle is a function of the absolute
            // shared-memory address, so a start address moved by whole rows still meets the pattern the TMA
            // wrote (base-offset field stays 0).
            int ri = 0, st = 0, kb = 0, stage = 0;
            uint32_t phase = 0;
            uint64_t adesc_cur = adesc_base, bdesc_cur = bdesc_base;       // the tile at hand
            const long long n_tiles = (long long)n_rows * n_st;
            for (long long tile = 0; tile < n_tiles && ok; ++tile) {
                const bool row_end = st == n_st - 1;
                const bool last_row = ri == n_rows - 1;
                // ---- first MMA group of the tile
                if (issuer && hdr.z > 0) {
                    umma_tile<DT, KSTEPS>(sa.x, adesc_cur, bdesc_cur + (uint64_t)sa.y, sa.z);
                    if (hdr.z > 1) {
                        umma_tile<DT, KSTEPS>(sa.w, adesc_cur, bdesc_cur + (uint64_t)sb.x, sb.y);
                        if (hdr.z > 2) umma_tile<DT, KSTEPS>(sb.z, adesc_cur, bdesc_cur + (uint64_t)sb.w, sc.x);
                        if (hdr.z > 3) umma_tile<DT, KSTEPS>(sc.y, adesc_cur, bdesc_cur + (uint64_t)sc.z, sc.w);
                    }
                }
                // ---- the next tile, worked out while those run
                int n_stage = stage + 1;
                uint32_t n_phase = phase;
                uint64_t adesc_nx = adesc_cur + a_stage_units;
                if (n_stage == nstage) { n_stage = 0; n_phase ^= 1u; adesc_nx = adesc_base; }
                uint64_t bdesc_nx = bdesc_cur + wtile_kb;
                int n_kbi = kb + 1;
                if (n_kbi == n_kb) { n_kbi = 0; bdesc_nx = bdesc_base; }
                uint32_t next_ok = 1u;
                if (!(last_row && row_end)) next_ok = mbar_test(bar_full + 8u * n_stage, n_phase);
                uint4 nh = hdr, na = sa, nb = sb, nc = sc;
                // schedule entries are published 32 rows at a time, ahead of the first copy of those rows
                const bool early_info = row_end && !last_row && ((ri + 1) & 31) != 0;
                const uint4* qn = (const uint4*)s_rowq[(ri + 1) & (ROWQ - 1)];
                if (early_info) { nh = qn[0]; na = qn[1]; nb = qn[2]; nc = qn[3]; }
                // ---- the other kx taps of the tile (row-shifted reads of the same box)
                {
                    uint64_t adesc = adesc_cur + kx_bytes, bdesc = bdesc_cur + wtile_kx;
                    for (int kxi = 1; kxi < n_kx; ++kxi, adesc += kx_bytes, bdesc += wtile_kx) {
                        if (issuer && hdr.z > 0) {
                            umma_tile<DT, KSTEPS>(sa.x, adesc, bdesc + (uint64_t)sa.y, sa.z);
                            if (hdr.z > 1) {
                                umma_tile<DT, KSTEPS>(sa.w, adesc, bdesc + (uint64_t)sb.x, sb.y);
                                if (hdr.z > 2) umma_tile<DT, KSTEPS>(sb.z, adesc, bdesc + (uint64_t)sb.w, sc.x);
                                if (hdr.z > 3) umma_tile<DT, KSTEPS>(sc.y, adesc, bdesc + (uint64_t)sc.z, sc.w);
                            }
                        }
                    }
                }
                if (issuer) {
                    umma_commit(bar_empty + 8u * stage);
                    if (row_end) {
                        // the accumulator this input row completed; on the block's last row also everything still open
                        // (to be parked in the ring, or emitted if only bottom padding was missing)
                        if (hdr.w) umma_commit(hdr.w);
                        if (last_row)
                            for (int orel = c_sched_rel; orel < c_n_orows; ++orel) umma_commit(bar_ready + 8u * (uint32_t)(orel % nslot));
                    }
                }
                if (!next_ok && !mbar_wait(bar_full + 8u * n_stage, n_phase, abort_flag)) { ok = false; break; }
                stage = n_stage; phase = n_phase; adesc_cur = adesc_nx; bdesc_cur = bdesc_nx; kb = n_kbi;
                if (row_end) {
                    if (last_row) break;
                    if (!early_info) { nh = qn[0]; na = qn[1]; nb = qn[2]; nc = qn[3]; }   // (published with the tile just waited for)
                    hdr = nh; sa = na; sb = nb; sc = nc;
                    st = 0; ++ri;
                    tc_fence_after();                            // the next row may start on a slot the epilogue has just cleared
                } else {
                    ++st;
                }
            }
        }
        __syncwarp();
    } else {
        // ------------------------------ epilogue: row finalisation -----------------------------
        // Groups of four warps (one warp per TMEM lane quarter) take the output rows in turn.
        // An emitted row is first laid out in the group's shared-memory tile (each thread writes its
        // own tile row, swizzled), then one thread hands the tile to a TMA store, which writes whole
        // lines and clips whatever lies outside the map.
        const int q = warp & 3;                          // TMEM lane quarter this warp may read
        const int grp = (warp - 2) >> 2;
        const bool leader = (warp - 2) == grp * 4 && lane == 0;
        const int m = q * 32 + lane;                     // row of the tile = TMEM lane
        const int bs = m / a.BXP, bx = m - bs * a.BXP;
        const int s = s0 + bs, x = x0 + bx;
        const bool in_tile = (bs < a.BS) && (bx < a.BX);
        const bool valid = in_tile && (s < a.S) && (x < a.Wout);
        const bool wide = (a.Ntile & 31) == 0;
        const TS* bias = a.bias ? (const TS*)a.bias + n0 : nullptr;
        const long long row_elems = (long long)a.Wout * a.Cout;
        TS* ring_pos = (TS*)a.ring + (long long)s * row_elems + (long long)x * a.Cout + n0;   // + ring slot * S * row_elems
        const long long ring_slot_stride = (long long)a.S * row_elems;
        const uint32_t tlane = tmem_base + ((uint32_t)(q * 32) << 16);
        const int md = bs * a.BX + bx;                   // row of the dense output tile
        StageSink sink;
        sink.pwb_log2 = 31u - (uint32_t)__clz(a.out_pwb);
        sink.panel_bytes = (uint32_t)a.out_stage_rows * (uint32_t)a.out_pwb;
        sink.row_base = sOut + (uint32_t)(grp * a.out_bufs) * a.out_stage_bytes + (uint32_t)md * a.out_pwb;
        sink.phase = a.out_pwb == 128 ? (uint32_t)(md & 7) : (a.out_pwb == 64 ? (uint32_t)((md >> 1) & 3)
                   : (a.out_pwb == 32 ? (uint32_t)((md >> 2) & 1) : 0u));
        uint32_t stg = sOut + (uint32_t)(grp * a.out_bufs) * a.out_stage_bytes;     // the staging tile in use
        uint32_t buf_step = a.out_bufs > 1 ? (uint32_t)a.out_stage_bytes : 0u;      // to the group's other tile (sign flips per store)
        const int panel_cols = a.out_pwb / a.out_esize;
        PoolCtx pc;
        pc.on = a.pool; pc.second = 0; pc.from_state = 0; pc.to_state = 0; pc.drop = 0;
        pc.writer = in_tile && !(bx & 1);
        const int mdp = bs * (a.BX >> 1) + (bx >> 1);   // row of the pooled tile
        pc.sink = sink;
        pc.sink.row_base = stg + (uint32_t)mdp * a.out_pwb;
        pc.sink.phase = a.out_pwb == 128 ? (uint32_t)(mdp & 7) : (a.out_pwb == 64 ? (uint32_t)((mdp >> 1) & 3)
                      : (a.out_pwb == 32 ? (uint32_t)((mdp >> 2) & 1) : 0u));
        const int wp = a.Wout >> 1;
        const bool state_ok = valid && (x >> 1) < wp;
        pc.state = (unsigned char*)a.pool_state + (((long long)s * wp + (x >> 1)) * a.Cout + n0) * a.out_esize;
        bool ok = true;
        // Every ring slot in tensor memory starts from what its row has so far (all MMAs accumulate): zero, or, for a
        // row begun by an earlier block, the partial sums that block left in the ring in global memory.  Taking those
        // up here, while weights and the first rows are still on their way, keeps the ring's read latency out of the
        // path between the last MMA and the emission; the three groups share the slots.
        {
            const long long carry_off0 = (const TS*)a.ring_in - (const TS*)a.ring;
            int rs = (a.ring_slot0 + c_oa) % a.ring_rows;
            for (int slot = 0; slot < (c_n_orows < a.nslot ? c_n_orows : a.nslot); ++slot) {
                const int rslot = rs;
                if (++rs == a.ring_rows) rs = 0;
                if (slot % MAX_GROUPS != grp) continue;
                // (carried_row is the same in all threads: the tensor-memory stores below are warp-wide instructions and
                // every branch around them must be uniform; what differs per thread is only whether it has values to load)
                const bool carried_row = c_r0_positive && (slot * a.stride - c_base_ty < 0);
                bool carried = carried_row && valid;
                const TS* rp = ring_pos + (long long)rslot * ring_slot_stride + carry_off0;
#ifdef IDF_BOUNDS
                if (carried && !IDF_OK_AT(a.status, (rp - carry_off0 - (const TS*)a.ring) + a.Ntile - 1, a.ring_elems)) carried = false;
#endif
                for (int c = 0; c < a.Ntile; c += 16) {
                    uint32_t v[16];
                    if (carried) {
                        uint32_t lo[8], hi[8];
                        ld_global_v8(rp + c, lo);
                        ld_global_v8(rp + c + 8, hi);
#pragma unroll
                        for (int j = 0; j < 8; ++j) { v[j] = lo[j]; v[8 + j] = hi[j]; }
                    } else {
#pragma unroll
                        for (int j = 0; j < 16; ++j) v[j] = 0u;
                    }
                    __syncwarp();
                    tmem_st16(tlane + (uint32_t)(slot * a.Ntile + c), v);
                }
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_free + 8u * slot);   // one arrival per warp
            }
        }
        // Rows left open by this block go back to the ring in global memory; those that meet in one ring slot stay in
        // one group, in order.  (Rows begun by an earlier block were read above, before the first MMA, so nothing
        // reads a ring slot any more once rows are written.)  The other rows go round the groups.
        const int n_cin = c_r0_positive ? (c_base_ty + a.stride - 1) / a.stride : 0;
        // Per-row bookkeeping is kept with small counters that step from row to row (a division or a 64-bit
        // operation per row and thread costs more than the row's arithmetic): TMEM slot and barrier parity of the row,
        // its ring slot in global memory, the parity of its absolute index, the group whose turn it is.
        const int G = a.out_groups;
        int slot_c = 0;                                       // orel mod nslot
        uint32_t par_c = 0;                                   // (orel div nslot) & 1
        int turn = 0;                                         // orel mod G
        int absp = (a.o_begin_par + c_oa) & 1;                // parity of the row's absolute index
        int pair_turn = (a.o_begin_half_mod + ((a.o_begin_par + c_oa) >> 1)) % G;   // (absolute index div 2) mod G
        int rslot_c = (a.ring_slot0 + c_oa) % a.ring_rows;    // absolute index mod ring_rows
        int rslot_g = rslot_c % G;                            // ... mod G: the group that owns the ring slot
        for (int orel = 0; orel < c_n_orows && ok && grp < G; ++orel) {
            int owner;
            if (!a.pool) {
                // (rows that meet in one ring slot stay in one group, which takes them in order)
                owner = (orel < n_cin || orel >= c_done_rel) ? rslot_g : turn;
            } else {
                // both rows of a pooling pair go to one group; pairs touching the global ring or the pool layer's state
                // (first < 0: the pair's first row came with an earlier launch) go to group 0
                const int first = orel - absp;
                owner = (first < 0 || first < n_cin || first + 1 >= c_done_rel) ? 0 : pair_turn;
                // a launch that emits at most one row has no pair to keep together and one row at most that touches the
                // pool layer's state: its rows spread over the groups by ring slot as above
                if (c_done_rel <= 1) owner = rslot_g;
            }
            const int slot = slot_c, rslot = rslot_c, row_odd = absp;
            const uint32_t par = par_c;
            // the counters move on to the next row
            if (++slot_c == a.nslot) { slot_c = 0; par_c ^= 1u; }
            if (++turn == G) turn = 0;
            if (++rslot_c == a.ring_rows) rslot_c = 0;
            if (++rslot_g == G) rslot_g = 0;
            if (rslot_c == 0) rslot_g = 0;
            if (absp && ++pair_turn == G) pair_turn = 0;
            absp ^= 1;
            if (owner != grp) continue;
            const bool emit = orel < c_done_rel;
            // one thread of the group polls the barrier; the named barrier below releases the other warps.
            // The tile must have been drained by the group's previous store before anyone writes it again: that
            // wait comes first, it overlaps the wait for the row.
            int got = 1;
            if (leader) {
                // (with two tiles the latest store may still be draining: it reads the other one)
                if (emit) {
                    if (a.out_bufs > 1) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                    else asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                }
                got = mbar_wait_relaxed(bar_ready + 8u * slot, par, abort_flag) ? 1 : 0;
            }
            // (the barrier also makes the whole group leave together if any of its waits ran out)
            if (!named_bar_and(1 + grp, 128, got != 0)) { ok = false; break; }
            tc_fence_after();
            const bool pool_emit = a.pool && emit;
            if (pool_emit) {
                pc.second = row_odd;
                pc.from_state = pc.second && orel == 0;
                const bool trailing = !pc.second && orel == c_done_rel - 1 && c_oa + c_done_rel == a.done_rel;   // the block's last emitted row
                pc.to_state = trailing && a.pool_keep;
                pc.drop = trailing && !a.pool_keep;
            }
            TS* rp = ring_pos + (long long)rslot * ring_slot_stride;
            const uint32_t trow = tlane + (uint32_t)(slot * a.Ntile);
            bool fine = true;           // range-checked build: false skips this row's accesses (the barriers still run)
#ifdef IDF_BOUNDS
            {
                fine = IDF_OK_AT(a.status, slot * a.Ntile + a.Ntile - 1, a.tmem_cols);
                if (valid && !emit) fine = fine && IDF_OK_AT(a.status, (rp - (TS*)a.ring) + a.Ntile - 1, a.ring_elems);
                if (pool_emit && state_ok && (pc.from_state || pc.to_state))
                    fine = fine && IDF_OK_AT(a.status, (pc.state - (unsigned char*)a.pool_state) + (long long)a.Ntile * a.out_esize - 1, a.pool_state_bytes);
                // (a launch that emits pooled rows stages them in the half-size tile; the full-size addresses are not used then)
                const uint32_t stage_row = a.pool ? pc.sink.row_base : sink.row_base;
                if (emit && (a.pool ? pc.writer != 0 : in_tile))
                    fine = fine && IDF_OK_AT(a.status, (stage_row - smem_u32(smem_raw)) + (uint32_t)(a.out_panels - 1) * sink.panel_bytes + a.out_pwb - 1,
                                             bars - smem_u32(smem_raw));
                fine = __all_sync(0xffffffffu, fine) != 0;     // (the tensor-memory loads below are warp-wide instructions)
            }
#endif
            {
                if (wide) {
                    for (int c = 0; c < a.Ntile; c += 32) {
                        uint32_t v[32];
                        if (!fine) continue;
                        __syncwarp();                         // (the finalisation of the previous chunk is per thread)
                        tmem_ld<32>(trow + c, v);
                        tmem_ld_wait();
                        tmem_st_zero<32>(trow + c);           // the slot's next row starts from zero
                        if (pool_emit || (emit ? in_tile : valid))
                            finalise_chunk<DT, 32, TS>(v, emit, rp + c, bias ? bias + c : nullptr, sink,
                                                       (uint32_t)(c * a.out_esize), a.out_elem, a.relu, a.shift, pc, state_ok);
                    }
                } else {
                    for (int c = 0; c < a.Ntile; c += 16) {
                        uint32_t v[16];
                        if (!fine) continue;
                        __syncwarp();
                        tmem_ld<16>(trow + c, v);
                        tmem_ld_wait();
                        tmem_st_zero<16>(trow + c);
                        if (pool_emit || (emit ? in_tile : valid))
                            finalise_chunk<DT, 16, TS>(v, emit, rp + c, bias ? bias + c : nullptr, sink,
                                                       (uint32_t)(c * a.out_esize), a.out_elem, a.relu, a.shift, pc, state_ok);
                    }
                }
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_free + 8u * slot);   // one arrival per warp
            }
            if (emit && (!a.pool || pc.second)) {      // with pooling only the second row of a pair sends a (pooled) row out
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                named_bar_sync(1 + grp, 128);
                if (leader) {
                    const int orow = a.pool ? a.pool_row_first + ((a.o_begin_par + c_oa + orel) >> 1) : a.out_row_first + c_oa + orel;
                    const int xc = a.pool ? (x0 >> 1) : x0;
                    for (int pnl = 0; pnl < a.out_panels; ++pnl) {
                        if (a.out_row_dim == 3)
                            tma_store_4d(&tmO, stg + (uint32_t)pnl * sink.panel_bytes, n0 + pnl * panel_cols, xc, s0, orow);
                        else
                            tma_store_4d(&tmO, stg + (uint32_t)pnl * sink.panel_bytes, n0 + pnl * panel_cols, xc, orow, s0);
                    }
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
                // the group's next row is laid out in its other tile
                stg += buf_step; sink.row_base += buf_step; pc.sink.row_base += buf_step;
                buf_step = 0u - buf_step;
            }
        }
        if (leader) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    }

    tc_fence_before();
    __syncthreads();
    if (s_abort) {
        if (threadIdx.x == 0) {
            // let this CTA's own copies land before its shared memory is given back (bounded)
            for (uint32_t i = 0; i < 4096 && !mbar_try_wait(bar_w, 0); ++i) __nanosleep(64);
            const int issued = s_issued;
            for (int st = 0; st < a.nstage; ++st) {
                int last = -1;
                for (int t = st; t < issued; t += a.nstage) last = t;
                if (last < 0) continue;
                const uint32_t par = (uint32_t)((last / a.nstage) & 1);
                for (uint32_t i = 0; i < 4096 && !mbar_try_wait(bar_full + 8u * st, par); ++i) __nanosleep(64);
            }
            atomicExch(a.status, 1u);
        }
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)a.tmem_cols) : "memory");
    }
}

// ------------------------------------------------------------------------------------------------
// Thin layers: the whole receptive field of an output position (Kh*Kw*Cin values) fits ONE swizzled
// shared-memory row of 32, 64 or 128 bytes - the first layers of nets that start from few channels.
// Such a layer is a plain contraction over that row (Eq. 4 for all taps of a unit at once), with so
// little arithmetic per output that the kernel is bound by the bytes it writes; what matters is that
// every role pays its fixed cost per BATCH of rows, not per row:
//   warps 0-3   build the im2col rows of R output rows of one 128-position tile in shared memory,
//               straight from the layer's input rows (zero where a tap falls on padding);
//   warp 4      issues R x ksteps tcgen05.mma (M = 128, N = Cout) into one of two accumulator sets;
//   warps 5-12  two epilogue groups taking work items in turn: tcgen05.ld, f(c + b), rounding or
//               requantisation, swizzled staging tile, one TMA store per row.
// The kernel handles only rows that this block's input rows determine completely (no ring row is read
// or written: rows begun by an earlier block or left open by this one go through the CUDA-core kernel),
// so rows are independent work items: item i = (row group, position tile), dealt round robin to a
// grid of one CTA per SM.
// ------------------------------------------------------------------------------------------------
constexpr int THIN_THREADS = 13 * 32;
constexpr int THIN_MAX_K = 128;              // bytes of an im2col row
constexpr int THIN_RAW_PER_THREAD = 16;      // input values a gather thread copies per work item (128 threads)
constexpr int THIN_RAW_BYTES = 128 * THIN_RAW_PER_THREAD * 2;

struct ThinArgs {
    const void* in;              // input rows of the block: [n_in][S][Win][Cin] in the activation type
    const void* bias;
    unsigned int* status;
    long long r0;                // absolute index of the first input row of the block
    long long o_first;           // absolute index of the first output row this launch computes
    int n_in, n_out;             // input rows in the block, output rows to compute: o_first + [0, n_out)
    int S, Win, Wout, Cin, Cout, Kh, Kw, stride, pad, stride_x, pad_x, relu, shift, out_elem;
    int kelems, swb, ksteps, BX, BS, n_xt, n_mt, R, nstage, tmem_cols;
    int out_esize, out_pwb, out_panels, out_tile_bytes;
    int out_row_dim, out_row_first;          // position of the row coordinate in the output tensor map; map row of o_first
};

template <int DT>
__global__ void __launch_bounds__(THIN_THREADS, 1)
conv_thin_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmO, const ThinArgs a)
{
    typedef typename Acc<DT>::S TS;
    constexpr int ES = DT == 1 ? 2 : 1;              // bytes of an activation
    extern __shared__ unsigned char smem_raw[];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    __shared__ short s_tab[THIN_MAX_K][2];            // value k of an im2col row: where it comes from, where it goes

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t row_tile_bytes = 128u * (uint32_t)a.swb;               // one im2col tile (128 positions)
    const uint32_t stage_bytes = (uint32_t)a.R * row_tile_bytes;
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sW = base;                                              // [Cout][swb]
    const uint32_t sA = (sW + (uint32_t)a.Cout * a.swb + 1023u) & ~1023u;
    const uint32_t sOut = sA + (uint32_t)a.nstage * stage_bytes;           // [group][buffer][R] staging tiles
    const uint32_t bars = sOut + 2u * 2u * (uint32_t)a.R * a.out_tile_bytes;
    const uint32_t bar_full = bars, bar_empty = bar_full + 8u * a.nstage, bar_w = bar_empty + 8u * a.nstage;
    const uint32_t bar_accfull = bar_w + 8u, bar_accfree = bar_accfull + 16u;

    if (threadIdx.x == 0) {
        s_abort = 0;
        for (int i = 0; i < a.nstage; ++i) { mbar_init(bar_full + 8u * i, 4); mbar_init(bar_empty + 8u * i, 1); }
        mbar_init(bar_w, 1);
        for (int i = 0; i < 2; ++i) { mbar_init(bar_accfull + 8u * i, 1); mbar_init(bar_accfree + 8u * i, 4); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_expect_tx(bar_w, (uint32_t)a.Cout * a.swb);                   // the parameters do not depend on earlier kernels
        tma_load_2d(sW, &tmW, bar_w, 0, 0);
    }
    for (int k = threadIdx.x; k < a.kelems; k += blockDim.x) {
        // value k of an im2col row: tap (ky, kx), channel ci -> its offset (in elements) from the position's corner in the
        // staging area [row][stream][position][channel], and its byte position in the row
        const int ci = k % a.Cin, t = k / a.Cin, ky = t / a.Kw, kx = t % a.Kw;
        const int XP = (a.BX - 1) * a.stride_x + a.Kw;
        s_tab[k][0] = (short)((ky * a.BS * XP + kx) * a.Cin + ci);
        s_tab[k][1] = (short)(k * ES);
    }
    if (warp == 4) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)), "r"((uint32_t)a.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // the zero padding behind the kelems values of every im2col row is written once
    for (uint32_t i = threadIdx.x; i < (uint32_t)a.nstage * stage_bytes / 16u; i += blockDim.x)
        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(sA + 16u * i), "r"(0u) : "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const uint32_t tmem_base = s_tmem_base;
    volatile int* abort_flag = &s_abort;
    const int n_groups = (a.n_out + a.R - 1) / a.R;
    const long long n_items = (long long)n_groups * a.n_mt;

    if (warp < 4) {
        // ------------------------------ im2col rows ---------------------------------------------
        // Two steps per work item.  (1) The 128 threads copy the input rows the item's R output rows reach - for the
        // tile's streams and positions, with the kx halo, zero where a tap falls on padding - into a small staging
        // area [row][stream][position][channel]: consecutive threads read consecutive elements, and the copy of the
        // NEXT item is already in flight (in registers) while the current one is worked on.  (2) Thread m builds the
        // im2col row of position m for each of the R output rows from that area: element k of a row sits at a fixed
        // offset from the position's corner (table s_tab), so a value costs two additions, a load and a store.
        const int m = warp * 32 + lane;                       // row of the tile = position
        const int bs = m / a.BX, bx = m - bs * a.BX;
        const bool in_tile = bs < a.BS;
        const uint32_t sw_phase = a.swb == 128 ? (uint32_t)(m & 7) : (a.swb == 64 ? (uint32_t)((m >> 1) & 3) : (uint32_t)((m >> 2) & 1));
        const unsigned char* in = (const unsigned char*)a.in;
        const int XP = (a.BX - 1) * a.stride_x + a.Kw;        // positions of a stream in the staging area
        const int run_s = XP * a.Cin, run_r = a.BS * run_s;   // elements per (row, stream) and per row
        const int n_r = (a.R - 1) * a.stride + a.Kh;
        const int raw_elems = n_r * run_r;
        const uint32_t m_r = 0xFFFFFFFFu / (uint32_t)run_r + 1u, m_s = 0xFFFFFFFFu / (uint32_t)run_s + 1u,
                       m_c = 0xFFFFFFFFu / (uint32_t)a.Cin + 1u;        // q = umulhi(n, m): n / d for the small n here
        const uint32_t corner = (uint32_t)((bs * XP + bx * a.stride_x) * a.Cin) * ES;
        const uint32_t sRaw = bars + 256u;                    // behind the barriers
        unsigned short held[THIN_RAW_PER_THREAD];             // the next item's share of the staging area
        auto fetch = [&](long long item) {
            const int g = (int)(item / a.n_mt), mt = (int)(item - (long long)g * a.n_mt);
            const int xt = mt % a.n_xt, st = mt / a.n_xt;
            const long long r_first = (a.o_first + (long long)g * a.R) * a.stride - a.pad - a.r0;     // row of the block
            const int x_first = xt * a.BX * a.stride_x - a.pad_x;
#pragma unroll
            for (int i = 0; i < THIN_RAW_PER_THREAD; ++i) {
                const uint32_t e = (uint32_t)(m + 128 * i);
                unsigned short v = 0;
                if (e < (uint32_t)raw_elems) {
                    const uint32_t rr = __umulhi(e, m_r), e1 = e - rr * (uint32_t)run_r;
                    const uint32_t ss = __umulhi(e1, m_s), e2 = e1 - ss * (uint32_t)run_s;
                    const uint32_t xp = __umulhi(e2, m_c), ci = e2 - xp * (uint32_t)a.Cin;
                    const long long r = r_first + rr;
                    const int sg = st * a.BS + (int)ss, ix = x_first + (int)xp;
                    if (r >= 0 && r < a.n_in && sg < a.S && ix >= 0 && ix < a.Win) {
                        const long long at = ((r * a.S + sg) * a.Win + ix) * (long long)a.Cin + ci;
                        if (IDF_OK_AT(a.status, at, (long long)a.n_in * a.S * a.Win * a.Cin))
                            v = ES == 2 ? *(const unsigned short*)(in + 2 * at) : (unsigned short)in[at];
                    }
                }
                held[i] = v;
            }
        };
        int it = 0;
        bool ok = true;
        if ((long long)blockIdx.x < n_items) fetch(blockIdx.x);
        for (long long item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++it) {
            const int stage = it % a.nstage;
            const uint32_t ph = (uint32_t)((it / a.nstage) & 1);
            const int g = (int)(item / a.n_mt), mt = (int)(item - (long long)g * a.n_mt);
            const int xt = mt % a.n_xt, st = mt / a.n_xt;
            const bool valid = in_tile && st * a.BS + bs < a.S && xt * a.BX + bx < a.Wout;
#pragma unroll
            for (int i = 0; i < THIN_RAW_PER_THREAD; ++i) {
                const uint32_t e = (uint32_t)(m + 128 * i);
                if (e < (uint32_t)raw_elems) {
                    if (ES == 2) asm volatile("st.shared.u16 [%0], %1;" ::"r"(sRaw + 2u * e), "h"(held[i]) : "memory");
                    else asm volatile("st.shared.u8 [%0], %1;" ::"r"(sRaw + e), "r"((uint32_t)held[i]) : "memory");
                }
            }
            named_bar_sync(3, 128);                               // the staging area is complete
            if (item + gridDim.x < n_items) fetch(item + gridDim.x);
            int got = 1;
            if (lane == 0) got = mbar_wait_relaxed(bar_empty + 8u * stage, ph ^ 1u, abort_flag) ? 1 : 0;
            got = __shfl_sync(0xffffffffu, got, 0);
            if (got && valid) {
                for (int j = 0; j < a.R; ++j) {
                    if (g * a.R + j >= a.n_out) break;
                    const uint32_t row_addr = sA + (uint32_t)stage * stage_bytes + (uint32_t)j * row_tile_bytes + (uint32_t)m * a.swb;
                    const uint32_t from = sRaw + corner + (uint32_t)(j * a.stride * run_r) * ES;
                    // eight values at a time: the loads of a batch are all issued before the first store needs its value
                    for (int k0 = 0; k0 < a.kelems; k0 += 8) {
                        uint32_t v[8], dst[8];
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            const int k = k0 + u < a.kelems ? k0 + u : a.kelems - 1;      // (the tail repeats the last value: same bytes, same place)
                            const uint32_t off = (uint32_t)(unsigned short)s_tab[k][0] * ES, to = (uint32_t)(unsigned short)s_tab[k][1];
                            dst[u] = row_addr + ((((to >> 4) ^ sw_phase)) << 4) + (to & 15u);
                            if (ES == 2) { unsigned short h; asm volatile("ld.shared.u16 %0, [%1];" : "=h"(h) : "r"(from + off)); v[u] = h; }
                            else asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v[u]) : "r"(from + off));
                        }
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            if (ES == 2) asm volatile("st.shared.u16 [%0], %1;" ::"r"(dst[u]), "h"((unsigned short)v[u]));
                            else asm volatile("st.shared.u8 [%0], %1;" ::"r"(dst[u]), "r"(v[u]));
                        }
                    }
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // the tensor core reads these rows through the async proxy
            // nobody reads the staging area any more; and if any warp's wait ran out, all four leave together
            if (!named_bar_and(3, 128, got != 0)) { ok = false; break; }
            if (lane == 0) mbar_arrive(bar_full + 8u * stage);
        }
    } else if (warp == 4) {
        // ------------------------------ MMA issuer ---------------------------------------------
        const uint64_t desc_hi = make_smem_desc(0, a.swb);
        const uint32_t idesc = (DT == 1 ? ((1u << 4) | (1u << 7) | (1u << 10)) : ((2u << 4) | (1u << 7) | (1u << 10))) |
                               ((128u >> 4) << 24) | ((uint32_t)(a.Cout >> 3) << 17);
        const uint64_t bdesc = desc_hi | (uint64_t)((sW & 0x3FFFFu) >> 4);
        bool ok = mbar_wait(bar_w, 0, abort_flag);
        const bool issuer = elect_one();
        int it = 0;
        for (long long item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++it) {
            const int stage = it % a.nstage;
            const uint32_t ph = (uint32_t)((it / a.nstage) & 1);
            const int acc = it & 1;
            const uint32_t aph = (uint32_t)((it >> 1) & 1);
            if (!mbar_wait(bar_accfree + 8u * acc, aph ^ 1u, abort_flag)) { ok = false; break; }   // the epilogue has read this accumulator set
            if (!mbar_wait(bar_full + 8u * stage, ph, abort_flag)) { ok = false; break; }
            tc_fence_after();
            if (issuer) {
                for (int j = 0; j < a.R; ++j) {
                    const uint64_t adesc = desc_hi | (uint64_t)(((sA + (uint32_t)stage * stage_bytes + (uint32_t)j * row_tile_bytes) & 0x3FFFFu) >> 4);
                    const uint32_t d = tmem_base + (uint32_t)((acc * a.R + j) * a.Cout);
                    for (int k = 0; k < a.ksteps; ++k) umma<DT>(d, adesc + 2u * k, bdesc + 2u * k, idesc, k > 0 ? 1u : 0u);
                }
                umma_commit(bar_empty + 8u * stage);
                umma_commit(bar_accfull + 8u * acc);
            }
            __syncwarp();
        }
    } else {
        // ------------------------------ epilogue -----------------------------------------------
        const int q = warp & 3;                           // TMEM lane quarter this warp may read
        const int grp = (warp - 5) >> 2;
        const bool leader = (warp - 5) == grp * 4 && lane == 0;
        const int m = q * 32 + lane;
        const int bs = m / a.BX, bx = m - bs * a.BX;
        const bool in_tile = bs < a.BS;
        const TS* bias = (const TS*)a.bias;
        const uint32_t tlane = tmem_base + ((uint32_t)(q * 32) << 16);
        StageSink sink;
        sink.pwb_log2 = 31u - (uint32_t)__clz(a.out_pwb);
        sink.panel_bytes = 128u * (uint32_t)a.out_pwb;
        const int md = bs * a.BX + bx;
        sink.phase = a.out_pwb == 128 ? (uint32_t)(md & 7) : (a.out_pwb == 64 ? (uint32_t)((md >> 1) & 3)
                   : (a.out_pwb == 32 ? (uint32_t)((md >> 2) & 1) : 0u));
        PoolCtx pc;
        pc.on = 0; pc.writer = 0; pc.second = 0; pc.from_state = 0; pc.to_state = 0; pc.drop = 0; pc.sink = sink; pc.state = nullptr;
        const int panel_cols = a.out_pwb / a.out_esize;
        const uint32_t grp_base = sOut + (uint32_t)grp * 2u * (uint32_t)a.R * a.out_tile_bytes;
        int buf = 0;
        bool ok = true;
        int it = 0;
        for (long long item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++it) {
            if ((it & 1) != grp) continue;
            const uint32_t aph = (uint32_t)((it >> 1) & 1);
            const int g = (int)(item / a.n_mt), mt = (int)(item - (long long)g * a.n_mt);
            const int xt = mt % a.n_xt, st = mt / a.n_xt;
            int got = 1;
            if (leader) {
                asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");     // the tiles of the store before last are free again
                got = mbar_wait_relaxed(bar_accfull + 8u * grp, aph, abort_flag) ? 1 : 0;
            }
            if (!named_bar_and(1 + grp, 128, got != 0)) { ok = false; break; }
            tc_fence_after();
            const uint32_t tiles = grp_base + (uint32_t)buf * (uint32_t)a.R * a.out_tile_bytes;
            for (int j = 0; j < a.R; ++j) {
                if (g * a.R + j >= a.n_out) break;
                sink.row_base = tiles + (uint32_t)j * a.out_tile_bytes + (uint32_t)md * a.out_pwb;
                const bool fine = IDF_OK_AT(a.status, (sink.row_base - smem_u32(smem_raw)) + (uint32_t)(a.out_panels - 1) * sink.panel_bytes + a.out_pwb - 1,
                                            bars - smem_u32(smem_raw));
                const uint32_t trow = tlane + (uint32_t)((grp * a.R + j) * a.Cout);
                if ((a.Cout & 31) == 0) {
                    for (int c = 0; c < a.Cout; c += 32) {
                        uint32_t v[32];
                        __syncwarp();
                        tmem_ld<32>(trow + c, v);
                        tmem_ld_wait();
                        if (in_tile && fine)
                            finalise_chunk<DT, 32, TS>(v, true, (TS*)nullptr, bias ? bias + c : nullptr, sink, (uint32_t)(c * a.out_esize),
                                                       a.out_elem, a.relu, a.shift, pc, false);
                    }
                } else {
                    for (int c = 0; c < a.Cout; c += 16) {
                        uint32_t v[16];
                        __syncwarp();
                        tmem_ld<16>(trow + c, v);
                        tmem_ld_wait();
                        if (in_tile && fine)
                            finalise_chunk<DT, 16, TS>(v, true, (TS*)nullptr, bias ? bias + c : nullptr, sink, (uint32_t)(c * a.out_esize),
                                                       a.out_elem, a.relu, a.shift, pc, false);
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_accfree + 8u * grp);           // one arrival per warp: the accumulator set may be overwritten
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            named_bar_sync(1 + grp, 128);
            if (leader) {
                for (int j = 0; j < a.R; ++j) {
                    const int orel = g * a.R + j;
                    if (orel >= a.n_out) break;
                    const uint32_t tile = tiles + (uint32_t)j * a.out_tile_bytes;
                    for (int pnl = 0; pnl < a.out_panels; ++pnl) {
                        if (a.out_row_dim == 3)
                            tma_store_4d(&tmO, tile + (uint32_t)pnl * sink.panel_bytes, pnl * panel_cols, xt * a.BX, st * a.BS, a.out_row_first + orel);
                        else
                            tma_store_4d(&tmO, tile + (uint32_t)pnl * sink.panel_bytes, pnl * panel_cols, xt * a.BX, a.out_row_first + orel, st * a.BS);
                    }
                }
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            }
            buf ^= 1;
        }
        if (leader) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    }

    tc_fence_before();
    __syncthreads();
    if (s_abort) {
        if (threadIdx.x == 0) {
            for (uint32_t i = 0; i < 4096 && !mbar_try_wait(bar_w, 0); ++i) __nanosleep(64);   // the CTA's own copy must land first
            atomicOr(a.status, 1u);
        }
        __syncthreads();
    }
    if (warp == 4) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)a.tmem_cols) : "memory");
    }
}

// ---- host side ---------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    });
    return fn;
}

CUtensorMapSwizzle swizzle_of(int swb)
{
    return swb == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : (swb == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
}

}  // namespace

bool tc_make_plan(int dtype, int S, int Win, int Wout, int Cin, int Cout, int Kh, int Kw, int stride_x, int ring_rows,
                  int out_esize, int pooled, TcPlan* p)
{
    *p = TcPlan{};
    if (dtype != 1 && dtype != 2) return false;
    const int esize = dtype == 1 ? 2 : 1;
    const int row_bytes = Cin * esize;
    if (stride_x < 1 || stride_x > 8) return false;     // (a tensor map's traversal stride is at most 8)
    if (!(row_bytes == 32 || row_bytes == 64 || (row_bytes >= 128 && row_bytes % 128 == 0))) return false;
    if (Kh * Kw > 32 || Cout % 16 != 0) return false;
    p->swb = row_bytes >= 128 ? 128 : row_bytes;
    p->KB = p->swb / esize;
    p->n_kb = Cin / p->KB;
    // With 128-byte rows one box per (input row, K block) carries the Kw-1 halo positions of every
    // stream in the tile and the kx taps read it at row offsets; narrower rows take one box per kx.
    p->shift_mode = (p->swb == 128 && Kw > 1) ? 1 : 0;
    const int halo = p->shift_mode ? Kw - 1 : 0;
    if (Wout >= 128) {
        p->n_xt = (Wout + 127) / 128;
        p->BX = (Wout + p->n_xt - 1) / p->n_xt;
        p->BS = 1;
    } else {
        p->n_xt = 1;
        p->BX = Wout;
        p->BS = 1 + (128 - Wout) / (Wout + halo);     // (BS-1)*(BX+halo) + BX <= 128 output lanes
        if (p->BS > S) p->BS = S;
    }
    p->BXP = p->BX + halo;
    // An x-strided layer needs one box per kx tap (the tap's positions x' * stride + kx - pad are then one strided
    // walk of the input row, which the tensor map does); the haloed tile of the row-shift mode has no such form.
    if (stride_x != 1 && (p->shift_mode || Kw == 1)) return false;
    p->sx = stride_x;
    if (p->BXP * stride_x > 256) return false;          // the box is given in input positions
    // A stage holds exactly the TMA box (BS streams x BXP positions).  The MMAs read 128 rows from row kx on,
    // so for the last positions they run past the box into whatever follows in shared memory: those are
    // lanes outside the tile, whose accumulators nobody reads.
    // kx taps that cannot share a haloed box (rows of 32 or 64 bytes, x-strided layers) get a box each, side by side in
    // the stage, under one barrier
    const int n_box = (!p->shift_mode && Kw > 1) ? Kw : 1;
    const size_t box_pitch = ((size_t)p->BS * p->BXP * p->swb + 1023) / 1024 * 1024;
    const size_t a_stage = (size_t)n_box * box_pitch;
    p->a_stage_bytes = (int)a_stage;
    p->n_box = n_box;
    p->a_box_pitch = (int)box_pitch;
    p->n_mt = p->n_xt * ((S + p->BS - 1) / p->BS);
    const int taps = Kh * Kw;
    // a launch that emits pooled rows stages half a tile of positions
    const int stage_rows = pooled ? 64 : 128;
    int best = 0, best_units = -1;
    const bool wide_for_1d = true;
    for (int nt = 256; nt >= 16; nt >>= 1) {
        if (Cout % nt) continue;
        if ((ring_rows + 1) * nt > 512) continue;
        if ((ring_rows + 256 / nt - 1) / (256 / nt) + 1 > 4) continue;   // at most 4 MMA segments per input row
        const size_t wb = (size_t)taps * p->n_kb * nt * p->swb;
        if (wb + 3 * a_stage + (size_t)stage_rows * nt * out_esize + 10240 > SMEM_LIMIT) continue;   // one staging tile at least
        const int units = p->n_mt * (Cout / nt);
        if (units >= 120) { best = nt; break; }          // enough CTAs for the 148 SMs: take the widest such tile
        // 1D nets come in long blocks of rows, which row chunks spread over the SMs: there the widest tile that fits
        // wins, because every channel slice fetches the Δ-rows again (audio1d's 128-channel layers with 16-channel
        // tiles moved 4.2 GB per layer through the L2)
        if (Win == 1 && wide_for_1d) { best = nt; break; }
        if (units > best_units) { best_units = units; best = nt; }
    }
    if (!best) return false;
    p->Ntile = best;
    p->n_nt = Cout / best;
    p->nslot = 512 / best;
    if (p->nslot > 16) p->nslot = 16;
    // as many resident rows as tensor memory holds: the fewer input rows whose window of ring rows
    // wraps around the slot array, the fewer split MMAs
    int cols = 32;
    while (cols < p->nslot * best) cols <<= 1;
    p->tmem_cols = cols;
    const size_t wb = ((size_t)taps * p->n_kb * best * p->swb + 1023) / 1024 * 1024;
    p->out_esize = out_esize;
    p->out_pwb = best * out_esize >= 128 ? 128 : best * out_esize;
    p->out_panels = best * out_esize / p->out_pwb;
    p->out_stage_rows = stage_rows;
    p->out_stage_bytes = p->out_panels * stage_rows * p->out_pwb;
    // as many epilogue groups (one staging tile each) as still leave three Δ-row stages
    p->out_groups = 1;
    p->out_bufs = 1;
    // layers with many short K blocks per row (little MMA work per tile) need a deeper pipeline to cover the
    // copy latency more than they need a second epilogue group
    const size_t want_stages = p->n_kb >= 4 ? 4 : 3;
    for (int g = MAX_GROUPS; g > 1; --g)
        if (wb + want_stages * a_stage + (size_t)g * p->out_stage_bytes + 10240 <= SMEM_LIMIT) { p->out_groups = g; break; }
    // a second staging tile per group where it still leaves one more Δ-row stage than wanted
    if (wb + (want_stages + 1) * a_stage + 2 * (size_t)p->out_groups * p->out_stage_bytes + 10240 <= SMEM_LIMIT) p->out_bufs = 2;
    // the MMAs' run past a small box (see a_stage) must end inside this CTA's shared memory: what follows the
    // last stage (the staging tiles) covers it, or padding is added behind them
    const size_t overrun = (size_t)(128 + halo) * p->swb > box_pitch ? (size_t)(128 + halo) * p->swb - box_pitch : 0;
    const size_t tail_have = (size_t)p->out_groups * p->out_bufs * p->out_stage_bytes;
    const size_t tail_pad = overrun > tail_have ? (overrun - tail_have + 1023) / 1024 * 1024 : 0;
    if (SMEM_LIMIT < 8192 + wb + 1024 + tail_have + tail_pad + 2 * a_stage) return false;
    const size_t room = SMEM_LIMIT - 8192 - wb - 1024 - tail_have - tail_pad;   // static shared memory and alignment slack stay free
    int nstage = (int)(room / a_stage);
    if (nstage > 8) nstage = 8;
    if (nstage < 2) return false;
    p->nstage = nstage;
    p->smem_bytes = 1024 + wb + (size_t)nstage * a_stage + tail_have + tail_pad + 8 * (2 * nstage + taps + 2 * p->nslot) + 64;
    p->w_bytes = (size_t)taps * Cout * Cin * esize;
    p->ok = 1;
    return true;
}

// Where tap (ky, kx) of a layer goes in the tensor-core copy of its parameters, [tap'][Cout][Cin]: kx by kx, and
// inside a kx the Kh tap rows in the order of the stacked weight tiles (weight_block), so that one copy delivers
// a channel slice with all its taps in the shared-memory order the MMA schedule addresses.
int tc_weight_slot(int ky, int kx, int Kh, int stride) { return kx * Kh + weight_block(ky, Kh, stride); }

int tc_encode_weights(const TcPlan& p, int dtype, const void* d_w, int taps, int Cin, int Cout, void* map_out)
{
    EncodeTiledFn enc = encode_fn();
    if (!enc) return -1;
    const int esize = dtype == 1 ? 2 : 1;
    if (taps > 256) return -1;
    cuuint64_t dims[3] = {(cuuint64_t)Cin, (cuuint64_t)Cout, (cuuint64_t)taps};
    cuuint64_t strides[2] = {(cuuint64_t)Cin * esize, (cuuint64_t)Cout * Cin * esize};
    cuuint32_t box[3] = {(cuuint32_t)p.KB, (cuuint32_t)p.Ntile, (cuuint32_t)taps};   // all taps of a channel slice and K block
    cuuint32_t es[3] = {1, 1, 1};
    CUresult r = enc((CUtensorMap*)map_out, dtype == 1 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8, 3,
                     const_cast<void*>(d_w), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_of(p.swb),
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? 0 : -1;
}

// Returns cudaErrorNotSupported when the launch cannot take this path (the caller then uses the
// CUDA-core kernel): unaligned input pointer or a tensor map the driver rejects.
cudaError_t launch_conv_tc(const ConvArgs& a, const TcPlan& p, int dtype, const void* w_map, int n_in_rows,
                           unsigned int* status, cudaStream_t st)
{
    EncodeTiledFn enc = encode_fn();
    if (!enc || !p.ok) return cudaErrorNotSupported;
    if (((uintptr_t)a.in & 15) != 0 || n_in_rows < 1) return cudaErrorNotSupported;
    const int esize = dtype == 1 ? 2 : 1;
    CUtensorMap tmA;
    cuuint64_t dims[4] = {(cuuint64_t)a.Cin, (cuuint64_t)a.Win, (cuuint64_t)a.S, (cuuint64_t)n_in_rows};
    cuuint64_t strides[3] = {(cuuint64_t)a.Cin * esize, (cuuint64_t)a.Win * a.Cin * esize,
                             (cuuint64_t)a.S * a.Win * a.Cin * esize};
    // (with a traversal stride the box is counted in input positions and delivers every sx-th of them)
    cuuint32_t box[4] = {(cuuint32_t)p.KB, (cuuint32_t)(p.BXP * p.sx), (cuuint32_t)p.BS, 1};
    cuuint32_t es[4] = {1, 1, 1, 1}, es_in[4] = {1, (cuuint32_t)p.sx, 1, 1};
    if (a.stride_x != p.sx) return cudaErrorNotSupported;
    CUresult r = enc(&tmA, dtype == 1 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8, 4,
                     const_cast<void*>(a.in), dims, strides, box, es_in, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_of(p.swb),
                     CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cudaErrorNotSupported;

    // emitted rows leave through a TMA store: [channel][x][stream][row] or [channel][x][row][stream]
    CUtensorMap tmO;
    const int row_dim = a.out_row_stride > a.out_stream_stride ? 3 : 2;
    {
        const int oes = p.out_esize;
        const int ow = a.pool_fused ? a.Wout / 2 : a.Wout;            // width of the rows that leave the kernel
        const int obx = a.pool_fused ? p.BX / 2 : p.BX;
        if (a.pool_fused && ((p.BX & 1) || ow < 1 || !a.pool_state)) return cudaErrorNotSupported;
        if ((a.pool_fused != 0) != (p.out_stage_rows == 64)) return cudaErrorNotSupported;   // the plan's staging tile must fit the rows that leave
        cuuint64_t od[4] = {(cuuint64_t)a.Cout, (cuuint64_t)ow, 0, 0};
        cuuint64_t os[3] = {(cuuint64_t)a.Cout * oes, 0, 0};
        cuuint32_t ob[4] = {(cuuint32_t)(p.out_pwb / oes), (cuuint32_t)obx, 1, 1};
        od[row_dim] = (cuuint64_t)a.out_rows_extent; od[5 - row_dim] = (cuuint64_t)a.S;
        os[row_dim - 1] = (cuuint64_t)a.out_row_stride * oes; os[4 - row_dim] = (cuuint64_t)a.out_stream_stride * oes;
        ob[5 - row_dim] = (cuuint32_t)p.BS;
        if (((uintptr_t)a.out & 15) != 0 || a.out_rows_extent < 1) return cudaErrorNotSupported;
        const CUtensorMapDataType odt = a.out_elem == E_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16
                                      : (a.out_elem == E_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_UINT8);
        const CUtensorMapSwizzle osw = p.out_pwb == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                     : (p.out_pwb == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                     : (p.out_pwb == 32 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE));
        CUresult ro = enc(&tmO, odt, 4, a.out, od, os, ob, es, CU_TENSOR_MAP_INTERLEAVE_NONE, osw,
                          CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (ro != CUDA_SUCCESS) return cudaErrorNotSupported;
    }

    TcArgs t{};
    t.bias = a.bias; t.ring = a.ring; t.out = a.out; t.status = status;
    t.out_row_stride = a.out_row_stride; t.out_stream_stride = a.out_stream_stride; t.out_row_base = a.out_row_base;
    t.o_begin = a.o_begin; t.r0_positive = a.r0 > 0; t.n_rows = (int)(a.r1 - a.r0); t.n_orows = (int)(a.o_end - a.o_begin);
    t.done_rel = (int)(a.done_end - a.o_begin);
    {
        // rows whose last tap is a real input row of this block (the others below done_end end on bottom padding)
        const long long q = a.r1 + a.pad - a.Kh;
        long long sched = q < 0 ? 0 : q / a.stride + 1;
        if (sched < a.o_begin) sched = a.o_begin;
        if (sched > a.done_end) sched = a.done_end;
        t.sched_rel = (int)(sched - a.o_begin);
    }
    t.base_ty = (int)(a.r0 + a.pad - a.o_begin * a.stride);
    t.S = a.S; t.Wout = a.Wout; t.Cout = a.Cout; t.Kh = a.Kh; t.Kw = a.Kw; t.stride = a.stride;
    t.pad_x = a.pad_x; t.relu = a.relu; t.shift = a.shift; t.ring_rows = a.ring_rows; t.out_elem = a.out_elem;
    t.BX = p.BX; t.BS = p.BS; t.n_xt = p.n_xt; t.Ntile = p.Ntile; t.n_nt = p.n_nt; t.KB = p.KB; t.n_kb = p.n_kb;
    t.swb = p.swb; t.nslot = p.nslot; t.nstage = p.nstage; t.tmem_cols = p.tmem_cols;
    t.BXP = p.BXP; t.shift_mode = p.shift_mode; t.sx = p.sx; t.a_stage_bytes = p.a_stage_bytes; t.n_box = p.n_box; t.a_box_pitch = p.a_box_pitch;
    t.out_esize = p.out_esize; t.out_pwb = p.out_pwb; t.out_panels = p.out_panels; t.out_stage_bytes = p.out_stage_bytes; t.out_stage_rows = p.out_stage_rows; t.out_groups = p.out_groups; t.out_bufs = p.out_bufs;
    t.out_row_dim = row_dim; t.out_row_first = (int)(a.o_begin - a.out_row_base);
    t.pool = a.pool_fused; t.pool_keep = a.pool_keep; t.pool_state = a.pool_state; t.pool_row_base = a.out_row_base;
    t.o_begin_par = (int)(a.o_begin & 1);
    t.o_begin_half_mod = (int)((a.o_begin >> 1) % p.out_groups);
    t.ring_slot0 = (int)(a.o_begin % a.ring_rows);
    t.pool_row_first = (int)((a.o_begin >> 1) - a.out_row_base);
    t.ring_elems = a.ring_elems; t.pool_state_bytes = a.pool_state_elems * p.out_esize; t.smem_bytes = (unsigned int)p.smem_bytes;
    // row chunks: a layer with few tiles (few streams, narrow rows) spreads the block's rows over more CTAs
    t.n_chunks = 1; t.chunk_rows = t.n_orows; t.chunk_shift = 0;
    {
        const int units = p.n_mt * p.n_nt;
        int min_rows = 2 * a.ring_rows + 2;
        if (min_rows < 16) min_rows = 16;
        const bool no_chunks = (debug_flags() & IDF_DEBUG_NO_ROW_CHUNKS) != 0;
        // (a block that continues rows of an earlier one needs room for the copy of the ring, see ring_in)
        // a launch that takes a first row out of the pool layer's state (its first row is the second of a pair) and
        // also parks one there (its last emitted row is the first of a pair) keeps both in one CTA: read before write
        const bool pool_state_rw = a.pool_fused && a.pool_keep && (a.o_begin & 1) && (a.done_end & 1);
        if (!no_chunks && !pool_state_rw && units < 120 && t.n_orows >= 2 * min_rows && (a.r0 == 0 || a.ring_scratch)) {
            int want = 296 / units;                                 // at most two full waves of CTAs on the 148 SMs
            if (want > t.n_orows / min_rows) want = t.n_orows / min_rows;
            if (want > 1) {
                int rows = (t.n_orows + want - 1) / want;
                rows += rows & 1;                                   // even: a pooling pair stays in one chunk
                t.chunk_shift = a.pool_fused ? (int)(a.o_begin & 1) : 0;
                t.chunk_rows = rows;
                t.n_chunks = (t.n_orows + t.chunk_shift + rows - 1) / rows;
            }
        }
    }
    t.ring_in = a.ring;
    if (t.n_chunks > 1 && a.r0 > 0) {
        const size_t ring_bytes = (size_t)a.ring_rows * a.S * a.Wout * a.Cout * 4;
        cudaError_t ce = cudaMemcpyAsync(a.ring_scratch, a.ring, ring_bytes, cudaMemcpyDeviceToDevice, st);
        if (ce != cudaSuccess) return ce;
        t.ring_in = a.ring_scratch;
    }
    const unsigned grid = (unsigned)(p.n_mt * p.n_nt * t.n_chunks);
    typedef void (*KernelFn)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const TcArgs);
    static const KernelFn kernels[2][4] = {
        {conv_tc_kernel<1, 1, 0>, conv_tc_kernel<1, 2, 0>, conv_tc_kernel<1, 4, 0>, conv_tc_kernel<1, 4, 1>},
        {conv_tc_kernel<2, 1, 0>, conv_tc_kernel<2, 2, 0>, conv_tc_kernel<2, 4, 0>, conv_tc_kernel<2, 4, 1>}};
    const int kidx = p.swb == 32 ? 0 : (p.swb == 64 ? 1 : ((p.shift_mode && a.Kw == 3) ? 3 : 2));
    const KernelFn fn = kernels[dtype - 1][kidx];
    static bool attr_set[2][4][64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!attr_set[dtype - 1][kidx][dev]) {
        cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(SMEM_LIMIT - 6144));
        if (e != cudaSuccess) return e;
        attr_set[dtype - 1][kidx][dev] = true;
    }
    // programmatic dependent launch: the kernel may be scheduled while its predecessor drains; it
    // touches nothing but its weights until griddepcontrol.wait
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(TC_THREADS); cfg.dynamicSmemBytes = p.smem_bytes; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    // (without the attribute the griddepcontrol instructions in the kernels are no-ops)
    const bool use_pdl = (debug_flags() & IDF_DEBUG_NO_PDL) == 0;
    cfg.attrs = attr; cfg.numAttrs = use_pdl ? 1 : 0;
    cudaError_t le = cudaLaunchKernelEx(&cfg, fn, tmA, *(const CUtensorMap*)w_map, tmO, t);
    if (le != cudaSuccess) return le;
    return cudaGetLastError();
}


// ---- thin layers: host side ----------------------------------------------------------------------
bool thin_make_plan(int dtype, int S, int Wout, int Cin, int Cout, int Kh, int Kw, int stride, int stride_x, int out_esize, ThinPlan* p)
{
    *p = ThinPlan{};
    if (dtype != 1 && dtype != 2) return false;
    const int esize = dtype == 1 ? 2 : 1;
    const int kbytes = Kh * Kw * Cin * esize;
    if (kbytes > THIN_MAX_K || Cout % 16 != 0 || Cout > 256 || Kh * Kw * Cin > THIN_MAX_K) return false;
    p->swb = kbytes <= 32 ? 32 : (kbytes <= 64 ? 64 : 128);
    p->kelems = Kh * Kw * Cin;
    p->ksteps = p->swb / 32;
    if (Wout >= 128) {
        p->n_xt = (Wout + 127) / 128;
        p->BX = (Wout + p->n_xt - 1) / p->n_xt;
        p->BS = 1;
    } else {
        p->n_xt = 1;
        p->BX = Wout;
        p->BS = 128 / Wout;
        if (p->BS > S) p->BS = S;
    }
    p->n_mt = p->n_xt * ((S + p->BS - 1) / p->BS);
    p->out_esize = out_esize;
    p->out_pwb = Cout * out_esize >= 128 ? 128 : Cout * out_esize;
    p->out_panels = Cout * out_esize / p->out_pwb;
    p->out_tile_bytes = p->out_panels * 128 * p->out_pwb;
    // rows per work item: as many as two accumulator sets in tensor memory and two staging sets per group allow
    const size_t wb = ((size_t)Cout * p->swb + 1023) / 1024 * 1024;
    int R = 256 / Cout;
    if (R > 4) R = 4;
    for (; R >= 1; --R) {
        const size_t need = 2048 + wb + 3 * (size_t)R * 128 * p->swb + 4 * (size_t)R * p->out_tile_bytes + 512 + THIN_RAW_BYTES + 4096;
        // the input values behind the item's rows (with the kx halo) must fit the staging area
        const long long raw = (long long)((R - 1) * stride + Kh) * p->BS * ((p->BX - 1) * stride_x + Kw) * Cin;
        if (need <= SMEM_LIMIT && raw <= 128 * THIN_RAW_PER_THREAD && raw * 4 < 32767) break;
    }
    if (R < 1) return false;
    p->R = R;
    p->nstage = 3;
    int cols = 32;
    while (cols < 2 * R * Cout) cols <<= 1;
    if (cols > 512) return false;
    p->tmem_cols = cols;
    p->smem_bytes = 1024 + wb + (size_t)p->nstage * R * 128 * p->swb + 4 * (size_t)R * p->out_tile_bytes + 256 + THIN_RAW_BYTES + 64;
    p->w_bytes = (size_t)Cout * p->swb;
    p->ok = 1;
    return true;
}

int thin_encode_weights(const ThinPlan& p, int dtype, const void* d_w, int Cout, void* map_out)
{
    EncodeTiledFn enc = encode_fn();
    if (!enc) return -1;
    const int esize = dtype == 1 ? 2 : 1;
    cuuint64_t dims[2] = {(cuuint64_t)(p.swb / esize), (cuuint64_t)Cout};
    cuuint64_t strides[1] = {(cuuint64_t)p.swb};
    cuuint32_t box[2] = {(cuuint32_t)(p.swb / esize), (cuuint32_t)Cout};
    cuuint32_t es[2] = {1, 1};
    CUresult r = enc((CUtensorMap*)map_out, dtype == 1 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8, 2,
                     const_cast<void*>(d_w), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_of(p.swb),
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? 0 : -1;
}

// Output rows [o_first, o_end) of the layer, each determined completely by the block's input rows a.in (rows
// a.r0 .. a.r1-1; taps outside them fall on zero padding).  cudaErrorNotSupported: use another kernel.
cudaError_t launch_conv_thin(const ConvArgs& a, const ThinPlan& p, int dtype, const void* w_map, long long o_first, long long o_end,
                             unsigned int* status, cudaStream_t st)
{
    EncodeTiledFn enc = encode_fn();
    if (!enc || !p.ok || o_end <= o_first) return cudaErrorNotSupported;
    if (((uintptr_t)a.out & 15) != 0 || a.out_rows_extent < 1 || a.pool_fused) return cudaErrorNotSupported;
    CUtensorMap tmO;
    const int row_dim = a.out_row_stride > a.out_stream_stride ? 3 : 2;
    {
        const int oes = p.out_esize;
        cuuint64_t od[4] = {(cuuint64_t)a.Cout, (cuuint64_t)a.Wout, 0, 0};
        cuuint64_t os[3] = {(cuuint64_t)a.Cout * oes, 0, 0};
        cuuint32_t ob[4] = {(cuuint32_t)(p.out_pwb / oes), (cuuint32_t)p.BX, 1, 1};
        cuuint32_t es[4] = {1, 1, 1, 1};
        od[row_dim] = (cuuint64_t)a.out_rows_extent; od[5 - row_dim] = (cuuint64_t)a.S;
        os[row_dim - 1] = (cuuint64_t)a.out_row_stride * oes; os[4 - row_dim] = (cuuint64_t)a.out_stream_stride * oes;
        ob[5 - row_dim] = (cuuint32_t)p.BS;
        const CUtensorMapDataType odt = a.out_elem == E_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16
                                      : (a.out_elem == E_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_UINT8);
        const CUtensorMapSwizzle osw = p.out_pwb == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                     : (p.out_pwb == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                     : (p.out_pwb == 32 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE));
        if (enc(&tmO, odt, 4, a.out, od, os, ob, es, CU_TENSOR_MAP_INTERLEAVE_NONE, osw, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorNotSupported;
    }
    ThinArgs t{};
    t.in = a.in; t.bias = a.bias; t.status = status;
    t.r0 = a.r0; t.o_first = o_first; t.n_in = (int)(a.r1 - a.r0); t.n_out = (int)(o_end - o_first);
    t.S = a.S; t.Win = a.Win; t.Wout = a.Wout; t.Cin = a.Cin; t.Cout = a.Cout; t.Kh = a.Kh; t.Kw = a.Kw;
    t.stride = a.stride; t.pad = a.pad; t.stride_x = a.stride_x; t.pad_x = a.pad_x; t.relu = a.relu; t.shift = a.shift;
    t.out_elem = a.out_elem;
    t.kelems = p.kelems; t.swb = p.swb; t.ksteps = p.ksteps; t.BX = p.BX; t.BS = p.BS; t.n_xt = p.n_xt; t.n_mt = p.n_mt;
    t.R = p.R; t.nstage = p.nstage; t.tmem_cols = p.tmem_cols;
    t.out_esize = p.out_esize; t.out_pwb = p.out_pwb; t.out_panels = p.out_panels; t.out_tile_bytes = p.out_tile_bytes;
    t.out_row_dim = row_dim; t.out_row_first = (int)(o_first - a.out_row_base);
    const long long n_items = (long long)((t.n_out + p.R - 1) / p.R) * p.n_mt;
    const unsigned grid = (unsigned)(n_items < 148 ? n_items : 148);
    typedef void (*KernelFn)(const CUtensorMap, const CUtensorMap, const ThinArgs);
    const KernelFn fn = dtype == 1 ? (KernelFn)conv_thin_kernel<1> : (KernelFn)conv_thin_kernel<2>;
    static bool attr_set[2][64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!attr_set[dtype - 1][dev]) {
        cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(SMEM_LIMIT - 6144));
        if (e != cudaSuccess) return e;
        attr_set[dtype - 1][dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(THIN_THREADS); cfg.dynamicSmemBytes = p.smem_bytes; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = (debug_flags() & IDF_DEBUG_NO_PDL) ? 0 : 1;
    cudaError_t le = cudaLaunchKernelEx(&cfg, fn, *(const CUtensorMap*)w_map, tmO, t);
    if (le != cudaSuccess) return le;
    return cudaGetLastError();
}

}  // namespace idf
