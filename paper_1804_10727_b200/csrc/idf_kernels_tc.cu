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
//   - when an input row was the last one an output row was waiting for, the epilogue warps read that
//     accumulator, add what the ring held from earlier blocks and the bias, apply f, round or
//     requantise, and write the row for the next layer; rows still open at the end of the block go
//     back to the ring in global memory.
// Warp roles: warp 0 = TMA producer, warp 1 = TMEM owner and MMA issuer, warps 2-5 = epilogue.
// Every wait is bounded; on expiry the kernel records IDF_ERR_TIMEOUT in the status word and leaves.
#include "idf_internal.h"

#include <cuda.h>
#include <mutex>

namespace idf {

namespace {

constexpr int TC_THREADS = 192;
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

struct TcArgs {
    const void* bias;
    void* ring;
    void* out;
    unsigned int* status;
    long long out_row_stride, out_stream_stride, out_row_base;
    long long o_begin;           // absolute index of the first visited output row
    int r0_positive;             // input rows arrived before this block (r0 > 0)
    int n_rows;                  // input rows in this block
    int n_orows;                 // visited output rows: o_begin + [0, n_orows)
    int done_rel;                // rows with relative index < done_rel are emitted, the others go back to the ring
    int base_ty;                 // r0 + pad - o_begin*stride: input row ri reaches relative output row
                                 // (base_ty + ri - ky) / stride through tap ky when that is a whole number >= 0
    int S, Wout, Cout, Kh, Kw, stride, pad_x, relu, shift, ring_rows, out_elem;
    int BX, BXP, BS, n_xt, Ntile, n_nt, KB, n_kb, swb, nslot, nstage, tmem_cols;
    int shift_mode;              // 1: one box per (row, K block) holds the kx halo, taps address it at row offsets
    int a_stage_bytes;
};

template <int DT> struct Acc;
template <> struct Acc<1> { typedef float S; };
template <> struct Acc<2> { typedef int S; };

template <int DT>
__global__ void __launch_bounds__(TC_THREADS, 1)
conv_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW, const TcArgs a)
{
    typedef typename Acc<DT>::S TS;
    extern __shared__ unsigned char smem_raw[];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    __shared__ int s_issued;
    __shared__ int s_tap_ky[32], s_tap_orel[32], s_tap_first[32];   // scratch of the MMA thread

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int taps = a.Kh * a.Kw;
    const uint32_t w_tile_bytes = (uint32_t)a.Ntile * a.swb;
    const uint32_t a_stage_bytes = (uint32_t)a.a_stage_bytes;
    const uint32_t a_box_bytes = (uint32_t)a.BXP * a.BS * a.swb;
    const int n_xload = a.shift_mode ? 1 : a.Kw;

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sW = base;
    const uint32_t sA = (sW + (uint32_t)taps * a.n_kb * w_tile_bytes + 1023u) & ~1023u;
    const uint32_t bars = sA + (uint32_t)a.nstage * a_stage_bytes;
    const uint32_t bar_full = bars;
    const uint32_t bar_empty = bar_full + 8u * a.nstage;
    const uint32_t bar_w = bar_empty + 8u * a.nstage;
    const uint32_t bar_ready = bar_w + 8u * taps;
    const uint32_t bar_free = bar_ready + 8u * a.nslot;

    const int nt = blockIdx.x % a.n_nt;
    const int mt = blockIdx.x / a.n_nt;
    const int xt = mt % a.n_xt, stile = mt / a.n_xt;
    const int x0 = xt * a.BX, s0 = stile * a.BS, n0 = nt * a.Ntile;

    if (threadIdx.x == 0) {
        s_abort = 0;
        s_issued = 0;
        for (int i = 0; i < a.nstage; ++i) { mbar_init(bar_full + 8u * i, 1); mbar_init(bar_empty + 8u * i, 1); }
        for (int i = 0; i < taps; ++i) mbar_init(bar_w + 8u * i, 1);
        for (int i = 0; i < a.nslot; ++i) { mbar_init(bar_ready + 8u * i, 1); mbar_init(bar_free + 8u * i, 128); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)), "r"((uint32_t)a.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;
    volatile int* abort_flag = &s_abort;
    const int n_rows = a.n_rows;

    if (warp == 0) {
        // ------------------------------ TMA producer -------------------------------------------
        if (lane == 0) {
            for (int kx = 0; kx < a.Kw; ++kx)
                for (int ky = 0; ky < a.Kh; ++ky) {
                    const int tap = ky * a.Kw + kx;
                    mbar_expect_tx(bar_w + 8u * tap, (uint32_t)a.n_kb * w_tile_bytes);
                    for (int kb = 0; kb < a.n_kb; ++kb)
                        tma_load_2d(sW + (uint32_t)(tap * a.n_kb + kb) * w_tile_bytes, &tmW, bar_w + 8u * tap,
                                    kb * a.KB, tap * a.Cout + n0);
                }
            int stage = 0, t = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int ri = 0; ri < n_rows && ok; ++ri)
                for (int xl = 0; xl < n_xload && ok; ++xl)
                    for (int kb = 0; kb < a.n_kb; ++kb) {
                        if (!mbar_wait(bar_empty + 8u * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
                        mbar_expect_tx(bar_full + 8u * stage, a_box_bytes);
                        tma_load_4d(sA + (uint32_t)stage * a_stage_bytes, &tmA, bar_full + 8u * stage,
                                    kb * a.KB, x0 - a.pad_x + xl, s0, ri);
                        s_issued = ++t;
                        if (++stage == a.nstage) { stage = 0; phase ^= 1u; }
                    }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ---------------------------------------------
        if (lane == 0) {
            const uint32_t idesc = (DT == 1 ? ((1u << 4) | (1u << 7) | (1u << 10)) : ((2u << 4) | (1u << 7) | (1u << 10))) |
                                   ((uint32_t)(a.Ntile >> 3) << 17) | ((128u >> 4) << 24);
            const int ksteps = a.swb / 32;
            const uint64_t desc_hi = make_smem_desc(0, a.swb);
            const int n_kx = a.shift_mode ? a.Kw : 1;
            uint32_t w_seen = 0;
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int ri = 0; ri < n_rows && ok; ++ri) {
                // output rows this input row reaches (a handful): slot, first touch, completion
                int n_t = 0;
                for (int ky = 0; ky < a.Kh && ok; ++ky) {
                    const int ty = a.base_ty + ri - ky;
                    if (ty < 0) break;
                    const int orel = ty / a.stride;
                    if (orel * a.stride != ty) continue;
                    int fr = orel * a.stride - a.base_ty;
                    if (fr < 0) fr = 0;
                    const int first = (ri == fr);
                    if (first && orel >= a.nslot) {      // the slot's previous row must have been read out
                        const int u = orel / a.nslot;
                        if (!mbar_wait(bar_free + 8u * (orel % a.nslot), (uint32_t)((u - 1) & 1), abort_flag)) { ok = false; break; }
                        tc_fence_after();
                    }
                    s_tap_ky[n_t] = ky; s_tap_orel[n_t] = orel; s_tap_first[n_t] = first;
                    ++n_t;
                }
                for (int xl = 0; xl < n_xload && ok; ++xl)
                    for (int kb = 0; kb < a.n_kb && ok; ++kb) {
                        if (!mbar_wait(bar_full + 8u * stage, phase, abort_flag)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t abase = sA + (uint32_t)stage * a_stage_bytes;
                        for (int kxi = 0; kxi < n_kx && ok; ++kxi) {
                            const int kx = a.shift_mode ? kxi : xl;
                            // tap kx reads the same tile kxi rows further down: the swizzle is a function of
                            // the absolute shared-memory address, so a start address moved by whole rows
                            // still meets the pattern the TMA wrote (base-offset field stays 0)
                            const uint32_t aaddr = abase + (uint32_t)kxi * a.swb;
                            const uint64_t adesc = desc_hi | (uint64_t)((aaddr & 0x3FFFFu) >> 4);
                            const bool first_tile = (xl == 0 && kxi == 0 && kb == 0);
                            for (int i = 0; i < n_t; ++i) {
                                const int tap = s_tap_ky[i] * a.Kw + kx;
                                if (!((w_seen >> tap) & 1u)) {
                                    if (!mbar_wait(bar_w + 8u * tap, 0, abort_flag)) { ok = false; break; }
                                    tc_fence_after();
                                    w_seen |= 1u << tap;
                                }
                                const uint32_t baddr = sW + (uint32_t)(tap * a.n_kb + kb) * w_tile_bytes;
                                const uint64_t bdesc = desc_hi | (uint64_t)((baddr & 0x3FFFFu) >> 4);
                                const uint32_t d = tmem_base + (uint32_t)((s_tap_orel[i] % a.nslot) * a.Ntile);
                                const uint32_t acc0 = (first_tile && s_tap_first[i]) ? 0u : 1u;
                                umma<DT>(d, adesc, bdesc, idesc, acc0);
                                for (int k = 1; k < ksteps; ++k)
                                    umma<DT>(d, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc, 1u);
                            }
                        }
                        if (ok) umma_commit(bar_empty + 8u * stage);
                        if (++stage == a.nstage) { stage = 0; phase ^= 1u; }
                    }
                if (!ok) break;
                // accumulators that this input row completed (on the block's last row: everything still open)
                for (int i = n_t - 1; i >= 0; --i) {
                    const int orel = s_tap_orel[i];
                    const int fin = (orel < a.done_rel) ? orel * a.stride - a.base_ty + a.Kh - 1 : n_rows - 1;
                    if (fin == ri) umma_commit(bar_ready + 8u * (uint32_t)(orel % a.nslot));
                }
            }
        }
        __syncwarp();
    } else {
        // ------------------------------ epilogue: row finalisation -----------------------------
        const int q = warp & 3;                          // TMEM lane quarter this warp may read
        const int m = q * 32 + lane;                     // row of the tile = TMEM lane
        const int bs = m / a.BXP, bx = m - bs * a.BXP;
        const int s = s0 + bs, x = x0 + bx;
        const bool valid = (bs < a.BS) && (bx < a.BX) && (s < a.S) && (x < a.Wout);
        const TS* bias = (const TS*)a.bias;
        TS* ring = (TS*)a.ring;
        const long long row_elems = (long long)a.Wout * a.Cout;
        bool ok = true;
        for (int orel = 0; orel < a.n_orows && ok; ++orel) {
            const long long o = a.o_begin + orel;
            const int slot = orel % a.nslot, u = orel / a.nslot;
            int got = 0;
            if (lane == 0) got = mbar_wait(bar_ready + 8u * slot, (uint32_t)(u & 1), abort_flag) ? 1 : 0;
            got = __shfl_sync(0xffffffffu, got, 0);
            if (!got) { ok = false; break; }
            tc_fence_after();
            const bool carried_in = a.r0_positive && (orel * a.stride - a.base_ty < 0);
            const bool emit = orel < a.done_rel;
            TS* rp = ring + ((o % a.ring_rows) * a.S + s) * row_elems + (long long)x * a.Cout + n0;
            const long long obase = (o - a.out_row_base) * a.out_row_stride + (long long)s * a.out_stream_stride +
                                    (long long)x * a.Cout + n0;
            for (int c = 0; c < a.Ntile; c += 16) {
                uint32_t v[16];
                tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(slot * a.Ntile + c), v);
                if (!valid) continue;
                TS acc[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) acc[j] = DT == 1 ? (TS)__uint_as_float(v[j]) : (TS)(int)v[j];
                if (carried_in) {
                    const int4* p4 = (const int4*)(rp + c);
#pragma unroll
                    for (int j4 = 0; j4 < 4; ++j4) {
                        const int4 t4 = p4[j4];
                        if (DT == 1) {
                            acc[4 * j4 + 0] += (TS)__int_as_float(t4.x); acc[4 * j4 + 1] += (TS)__int_as_float(t4.y);
                            acc[4 * j4 + 2] += (TS)__int_as_float(t4.z); acc[4 * j4 + 3] += (TS)__int_as_float(t4.w);
                        } else {
                            acc[4 * j4 + 0] += (TS)t4.x; acc[4 * j4 + 1] += (TS)t4.y;
                            acc[4 * j4 + 2] += (TS)t4.z; acc[4 * j4 + 3] += (TS)t4.w;
                        }
                    }
                }
                if (!emit) {
                    int4* p4 = (int4*)(rp + c);
#pragma unroll
                    for (int j4 = 0; j4 < 4; ++j4) {
                        int4 t4;
                        if (DT == 1) {
                            t4.x = __float_as_int((float)acc[4 * j4 + 0]); t4.y = __float_as_int((float)acc[4 * j4 + 1]);
                            t4.z = __float_as_int((float)acc[4 * j4 + 2]); t4.w = __float_as_int((float)acc[4 * j4 + 3]);
                        } else {
                            t4.x = (int)acc[4 * j4 + 0]; t4.y = (int)acc[4 * j4 + 1];
                            t4.z = (int)acc[4 * j4 + 2]; t4.w = (int)acc[4 * j4 + 3];
                        }
                        p4[j4] = t4;
                    }
                    continue;
                }
                if (DT == 1) {
                    float f[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        float t = (float)acc[j] + (bias ? (float)bias[n0 + c + j] : 0.f);
                        f[j] = (a.relu && t < 0.f) ? 0.f : t;
                    }
                    if (a.out_elem == E_BF16) {
                        __nv_bfloat16* op = (__nv_bfloat16*)a.out + obase + c;
                        uint32_t pk[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            __nv_bfloat162 h2 = __floats2bfloat162_rn(f[2 * j], f[2 * j + 1]);
                            pk[j] = *(uint32_t*)&h2;
                        }
                        ((int4*)op)[0] = make_int4((int)pk[0], (int)pk[1], (int)pk[2], (int)pk[3]);
                        ((int4*)op)[1] = make_int4((int)pk[4], (int)pk[5], (int)pk[6], (int)pk[7]);
                    } else {
                        float* op = (float*)a.out + obase + c;
#pragma unroll
                        for (int j4 = 0; j4 < 4; ++j4)
                            ((float4*)op)[j4] = make_float4(f[4 * j4], f[4 * j4 + 1], f[4 * j4 + 2], f[4 * j4 + 3]);
                    }
                } else {
                    uint32_t pk[4] = {0, 0, 0, 0};
                    const int lo = a.relu ? 0 : -127;
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        int t = (int)acc[j] + (bias ? (int)bias[n0 + c + j] : 0);
                        if (a.relu && t < 0) t = 0;
                        if (a.shift > 0) t = (t + (1 << (a.shift - 1))) >> a.shift;
                        t = t < lo ? lo : (t > 127 ? 127 : t);
                        pk[j >> 2] |= ((uint32_t)t & 0xffu) << (8 * (j & 3));
                    }
                    int8_t* op = (int8_t*)a.out + obase + c;
                    *(int4*)op = make_int4((int)pk[0], (int)pk[1], (int)pk[2], (int)pk[3]);
                }
            }
            tc_fence_before();
            mbar_arrive(bar_free + 8u * slot);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (s_abort) {
        if (threadIdx.x == 0) {
            // let this CTA's own copies land before its shared memory is given back (bounded)
            for (int tap = 0; tap < taps; ++tap)
                for (uint32_t i = 0; i < 4096 && !mbar_try_wait(bar_w + 8u * tap, 0); ++i) __nanosleep(64);
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
                  TcPlan* p)
{
    *p = TcPlan{};
    if (dtype != 1 && dtype != 2) return false;
    const int esize = dtype == 1 ? 2 : 1;
    const int row_bytes = Cin * esize;
    if (stride_x != 1) return false;
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
    if (p->BXP > 256) return false;
    const size_t a_stage = ((size_t)((128 + halo + 7) / 8 * 8) * p->swb + 1023) / 1024 * 1024;
    p->a_stage_bytes = (int)a_stage;
    p->n_mt = p->n_xt * ((S + p->BS - 1) / p->BS);
    const int taps = Kh * Kw;
    int best = 0, best_units = -1;
    for (int nt = 256; nt >= 16; nt >>= 1) {
        if (Cout % nt) continue;
        if ((ring_rows + 1) * nt > 512) continue;
        const size_t wb = (size_t)taps * p->n_kb * nt * p->swb;
        if (wb + 3 * a_stage + 4096 > SMEM_LIMIT) continue;
        const int units = p->n_mt * (Cout / nt);
        if (units >= 120) { best = nt; break; }          // enough CTAs for the 148 SMs: take the widest such tile
        if (units > best_units) { best_units = units; best = nt; }
    }
    if (!best) return false;
    p->Ntile = best;
    p->n_nt = Cout / best;
    p->nslot = 512 / best;
    if (p->nslot > 16) p->nslot = 16;
    if (p->nslot > ring_rows + 3) p->nslot = ring_rows + 3;
    int cols = 32;
    while (cols < p->nslot * best) cols <<= 1;
    p->tmem_cols = cols;
    const size_t wb = ((size_t)taps * p->n_kb * best * p->swb + 1023) / 1024 * 1024;
    const size_t room = SMEM_LIMIT - 2048 - wb - 1024;
    int nstage = (int)(room / a_stage);
    if (nstage > 8) nstage = 8;
    if (nstage < 2) return false;
    p->nstage = nstage;
    p->smem_bytes = 1024 + wb + (size_t)nstage * a_stage + 8 * (2 * nstage + taps + 2 * p->nslot) + 64;
    p->w_bytes = (size_t)taps * Cout * Cin * esize;
    p->ok = 1;
    return true;
}

int tc_encode_weights(const TcPlan& p, int dtype, const void* d_w, int taps, int Cin, int Cout, void* map_out)
{
    EncodeTiledFn enc = encode_fn();
    if (!enc) return -1;
    const int esize = dtype == 1 ? 2 : 1;
    cuuint64_t dims[2] = {(cuuint64_t)Cin, (cuuint64_t)taps * Cout};
    cuuint64_t strides[1] = {(cuuint64_t)Cin * esize};
    cuuint32_t box[2] = {(cuuint32_t)p.KB, (cuuint32_t)p.Ntile};
    cuuint32_t es[2] = {1, 1};
    CUresult r = enc((CUtensorMap*)map_out, dtype == 1 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8, 2,
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
    cuuint32_t box[4] = {(cuuint32_t)p.KB, (cuuint32_t)p.BXP, (cuuint32_t)p.BS, 1};
    cuuint32_t es[4] = {1, 1, 1, 1};
    CUresult r = enc(&tmA, dtype == 1 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8, 4,
                     const_cast<void*>(a.in), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_of(p.swb),
                     CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cudaErrorNotSupported;

    TcArgs t{};
    t.bias = a.bias; t.ring = a.ring; t.out = a.out; t.status = status;
    t.out_row_stride = a.out_row_stride; t.out_stream_stride = a.out_stream_stride; t.out_row_base = a.out_row_base;
    t.o_begin = a.o_begin; t.r0_positive = a.r0 > 0; t.n_rows = (int)(a.r1 - a.r0); t.n_orows = (int)(a.o_end - a.o_begin);
    t.done_rel = (int)(a.done_end - a.o_begin); t.base_ty = (int)(a.r0 + a.pad - a.o_begin * a.stride);
    t.S = a.S; t.Wout = a.Wout; t.Cout = a.Cout; t.Kh = a.Kh; t.Kw = a.Kw; t.stride = a.stride;
    t.pad_x = a.pad_x; t.relu = a.relu; t.shift = a.shift; t.ring_rows = a.ring_rows; t.out_elem = a.out_elem;
    t.BX = p.BX; t.BS = p.BS; t.n_xt = p.n_xt; t.Ntile = p.Ntile; t.n_nt = p.n_nt; t.KB = p.KB; t.n_kb = p.n_kb;
    t.swb = p.swb; t.nslot = p.nslot; t.nstage = p.nstage; t.tmem_cols = p.tmem_cols;
    t.BXP = p.BXP; t.shift_mode = p.shift_mode; t.a_stage_bytes = p.a_stage_bytes;
    const unsigned grid = (unsigned)(p.n_mt * p.n_nt);
    static bool attr_set[2][64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!attr_set[dtype - 1][dev]) {
        cudaError_t e = dtype == 1
            ? cudaFuncSetAttribute(conv_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(SMEM_LIMIT - 1024))
            : cudaFuncSetAttribute(conv_tc_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(SMEM_LIMIT - 1024));
        if (e != cudaSuccess) return e;
        attr_set[dtype - 1][dev] = true;
    }
    if (dtype == 1) conv_tc_kernel<1><<<grid, TC_THREADS, p.smem_bytes, st>>>(tmA, *(const CUtensorMap*)w_map, t);
    else conv_tc_kernel<2><<<grid, TC_THREADS, p.smem_bytes, st>>>(tmA, *(const CUtensorMap*)w_map, t);
    return cudaGetLastError();
}

}  // namespace idf
