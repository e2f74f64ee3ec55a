// CUDA-core kernels: the general path for every type and shape.
//
//  conv_rows_kernel    dense Δ-row update + row finalisation (Eq. 4 applied tap by tap, then Eq. 2-3
//                      once per unit), one thread per ring-slot element
//  conv_sparse_kernel  compaction of the non-zero Δ-events of a row (warp ballot + prefix sum) and
//                      scatter of w*Δh into the ring (Eq. 4 event by event), one CTA per stream
//  pool_rows_kernel    2x2 max-pool fold with a one-row running maximum
#include "idf_internal.h"

#include <climits>

namespace idf {

__device__ __forceinline__ float to_acc(float v) { return v; }
__device__ __forceinline__ float to_acc(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ int to_acc(int8_t v) { return (int)v; }

template <typename TO, typename TS>
struct Emit;
template <>
struct Emit<float, float> {
    static __device__ __forceinline__ float run(float c, float b, int relu, int) {
        float v = c + b;
        return (relu && v < 0.f) ? 0.f : v;
    }
};
template <>
struct Emit<__nv_bfloat16, float> {
    static __device__ __forceinline__ __nv_bfloat16 run(float c, float b, int relu, int) {
        float v = c + b;
        if (relu && v < 0.f) v = 0.f;
        return __float2bfloat16_rn(v);
    }
};
template <>
struct Emit<int8_t, int> {
    static __device__ __forceinline__ int8_t run(int c, int b, int relu, int shift) {
        int v = c + b;
        if (relu && v < 0) v = 0;
        if (shift > 0) v = (v + (1 << (shift - 1))) >> shift;   // arithmetic shift = floor division
        const int lo = relu ? 0 : -127;
        v = v < lo ? lo : (v > 127 ? 127 : v);
        return (int8_t)v;
    }
};

// ------------------------------------------------------------------------------------------------
// Dense update + finalisation.  The first `edge_blocks` CTAs: one thread owns one element (slot, stream,
// x, co) of the ring and walks, in order, every output row of this block that lives in that slot and
// exchanges state with the ring (begun by an earlier block, or left open by this one), so a slot is
// never read and written by different threads.  The other CTAs take the interior rows [int_begin, int_end):
// rows begun AND completed by this block's input never touch the ring (Eq. 1 restricted to the block), so
// each (row, stream, x, co) has a thread of its own - with few streams and narrow rows that is where the
// parallelism is.  Weights: [Kh][Kw][Cin][Cout] (threads of a warp differ in co).
// ------------------------------------------------------------------------------------------------
template <typename TI, typename TW, typename TS, typename TO>
__global__ void __launch_bounds__(256) conv_rows_kernel(ConvArgs a, long long int_begin, long long int_end, unsigned edge_blocks)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const TI* __restrict__ in = (const TI*)a.in;
    const TW* __restrict__ w = (const TW*)a.w;
    const TS* __restrict__ bias = (const TS*)a.bias;
    TS* ring = (TS*)a.ring;
    TO* out = (TO*)a.out;
    const long long row_elems = (long long)a.Wout * a.Cout;
    if (blockIdx.x >= edge_blocks) {
        const long long n_int = (int_end - int_begin) * a.S * row_elems;
        for (long long idx = (long long)(blockIdx.x - edge_blocks) * blockDim.x + threadIdx.x; idx < n_int;
             idx += (long long)(gridDim.x - edge_blocks) * blockDim.x) {
            const int co = (int)(idx % a.Cout);
            long long t = idx / a.Cout;
            const int x = (int)(t % a.Wout);
            t /= a.Wout;
            const int s = (int)(t % a.S);
            const long long o = int_begin + t / a.S;
            TS acc = 0;
            for (int ky = 0; ky < a.Kh; ++ky) {
                const long long r = o * a.stride - a.pad + ky;
                if (r < a.r0 || r >= a.r1) continue;             // zero padding above the first or below the last row
                const TI* row = in + ((r - a.r0) * a.S + s) * (long long)a.Win * a.Cin;
                for (int kx = 0; kx < a.Kw; ++kx) {
                    const int ix = x * a.stride_x - a.pad_x + kx;
                    if (ix < 0 || ix >= a.Win) continue;
                    const TI* ap = row + (long long)ix * a.Cin;
                    if (!IDF_OK_AT(a.status, (ap - in) + a.Cin - 1, a.in_elems)) continue;
                    const TW* wp = w + ((long long)(ky * a.Kw + kx) * a.Cin) * a.Cout + co;
                    for (int ci = 0; ci < a.Cin; ++ci) acc += to_acc(ap[ci]) * to_acc(wp[(long long)ci * a.Cout]);
                }
            }
            const long long oi = (o - a.out_row_base) * a.out_row_stride + (long long)s * a.out_stream_stride + (long long)x * a.Cout + co;
            if (IDF_OK_AT(a.status, oi, a.out_elems)) out[oi] = Emit<TO, TS>::run(acc, bias ? bias[co] : (TS)0, a.relu, a.shift);
        }
        return;
    }
    const long long total = (long long)a.ring_rows * a.S * row_elems;
    const int slot_of_first = (int)(a.o_begin % a.ring_rows);      // (one 64-bit division per thread instead of five)
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (long long)edge_blocks * blockDim.x) {
        int co, x, s, slot;
        if (total <= 0x7fffffffLL) {
            unsigned t = (unsigned)idx;
            co = (int)(t % (unsigned)a.Cout); t /= (unsigned)a.Cout;
            x = (int)(t % (unsigned)a.Wout); t /= (unsigned)a.Wout;
            s = (int)(t % (unsigned)a.S);
            slot = (int)(t / (unsigned)a.S);
        } else {
            co = (int)(idx % a.Cout);
            long long t = idx / a.Cout;
            x = (int)(t % a.Wout);
            t /= a.Wout;
            s = (int)(t % a.S);
            slot = (int)(t / a.S);
        }
        const TS b = bias ? bias[co] : (TS)0;
        // first visited row that lives in this slot
        long long o = a.o_begin + ((slot - slot_of_first) + a.ring_rows) % a.ring_rows;
        bool dirty = false;
        TS leave = 0;
        TS* rp = ring + ((long long)slot * a.S + s) * row_elems + (long long)x * a.Cout + co;
        if (!IDF_OK_AT(a.status, rp - ring, a.ring_elems)) continue;
        for (; o < a.o_end; o += a.ring_rows) {
            if (o >= int_begin && o < int_end) {                 // interior rows are another CTA's: on to the slot's first row behind them
                o += (long long)((unsigned)(int_end - 1 - o) / (unsigned)a.ring_rows) * a.ring_rows;      // (a block has far fewer than 2^32 rows)
                continue;
            }
            TS acc = 0;
            for (int ky = 0; ky < a.Kh; ++ky) {
                const long long r = o * a.stride - a.pad + ky;
                if (r < a.r0 || r >= a.r1) continue;
                const TI* row = in + ((r - a.r0) * a.S + s) * (long long)a.Win * a.Cin;
                for (int kx = 0; kx < a.Kw; ++kx) {
                    const int ix = x * a.stride_x - a.pad_x + kx;
                    if (ix < 0 || ix >= a.Win) continue;
                    const TI* ap = row + (long long)ix * a.Cin;
                    if (!IDF_OK_AT(a.status, (ap - in) + a.Cin - 1, a.in_elems)) continue;
                    const TW* wp = w + ((long long)(ky * a.Kw + kx) * a.Cin) * a.Cout + co;
                    for (int ci = 0; ci < a.Cin; ++ci) acc += to_acc(ap[ci]) * to_acc(wp[(long long)ci * a.Cout]);
                }
            }
            const bool carried_in = (a.r0 > 0) && (o * a.stride - a.pad < a.r0);
            const TS c = acc + (carried_in ? *rp : (TS)0);
            if (o < a.done_end) {
                const long long oi = (o - a.out_row_base) * a.out_row_stride + (long long)s * a.out_stream_stride + (long long)x * a.Cout + co;
                if (IDF_OK_AT(a.status, oi, a.out_elems)) out[oi] = Emit<TO, TS>::run(c, b, a.relu, a.shift);
                if (carried_in) { dirty = true; leave = 0; }
            } else {
                dirty = true;
                leave = c;
            }
        }
        if (dirty) *rp = leave;
    }
}

// End-of-input completion when no input rows arrive: the visited rows only wait for bottom
// padding, so each is read from its ring slot, emitted and its slot cleared.  Four channels per thread.
template <typename TS, typename TO>
__global__ void __launch_bounds__(256) conv_flush_kernel(ConvArgs a)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const TS* __restrict__ bias = (const TS*)a.bias;
    TS* ring = (TS*)a.ring;
    TO* out = (TO*)a.out;
    const int c4n = a.Cout / 4;
    const long long row_elems = (long long)a.Wout * a.Cout;
    const long long total = (a.o_end - a.o_begin) * a.S * a.Wout * c4n;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const int co = (int)(idx % c4n) * 4;
        long long t = idx / c4n;
        const int x = (int)(t % a.Wout);
        t /= a.Wout;
        const int s = (int)(t % a.S);
        const long long o = a.o_begin + t / a.S;
        TS* rp = ring + ((o % a.ring_rows) * a.S + s) * row_elems + (long long)x * a.Cout + co;
        if (!IDF_OK_AT(a.status, (rp - ring) + 3, a.ring_elems)) continue;
        __align__(16) TS c[4];
        *(int4*)c = *(const int4*)rp;
        if (o >= a.done_end) continue;               // a row that can never complete: left as it is
        *(int4*)rp = make_int4(0, 0, 0, 0);
        TO* op = out + (o - a.out_row_base) * a.out_row_stride + (long long)s * a.out_stream_stride + (long long)x * a.Cout + co;
        if (!IDF_OK_AT(a.status, (op - out) + 3, a.out_elems)) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) op[j] = Emit<TO, TS>::run(c[j], bias ? bias[co + j] : (TS)0, a.relu, a.shift);
    }
}

template <typename TI, typename TW, typename TS, typename TO>
static cudaError_t launch_rows(const ConvArgs& a, cudaStream_t st)
{
    if (a.r0 == a.r1 && a.r0 > 0 && a.Cout % 4 == 0 && a.o_end - a.o_begin <= a.ring_rows) {
        // no taps in this call: every visited row was started by earlier input rows
        const long long tot = (a.o_end - a.o_begin) * a.S * a.Wout * (a.Cout / 4);
        if (tot <= 0) return cudaSuccess;
        long long blocks = (tot + 255) / 256;
        if (blocks > 148LL * 64) blocks = 148LL * 64;
        conv_flush_kernel<TS, TO><<<(unsigned)blocks, 256, 0, st>>>(a);
        return cudaGetLastError();
    }
    const long long total = (long long)a.ring_rows * a.S * a.Wout * a.Cout;
    if (total == 0 || a.o_end <= a.o_begin) return cudaSuccess;
    long long blocks = (total + 255) / 256;
    if (blocks > 148LL * 64) blocks = 148LL * 64;
    // interior rows: not begun by an earlier block (first tap row o*stride - pad >= r0) and completed by this one
    long long int_begin = a.r0 > 0 ? (a.r0 + a.pad + a.stride - 1) / a.stride : a.o_begin;
    if (int_begin < a.o_begin) int_begin = a.o_begin;
    long long int_end = a.done_end;
    long long int_blocks = 0;
    if (int_end - int_begin >= 2LL * a.ring_rows) {
        const long long n_int = (int_end - int_begin) * a.S * a.Wout * a.Cout;
        int_blocks = (n_int + 255) / 256;
        if (int_blocks > 148LL * 64) int_blocks = 148LL * 64;
    } else {
        int_begin = int_end = 0;
    }
    conv_rows_kernel<TI, TW, TS, TO><<<(unsigned)(blocks + int_blocks), 256, 0, st>>>(a, int_begin, int_end, (unsigned)blocks);
    return cudaGetLastError();
}

template <typename TI, typename TW, typename TS, typename TO>
static cudaError_t launch_edges_t(const ConvArgs& a, long long skip_begin, long long skip_end, cudaStream_t st)
{
    const long long total = (long long)a.ring_rows * a.S * a.Wout * a.Cout;
    if (total == 0 || a.o_end <= a.o_begin) return cudaSuccess;
    long long blocks = (total + 255) / 256;
    if (blocks > 148LL * 64) blocks = 148LL * 64;
    conv_rows_kernel<TI, TW, TS, TO><<<(unsigned)blocks, 256, 0, st>>>(a, skip_begin, skip_end, (unsigned)blocks);
    return cudaGetLastError();
}

cudaError_t launch_conv_edges(const ConvArgs& a, int dtype, long long skip_begin, long long skip_end, cudaStream_t st)
{
    if (dtype == 0) return launch_edges_t<float, float, float, float>(a, skip_begin, skip_end, st);
    if (dtype == 1) {
        if (a.in_elem != E_BF16) return cudaErrorInvalidValue;
        if (a.out_elem == E_BF16) return launch_edges_t<__nv_bfloat16, float, float, __nv_bfloat16>(a, skip_begin, skip_end, st);
        return launch_edges_t<__nv_bfloat16, float, float, float>(a, skip_begin, skip_end, st);
    }
    return launch_edges_t<int8_t, int8_t, int, int8_t>(a, skip_begin, skip_end, st);
}

cudaError_t launch_conv_simple(const ConvArgs& a, int dtype, cudaStream_t st)
{
    if (dtype == 0) return launch_rows<float, float, float, float>(a, st);
    if (dtype == 1) {
        if (a.in_elem != E_BF16) return cudaErrorInvalidValue;
        if (a.out_elem == E_BF16) return launch_rows<__nv_bfloat16, float, float, __nv_bfloat16>(a, st);
        return launch_rows<__nv_bfloat16, float, float, float>(a, st);
    }
    return launch_rows<int8_t, int8_t, int, int8_t>(a, st);
}

// ------------------------------------------------------------------------------------------------
// Sparse-event path.  One CTA owns one stream and takes the block's input rows in order:
//   1. compaction: each warp looks at 32 input components at a time, ballots "non-zero", and
//      appends the survivors (position, channel, value) to a list in shared memory at the offset
//      given by the prefix popcount of the ballot (Eq. 3: only non-zero events are sent);
//   2. scatter: every (event, kernel tap, output channel) triple adds w*Δh to the ring row it
//      reaches (Eq. 4) with shared-memory atomics (or global atomics when the ring is too large
//      for shared memory; the ring of a stream is private to its CTA either way);
//   3. finalisation of the ring rows that this input row completed: emit f(c + b), zero the slot.
// Rows still open at the end of the block go back to the ring in global memory.
// ------------------------------------------------------------------------------------------------
constexpr int SPARSE_MAX_THREADS = 512;
constexpr int SPARSE_MAX_EVENTS = 1024;   // list capacity per pass; longer rows take several passes

template <typename TS> __device__ __forceinline__ void atomic_add(TS* p, TS v) { atomicAdd(p, v); }
// The same on an address known to lie in shared memory: a reduction in the shared state space (the generic
// form has to find out at run time which space the pointer belongs to).  No memory clobber: the statements are
// volatile, so they keep their order, and whoever reads the sums does so behind a __syncthreads().
__device__ __forceinline__ void atomic_add_shared(int* p, int v)
{
    asm volatile("red.shared.add.s32 [%0], %1;" ::"r"((uint32_t)__cvta_generic_to_shared(p)), "r"(v));
}
__device__ __forceinline__ void atomic_add_shared(float* p, float v)
{
    asm volatile("red.shared.add.f32 [%0], %1;" ::"r"((uint32_t)__cvta_generic_to_shared(p)), "f"(v));
}
constexpr int SPARSE_W_SMEM = 1024;       // weights of a thin layer (Kh*Kw*Cin*Cout values at most this many) are kept in shared memory

template <typename TI, typename TW, typename TS, typename TO, bool RING_IN_SMEM>
__global__ void __launch_bounds__(SPARSE_MAX_THREADS) conv_sparse_kernel(ConvArgs a)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ short ev_x[SPARSE_MAX_EVENTS], ev_ci[SPARSE_MAX_EVENTS];   // position and channel of the event
    __shared__ TS ev_val[SPARSE_MAX_EVENTS];
    __shared__ int ev_count[2];
    __shared__ unsigned long long ev_total;
    __shared__ TS w_s[SPARSE_W_SMEM];

    const int s = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31;
    const int SPARSE_THREADS = blockDim.x;      // 64 to 512 by row length: wide rows want many warps for the finalisation, short rows many small CTAs per SM
    const TI* __restrict__ in = (const TI*)a.in;
    const TW* __restrict__ w = (const TW*)a.w;
    const TS* __restrict__ bias = (const TS*)a.bias;
    TO* out = (TO*)a.out;
    const int row_elems = a.Wout * a.Cout;
    TS* gring = (TS*)a.ring;     // element (slot, s, x, co) at ((slot*S + s)*row_elems + x*Cout + co)
    TS* ring = RING_IN_SMEM ? (TS*)smem_raw : gring;
    const long long slot_stride = RING_IN_SMEM ? row_elems : (long long)a.S * row_elems;
    const long long ring_base = RING_IN_SMEM ? 0 : (long long)s * row_elems;

    if (tid == 0) { ev_total = 0; ev_count[0] = 0; ev_count[1] = 0; }
    const int n_w = a.Kh * a.Kw * a.Cin * a.Cout;
    const bool w_in_smem = n_w <= SPARSE_W_SMEM;
    if (w_in_smem)
        for (int i = tid; i < n_w; i += SPARSE_THREADS) w_s[i] = (TS)to_acc(w[i]);
    if (RING_IN_SMEM) {
        for (int i = tid; i < a.ring_rows * row_elems; i += SPARSE_THREADS) {
            const int slot = i / row_elems, e = i - slot * row_elems;
            const long long gi = ((long long)slot * a.S + s) * row_elems + e;
            if (IDF_OK_AT(a.status, gi, a.ring_elems)) ring[i] = gring[gi];
        }
    }
    __syncthreads();

    const int n_comp = a.Win * a.Cin;
    const int taps = a.Kh * a.Kw;
    const int slot0 = (int)(a.o_begin % a.ring_rows);     // ring slot of the first visited row
    // Row bookkeeping relative to the block (32-bit, stepping counters: a 64-bit division per row and thread costs as
    // much as the row's own work): rows are counted from o_begin, input rows from r0.
    int done = 0;                                    // visited rows below `done` have been emitted
    int done_slot = slot0;                           // ring slot of visited row `done`
    const int done_end_rel = (int)(a.done_end - a.o_begin), n_in = (int)(a.r1 - a.r0);
    const int c_q = (int)(a.r0 + a.pad - a.Kh - a.o_begin * a.stride);       // r + pad - Kh - o_begin*stride for r = r0
    // finalisation of the visited rows below `upto`: emit f(c + b), zero the slot
    auto finalise_upto = [&](int upto) {
        for (; done < upto; ++done) {
            const int slot = done_slot;
            if (++done_slot == a.ring_rows) done_slot = 0;
            TO* orow = out + (a.o_begin + done - a.out_row_base) * a.out_row_stride + (long long)s * a.out_stream_stride;
            if (!IDF_OK_AT(a.status, (orow - out) + row_elems - 1, a.out_elems) || !IDF_OK_AT(a.status, orow - out, a.out_elems) ||
                !IDF_OK_AT(a.status, (slot + 1) * (long long)row_elems - 1, (long long)a.ring_rows * row_elems)) continue;
            if (sizeof(TO) == 1 && (a.Cout & 3) == 0 && (((uintptr_t)orow) & 3) == 0) {
                // int8 rows: four channels per thread, one 4-byte store
                const bool pow2 = (a.Cout & (a.Cout - 1)) == 0;
                if (RING_IN_SMEM && !bias && a.relu) {
                    // the usual case (ReLU, no bias): max, rounding shift, min on four words, three byte permutes to pack
                    const int rnd = a.shift > 0 ? 1 << (a.shift - 1) : 0;
                    const int4* src = (const int4*)(smem_raw) + (int)slot * (row_elems >> 2);
                    uint32_t* dst = (uint32_t*)orow;
                    if (a.shift == 0) {
                        // no requantisation shift (first layers fed with small integers): clamp and pack only
                        for (int i = tid; i < (row_elems >> 2); i += SPARSE_THREADS) {
                            const int4 c = src[i];
                            ((int4*)src)[i] = make_int4(0, 0, 0, 0);
                            uint32_t hi2, all4;
                            asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, 0;" : "=r"(hi2) : "r"(c.w), "r"(c.z));
                            asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(all4) : "r"(c.y), "r"(c.x), "r"(hi2));
                            dst[i] = __vminu4(all4, 0x7f7f7f7fu);
                        }
                    } else
                    for (int i = tid; i < (row_elems >> 2); i += SPARSE_THREADS) {
                        const int4 c = src[i];
                        ((int4*)src)[i] = make_int4(0, 0, 0, 0);
                        // (c + rnd) >> shift is negative exactly when max(c, 0) + rnd >> shift would be 0 (c < 0 means
                        // c + rnd < 2^shift), so the ReLU is the saturating pack's lower bound; the upper bound is 127
                        const int v0 = (c.x + rnd) >> a.shift, v1 = (c.y + rnd) >> a.shift, v2 = (c.z + rnd) >> a.shift, v3 = (c.w + rnd) >> a.shift;
                        uint32_t hi2, all4;
                        asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, 0;" : "=r"(hi2) : "r"(v3), "r"(v2));
                        asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(all4) : "r"(v1), "r"(v0), "r"(hi2));
                        dst[i] = __vminu4(all4, 0x7f7f7f7fu);
                    }
                } else
                for (int i = tid * 4; i < row_elems; i += SPARSE_THREADS * 4) {
                    TS* p = &ring[ring_base + slot * slot_stride + i];
                    const int co = pow2 ? (i & (a.Cout - 1)) : i % a.Cout;
                    // (16-byte accesses: the ring row starts on a 16-byte boundary and i is a multiple of 4)
                    __align__(16) TS c[4];
                    *(int4*)c = *(const int4*)p;
                    *(int4*)p = make_int4(0, 0, 0, 0);
                    uint32_t pk = 0;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const TO v = Emit<TO, TS>::run(c[j], bias ? bias[co + j] : (TS)0, a.relu, a.shift);
                        pk |= ((uint32_t)(*(const unsigned char*)&v)) << (8 * j);
                    }
                    *(uint32_t*)(orow + i) = pk;
                }
            } else {
                for (int i = tid; i < row_elems; i += SPARSE_THREADS) {
                    TS* p = &ring[ring_base + slot * slot_stride + i];
                    const TS c = *p;
                    *p = 0;
                    const int co = i % a.Cout;
                    orow[i] = Emit<TO, TS>::run(c, bias ? bias[co] : (TS)0, a.relu, a.shift);
                }
            }
        }
    };
    // Per input row two block-wide phases: (A) the row's non-zero components are compacted into the event list
    // while the rows that the PREVIOUS input row completed are finalised (independent work: the loads of one
    // hide behind the arithmetic of the other); (B) the events are scattered into the ring.  The event
    // counter is double-buffered so that it can be cleared for the next pass while this one's is still read.
    const int cin_shift = (a.Cin & (a.Cin - 1)) == 0 ? 31 - __clz(a.Cin) : -1;     // (no division per event where Cin is a power of two)
    int cb = 0;
    int top_row = INT_MIN, top_slot = 0;             // 3x3 stride-1 scatter: the highest row the coming input row reaches, and its ring slot
    for (int rr = 0; rr <= n_in; ++rr) {
        // rr == n_in is the closing pass: no input, everything below done_end is finalised
        const bool have = rr < n_in;
        int upto = done_end_rel;
        if (have) {
            // row o completes at input row o*stride - pad + Kh - 1, here: <= r - 1; relative to o_begin:
            // floor((r + pad - Kh) / stride) + 1 - o_begin, not below 0
            const int q = rr + c_q;
            if (a.stride == 1) upto = q + 1;           // (a division per row and thread costs as much as the scatter of an event)
            else upto = q < 0 ? -((-q + a.stride - 1) / a.stride) + 1 : q / a.stride + 1;
            if (upto < 0) upto = 0;
            if (upto > done_end_rel) upto = done_end_rel;
        }
        const TI* row = in + ((long long)rr * a.S + s) * (long long)n_comp;
        if (have && !IDF_OK_AT(a.status, (row - in) + n_comp - 1, a.in_elems)) continue;
        const int n_pass = have ? (n_comp + SPARSE_MAX_EVENTS - 1) / SPARSE_MAX_EVENTS : 1;
        for (int pass = 0; pass < n_pass; ++pass) {
            const int base = pass * SPARSE_MAX_EVENTS;
            const int lim = min(n_comp, base + SPARSE_MAX_EVENTS);
            TS v_first = (TS)0;
            if (have && base + tid < lim) v_first = (TS)to_acc(row[base + tid]);      // in flight during the finalisation
            if (pass == 0) finalise_upto(upto);
            if (have) {
                for (int i0 = base + (tid - lane); i0 < lim; i0 += SPARSE_THREADS) {
                    const int i = i0 + lane;
                    const TS v = (i0 == base + (tid - lane)) ? v_first : ((i < lim) ? (TS)to_acc(row[i]) : (TS)0);
                    const unsigned m = __ballot_sync(0xffffffffu, v != (TS)0);
                    if (m) {
                        int off = 0;
                        if (lane == 0) off = atomicAdd(&ev_count[cb], __popc(m));
                        off = __shfl_sync(0xffffffffu, off, 0);
                        if (v != (TS)0) {
                            const int k = off + __popc(m & ((1u << lane) - 1u));
                            if (!IDF_OK_AT(a.status, k, SPARSE_MAX_EVENTS)) continue;
                            const int x = cin_shift >= 0 ? i >> cin_shift : i / a.Cin;
                            ev_x[k] = (short)x;
                            ev_ci[k] = (short)(i - x * a.Cin);
                            ev_val[k] = v;
                        }
                    }
                }
            }
            __syncthreads();
            if (have) {
                const int n_ev = ev_count[cb];
                if (tid == 0) { ev_total += (unsigned long long)n_ev; ev_count[cb ^ 1] = 0; }
            // scatter: a warp takes one event at a time and walks its kernel taps, the lanes take the output
            // channels; target row, ring slot and target x are worked out once per tap row / tap (no
            // per-channel index arithmetic, no division when the stride is 1)
            const int ty0 = rr + c_q + a.Kh;                                  // = r + pad - o_begin*stride: tap ky reaches relative row (ty0 - ky) / stride
            if (RING_IN_SMEM && w_in_smem && a.stride == 1 && a.stride_x == 1 && a.Kh == 3 && a.Kw == 3) {
                // the common 3x3, stride-1 case with everything in shared memory, unrolled: the three target rows'
                // slot offsets are worked out once per input row, a tap costs an address, a weight, a reduction
                // (the slot of row ty0 steps with the input row: three runtime modulos per row and thread took longer than
                // the events themselves)
                int soff[3];
                if (ty0 != top_row) { top_row = ty0; top_slot = ty0 >= 0 ? (slot0 + ty0) % a.ring_rows : 0; }
                {
                    int sl = top_slot;
#pragma unroll
                    for (int ky = 0; ky < 3; ++ky) {
                        soff[ky] = ty0 - ky >= 0 ? sl * row_elems : -1;
                        if (--sl < 0) sl = a.ring_rows - 1;
                    }
                }
                if (ty0 >= 0) {                                  // the next input row reaches one row further
                    ++top_row;
                    if (++top_slot == a.ring_rows) top_slot = 0;
                } else {
                    top_row = INT_MIN;
                }
                const int tap_w = a.Cin * a.Cout;
                TS* ring_s = (TS*)smem_raw;
                for (int e = tid >> 5; e < n_ev; e += SPARSE_THREADS / 32) {
                    const int x = ev_x[e] + a.pad_x;
                    const TS val = ev_val[e];
                    const TS* wp = w_s + ev_ci[e] * a.Cout;
                    for (int co = lane; co < a.Cout; co += 32) {
#pragma unroll
                        for (int ky = 0; ky < 3; ++ky) {
                            if (soff[ky] < 0) continue;
#pragma unroll
                            for (int kx = 0; kx < 3; ++kx) {
                                const int ox = x - kx;
                                if (ox < 0 || ox >= a.Wout) continue;
                                if (!IDF_OK_AT(a.status, soff[ky] + ox * a.Cout + co, (long long)a.ring_rows * row_elems)) continue;
                                atomic_add_shared(ring_s + soff[ky] + ox * a.Cout + co, val * wp[(ky * 3 + kx) * tap_w + co]);
                            }
                        }
                    }
                }
            } else
            for (int e = tid >> 5; e < n_ev; e += SPARSE_THREADS / 32) {
                const int x = ev_x[e], ci = ev_ci[e];
                const TS val = ev_val[e];
                for (int ky = 0; ky < a.Kh; ++ky) {
                    const int ty = ty0 - ky;
                    if (ty < 0) break;
                    int orel = ty;
                    if (a.stride != 1) { orel = ty / a.stride; if (orel * a.stride != ty) continue; }
                    const int slot = (slot0 + orel) % a.ring_rows;
                    TS* drow = &ring[ring_base + slot * slot_stride];
                    const int wrow_i = (ky * a.Kw * a.Cin + ci) * a.Cout;
                    const TW* wrow = w + wrow_i;
                    for (int kx = 0; kx < a.Kw; ++kx) {
                        const int tx = x + a.pad_x - kx;
                        if (tx < 0) break;
                        int ox = tx;
                        if (a.stride_x != 1) { ox = tx / a.stride_x; if (ox * a.stride_x != tx) continue; }
                        if (ox >= a.Wout) continue;
                        const int wofs = kx * a.Cin * a.Cout;
                        TS* dst = drow + ox * a.Cout;
                        if (!IDF_OK_AT(a.status, (dst - ring) + a.Cout - 1, RING_IN_SMEM ? (long long)a.ring_rows * row_elems : a.ring_elems)) continue;
                        for (int co = lane; co < a.Cout; co += 32) {
                            const TS wv = w_in_smem ? w_s[wrow_i + wofs + co] : (TS)to_acc(wrow[wofs + co]);
                            if (RING_IN_SMEM) atomic_add_shared(dst + co, val * wv);
                            else atomic_add(dst + co, val * wv);
                        }
                    }
                }
            }
                __syncthreads();
                cb ^= 1;
            }
        }
    }
    if (RING_IN_SMEM) {
        for (int i = tid; i < a.ring_rows * row_elems; i += SPARSE_THREADS) {
            const int slot = i / row_elems, e = i - slot * row_elems;
            const long long gi = ((long long)slot * a.S + s) * row_elems + e;
            if (IDF_OK_AT(a.status, gi, a.ring_elems)) gring[gi] = ring[i];
        }
    }
    if (tid == 0 && a.event_counter && ev_total) atomicAdd(a.event_counter, ev_total);
}

size_t conv_sparse_max_smem() { return 200 * 1024; }

template <typename TI, typename TW, typename TS, typename TO>
static cudaError_t launch_sparse_t(const ConvArgs& a, cudaStream_t st)
{
    if (a.S == 0) return cudaSuccess;
    const size_t ring_bytes = (size_t)a.ring_rows * a.Wout * a.Cout * sizeof(TS);
    const long long row_words = (long long)a.Wout * a.Cout;
    const int nthr = row_words >= 4096 ? SPARSE_MAX_THREADS : (row_words >= 1024 ? 256 : (row_words >= 512 ? 128 : 64));     // short rows: more, smaller CTAs per SM
    if (ring_bytes <= conv_sparse_max_smem()) {
        auto k = conv_sparse_kernel<TI, TW, TS, TO, true>;
        cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ring_bytes);
        if (e != cudaSuccess) return e;
        k<<<a.S, nthr, ring_bytes, st>>>(a);
    } else {
        conv_sparse_kernel<TI, TW, TS, TO, false><<<a.S, nthr, 0, st>>>(a);
    }
    return cudaGetLastError();
}

cudaError_t launch_conv_sparse(const ConvArgs& a, int dtype, cudaStream_t st)
{
    // (the event list keeps positions and channels in 16 bits; beyond that the dense kernel gives the same result)
    if (a.Win > 32767 || a.Cin > 32767) return launch_conv_simple(a, dtype, st);
    if (dtype == 0) return launch_sparse_t<float, float, float, float>(a, st);
    if (dtype == 1) {
        if (a.in_elem != E_BF16) return cudaErrorInvalidValue;
        if (a.out_elem == E_BF16) return launch_sparse_t<__nv_bfloat16, float, float, __nv_bfloat16>(a, st);
        return launch_sparse_t<__nv_bfloat16, float, float, float>(a, st);
    }
    return launch_sparse_t<int8_t, int8_t, int, int8_t>(a, st);
}

// ------------------------------------------------------------------------------------------------
// x-unfold in front of the tensor-core kernel for thin or x-strided layers: every output position
// gets its Kw*Cin input values side by side (zero padded to kpad), so that the channel contraction
// has a K the tensor cores accept and needs no stride in x.  One thread writes 16 bytes.
// ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) unfold_rows_kernel(const T* __restrict__ in, T* __restrict__ out, long long n_pos,
                                                          int Win, int Wout, int Cin, int Kw, int stride_x, int pad_x, int kpad,
                                                          long long in_elems, unsigned int* status)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    constexpr int V = 16 / (int)sizeof(T);
    const int vecs = kpad / V;
    const long long total = n_pos * vecs;
    const bool vec_ok = (Cin % V) == 0 && (((uintptr_t)in) & 15) == 0;     // channels of a position in whole 16-byte groups
    const bool small = total <= 0x7fffffffLL;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        // (v, x', (row, stream)) of this 16-byte piece; in 32 bits where the launch allows: the four 64-bit divisions
        // cost more than the copy
        int v, xo;
        long long p, rs;
        if (small) {
            const unsigned int i = (unsigned int)idx, pp = i / (unsigned int)vecs, r = pp / (unsigned int)Wout;
            v = (int)(i - pp * (unsigned int)vecs);
            xo = (int)(pp - r * (unsigned int)Wout);
            p = pp; rs = r;
        } else {
            v = (int)(idx % vecs);
            p = idx / vecs;                          // (row, stream, x') flattened
            xo = (int)(p % Wout);
            rs = p / Wout;                           // (row, stream)
        }
        const T* row = in + rs * (long long)Win * Cin;
        __align__(16) T vals[V];
        if (vec_ok) {
            // a 16-byte group never straddles two taps: it is one aligned 16-byte piece of an input position
            const int k0 = v * V;
            const int kx = k0 / Cin, ci = k0 - kx * Cin;
            const int ix = xo * stride_x - pad_x + kx;
            int4 q = make_int4(0, 0, 0, 0);
            if (kx < Kw && ix >= 0 && ix < Win && IDF_OK_AT(status, (row - in) + (long long)ix * Cin + ci + V - 1, in_elems))
                q = *(const int4*)(row + (long long)ix * Cin + ci);
            *(int4*)(out + p * kpad + (long long)v * V) = q;
            continue;
        }
        // the Kw*Cin values of an output position are one contiguous run of the input row, starting at position
        // xo*stride - pad: element k of the run lies outside the row exactly when its position does
        const int e0 = (xo * stride_x - pad_x) * Cin + v * V;
        const int k_end = Kw * Cin - v * V, e_end = Win * Cin;
#pragma unroll
        for (int j = 0; j < V; ++j) {
            const int e = e0 + j;
            vals[j] = (j < k_end && e >= 0 && e < e_end && IDF_OK_AT(status, (row - in) + e, in_elems)) ? row[e] : (T)0;
        }
        *(int4*)(out + p * kpad + (long long)v * V) = *(const int4*)vals;
    }
}

// The same for layers whose positions are not whole 16-byte groups (three channels, say), where the kernel above would
// fetch every value with a load of its own: a block takes one input row of one stream at a time, brings it into shared
// memory with 16-byte loads, and every thread puts its 16-byte pieces together from there.
constexpr int UNFOLD_ROW_BYTES = 16384;      // longest input row this form takes
template <typename T>
__global__ void __launch_bounds__(256) unfold_rows_staged_kernel(const T* __restrict__ in, T* __restrict__ out, int n_rs,
                                                                 int Win, int Wout, int Cin, int Kw, int stride_x, int pad_x, int kpad,
                                                                 long long in_elems, unsigned int* status)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    __shared__ __align__(16) unsigned char raw[UNFOLD_ROW_BYTES];
    constexpr int V = 16 / (int)sizeof(T);
    const int vecs = kpad / V;
    const int row_elems = Win * Cin, n16 = row_elems * (int)sizeof(T) / 16, pieces = Wout * vecs;
    const int k_all = Kw * Cin;
    const T* rawT = (const T*)raw;
    for (int rs = blockIdx.x; rs < n_rs; rs += gridDim.x) {
        const T* row = in + (long long)rs * row_elems;
        if (IDF_OK_AT(status, (long long)rs * row_elems + row_elems - 1, in_elems))
            for (int i = threadIdx.x; i < n16; i += 256) ((int4*)raw)[i] = ((const int4*)row)[i];
        __syncthreads();
        T* orow = out + (long long)rs * Wout * kpad;
        for (int pc = threadIdx.x; pc < pieces; pc += 256) {
            const int xo = pc / vecs, v = pc - xo * vecs;
            const int e0 = (xo * stride_x - pad_x) * Cin + v * V, k_end = k_all - v * V;
            __align__(16) T vals[V];
#pragma unroll
            for (int j = 0; j < V; ++j) {
                const int e = e0 + j;
                vals[j] = (j < k_end && e >= 0 && e < row_elems) ? rawT[e] : (T)0;
            }
            ((int4*)orow)[pc] = *(const int4*)vals;
        }
        __syncthreads();
    }
}

cudaError_t launch_unfold(const ConvArgs& a, int n_rows, int kpad, void* out, cudaStream_t st)
{
    const long long n_pos = (long long)n_rows * a.S * a.Wout;
    if (n_pos == 0) return cudaSuccess;
    const int esize = a.in_elem == E_BF16 ? 2 : 1;
    const long long total = n_pos * (kpad * esize / 16);
    long long blocks = (total + 255) / 256;
    if (blocks > 148LL * 32) blocks = 148LL * 32;
    // rows whose positions are not whole 16-byte groups: staged through shared memory, a block per (row, stream)
    const long long n_rs = (long long)n_rows * a.S;
    const long long row_bytes = (long long)a.Win * a.Cin * esize;
    if ((a.Cin * esize) % 16 != 0 && row_bytes % 16 == 0 && row_bytes <= UNFOLD_ROW_BYTES && (((uintptr_t)a.in) & 15) == 0 &&
        n_rs <= 0x7fffffffLL && (long long)a.Wout * (kpad * esize / 16) <= 0x7fffffffLL) {
        const unsigned grid = (unsigned)(n_rs < 148LL * 8 ? n_rs : 148LL * 8);
        if (a.in_elem == E_BF16)
            unfold_rows_staged_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)a.in, (__nv_bfloat16*)out, (int)n_rs, a.Win, a.Wout,
                                                                         a.Cin, a.Kw, a.stride_x, a.pad_x, kpad, a.in_elems, a.status);
        else if (a.in_elem == E_I8)
            unfold_rows_staged_kernel<int8_t><<<grid, 256, 0, st>>>((const int8_t*)a.in, (int8_t*)out, (int)n_rs, a.Win, a.Wout, a.Cin, a.Kw,
                                                                  a.stride_x, a.pad_x, kpad, a.in_elems, a.status);
        else
            return cudaErrorInvalidValue;
        return cudaGetLastError();
    }
    if (a.in_elem == E_BF16)
        unfold_rows_kernel<__nv_bfloat16><<<(unsigned)blocks, 256, 0, st>>>((const __nv_bfloat16*)a.in, (__nv_bfloat16*)out, n_pos,
                                                                          a.Win, a.Wout, a.Cin, a.Kw, a.stride_x, a.pad_x, kpad, a.in_elems, a.status);
    else if (a.in_elem == E_I8)
        unfold_rows_kernel<int8_t><<<(unsigned)blocks, 256, 0, st>>>((const int8_t*)a.in, (int8_t*)out, n_pos, a.Win, a.Wout,
                                                                   a.Cin, a.Kw, a.stride_x, a.pad_x, kpad, a.in_elems, a.status);
    else
        return cudaErrorInvalidValue;
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Max-pool fold: the x-pair is reduced at once; the first row of a y-pair waits in a one-row
// running maximum; the second row emits.  Width-1 maps pool over rows only.
// ------------------------------------------------------------------------------------------------
template <typename T> __device__ __forceinline__ T max_of(T a, T b) { return a > b ? a : b; }
template <> __device__ __forceinline__ __nv_bfloat16 max_of(__nv_bfloat16 a, __nv_bfloat16 b)
{
    return __bfloat162float(a) > __bfloat162float(b) ? a : b;
}

template <typename T>
__global__ void __launch_bounds__(256) pool_rows_kernel(PoolArgs a)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const T* __restrict__ in = (const T*)a.in;
    T* state = (T*)a.state;
    T* out = (T*)a.out;
    const int px = (a.Win == 1) ? 1 : 2;
    const long long total = (long long)a.S * a.Wout * a.C;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(idx % a.C);
        long long t = idx / a.C;
        const int ox = (int)(t % a.Wout);
        const int s = (int)(t / a.Wout);
        for (long long o = a.o_begin; o < a.o_end; ++o) {
            bool have = false;
            T m = (T)0;
            if (!IDF_OK_AT(a.status, idx, a.state_elems)) continue;
            if (2 * o < a.r0) { m = state[idx]; have = true; }
            for (int dy = 0; dy < 2; ++dy) {
                const long long r = 2 * o + dy;
                if (r < a.r0 || r >= a.r1) continue;
                const T* row = in + ((r - a.r0) * a.S + s) * (long long)a.Win * a.C;
                for (int dx = 0; dx < px; ++dx) {
                    if (!IDF_OK_AT(a.status, (row - in) + (long long)(px * ox + dx) * a.C + c, a.in_elems)) continue;
                    const T v = row[(long long)(px * ox + dx) * a.C + c];
                    m = have ? max_of(m, v) : v;
                    have = true;
                }
            }
            const long long oi = (o - a.out_row_base) * a.out_row_stride + (long long)s * a.out_stream_stride + (long long)ox * a.C + c;
            if (o < a.done_end) { if (IDF_OK_AT(a.status, oi, a.out_elems)) out[oi] = m; }
            else state[idx] = m;
        }
    }
}

// 16 bytes of channels per thread (the layout is channels-innermost, so a position's channels are
// contiguous): the same fold, vectorised, with a thread per output row.  Used when C * sizeof(T) is a
// multiple of 16.  The one state row can be read (the first visited row, when its first half came with an
// earlier launch) and written (the last visited row, when its second half is still to come) in the same
// launch; when both happen the reading thread also handles the writing row, after its own, so the two
// accesses to a state element are ordered inside one thread whatever the CTAs' order.
template <typename T>
__global__ void __launch_bounds__(256) pool_rows_vec_kernel(PoolArgs a)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    constexpr int V = 16 / (int)sizeof(T);
    const T* __restrict__ in = (const T*)a.in;
    T* state = (T*)a.state;
    T* out = (T*)a.out;
    const int px = (a.Win == 1) ? 1 : 2;
    const int cv = a.C / V;
    long long n_o = a.o_end - a.o_begin;
    const bool carried_in = 2 * a.o_begin < a.r0;
    const bool carried_out = a.o_end - 1 >= a.done_end;
    const bool chained = carried_in && carried_out && n_o >= 2;     // the first row's thread takes the last row too
    if (chained) n_o -= 1;
    const long long total = n_o * a.S * a.Wout * cv;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(idx % cv) * V;
        long long t = idx / cv;
        const int ox = (int)(t % a.Wout);
        t /= a.Wout;
        const int s = (int)(t % a.S);
        long long o = a.o_begin + t / a.S;
        const long long sidx = ((long long)s * a.Wout + ox) * a.C + c;
        for (int turn = 0; turn < 2; ++turn) {
            __align__(16) T m[V];
            bool have = false;
            if (!IDF_OK_AT(a.status, sidx + V - 1, a.state_elems)) break;
            if (2 * o < a.r0) { *(int4*)m = *(const int4*)(state + sidx); have = true; }
            for (int dy = 0; dy < 2; ++dy) {
                const long long r = 2 * o + dy;
                if (r < a.r0 || r >= a.r1) continue;
                const T* row = in + ((r - a.r0) * a.S + s) * (long long)a.Win * a.C;
                for (int dx = 0; dx < px; ++dx) {
                    __align__(16) T v[V];
                    if (!IDF_OK_AT(a.status, (row - in) + (long long)(px * ox + dx) * a.C + c + V - 1, a.in_elems)) continue;
                    *(int4*)v = *(const int4*)(row + (long long)(px * ox + dx) * a.C + c);
#pragma unroll
                    for (int j = 0; j < V; ++j) m[j] = have ? max_of(m[j], v[j]) : v[j];
                    have = true;
                }
            }
            const long long oi = (o - a.out_row_base) * a.out_row_stride + (long long)s * a.out_stream_stride + (long long)ox * a.C + c;
            if (o < a.done_end) { if (IDF_OK_AT(a.status, oi + V - 1, a.out_elems)) *(int4*)(out + oi) = *(const int4*)m; }
            else *(int4*)(state + sidx) = *(const int4*)m;
            if (!(chained && o == a.o_begin)) break;
            o = a.o_end - 1;
        }
    }
}

template <typename T>
static cudaError_t launch_pool_t(const PoolArgs& a, cudaStream_t st)
{
    const long long total = (long long)a.S * a.Wout * a.C;
    if (total == 0 || a.o_end <= a.o_begin) return cudaSuccess;
    constexpr int V = 16 / (int)sizeof(T);
    const bool aligned = (a.C % V == 0) && (((uintptr_t)a.in | (uintptr_t)a.out | (uintptr_t)a.state) & 15) == 0 &&
                         ((a.out_row_stride | a.out_stream_stride) % V == 0);
    // (the vector kernel gives each output row a thread; it orders the one read and the one write of the state
    // row itself, see there)
    if (aligned) {
        const long long tv = (a.o_end - a.o_begin) * a.S * a.Wout * (a.C / V);
        long long blocks = (tv + 255) / 256;
        if (blocks > 148LL * 64) blocks = 148LL * 64;
        pool_rows_vec_kernel<T><<<(unsigned)blocks, 256, 0, st>>>(a);
        return cudaGetLastError();
    }
    long long blocks = (total + 255) / 256;
    if (blocks > 148LL * 32) blocks = 148LL * 32;
    pool_rows_kernel<T><<<(unsigned)blocks, 256, 0, st>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_pool(const PoolArgs& a, cudaStream_t st)
{
    switch (a.elem) {
        case E_F32: return launch_pool_t<float>(a, st);
        case E_BF16: return launch_pool_t<__nv_bfloat16>(a, st);
        case E_I8: return launch_pool_t<int8_t>(a, st);
        default: return cudaErrorInvalidValue;
    }
}

// ------------------------------------------------------------------------------------------------
// Global-average sink (the averaging output unit of the paper's Fig. 1): c_out += dh for every
// arriving value, one running sum per (stream, channel); the mean over the positions received so
// far is written after every launch, so the output can be read at any time.
// One thread per (stream, channel); channels are innermost, so a warp reads consecutive addresses.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ float avg_term(float v) { return v; }
__device__ __forceinline__ float avg_term(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ int avg_term(int8_t v) { return (int)v; }

template <typename TI, typename TS>
__global__ void __launch_bounds__(256) avg_rows_kernel(AvgArgs a)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const TI* __restrict__ in = (const TI*)a.in;
    TS* sum = (TS*)a.sum;
    const long long total = (long long)a.S * a.C;
    const double count = (double)a.rows_total * (double)a.W;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(idx % a.C);
        const long long s = idx / a.C;
        if (!IDF_OK_AT(a.status, idx, a.sum_elems)) continue;
        TS acc = sum[idx];
        for (long long r = 0; r < a.n_rows; ++r) {
            const TI* row = in + (r * a.S + s) * (long long)a.W * a.C + c;
            if (!IDF_OK_AT(a.status, (row - in) + (long long)(a.W - 1) * a.C, a.in_elems)) continue;
            for (int x = 0; x < a.W; ++x) acc += avg_term(row[(long long)x * a.C]);
        }
        sum[idx] = acc;
        if (IDF_OK_AT(a.status, s * a.out_stream_stride + c, a.out_elems)) a.out[s * a.out_stream_stride + c] = (float)((double)acc / count);
    }
}
cudaError_t launch_avg(const AvgArgs& a, cudaStream_t st)
{
    const long long total = (long long)a.S * a.C;
    if (total == 0 || a.n_rows <= 0) return cudaSuccess;
    long long blocks = (total + 255) / 256;
    if (blocks > 148LL * 32) blocks = 148LL * 32;
    switch (a.elem) {
        case E_F32: avg_rows_kernel<float, float><<<(unsigned)blocks, 256, 0, st>>>(a); break;
        case E_BF16: avg_rows_kernel<__nv_bfloat16, float><<<(unsigned)blocks, 256, 0, st>>>(a); break;
        case E_I8: avg_rows_kernel<int8_t, int><<<(unsigned)blocks, 256, 0, st>>>(a); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

}  // namespace idf
