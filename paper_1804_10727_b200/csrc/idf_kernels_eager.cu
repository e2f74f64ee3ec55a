// Eager (anytime) emission: the paper's literal rule, one segment at a time.
//
// Every unit keeps its state c (Eq. 2) and the activation it last announced.  After a segment has
// been applied, a unit whose activation f(c) differs from the announced one sends the difference
// dh = h(t) - h(t-1) to the layer above (Eq. 3), which adds w * dh to its own states (Eq. 4) and
// re-evaluates in turn (Eq. 5 and the sentence after it), layer by layer, within the same push.  So
// the net's output is available - and converges - while the input still arrives (Section
// "Experimental verification").  Units announce partial sums here, so a layer keeps every row that
// present or future input can still reach: the rows of the input cone, not just ceil(Kh/stride).
//
// Per layer three rings of `cap` rows (slot = row mod cap), 32-bit words (fp32 / int32):
//   c  the state variable,  h  the announced activation,  d  the change announced in this push.
// A push of one segment touches, in every layer, exactly the rows whose receptive field contains
// that segment; the host works the row intervals out and launches one kernel per layer.
#include "idf_internal.h"

namespace idf {

namespace {

__device__ __forceinline__ float eager_act(float c, float b, int relu, int, int round_bf16)
{
    float v = c + b;
    if (relu && v < 0.f) v = 0.f;
    if (round_bf16) v = __bfloat162float(__float2bfloat16_rn(v));
    return v;
}
__device__ __forceinline__ int eager_act(int c, int b, int relu, int shift, int)
{
    int v = c + b;
    if (relu && v < 0) v = 0;
    if (shift > 0) v = (v + (1 << (shift - 1))) >> shift;
    const int lo = relu ? 0 : -127;
    return v < lo ? lo : (v > 127 ? 127 : v);
}
__device__ __forceinline__ float w_val(float w) { return w; }
__device__ __forceinline__ int w_val(int8_t w) { return (int)w; }

// one count per warp instead of one atomic per thread
__device__ __forceinline__ void count_events(unsigned long long* counter, bool nonzero)
{
    const unsigned m = __ballot_sync(__activemask(), nonzero);
    if (counter && m && (threadIdx.x & 31) == (__ffs(m) - 1)) atomicAdd(counter, (unsigned long long)__popc(m));
}

__device__ __forceinline__ void write_out(const EagerArgs& a, long long o, int s, int x, int co, float h)
{
    const long long i = (long long)s * a.out_stream_stride + o * a.out_row_stride + (long long)x * a.Cout + co;
    if (IDF_OK_AT(a.status, i, a.out_elems)) ((float*)a.out)[i] = h;
}
__device__ __forceinline__ void write_out(const EagerArgs& a, long long o, int s, int x, int co, int h)
{
    const long long i = (long long)s * a.out_stream_stride + o * a.out_row_stride + (long long)x * a.Cout + co;
    if (IDF_OK_AT(a.status, i, a.out_elems)) ((int8_t*)a.out)[i] = (int8_t)h;
}

// The pushed segment as the input layer's announcement: input units start at 0, so dh = x (paragraph after Eq. 3).
template <typename TI, typename TS>
__global__ void __launch_bounds__(256) eager_input_kernel(const TI* __restrict__ in, TS* __restrict__ d, long long n,
                                                          unsigned long long* events)
{
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < (n + 31) / 32 * 32;
         i += (long long)gridDim.x * blockDim.x) {
        TS v = 0;
        if (i < n) {
            if constexpr (sizeof(TI) == 2) v = (TS)__bfloat162float(in[i]);
            else v = (TS)in[i];
            d[i] = v;
        }
        count_events(events, v != (TS)0);
    }
}

// Conv layer: rows [o_lo, o_hi] take up the changes of rows [in_lo, in_hi] of the layer below (Eq. 4, zero
// changes skipped), re-evaluate, and announce their own change (Eq. 3).  One thread per unit.
template <typename TS, typename TW>
__global__ void __launch_bounds__(256) eager_conv_kernel(EagerArgs a)
{
    const TS* __restrict__ din = (const TS*)a.din;
    const TW* __restrict__ w = (const TW*)a.w;
    const TS* __restrict__ bias = (const TS*)a.bias;
    TS* cr = (TS*)a.c;
    TS* hr = (TS*)a.h;
    TS* dr = (TS*)a.d;
    const long long row_elems = (long long)a.Wout * a.Cout;
    const long long n = (a.o_hi - a.o_lo + 1) * a.S * row_elems;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < (n + 31) / 32 * 32;
         idx += (long long)gridDim.x * blockDim.x) {
        bool emitted = false;
        if (idx < n) {
            const int co = (int)(idx % a.Cout);
            long long t = idx / a.Cout;
            const int x = (int)(t % a.Wout);
            t /= a.Wout;
            const int s = (int)(t % a.S);
            const long long o = a.o_lo + t / a.S;
            TS acc = 0;
            if (a.in_lo <= a.in_hi)
                for (int ky = 0; ky < a.Kh; ++ky) {
                    const long long i = o * a.stride - a.pad + ky;
                    if (i < a.in_lo || i > a.in_hi) continue;
                    const TS* drow = din + ((i % a.cap_in) * a.S + s) * (long long)a.Win * a.Cin;
                    if (!IDF_OK_AT(a.status, (drow - din) + (long long)a.Win * a.Cin - 1, a.in_elems)) continue;
                    for (int kx = 0; kx < a.Kw; ++kx) {
                        const int ix = x * a.stride_x - a.pad_x + kx;
                        if (ix < 0 || ix >= a.Win) continue;
                        const TS* dp = drow + (long long)ix * a.Cin;
                        const TW* wp = w + ((long long)(ky * a.Kw + kx) * a.Cin) * a.Cout + co;
                        for (int ci = 0; ci < a.Cin; ++ci) {
                            const TS dv = dp[ci];
                            if (dv != (TS)0) acc += w_val(wp[(long long)ci * a.Cout]) * dv;     // only non-zero events cost work
                        }
                    }
                }
            const long long e = (((o % a.cap) * a.S + s) * a.Wout + x) * (long long)a.Cout + co;
            if (!IDF_OK_AT(a.status, e, a.ring_elems)) continue;
            const bool fresh = o >= a.o_new;                        // first touch: the slot still holds an older row
            const TS cn = (fresh ? (TS)0 : cr[e]) + acc;
            const TS hold = fresh ? (TS)0 : hr[e];
            const TS hn = o >= a.o_cut ? (TS)0 : eager_act(cn, bias ? bias[co] : (TS)0, a.relu, a.shift, a.round_bf16);
            cr[e] = cn;
            hr[e] = hn;
            dr[e] = hn - hold;
            emitted = hn != hold;
            if (a.out) write_out(a, o, s, x, co, hn);
        }
        count_events(a.events, emitted);
    }
}

// Max-pool unit: it holds its four current inputs (the announced activations of the layer below, 0 for units
// that have not announced anything yet) and announces max_new - max_old.
template <typename TS>
__global__ void __launch_bounds__(256) eager_pool_kernel(EagerArgs a)
{
    const TS* __restrict__ hin = (const TS*)a.hin;
    TS* hr = (TS*)a.h;
    TS* dr = (TS*)a.d;
    const int px = a.Win == 1 ? 1 : 2;
    const long long row_elems = (long long)a.Wout * a.Cout;
    const long long n = (a.o_hi - a.o_lo + 1) * a.S * row_elems;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < (n + 31) / 32 * 32;
         idx += (long long)gridDim.x * blockDim.x) {
        bool emitted = false;
        if (idx < n) {
            const int c = (int)(idx % a.Cout);
            long long t = idx / a.Cout;
            const int x = (int)(t % a.Wout);
            t /= a.Wout;
            const int s = (int)(t % a.S);
            const long long o = a.o_lo + t / a.S;
            TS m = 0;
            bool have = false;
            for (int dy = 0; dy < 2; ++dy) {
                const long long i = 2 * o + dy;
                for (int dx = 0; dx < px; ++dx) {
                    TS v = 0;                                          // a unit that has announced nothing stands at 0
                    const long long hi_at = (((i % a.cap_in) * a.S + s) * a.Win + (px * x + dx)) * (long long)a.Cin + c;
                    if (i <= a.in_hi && IDF_OK_AT(a.status, hi_at, a.in_elems)) v = hin[hi_at];
                    m = have ? (v > m ? v : m) : v;
                    have = true;
                }
            }
            const long long e = (((o % a.cap) * a.S + s) * a.Wout + x) * (long long)a.Cout + c;
            if (!IDF_OK_AT(a.status, e, a.ring_elems)) continue;
            const TS hold = o >= a.o_new ? (TS)0 : hr[e];
            const TS hn = o >= a.o_cut ? (TS)0 : m;
            hr[e] = hn;
            dr[e] = hn - hold;
            emitted = hn != hold;
            if (a.out) write_out(a, o, s, x, c, hn);
        }
        count_events(a.events, emitted);
    }
}

unsigned blocks_for(long long n)
{
    long long b = (n + 255) / 256;
    return (unsigned)(b < 1 ? 1 : (b > 148LL * 32 ? 148LL * 32 : b));
}

}  // namespace

cudaError_t launch_eager_input(const void* in, int in_elem, void* d, long long n, unsigned long long* events, cudaStream_t st)
{
    if (n <= 0) return cudaSuccess;
    switch (in_elem) {
        case E_F32: eager_input_kernel<float, float><<<blocks_for(n), 256, 0, st>>>((const float*)in, (float*)d, n, events); break;
        case E_BF16: eager_input_kernel<__nv_bfloat16, float><<<blocks_for(n), 256, 0, st>>>((const __nv_bfloat16*)in, (float*)d, n, events); break;
        case E_I8: eager_input_kernel<int8_t, int><<<blocks_for(n), 256, 0, st>>>((const int8_t*)in, (int*)d, n, events); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

cudaError_t launch_eager_layer(const EagerArgs& a, int is_pool, int int_net, cudaStream_t st)
{
    if (a.o_hi < a.o_lo) return cudaSuccess;
    const long long n = (a.o_hi - a.o_lo + 1) * a.S * (long long)a.Wout * a.Cout;
    if (is_pool) {
        if (int_net) eager_pool_kernel<int><<<blocks_for(n), 256, 0, st>>>(a);
        else eager_pool_kernel<float><<<blocks_for(n), 256, 0, st>>>(a);
    } else {
        if (int_net) eager_conv_kernel<int, int8_t><<<blocks_for(n), 256, 0, st>>>(a);
        else eager_conv_kernel<float, float><<<blocks_for(n), 256, 0, st>>>(a);
    }
    return cudaGetLastError();
}

}  // namespace idf
