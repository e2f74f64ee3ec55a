// Depth-first over ALL layers in one launch, with every layer's rolling state on chip.
//
// The paper pushes each arriving segment through the whole net before the next one is looked at, and
// keeps only the partial activations that present or future input can still influence (Section
// "Asynchronous incremental updates", first paragraph; Discussion: "activation subset buffers").  For
// nets whose per-stream state is small this kernel does exactly that on one SM: a CTA owns a group of
// streams, loads their rings (and pooling rows) into shared memory, and then takes the pushed
// segments one at a time: the segment's events update the first layer's ring rows (Eq. 4), a row
// that is complete is finalised (Eq. 2-3) into a shared-memory row buffer, which is the next layer's
// input at once, and so on up to the output row, which is the only thing written to global memory
// besides the state at the end of the launch.  Between layers nothing leaves the SM.
//
// State in global memory has the layout of the per-layer kernels (rings [slot][stream][x][c] of
// 32-bit words without the bias, pooling rows [stream][x][c] in the layer's element type), so a
// stream may be advanced by this kernel and by the per-layer kernels in turn.
#include "idf_internal.h"

namespace idf {

namespace {

template <typename TS> struct WeightOf;
template <> struct WeightOf<float> { typedef float T; };
template <> struct WeightOf<int> { typedef int8_t T; };

__device__ __forceinline__ float fused_act(float c, float b, int relu, int, int round_bf16)
{
    float v = c + b;
    if (relu && v < 0.f) v = 0.f;
    if (round_bf16) v = __bfloat162float(__float2bfloat16_rn(v));
    return v;
}
__device__ __forceinline__ int fused_act(int c, int b, int relu, int shift, int)
{
    int v = c + b;
    if (relu && v < 0) v = 0;
    if (shift > 0) v = (v + (1 << (shift - 1))) >> shift;
    const int lo = relu ? 0 : -127;
    return v < lo ? lo : (v > 127 ? 127 : v);
}
__device__ __forceinline__ float fw(float w) { return w; }
__device__ __forceinline__ int fw(int8_t w) { return (int)w; }

template <typename TS>
__device__ __forceinline__ TS load_elem(const void* p, long long i, int elem)
{
    if (elem == E_F32) return (TS)((const float*)p)[i];
    if (elem == E_BF16) return (TS)__bfloat162float(((const __nv_bfloat16*)p)[i]);
    return (TS)((const int8_t*)p)[i];
}
template <typename TS>
__device__ __forceinline__ void store_elem(void* p, long long i, int elem, TS v)
{
    if (elem == E_F32) ((float*)p)[i] = (float)v;
    else if (elem == E_BF16) ((__nv_bfloat16*)p)[i] = __float2bfloat16_rn((float)v);
    else ((int8_t*)p)[i] = (int8_t)v;
}

// Layer i takes the row `in` ([G][Win][Cin] words in shared memory) as its input row number rows_in[i].
// Returns true if it completed a row, which then stands in the layer's row buffer.
template <typename TS>
__device__ bool fused_feed(const FusedArgs& a, int i, const TS* in, TS* smem, long long* rows_in, long long* rows_done,
                           int G, int g0, unsigned long long* ev_local)
{
    typedef typename WeightOf<TS>::T TW;
    const FusedLayer& L = a.layer[i];
    const long long r = rows_in[i];
    rows_in[i] = r + 1;
    TS* rowbuf = smem + L.rowbuf_soff;
    if (L.count_events) {
        // the layer's input events: the non-zero components of the row (Eq. 3)
        unsigned n = 0;
        for (int e = threadIdx.x; e < G * L.Win * L.Cin; e += blockDim.x) n += in[e] != (TS)0;
        for (int o = 16; o; o >>= 1) n += __shfl_xor_sync(0xffffffffu, n, o);
        if ((threadIdx.x & 31) == 0 && n) atomicAdd(&ev_local[i], (unsigned long long)n);
    }
    if (L.kind == 1) {
        // 2x2 max-pool fold: the x-pooled first row of a pair waits in the pool state
        TS* st = smem + L.state_soff;
        const int px = L.Win == 1 ? 1 : 2;
        const bool second = (r & 1) != 0;
        for (int e = threadIdx.x; e < G * L.Wout * L.Cout; e += blockDim.x) {
            const int c = e % L.Cout, t = e / L.Cout, x = t % L.Wout, g = t / L.Wout;
            const TS* p = in + ((g * L.Win + px * x) * L.Cin + c);
            TS m = p[0];
            if (px == 2) { const TS v = p[L.Cin]; m = v > m ? v : m; }
            if (second) { const TS f = st[e]; rowbuf[e] = f > m ? f : m; }
            else st[e] = m;
        }
        __syncthreads();
        if (second) rows_done[i] += 1;
        return second;
    }
    // conv: Eq. 4 for every event of the row, tap by tap, then Eq. 2-3 for the row this input row completes
    const TW* __restrict__ w = (const TW*)a.weights + L.w_off;
    const TS* __restrict__ bias = L.bias_off >= 0 ? (const TS*)((const unsigned char*)a.weights + L.bias_off) : nullptr;
    TS* ring = smem + L.state_soff;
    const int row_elems = L.Wout * L.Cout;
    const long long o_hi = (r + L.pad) / L.stride;
    long long o_lo = r + L.pad - L.Kh + 1;
    o_lo = o_lo <= 0 ? 0 : (o_lo + L.stride - 1) / L.stride;
    const long long tf = r + L.pad - (L.Kh - 1);
    const bool completes = tf >= 0 && tf % L.stride == 0;           // output row tf / stride has now received its last tap
    const long long o_done = completes ? tf / L.stride : -1;
    for (int e = threadIdx.x; e < G * row_elems; e += blockDim.x) {
        const int co = e % L.Cout, t = e / L.Cout, x = t % L.Wout, g = t / L.Wout;
        for (long long o = o_lo; o <= o_hi; ++o) {
            const int ky = (int)(r + L.pad - o * L.stride);
            TS acc = 0;
            for (int kx = 0; kx < L.Kw; ++kx) {
                const int ix = x * L.stride_x - L.pad_x + kx;
                if (ix < 0 || ix >= L.Win) continue;
                const TS* ip = in + (g * L.Win + ix) * L.Cin;
                const TW* wp = w + ((ky * L.Kw + kx) * L.Cin) * L.Cout + co;
                for (int ci = 0; ci < L.Cin; ++ci) {
                    const TS v = ip[ci];
                    if (v != (TS)0) acc += fw(wp[ci * L.Cout]) * v;       // zero components send no event
                }
            }
            TS* cp = ring + ((int)(o % L.ring_rows) * G + g) * row_elems + x * L.Cout + co;
            const TS c = *cp + acc;
            if (o == o_done) {
                rowbuf[e] = fused_act(c, bias ? bias[co] : (TS)0, L.relu, L.shift, L.round_bf16);
                *cp = 0;                                               // the slot is free for row o + ring_rows
            } else {
                *cp = c;
            }
        }
    }
    __syncthreads();
    if (completes) rows_done[i] += 1;
    return completes;
}

// The row standing in layer i's buffer goes up through the layers above; the net's output row is written out.
template <typename TS>
__device__ void fused_cascade(const FusedArgs& a, int i, TS* smem, long long* rows_in, long long* rows_done, int G, int g0,
                              unsigned long long* ev_local)
{
    const TS* cur = smem + a.layer[i].rowbuf_soff;
    for (int k = i + 1; k < a.n_layers; ++k) {
        if (!fused_feed<TS>(a, k, cur, smem, rows_in, rows_done, G, g0, ev_local)) return;
        cur = smem + a.layer[k].rowbuf_soff;
    }
    // a finished row of the last layer
    const FusedLayer& Z = a.layer[a.n_layers - 1];
    const long long o = rows_done[a.n_layers - 1] - 1 - a.out_base;
    const int row_elems = Z.Wout * Z.Cout;
    for (int e = threadIdx.x; e < G * row_elems; e += blockDim.x) {
        const int g = e / row_elems, q = e - g * row_elems;
        const long long at = ((long long)(g0 + g) * a.out_cap + o) * row_elems + q;
        if (IDF_OK_AT(a.status, at, (long long)a.S * a.out_cap * row_elems)) store_elem<TS>(a.out, at, a.out_elem, cur[e]);
    }
    __syncthreads();
}

template <typename TS>
__global__ void __launch_bounds__(512) depth_first_kernel(const FusedArgs a)
{
    extern __shared__ __align__(16) unsigned char fsmem[];
    __shared__ unsigned long long ev_local[FUSED_MAX_LAYERS];
    TS* smem = (TS*)fsmem;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int g0 = blockIdx.x * a.G;
    const int G = min(a.G, a.S - g0);
    long long rows_in[FUSED_MAX_LAYERS], rows_done[FUSED_MAX_LAYERS];
    for (int i = 0; i < a.n_layers; ++i) { rows_in[i] = a.layer[i].rows_in; rows_done[i] = a.layer[i].rows_done; }
    if (threadIdx.x < FUSED_MAX_LAYERS) ev_local[threadIdx.x] = 0;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // ---- the group's rolling state comes on chip
    for (int i = 0; i < a.n_layers; ++i) {
        const FusedLayer& L = a.layer[i];
        TS* st = smem + L.state_soff;
        const int row_elems = L.Wout * L.Cout;
        if (L.kind == 0) {
            const TS* gr = (const TS*)L.state;
            for (int e = threadIdx.x; e < L.ring_rows * G * row_elems; e += blockDim.x) {
                const int slot = e / (G * row_elems), q = e - slot * (G * row_elems);
                const long long at = ((long long)slot * a.S + g0) * row_elems + q;
                if (IDF_OK_AT(a.status, at, (long long)L.ring_rows * a.S * row_elems)) st[e] = gr[at];
            }
        } else {
            for (int e = threadIdx.x; e < G * row_elems; e += blockDim.x) {
                const long long at = (long long)g0 * row_elems + e;
                if (IDF_OK_AT(a.status, at, (long long)a.S * row_elems)) st[e] = load_elem<TS>(L.state, at, L.out_elem);
            }
        }
    }
    __syncthreads();
    // ---- segments, one at a time, each through every layer it can reach
    TS* inrow = smem + a.in_soff;
    const int in_elems = a.in_w * a.in_c;
    for (int seg = 0; seg < a.n_seg; ++seg) {
        for (int e = threadIdx.x; e < G * in_elems; e += blockDim.x) {
            const long long at = ((long long)seg * a.S + g0) * in_elems + e;
            if (IDF_OK_AT(a.status, at, (long long)a.n_seg * a.S * in_elems)) inrow[e] = load_elem<TS>(a.in, at, a.in_elem);
        }
        __syncthreads();
        if (fused_feed<TS>(a, 0, inrow, smem, rows_in, rows_done, G, g0, ev_local))
            fused_cascade<TS>(a, 0, smem, rows_in, rows_done, G, g0, ev_local);
    }
    // ---- end of input: rows that wait only for bottom zero padding are complete as they stand, in depth order
    if (a.flush) {
        for (int i = 0; i < a.n_layers; ++i) {
            const FusedLayer& L = a.layer[i];
            if (L.kind != 0) continue;                   // (an unpaired pooling row is dropped)
            const long long q = rows_in[i] + 2LL * L.pad - L.Kh;
            const long long total = rows_in[i] <= 0 || q < 0 ? 0 : q / L.stride + 1;
            const int row_elems = L.Wout * L.Cout;
            const TS* bias = L.bias_off >= 0 ? (const TS*)((const unsigned char*)a.weights + L.bias_off) : nullptr;
            while (rows_done[i] < total) {
                const long long o = rows_done[i];
                TS* ring = smem + L.state_soff;
                TS* rowbuf = smem + L.rowbuf_soff;
                for (int e = threadIdx.x; e < G * row_elems; e += blockDim.x) {
                    const int g = e / row_elems, q2 = e - g * row_elems;
                    TS* cp = ring + ((int)(o % L.ring_rows) * G + g) * row_elems + q2;
                    rowbuf[e] = fused_act(*cp, bias ? bias[q2 % L.Cout] : (TS)0, L.relu, L.shift, L.round_bf16);
                    *cp = 0;
                }
                __syncthreads();
                rows_done[i] = o + 1;
                fused_cascade<TS>(a, i, smem, rows_in, rows_done, G, g0, ev_local);
            }
        }
    }
    // ---- the state goes back
    for (int i = 0; i < a.n_layers; ++i) {
        const FusedLayer& L = a.layer[i];
        const TS* st = smem + L.state_soff;
        const int row_elems = L.Wout * L.Cout;
        if (L.kind == 0) {
            TS* gr = (TS*)L.state;
            for (int e = threadIdx.x; e < L.ring_rows * G * row_elems; e += blockDim.x) {
                const int slot = e / (G * row_elems), q = e - slot * (G * row_elems);
                const long long at = ((long long)slot * a.S + g0) * row_elems + q;
                if (IDF_OK_AT(a.status, at, (long long)L.ring_rows * a.S * row_elems)) gr[at] = st[e];
            }
        } else {
            for (int e = threadIdx.x; e < G * row_elems; e += blockDim.x) {
                const long long at = (long long)g0 * row_elems + e;
                if (IDF_OK_AT(a.status, at, (long long)a.S * row_elems)) store_elem<TS>(L.state, at, L.out_elem, st[e]);
            }
        }
    }
    __syncthreads();
    if (threadIdx.x < a.n_layers && ev_local[threadIdx.x] && a.counters) atomicAdd(a.counters + threadIdx.x, ev_local[threadIdx.x]);
}

}  // namespace

cudaError_t launch_depth_first(const FusedArgs& a, int int_net, int threads, size_t smem_bytes, cudaStream_t st)
{
    if (a.S <= 0 || (a.n_seg <= 0 && !a.flush)) return cudaSuccess;
    const unsigned grid = (unsigned)((a.S + a.G - 1) / a.G);
    auto kf = int_net ? depth_first_kernel<int> : depth_first_kernel<float>;
    static bool attr_set[2][64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!attr_set[int_net ? 1 : 0][dev]) {
        cudaError_t e = cudaFuncSetAttribute(kf, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)FUSED_SMEM_LIMIT);
        if (e != cudaSuccess) return e;
        attr_set[int_net ? 1 : 0][dev] = true;
    }
    kf<<<grid, threads, smem_bytes, st>>>(a);
    return cudaGetLastError();
}

}  // namespace idf
