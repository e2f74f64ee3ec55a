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
//
// Rows travel between layers in shared memory as fp32 values (float nets; bf16 layers hold
// bf16-representable values) or int8 (int nets, four channels to a word for dp4a).  Row bookkeeping
// (which ring slots a row reaches, which row it completes) is kept in small counters that step from
// row to row: no division in the loop over segments.
#include "idf_internal.h"

namespace idf {

namespace {

template <typename TS> struct RowOf;
template <> struct RowOf<float> { typedef float T; typedef float W; };
template <> struct RowOf<int> { typedef int8_t T; typedef int8_t W; };

__device__ __forceinline__ float fused_act(float c, float b, int relu, int, int round_bf16)
{
    float v = c + b;
    if (relu && v < 0.f) v = 0.f;
    if (round_bf16) v = __bfloat162float(__float2bfloat16_rn(v));
    return v;
}
__device__ __forceinline__ int8_t fused_act(int c, int b, int relu, int shift, int)
{
    int v = c + b;
    if (relu && v < 0) v = 0;
    if (shift > 0) v = (v + (1 << (shift - 1))) >> shift;
    const int lo = relu ? 0 : -127;
    return (int8_t)(v < lo ? lo : (v > 127 ? 127 : v));
}

template <typename TR>
__device__ __forceinline__ TR load_elem(const void* p, long long i, int elem)
{
    if (elem == E_F32) return (TR)((const float*)p)[i];
    if (elem == E_BF16) return (TR)__bfloat162float(((const __nv_bfloat16*)p)[i]);
    return (TR)((const int8_t*)p)[i];
}
template <typename TR>
__device__ __forceinline__ void store_elem(void* p, long long i, int elem, TR v)
{
    if (elem == E_F32) ((float*)p)[i] = (float)v;
    else if (elem == E_BF16) ((__nv_bfloat16*)p)[i] = __float2bfloat16_rn((float)v);
    else ((int8_t*)p)[i] = (int8_t)v;
}

// progress of one layer inside the launch (the same in every thread)
struct LayerClock {
    int ph;        // conv: (rows received + pad) mod stride = the first tap ky of the next input row; pool: rows received mod 2
    int hi_slot;   // conv: ring slot of the newest row the next input row reaches
    int hi_sat;    // conv: index of that newest row, saturated (only "how many older rows exist" matters)
    int phf;       // conv: (rows received + pad - (Kh-1)) mod stride: 0 when the next input row completes a row
    int tf_neg;    // conv: input rows still to come before the first row can complete
    int done_slot; // conv: ring slot of the oldest open row (the next to complete)
};

constexpr int FUSED_TAPS = 3;      // rows one input row reaches in the fast loops (ceil(Kh/stride) <= 3); more take the plain loop

// Layer i takes the row `in` ([G][Win][Cin]) as its next input row.  Returns true if it completed a row, which then
// stands in the layer's row buffer.
template <typename TS>
__device__ bool fused_feed(const FusedArgs& a, int i, const typename RowOf<TS>::T* in, unsigned char* smem, LayerClock& k, int G,
                           unsigned long long* ev_local)
{
    typedef typename RowOf<TS>::T TR;
    typedef typename RowOf<TS>::W TW;
    const FusedLayer& L = a.layer[i];
    TR* rowbuf = (TR*)(smem + L.rowbuf_soff);
    if (L.count_events) {
        // the layer's input events: the non-zero components of the row (Eq. 3)
        unsigned n = 0;
        for (int e = threadIdx.x; e < G * L.Win * L.Cin; e += blockDim.x) n += in[e] != (TR)0;
        for (int o = 16; o; o >>= 1) n += __shfl_xor_sync(0xffffffffu, n, o);
        if ((threadIdx.x & 31) == 0 && n) atomicAdd(&ev_local[i], (unsigned long long)n);
    }
    if (L.kind == 1) {
        // 2x2 max-pool fold: the x-pooled first row of a pair waits in the pool state
        TR* st = (TR*)(smem + L.state_soff);
        const int px = L.Win == 1 ? 1 : 2;
        const bool second = k.ph != 0;
        for (int e = threadIdx.x; e < G * L.Wout * L.Cout; e += blockDim.x) {
            const int c = e % L.Cout, t = e / L.Cout, x = t % L.Wout, g = t / L.Wout;
            const TR* p = in + ((g * L.Win + px * x) * L.Cin + c);
            TR m = p[0];
            if (px == 2) { const TR v = p[L.Cin]; m = v > m ? v : m; }
            if (second) { const TR f = st[e]; rowbuf[e] = f > m ? f : m; }
            else st[e] = m;
        }
        __syncthreads();
        k.ph ^= 1;
        return second;
    }
    // conv: Eq. 4 for every event of the row, tap by tap, then Eq. 2-3 for the row this input row completes
    const TS* __restrict__ bias = L.bias_off >= 0 ? (const TS*)((const unsigned char*)a.weights + L.bias_off) : nullptr;
    TS* ring = (TS*)(smem + L.state_soff);
    const int row_elems = L.Wout * L.Cout;
    // taps ky = ph, ph + s, ... < Kh; tap j reaches the row j below the newest one (if that many rows exist)
    int nt = (L.Kh - k.ph + L.stride - 1) / L.stride;
    if (nt > k.hi_sat + 1) nt = k.hi_sat + 1;
    const bool completes = k.phf == 0 && k.tf_neg == 0;      // ... and the oldest row reached then has its last tap
    const int Cq = L.Cin >> 2;
    const bool quads = (L.Cin & 3) == 0 && !L.count_events && L.wq_off >= 0;
    if (nt <= FUSED_TAPS && quads) {
        // four input channels at a time (dp4a / four FMAs), the input fetched once for all taps
        const int* __restrict__ wq = (const int*)((const unsigned char*)a.weights + L.wq_off);     // int nets: [ky][kx][ci/4][co] packed words
        const float* __restrict__ wf = (const float*)a.weights + L.w_off;                          // float nets: [ky][kx][ci][co]
        for (int e = threadIdx.x; e < G * row_elems; e += blockDim.x) {
            const int co = e % L.Cout, t = e / L.Cout, x = t % L.Wout, g = t / L.Wout;
            TS acc[FUSED_TAPS] = {0, 0, 0};
            for (int kx = 0; kx < L.Kw; ++kx) {
                const int ix = x * L.stride_x - L.pad_x + kx;
                if (ix < 0 || ix >= L.Win) continue;
                const TR* ip = in + (g * L.Win + ix) * L.Cin;
                for (int c4 = 0; c4 < Cq; ++c4) {
                    if constexpr (sizeof(TR) == 1) {
                        const int v = ((const int*)ip)[c4];
#pragma unroll
                        for (int j = 0; j < FUSED_TAPS; ++j)
                            if (j < nt) acc[j] = __dp4a(v, __ldg(wq + (((k.ph + j * L.stride) * L.Kw + kx) * Cq + c4) * L.Cout + co), acc[j]);
                    } else {
                        const float4 v = ((const float4*)ip)[c4];
#pragma unroll
                        for (int j = 0; j < FUSED_TAPS; ++j)
                            if (j < nt) {
                                const float* wp = wf + (((k.ph + j * L.stride) * L.Kw + kx) * L.Cin + 4 * c4) * L.Cout + co;
                                acc[j] += __ldg(wp) * v.x; acc[j] += __ldg(wp + L.Cout) * v.y;
                                acc[j] += __ldg(wp + 2 * L.Cout) * v.z; acc[j] += __ldg(wp + 3 * L.Cout) * v.w;
                            }
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < FUSED_TAPS; ++j) {
                if (j >= nt) break;
                int slot = k.hi_slot - j;
                if (slot < 0) slot += L.ring_rows;
                TS* cp = ring + (slot * G + g) * row_elems + x * L.Cout + co;
                const TS c = *cp + acc[j];
                if (completes && j == nt - 1) {
                    rowbuf[e] = fused_act(c, bias ? bias[co] : (TS)0, L.relu, L.shift, L.round_bf16);
                    *cp = 0;                                           // the slot is free for the row ring_rows further on
                } else {
                    *cp = c;
                }
            }
        }
    } else {
        const TW* __restrict__ w = (const TW*)a.weights + L.w_off;
        for (int e = threadIdx.x; e < G * row_elems; e += blockDim.x) {
            const int co = e % L.Cout, t = e / L.Cout, x = t % L.Wout, g = t / L.Wout;
            for (int j = 0; j < nt; ++j) {
                const int ky = k.ph + j * L.stride;
                TS acc = 0;
                for (int kx = 0; kx < L.Kw; ++kx) {
                    const int ix = x * L.stride_x - L.pad_x + kx;
                    if (ix < 0 || ix >= L.Win) continue;
                    const TR* ip = in + (g * L.Win + ix) * L.Cin;
                    const TW* wp = w + ((ky * L.Kw + kx) * L.Cin) * L.Cout + co;
                    for (int ci = 0; ci < L.Cin; ++ci) {
                        const TS v = (TS)ip[ci];
                        if (v != (TS)0) acc += (TS)wp[ci * L.Cout] * v;       // zero components send no event
                    }
                }
                int slot = k.hi_slot - j % L.ring_rows;
                if (slot < 0) slot += L.ring_rows;
                TS* cp = ring + (slot * G + g) * row_elems + x * L.Cout + co;
                const TS c = *cp + acc;
                if (completes && j == nt - 1) {
                    rowbuf[e] = fused_act(c, bias ? bias[co] : (TS)0, L.relu, L.shift, L.round_bf16);
                    *cp = 0;
                } else {
                    *cp = c;
                }
            }
        }
    }
    __syncthreads();
    // the clock moves on to the next input row
    if (++k.ph == L.stride) {
        k.ph = 0;
        if (++k.hi_slot == L.ring_rows) k.hi_slot = 0;
        if (k.hi_sat < (1 << 20)) ++k.hi_sat;
    }
    if (k.tf_neg > 0) --k.tf_neg;
    else if (++k.phf == L.stride) k.phf = 0;
    if (completes && ++k.done_slot == L.ring_rows) k.done_slot = 0;
    return completes;
}

// The row standing in layer i's buffer goes up through the layers above; the net's output row is written out.
template <typename TS>
__device__ void fused_cascade(const FusedArgs& a, int i, unsigned char* smem, LayerClock* clk, int G, int g0, int& out_row,
                              unsigned long long* ev_local)
{
    typedef typename RowOf<TS>::T TR;
    const TR* cur = (const TR*)(smem + a.layer[i].rowbuf_soff);
    for (int n = i + 1; n < a.n_layers; ++n) {
        if (!fused_feed<TS>(a, n, cur, smem, clk[n], G, ev_local)) return;
        cur = (const TR*)(smem + a.layer[n].rowbuf_soff);
    }
    // a finished row of the last layer
    const FusedLayer& Z = a.layer[a.n_layers - 1];
    const int row_elems = Z.Wout * Z.Cout;
    for (int e = threadIdx.x; e < G * row_elems; e += blockDim.x) {
        const int g = e / row_elems, q = e - g * row_elems;
        const long long at = ((long long)(g0 + g) * a.out_cap + out_row) * row_elems + q;
        if (IDF_OK_AT(a.status, at, (long long)a.S * a.out_cap * row_elems)) store_elem<TR>(a.out, at, a.out_elem, cur[e]);
    }
    out_row += 1;
    __syncthreads();
}

template <typename TS>
__global__ void __launch_bounds__(512) depth_first_kernel(const FusedArgs a)
{
    typedef typename RowOf<TS>::T TR;
    extern __shared__ __align__(16) unsigned char fsmem[];
    __shared__ unsigned long long ev_local[FUSED_MAX_LAYERS];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int g0 = blockIdx.x * a.G;
    const int G = min(a.G, a.S - g0);
    LayerClock clk[FUSED_MAX_LAYERS];
    for (int i = 0; i < a.n_layers; ++i) {
        const FusedLayer& L = a.layer[i];
        clk[i].ph = L.ph0; clk[i].hi_slot = L.hi_slot0; clk[i].hi_sat = L.hi_sat0; clk[i].phf = L.phf0; clk[i].tf_neg = L.tf_neg0;
        clk[i].done_slot = L.done_slot0;
    }
    int out_row = a.out_row0;
    if (threadIdx.x < FUSED_MAX_LAYERS) ev_local[threadIdx.x] = 0;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // ---- the group's rolling state comes on chip
    for (int i = 0; i < a.n_layers; ++i) {
        const FusedLayer& L = a.layer[i];
        const int row_elems = L.Wout * L.Cout;
        if (L.kind == 0) {
            TS* st = (TS*)(fsmem + L.state_soff);
            const TS* gr = (const TS*)L.state;
            for (int e = threadIdx.x; e < L.ring_rows * G * row_elems; e += blockDim.x) {
                const int slot = e / (G * row_elems), q = e - slot * (G * row_elems);
                const long long at = ((long long)slot * a.S + g0) * row_elems + q;
                if (IDF_OK_AT(a.status, at, (long long)L.ring_rows * a.S * row_elems)) st[e] = gr[at];
            }
        } else {
            TR* st = (TR*)(fsmem + L.state_soff);
            for (int e = threadIdx.x; e < G * row_elems; e += blockDim.x) {
                const long long at = (long long)g0 * row_elems + e;
                if (IDF_OK_AT(a.status, at, (long long)a.S * row_elems)) st[e] = load_elem<TR>(L.state, at, L.out_elem);
            }
        }
    }
    __syncthreads();
    // ---- segments, one at a time, each through every layer it can reach
    TR* inrow = (TR*)(fsmem + a.in_soff);
    const int in_elems = a.in_w * a.in_c;
    for (int seg = 0; seg < a.n_seg; ++seg) {
        for (int e = threadIdx.x; e < G * in_elems; e += blockDim.x) {
            const long long at = ((long long)seg * a.S + g0) * in_elems + e;
            if (IDF_OK_AT(a.status, at, (long long)a.n_seg * a.S * in_elems)) inrow[e] = load_elem<TR>(a.in, at, a.in_elem);
        }
        __syncthreads();
        if (fused_feed<TS>(a, 0, inrow, fsmem, clk[0], G, ev_local)) fused_cascade<TS>(a, 0, fsmem, clk, G, g0, out_row, ev_local);
    }
    // ---- end of input: rows that wait only for bottom zero padding are complete as they stand, in depth order
    // (how many each layer has is a matter of row counts: worked out by the host for the rows the layer will have received)
    if (a.flush) {
        for (int i = 0; i < a.n_layers; ++i) {
            const FusedLayer& L = a.layer[i];
            if (L.kind != 0) continue;                   // (an unpaired pooling row is dropped)
            const int row_elems = L.Wout * L.Cout;
            const TS* bias = L.bias_off >= 0 ? (const TS*)((const unsigned char*)a.weights + L.bias_off) : nullptr;
            for (int n = 0; n < L.n_flush; ++n) {
                TS* ring = (TS*)(fsmem + L.state_soff);
                TR* rowbuf = (TR*)(fsmem + L.rowbuf_soff);
                for (int e = threadIdx.x; e < G * row_elems; e += blockDim.x) {
                    const int g = e / row_elems, q2 = e - g * row_elems;
                    TS* cp = ring + (clk[i].done_slot * G + g) * row_elems + q2;
                    rowbuf[e] = fused_act(*cp, bias ? bias[q2 % L.Cout] : (TS)0, L.relu, L.shift, L.round_bf16);
                    *cp = 0;
                }
                __syncthreads();
                if (++clk[i].done_slot == L.ring_rows) clk[i].done_slot = 0;
                fused_cascade<TS>(a, i, fsmem, clk, G, g0, out_row, ev_local);
            }
        }
    }
    // ---- the state goes back
    for (int i = 0; i < a.n_layers; ++i) {
        const FusedLayer& L = a.layer[i];
        const int row_elems = L.Wout * L.Cout;
        if (L.kind == 0) {
            const TS* st = (const TS*)(fsmem + L.state_soff);
            TS* gr = (TS*)L.state;
            for (int e = threadIdx.x; e < L.ring_rows * G * row_elems; e += blockDim.x) {
                const int slot = e / (G * row_elems), q = e - slot * (G * row_elems);
                const long long at = ((long long)slot * a.S + g0) * row_elems + q;
                if (IDF_OK_AT(a.status, at, (long long)L.ring_rows * a.S * row_elems)) gr[at] = st[e];
            }
        } else {
            const TR* st = (const TR*)(fsmem + L.state_soff);
            for (int e = threadIdx.x; e < G * row_elems; e += blockDim.x) {
                const long long at = (long long)g0 * row_elems + e;
                if (IDF_OK_AT(a.status, at, (long long)a.S * row_elems)) store_elem<TR>(L.state, at, L.out_elem, st[e]);
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
