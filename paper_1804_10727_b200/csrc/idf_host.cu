// Host side of the C ABI: spec validation, shape inference, workspace layout, parameter packing
// and the depth-first schedule that walks every block of pushed segments through all layers.
#include "../../include/idf.h"
#include "idf_internal.h"

#include <algorithm>
#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <string>
#include <vector>

using namespace idf;

namespace {

thread_local std::string g_err;

int fail(int code, const char* fmt, ...)
{
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    g_err = buf;
    return code;
}

size_t align_up(size_t v, size_t a = 256) { return (v + a - 1) / a * a; }

struct LayerPlan {
    idf_layer l;
    int in_w, out_w, in_c, out_c;
    int ring_rows;           // conv: ceil(kh/stride); pool: 1
    int in_elem, out_elem;   // Elem of the rows this layer receives / emits
    int use_sparse;
    TcPlan tc;                              // tensor-core path (tc.ok) for the dense update
    std::vector<unsigned char> wtc_packed;  // [tap slot][Cout][Cin] in the activation type, tap slots in the order of tc_weight_slot
    size_t wtc_off = 0;
    alignas(64) unsigned char w_map[128];   // TMA descriptor of wtc in the workspace (made at open)
    TcPlan tc_pool;                         // plan of the launches that also emit the following max-pool's rows
    alignas(64) unsigned char w_map_pool[128];
    long long tc_launches = 0;
    // thin layers (the whole receptive field of an output position in one shared-memory row): a kernel of its own for
    // the rows a block determines completely
    std::vector<unsigned char> wq_packed;      // int nets, Cin % 4 == 0: [Kh][Kw][Cin/4][Cout] words of four int8 (all-layers launch)
    size_t wq_off = 0;
    ThinPlan thin;
    std::vector<unsigned char> wthin_packed;   // [Cout][row bytes] in the activation type, zero padded
    size_t wthin_off = 0;
    alignas(64) unsigned char w_map_thin[128];
    // x-unfold in front of the tensor-core kernel (thin or x-strided layers): the Kw taps of every
    // output position are laid side by side as kpad channels, the conv then has Kw = 1, stride_x = 1
    int unfold = 0, kpad = 0, in_cap_rows = 0;
    size_t unf_off = 0;
    // host copies of the packed parameters
    std::vector<unsigned char> w_packed;   // [Kh][Kw][Cin][Cout] float (float nets) or int8
    std::vector<unsigned char> b_packed;   // [Cout] float / int32 (empty = zero bias)
    // workspace offsets
    size_t w_off = 0, b_off = 0, state_off = 0, out_off = 0;
    size_t state_bytes_all = 0;            // all streams
    size_t state_bytes_stream = 0;
    int out_cap_rows = 0;                  // capacity of the buffer this layer emits into
    // progress (identical for all streams)
    long long rows_in = 0, rows_done = 0;
    long long pending = 0;                 // rows waiting in this layer's input buffer
    int fire_rows = 0;                     // the layer runs once this many rows wait (or when a push ends)
    int fuse_pool = 0;                     // conv layer whose tensor-core launch may emit the following 2x2 max-pool's rows
    // eager emission: rings of e_cap rows for the state, the announced activation and the change of the current step
    int e_cap = 0, e_window = 0;           // ring capacity in rows; most rows one segment can touch (the input cone)
    size_t e_c_off = 0, e_h_off = 0, e_d_off = 0;
    long long e_hi = -1;                   // last row touched so far
};

enum Phase { CREATED = 0, OPEN = 1, FINISHED = 2 };

}  // namespace

struct idf_net {
    int dtype = 0, in_w = 0, in_c = 0, n_streams = 0, row_block = 0;
    // depth-first over all layers in one launch (nets whose per-stream state is small): plan made at create
    int fused_ok = 0, fused_G = 0, fused_threads = 0, fused_in_soff = 0;
    size_t fused_smem = 0;
    std::vector<int> fused_state_soff, fused_rowbuf_soff;
    double macs_per_row = 0;               // multiply-accumulates one segment of one stream costs (all layers, steady state)
    int eager = 0;                         // emission policy: 0 = once per unit (deferred), 1 = after every segment (eager)
    size_t eager_in_off = 0;               // the pushed segment as words (the input layer's announcement)
    std::vector<LayerPlan> L;
    size_t workspace_bytes = 0, state_region_off = 0, state_region_bytes = 0, counters_off = 0, status_off = 0;
    size_t ring_scratch_off = 0;           // room for a copy of the largest tensor-core layer's ring (row-chunked launches)
    size_t state_bytes_stream = 0;
    unsigned char* ws = nullptr;
    cudaStream_t stream = nullptr;
    int phase = CREATED;
    long long launches = 0;
    long long out_rows_total = 0;
    long long out_base = 0;                // output row written at index 0 of the caller's buffer (idf_stream_set_out_base)
    // optional per-launch timing (CUDA events on the handle's stream)
    bool timing = false;
    struct Timed { int layer; cudaEvent_t a, b; };
    std::vector<Timed> timed;
    std::vector<cudaEvent_t> event_pool;
    // idf_run_host: copy streams and ordering events, made at the first call (no device memory involved)
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
    std::vector<cudaEvent_t> order_events;
};

namespace {

float bf16_bits_to_float(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

long long conv_done_after(const idf_layer& l, long long rows_in)
{
    // number of output rows whose last tap (row o*stride - pad + Kh - 1) lies below rows_in
    const long long q = rows_in + l.pad - l.kh;
    return q < 0 ? 0 : q / l.stride + 1;
}

long long conv_rows_at_flush(const idf_layer& l, long long rows_in)
{
    // floor((H + 2 pad - Kh) / stride) + 1 rows exist once the input is known to have H rows
    if (rows_in <= 0) return 0;
    const long long q = rows_in + 2LL * l.pad - l.kh;
    return q < 0 ? 0 : q / l.stride + 1;
}

// (a global-average sink has one output row, rewritten with the running mean whenever rows arrive)
long long layer_done_after(const LayerPlan& P, long long rows_in)
{
    return P.l.kind == IDF_CONV ? conv_done_after(P.l, rows_in) : P.l.kind == IDF_MAXPOOL2 ? rows_in / 2 : (rows_in > 0 ? 1 : 0);
}
long long layer_rows_at_flush(const LayerPlan& P, long long rows_in)
{
    return P.l.kind == IDF_CONV ? conv_rows_at_flush(P.l, rows_in) : P.l.kind == IDF_MAXPOOL2 ? rows_in / 2 : (rows_in > 0 ? 1 : 0);
}

// Enqueue one layer on n_in input rows found at in_ptr (slots 0..n_in-1).  With `flush` (n_in == 0)
// the layer learns that its input has ended and completes the rows that wait only for bottom padding.
// Rows it emits go to the next layer's buffer starting at slot `out_slot` (or to the caller's output
// at their absolute row index).  Updates the layer's row counters; *n_out_p = rows emitted.
int launch_layer(idf_net* net, size_t i, const void* in_ptr, long long n_in, bool flush, void* final_out,
                 long long out_cap, long long out_slot, long long* n_out_p)
{
    LayerPlan& P = net->L[i];
    const bool last = (i + 1 == net->L.size());
    const long long r0 = P.rows_in, r1 = r0 + n_in;
    long long done_end, o_end;
    if (P.l.kind == IDF_CONV) {
        done_end = flush ? conv_rows_at_flush(P.l, r1) : conv_done_after(P.l, r1);
        const long long started = r1 > 0 ? (r1 - 1 + P.l.pad) / P.l.stride + 1 : 0;   // rows reached so far
        o_end = std::max(started, done_end);
    } else if (P.l.kind == IDF_MAXPOOL2) {
        done_end = r1 / 2;
        o_end = (r1 + 1) / 2;
    } else {
        done_end = o_end = r1 > 0 ? 1 : 0;
    }
    const long long o_begin = P.rows_done;
    if (done_end < o_begin) done_end = o_begin;
    const long long n_out = done_end - o_begin;
    *n_out_p = n_out;
    if (last && done_end - net->out_base > out_cap)
        return fail(IDF_ERR_CAPACITY, "output row %lld does not fit out_capacity_rows=%lld", done_end - 1, out_cap);
    if (!last && n_out + out_slot > P.out_cap_rows)
        return fail(IDF_ERR_CAPACITY, "internal: layer %zu emits %lld rows at slot %lld of a %d-row buffer", i, n_out,
                    out_slot, P.out_cap_rows);
    P.rows_in = r1;
    P.rows_done = done_end;
    if (n_in == 0 && n_out == 0) return IDF_OK;

    const long long S = net->n_streams;
    void* out_ptr;
    long long row_stride, stream_stride, row_base;
    if (last) {
        out_ptr = final_out;
        row_stride = (long long)P.out_w * P.out_c;
        stream_stride = out_cap * row_stride;
        row_base = net->out_base;
    } else {
        out_ptr = net->ws + P.out_off;
        stream_stride = (long long)P.out_w * P.out_c;
        row_stride = S * stream_stride;
        row_base = o_begin - out_slot;             // emitted rows are appended slot after slot
    }
    // extents of the buffers this launch addresses (the range-checked build compares every index with them)
    const long long in_elems = n_in * S * P.in_w * P.in_c;
    const long long out_elems = last ? S * out_cap * P.out_w * P.out_c : (long long)P.out_cap_rows * S * P.out_w * P.out_c;
    unsigned int* status = (unsigned int*)(net->ws + net->status_off);
    cudaError_t ce;
    cudaEvent_t ev_a = nullptr, ev_b = nullptr;
    if (net->timing) {
        for (cudaEvent_t* e : {&ev_a, &ev_b}) {
            if (!net->event_pool.empty()) { *e = net->event_pool.back(); net->event_pool.pop_back(); }
            else if (cudaEventCreate(e) != cudaSuccess) return fail(IDF_ERR_CUDA, "cudaEventCreate failed");
        }
        cudaEventRecord(ev_a, net->stream);
    }
    if (P.l.kind == IDF_CONV) {
        ConvArgs a{};
        a.in_elems = in_elems; a.out_elems = out_elems; a.status = status;
        a.ring_elems = (long long)P.ring_rows * S * P.out_w * P.out_c;
        a.in = in_ptr;
        a.w = net->ws + P.w_off;
        a.bias = P.b_packed.empty() ? nullptr : net->ws + P.b_off;
        a.ring = net->ws + P.state_off;
        a.ring_scratch = net->ring_scratch_off ? net->ws + net->ring_scratch_off : nullptr;
        a.out = out_ptr;
        a.out_row_stride = row_stride; a.out_stream_stride = stream_stride; a.out_row_base = row_base;
        a.out_rows_extent = last ? out_cap : P.out_cap_rows;
        a.event_counter = (unsigned long long*)(net->ws + net->counters_off) + i;
        a.S = (int)S; a.Win = P.in_w; a.Wout = P.out_w; a.Cin = P.in_c; a.Cout = P.out_c;
        a.Kh = P.l.kh; a.Kw = P.l.kw; a.stride = P.l.stride; a.pad = P.l.pad; a.relu = P.l.relu; a.shift = P.l.shift;
        a.stride_x = P.in_w == 1 ? 1 : P.l.stride; a.pad_x = P.in_w == 1 ? 0 : P.l.pad;
        a.ring_rows = P.ring_rows; a.in_elem = P.in_elem; a.out_elem = P.out_elem;
        a.r0 = r0; a.r1 = r1; a.o_begin = o_begin; a.o_end = o_end; a.done_end = done_end;
        ce = cudaErrorNotSupported;
        if (P.thin.ok && !P.use_sparse && n_in > 0) {
            // rows not begun by an earlier block (first tap row o*stride - pad >= r0) and completed by this one: the
            // thin-layer kernel computes them from the block's rows alone; the others exchange state with the ring
            long long int_begin = r0 > 0 ? (r0 + P.l.pad + P.l.stride - 1) / P.l.stride : o_begin;
            if (int_begin < o_begin) int_begin = o_begin;
            const long long int_end = done_end;
            if (int_end - int_begin >= 4) {
                ce = launch_conv_thin(a, P.thin, net->dtype, P.w_map_thin, int_begin, int_end, status, net->stream);
                if (ce == cudaSuccess) {
                    net->launches += 1;
                    P.tc_launches += 1;
                    ce = launch_conv_edges(a, net->dtype, int_begin, int_end, net->stream);
                }
            }
        }
        if (ce == cudaErrorNotSupported && P.tc.ok && !P.use_sparse && n_in > 0) {
            ConvArgs t = a;
            if (P.unfold && n_in <= P.in_cap_rows) {
                ce = launch_unfold(a, (int)n_in, P.kpad, net->ws + P.unf_off, net->stream);
                t.in = net->ws + P.unf_off;
                t.Win = a.Wout; t.Cin = P.kpad; t.Kw = 1; t.stride_x = 1; t.pad_x = 0;
                if (ce == cudaSuccess) {
                    net->launches += 1;
                    ce = launch_conv_tc(t, P.tc, net->dtype, P.w_map, (int)n_in, (unsigned int*)(net->ws + net->status_off), net->stream);
                }
            } else if (!P.unfold) {
                ce = launch_conv_tc(t, P.tc, net->dtype, P.w_map, (int)n_in, (unsigned int*)(net->ws + net->status_off), net->stream);
            }
            if (ce == cudaSuccess) P.tc_launches += 1;
        }
        if (ce == cudaErrorNotSupported)
            ce = P.use_sparse ? launch_conv_sparse(a, net->dtype, net->stream) : launch_conv_simple(a, net->dtype, net->stream);
    } else if (P.l.kind == IDF_GLOBAL_AVG) {
        AvgArgs a{};
        a.in_elems = in_elems; a.out_elems = out_elems; a.sum_elems = S * P.in_c; a.status = status;
        a.in = in_ptr;
        a.sum = net->ws + P.state_off;
        a.out = (float*)out_ptr;
        a.out_stream_stride = stream_stride;
        a.S = (int)S; a.W = P.in_w; a.C = P.in_c; a.elem = P.in_elem;
        a.n_rows = n_in; a.rows_total = r1;
        ce = launch_avg(a, net->stream);
    } else {
        PoolArgs a{};
        a.in_elems = in_elems; a.out_elems = out_elems; a.state_elems = S * P.out_w * P.out_c; a.status = status;
        a.in = in_ptr;
        a.state = net->ws + P.state_off;
        a.out = out_ptr;
        a.out_row_stride = row_stride; a.out_stream_stride = stream_stride; a.out_row_base = row_base;
        a.S = (int)S; a.Win = P.in_w; a.Wout = P.out_w; a.C = P.in_c; a.elem = P.in_elem;
        a.r0 = r0; a.r1 = r1; a.o_begin = o_begin; a.o_end = o_end; a.done_end = done_end;
        ce = launch_pool(a, net->stream);
    }
    if (net->timing) {
        cudaEventRecord(ev_b, net->stream);
        net->timed.push_back({(int)i, ev_a, ev_b});
    }
    if (ce != cudaSuccess) return fail(IDF_ERR_CUDA, "kernel launch failed at layer %zu: %s", i, cudaGetErrorString(ce));
    net->launches += 1;
    return IDF_OK;
}

// A conv layer followed by a 2x2 max-pool, as ONE tensor-core launch that emits the pooled rows (into the
// buffer behind the pool layer, or the caller's output).  Both layers' row counters advance as if the
// two had run one after the other; a trailing unpaired row waits x-pooled in the pool layer's state,
// exactly as the stand-alone pool kernel leaves it, so fused and unfused launches may alternate.
// Returns 1 (no row counter changed) when this launch cannot take the fused path.
int launch_conv_pool(idf_net* net, size_t i, const void* in_ptr, long long n_in, bool flush, void* final_out,
                     long long out_cap, long long out_slot, long long* n_out_p)
{
    LayerPlan& P = net->L[i];
    LayerPlan& Q = net->L[i + 1];
    const bool last = (i + 2 == net->L.size());
    if (!P.fuse_pool || !P.tc_pool.ok || n_in <= 0 || (P.unfold && n_in > P.in_cap_rows) || Q.rows_in != P.rows_done) return 1;
    const long long r0 = P.rows_in, r1 = r0 + n_in;
    long long done_end = flush ? conv_rows_at_flush(P.l, r1) : conv_done_after(P.l, r1);
    const long long started = (r1 - 1 + P.l.pad) / P.l.stride + 1;
    const long long o_begin = P.rows_done;
    if (done_end < o_begin) done_end = o_begin;
    const long long o_end = std::max(started, done_end);
    const long long q_begin = Q.rows_done, q_done = done_end / 2;
    const long long n_out = q_done - q_begin;
    if (last && q_done - net->out_base > out_cap)
        return fail(IDF_ERR_CAPACITY, "output row %lld does not fit out_capacity_rows=%lld", q_done - 1, out_cap);
    if (!last && n_out + out_slot > Q.out_cap_rows)
        return fail(IDF_ERR_CAPACITY, "internal: layer %zu emits %lld rows at slot %lld of a %d-row buffer", i + 1, n_out,
                    out_slot, Q.out_cap_rows);
    const long long S = net->n_streams;
    ConvArgs a{};
    a.in = in_ptr;
    a.w = net->ws + P.w_off;
    a.bias = P.b_packed.empty() ? nullptr : net->ws + P.b_off;
    a.ring = net->ws + P.state_off;
        a.ring_scratch = net->ring_scratch_off ? net->ws + net->ring_scratch_off : nullptr;
    if (last) {
        a.out = final_out;
        a.out_row_stride = (long long)Q.out_w * Q.out_c;
        a.out_stream_stride = out_cap * a.out_row_stride;
        a.out_row_base = net->out_base;
        a.out_rows_extent = out_cap;
    } else {
        a.out = net->ws + Q.out_off;
        a.out_stream_stride = (long long)Q.out_w * Q.out_c;
        a.out_row_stride = S * a.out_stream_stride;
        a.out_row_base = q_begin - out_slot;
        a.out_rows_extent = Q.out_cap_rows;
    }
    a.event_counter = (unsigned long long*)(net->ws + net->counters_off) + i;
    a.S = (int)S; a.Win = P.in_w; a.Wout = P.out_w; a.Cin = P.in_c; a.Cout = P.out_c;
    a.Kh = P.l.kh; a.Kw = P.l.kw; a.stride = P.l.stride; a.pad = P.l.pad; a.relu = P.l.relu; a.shift = P.l.shift;
    a.stride_x = P.l.stride; a.pad_x = P.l.pad;
    a.ring_rows = P.ring_rows; a.in_elem = P.in_elem; a.out_elem = P.out_elem;
    a.r0 = r0; a.r1 = r1; a.o_begin = o_begin; a.o_end = o_end; a.done_end = done_end;
    a.pool_fused = 1; a.pool_keep = flush ? 0 : 1; a.pool_state = net->ws + Q.state_off;
    a.in_elems = n_in * S * P.in_w * P.in_c;
    a.out_elems = last ? S * out_cap * Q.out_w * Q.out_c : (long long)Q.out_cap_rows * S * Q.out_w * Q.out_c;
    a.ring_elems = (long long)P.ring_rows * S * P.out_w * P.out_c;
    a.pool_state_elems = S * Q.out_w * Q.out_c;
    a.status = (unsigned int*)(net->ws + net->status_off);
    if (a.out_rows_extent < 1) return 1;
    cudaEvent_t ev_a = nullptr, ev_b = nullptr;
    if (net->timing) {
        for (cudaEvent_t* e : {&ev_a, &ev_b}) {
            if (!net->event_pool.empty()) { *e = net->event_pool.back(); net->event_pool.pop_back(); }
            else if (cudaEventCreate(e) != cudaSuccess) return fail(IDF_ERR_CUDA, "cudaEventCreate failed");
        }
        cudaEventRecord(ev_a, net->stream);
    }
    cudaError_t ce;
    ConvArgs t = a;
    if (P.unfold) {
        // (if the conv launch below declines, this pass has only filled its own buffer: harmless)
        ce = launch_unfold(a, (int)n_in, P.kpad, net->ws + P.unf_off, net->stream);
        if (ce != cudaSuccess) return fail(IDF_ERR_CUDA, "kernel launch failed at layer %zu: %s", i, cudaGetErrorString(ce));
        net->launches += 1;
        t.in = net->ws + P.unf_off;
        t.Win = a.Wout; t.Cin = P.kpad; t.Kw = 1; t.stride_x = 1; t.pad_x = 0;
    }
    ce = launch_conv_tc(t, P.tc_pool, net->dtype, P.w_map_pool, (int)n_in, (unsigned int*)(net->ws + net->status_off), net->stream);
    if (net->timing) {
        if (ce == cudaSuccess) {
            cudaEventRecord(ev_b, net->stream);
            net->timed.push_back({(int)i, ev_a, ev_b});
        } else {
            // a declined launch is no layer time: the layer runs again through launch_layer, which records its own pair
            net->event_pool.push_back(ev_a);
            net->event_pool.push_back(ev_b);
        }
    }
    if (ce == cudaErrorNotSupported) return 1;
    if (ce != cudaSuccess) return fail(IDF_ERR_CUDA, "kernel launch failed at layer %zu: %s", i, cudaGetErrorString(ce));
    net->launches += 1;
    P.tc_launches += 1;
    P.rows_in = r1; P.rows_done = done_end;
    Q.rows_in = done_end; Q.rows_done = q_done;
    *n_out_p = n_out;
    return IDF_OK;
}

// Depth-first schedule.  Rows a layer emits wait in the next layer's buffer; that layer runs ("fires")
// once a block's worth of rows (fire_rows) has gathered, when a push ends, or when its buffer could not
// take what is about to arrive.  So a pooled, narrower layer runs less often on as many rows, and a
// push of one segment still walks every layer it can reach before the call returns.
int fire(idf_net* net, size_t i, const void* in_ptr, long long n_in, bool flush, void* d_out, long long out_cap,
         long long* emitted);
int run_segments_eager(idf_net* net, const void* d_segments, long long n_seg, bool flush, void* d_out, long long out_cap,
                       long long* emitted);
int run_segments_fused(idf_net* net, const void* d_segments, long long n_seg, bool flush, void* d_out, long long out_cap,
                       long long* emitted);

int ensure_space(idf_net* net, size_t m, long long need, void* d_out, long long out_cap, long long* emitted)
{
    LayerPlan& Q = net->L[m];
    if (Q.pending + need <= net->L[m - 1].out_cap_rows) return IDF_OK;
    return fire(net, m, net->ws + net->L[m - 1].out_off, Q.pending, false, d_out, out_cap, emitted);
}

int fire(idf_net* net, size_t i, const void* in_ptr, long long n_in, bool flush, void* d_out, long long out_cap,
         long long* emitted)
{
    LayerPlan& P = net->L[i];
    const bool last = (i + 1 == net->L.size());
    const long long r1 = P.rows_in + n_in;
    const long long n1 = std::max(0LL, layer_done_after(P, r1) - P.rows_done);
    const long long n2 = flush ? std::max(0LL, layer_rows_at_flush(P, r1) - std::max(P.rows_done, layer_done_after(P, r1))) : 0;
    if (P.fuse_pool && n_in > 0 && net->L[i + 1].pending == 0 && net->L[i + 1].rows_in == P.rows_done) {
        // conv + pool in one launch: the pooled rows go straight to the buffer behind the pool layer
        LayerPlan& Q = net->L[i + 1];
        const bool qlast = (i + 2 == net->L.size());
        const long long n_pool = (P.rows_done + n1 + n2) / 2 - Q.rows_done;
        if (!qlast) {
            int rc = ensure_space(net, i + 2, n_pool, d_out, out_cap, emitted);
            if (rc != IDF_OK) return rc;
        }
        long long got = 0;
        int rc = launch_conv_pool(net, i, in_ptr, n_in, flush, d_out, out_cap, qlast ? 0 : net->L[i + 2].pending, &got);
        if (rc < 0) return rc;
        if (rc == IDF_OK) {
            if (i > 0) P.pending = 0;
            if (qlast) *emitted += got; else net->L[i + 2].pending += got;
            return IDF_OK;
        }
    }
    if (!last) {
        int rc = ensure_space(net, i + 1, n1 + n2, d_out, out_cap, emitted);
        if (rc != IDF_OK) return rc;
    }
    if (i > 0) P.pending = 0;
    long long got = 0;
    if (n_in > 0) {
        // When the end of input comes with the layer's last rows, one launch of a dense layer does both:
        // it applies the rows and completes what then only waits for bottom padding.
        const bool fused = flush && P.l.kind == IDF_CONV && !P.use_sparse;
        int rc = launch_layer(net, i, in_ptr, n_in, fused, d_out, out_cap, last ? 0 : net->L[i + 1].pending, &got);
        if (rc != IDF_OK) return rc;
        if (last) *emitted += got; else net->L[i + 1].pending += got;
        if (fused) flush = false;
    }
    if (flush) {
        // the arriving rows took the ordinary path above; what is left is the padding-only completion
        int rc = launch_layer(net, i, nullptr, 0, true, d_out, out_cap, last ? 0 : net->L[i + 1].pending, &got);
        if (rc != IDF_OK) return rc;
        if (last) *emitted += got; else net->L[i + 1].pending += got;
    }
    return IDF_OK;
}

int run_segments(idf_net* net, const void* d_segments, long long n_seg, bool flush, void* d_out,
                 long long out_cap, long long* emitted)
{
    const size_t nl = net->L.size();
    if (net->eager) return run_segments_eager(net, d_segments, n_seg, flush, d_out, out_cap, emitted);
    if (net->fused_ok && !(debug_flags() & IDF_DEBUG_NO_FUSED) && n_seg <= 65535) {
        // Pushes of one or two segments with so little arithmetic that the per-layer kernels' launches are all there is to
        // them (a small net, a stream or two) take the single launch that keeps the state on chip (measured, one segment
        // per push: toy1d 17.2 -> 12.3 us per push).  Anything larger is better off with the per-layer kernels, which work
        // on all rows and streams of a layer at once, on the tensor cores (mnist2d, one image row per push: 8 streams
        // 26 us per-layer against 30 us in one launch; 4096 streams 114 against 425 us).
        const bool small = n_seg <= 2 && net->macs_per_row * (double)n_seg * net->n_streams < 2e5;
        if (small || (debug_flags() & IDF_DEBUG_FORCE_FUSED)) return run_segments_fused(net, d_segments, n_seg, flush, d_out, out_cap, emitted);
    }
    // capacity of the caller's output first: the rows complete after this call do not depend on the schedule
    {
        long long r = net->L[0].rows_in + n_seg;
        for (size_t i = 0; i < nl; ++i) r = flush ? layer_rows_at_flush(net->L[i], r) : layer_done_after(net->L[i], r);
        if (r - net->out_base > out_cap)
            return fail(IDF_ERR_CAPACITY, "output row %lld does not fit out_capacity_rows=%lld", r - 1, out_cap);
    }
    const size_t seg_bytes = (size_t)net->n_streams * net->in_w * net->in_c * elem_size(net->L[0].in_elem);
    int rc = IDF_OK;
    for (long long s0 = 0; s0 < n_seg && rc == IDF_OK; s0 += net->row_block) {
        const long long n = std::min<long long>(net->row_block, n_seg - s0);
        const bool last_block = s0 + n >= n_seg;
        const bool fin = flush && last_block;          // the input ends with this block: every layer also flushes
        rc = fire(net, 0, (const unsigned char*)d_segments + (size_t)s0 * seg_bytes, n, fin, d_out, out_cap, emitted);
        for (size_t i = 1; i < nl && rc == IDF_OK; ++i) {
            LayerPlan& P = net->L[i];
            if (fin || (P.pending > 0 && (P.pending >= P.fire_rows || last_block)))
                rc = fire(net, i, net->ws + net->L[i - 1].out_off, P.pending, fin, d_out, out_cap, emitted);
        }
    }
    if (flush && n_seg == 0)
        for (size_t i = 0; i < nl && rc == IDF_OK; ++i)
            rc = fire(net, i, i ? net->ws + net->L[i - 1].out_off : nullptr, i ? net->L[i].pending : 0, true, d_out, out_cap, emitted);
    if (rc != IDF_OK) net->phase = FINISHED;      // counters and buffers are no longer consistent: reopen to go on
    return rc;
}

}  // namespace

namespace {

// Rows of layer P reached by rows [lo, hi] of the layer below (its input cone, clipped at the top of the map).
void reach(const LayerPlan& P, long long lo, long long hi, long long* o_lo, long long* o_hi)
{
    if (P.l.kind == IDF_CONV) {
        const long long a = lo + P.l.pad - P.l.kh + 1;
        *o_lo = a <= 0 ? 0 : (a + P.l.stride - 1) / P.l.stride;
        *o_hi = (hi + P.l.pad) / P.l.stride;
    } else {
        *o_lo = lo / 2;
        *o_hi = hi / 2;
    }
}

// Eager emission, one segment at a time: the segment is the input layer's announcement; every layer in turn takes up
// the changes of the rows below that moved, re-evaluates the rows of its cone and announces their changes.
int eager_step(idf_net* net, const void* seg, long long r, void* d_out, long long out_cap)
{
    const long long S = net->n_streams;
    const bool int_net = net->dtype == IDF_I8_I32;
    unsigned long long* counters = (unsigned long long*)(net->ws + net->counters_off);
    cudaError_t ce = launch_eager_input(seg, net->L[0].in_elem, net->ws + net->eager_in_off, S * net->in_w * net->in_c,
                                        counters, net->stream);
    if (ce != cudaSuccess) return fail(IDF_ERR_CUDA, "kernel launch failed (eager input): %s", cudaGetErrorString(ce));
    net->launches += 1;
    long long lo = r, hi = r;
    for (size_t i = 0; i < net->L.size(); ++i) {
        LayerPlan& P = net->L[i];
        const bool last = i + 1 == net->L.size();
        long long o_lo, o_hi;
        reach(P, lo, hi, &o_lo, &o_hi);
        EagerArgs a{};
        a.din = i == 0 ? net->ws + net->eager_in_off : net->ws + net->L[i - 1].e_d_off;
        a.hin = i == 0 ? nullptr : net->ws + net->L[i - 1].e_h_off;
        a.c = net->ws + P.e_c_off; a.h = net->ws + P.e_h_off; a.d = net->ws + P.e_d_off;
        a.w = net->ws + P.w_off;
        a.bias = P.b_packed.empty() ? nullptr : net->ws + P.b_off;
        a.out = last ? d_out : nullptr;
        a.out_row_stride = (long long)P.out_w * P.out_c;
        a.out_stream_stride = out_cap * a.out_row_stride;
        a.events = last ? nullptr : counters + i + 1;
        a.S = (int)S; a.Win = P.in_w; a.Wout = P.out_w; a.Cin = P.in_c; a.Cout = P.out_c;
        a.Kh = P.l.kh; a.Kw = P.l.kw; a.stride = P.l.stride; a.pad = P.l.pad;
        a.stride_x = P.in_w == 1 ? 1 : P.l.stride; a.pad_x = P.in_w == 1 ? 0 : P.l.pad;
        a.relu = P.l.relu; a.shift = P.l.shift; a.round_bf16 = P.out_elem == E_BF16;
        a.cap_in = i == 0 ? 1 : net->L[i - 1].e_cap; a.cap = P.e_cap;
        a.in_lo = lo; a.in_hi = P.l.kind == IDF_MAXPOOL2 ? net->L[i - 1].e_hi : hi;
        a.o_lo = o_lo; a.o_hi = o_hi; a.o_new = P.e_hi + 1; a.o_cut = (1LL << 62);
        a.in_elems = i == 0 ? S * net->in_w * net->in_c : (long long)net->L[i - 1].e_cap * S * P.in_w * P.in_c;
        a.ring_elems = (long long)P.e_cap * S * P.out_w * P.out_c;
        a.out_elems = S * out_cap * P.out_w * P.out_c;
        a.status = (unsigned int*)(net->ws + net->status_off);
        if (o_hi - o_lo + 1 > P.e_window) return fail(IDF_ERR_CAPACITY, "internal: layer %zu cone of %lld rows exceeds %d", i, o_hi - o_lo + 1, P.e_window);
        ce = launch_eager_layer(a, P.l.kind == IDF_MAXPOOL2, int_net, net->stream);
        if (ce != cudaSuccess) return fail(IDF_ERR_CUDA, "kernel launch failed at layer %zu: %s", i, cudaGetErrorString(ce));
        net->launches += 1;
        if (o_hi > P.e_hi) P.e_hi = o_hi;
        lo = o_lo; hi = o_hi;
    }
    return IDF_OK;
}

// Rows of the last layer that no later segment can reach once `rows` segments have arrived.
long long eager_final_rows(const idf_net* net, long long rows)
{
    long long lo = rows, hi = rows;
    for (const auto& P : net->L) reach(P, lo, hi, &lo, &hi);
    return lo;
}

// End of input: units of rows that turn out to lie beyond the maps (their receptive field was cut off by the end of
// the input, or they only existed as a first half of a pooling pair) take back what they announced, layer by layer.
int eager_finish(idf_net* net, void* d_out, long long out_cap)
{
    const long long S = net->n_streams;
    const bool int_net = net->dtype == IDF_I8_I32;
    unsigned long long* counters = (unsigned long long*)(net->ws + net->counters_off);
    long long h = net->L[0].rows_in;
    bool changed = false;
    long long lo = 0, hi = -1;
    for (size_t i = 0; i < net->L.size(); ++i) {
        LayerPlan& P = net->L[i];
        const bool last = i + 1 == net->L.size();
        h = layer_rows_at_flush(P, h);                       // rows this layer's map really has
        long long p_lo = (1LL << 62), p_hi = -1;
        if (changed) reach(P, lo, hi, &p_lo, &p_hi);
        if (p_hi > P.e_hi) p_hi = P.e_hi;
        if (P.e_hi >= h) { p_lo = std::min(p_lo, h); p_hi = P.e_hi; }
        if (p_hi < p_lo) { changed = false; continue; }
        EagerArgs a{};
        a.din = i == 0 ? net->ws + net->eager_in_off : net->ws + net->L[i - 1].e_d_off;
        a.hin = i == 0 ? nullptr : net->ws + net->L[i - 1].e_h_off;
        a.c = net->ws + P.e_c_off; a.h = net->ws + P.e_h_off; a.d = net->ws + P.e_d_off;
        a.w = net->ws + P.w_off;
        a.bias = P.b_packed.empty() ? nullptr : net->ws + P.b_off;
        a.out = last ? d_out : nullptr;
        a.out_row_stride = (long long)P.out_w * P.out_c;
        a.out_stream_stride = out_cap * a.out_row_stride;
        a.events = last ? nullptr : counters + i + 1;
        a.S = (int)S; a.Win = P.in_w; a.Wout = P.out_w; a.Cin = P.in_c; a.Cout = P.out_c;
        a.Kh = P.l.kh; a.Kw = P.l.kw; a.stride = P.l.stride; a.pad = P.l.pad;
        a.stride_x = P.in_w == 1 ? 1 : P.l.stride; a.pad_x = P.in_w == 1 ? 0 : P.l.pad;
        a.relu = P.l.relu; a.shift = P.l.shift; a.round_bf16 = P.out_elem == E_BF16;
        a.cap_in = i == 0 ? 1 : net->L[i - 1].e_cap; a.cap = P.e_cap;
        a.in_lo = changed ? lo : 1; a.in_hi = changed ? hi : 0;
        if (P.l.kind == IDF_MAXPOOL2) a.in_hi = net->L[i - 1].e_hi;
        a.o_lo = p_lo; a.o_hi = p_hi; a.o_new = P.e_hi + 1; a.o_cut = h;
        a.in_elems = i == 0 ? S * net->in_w * net->in_c : (long long)net->L[i - 1].e_cap * S * P.in_w * P.in_c;
        a.ring_elems = (long long)P.e_cap * S * P.out_w * P.out_c;
        a.out_elems = S * out_cap * P.out_w * P.out_c;
        a.status = (unsigned int*)(net->ws + net->status_off);
        // (rows beyond the caller's buffer are not written: they hold nothing the caller will read)
        if (last && a.o_hi >= out_cap) a.o_hi = out_cap - 1;
        cudaError_t ce = launch_eager_layer(a, P.l.kind == IDF_MAXPOOL2, int_net, net->stream);
        if (ce != cudaSuccess) return fail(IDF_ERR_CUDA, "kernel launch failed at layer %zu: %s", i, cudaGetErrorString(ce));
        net->launches += 1;
        changed = true; lo = p_lo; hi = p_hi;
    }
    return IDF_OK;
}

int run_segments_eager(idf_net* net, const void* d_segments, long long n_seg, bool flush, void* d_out, long long out_cap,
                       long long* emitted)
{
    const size_t seg_bytes = (size_t)net->n_streams * net->in_w * net->in_c * elem_size(net->L[0].in_elem);
    const long long r0 = net->L[0].rows_in;
    // every row the pushed segments touch in the last layer is written (finished rows and, above them, the rows of
    // the cone with their current partial activations): all of them must fit the caller's buffer
    if (n_seg > 0) {
        long long lo = r0 + n_seg - 1, hi = lo;
        for (const auto& P : net->L) reach(P, lo, hi, &lo, &hi);
        if (hi + 1 > out_cap)
            return fail(IDF_ERR_CAPACITY, "eager emission writes output rows up to %lld: out_capacity_rows=%lld is too small", hi, out_cap);
    }
    int rc = IDF_OK;
    for (long long k = 0; k < n_seg && rc == IDF_OK; ++k) {
        rc = eager_step(net, (const unsigned char*)d_segments + (size_t)k * seg_bytes, r0 + k, d_out, out_cap);
        if (rc == IDF_OK) net->L[0].rows_in = r0 + k + 1;
    }
    long long done = eager_final_rows(net, net->L[0].rows_in);
    if (rc == IDF_OK && flush) {
        rc = eager_finish(net, d_out, out_cap);
        long long h = net->L[0].rows_in;
        for (const auto& P : net->L) h = layer_rows_at_flush(P, h);
        done = h;
        if (rc == IDF_OK && done > out_cap) rc = fail(IDF_ERR_CAPACITY, "output row %lld does not fit out_capacity_rows=%lld", done - 1, out_cap);
    }
    if (rc != IDF_OK) { net->phase = FINISHED; return rc; }
    LayerPlan& Z = net->L.back();
    if (done < Z.rows_done) done = Z.rows_done;
    *emitted += done - Z.rows_done;
    Z.rows_done = done;
    return IDF_OK;
}

}  // namespace

namespace {

// One launch for the whole push: every segment through every layer, state in shared memory (depth_first_kernel).
int run_segments_fused(idf_net* net, const void* d_segments, long long n_seg, bool flush, void* d_out, long long out_cap,
                       long long* emitted)
{
    const size_t nl = net->L.size();
    // rows complete after this call, layer by layer (the schedule inside the kernel follows the same closed forms)
    std::vector<long long> in_after(nl), done_after(nl);
    long long r = net->L[0].rows_in + n_seg;
    for (size_t i = 0; i < nl; ++i) {
        in_after[i] = r;
        r = flush ? layer_rows_at_flush(net->L[i], r) : layer_done_after(net->L[i], r);
        r = std::max(r, net->L[i].rows_done);
        done_after[i] = r;
    }
    if (r - net->out_base > out_cap)
        return fail(IDF_ERR_CAPACITY, "output row %lld does not fit out_capacity_rows=%lld", r - 1, out_cap);
    if (n_seg == 0 && !flush) return IDF_OK;
    FusedArgs a{};
    a.n_layers = (int)nl; a.S = net->n_streams; a.G = net->fused_G;
    a.in = d_segments; a.n_seg = (int)n_seg; a.in_w = net->in_w; a.in_c = net->in_c; a.in_elem = net->L[0].in_elem;
    a.in_soff = net->fused_in_soff; a.flush = flush ? 1 : 0;
    a.weights = net->ws;
    a.out = d_out; a.out_cap = out_cap; a.out_elem = net->L.back().out_elem;
    a.out_row0 = (int)(net->L.back().rows_done - net->out_base);
    a.counters = (unsigned long long*)(net->ws + net->counters_off);
    a.status = (unsigned int*)(net->ws + net->status_off);
    for (size_t i = 0; i < nl; ++i) {
        const LayerPlan& P = net->L[i];
        FusedLayer& F = a.layer[i];
        F.kind = P.l.kind == IDF_CONV ? 0 : 1;
        F.Cin = P.in_c; F.Cout = P.out_c; F.Kh = P.l.kh; F.Kw = P.l.kw; F.stride = P.l.stride; F.pad = P.l.pad;
        F.stride_x = P.in_w == 1 ? 1 : P.l.stride; F.pad_x = P.in_w == 1 ? 0 : P.l.pad;
        F.relu = P.l.relu; F.shift = P.l.shift; F.round_bf16 = P.out_elem == E_BF16;
        F.Win = P.in_w; F.Wout = P.out_w; F.ring_rows = P.ring_rows; F.count_events = P.use_sparse; F.out_elem = P.out_elem;
        F.state_soff = net->fused_state_soff[i]; F.rowbuf_soff = net->fused_rowbuf_soff[i];
        F.w_off = (long long)(net->dtype == IDF_I8_I32 ? P.w_off : P.w_off / 4);
        F.wq_off = net->dtype == IDF_I8_I32 ? (P.wq_packed.empty() ? -1 : (long long)P.wq_off) : 0;
        F.bias_off = P.b_packed.empty() ? -1 : (long long)P.b_off;
        F.state = net->ws + P.state_off;
        if (F.kind == 0) {
            const long long t0 = P.rows_in + P.l.pad, hi = t0 / P.l.stride, tf = t0 - (P.l.kh - 1);
            F.ph0 = (int)(t0 % P.l.stride);
            F.hi_slot0 = (int)(hi % P.ring_rows);
            F.hi_sat0 = (int)std::min<long long>(hi, 1 << 20);
            F.tf_neg0 = tf < 0 ? (int)-tf : 0;
            F.phf0 = tf < 0 ? 0 : (int)(tf % P.l.stride);
            F.done_slot0 = (int)(P.rows_done % P.ring_rows);
            // rows that complete only because the input ends: those of the final map that the rows received do not complete
            F.n_flush = flush ? (int)std::max<long long>(0, conv_rows_at_flush(P.l, in_after[i]) -
                                                             std::max(conv_done_after(P.l, in_after[i]), P.rows_done)) : 0;
        } else {
            F.ph0 = (int)(P.rows_in & 1);
        }
    }
    cudaError_t ce = launch_depth_first(a, net->dtype == IDF_I8_I32, net->fused_threads, net->fused_smem, net->stream);
    if (ce != cudaSuccess) { net->phase = FINISHED; return fail(IDF_ERR_CUDA, "kernel launch failed (all layers in one): %s", cudaGetErrorString(ce)); }
    net->launches += 1;
    const long long before = net->L.back().rows_done;
    for (size_t i = 0; i < nl; ++i) { net->L[i].rows_in = in_after[i]; net->L[i].rows_done = done_after[i]; net->L[i].pending = 0; }
    *emitted += net->L.back().rows_done - before;
    return IDF_OK;
}

}  // namespace

namespace {
std::atomic<unsigned> g_debug_flags{0};
}
namespace idf {
int set_last_error(int code, const char* msg) { return fail(code, "%s", msg); }
unsigned debug_flags() { return g_debug_flags.load(std::memory_order_relaxed); }
}  // namespace idf

extern "C" {

const char* idf_last_error(void) { return g_err.c_str(); }

int idf_set_debug_flags(unsigned int flags)
{
    if (flags & ~(unsigned)(IDF_DEBUG_NO_TENSOR_CORES | IDF_DEBUG_NO_POOL_FUSION | IDF_DEBUG_NO_ROW_CHUNKS | IDF_DEBUG_NO_PDL | IDF_DEBUG_PREFER_THIN | IDF_DEBUG_NO_FUSED | IDF_DEBUG_FORCE_FUSED))
        return fail(IDF_ERR_ARG, "unknown debug flag in 0x%x", flags);
    g_debug_flags.store(flags, std::memory_order_relaxed);
    return IDF_OK;
}

int idf_net_create(const idf_spec* spec, const void* const* weights, const void* const* biases, idf_net** out)
{
    if (!spec || !out) return fail(IDF_ERR_ARG, "spec and out must not be NULL");
    *out = nullptr;
    if (!spec->layers || spec->n_layers < 1 || spec->n_layers > 256) return fail(IDF_ERR_ARG, "n_layers must be 1..256");
    if (!weights) return fail(IDF_ERR_ARG, "weights must not be NULL");
    if (spec->dtype < IDF_F32 || spec->dtype > IDF_I8_I32) return fail(IDF_ERR_SPEC, "unknown dtype %d", spec->dtype);
    if (spec->in_w < 1 || spec->in_c < 1) return fail(IDF_ERR_SPEC, "in_w and in_c must be positive");
    if (spec->n_streams < 1) return fail(IDF_ERR_SPEC, "n_streams must be positive");
    if (spec->row_block < 0 || spec->row_block > 4096) return fail(IDF_ERR_SPEC, "row_block must be 0..4096");
    if (spec->emission != IDF_EMIT_DEFERRED && spec->emission != IDF_EMIT_EAGER) return fail(IDF_ERR_SPEC, "unknown emission policy %d", spec->emission);
    if (spec->emission == IDF_EMIT_EAGER) {
        if (spec->layers[0].kind != IDF_CONV) return fail(IDF_ERR_UNSUPPORTED, "eager emission: the first layer must be a conv layer");
        for (int i = 0; i < spec->n_layers; ++i)
            if (spec->layers[i].kind == IDF_GLOBAL_AVG) return fail(IDF_ERR_UNSUPPORTED, "eager emission: no global-average sink (use a whole-map conv layer as the output unit)");
    }

    idf_net* net = new (std::nothrow) idf_net();
    if (!net) return fail(IDF_ERR_ARG, "out of host memory");
    net->dtype = spec->dtype; net->in_w = spec->in_w; net->in_c = spec->in_c; net->n_streams = spec->n_streams;
    net->eager = spec->emission == IDF_EMIT_EAGER;
    // default: about 25 000 positions per stream and block (112 rows of a 224-wide image, 1024 samples of a 1D
    // signal): long enough that a launch's fixed cost (weights into shared memory, ring rows in and out) is small
    // (1D signals: 4096 samples - fewer launches and fewer rows read twice at the edges of row chunks; audio1d 2.9 -> 2.3 ms)
    net->row_block = spec->row_block > 0 ? spec->row_block : (spec->in_w == 1 ? 4096 : std::min(1024, std::max(32, 25088 / spec->in_w)));
    const int act_elem = spec->dtype == IDF_F32 ? E_F32 : (spec->dtype == IDF_BF16_F32 ? E_BF16 : E_I8);
    const size_t state_word = 4;

    int last_conv = -1;
    for (int i = 0; i < spec->n_layers; ++i)
        if (spec->layers[i].kind == IDF_CONV) last_conv = i;
    if (last_conv < 0) { delete net; return fail(IDF_ERR_SPEC, "a net needs at least one conv layer"); }

    int w = spec->in_w, c = spec->in_c, elem = act_elem;
    int cap = net->row_block;
    net->L.resize(spec->n_layers);
    for (int i = 0; i < spec->n_layers; ++i) {
        LayerPlan& P = net->L[i];
        P.l = spec->layers[i];
        P.in_w = w; P.in_c = c; P.in_elem = elem;
        const idf_layer& l = P.l;
        if (l.kind == IDF_CONV) {
            if (l.cin != c) { delete net; return fail(IDF_ERR_SPEC, "layer %d: cin=%d but the incoming map has %d channels", i, l.cin, c); }
            if (l.cout < 1 || l.kh < 1 || l.kw < 1) { delete net; return fail(IDF_ERR_SPEC, "layer %d: cout, kh, kw must be positive", i); }
            if (l.stride < 1 || l.stride > l.kh) { delete net; return fail(IDF_ERR_SPEC, "layer %d: stride must be 1..kh", i); }
            if (l.pad < 0 || l.pad >= l.kh) { delete net; return fail(IDF_ERR_SPEC, "layer %d: pad must be 0..kh-1", i); }
            if (w == 1 && l.kw != 1) { delete net; return fail(IDF_ERR_SPEC, "layer %d: a width-1 map needs kw == 1", i); }
            if (l.shift < 0 || l.shift > 30) { delete net; return fail(IDF_ERR_SPEC, "layer %d: shift must be 0..30", i); }
            if (l.path < IDF_PATH_AUTO || l.path > IDF_PATH_SPARSE) { delete net; return fail(IDF_ERR_SPEC, "layer %d: unknown path", i); }
            if (!weights[i]) { delete net; return fail(IDF_ERR_ARG, "layer %d: weights missing", i); }
            const int padw = (w == 1) ? 0 : l.pad;     // 1D nets pad the streaming axis only
            if (w + 2 * padw < l.kw) { delete net; return fail(IDF_ERR_SPEC, "layer %d: kernel wider than the padded row", i); }
            P.out_w = (w + 2 * padw - l.kw) / l.stride + 1;
            if (w == 1) P.out_w = 1;
            P.out_c = l.cout;
            P.ring_rows = (l.kh + l.stride - 1) / l.stride;
            P.out_elem = spec->dtype == IDF_F32 ? E_F32
                       : spec->dtype == IDF_I8_I32 ? E_I8
                       : (i == last_conv ? E_F32 : E_BF16);
            // sparse path by default only for the thin first layer of an integer net (raw, sparse input)
            P.use_sparse = l.path == IDF_PATH_SPARSE ||
                           (l.path == IDF_PATH_AUTO && i == 0 && spec->dtype == IDF_I8_I32 && l.cin <= 4);
            P.state_bytes_stream = (size_t)P.ring_rows * P.out_w * P.out_c * state_word;
            cap = std::max(2 * net->row_block + 8, (cap + l.stride - 1) / l.stride + 1 + P.ring_rows);
            // parameters -> [Kh][Kw][Cin][Cout]
            const size_t nw = (size_t)l.cout * l.kh * l.kw * l.cin;
            if (spec->dtype == IDF_I8_I32) {
                P.w_packed.resize(nw);
                const int8_t* src = (const int8_t*)weights[i];
                for (int co = 0; co < l.cout; ++co)
                    for (int k = 0; k < l.kh * l.kw; ++k)
                        for (int ci = 0; ci < l.cin; ++ci)
                            ((int8_t*)P.w_packed.data())[((size_t)k * l.cin + ci) * l.cout + co] =
                                src[((size_t)co * l.kh * l.kw + k) * l.cin + ci];
            } else {
                P.w_packed.resize(nw * 4);
                float* dst = (float*)P.w_packed.data();
                for (int co = 0; co < l.cout; ++co)
                    for (int k = 0; k < l.kh * l.kw; ++k)
                        for (int ci = 0; ci < l.cin; ++ci) {
                            const size_t si = ((size_t)co * l.kh * l.kw + k) * l.cin + ci;
                            const float v = spec->dtype == IDF_F32 ? ((const float*)weights[i])[si]
                                                                  : bf16_bits_to_float(((const uint16_t*)weights[i])[si]);
                            dst[((size_t)k * l.cin + ci) * l.cout + co] = v;
                        }
            }
            // tensor-core layout [tap slot][Cout][Cin], activation type, when the layer qualifies
            const int in_cap = i == 0 ? net->row_block : net->L[i - 1].out_cap_rows;
            const bool tc_allowed = !P.use_sparse && !(debug_flags() & IDF_DEBUG_NO_TENSOR_CORES) && spec->dtype != IDF_F32 && !net->eager;
            const size_t es = spec->dtype == IDF_I8_I32 ? 1 : 2;
            const int taps = l.kh * l.kw;
            const bool pool_next = i + 1 < spec->n_layers && spec->layers[i + 1].kind == IDF_MAXPOOL2;
            if (tc_allowed && tc_make_plan(spec->dtype, net->n_streams, w, P.out_w, l.cin, l.cout, l.kh, l.kw,
                                           w == 1 ? 1 : l.stride, P.ring_rows, (int)elem_size(P.out_elem), 0, &P.tc)) {
                if (pool_next)
                    tc_make_plan(spec->dtype, net->n_streams, w, P.out_w, l.cin, l.cout, l.kh, l.kw, w == 1 ? 1 : l.stride,
                                 P.ring_rows, (int)elem_size(P.out_elem), 1, &P.tc_pool);
                P.wtc_packed.resize(nw * es);
                for (int co = 0; co < l.cout; ++co)
                    for (int k = 0; k < taps; ++k)
                        memcpy(P.wtc_packed.data() + (((size_t)tc_weight_slot(k / l.kw, k % l.kw, l.kh, l.stride) * l.cout + co) * l.cin) * es,
                               (const unsigned char*)weights[i] + (((size_t)co * taps + k) * l.cin) * es, (size_t)l.cin * es);
            } else if (tc_allowed) {
                // thin (Cin*Kw below a tensor-core K step) or x-strided layer: unfold x first
                const size_t kbytes = (size_t)l.kw * l.cin * es;
                const size_t padded = kbytes <= 32 ? 32 : (kbytes <= 64 ? 64 : (kbytes + 127) / 128 * 128);
                const int kpad = (int)(padded / es);
                if (padded <= 1024 &&
                    tc_make_plan(spec->dtype, net->n_streams, P.out_w, P.out_w, kpad, l.cout, l.kh, 1, 1, P.ring_rows,
                                 (int)elem_size(P.out_elem), 0, &P.tc)) {
                    if (pool_next)
                        tc_make_plan(spec->dtype, net->n_streams, P.out_w, P.out_w, kpad, l.cout, l.kh, 1, 1, P.ring_rows,
                                     (int)elem_size(P.out_elem), 1, &P.tc_pool);
                    P.unfold = 1;
                    P.kpad = kpad;
                    P.in_cap_rows = in_cap;
                    P.wtc_packed.assign((size_t)l.kh * l.cout * kpad * es, 0);      // [ky][Cout][kx*Cin + ci], zero padded
                    for (int co = 0; co < l.cout; ++co)
                        for (int ky = 0; ky < l.kh; ++ky)
                            memcpy(P.wtc_packed.data() + (((size_t)tc_weight_slot(ky, 0, l.kh, l.stride) * l.cout + co) * kpad) * es,
                                   (const unsigned char*)weights[i] + (((size_t)co * l.kh + ky) * l.kw * l.cin) * es,
                                   (size_t)l.kw * l.cin * es);
                }
            }
            // A layer whose whole receptive field fits one 128-byte row gets the thin-layer kernel where the row-ring kernel
            // has no good form for it: 1D nets (behind an x-unfold pass every tap row would carry Cin values padded to a
            // K step: audio1d's first layer 1.68 -> 0.84 ms) and shapes it cannot take at all.  2D layers with kx taps stay
            // with x-unfold + row ring (vgg2d conv1: 0.19 ms against 0.52 ms: building 27-value rows element by element
            // costs more than the unfold pass saves).
            const bool prefer_thin = (debug_flags() & IDF_DEBUG_PREFER_THIN) != 0;
            if (tc_allowed && ((P.unfold && (w == 1 || prefer_thin)) || !P.tc.ok) && !(pool_next && P.tc_pool.ok) &&
                thin_make_plan(spec->dtype, net->n_streams, P.out_w, l.cin, l.cout, l.kh, l.kw, l.stride, w == 1 ? 1 : l.stride,
                               (int)elem_size(P.out_elem), &P.thin)) {
                P.wthin_packed.assign((size_t)l.cout * P.thin.swb, 0);
                for (int co = 0; co < l.cout; ++co)
                    memcpy(P.wthin_packed.data() + (size_t)co * P.thin.swb, (const unsigned char*)weights[i] + (size_t)co * taps * l.cin * es,
                           (size_t)taps * l.cin * es);
            }
            if (spec->dtype == IDF_I8_I32 && l.cin % 4 == 0) {
                P.wq_packed.resize((size_t)taps * l.cin * l.cout);
                const int8_t* src = (const int8_t*)weights[i];
                for (int co = 0; co < l.cout; ++co)
                    for (int k = 0; k < taps; ++k)
                        for (int ci = 0; ci < l.cin; ++ci)
                            P.wq_packed[((((size_t)k * (l.cin / 4) + ci / 4) * l.cout + co) * 4) + (ci & 3)] =
                                (unsigned char)src[((size_t)co * taps + k) * l.cin + ci];
            }
            if (biases && biases[i]) {
                // an all-zero bias is no bias: the kernels then skip the add (state words: +0.0f and 0 are all-zero bits)
                bool any = false;
                for (size_t k = 0; k < (size_t)l.cout * 4 && !any; ++k) any = ((const unsigned char*)biases[i])[k] != 0;
                if (any) {
                    P.b_packed.resize((size_t)l.cout * 4);
                    memcpy(P.b_packed.data(), biases[i], (size_t)l.cout * 4);
                }
            }
        } else if (l.kind == IDF_MAXPOOL2) {
            P.out_w = (w == 1) ? 1 : w / 2;
            if (P.out_w < 1) { delete net; return fail(IDF_ERR_SPEC, "layer %d: pooling an empty row", i); }
            P.out_c = c;
            P.ring_rows = 1;
            P.out_elem = elem;
            P.use_sparse = 0;
            P.state_bytes_stream = (size_t)P.out_w * P.out_c * elem_size(elem);
            cap = std::max(2 * net->row_block + 8, cap / 2 + 1);
        } else if (l.kind == IDF_GLOBAL_AVG) {
            if (i + 1 != spec->n_layers) { delete net; return fail(IDF_ERR_SPEC, "layer %d: a global-average sink must be the last layer", i); }
            P.out_w = 1;
            P.out_c = c;
            P.ring_rows = 1;
            P.out_elem = E_F32;
            P.use_sparse = 0;
            P.state_bytes_stream = (size_t)c * state_word;      // one running sum per channel
        } else {
            delete net;
            return fail(IDF_ERR_SPEC, "layer %d: unknown kind %d", i, l.kind);
        }
        P.out_cap_rows = cap;      // rows the buffer behind this layer holds: a block in waiting plus one arrival
        P.fire_rows = net->row_block;
        P.state_bytes_all = P.state_bytes_stream * (size_t)net->n_streams;
        net->state_bytes_stream += P.state_bytes_stream;
        w = P.out_w; c = P.out_c; elem = P.out_elem;
    }
    if (net->eager) {
        // rows of every layer that one segment can touch (its input cone): the most over a long run of segments
        for (long long r = 0; r < 4096; ++r) {
            long long lo = r, hi = r;
            for (auto& P : net->L) {
                reach(P, lo, hi, &lo, &hi);
                P.e_window = std::max<long long>(P.e_window, hi - lo + 1);
            }
        }
        net->state_bytes_stream = 0;
        for (auto& P : net->L) {
            P.e_cap = P.e_window + 2;      // (a pooling layer above still reads the two rows below its oldest open pair)
            P.out_cap_rows = 0;
            P.state_bytes_stream = (size_t)P.e_window * P.out_w * P.out_c * 8;       // state and announced activation
            P.state_bytes_all = (size_t)3 * P.e_cap * net->n_streams * P.out_w * P.out_c * 4;
            net->state_bytes_stream += P.state_bytes_stream;
        }
    }
    // a dense tensor-core conv layer directly followed by a 2x2 max-pool emits the pooled rows itself
    {
        const bool no_fuse = (debug_flags() & IDF_DEBUG_NO_POOL_FUSION) != 0;
        for (size_t i = 0; i + 1 < net->L.size(); ++i) {
            LayerPlan& P = net->L[i];
            P.fuse_pool = P.l.kind == IDF_CONV && net->L[i + 1].l.kind == IDF_MAXPOOL2 && P.tc.ok && P.tc_pool.ok && !P.use_sparse &&
                          P.out_w >= 2 && (P.tc_pool.BX % 2) == 0 && !no_fuse && !net->eager;
        }
    }
    // one launch for all layers, state in shared memory: possible when a stream's rings, pooling rows and one row per
    // layer boundary are small enough for at least one stream per CTA
    if (!net->eager && (int)net->L.size() <= FUSED_MAX_LAYERS) {
        bool ok = true;
        size_t words = (size_t)net->in_w * net->in_c;
        double macs = 0, rate = 1;
        for (const auto& P : net->L) {
            if (P.l.kind == IDF_GLOBAL_AVG) { ok = false; break; }
            words += (size_t)(P.l.kind == IDF_CONV ? P.ring_rows : 1) * P.out_w * P.out_c + (size_t)P.out_w * P.out_c;
            if (P.l.kind == IDF_CONV) { rate /= P.l.stride; macs += rate * P.out_w * P.out_c * (double)P.l.kh * P.l.kw * P.l.cin; }
            else rate /= 2;
        }
        net->macs_per_row = macs;
        // rows between layers: fp32 values or int8; rings: words
        const size_t rs = spec->dtype == IDF_I8_I32 ? 1 : 4;
        size_t per_stream = (size_t)net->in_w * net->in_c * rs;
        for (const auto& P : net->L)
            per_stream += (P.l.kind == IDF_CONV ? (size_t)P.ring_rows * P.out_w * P.out_c * 4 : (size_t)P.out_w * P.out_c * rs) +
                          (size_t)P.out_w * P.out_c * rs;
        (void)words;
        if (ok && per_stream + 64 * net->L.size() <= FUSED_SMEM_LIMIT) {
            int G = (int)std::min<size_t>((FUSED_SMEM_LIMIT - 64 * net->L.size()) / per_stream, 32);
            G = std::min(G, net->n_streams);
            // (enough CTAs for the SMs before more streams per CTA)
            while (G > 1 && (net->n_streams + G - 1) / G < 2 * 148) --G;
            net->fused_G = G;
            auto up16 = [](size_t v) { return (v + 15) / 16 * 16; };
            size_t off = 0;
            net->fused_in_soff = 0; off = up16((size_t)G * net->in_w * net->in_c * rs);
            size_t widest = (size_t)G * net->in_w * net->in_c;
            for (const auto& P : net->L) {
                net->fused_state_soff.push_back((int)off);
                off = up16(off + (P.l.kind == IDF_CONV ? (size_t)P.ring_rows * G * P.out_w * P.out_c * 4 : (size_t)G * P.out_w * P.out_c * rs));
                net->fused_rowbuf_soff.push_back((int)off);
                off = up16(off + (size_t)G * P.out_w * P.out_c * rs);
                widest = std::max(widest, (size_t)G * P.out_w * P.out_c);
            }
            net->fused_smem = off;
            net->fused_threads = (int)std::min<size_t>(512, std::max<size_t>(64, (widest + 31) / 32 * 32));
            net->fused_ok = off <= FUSED_SMEM_LIMIT;
        }
    }
    // workspace: [parameters][state of all streams][rows travelling between layers][counters]
    size_t off = 0;
    for (auto& P : net->L) {
        P.w_off = off; off = align_up(off + P.w_packed.size());
        P.b_off = off; off = align_up(off + P.b_packed.size());
        P.wtc_off = off; off = align_up(off + P.wtc_packed.size(), 1024);
        P.wthin_off = off; off = align_up(off + P.wthin_packed.size(), 1024);
        P.wq_off = off; off = align_up(off + P.wq_packed.size());
    }
    net->state_region_off = off;
    for (auto& P : net->L) {
        P.state_off = off;
        if (net->eager) {
            const size_t ring = P.state_bytes_all / 3;
            P.e_c_off = off; P.e_h_off = off + ring; P.e_d_off = off + 2 * ring;
        }
        off = align_up(off + P.state_bytes_all);
    }
    net->state_region_bytes = off - net->state_region_off;
    if (net->eager) { net->eager_in_off = off; off = align_up(off + (size_t)net->n_streams * net->in_w * net->in_c * 4); }
    for (size_t i = 0; i + 1 < net->L.size(); ++i) {
        LayerPlan& P = net->L[i];
        P.out_off = off;
        off = align_up(off + (size_t)P.out_cap_rows * net->n_streams * P.out_w * P.out_c * elem_size(P.out_elem));
    }
    for (auto& P : net->L)
        if (P.unfold) {
            P.unf_off = off;
            off = align_up(off + (size_t)P.in_cap_rows * net->n_streams * P.out_w * P.kpad * elem_size(P.in_elem), 1024);
        }
    {
        size_t biggest = 0;
        for (auto& P : net->L)
            if (P.l.kind == IDF_CONV && P.tc.ok) biggest = std::max(biggest, P.state_bytes_all);
        if (biggest) { net->ring_scratch_off = off; off = align_up(off + biggest); }
    }
    net->counters_off = off;
    off = align_up(off + net->L.size() * sizeof(unsigned long long));
    net->status_off = off;
    off = align_up(off + sizeof(unsigned int));
    net->workspace_bytes = off;
    *out = net;
    return IDF_OK;
}

int idf_net_destroy(idf_net* net)
{
    if (net) {
        for (auto& t : net->timed) { cudaEventDestroy(t.a); cudaEventDestroy(t.b); }
        for (auto e : net->event_pool) cudaEventDestroy(e);
        for (auto e : net->order_events) cudaEventDestroy(e);
        if (net->copy_in) cudaStreamDestroy(net->copy_in);
        if (net->copy_out) cudaStreamDestroy(net->copy_out);
    }
    delete net;
    return IDF_OK;
}

size_t idf_net_state_bytes(const idf_net* net) { return net ? net->state_bytes_stream : 0; }

size_t idf_net_workspace_bytes(const idf_net* net) { return net ? net->workspace_bytes : 0; }

int idf_out_shape(const idf_net* net, long long in_rows, long long* out_rows, int* out_w, int* out_c)
{
    if (!net) return fail(IDF_ERR_ARG, "net must not be NULL");
    if (in_rows < 0) return fail(IDF_ERR_ARG, "in_rows must not be negative");
    long long h = in_rows;
    for (const auto& P : net->L) h = layer_rows_at_flush(P, h);
    if (out_rows) *out_rows = h;
    if (out_w) *out_w = net->L.back().out_w;
    if (out_c) *out_c = net->L.back().out_c;
    return IDF_OK;
}

long long idf_out_rows_needed(const idf_net* net, long long in_rows)
{
    if (!net || in_rows < 0) return -1;
    long long h = in_rows;
    for (const auto& P : net->L) h = layer_rows_at_flush(P, h);
    if (net->eager && in_rows > 0) {
        long long lo = in_rows - 1, hi = lo;
        for (const auto& P : net->L) reach(P, lo, hi, &lo, &hi);
        h = std::max(h, hi + 1);
    }
    return h;
}

int idf_stream_open(idf_net* net, void* d_workspace, size_t workspace_bytes, void* cuda_stream)
{
    if (!net || !d_workspace) return fail(IDF_ERR_ARG, "net and d_workspace must not be NULL");
    if (workspace_bytes < net->workspace_bytes)
        return fail(IDF_ERR_CAPACITY, "workspace has %zu bytes, %zu needed", workspace_bytes, net->workspace_bytes);
    if (((uintptr_t)d_workspace & 255) != 0) return fail(IDF_ERR_ARG, "d_workspace must be 256-byte aligned");
    net->ws = (unsigned char*)d_workspace;
    net->stream = (cudaStream_t)cuda_stream;
    cudaError_t e = cudaSuccess;
    for (auto& P : net->L) {
        if (!P.w_packed.empty() && e == cudaSuccess)
            e = cudaMemcpyAsync(net->ws + P.w_off, P.w_packed.data(), P.w_packed.size(), cudaMemcpyHostToDevice, net->stream);
        if (!P.b_packed.empty() && e == cudaSuccess)
            e = cudaMemcpyAsync(net->ws + P.b_off, P.b_packed.data(), P.b_packed.size(), cudaMemcpyHostToDevice, net->stream);
        if (!P.wtc_packed.empty() && e == cudaSuccess) {
            e = cudaMemcpyAsync(net->ws + P.wtc_off, P.wtc_packed.data(), P.wtc_packed.size(), cudaMemcpyHostToDevice, net->stream);
            if (tc_encode_weights(P.tc, net->dtype, net->ws + P.wtc_off, P.unfold ? P.l.kh : P.l.kh * P.l.kw,
                                  P.unfold ? P.kpad : P.l.cin, P.l.cout, P.w_map) != 0)
                P.tc.ok = 0;               // no TMA descriptor: this layer stays on the CUDA-core kernel
            if (P.tc_pool.ok && tc_encode_weights(P.tc_pool, net->dtype, net->ws + P.wtc_off, P.unfold ? P.l.kh : P.l.kh * P.l.kw,
                                                  P.unfold ? P.kpad : P.l.cin, P.l.cout, P.w_map_pool) != 0)
                P.tc_pool.ok = 0;
        }
        if (!P.wq_packed.empty() && e == cudaSuccess)
            e = cudaMemcpyAsync(net->ws + P.wq_off, P.wq_packed.data(), P.wq_packed.size(), cudaMemcpyHostToDevice, net->stream);
        if (!P.wthin_packed.empty() && e == cudaSuccess) {
            e = cudaMemcpyAsync(net->ws + P.wthin_off, P.wthin_packed.data(), P.wthin_packed.size(), cudaMemcpyHostToDevice, net->stream);
            if (thin_encode_weights(P.thin, net->dtype, net->ws + P.wthin_off, P.l.cout, P.w_map_thin) != 0) P.thin.ok = 0;
        }
    }
    if (e != cudaSuccess) { net->phase = CREATED; return fail(IDF_ERR_CUDA, "stream_open: %s", cudaGetErrorString(e)); }
    net->phase = FINISHED;                 // a bound workspace with uploaded parameters: ready for a reset
    return idf_stream_reset(net);
}

int idf_stream_reset(idf_net* net)
{
    if (!net) return fail(IDF_ERR_ARG, "net must not be NULL");
    if (net->phase == CREATED) return fail(IDF_ERR_STATE, "reset before stream_open");
    for (auto& P : net->L) { P.rows_in = 0; P.rows_done = 0; P.tc_launches = 0; P.pending = 0; P.e_hi = -1; }
    cudaError_t e = cudaMemsetAsync(net->ws + net->status_off, 0, sizeof(unsigned int), net->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(net->ws + net->state_region_off, 0, net->state_region_bytes, net->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(net->ws + net->counters_off, 0, net->L.size() * sizeof(unsigned long long), net->stream);
    if (e != cudaSuccess) { net->phase = CREATED; return fail(IDF_ERR_CUDA, "stream_reset: %s", cudaGetErrorString(e)); }
    net->phase = OPEN;
    net->launches = 0;
    net->out_rows_total = 0;
    net->out_base = 0;
    return IDF_OK;
}

int idf_stream_push(idf_net* net, const void* d_segments, int n_seg, void* d_out, long long out_capacity_rows,
                    int* rows_emitted)
{
    if (!net) return fail(IDF_ERR_ARG, "net must not be NULL");
    if (net->phase != OPEN) return fail(IDF_ERR_STATE, net->phase == CREATED ? "push before stream_open" : "push after stream_finish");
    if (n_seg < 0 || out_capacity_rows < 0) return fail(IDF_ERR_ARG, "negative count");
    if (rows_emitted) *rows_emitted = 0;
    if (n_seg == 0) return IDF_OK;
    if (!d_segments || !d_out) return fail(IDF_ERR_ARG, "d_segments and d_out must not be NULL");
    long long em = 0;
    int rc = run_segments(net, d_segments, n_seg, false, d_out, out_capacity_rows, &em);
    if (rc != IDF_OK) return rc;
    net->out_rows_total += em;
    if (rows_emitted) *rows_emitted = (int)em;
    return IDF_OK;
}

int idf_stream_set_out_base(idf_net* net, long long first_row)
{
    if (!net) return fail(IDF_ERR_ARG, "net must not be NULL");
    if (net->phase != OPEN) return fail(IDF_ERR_STATE, "set_out_base needs open streams");
    if (net->eager && first_row != 0) return fail(IDF_ERR_UNSUPPORTED, "eager emission keeps the output window at row 0");
    if (first_row < 0 || first_row > net->out_rows_total)
        return fail(IDF_ERR_ARG, "first_row=%lld: only rows emitted so far (%lld) can be left behind", first_row, net->out_rows_total);
    net->out_base = first_row;
    return IDF_OK;
}

int idf_stream_finish(idf_net* net, void* d_out, long long out_capacity_rows, long long* total_rows)
{
    if (!net) return fail(IDF_ERR_ARG, "net must not be NULL");
    if (net->phase != OPEN) return fail(IDF_ERR_STATE, net->phase == CREATED ? "finish before stream_open" : "finish called twice");
    if (!d_out || out_capacity_rows < 0) return fail(IDF_ERR_ARG, "d_out must not be NULL");
    long long em = 0;
    int rc = run_segments(net, nullptr, 0, true, d_out, out_capacity_rows, &em);
    if (rc != IDF_OK) return rc;
    net->out_rows_total += em;
    net->phase = FINISHED;
    if (total_rows) *total_rows = net->out_rows_total;
    return IDF_OK;
}

int idf_stream_push_last(idf_net* net, const void* d_segments, int n_seg, void* d_out, long long out_capacity_rows,
                         long long* total_rows)
{
    if (!net) return fail(IDF_ERR_ARG, "net must not be NULL");
    if (net->phase != OPEN) return fail(IDF_ERR_STATE, net->phase == CREATED ? "push before stream_open" : "push after stream_finish");
    if (n_seg < 0 || out_capacity_rows < 0) return fail(IDF_ERR_ARG, "negative count");
    if (!d_out || (n_seg > 0 && !d_segments)) return fail(IDF_ERR_ARG, "d_segments and d_out must not be NULL");
    long long em = 0;
    int rc = run_segments(net, d_segments, n_seg, true, d_out, out_capacity_rows, &em);
    if (rc != IDF_OK) return rc;
    net->out_rows_total += em;
    net->phase = FINISHED;
    if (total_rows) *total_rows = net->out_rows_total;
    return IDF_OK;
}

int idf_run_host(idf_net* net, const void* h_segments, int n_seg, void* d_segments, void* h_out, void* d_out,
                 long long out_capacity_rows, long long* total_rows)
{
    if (!net || !h_segments || !d_segments || !h_out || !d_out) return fail(IDF_ERR_ARG, "NULL argument");
    if (net->phase != OPEN || net->L[0].rows_in != 0) return fail(IDF_ERR_STATE, "run_host needs a freshly opened handle");
    if (n_seg < 0) return fail(IDF_ERR_ARG, "negative count");
    // Pipeline over row blocks: while block b is computed on the handle's stream, block b + 1 travels to the
    // device on a second stream and the output rows block b - 1 completed travel back on a third.
    // Half a row block per step: the first block's way in and the last block's way out are the part of the copies
    // that nothing overlaps, and they shrink with the block, while the launches grow only a little more numerous
    // (vgg2d: 2.20 -> 1.98 ms per batch; a quarter block is slower again).
    const long long pipe = net->row_block >= 2 ? net->row_block / 2 : 1;
    // ... and the first and the last step take half of that again when there are steps enough
    std::vector<long long> cut;                      // segment index where step b starts; cut.back() = n_seg
    {
        const long long edge = (n_seg >= 3 * pipe && pipe >= 2) ? pipe / 2 : 0;
        long long pos = 0;
        cut.push_back(0);
        if (edge) { pos = edge; cut.push_back(pos); }
        while (pos < n_seg - edge) { pos = std::min<long long>(pos + pipe, n_seg - edge); cut.push_back(pos); }
        if (edge) cut.push_back(n_seg);
        if (cut.size() < 2) cut.push_back(n_seg);
    }
    const long long nb = (long long)cut.size() - 1;
    if (!net->copy_in) {
        if (cudaStreamCreateWithFlags(&net->copy_in, cudaStreamNonBlocking) != cudaSuccess ||
            cudaStreamCreateWithFlags(&net->copy_out, cudaStreamNonBlocking) != cudaSuccess)
            return fail(IDF_ERR_CUDA, "run_host: cannot create the copy streams");
    }
    while ((long long)net->order_events.size() < 2 * nb + 1) {
        cudaEvent_t e;
        if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return fail(IDF_ERR_CUDA, "cudaEventCreate failed");
        net->order_events.push_back(e);
    }
    const LayerPlan& P = net->L.back();
    const size_t seg_bytes = (size_t)net->n_streams * net->in_w * net->in_c * elem_size(net->L[0].in_elem);
    const size_t orow_bytes = (size_t)P.out_w * P.out_c * elem_size(P.out_elem);
    const size_t opitch = (size_t)out_capacity_rows * orow_bytes;
    cudaError_t e = cudaEventRecord(net->order_events[0], net->stream);      // earlier work on the caller's stream comes first
    if (e == cudaSuccess) e = cudaStreamWaitEvent(net->copy_in, net->order_events[0], 0);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(net->copy_out, net->order_events[0], 0);
    if (e != cudaSuccess) return fail(IDF_ERR_CUDA, "run_host: %s", cudaGetErrorString(e));
    long long tot = 0, copied = 0;
    for (long long b = 0; b < nb; ++b) {
        const long long s0 = cut[b], n = cut[b + 1] - cut[b];
        const bool last_block = b + 1 == nb;
        cudaEvent_t ev_in = net->order_events[1 + 2 * b], ev_done = net->order_events[2 + 2 * b];
        if (n > 0) {
            e = cudaMemcpyAsync((unsigned char*)d_segments + (size_t)s0 * seg_bytes, (const unsigned char*)h_segments + (size_t)s0 * seg_bytes,
                                (size_t)n * seg_bytes, cudaMemcpyHostToDevice, net->copy_in);
            if (e == cudaSuccess) e = cudaEventRecord(ev_in, net->copy_in);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(net->stream, ev_in, 0);
            if (e != cudaSuccess) return fail(IDF_ERR_CUDA, "run_host h2d: %s", cudaGetErrorString(e));
        }
        const void* blk = (const unsigned char*)d_segments + (size_t)s0 * seg_bytes;
        int rc;
        if (last_block) {
            rc = idf_stream_push_last(net, blk, (int)std::max<long long>(n, 0), d_out, out_capacity_rows, &tot);
        } else {
            int em = 0;
            rc = idf_stream_push(net, blk, (int)n, d_out, out_capacity_rows, &em);
            tot = net->out_rows_total;
        }
        if (rc != IDF_OK) { cudaStreamSynchronize(net->copy_in); cudaStreamSynchronize(net->copy_out); return rc; }
        // (a global-average sink rewrites its one row with every push: it travels once, at the end)
        if (tot > copied && (P.l.kind != IDF_GLOBAL_AVG || last_block)) {
            // output rows [copied, tot) of every stream: a strided copy (one run of rows per stream)
            e = cudaEventRecord(ev_done, net->stream);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(net->copy_out, ev_done, 0);
            if (e == cudaSuccess)
                e = cudaMemcpy2DAsync((unsigned char*)h_out + (size_t)copied * orow_bytes, opitch,
                                      (const unsigned char*)d_out + (size_t)copied * orow_bytes, opitch,
                                      (size_t)(tot - copied) * orow_bytes, (size_t)net->n_streams, cudaMemcpyDeviceToHost, net->copy_out);
            if (e != cudaSuccess) return fail(IDF_ERR_CUDA, "run_host d2h: %s", cudaGetErrorString(e));
            copied = tot;
        }
    }
    e = cudaStreamSynchronize(net->copy_out);
    if (e == cudaSuccess) e = cudaStreamSynchronize(net->copy_in);
    if (e == cudaSuccess) e = cudaStreamSynchronize(net->stream);
    if (e != cudaSuccess) return fail(IDF_ERR_CUDA, "run_host: %s", cudaGetErrorString(e));
    if (total_rows) *total_rows = tot;
    return IDF_OK;
}

int idf_event_counts(idf_net* net, long long* events)
{
    if (!net || !events) return fail(IDF_ERR_ARG, "NULL argument");
    if (net->phase == CREATED) return fail(IDF_ERR_STATE, "no open stream");
    cudaError_t e = cudaMemcpyAsync(events, net->ws + net->counters_off, net->L.size() * sizeof(long long),
                                    cudaMemcpyDeviceToHost, net->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(net->stream);
    if (e != cudaSuccess) return fail(IDF_ERR_CUDA, "event_counts: %s", cudaGetErrorString(e));
    return IDF_OK;
}

long long idf_launch_count(const idf_net* net) { return net ? net->launches : 0; }

int idf_stream_status(idf_net* net, long long* tensor_core_launches)
{
    if (!net) return fail(IDF_ERR_ARG, "net must not be NULL");
    if (net->phase == CREATED) return fail(IDF_ERR_STATE, "no open stream");
    unsigned int st = 0;
    cudaError_t e = cudaMemcpyAsync(&st, net->ws + net->status_off, sizeof st, cudaMemcpyDeviceToHost, net->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(net->stream);
    if (e != cudaSuccess) return fail(IDF_ERR_CUDA, "stream_status: %s", cudaGetErrorString(e));
    if (tensor_core_launches)
        for (size_t i = 0; i < net->L.size(); ++i) tensor_core_launches[i] = net->L[i].tc_launches;
    if (st & 2u) return fail(IDF_ERR_BOUNDS, "an index check of the range-checked build failed (the access was skipped; results are invalid)");
    if (st != 0) return fail(IDF_ERR_TIMEOUT, "a bounded device-side wait ran out (kernel gave up)");
    return IDF_OK;
}

// Snapshot of the streams' progress: a fixed header (what net it belongs to, how far every layer has
// come) followed by the rolling state of all streams and the sparse-path event counters.
namespace {
struct SnapshotHeader {
    unsigned long long magic;
    unsigned long long fingerprint;        // of the net's shape: a snapshot only fits a net built from the same spec
    unsigned long long state_region_bytes;
    unsigned long long n_layers;
    long long out_rows_total;
};
constexpr unsigned long long SNAPSHOT_MAGIC = 0x3154504e53464449ULL;      // "IDFSNPT1"

unsigned long long mix(unsigned long long h, unsigned long long v)
{
    h ^= v + 0x9e3779b97f4a7c15ULL + (h << 6) + (h >> 2);
    return h;
}
unsigned long long net_fingerprint(const idf_net* net)
{
    unsigned long long h = 0x1234;
    for (long long v : {(long long)net->dtype, (long long)net->in_w, (long long)net->in_c, (long long)net->n_streams, (long long)net->L.size()})
        h = mix(h, (unsigned long long)v);
    for (const auto& P : net->L) {
        const idf_layer& l = P.l;
        for (long long v : {(long long)l.kind, (long long)l.cin, (long long)l.cout, (long long)l.kh, (long long)l.kw, (long long)l.stride,
                            (long long)l.pad, (long long)l.relu, (long long)l.shift, (long long)P.use_sparse, (long long)P.state_bytes_all})
            h = mix(h, (unsigned long long)v);
    }
    return h;
}
size_t snapshot_bytes(const idf_net* net)
{
    return sizeof(SnapshotHeader) + net->L.size() * 3 * sizeof(long long) + net->state_region_bytes;
}
}  // namespace

size_t idf_state_snapshot_bytes(const idf_net* net) { return net ? snapshot_bytes(net) : 0; }

int idf_state_save(idf_net* net, void* h_snapshot, size_t bytes)
{
    if (!net || !h_snapshot) return fail(IDF_ERR_ARG, "net and h_snapshot must not be NULL");
    if (net->eager) return fail(IDF_ERR_UNSUPPORTED, "state snapshots are not available with eager emission");
    if (net->phase != OPEN) return fail(IDF_ERR_STATE, "state_save needs open streams (after open/reset/push, before finish)");
    if (bytes < snapshot_bytes(net)) return fail(IDF_ERR_CAPACITY, "snapshot needs %zu bytes, %zu given", snapshot_bytes(net), bytes);
    for (const auto& P : net->L)
        if (P.pending != 0) return fail(IDF_ERR_STATE, "internal: rows in flight between layers");   // (a push leaves none behind)
    unsigned char* p = (unsigned char*)h_snapshot;
    SnapshotHeader h{SNAPSHOT_MAGIC, net_fingerprint(net), net->state_region_bytes, net->L.size(), net->out_rows_total};
    memcpy(p, &h, sizeof h);
    p += sizeof h;
    long long* prog = (long long*)p;                     // per layer: rows received, rows emitted, events applied
    for (size_t i = 0; i < net->L.size(); ++i) { prog[3 * i] = net->L[i].rows_in; prog[3 * i + 1] = net->L[i].rows_done; }
    std::vector<unsigned long long> ev(net->L.size());
    cudaError_t e = cudaMemcpyAsync(ev.data(), net->ws + net->counters_off, ev.size() * sizeof(unsigned long long),
                                    cudaMemcpyDeviceToHost, net->stream);
    p += net->L.size() * 3 * sizeof(long long);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(p, net->ws + net->state_region_off, net->state_region_bytes, cudaMemcpyDeviceToHost, net->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(net->stream);
    if (e != cudaSuccess) return fail(IDF_ERR_CUDA, "state_save: %s", cudaGetErrorString(e));
    for (size_t i = 0; i < net->L.size(); ++i) prog[3 * i + 2] = (long long)ev[i];
    return IDF_OK;
}

int idf_state_restore(idf_net* net, const void* h_snapshot, size_t bytes)
{
    if (!net || !h_snapshot) return fail(IDF_ERR_ARG, "net and h_snapshot must not be NULL");
    if (net->eager) return fail(IDF_ERR_UNSUPPORTED, "state snapshots are not available with eager emission");
    if (net->phase == CREATED) return fail(IDF_ERR_STATE, "state_restore before stream_open");
    if (bytes < sizeof(SnapshotHeader)) return fail(IDF_ERR_ARG, "not a snapshot (too short)");
    SnapshotHeader h;
    memcpy(&h, h_snapshot, sizeof h);
    if (h.magic != SNAPSHOT_MAGIC) return fail(IDF_ERR_ARG, "not a snapshot (bad magic)");
    if (h.fingerprint != net_fingerprint(net) || h.n_layers != net->L.size() || h.state_region_bytes != net->state_region_bytes)
        return fail(IDF_ERR_SPEC, "the snapshot was taken from a net with a different spec or stream count");
    if (bytes < snapshot_bytes(net)) return fail(IDF_ERR_ARG, "snapshot truncated: %zu of %zu bytes", bytes, snapshot_bytes(net));
    const unsigned char* p = (const unsigned char*)h_snapshot + sizeof h;
    const long long* prog = (const long long*)p;
    // the progress record must be one the schedule can produce: every layer has emitted exactly the rows
    // complete after its input rows, and its successor has received them all
    long long r = prog[0];
    if (r < 0) return fail(IDF_ERR_ARG, "snapshot corrupt (negative row count)");
    for (size_t i = 0; i < net->L.size(); ++i) {
        if (prog[3 * i] != r) return fail(IDF_ERR_ARG, "snapshot corrupt (layer %zu row count)", i);
        r = layer_done_after(net->L[i], r);
        if (prog[3 * i + 1] != r) return fail(IDF_ERR_ARG, "snapshot corrupt (layer %zu rows emitted)", i);
    }
    if (h.out_rows_total != r) return fail(IDF_ERR_ARG, "snapshot corrupt (output row count)");
    p += net->L.size() * 3 * sizeof(long long);
    std::vector<unsigned long long> ev(net->L.size());
    for (size_t i = 0; i < net->L.size(); ++i) ev[i] = (unsigned long long)prog[3 * i + 2];
    cudaError_t e = cudaMemsetAsync(net->ws + net->status_off, 0, sizeof(unsigned int), net->stream);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(net->ws + net->state_region_off, p, net->state_region_bytes, cudaMemcpyHostToDevice, net->stream);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(net->ws + net->counters_off, ev.data(), ev.size() * sizeof(unsigned long long), cudaMemcpyHostToDevice, net->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(net->stream);      // (ev and possibly the caller's buffer are pageable)
    if (e != cudaSuccess) { net->phase = CREATED; return fail(IDF_ERR_CUDA, "state_restore: %s", cudaGetErrorString(e)); }
    for (size_t i = 0; i < net->L.size(); ++i) {
        LayerPlan& P = net->L[i];
        P.rows_in = prog[3 * i]; P.rows_done = prog[3 * i + 1]; P.pending = 0;
    }
    net->out_rows_total = h.out_rows_total;
    net->out_base = 0;
    net->phase = OPEN;
    return IDF_OK;
}

int idf_set_timing(idf_net* net, int on)
{
    if (!net) return fail(IDF_ERR_ARG, "net must not be NULL");
    net->timing = on != 0;
    return IDF_OK;
}

int idf_layer_times(idf_net* net, double* ms, long long* launches)
{
    if (!net || !ms || !launches) return fail(IDF_ERR_ARG, "NULL argument");
    for (size_t i = 0; i < net->L.size(); ++i) { ms[i] = 0.0; launches[i] = 0; }
    if (net->timed.empty()) return IDF_OK;
    cudaError_t e = cudaStreamSynchronize(net->stream);
    if (e != cudaSuccess) return fail(IDF_ERR_CUDA, "layer_times: %s", cudaGetErrorString(e));
    for (auto& t : net->timed) {
        float f = 0.f;
        if (cudaEventElapsedTime(&f, t.a, t.b) == cudaSuccess) { ms[t.layer] += f; launches[t.layer] += 1; }
        net->event_pool.push_back(t.a);
        net->event_pool.push_back(t.b);
    }
    net->timed.clear();
    return IDF_OK;
}

}  // extern "C"
