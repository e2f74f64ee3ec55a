// Internal declarations shared by the host side of the library and its kernels.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

namespace idf {

// element types of activation rows travelling between layers
enum Elem : int { E_F32 = 0, E_BF16 = 1, E_I8 = 2, E_I32 = 3 };

// Range-checked build (-DIDF_BOUNDS): every index into a ring, a row buffer, shared memory or tensor memory is
// compared with the extent of what it indexes before the access; a violation sets bit 1 of the handle's status
// word (idf_stream_status then reports IDF_ERR_BOUNDS) and the access is skipped - never a trap, never a wild
// access.  In the regular build the checks compile to nothing.
#ifdef __CUDACC__
#ifdef IDF_BOUNDS
__device__ __forceinline__ bool bounds_ok(unsigned int* status, long long idx, long long extent)
{
    if (idx >= 0 && idx < extent) return true;
    if (status) atomicOr(status, 2u);
    return false;
}
#define IDF_OK_AT(status, idx, extent) idf::bounds_ok((status), (long long)(idx), (long long)(extent))
#else
#define IDF_OK_AT(status, idx, extent) true
#endif
#endif

// process-wide debug switches (bits of idf_debug_flag), set through idf_set_debug_flags
unsigned debug_flags();

inline size_t elem_size(int e) { return e == E_F32 || e == E_I32 ? 4 : (e == E_BF16 ? 2 : 1); }

// How one conv layer advances by a block of input rows.  All row indices are absolute
// (counted since idf_stream_open) and identical for every stream.
//
// Row bookkeeping (0-based): input row r reaches output rows o with 0 <= r + pad - o*stride < Kh
// through tap ky = r + pad - o*stride; row o is complete once input row o*stride - pad + Kh - 1 has
// been applied (or at flush if only bottom padding is missing); its ring slot is o % ring_rows.
// A free ring slot holds zeros; the state excludes the bias, which joins at emission.
struct ConvArgs {
    const void* in;        // input rows of this block: [r - r0][S][Win][Cin]
    const void* w;         // packed weights (layout depends on the kernel)
    const void* bias;      // [Cout] in the state type, or nullptr
    void* ring;            // [ring_rows][S][Wout][Cout] state words
    void* ring_scratch;    // tensor-core kernel: room for a copy of the ring (same size), or nullptr
    void* out;             // emitted rows
    long long out_row_stride, out_stream_stride, out_row_base;  // element strides; row o goes to (o - out_row_base)
    long long out_rows_extent;   // rows the output buffer holds per stream
    unsigned long long* event_counter;  // sparse path: number of non-zero events applied
    int S, Win, Wout, Cin, Cout, Kh, Kw, stride, pad, relu, shift, ring_rows;
    int stride_x, pad_x;   // x axis: equal to stride/pad, except 1 and 0 on width-1 (1D) maps
    int in_elem, out_elem; // Elem
    long long r0, r1;      // input rows [r0, r1) arrive in this block
    long long o_begin, o_end;  // output rows [o_begin, o_end) are visited
    long long done_end;    // rows o < done_end are complete after this block: emit them, free their slots
    // Tensor-core kernel only: 2x2 max-pooling folded into the emission.  `out` and its strides, row base and
    // row extent then describe the POOLED rows (pooled row p = o / 2 goes to p - out_row_base).
    int pool_fused;        // 1: emit pooled rows
    int pool_keep;         // 1: more input may follow (a trailing first row of a pair waits in pool_state); 0: end of input
    void* pool_state;      // the pool layer's state: [S][Wout/2][Cout] in the output type
    // extents in elements of what the pointers above address (range-checked build) and the handle's status word
    long long in_elems, out_elems, ring_elems, pool_state_elems;
    unsigned int* status;
};

struct PoolArgs {
    const void* in;        // [r - r0][S][Win][C]
    void* state;           // [S][Wout][C] running maximum of the first row of a pair
    void* out;
    long long out_row_stride, out_stream_stride, out_row_base;
    int S, Win, Wout, C, elem;
    long long r0, r1, o_begin, o_end, done_end;
    long long in_elems, out_elems, state_elems;   // extents (range-checked build)
    unsigned int* status;
};

// Global-average sink: every arriving row is added into one running sum per (stream, channel); the
// output row holds the mean over all positions received so far.
struct AvgArgs {
    const void* in;        // [n_rows][S][W][C] in the element type `elem`
    void* sum;             // [S][C] state words (fp32, or int32 for E_I8 rows)
    float* out;            // mean of stream s at out + s * out_stream_stride, C floats
    long long out_stream_stride;
    int S, W, C, elem;
    long long n_rows;      // rows arriving in this launch
    long long rows_total;  // rows received since open, these included
    long long in_elems, out_elems, sum_elems;     // extents (range-checked build)
    unsigned int* status;
};

// Eager emission (one segment per step): how one layer re-evaluates the rows of its input cone.
// Rings hold 32-bit words (fp32 for float nets, int32 for int nets), slot = row mod capacity.
struct EagerArgs {
    const void* din;       // changes announced by the layer below in this step: [cap_in][S][Win][Cin] (conv)
    const void* hin;       // activations announced so far by the layer below: [cap_in][S][Win][Cin] (pool)
    void* c;               // state variables: [cap][S][Wout][Cout] (conv)
    void* h;               // activations this layer has announced: [cap][S][Wout][Cout]
    void* d;               // the change it announces in this step: [cap][S][Wout][Cout]
    const void* w;         // [Kh][Kw][Cin][Cout] fp32 or int8
    const void* bias;      // [Cout] words or nullptr
    void* out;             // last layer: the caller's output [S][rows][Wout][Cout] (fp32 / int8), else nullptr
    long long out_row_stride, out_stream_stride;
    unsigned long long* events;   // count of non-zero changes announced (or nullptr)
    int S, Win, Wout, Cin, Cout, Kh, Kw, stride, pad, stride_x, pad_x, relu, shift, round_bf16;
    int cap_in, cap;       // ring capacities in rows
    long long in_lo, in_hi;   // rows of the layer below that changed in this step (conv; empty if in_lo > in_hi);
                              // pool: in_hi = last row of the layer below that has announced anything
    long long o_lo, o_hi;     // rows of this layer to re-evaluate
    long long o_new;          // rows >= o_new are touched for the first time (their slots hold an older row)
    long long o_cut;          // rows >= o_cut turn out not to exist (end of input): their activation goes back to 0
    long long in_elems, ring_elems, out_elems;    // extents of din/hin, of each of c/h/d, of out (range-checked build)
    unsigned int* status;
};
cudaError_t launch_eager_input(const void* in, int in_elem, void* d, long long n, unsigned long long* events, cudaStream_t st);
cudaError_t launch_eager_layer(const EagerArgs& a, int is_pool, int int_net, cudaStream_t st);

// Depth-first over all layers in one launch (state of a group of streams in shared memory).
constexpr int FUSED_MAX_LAYERS = 12;
constexpr size_t FUSED_SMEM_LIMIT = 200 * 1024;
struct FusedLayer {
    int kind;              // 0 conv, 1 max-pool
    int Cin, Cout, Kh, Kw, stride, pad, stride_x, pad_x, relu, shift, round_bf16, Win, Wout, ring_rows;
    int count_events;      // the layer reports its input events (sparse-path layers)
    int out_elem;          // element type of the rows the layer emits (pool state in global memory has this type)
    int state_soff, rowbuf_soff;   // shared memory, in bytes: ring [slot][G][Wout][Cout] words or pool row [G][Wout][C]; emitted row [G][Wout][Cout]
    long long w_off;       // weights [Kh][Kw][Cin][Cout]: element offset from FusedArgs::weights (fp32 or int8 elements)
    long long wq_off;      // int nets: the same weights, four input channels to a word [Kh][Kw][Cin/4][Cout], BYTE offset; -1: none
    long long bias_off;    // bias [Cout] words: BYTE offset from FusedArgs::weights, or -1
    void* state;           // the layer's state in global memory
    // the layer's progress when the launch begins, as the small counters the kernel steps (see LayerClock)
    int ph0, hi_slot0, hi_sat0, phf0, tf_neg0, done_slot0;
    int n_flush;           // rows the layer completes on bottom padding if the input ends with this launch
};
struct FusedArgs {
    FusedLayer layer[FUSED_MAX_LAYERS];
    int n_layers, S, G;    // streams in all, streams per CTA
    const void* in;        // pushed segments [n_seg][S][in_w][in_c] in the element type in_elem
    int n_seg, in_w, in_c, in_elem, in_soff;
    int flush;             // the input ends with these segments
    const void* weights;   // base of the parameter area
    void* out;             // [S][out_cap][Wout][Cout] in out_elem (fp32 / int8)
    long long out_cap;
    int out_row0;          // index in the caller's buffer of the next output row
    int out_elem;
    unsigned long long* counters;   // per layer: input events applied (sparse-path layers)
    unsigned int* status;
};
cudaError_t launch_depth_first(const FusedArgs& a, int int_net, int threads, size_t smem_bytes, cudaStream_t st);

// Static plan of the tensor-core path for one conv layer (tile shapes, shared-memory budget).
struct TcPlan {
    int ok = 0;
    int BX = 0, BS = 0;      // a 128-row M tile = BS streams x BX consecutive x positions
    int BXP = 0;             // positions per stream held in the shared-memory tile (BX + kx halo)
    int shift_mode = 0;      // kx taps read one haloed tile at row offsets instead of one box per kx
    int sx = 1;              // x stride (> 1 only without shift_mode: the tensor map walks the input row in steps of sx)
    int a_stage_bytes = 0;
    int n_box = 1, a_box_pitch = 0;   // TMA boxes per stage (one per kx tap where the taps cannot share a haloed box), their distance
    int n_xt = 0, n_mt = 0;  // x tiles per row, M tiles in all
    int Ntile = 0, n_nt = 0; // output channels per CTA, N tiles
    int KB = 0, n_kb = 0;    // input channels per K block (one swizzled shared-memory row), K blocks
    int swb = 0;             // bytes of one K-block row: 32, 64 or 128 = the swizzle span
    int nslot = 0;           // ring rows resident in tensor memory at once (>= ring rows + 1)
    int nstage = 0;          // Δ-row tiles in flight
    int tmem_cols = 0;
    int out_groups = 0;
    int out_bufs = 1;        // staging tiles per epilogue group (2: a row is laid out while the previous store still drains)
    int out_esize = 0, out_pwb = 0, out_panels = 0, out_stage_bytes = 0;   // staging of emitted rows for the TMA store
    int out_stage_rows = 0;  // rows of one staging panel: 128, or 64 in a plan for launches that emit pooled rows
    size_t smem_bytes = 0;
    size_t w_bytes = 0;      // device weights for this path: [tap slot][Cout][Cin] in the activation type
};
bool tc_make_plan(int dtype, int S, int Win, int Wout, int Cin, int Cout, int Kh, int Kw, int stride_x, int ring_rows,
                  int out_esize, int pooled, TcPlan* p);
int tc_weight_slot(int ky, int kx, int Kh, int stride);
int tc_encode_weights(const TcPlan& p, int dtype, const void* d_w, int taps, int Cin, int Cout, void* map_out);
cudaError_t launch_conv_tc(const ConvArgs& a, const TcPlan& p, int dtype, const void* w_map, int n_in_rows,
                           unsigned int* status, cudaStream_t st);

// Static plan of the thin-layer kernel (the whole Kh*Kw*Cin-wide receptive field in one swizzled shared-memory row).
struct ThinPlan {
    int ok = 0;
    int swb = 0;             // bytes of one im2col row: 32, 64 or 128 (the swizzle span)
    int kelems = 0;          // Kh*Kw*Cin values of a row, zero padded to swb bytes
    int ksteps = 0;          // 32-byte MMA K steps
    int BX = 0, BS = 0, n_xt = 0, n_mt = 0;   // a 128-position tile = BS streams x BX consecutive x positions
    int R = 0;               // output rows per work item
    int nstage = 0, tmem_cols = 0;
    int out_esize = 0, out_pwb = 0, out_panels = 0, out_tile_bytes = 0;
    size_t smem_bytes = 0, w_bytes = 0;      // w_bytes: device weights [Cout][swb] in the activation type
};
bool thin_make_plan(int dtype, int S, int Wout, int Cin, int Cout, int Kh, int Kw, int stride, int stride_x, int out_esize, ThinPlan* p);
int thin_encode_weights(const ThinPlan& p, int dtype, const void* d_w, int Cout, void* map_out);
cudaError_t launch_conv_thin(const ConvArgs& a, const ThinPlan& p, int dtype, const void* w_map, long long o_first, long long o_end,
                             unsigned int* status, cudaStream_t st);
// CUDA-core conv kernel on the rows that exchange state with the ring only: rows [skip_begin, skip_end) are left to
// another kernel
cudaError_t launch_conv_edges(const ConvArgs& a, int dtype, long long skip_begin, long long skip_end, cudaStream_t st);

// x-unfold: out[row][s][x'][kx*Cin + ci] = in[row][s][x'*stride_x - pad_x + kx][ci] (0 outside the row or
// beyond Kw*Cin), kpad channels per position, in the activation type
cudaError_t launch_unfold(const ConvArgs& a, int n_rows, int kpad, void* out, cudaStream_t st);

// CUDA-core kernels (every type, every shape)
cudaError_t launch_conv_simple(const ConvArgs& a, int dtype, cudaStream_t st);
cudaError_t launch_conv_sparse(const ConvArgs& a, int dtype, cudaStream_t st);
cudaError_t launch_pool(const PoolArgs& a, cudaStream_t st);
cudaError_t launch_avg(const AvgArgs& a, cudaStream_t st);
size_t conv_sparse_max_smem();

}  // namespace idf
