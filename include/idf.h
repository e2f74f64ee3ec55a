/*
 * idf - incremental depth-first CNN inference (Binas & Bengio, arXiv 1804.10727)
 * C ABI of the CUDA (sm_100a) library.
 *
 * The paper's "streaming core" takes input segments as they arrive and updates
 * its output incrementally (Introduction, last paragraph; Discussion, second
 * paragraph).  A segment is one sample of a 1D signal or one row of a 2D image
 * (Section "Asynchronous incremental updates", the 1D/2D paragraphs and Fig. 2).
 * Every unit keeps a state variable c (Eq. 2); an arriving event dh is added as
 * c += w * dh (Eq. 4); a unit whose activation f(c) has changed passes the
 * change on to the next layer (Eq. 3, Eq. 5).  This library uses the
 * segment-synchronous form of that rule: a unit emits once, when no present or
 * future segment can reach it any more, so every conv layer keeps only
 * ceil(Kh/stride) rows of state ("activation subset buffers", Discussion) and the
 * result equals conventional layer-by-layer inference (Eq. 1).
 *
 * Many independent streams advance in lockstep: every call handles the same
 * number of segments for each of n_streams streams.
 *
 * Conventions
 *   - All functions return IDF_OK (0) or a negative idf_status; no exceptions, no abort,
 *     no device traps.  idf_last_error() gives a message for the calling thread's last failure.
 *   - "host" / "device" in a parameter comment says where the pointer must live.
 *   - The library allocates no device memory: the caller passes the workspace, the segment
 *     buffer and the output buffer (device memory it owns) and the CUDA stream all work is
 *     enqueued on.  A handle is not thread-safe; distinct handles are independent.
 *   - There is no CPU fallback and no other backend.
 *   - Layouts have channels innermost.  Weights: [Cout][Kh][Kw][Cin], cross-correlation
 *     (no kernel flip), zero padding `pad` on all four sides, one stride for both axes,
 *     output extent floor((n + 2 pad - k) / stride) + 1.  A 1D net has in_w == 1 and kw == 1.
 */
#ifndef IDF_H
#define IDF_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct idf_net idf_net;   /* opaque; owns packed host copies of the parameters and the layout */

/* activation/weight type _ state type */
typedef enum {
    IDF_F32 = 0,       /* fp32 activations and weights, fp32 state                                   */
    IDF_BF16_F32 = 1,  /* bf16 activations and weights, fp32 state; a conv layer that feeds a later  */
                       /* conv layer rounds f(c) to bf16 (nearest even); the last conv layer and     */
                       /* whatever follows it stay fp32; the net's output is fp32                    */
    IDF_I8_I32 = 2     /* int8 activations and weights, int32 state; per conv layer                  */
                       /* q = clamp((c + 2^(shift-1)) >> shift, relu ? 0 : -127, 127); output int8   */
} idf_dtype;

typedef enum {
    IDF_CONV = 0,
    IDF_MAXPOOL2 = 1,    /* 2x2 max pool, stride 2, floor; rows only when width is 1 */
    IDF_GLOBAL_AVG = 2   /* output sink, last layer only: the averaging output unit of the paper's Fig. 1.  Every value
                            arriving from the layer below is added to one running sum per stream and channel
                            (c_out += dh, Eq. 4 with weight 1; 4 bytes of state per channel).  The net's output is then
                            ONE row [n_streams][out_capacity_rows >= 1][1][C] of fp32 (for every idf_dtype; for int
                            nets the exact int32 sum divided in double precision and rounded once): the mean over all
                            positions received so far.  It is rewritten by every push that brings it new rows, so it
                            can be read between pushes (the paper's output that converges while the input arrives,
                            Section "Experimental verification"), and is final after idf_stream_finish. */
} idf_kind;
/* A fully connected output layer over a map of known size H x W x C (the paper's 10 output units) is an IDF_CONV layer
 * with kh = H, kw = W, stride = H, pad = 0 and weights [n_out][H][W][C]: one output row of width 1, one ring row of
 * state, and every arriving row adds its share w * dh at once. */
typedef enum { IDF_PATH_AUTO = 0, IDF_PATH_DENSE = 1, IDF_PATH_SPARSE = 2 } idf_path;

/* When a unit passes a change of its activation on.
 *   IDF_EMIT_DEFERRED  once, when no present or future segment can reach it any more (see the file header): state of
 *                      ceil(Kh/stride) rows per conv layer, the operation count of conventional inference, every
 *                      kernel of the library.  Output rows appear when they are final.
 *   IDF_EMIT_EAGER     the paper's literal rule (Eq. 3-5): after every segment each unit whose activation f(c) has
 *                      changed announces dh = h(t) - h(t-1), the layer above adds w * dh to its states (Eq. 4) and
 *                      re-evaluates in turn, within the same push.  The net's output is then an ANYTIME output: after
 *                      every idf_stream_push, d_out holds, below the finished rows, also the rows a later segment can
 *                      still reach, with the activation they have announced so far, and converges to the conventional
 *                      result as the input arrives (Section "Experimental verification", Fig. 3-4); rows_emitted still
 *                      counts finished rows only, and out_capacity_rows must cover every row touched.  A unit
 *                      announces partial sums, so a layer keeps all rows of its input cone (state and announced
 *                      activation: idf_net_state_bytes reports them) and a unit is updated once per segment of its
 *                      receptive field.  Units of rows that turn out to lie beyond the end of the input (known only
 *                      at idf_stream_finish) take back what they announced.  A max-pool unit holds its four current
 *                      inputs (0 for units that have announced nothing) and announces max_new - max_old.  Runs on
 *                      CUDA cores, one launch per layer and segment; IDF_GLOBAL_AVG, idf_stream_set_out_base and the
 *                      snapshot calls are not available (IDF_ERR_UNSUPPORTED), the first layer must be a conv
 *                      layer.  idf_event_counts: events[i] = non-zero changes layer i has received. */
typedef enum { IDF_EMIT_DEFERRED = 0, IDF_EMIT_EAGER = 1 } idf_emission;

typedef enum {
    IDF_OK = 0,
    IDF_ERR_ARG = -1,          /* null pointer, negative count, ...                                   */
    IDF_ERR_SPEC = -2,         /* inconsistent layer spec (channel mismatch, empty map, ...)          */
    IDF_ERR_STATE = -3,        /* push before open or after finish                                    */
    IDF_ERR_CAPACITY = -4,     /* workspace or output buffer too small                                */
    IDF_ERR_UNSUPPORTED = -5,  /* valid request this build cannot serve                               */
    IDF_ERR_CUDA = -6,         /* a CUDA call failed                                                  */
    IDF_ERR_TIMEOUT = -7,      /* a bounded device-side wait ran out                                  */
    IDF_ERR_BOUNDS = -8        /* range-checked build only (libidf_bounds.so): an index lay outside   */
                               /* the ring, row buffer, shared or tensor memory it addresses; the     */
                               /* access was skipped and recorded, never performed                    */
} idf_status;

typedef struct {
    int kind;      /* idf_kind                                                        */
    int cin, cout; /* conv only                                                       */
    int kh, kw;    /* conv only; kw == 1 for 1D nets                                  */
    int stride;    /* conv only; 1 <= stride <= kh                                    */
    int pad;       /* conv only; 0 <= pad < kh                                        */
    int relu;      /* conv only; f = ReLU if non-zero, identity otherwise             */
    int shift;     /* conv only, IDF_I8_I32: requantisation shift, 0..30              */
    int path;      /* conv only; idf_path: how the layer's events are applied         */
} idf_layer;

typedef struct {
    int n_layers;
    const idf_layer* layers;   /* host */
    int dtype;                 /* idf_dtype */
    int in_w, in_c;            /* segment width (1 for 1D) and channels */
    int n_streams;             /* streams advanced together by every call */
    int row_block;             /* most segments pushed through all layers at once (bounds the   */
                               /* transient workspace); 0 = library default: about 25 000       */
                               /* positions per stream (112 rows of a 224-wide image, at most   */
                               /* 1024 rows), 4096 samples for 1D nets.  The buffers between    */
                               /* layers hold 2 * row_block + 8 rows of every stream whatever   */
                               /* the streams' real length: for short streams (a 28-row image)  */
                               /* give the real row count and the workspace shrinks with it     */
    int emission;              /* idf_emission; 0 = IDF_EMIT_DEFERRED                           */
} idf_spec;

/* Build a net from a layer list and the parameters of a conventionally trained CNN
 * (Section "Experimental verification": learned parameters are copied into the incremental
 * model).  weights[i] / biases[i] belong to layers[i]; entries of non-conv layers are ignored.
 *   weights: host, per conv layer [Cout][Kh][Kw][Cin] in the activation type (fp32 / bf16 bits / int8)
 *   biases : host, per conv layer [Cout] in the state type (fp32 / int32); the array or an entry may
 *            be NULL = zero bias.  The paper takes b = 0 without loss of generality; here the bias
 *            joins at emission, h = f(c + b).
 * Everything is copied; the caller may free its buffers on return.  *out receives the handle. */
int idf_net_create(const idf_spec* spec, const void* const* weights, const void* const* biases, idf_net** out);

/* Release the handle (host memory only; device buffers belong to the caller). */
int idf_net_destroy(idf_net* net);

/* Rolling state PER STREAM in bytes: sum over conv layers of ceil(Kh/stride) rows of Wout*Cout
 * state words, plus one row per pooling layer.  Constant in the number of segments (1D: constant;
 * 2D: proportional to the row width), as the paper's abstract claims.  0 if net is NULL. */
size_t idf_net_state_bytes(const idf_net* net);

/* Device bytes the caller must provide to idf_stream_open: all streams' rolling state (the "activation
 * subset buffers" of the paper's Discussion, idf_net_state_bytes per stream), the packed parameters, and
 * the transient buffers of at most 2 * row_block + 8 rows between layers that carry the events of Eq. 3
 * from one layer to the next (sentence after Eq. 5).  Independent of the number of segments.  0 if net
 * is NULL. */
size_t idf_net_workspace_bytes(const idf_net* net);

/* Shape of the output map once in_rows segments and the end of input have been seen: the extent of the
 * conventional layer-by-layer result (Eq. 1 with the conv connectivity of Section "Asynchronous
 * incremental updates"), which the incremental result equals ("identical to the original output",
 * Introduction).  out_rows may be 0.  Any out pointer may be NULL.  IDF_ERR_ARG for a NULL net or
 * negative in_rows. */
int idf_out_shape(const idf_net* net, long long in_rows, long long* out_rows, int* out_w, int* out_c);

/* Rows per stream the output buffer must hold (out_capacity_rows) for streams of in_rows segments: the rows of the
 * final map (idf_out_shape) and, with IDF_EMIT_EAGER, also the rows above them that the last segments touch with
 * partial activations before the end of input takes those back.  -1 for a NULL net or negative in_rows. */
long long idf_out_rows_needed(const idf_net* net, long long in_rows);

/* Start streams: every unit's state variable c and activation begin at zero (the paper's convention
 * in the paragraph after Eq. 3: all units start at 0, so the first events are the inputs themselves).
 * Binds a workspace (device, 256-byte aligned, >= idf_net_workspace_bytes; owned by the caller, who must
 * keep it alive and unmodified until the streams are finished) and a CUDA stream (a cudaStream_t passed as
 * void*, NULL = default stream); uploads the parameters, zeroes all state, resets the segment counters.
 * May be called again after idf_stream_finish to start new streams.  Errors: IDF_ERR_ARG (NULL or
 * misaligned workspace), IDF_ERR_CAPACITY (workspace too small), IDF_ERR_CUDA. */
int idf_stream_open(idf_net* net, void* d_workspace, size_t workspace_bytes, void* cuda_stream);

/* Start new streams on the workspace and CUDA stream bound by the last idf_stream_open: zero all
 * rolling state (every unit starts at 0, the paper's convention after Eq. 3) and the segment
 * counters.  The parameters uploaded by idf_stream_open stay where they are, so the caller must
 * not have written to the workspace since.  Valid in any state after the first idf_stream_open
 * (also in the middle of streams, which are then abandoned); IDF_ERR_STATE before it. */
int idf_stream_reset(idf_net* net);

/* Push n_seg consecutive segments of every stream through all layers, depth first: the paper's
 * streaming core "can process small segments of the input as they arrive" (Introduction, last
 * paragraph); a segment is a sample or an image row (Fig. 2 and its caption), its non-zero components
 * are the events of Eq. 3, each layer adds them into its state (Eq. 4), and rows of units that no present
 * or future segment can reach any more are finalised and passed up at once (sentence after Eq. 5; Fig. 2
 * caption: such units are fully processed and can be forgotten).
 *   d_segments: device, [n_seg][n_streams][in_w][in_c] in the activation type
 *   d_out     : device, [n_streams][out_capacity_rows][out_w][out_c], fp32 (float nets) or int8;
 *               output rows that become complete are written at their absolute row index
 *   rows_emitted: host, may be NULL; receives the number of output rows completed by this call.
 *               The count is known on the host, so no synchronisation is implied; the work is
 *               enqueued on the stream given to idf_stream_open.
 * The result does not depend on how segments are grouped into calls (bit-exact for int nets).
 * Errors: IDF_ERR_STATE before open / after finish; IDF_ERR_CAPACITY if a completed row would not
 * fit out_capacity_rows (nothing is enqueued in that case). */
int idf_stream_push(idf_net* net, const void* d_segments, int n_seg,
                    void* d_out, long long out_capacity_rows, int* rows_emitted);

/* Output window for streams of unbounded length (the paper's 1D case: state constant in the input length, so the
 * output buffer should be too).  By default output row o of a stream is written at row index o of d_out.  After
 * this call rows are written at index o - first_row instead: the caller has consumed the rows below first_row and
 * reuses the buffer from its start.  first_row must not exceed the number of rows emitted so far (IDF_ERR_ARG), so
 * that no row still to come would land below index 0; IDF_ERR_STATE unless streams are open.  The capacity check of
 * the push calls counts from first_row.  idf_stream_open, idf_stream_reset and idf_state_restore set it back to 0.
 * A global-average sink always writes its single row at index 0. */
int idf_stream_set_out_base(idf_net* net, long long first_row);

/* End of input.  The length of a stream is not known while it runs (segments are taken as they
 * arrive, Introduction and Discussion), yet the result must equal the conventional output (Introduction:
 * "identical"; Eq. 1), whose last rows see zero padding below the input.  So this call completes the rows
 * that wait only for bottom zero padding, in depth order, and drops rows that can never complete.  total_rows (host, may be NULL) receives the number of output
 * rows per stream since open.  After this call only idf_stream_open or idf_net_destroy are valid. */
int idf_stream_finish(idf_net* net, void* d_out, long long out_capacity_rows, long long* total_rows);

/* The last n_seg segments of every stream together with the end of input: the same results as
 * idf_stream_push followed by idf_stream_finish (the paper's output is defined by the whole input,
 * Eq. 1; how the rows are grouped into calls changes nothing), but every dense layer completes the
 * rows that wait only for bottom zero padding in the launch that applies its last rows, instead of
 * a second pass through the layers.  n_seg may be 0 (then this is idf_stream_finish).  Arguments,
 * layouts, ownership and errors as for idf_stream_push; total_rows as for idf_stream_finish.  After
 * this call only idf_stream_open or idf_net_destroy are valid. */
int idf_stream_push_last(idf_net* net, const void* d_segments, int n_seg,
                         void* d_out, long long out_capacity_rows, long long* total_rows);

/* Whole streams from host memory: copy h_segments ([n_seg][n_streams][in_w][in_c], host, ideally
 * pinned) to d_segments, push every segment and the end of input (as idf_stream_push_last), copy the
 * completed output rows back to h_out ([n_streams][out_capacity_rows][out_w][out_c], host, ideally
 * pinned; rows beyond the last completed one are left as they are) and wait until all of it is done.
 * The work is pipelined over steps of row_block / 2 segments (the first and the last step half of
 * that, so that the copies nothing overlaps are short): while one step is computed on the handle's
 * stream, the next one travels to the device and the output rows of the one before travel back, on two copy streams the handle creates at its first idf_run_host (streams and events only,
 * no device memory) and orders after whatever was enqueued on the handle's stream before the call.
 * d_segments and d_out are device staging buffers of the same sizes, owned by the caller.  The handle
 * must be freshly opened or reset. */
int idf_run_host(idf_net* net, const void* h_segments, int n_seg, void* d_segments,
                 void* h_out, void* d_out, long long out_capacity_rows, long long* total_rows);

/* Counters of the sparse-event path since open, read back from the device (synchronises the
 * stream): events[i] = number of non-zero input events layer i has applied; entries of layers on
 * the dense path are 0.  events: host, n_layers entries. */
int idf_event_counts(idf_net* net, long long* events);

/* Kernel launches enqueued by this handle since open. */
long long idf_launch_count(const idf_net* net);

/* Wait for the stream and report whether any kernel of this handle gave up on a bounded device-side
 * wait since idf_stream_open (IDF_ERR_TIMEOUT; results are then invalid) or, in the range-checked build
 * of the library (compiled with -DIDF_BOUNDS: every index into a ring, row buffer, shared or tensor
 * memory is compared with its extent before the access), skipped an access whose index was out of range
 * (IDF_ERR_BOUNDS).  tensor_core_launches
 * (host, n_layers entries, may be NULL) receives per layer how many launches took the tcgen05 path. */
int idf_stream_status(idf_net* net, long long* tensor_core_launches);

/* Per-layer device time.  With timing on, every kernel launch of the handle is bracketed by CUDA
 * events on its stream.  idf_layer_times synchronises the stream, adds up the elapsed time of the
 * launches recorded since the last query into ms[i] (milliseconds, host, n_layers entries) and
 * their number into launches[i], and clears the record. */
int idf_set_timing(idf_net* net, int on);
int idf_layer_times(idf_net* net, double* ms, long long* launches);

/* Checkpoint of running streams.  The paper's Discussion reads the method as a recurrent model whose
 * hidden state is the set of partially computed activations; that state (all streams' ring rows and
 * pooling rows) together with the per-layer row counters is everything a stream needs to go on, so
 * it can be taken off the device between two pushes and put back later, on this handle or on
 * another handle created from the same spec and parameters (another workspace, another GPU).
 *
 *   idf_state_snapshot_bytes  size of a snapshot of this net in bytes (0 if net is NULL): a small
 *                             header plus the state of all streams (n_streams * idf_net_state_bytes,
 *                             each layer rounded up to 256 bytes).
 *   idf_state_save     h_snapshot: host, at least idf_state_snapshot_bytes, owned by the caller.
 *                      Valid while streams are open (after open/reset/push, before finish), else
 *                      IDF_ERR_STATE; IDF_ERR_CAPACITY if bytes is too small.  Copies on the handle's
 *                      stream and waits for it.  The streams go on unchanged.
 *   idf_state_restore  h_snapshot: host.  The handle must have a workspace bound (idf_stream_open);
 *                      whatever streams it was running are abandoned and replaced by the saved ones,
 *                      which are then open.  IDF_ERR_ARG if the buffer is not a snapshot or is
 *                      truncated or inconsistent, IDF_ERR_SPEC if it was taken from a net of another
 *                      shape (layers, types, widths, stream count).  Parameters are not part of a
 *                      snapshot: the restoring handle uses its own.  Waits for the stream.
 * Output rows completed before the snapshot are not written again: later pushes write the rows that
 * follow, at their absolute row index, into whatever d_out the caller passes then.  Continuing from
 * a snapshot gives bit-identical results to continuing without the interruption. */
size_t idf_state_snapshot_bytes(const idf_net* net);
int idf_state_save(idf_net* net, void* h_snapshot, size_t bytes);
int idf_state_restore(idf_net* net, const void* h_snapshot, size_t bytes);

/* One fp32 conv layer over whole streams, for callers that cannot allocate device memory.
 * (The paper has no counterpart to this call; it exists for deployment reasons only.)
 *
 * Some callers hold nothing but their input and output buffers at the moment they need a result:
 * a plugin handed two pointers by its host program, code inside a pre-partitioned memory pool, a
 * latency-critical loop that must keep away from the allocator.  They cannot supply the workspace
 * the regular calls need, and this call needs none: the rolling state (ceil(kh/stride) rows per
 * stream) and the repacked weights live in a fixed array inside the library image, of
 * IDF_NOALLOC_SCRATCH_BYTES bytes, which every GPU that loads the library holds until exit.
 * The call allocates and frees nothing, on the device or through any library.
 *
 *   d_in      device, [n_rows][n_streams][in_w][cin] fp32 - all segments of every stream
 *   d_weights device, [cout][kh][kw][cin] fp32;  d_bias device, [cout] fp32 or NULL
 *   d_out     device, [n_streams][out_capacity_rows][out_w][cout] fp32; receives every output row
 *             (the end-of-input flush is included), f = ReLU if relu != 0
 *   out_rows  host, may be NULL: floor((n_rows + 2 pad - kh) / stride) + 1 (0 if negative)
 *   cuda_stream  a cudaStream_t as void*, NULL = default stream; the work is enqueued, not awaited
 *
 * Limits and sharing: ring bytes (rounded up to 256) + weight bytes must fit the array, else
 * IDF_ERR_CAPACITY and nothing is enqueued.  All calls on a device share the one array, which keeps
 * the previous call's contents; the call clears the part that must start at zero itself.  Two calls
 * whose GPU work overlaps in time (different streams, different threads) race on the array and give
 * wrong results: serialise them.  The first call on each device resolves the array's device address
 * (a one-time set-up step with that device current); make that first call before any CUDA stream
 * capture begins.  Results equal those of a one-layer IDF_F32 net run through
 * idf_stream_push + idf_stream_finish. */
#define IDF_NOALLOC_SCRATCH_BYTES (8u << 20)
int idf_conv_rows_noalloc(const float* d_in, int n_rows, int n_streams, int in_w, int cin,
                          const float* d_weights, const float* d_bias, int cout, int kh, int kw,
                          int stride, int pad, int relu, float* d_out, long long out_capacity_rows,
                          long long* out_rows, void* cuda_stream);

/* Debug only.  Process-wide switches that route work away from the default kernels so that tests can compare
 * the paths with one another; results are the same with any combination (bit-exact for int nets), only the
 * kernels and launch counts differ.  Not for production use; the paper has no counterpart.  flags is a
 * combination of the bits below (0 = defaults); IDF_DEBUG_NO_TENSOR_CORES, IDF_DEBUG_NO_POOL_FUSION and
 * IDF_DEBUG_PREFER_THIN are read by idf_net_create (they affect nets created afterwards), the others at every push or launch.
 * IDF_ERR_ARG for an unknown bit (nothing changes). */
typedef enum {
    IDF_DEBUG_NO_TENSOR_CORES = 1,  /* dense layers stay on the CUDA-core kernel                              */
    IDF_DEBUG_NO_POOL_FUSION = 2,   /* max-pool layers run as launches of their own                           */
    IDF_DEBUG_NO_ROW_CHUNKS = 4,    /* a block's rows stay in one CTA per tile                                */
    IDF_DEBUG_NO_PDL = 8,           /* no programmatic dependent launch                                       */
    IDF_DEBUG_PREFER_THIN = 16,     /* thin layers (receptive field of at most 128 bytes) take the thin-layer */
                                    /* kernel also where x-unfold + row ring is the default (2D nets)          */
    IDF_DEBUG_NO_FUSED = 32,        /* never the single launch over all layers (state in shared memory)       */
    IDF_DEBUG_FORCE_FUSED = 64      /* ... always, where a stream's state fits (by default: small pushes only) */
} idf_debug_flag;
int idf_set_debug_flags(unsigned int flags);

/* Message for the most recent failure on the calling thread ("" if none). */
const char* idf_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* IDF_H */
