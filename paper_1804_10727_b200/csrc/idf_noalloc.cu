// One conv layer over whole streams with NO device allocation anywhere on the way.
//
// Who this is for: callers that are not allowed to allocate device memory at the point where they
// need inference -- code running inside a memory pool that has already been carved up, a plugin
// that only receives input and output buffers from its host application, a real-time loop that
// must not touch the allocator.  The regular entry points ask such a caller for a workspace, which
// it cannot provide.  Here the rolling state (the ring of ceil(Kh/stride) rows per stream) and the
// repacked weights live in a fixed array that is part of the library image itself, so every GPU
// that loads the library carries IDF_NOALLOC_SCRATCH_BYTES of it until the process exits.
#include "../../include/idf.h"
#include "idf_internal.h"

#include <mutex>

using namespace idf;

namespace {

constexpr size_t kScratchBytes = IDF_NOALLOC_SCRATCH_BYTES;
constexpr int kMaxDevices = 64;

// The scratch itself.  In host code this name is only a handle for the runtime; the device address
// comes from cudaGetSymbolAddress below and is what the kernels receive.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

std::mutex g_mu;
unsigned char* g_scratch_ptr[kMaxDevices] = {};

// weights arrive in the public layout [Cout][Kh][Kw][Cin]; the row kernel reads [Kh][Kw][Cin][Cout]
__global__ void repack_weights_kernel(const float* __restrict__ src, float* __restrict__ dst, int cout, int taps, int cin)
{
    const long long n = (long long)cout * taps * cin;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
        const int ci = (int)(i % cin);
        const long long t = i / cin;
        const int k = (int)(t % taps);
        const int co = (int)(t / taps);
        dst[((long long)k * cin + ci) * cout + co] = src[i];
    }
}

}  // namespace

// defined in idf_host.cu: records the message idf_last_error() returns and hands the code back
namespace idf { int set_last_error(int code, const char* msg); }

extern "C" int idf_conv_rows_noalloc(const float* d_in, int n_rows, int n_streams, int in_w, int cin,
                                     const float* d_weights, const float* d_bias, int cout, int kh, int kw,
                                     int stride, int pad, int relu, float* d_out, long long out_capacity_rows,
                                     long long* out_rows, void* cuda_stream)
{
    if (!d_in || !d_weights || !d_out) return set_last_error(IDF_ERR_ARG, "noalloc: d_in, d_weights and d_out must not be NULL");
    if (n_rows < 1 || n_streams < 1 || in_w < 1 || cin < 1 || cout < 1 || kh < 1 || kw < 1)
        return set_last_error(IDF_ERR_ARG, "noalloc: sizes must be positive");
    if (stride < 1 || stride > kh || pad < 0 || pad >= kh) return set_last_error(IDF_ERR_SPEC, "noalloc: need 1 <= stride <= kh and 0 <= pad < kh");
    if (in_w == 1 && kw != 1) return set_last_error(IDF_ERR_SPEC, "noalloc: a width-1 map needs kw == 1");
    const int stride_x = in_w == 1 ? 1 : stride, pad_x = in_w == 1 ? 0 : pad;
    if (in_w + 2 * pad_x < kw) return set_last_error(IDF_ERR_SPEC, "noalloc: kernel wider than the padded row");
    const int out_w = (in_w + 2 * pad_x - kw) / stride_x + 1;
    const int ring_rows = (kh + stride - 1) / stride;
    const size_t ring_bytes = ((size_t)ring_rows * n_streams * out_w * cout * sizeof(float) + 255) / 256 * 256;
    const size_t w_bytes = (size_t)cout * kh * kw * cin * sizeof(float);
    if (ring_bytes + w_bytes > kScratchBytes)
        return set_last_error(IDF_ERR_CAPACITY, "noalloc: ring + weights exceed the built-in scratch (IDF_NOALLOC_SCRATCH_BYTES)");
    const long long q = (long long)n_rows + 2LL * pad - kh;
    const long long rows_out = q < 0 ? 0 : q / stride + 1;
    if (rows_out > out_capacity_rows) return set_last_error(IDF_ERR_CAPACITY, "noalloc: out_capacity_rows too small");

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices)
        return set_last_error(IDF_ERR_CUDA, "noalloc: cudaGetDevice failed");
    unsigned char* scratch;
    {
        // set-up, once per device, with that device current: turn the symbol into a device address
        std::lock_guard<std::mutex> lk(g_mu);
        if (!g_scratch_ptr[dev]) {
            void* p = nullptr;
            cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
            if (e != cudaSuccess || !p) return set_last_error(IDF_ERR_CUDA, "noalloc: cudaGetSymbolAddress failed");
            g_scratch_ptr[dev] = (unsigned char*)p;
        }
        scratch = g_scratch_ptr[dev];
    }
    cudaStream_t st = (cudaStream_t)cuda_stream;
    float* ring = (float*)scratch;
    float* w_packed = (float*)(scratch + ring_bytes);
    // the array keeps whatever the previous call left: the ring must start at zero
    cudaError_t e = cudaMemsetAsync(ring, 0, ring_bytes, st);
    if (e != cudaSuccess) return set_last_error(IDF_ERR_CUDA, "noalloc: memset failed");
    const long long nw = (long long)cout * kh * kw * cin;
    repack_weights_kernel<<<(unsigned)((nw + 255) / 256 > 1184 ? 1184 : (nw + 255) / 256), 256, 0, st>>>(d_weights, w_packed, cout, kh * kw, cin);
    if (cudaGetLastError() != cudaSuccess) return set_last_error(IDF_ERR_CUDA, "noalloc: repack launch failed");

    // the same row-block walk as idf_stream_push + idf_stream_finish for a single layer
    // (blocks as long as the regular entry points' default: neither the ring nor the scratch depends on the length)
    const int row_block = 25088 / in_w < 32 ? 32 : (25088 / in_w > 1024 ? 1024 : 25088 / in_w);
    long long rows_done = 0;
    for (long long r0 = 0; r0 < n_rows; r0 += row_block) {
        const long long r1 = r0 + row_block < n_rows ? r0 + row_block : n_rows;
        const bool last = (r1 == n_rows);
        const long long qq = r1 + pad - kh;
        long long done_end = last ? rows_out : (qq < 0 ? 0 : qq / stride + 1);
        if (done_end < rows_done) done_end = rows_done;
        const long long started = (r1 - 1 + pad) / stride + 1;
        ConvArgs a{};
        a.in = d_in + (size_t)r0 * n_streams * in_w * cin;
        a.w = w_packed; a.bias = d_bias; a.ring = ring; a.out = d_out;
        a.out_row_stride = (long long)out_w * cout;
        a.out_stream_stride = out_capacity_rows * a.out_row_stride;
        a.out_row_base = 0;
        a.event_counter = nullptr;
        a.S = n_streams; a.Win = in_w; a.Wout = out_w; a.Cin = cin; a.Cout = cout; a.Kh = kh; a.Kw = kw;
        a.stride = stride; a.pad = pad; a.relu = relu; a.shift = 0; a.ring_rows = ring_rows;
        a.stride_x = stride_x; a.pad_x = pad_x; a.in_elem = E_F32; a.out_elem = E_F32;
        a.in_elems = (r1 - r0) * (long long)n_streams * in_w * cin;
        a.out_elems = (long long)n_streams * out_capacity_rows * out_w * cout;
        a.ring_elems = (long long)ring_rows * n_streams * out_w * cout;
        a.status = nullptr;          // (no handle, no status word: the range-checked build still skips what is out of range)
        a.r0 = r0; a.r1 = r1; a.o_begin = rows_done; a.o_end = started > done_end ? started : done_end; a.done_end = done_end;
        e = launch_conv_simple(a, IDF_F32, st);
        if (e != cudaSuccess) return set_last_error(IDF_ERR_CUDA, "noalloc: kernel launch failed");
        rows_done = done_end;
        if (last) break;
    }
    if (out_rows) *out_rows = rows_out;
    return IDF_OK;
}
