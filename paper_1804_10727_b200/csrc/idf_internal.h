// Internal declarations shared by the host side of the library and its kernels.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

namespace idf {

// element types of activation rows travelling between layers
enum Elem : int { E_F32 = 0, E_BF16 = 1, E_I8 = 2, E_I32 = 3 };

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
    void* out;             // emitted rows
    long long out_row_stride, out_stream_stride, out_row_base;  // element strides; row o goes to (o - out_row_base)
    unsigned long long* event_counter;  // sparse path: number of non-zero events applied
    int S, Win, Wout, Cin, Cout, Kh, Kw, stride, pad, relu, shift, ring_rows;
    int stride_x, pad_x;   // x axis: equal to stride/pad, except 1 and 0 on width-1 (1D) maps
    int in_elem, out_elem; // Elem
    long long r0, r1;      // input rows [r0, r1) arrive in this block
    long long o_begin, o_end;  // output rows [o_begin, o_end) are visited
    long long done_end;    // rows o < done_end are complete after this block: emit them, free their slots
};

struct PoolArgs {
    const void* in;        // [r - r0][S][Win][C]
    void* state;           // [S][Wout][C] running maximum of the first row of a pair
    void* out;
    long long out_row_stride, out_stream_stride, out_row_base;
    int S, Win, Wout, C, elem;
    long long r0, r1, o_begin, o_end, done_end;
};

// CUDA-core kernels (every type, every shape)
cudaError_t launch_conv_simple(const ConvArgs& a, int dtype, cudaStream_t st);
cudaError_t launch_conv_sparse(const ConvArgs& a, int dtype, cudaStream_t st);
cudaError_t launch_pool(const PoolArgs& a, cudaStream_t st);
size_t conv_sparse_max_smem();

}  // namespace idf
