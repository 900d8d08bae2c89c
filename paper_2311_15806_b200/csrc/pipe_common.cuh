// Shared host/device helpers of libpipe (internal; the public surface is include/pipe.h).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "pipe.h"

namespace pipe {

constexpr uint32_t kBlobMagic = 0x50495045u;  // "PIPE"
constexpr int kHeaderBytes = 1024;
constexpr int kKernelKAlign = 128;  // kernel-layout rows are padded to this many codes

// Resolved, validated view of a pipe_layer_desc.
struct LayerInfo {
  int O, I, bits, K, g, G, n_keep, M;
  int qmax;
  int branch_begin[PIPE_MAX_ORDERS + 1];  // first order (0-based) of every branch, then K
  pipe_layer_layout lay;
};

pipe_status resolve_layer(const pipe_layer_desc* desc, LayerInfo* out);

// Device status word of the current device.
int* device_status_word();
void count_launch(int n = 1);
int kernel_choice();

inline pipe_status cuda_ok(cudaError_t e) { return e == cudaSuccess ? PIPE_OK : PIPE_ERR_CUDA; }

inline pipe_status launch_status() { return cuda_ok(cudaGetLastError()); }

template <typename T>
__host__ __device__ inline T ceil_div(T a, T b) {
  return (a + b - 1) / b;
}

template <typename T>
__host__ __device__ inline T round_up(T a, T b) {
  return ceil_div(a, b) * b;
}

// Raise a device-side error: first error wins.
__device__ inline void raise_status(int* status, int code) { atomicCAS(status, 0, code); }

// Per-order pointers into a blob, passed to kernels by value.
struct OrderView {
  const uint8_t* codes;   // canonical packed codes
  const uint8_t* kcodes;  // kernel-layout codes
  const float* scales;
  const int32_t* cum;     // [G+1]
  int rows;
  int row_off;            // column offset of this order in the partials matrix
};

inline OrderView order_view(const LayerInfo& L, const void* blob, int k) {
  const uint8_t* b = static_cast<const uint8_t*>(blob);
  OrderView v;
  v.codes = b + L.lay.codes_off[k];
  v.kcodes = b + L.lay.kcodes_off[k];
  v.scales = reinterpret_cast<const float*>(b + L.lay.scales_off[k]);
  v.cum = reinterpret_cast<const int32_t*>(b + L.lay.cum_off[k]);
  v.rows = L.lay.rows[k];
  int off = 0;
  for (int j = 0; j < k; ++j) off += L.lay.rows[j];
  v.row_off = off;
  return v;
}

// One ensemble branch of a forward call.
struct BranchArgs {
  const int8_t* xq;
  const float* sx;
  float* y;
  int k_begin, k_end;
  int add_bias;    // bias enters this branch
  int accumulate;  // y += result (summed ensemble, branches after the first)
};

struct ForwardArgs {
  OrderView order[PIPE_MAX_ORDERS];
  BranchArgs branch[PIPE_MAX_ORDERS];
  int num_branches;
  int O, I, bits, g, G;
  int64_t T, ldxq, ldy;
  const float* bias;
  int32_t* partials;
  int total_rows;
  int kernel_row_bytes, canon_row_bytes;
  int* status;
  // implicit convolution (conv_on != 0): branch[0].xq is the NHWC input, T = N*H*W
  int conv_on, cN, cH, cW, cC, ckh, ckw, cph, cpw;
  int cHo, cWo, csh, csw;   // output height / width and the strides
};

// Tensor map of a row-major byte matrix [rows, inner_bytes] with row pitch pitch_bytes (a multiple of 16) and
// a box of box_inner x box_rows bytes; swizzle128 selects the 128-byte swizzle.  False when the driver entry
// point is missing or the encoding fails.
bool make_tensor_map_2d_u8(CUtensorMap* map, const void* base, uint64_t inner_bytes, uint64_t rows, uint64_t pitch_bytes,
                           uint32_t box_inner, uint32_t box_rows, bool swizzle128);

// GEMM back ends (each returns PIPE_ERR_UNSUPPORTED when it cannot take the request).
pipe_status forward_reference(const ForwardArgs& a, cudaStream_t stream);
pipe_status forward_tcgen05(const ForwardArgs& a, cudaStream_t stream);
pipe_status forward_tcgen05_pair(const ForwardArgs& a, cudaStream_t stream);   // two-SM form (clusters of two CTAs)
pipe_status forward_stream(const ForwardArgs& a, cudaStream_t stream);

}  // namespace pipe
