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
  int O, I, bits, K, g, G, n_keep, M;   // bits: the storage format of the codes (8, 4 or 2)
  int wbits;             // b of the quantizer (8, 6, 4, 3 or 2): qmax = 2^(b-1) - 1
  int score_mode, keep_elems;
  int qmax;
  int branch_begin[PIPE_MAX_ORDERS + 1];  // first order (0-based) of every branch, then K
  pipe_layer_layout lay;
};

pipe_status resolve_layer(const pipe_layer_desc* desc, LayerInfo* out);

constexpr int kPlanSMs = 148;   // SMs of the B200 the decode plan is laid out for

// Device status word of the current device.
int* device_status_word();
void count_launch(int n = 1);
int kernel_choice();
// Streams whose last library call was an expansion (which writes the blob a forward call on the same stream may be about
// to read): an expansion marks its stream, every other call on a stream takes the mark away and learns whether it was there.
void mark_expansion(cudaStream_t stream);
bool take_expansion_mark(cudaStream_t stream);
bool expansion_marked(cudaStream_t stream);   // the same question without clearing the mark

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

// Block records of a channel-block table (layout in pipe.h).
constexpr int kRecHeaderInts = 32;
constexpr int kRecRowbase = 8, kRecStart = 16;              // header words of rowbase[0..7], start[0..7]
constexpr int kRecColmapOff = kRecHeaderInts * 4;           // bytes
constexpr int kRecColmapEntries = 8 * (PIPE_BLOCK_CHANNELS / 8);
constexpr int kRecScaleOff = kRecColmapOff + kRecColmapEntries * 2;
constexpr int kRecBytes = kRecScaleOff + PIPE_BLOCK_ROWS * 4;
static_assert(kRecBytes == PIPE_BLOCK_RECORD_BYTES && kRecBytes % 16 == 0, "record layout");

// Row limit of the blocks of a channel-block table (the definition in pipe.h): R rows kept by the cluster's nk orders.
inline int block_row_limit(int64_t R, int O, int nk, int g) {
  // A cluster of a few blocks (at most PIPE_EVEN_BLOCKS) is cut into blocks of ONE size: a block is closed when the
  // next group would take it beyond the limit, so it ends up to one group (at most nk * g rows) short of it, half a
  // group on average; n blocks of that average size hold the rows, and the limit is the mean block plus that half
  // group.  (Filled to PIPE_BLOCK_ROWS instead, the last block of such a cluster is a small one that costs a tile
  // like the others.)  A cluster of many blocks keeps the widest blocks: there the MMA's width is worth more.
  {
    const int64_t half = (static_cast<int64_t>(nk) * g) / 2;
    const int64_t room = PIPE_BLOCK_ROWS - half > 0 ? PIPE_BLOCK_ROWS - half : 1;
    const int64_t ner = ceil_div<int64_t>(R, room), nec = ceil_div<int64_t>(O, PIPE_BLOCK_CHANNELS);
    const int64_t ne = ner > nec ? ner : nec;
    if (ne >= 1 && ne <= PIPE_EVEN_BLOCKS) {
      const int64_t even = ceil_div<int64_t>(R, ne) + half;
      return static_cast<int>(even < PIPE_BLOCK_ROWS ? even : PIPE_BLOCK_ROWS);
    }
  }
  const int64_t n0r = ceil_div<int64_t>(R, PIPE_BLOCK_ROWS), n0c = ceil_div<int64_t>(O, PIPE_BLOCK_CHANNELS);
  const int64_t n0 = n0r > n0c ? n0r : n0c;
  const int64_t even = round_up<int64_t>(ceil_div<int64_t>(R, n0 > 0 ? n0 : 1), 16) + static_cast<int64_t>(nk) * g;
  return static_cast<int>(even < PIPE_BLOCK_ROWS ? even : PIPE_BLOCK_ROWS);
}
// A bound on the blocks the cut can make: a block closed by its rows stacks more than limit - nk * g of them (the
// next group would have added nk * g at most), a block closed by its channels holds PIPE_BLOCK_CHANNELS / g groups,
// and one block is left open at the end.
inline int block_count_bound(int64_t R, int O, int G, int nk, int g) {
  const int64_t per = block_row_limit(R, O, nk, g) - static_cast<int64_t>(nk) * g;
  const int64_t maxg = PIPE_BLOCK_CHANNELS / g > 0 ? PIPE_BLOCK_CHANNELS / g : 1;
  const int64_t n = R / (per > 0 ? per + 1 : 1) + G / maxg + 2;
  return static_cast<int>(n < G ? n : G);
}

// Raise a device-side error: first error wins.
__device__ inline void raise_status(int* status, int code) { atomicCAS(status, 0, code); }

// clamp(rne(v / s)) as an int8 lane.  The IEEE quotient is what defines the code (Eq. 1 with true
// division), but a division costs an order of magnitude more than a multiplication, so the quotient is
// first estimated as t = v * r with r = rn(1 / s): t is within a relative 2^-22.9 of the real quotient,
// as is the IEEE quotient itself (2^-24), so both round to the same integer unless the estimate lies
// within |t| * 2^-21 of a rounding boundary (an odd multiple of one half) -- only then, a few times in a
// hundred thousand, is the division carried out.  Beyond +-130 both clamp.
__device__ __forceinline__ uint32_t quant_lane(float v, float s, float r) {
  const float t = __fmul_rn(v, r);
  float q = rintf(t);
  const float at = fabsf(t);
  if (at > 130.f) {
    q = copysignf(127.f, t);
  } else if (0.5f - fabsf(__fsub_rn(t, q)) <= at * 4.76837158203125e-07f) {
    q = rintf(__fdiv_rn(v, s));
  }
  q = fminf(fmaxf(q, -127.f), 127.f);
  return static_cast<uint32_t>(static_cast<int>(q)) & 0xffu;
}

// The same code with the division always carried out; a zero step gives the code 0 (Eq. 1 on an all-zero tensor).
__device__ __forceinline__ uint32_t quant_lane_exact(float v, float s) {
  float q = 0.f;
  if (s != 0.f) q = fminf(fmaxf(rintf(__fdiv_rn(v, s)), -127.f), 127.f);
  return static_cast<uint32_t>(static_cast<int>(q)) & 0xffu;
}

// The estimate needs a reciprocal that neither overflows nor is subnormal.
__device__ __forceinline__ bool quant_step_is_fast(float s) { return s >= 1e-30f && s <= 1e30f; }

// Four codes as the bytes of one word, lowest address first.
__device__ __forceinline__ uint32_t quant4(const float4& f, float s, float r, bool fast) {
  if (fast) return quant_lane(f.x, s, r) | (quant_lane(f.y, s, r) << 8) | (quant_lane(f.z, s, r) << 16) | (quant_lane(f.w, s, r) << 24);
  return quant_lane_exact(f.x, s) | (quant_lane_exact(f.y, s) << 8) | (quant_lane_exact(f.z, s) << 16) | (quant_lane_exact(f.w, s) << 24);
}

// sigma of Eq. 9 for an inner layer (Sec. 3.2 names ReLU, SiLU, GeLU and sigmoid), in binary32: kind 0 identity,
// 1 ReLU, 2 SiLU v / (1 + exp(-v)), 3 GeLU v (1 + erf(v / sqrt 2)) / 2, 4 sigmoid 1 / (1 + exp(-v)).
__device__ __forceinline__ float apply_activation(float v, int kind) {
  switch (kind) {
    case 1: return fmaxf(v, 0.f);
    case 2: return __fdiv_rn(v, __fadd_rn(1.f, expf(-v)));
    case 3: return __fmul_rn(__fmul_rn(0.5f, v), __fadd_rn(1.f, erff(__fmul_rn(v, 0.70710678118654752f))));
    case 4: return __fdiv_rn(1.f, __fadd_rn(1.f, expf(-v)));
    default: return v;
  }
}

// Per-order pointers into a blob, passed to kernels by value.
struct OrderView {
  const uint8_t* codes;   // canonical packed codes
  const uint8_t* kcodes;  // kernel-layout codes
  const uint8_t* wcodes;  // int8 copy in the tensor-core operand layout, or nullptr
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
  v.wcodes = L.lay.wcodes_off[k] ? b + L.lay.wcodes_off[k] : nullptr;
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
  int8_t* yq;              // re-quantized output (ForwardArgs::q8_out), else unused
  const float* out_scale;  // its step: one float on the device
  int k_begin, k_end;
  const int32_t* zp;       // zero point of asymmetric activation codes (one int on the device), or nullptr for 0
  const int32_t* dec;      // decode-unit table of this branch's cluster of orders (n, b_0 .. b_n), or nullptr
  const int32_t* blk;      // channel-block table of this branch's cluster of orders (n, b_0 .. b_n), or nullptr
  const uint8_t* rec;      // the table's block records (PIPE_BLOCK_RECORD_BYTES each), or nullptr
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
  // fused inner-layer epilogue (q8_out != 0): yq = clamp(rne(act(y) / out_scale)) as int8, row pitch ldyq; y is not written
  int decode_split;   // CTAs that share a decode unit's reduction axis (from the layout; 0 = no decode tables)
  int blob_settled;   // the library's last call on this stream was no expansion: a kernel launched with programmatic stream
                      // serialization may read the expanded layer before it waits for the launch before it
  int q8_out, relu;   // relu: the activation kind (see apply_activation; the name is from the first version)
  // the channel-block table and block records of the cluster of ALL orders, for a summed ensemble whose predictors
  // share one input (nullptr: the layer has none, or the call is no such ensemble)
  const int32_t* sum_blk;
  const uint8_t* sum_rec;
  int64_t ldyq;
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
pipe_status forward_decode_tc(const ForwardArgs& a, cudaStream_t stream);      // T <= 16 on tcgen05 (decode-unit tables)

}  // namespace pipe
