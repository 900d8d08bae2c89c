// pipe_quantize_act: per-tensor symmetric int8 quantization of the layer input
// (Appendix B, Eq. 9: the layer consumes Q(x) and one scale lambda_x).
//
// Two HBM-bound passes: (1) grid-wide max|x| through an order-free unsigned atomicMax on the
// magnitude bits, (2) divide / round-half-even / clamp / 16-byte int8 stores.  Tensors that
// fit the 126 MB L2 are read from HBM once.
#include "pipe_common.cuh"

namespace pipe {

constexpr int kQThreads = 256;

__device__ __forceinline__ uint32_t q_abs_key(float v) { return __float_as_uint(v) & 0x7fffffffu; }

struct QuantArgs {
  const float* x;
  int8_t* xq;
  int64_t T, ldx, ldxq;
  int I;
  int chunks_per_row;   // ceil(I / 16)
  int64_t total_chunks;
  int vec_in, vec_out;  // rows are 16-byte aligned on the input / output side
};

__device__ __forceinline__ void load16(const QuantArgs& p, int64_t c, float (&v)[16], int64_t& t, int& i0) {
  t = c / p.chunks_per_row;
  i0 = static_cast<int>(c - t * p.chunks_per_row) * 16;
  const float* row = p.x + t * p.ldx;
  if (p.vec_in && i0 + 16 <= p.I) {
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const float4 f = __ldg(reinterpret_cast<const float4*>(row + i0) + w);
      v[4 * w] = f.x; v[4 * w + 1] = f.y; v[4 * w + 2] = f.z; v[4 * w + 3] = f.w;
    }
  } else {
#pragma unroll
    for (int e = 0; e < 16; ++e) v[e] = (i0 + e < p.I) ? row[i0 + e] : 0.f;
  }
}

// ws[0] = max over the tensor of the magnitude bits (ws[0] must be zero on entry).
__global__ void __launch_bounds__(kQThreads) act_absmax_kernel(const QuantArgs p, uint32_t* ws) {
  uint32_t m = 0;
  for (int64_t c = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; c < p.total_chunks;
       c += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    float v[16];
    int64_t t;
    int i0;
    load16(p, c, v, t, i0);
#pragma unroll
    for (int e = 0; e < 16; ++e) m = max(m, q_abs_key(v[e]));
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, d));
  __shared__ uint32_t part[kQThreads / 32];
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < kQThreads / 32; ++w) m = max(m, part[w]);
    if (m) atomicMax(ws, m);
  }
}

// lambda_x = absmax / 127 (or the static scale); xq = clamp(rne(x / lambda_x), -127, 127).
__global__ void __launch_bounds__(kQThreads) act_quantize_kernel(const QuantArgs p, const uint32_t* ws,
                                                                 const float* static_scale, float* sx_out, int* status) {
  const uint32_t mbits = ws[0];
  float s;
  if (static_scale) s = *static_scale;
  else s = __fdiv_rn(__uint_as_float(mbits), 127.f);
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    *sx_out = s;
    if (mbits >= 0x7f800000u) raise_status(status, PIPE_ERR_NONFINITE);
    if (static_scale && !(s >= 0.f && s < __uint_as_float(0x7f800000u))) raise_status(status, PIPE_ERR_INVALID_ARG);
  }
  for (int64_t c = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; c < p.total_chunks;
       c += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    float v[16];
    int64_t t;
    int i0;
    load16(p, c, v, t, i0);
    uint32_t w[4] = {0, 0, 0, 0};
#pragma unroll
    for (int e = 0; e < 16; ++e) {
      float q = 0.f;
      if (s != 0.f) {
        q = rintf(__fdiv_rn(v[e], s));
        q = fminf(fmaxf(q, -127.f), 127.f);
      }
      w[e >> 2] |= (static_cast<uint32_t>(static_cast<int>(q)) & 0xffu) << (8 * (e & 3));
    }
    int8_t* orow = p.xq + t * p.ldxq;
    if (p.vec_out && i0 + 16 <= p.I) {
      *reinterpret_cast<uint4*>(orow + i0) = make_uint4(w[0], w[1], w[2], w[3]);
    } else {
#pragma unroll
      for (int e = 0; e < 16; ++e)
        if (i0 + e < p.I) orow[i0 + e] = static_cast<int8_t>(w[e >> 2] >> (8 * (e & 3)));
    }
  }
}

// ---- contiguous tensors (ldx == ldxq == I, I a multiple of 4, 16-byte aligned input): the tensor is one
// flat array, a thread takes one float4 per trip (a warp reads 512 and writes 128 contiguous bytes per
// instruction) and keeps four trips in flight.
constexpr int kFlatUnroll = 4;

__global__ void __launch_bounds__(kQThreads) act_absmax_flat_kernel(const float4* __restrict__ x, int64_t n4, uint32_t* ws) {
  uint32_t m = 0;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x;
  for (; i + (kFlatUnroll - 1) * stride < n4; i += kFlatUnroll * stride) {
    float4 f[kFlatUnroll];
#pragma unroll
    for (int u = 0; u < kFlatUnroll; ++u) f[u] = __ldg(x + i + u * stride);
#pragma unroll
    for (int u = 0; u < kFlatUnroll; ++u)
      m = max(max(m, max(q_abs_key(f[u].x), q_abs_key(f[u].y))), max(q_abs_key(f[u].z), q_abs_key(f[u].w)));
  }
  for (; i < n4; i += stride) {
    const float4 f = __ldg(x + i);
    m = max(max(m, max(q_abs_key(f.x), q_abs_key(f.y))), max(q_abs_key(f.z), q_abs_key(f.w)));
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, d));
  __shared__ uint32_t part[kQThreads / 32];
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < kQThreads / 32; ++w) m = max(m, part[w]);
    if (m) atomicMax(ws, m);
  }
}

__global__ void __launch_bounds__(kQThreads) act_quantize_flat_kernel(const float4* __restrict__ x, int64_t n4,
                                                                      uint32_t* __restrict__ xq, const uint32_t* ws,
                                                                      const float* static_scale, float* sx_out, int* status) {
  const uint32_t mbits = ws[0];
  float s;
  if (static_scale) s = *static_scale;
  else s = __fdiv_rn(__uint_as_float(mbits), 127.f);
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    *sx_out = s;
    if (mbits >= 0x7f800000u) raise_status(status, PIPE_ERR_NONFINITE);
    if (static_scale && !(s >= 0.f && s < __uint_as_float(0x7f800000u))) raise_status(status, PIPE_ERR_INVALID_ARG);
  }
  const bool fast = quant_step_is_fast(s);
  const float r = fast ? __frcp_rn(s) : 0.f;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x;
  for (; i + (kFlatUnroll - 1) * stride < n4; i += kFlatUnroll * stride) {
    float4 f[kFlatUnroll];
#pragma unroll
    for (int u = 0; u < kFlatUnroll; ++u) f[u] = __ldg(x + i + u * stride);
#pragma unroll
    for (int u = 0; u < kFlatUnroll; ++u) xq[i + u * stride] = quant4(f[u], s, r, fast);
  }
  for (; i < n4; i += stride) xq[i] = quant4(__ldg(x + i), s, r, fast);
}

__global__ void act_empty_kernel(const float* static_scale, float* sx_out) {
  if (threadIdx.x == 0) *sx_out = static_scale ? *static_scale : 0.f;
}

pipe_status quantize_act_impl(const float* d_x, int64_t T, int32_t I, int64_t ldx, const float* d_static_scale,
                              int8_t* d_xq, int64_t ldxq, float* d_sx, uint32_t* d_scratch, cudaStream_t s) {
  int* status = device_status_word();
  if (!status) return PIPE_ERR_CUDA;
  if (T == 0) {
    act_empty_kernel<<<1, 32, 0, s>>>(d_static_scale, d_sx);
    count_launch(1);
    return launch_status();
  }
  QuantArgs p;
  p.x = d_x; p.xq = d_xq; p.T = T; p.ldx = ldx; p.ldxq = ldxq; p.I = I;
  p.chunks_per_row = ceil_div(I, 16);
  p.total_chunks = T * p.chunks_per_row;
  p.vec_in = ((reinterpret_cast<uintptr_t>(d_x) & 15) == 0) && (ldx % 4 == 0);
  p.vec_out = ((reinterpret_cast<uintptr_t>(d_xq) & 15) == 0) && (ldxq % 16 == 0);
  int sms = 148;
  int dev = 0;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int64_t want = ceil_div<int64_t>(p.total_chunks, kQThreads);
  const int grid = static_cast<int>(want < static_cast<int64_t>(sms) * 8 ? want : static_cast<int64_t>(sms) * 8);
  if (cudaMemsetAsync(d_scratch, 0, 16, s) != cudaSuccess) return PIPE_ERR_CUDA;
  if (ldx == I && ldxq == I && I % 4 == 0 && p.vec_in && (reinterpret_cast<uintptr_t>(d_xq) & 3) == 0) {
    const int64_t n4 = T * (I / 4);
    const int64_t want4 = ceil_div<int64_t>(n4, kQThreads * kFlatUnroll);
    const int g4 = static_cast<int>(want4 < static_cast<int64_t>(sms) * 8 ? want4 : static_cast<int64_t>(sms) * 8);
    // (with a static scale the first pass still serves the non-finite check of the input)
    act_absmax_flat_kernel<<<g4, kQThreads, 0, s>>>(reinterpret_cast<const float4*>(d_x), n4, d_scratch);
    act_quantize_flat_kernel<<<g4, kQThreads, 0, s>>>(reinterpret_cast<const float4*>(d_x), n4, reinterpret_cast<uint32_t*>(d_xq),
                                                      d_scratch, d_static_scale, d_sx, status);
    count_launch(2);
    return launch_status();
  }
  if (!d_static_scale) {
    act_absmax_kernel<<<grid, kQThreads, 0, s>>>(p, d_scratch);
    count_launch(1);
  } else {
    // a static scale still needs the non-finite check of the input
    act_absmax_kernel<<<grid, kQThreads, 0, s>>>(p, d_scratch);
    count_launch(1);
  }
  act_quantize_kernel<<<grid, kQThreads, 0, s>>>(p, d_scratch, d_static_scale, d_sx, status);
  count_launch(1);
  return launch_status();
}

// ---- the other activation quantizers of Sec. 4.3 (A6 / A4, asymmetric): same two passes, division always carried
// out.  ws[0] = largest magnitude key (non-finite check, symmetric scale), ws[1] = bits of max(x, 0),
// ws[2] = bits of max(-x, 0); all three are non-negative floats, whose order is the order of their bit patterns.
__global__ void __launch_bounds__(kQThreads) act_range_kernel(const QuantArgs p, uint32_t* ws) {
  uint32_t m = 0, hi = 0, nlo = 0;
  for (int64_t c = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; c < p.total_chunks;
       c += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    float v[16];
    int64_t t;
    int i0;
    load16(p, c, v, t, i0);
#pragma unroll
    for (int e = 0; e < 16; ++e) {
      m = max(m, q_abs_key(v[e]));
      hi = max(hi, __float_as_uint(fmaxf(v[e], 0.f)) & 0x7fffffffu);   // (the mask turns a -0 into +0)
      nlo = max(nlo, __float_as_uint(fmaxf(-v[e], 0.f)) & 0x7fffffffu);
    }
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) {
    m = max(m, __shfl_xor_sync(0xffffffffu, m, d));
    hi = max(hi, __shfl_xor_sync(0xffffffffu, hi, d));
    nlo = max(nlo, __shfl_xor_sync(0xffffffffu, nlo, d));
  }
  if ((threadIdx.x & 31) == 0) {
    if (m) atomicMax(ws, m);
    if (hi) atomicMax(ws + 1, hi);
    if (nlo) atomicMax(ws + 2, nlo);
  }
}

__global__ void __launch_bounds__(kQThreads) act_quantize_ex_kernel(const QuantArgs p, const uint32_t* ws, int act_bits, int asym,
                                                                    const float* static_scale, const float* static_range,
                                                                    float* sx_out, int32_t* zp_out, int* status) {
  const uint32_t mbits = ws[0];
  const float half = static_cast<float>(1 << (act_bits - 1));
  float s, z = 0.f, cmin, cmax;
  bool bad_arg = false;
  if (!asym) {
    const float qx = half - 1.f;
    s = static_scale ? *static_scale : __fdiv_rn(__uint_as_float(mbits), qx);
    bad_arg = static_scale && !(s >= 0.f && s < __uint_as_float(0x7f800000u));
    cmin = -qx;
    cmax = qx;
  } else {
    float lo = -__uint_as_float(ws[2]), hi = __uint_as_float(ws[1]);
    if (static_range) {
      lo = static_range[0];
      hi = static_range[1];
      bad_arg = !(lo <= 0.f && hi >= 0.f && lo > -__uint_as_float(0x7f800000u) && hi < __uint_as_float(0x7f800000u));
    }
    s = __fdiv_rn(__fsub_rn(hi, lo), 2.f * half - 1.f);
    cmin = -half;
    cmax = half - 1.f;
    if (s != 0.f) z = fminf(fmaxf(rintf(__fsub_rn(-half, __fdiv_rn(lo, s))), cmin), cmax);
  }
  if (bad_arg) s = 0.f, z = 0.f;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    *sx_out = s;
    *zp_out = static_cast<int32_t>(z);
    if (mbits >= 0x7f800000u) raise_status(status, PIPE_ERR_NONFINITE);
    if (bad_arg) raise_status(status, PIPE_ERR_INVALID_ARG);
  }
  for (int64_t c = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; c < p.total_chunks;
       c += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    float v[16];
    int64_t t;
    int i0;
    load16(p, c, v, t, i0);
    uint32_t w[4] = {0, 0, 0, 0};
#pragma unroll
    for (int e = 0; e < 16; ++e) {
      float q = z;
      if (s != 0.f) q = fminf(fmaxf(__fadd_rn(rintf(__fdiv_rn(v[e], s)), z), cmin), cmax);
      w[e >> 2] |= (static_cast<uint32_t>(static_cast<int>(q)) & 0xffu) << (8 * (e & 3));
    }
    int8_t* orow = p.xq + t * p.ldxq;
    if (p.vec_out && i0 + 16 <= p.I) {
      *reinterpret_cast<uint4*>(orow + i0) = make_uint4(w[0], w[1], w[2], w[3]);
    } else {
#pragma unroll
      for (int e = 0; e < 16; ++e)
        if (i0 + e < p.I) orow[i0 + e] = static_cast<int8_t>(w[e >> 2] >> (8 * (e & 3)));
    }
  }
}

__global__ void act_empty_ex_kernel(const float* static_scale, float* sx_out, int32_t* zp_out) {
  if (threadIdx.x == 0) {
    *sx_out = static_scale ? *static_scale : 0.f;
    *zp_out = 0;
  }
}

}  // namespace pipe

using namespace pipe;

extern "C" pipe_status pipe_quantize_act(const float* d_x, int64_t T, int32_t I, int64_t ldx, const float* d_static_scale,
                                         int8_t* d_xq, int64_t ldxq, float* d_sx, void* d_ws, size_t ws_bytes,
                                         void* stream) {
  if (T < 0 || I <= 0) return PIPE_ERR_INVALID_ARG;
  if (!d_sx || !d_ws) return PIPE_ERR_INVALID_ARG;
  if (T > 0 && (!d_x || !d_xq)) return PIPE_ERR_INVALID_ARG;
  if (ldx < I || ldxq < I) return PIPE_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(d_x) & 3) || (reinterpret_cast<uintptr_t>(d_ws) & 255) ||
      (reinterpret_cast<uintptr_t>(d_sx) & 3))
    return PIPE_ERR_ALIGNMENT;
  if (ws_bytes < 256) return PIPE_ERR_WORKSPACE;
  const pipe_status st = quantize_act_impl(d_x, T, I, ldx, d_static_scale, d_xq, ldxq, d_sx, static_cast<uint32_t*>(d_ws),
                                           static_cast<cudaStream_t>(stream));
  // (this call's kernels now stand between an expansion and what follows)
  if (st == PIPE_OK) take_expansion_mark(static_cast<cudaStream_t>(stream));
  return st;
}

extern "C" pipe_status pipe_quantize_act_ex(const float* d_x, int64_t T, int32_t I, int64_t ldx, int32_t act_bits,
                                            int32_t asymmetric, const float* d_static_scale, const float* d_static_range,
                                            int8_t* d_xq, int64_t ldxq, float* d_sx, int32_t* d_zp, void* d_ws,
                                            size_t ws_bytes, void* stream) {
  if (T < 0 || I <= 0) return PIPE_ERR_INVALID_ARG;
  if (!(act_bits == 8 || act_bits == 6 || act_bits == 4)) return PIPE_ERR_INVALID_ARG;
  if (!d_sx || !d_zp || !d_ws) return PIPE_ERR_INVALID_ARG;
  if (T > 0 && (!d_x || !d_xq)) return PIPE_ERR_INVALID_ARG;
  if (ldx < I || ldxq < I) return PIPE_ERR_INVALID_ARG;
  if (asymmetric ? d_static_scale != nullptr : d_static_range != nullptr) return PIPE_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(d_x) & 3) || (reinterpret_cast<uintptr_t>(d_ws) & 255) || (reinterpret_cast<uintptr_t>(d_sx) & 3) ||
      (reinterpret_cast<uintptr_t>(d_zp) & 3) || (reinterpret_cast<uintptr_t>(d_static_scale) & 3) ||
      (reinterpret_cast<uintptr_t>(d_static_range) & 3))
    return PIPE_ERR_ALIGNMENT;
  if (ws_bytes < 256) return PIPE_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int* status = device_status_word();
  if (!status) return PIPE_ERR_CUDA;
  take_expansion_mark(s);   // (kernels follow: they stand between an expansion and what comes next on the stream)
  if (T == 0) {
    act_empty_ex_kernel<<<1, 32, 0, s>>>(d_static_scale, d_sx, d_zp);
    count_launch(1);
    return launch_status();
  }
  QuantArgs p;
  p.x = d_x; p.xq = d_xq; p.T = T; p.ldx = ldx; p.ldxq = ldxq; p.I = I;
  p.chunks_per_row = ceil_div(I, 16);
  p.total_chunks = T * p.chunks_per_row;
  p.vec_in = ((reinterpret_cast<uintptr_t>(d_x) & 15) == 0) && (ldx % 4 == 0);
  p.vec_out = ((reinterpret_cast<uintptr_t>(d_xq) & 15) == 0) && (ldxq % 16 == 0);
  int sms = 148, dev = 0;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int64_t want = ceil_div<int64_t>(p.total_chunks, kQThreads);
  const int grid = static_cast<int>(want < static_cast<int64_t>(sms) * 8 ? want : static_cast<int64_t>(sms) * 8);
  uint32_t* scratch = static_cast<uint32_t*>(d_ws);
  if (cudaMemsetAsync(scratch, 0, 16, s) != cudaSuccess) return PIPE_ERR_CUDA;
  act_range_kernel<<<grid, kQThreads, 0, s>>>(p, scratch);
  act_quantize_ex_kernel<<<grid, kQThreads, 0, s>>>(p, scratch, act_bits, asymmetric ? 1 : 0, d_static_scale, d_static_range, d_sx,
                                                    d_zp, status);
  count_launch(2);
  return launch_status();
}

// ------------------------------------------------------------------------------------------------
// Explicit lowering of a quantized NHWC tensor to the rows of the convolution's GEMM, for the geometries the implicit
// convolution does not take (channel counts that are not multiples of 128: a network's first layer, narrow layers).
namespace pipe {

struct LowerArgs {
  const int8_t* x;
  int8_t* rows;
  int64_t ld_rows, total;   // total = T * kh * kw * ceil(C / 16) pieces of up to 16 channels
  int N, H, W, C, kh, kw, ph, pw, sh, sw, Ho, Wo, cpieces;
  int vec;                  // 16-byte loads and stores are possible (C % 16 == 0, aligned pointers and pitch)
};

__global__ void __launch_bounds__(256) lower_conv_input_kernel(const __grid_constant__ LowerArgs a) {
  for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < a.total; i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int piece = static_cast<int>(i % a.cpieces);
    int64_t r = i / a.cpieces;
    const int tap = static_cast<int>(r % (a.kh * a.kw));
    const int64_t t = r / (a.kh * a.kw);
    const int wo = static_cast<int>(t % a.Wo);
    const int ho = static_cast<int>((t / a.Wo) % a.Ho);
    const int n = static_cast<int>(t / (static_cast<int64_t>(a.Wo) * a.Ho));
    const int h = a.sh * ho + tap / a.kw - a.ph, w = a.sw * wo + tap % a.kw - a.pw;
    const bool in = h >= 0 && h < a.H && w >= 0 && w < a.W;
    const int c0 = piece * 16, nc = min(16, a.C - c0);
    int8_t* dst = a.rows + t * a.ld_rows + static_cast<int64_t>(tap) * a.C + c0;
    const int8_t* src = a.x + ((static_cast<int64_t>(n) * a.H + h) * a.W + w) * a.C + c0;
    if (a.vec) {
      *reinterpret_cast<uint4*>(dst) = in ? __ldg(reinterpret_cast<const uint4*>(src)) : make_uint4(0, 0, 0, 0);
    } else {
      for (int c = 0; c < nc; ++c) dst[c] = in ? __ldg(src + c) : static_cast<int8_t>(0);
    }
  }
}

}  // namespace pipe

extern "C" pipe_status pipe_lower_conv_input(const pipe_conv_geom* geom, const int8_t* d_xq, int8_t* d_rows, int64_t ld_rows,
                                             void* stream) {
  if (!geom || !d_xq || !d_rows) return PIPE_ERR_INVALID_ARG;
  if (geom->batch < 1 || geom->height < 1 || geom->width < 1 || geom->channels < 1 || geom->kernel_h < 1 || geom->kernel_w < 1 ||
      geom->stride_h < 0 || geom->stride_w < 0 || geom->pad_h < 0 || geom->pad_w < 0)
    return PIPE_ERR_INVALID_ARG;
  const int sh = geom->stride_h > 0 ? geom->stride_h : 1, sw = geom->stride_w > 0 ? geom->stride_w : 1;
  if (geom->pad_h >= geom->kernel_h || geom->pad_w >= geom->kernel_w) return PIPE_ERR_SHAPE;
  if (geom->height + 2 * geom->pad_h < geom->kernel_h || geom->width + 2 * geom->pad_w < geom->kernel_w) return PIPE_ERR_SHAPE;
  const int64_t I = static_cast<int64_t>(geom->kernel_h) * geom->kernel_w * geom->channels;
  if (I > INT32_MAX || ld_rows < I) return PIPE_ERR_INVALID_ARG;
  LowerArgs a;
  a.x = d_xq; a.rows = d_rows; a.ld_rows = ld_rows;
  a.N = geom->batch; a.H = geom->height; a.W = geom->width; a.C = geom->channels;
  a.kh = geom->kernel_h; a.kw = geom->kernel_w; a.ph = geom->pad_h; a.pw = geom->pad_w; a.sh = sh; a.sw = sw;
  a.Ho = (a.H + 2 * a.ph - a.kh) / sh + 1;
  a.Wo = (a.W + 2 * a.pw - a.kw) / sw + 1;
  a.cpieces = ceil_div(a.C, 16);
  a.total = static_cast<int64_t>(a.N) * a.Ho * a.Wo * a.kh * a.kw * a.cpieces;
  a.vec = (a.C % 16 == 0 && ld_rows % 16 == 0 && !(reinterpret_cast<uintptr_t>(d_xq) & 15) && !(reinterpret_cast<uintptr_t>(d_rows) & 15)) ? 1 : 0;
  int sms = 148, dev = 0;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int64_t want = ceil_div<int64_t>(a.total, 256);
  const int grid = static_cast<int>(want < static_cast<int64_t>(sms) * 16 ? want : static_cast<int64_t>(sms) * 16);
  take_expansion_mark(static_cast<cudaStream_t>(stream));
  lower_conv_input_kernel<<<grid > 0 ? grid : 1, 256, 0, static_cast<cudaStream_t>(stream)>>>(a);
  count_launch(1);
  return launch_status();
}
