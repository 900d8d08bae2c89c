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
  return quantize_act_impl(d_x, T, I, ldx, d_static_scale, d_xq, ldxq, d_sx, static_cast<uint32_t*>(d_ws),
                           static_cast<cudaStream_t>(stream));
}
