// CUDA-core (dp4a) kernel of the expanded layer (Appendix B, Eq. 9; Sec. 3.2 for the branches).
//
// The straightforward statement of the forward pass on the GPU: one order at a time, codes
// read from the CANONICAL packed section, one int32 accumulator per (token, channel, order),
// fixed-order fp32 epilogue.  It takes every shape the ABI allows, so it is the path for
// odd sizes, and because it shares neither the code layout nor the tiling of the tensor-core
// kernels it doubles as a full-size cross-check for them.
#include "pipe_common.cuh"

namespace pipe {

constexpr int kRefT = 64;        // tokens per block
constexpr int kRefC = 64;        // channels per block
constexpr int kRefKB = 64;       // reduction bytes (int8 lanes) per step
constexpr int kRefWords = kRefKB / 4;
constexpr int kRefPitch = kRefWords + 1;

// Codes i..i+3 of a canonical row (two's complement b-bit fields, element e at bit e*b of the
// row's little-endian bit stream) as four sign-extended int8 lanes; lanes at or beyond I are 0.
__device__ __forceinline__ uint32_t canon_lanes(const uint8_t* row, int i, int I, int bits) {
  uint32_t out = 0;
  const int per = 8 / bits;
  const uint32_t mask = (1u << bits) - 1u, sign = 1u << (bits - 1);
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const int el = i + e;
    if (el >= I) break;
    const uint32_t f = (static_cast<uint32_t>(row[el / per]) >> ((el % per) * bits)) & mask;
    const int v = static_cast<int>(f ^ sign) - static_cast<int>(sign);
    out |= (static_cast<uint32_t>(v) & 0xffu) << (8 * e);
  }
  return out;
}

__global__ void __launch_bounds__(256) ref_forward_kernel(const ForwardArgs a, const int sum_mode) {
  __shared__ uint32_t xs[kRefT][kRefPitch];
  __shared__ uint32_t wsm[kRefC][kRefPitch];
  __shared__ int crow[kRefC];

  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  const int c0 = blockIdx.x * kRefC;
  const int64_t t0 = static_cast<int64_t>(blockIdx.y) * kRefT;
  const int m_first = sum_mode ? 0 : blockIdx.z;
  const int m_last = sum_mode ? a.num_branches : blockIdx.z + 1;

  float total[4][4];
  for (int m = m_first; m < m_last; ++m) {
    const BranchArgs br = a.branch[m];
    const float sx = *br.sx;
    // asymmetric activation codes (Sec. 4.3): sum_i (c - z) q = sum_i c q - z * sum_i q; the row sum of the weight
    // codes comes out of the same loop (dp4a against four ones)
    const int zp = br.zp ? *br.zp : 0;
    float out_step = 0.f;
    if (a.q8_out) {
      out_step = *br.out_scale;
      if (!(out_step >= 0.f && out_step < __uint_as_float(0x7f800000u)) && tid == 0 && blockIdx.x == 0 && blockIdx.y == 0)
        raise_status(a.status, PIPE_ERR_INVALID_ARG);
    }
    float yv[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) yv[i][j] = 0.f;

    for (int k = br.k_begin; k < br.k_end; ++k) {
      const OrderView ov = a.order[k];
      __syncthreads();
      if (tid < kRefC) {
        const int c = c0 + tid;
        int r = -1;
        if (c < a.O) {
          const int grp = c / a.g;
          const int lo = ov.cum[grp];
          if (ov.cum[grp + 1] > lo) r = lo * a.g + c % a.g;
        }
        crow[tid] = r;
      }
      __syncthreads();
      int acc[4][4];
      int rsum[4] = {0, 0, 0, 0};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0;

      for (int kb = 0; kb < a.I; kb += kRefKB) {
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          const int idx = tid + 256 * r;
          const int row = idx / kRefWords, w = idx % kRefWords;
          const int i = kb + 4 * w;
          uint32_t xv = 0, wv = 0;
          const int64_t t = t0 + row;
          if (t < a.T && i < a.I) {
            const int8_t* xr = br.xq + t * a.ldxq;
#pragma unroll
            for (int e = 0; e < 4; ++e)
              if (i + e < a.I) xv |= (static_cast<uint32_t>(static_cast<uint8_t>(xr[i + e]))) << (8 * e);
          }
          const int cr = crow[row];
          if (cr >= 0 && i < a.I)
            wv = canon_lanes(ov.codes + static_cast<int64_t>(cr) * a.canon_row_bytes, i, a.I, a.bits);
          xs[row][w] = xv;
          wsm[row][w] = wv;
        }
        __syncthreads();
#pragma unroll
        for (int w = 0; w < kRefWords; ++w) {
          int xa[4], wb[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) xa[i] = static_cast<int>(xs[4 * ty + i][w]);
#pragma unroll
          for (int j = 0; j < 4; ++j) wb[j] = static_cast<int>(wsm[4 * tx + j][w]);
#pragma unroll
          for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = __dp4a(xa[i], wb[j], acc[i][j]);
          if (zp != 0) {
#pragma unroll
            for (int j = 0; j < 4; ++j) rsum[j] = __dp4a(0x01010101, wb[j], rsum[j]);
          }
        }
        __syncthreads();
      }
      // order epilogue: scale product first, one FMA per term, ascending k
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int cr = crow[4 * tx + j];
        if (cr < 0) continue;
        const float cs = __fmul_rn(ov.scales[cr], sx);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int64_t t = t0 + 4 * ty + i;
          if (t >= a.T) continue;
          const int av = acc[i][j] - zp * rsum[j];
          yv[i][j] = __fmaf_rn(__int2float_rn(av), cs, yv[i][j]);
          if (a.partials) a.partials[t * a.total_rows + ov.row_off + cr] = av;
        }
      }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int c = c0 + 4 * tx + j;
      if (c >= a.O) continue;
      const float b = (br.add_bias && a.bias) ? a.bias[c] : 0.f;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int64_t t = t0 + 4 * ty + i;
        if (t >= a.T) continue;
        float v = yv[i][j];
        if (br.add_bias && a.bias) v = __fadd_rn(v, b);
        if (sum_mode) {
          total[i][j] = (m == 0) ? v : __fadd_rn(total[i][j], v);
          if (m + 1 == m_last) a.branch[0].y[t * a.ldy + c] = total[i][j];
        } else if (a.q8_out) {
          // inner layer of a branch: activation, then the next layer's input quantizer (division carried out)
          v = apply_activation(v, a.relu);
          br.yq[t * a.ldyq + c] = static_cast<int8_t>(quant_lane_exact(v, out_step));
        } else {
          br.y[t * a.ldy + c] = v;
        }
      }
    }
  }
}

pipe_status forward_reference(const ForwardArgs& a, cudaStream_t stream) {
  if (a.T == 0) return PIPE_OK;
  const int sum_mode = a.num_branches > 1 && a.branch[1].accumulate;
  const int64_t tb = ceil_div<int64_t>(a.T, kRefT);
  if (tb > 65535) {
    // split the token range so that gridDim.y stays legal
    ForwardArgs part = a;
    const int64_t step = 65535LL * kRefT;
    for (int64_t t = 0; t < a.T; t += step) {
      part.T = (a.T - t < step) ? a.T - t : step;
      for (int m = 0; m < a.num_branches; ++m) {
        part.branch[m].xq = a.branch[m].xq + t * a.ldxq;
        part.branch[m].y = a.branch[m].y ? a.branch[m].y + t * a.ldy : nullptr;
        part.branch[m].yq = a.branch[m].yq ? a.branch[m].yq + t * a.ldyq : nullptr;
      }
      part.partials = a.partials ? a.partials + t * a.total_rows : nullptr;
      pipe_status st = forward_reference(part, stream);
      if (st != PIPE_OK) return st;
    }
    return PIPE_OK;
  }
  dim3 grid(ceil_div(a.O, kRefC), static_cast<unsigned>(tb), sum_mode ? 1 : a.num_branches);
  ref_forward_kernel<<<grid, 256, 0, stream>>>(a, sum_mode);
  count_launch(1);
  return launch_status();
}

}  // namespace pipe
