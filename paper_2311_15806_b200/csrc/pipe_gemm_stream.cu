// Small-token kernel of the expanded layer (Appendix B, Eq. 9; Sec. 3.2 for the branches), T <= 16.
//
// With a handful of tokens the layer is bound by streaming the packed weight codes from HBM once.
// The kernel therefore moves weights global -> registers with coalesced 16-byte loads (many in
// flight per warp), unpacks them in registers with the shift-and-mask layout and feeds legacy
// warp-level integer MMAs (mma.sync m16n8k32, weights as the 16-row operand, tokens as the
// 8-column operand): the tensor pipe is nowhere near a limit here, the byte stream is.
//
// Work unit: a "slab" = 8 consecutive output channels of one branch.  In every order of the branch
// that keeps the slab's group, the slab is 8 consecutive compacted rows.  Two such 8-row chunks
// (two orders, ascending) form one 16-row MMA tile, so both orders of a pair accumulate in the same
// thread and the fixed-order fp32 epilogue is thread-local.  A CTA of 16 warps works on 4 slabs at a
// time; the 4 warps of a slab split the reduction axis and add their exact int32 partial sums
// through shared memory.  The quantized activations sit in shared memory in MMA-fragment order.
#include "pipe_common.cuh"

namespace pipe {

namespace st {

constexpr int kThreads = 512;
constexpr int kSlabsPerCta = 4;
constexpr int kSlices = 4;        // warps per slab, each owns a contiguous range of macro steps
constexpr int kMaxPairs = 4;      // up to 8 orders per branch
constexpr int kBatch = 8;         // macro steps whose loads are issued together

struct Params {
  ForwardArgs f;
  int nt;            // 8-token MMA column tiles: 1 (T <= 8) or 2
  int chk;           // codes per 16-byte chunk: 16 (int8), 32 (int4), 64 (ternary)
  int nmma;          // MMAs per macro step = chk / 8
  int nms;           // macro steps: ceil(I_pad / (4 * chk))
  int kblocks;       // I_pad / 128
  int pk;            // packed bytes of one row of one 128-code block
  int shift;         // 8 - b
  int slabs_per_branch, total_slabs;
  int xs_bytes, red_bytes;
};

__device__ __forceinline__ void mma_s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                       uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// int8 lanes (times 2^(8-b)) of the codes held by 16 packed bytes: reg[2m] covers reduction
// offsets 8m..8m+3 of the chunk, reg[2m+1] covers 8m+4..8m+7 (see the streaming layout).
template <int BITS>
__device__ __forceinline__ void unpack_chunk(const uint4& w, uint32_t (&reg)[16]) {
  const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
  if (BITS == 8) {
#pragma unroll
    for (int j = 0; j < 4; ++j) reg[j] = ww[j];
  } else if (BITS == 4) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      reg[2 * j] = (ww[j] << 4) & 0xF0F0F0F0u;
      reg[2 * j + 1] = ww[j] & 0xF0F0F0F0u;
    }
  } else {
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int h = 0; h < 4; ++h) reg[4 * j + h] = (ww[j] << (6 - 2 * h)) & 0xC0C0C0C0u;
  }
}

template <int BITS, int NT>
__global__ void __launch_bounds__(kThreads, 1) stream_forward_kernel(const Params p) {
  constexpr int CHK = 128 / BITS;        // codes per 16-byte chunk
  constexpr int NMMA = CHK / 8;          // MMAs per macro step
  extern __shared__ uint4 smem_u4[];
  uint2* xs = reinterpret_cast<uint2*>(smem_u4);                                  // [nms][NMMA][NT][32] 8-byte fragments
  int* red = reinterpret_cast<int*>(reinterpret_cast<uint8_t*>(smem_u4) + p.xs_bytes);  // [slab][slice-1][pair][lane][4*NT]
  __shared__ int slab_meta[kSlabsPerCta][2 + 2 * kMaxPairs * 2];  // per slab: branch, npairs, then (order, row0) per chunk

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gid = lane >> 2, tig = lane & 3;
  const int slab_local = warp / kSlices, slice = warp % kSlices;
  const int I = p.f.I;
  int cur_branch_loaded = -1;

  const int groups = (p.total_slabs + kSlabsPerCta - 1) / kSlabsPerCta;
  for (int grp = blockIdx.x; grp < groups; grp += gridDim.x) {
    const int slab = grp * kSlabsPerCta + slab_local;
    // slabs_per_branch is padded to a multiple of 4, so a group never straddles two branches; the
    // padding slabs (channels beyond O) do nothing.
    const int branch = (grp * kSlabsPerCta) / p.slabs_per_branch;
    const bool slab_ok = (slab - branch * p.slabs_per_branch) * 8 < p.f.O;
    const BranchArgs& br = p.f.branch[branch];

    // ---- stage the activations of this branch in fragment order (once per branch change)
    if (branch != cur_branch_loaded) {
      __syncthreads();
      const int units = p.nms * NMMA * NT * 32;
      for (int u = threadIdx.x; u < units; u += kThreads) {
        const int l = u & 31;
        const int nt = (u >> 5) % NT;
        const int m = ((u >> 5) / NT) % NMMA;
        const int ms = (u >> 5) / NT / NMMA;
        const int n = (l >> 2) + 8 * nt;
        const int k0 = ms * 4 * CHK + (l & 3) * CHK + 8 * m;
        uint32_t lo = 0, hi = 0;
        if (n < p.f.T) {
          const int8_t* xr = br.xq + static_cast<int64_t>(n) * p.f.ldxq;
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            if (k0 + e < I) lo |= static_cast<uint32_t>(static_cast<uint8_t>(xr[k0 + e])) << (8 * e);
            if (k0 + 4 + e < I) hi |= static_cast<uint32_t>(static_cast<uint8_t>(xr[k0 + 4 + e])) << (8 * e);
          }
        }
        xs[u] = make_uint2(lo, hi);
      }
      cur_branch_loaded = branch;
    }
    // ---- slab metadata: which orders keep this slab's group, and where its 8 rows start
    if (slice == 0 && lane == 0) {
      int nchunks = 0;
      if (slab_ok) {
        const int c0 = (slab - branch * p.slabs_per_branch) * 8;
        const int j = c0 / p.f.g;
        for (int k = br.k_begin; k < br.k_end; ++k) {
          const int32_t* cum = p.f.order[k].cum;
          const int lo = __ldg(cum + j), hi = __ldg(cum + j + 1);
          if (hi > lo) {
            slab_meta[slab_local][2 + 2 * nchunks] = k;
            slab_meta[slab_local][3 + 2 * nchunks] = lo * p.f.g + c0 % p.f.g;
            ++nchunks;
          }
        }
      }
      slab_meta[slab_local][0] = branch;
      slab_meta[slab_local][1] = nchunks;
    }
    __syncthreads();
    const int nchunks = slab_meta[slab_local][1];
    const int npairs = (nchunks + 1) >> 1;

    int acc[kMaxPairs][NT][4];
#pragma unroll
    for (int q = 0; q < kMaxPairs; ++q)
#pragma unroll
      for (int t = 0; t < NT; ++t)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[q][t][e] = 0;

    // macro steps of this warp's slice
    const int per = (p.nms + kSlices - 1) / kSlices;
    const int ms_begin = min(slice * per, p.nms), ms_end = min(ms_begin + per, p.nms);

#pragma unroll
    for (int q = 0; q < kMaxPairs; ++q) {
      if (q >= npairs) break;
      const int k_a = slab_meta[slab_local][2 + 4 * q], row_a = slab_meta[slab_local][3 + 4 * q];
      const bool has_b = 2 * q + 1 < nchunks;
      const int k_b = has_b ? slab_meta[slab_local][4 + 4 * q] : k_a;
      const int row_b = has_b ? slab_meta[slab_local][5 + 4 * q] : row_a;
      const OrderView& oa = p.f.order[k_a];
      const OrderView& ob = p.f.order[k_b];
      for (int ms0 = ms_begin; ms0 < ms_end; ms0 += kBatch) {
        uint4 wa[kBatch], wb[kBatch];
#pragma unroll
        for (int s = 0; s < kBatch; ++s) {
          const int ms = ms0 + s;
          wa[s] = make_uint4(0, 0, 0, 0);
          wb[s] = make_uint4(0, 0, 0, 0);
          if (ms < ms_end) {
            // byte position of this thread's chunk: reduction offset ms*4*CHK + tig*CHK
            const int kcode = ms * 4 * CHK + tig * CHK;
            const int kb = kcode >> 7;
            if (kb < p.kblocks) {
              const int inblk = ((kcode & 127) * BITS) >> 3;
              const size_t oa_off = (static_cast<size_t>(kb) * oa.rows + row_a + gid) * p.pk + inblk;
              wa[s] = __ldg(reinterpret_cast<const uint4*>(oa.kcodes + oa_off));
              if (has_b) {
                const size_t ob_off = (static_cast<size_t>(kb) * ob.rows + row_b + gid) * p.pk + inblk;
                wb[s] = __ldg(reinterpret_cast<const uint4*>(ob.kcodes + ob_off));
              }
            }
          }
        }
#pragma unroll
        for (int s = 0; s < kBatch; ++s) {
          const int ms = ms0 + s;
          if (ms >= ms_end) break;
          uint32_t ra[16], rb[16];
          unpack_chunk<BITS>(wa[s], ra);
          unpack_chunk<BITS>(wb[s], rb);
          const uint2* xf = xs + static_cast<size_t>(ms) * NMMA * NT * 32 + lane;
#pragma unroll
          for (int m = 0; m < NMMA; ++m)
#pragma unroll
            for (int t = 0; t < NT; ++t) {
              const uint2 b = xf[(m * NT + t) * 32];
              // tile rows 0-7: order k_a, rows 8-15: order k_b
              mma_s8(acc[q][t], ra[2 * m], rb[2 * m], ra[2 * m + 1], rb[2 * m + 1], b.x, b.y);
            }
        }
      }
    }

    // ---- add the slices' exact partial sums; slice 0 keeps the total
    if (slice != 0) {
#pragma unroll
      for (int q = 0; q < kMaxPairs; ++q) {
        if (q >= npairs) break;
        int* dst = red + ((((slab_local * (kSlices - 1) + slice - 1) * kMaxPairs + q) * 32 + lane) * (4 * NT));
#pragma unroll
        for (int t = 0; t < NT; ++t)
#pragma unroll
          for (int e = 0; e < 4; ++e) dst[t * 4 + e] = acc[q][t][e];
      }
    }
    __syncthreads();
    if (slice == 0 && slab_ok) {
      const float sx = __ldg(br.sx);
      const int c = (slab - branch * p.slabs_per_branch) * 8 + gid;   // this thread's output channel
      float y[NT][2];
#pragma unroll
      for (int t = 0; t < NT; ++t) y[t][0] = y[t][1] = 0.f;
#pragma unroll
      for (int q = 0; q < kMaxPairs; ++q) {
        if (q >= npairs) break;
#pragma unroll
        for (int sl = 1; sl < kSlices; ++sl) {
          const int* src = red + ((((slab_local * (kSlices - 1) + sl - 1) * kMaxPairs + q) * 32 + lane) * (4 * NT));
#pragma unroll
          for (int t = 0; t < NT; ++t)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[q][t][e] += src[t * 4 + e];
        }
        // accumulator registers 0,1: tile row gid (order k_a); 2,3: tile row gid + 8 (order k_b);
        // columns 2*tig, 2*tig + 1 of token tile t.  Ascending order: k_a first, then k_b.
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          if (2 * q + half >= nchunks) break;
          const int k = slab_meta[slab_local][2 + 2 * (2 * q + half)];
          const int row = slab_meta[slab_local][3 + 2 * (2 * q + half)] + gid;
          const OrderView& ov = p.f.order[k];
          const float cs = __fmul_rn(__ldg(ov.scales + row), sx);
#pragma unroll
          for (int t = 0; t < NT; ++t)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              const int a = acc[q][t][2 * half + e] >> p.shift;   // exact: the sum carries a factor 2^shift
              y[t][e] = __fmaf_rn(__int2float_rn(a), cs, y[t][e]);
              const int tok = 8 * t + 2 * tig + e;
              if (p.f.partials && tok < p.f.T) p.f.partials[static_cast<int64_t>(tok) * p.f.total_rows + ov.row_off + row] = a;
            }
        }
      }
      const bool bias = br.add_bias && p.f.bias;
      const float bv = bias ? __ldg(p.f.bias + c) : 0.f;
#pragma unroll
      for (int t = 0; t < NT; ++t)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int tok = 8 * t + 2 * tig + e;
          if (tok >= p.f.T) continue;
          float v = y[t][e];
          if (bias) v = __fadd_rn(v, bv);
          float* dst = br.y + static_cast<int64_t>(tok) * p.f.ldy + c;
          if (br.accumulate) v = __fadd_rn(*dst, v);
          *dst = v;
        }
    }
    __syncthreads();   // red[] and slab_meta[] are reused by the next group
  }
}

}  // namespace st

static pipe_status launch_stream(const ForwardArgs& a, cudaStream_t stream) {
  using namespace st;
  if (a.T > 16 || a.g % 8 != 0) return PIPE_ERR_UNSUPPORTED;
  int max_cluster = 0;
  for (int m = 0; m < a.num_branches; ++m) max_cluster = max(max_cluster, a.branch[m].k_end - a.branch[m].k_begin);
  if (max_cluster > 2 * kMaxPairs) return PIPE_ERR_UNSUPPORTED;
  Params p;
  p.f = a;
  p.nt = a.T <= 8 ? 1 : 2;
  p.chk = 128 / a.bits;
  p.nmma = p.chk / 8;
  p.kblocks = ceil_div(a.I, 128);
  p.nms = ceil_div(p.kblocks * 128, 4 * p.chk);
  p.pk = 128 * a.bits / 8;
  p.shift = 8 - a.bits;
  // groups of 4 slabs must not straddle branches: pad every branch to a multiple of 4 slabs
  p.slabs_per_branch = round_up(a.O / 8, kSlabsPerCta);
  p.total_slabs = p.slabs_per_branch * a.num_branches;
  p.xs_bytes = round_up(p.nms * p.nmma * p.nt * 32 * 8, 16);
  p.red_bytes = kSlabsPerCta * (kSlices - 1) * kMaxPairs * 32 * 4 * p.nt * 4;
  const int dyn = p.xs_bytes + p.red_bytes;
  int dev = 0, smem_max = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return PIPE_ERR_CUDA;
  cudaDeviceGetAttribute(&smem_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (dyn + 2048 > smem_max) return PIPE_ERR_UNSUPPORTED;
  const int groups = p.total_slabs / kSlabsPerCta;
  const int grid = groups < sms ? groups : sms;

  void (*kern)(const Params) = nullptr;
  if (a.bits == 8) kern = p.nt == 1 ? stream_forward_kernel<8, 1> : stream_forward_kernel<8, 2>;
  else if (a.bits == 4) kern = p.nt == 1 ? stream_forward_kernel<4, 1> : stream_forward_kernel<4, 2>;
  else kern = p.nt == 1 ? stream_forward_kernel<2, 1> : stream_forward_kernel<2, 2>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn) != cudaSuccess) return PIPE_ERR_CUDA;
  kern<<<grid, kThreads, dyn, stream>>>(p);
  count_launch(1);
  return launch_status();
}

pipe_status forward_stream(const ForwardArgs& a, cudaStream_t stream) {
  if (a.T == 0) return PIPE_OK;
  const bool sum_mode = a.num_branches > 1 && a.branch[1].accumulate;
  if (!sum_mode) return launch_stream(a, stream);
  for (int m = 0; m < a.num_branches; ++m) {
    ForwardArgs one = a;
    one.num_branches = 1;
    one.branch[0] = a.branch[m];
    pipe_status st = launch_stream(one, stream);
    if (st != PIPE_OK) return st;
  }
  return PIPE_OK;
}

}  // namespace pipe
