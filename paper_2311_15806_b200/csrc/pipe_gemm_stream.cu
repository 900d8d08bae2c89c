// Small-token kernel of the expanded layer (Appendix B, Eq. 9; Sec. 3.2 for the branches), T <= 16.
//
// With a handful of tokens the layer is bound by streaming the packed weight codes from HBM once.
// The kernel therefore moves weights global -> registers with coalesced 16-byte loads (the loads of
// the next batch are always in flight while the current batch is consumed), unpacks them in
// registers with the shift-and-mask layout and feeds legacy warp-level integer MMAs
// (mma.sync m16n8k32, weights as the 16-row operand, tokens as the 8-column operand): the tensor
// pipe is nowhere near a limit here, the byte stream is.
//
// Work unit: a "slab" = 8 consecutive output channels of one branch.  In every order of the branch
// that keeps the slab's group, the slab is 8 consecutive compacted rows.  Two such 8-row chunks
// (two orders, ascending) form one 16-row MMA tile, so both orders of a pair accumulate in the same
// thread and the fixed-order fp32 epilogue is thread-local.  A persistent CTA walks groups of 4
// slabs: 16 streaming warps (4 per slab, each owning a range of the reduction axis) drop their exact
// int32 partial sums into a double-buffered shared-memory area; 4 epilogue warps (one per slab)
// add the four ranges, apply the scales in ascending order and store, while the streaming warps
// are already on the next group.  The quantized activations (at most 16 rows) are read as MMA
// fragments straight from global memory: they stay resident in L1.  All slab metadata and scale
// products of the CTA are gathered once, up front, with independent loads.
#include "pipe_common.cuh"

namespace pipe {

namespace st {

constexpr int kStreamWarps = 16;
constexpr int kEpiWarps = 4;
constexpr int kThreads = 32 * (kStreamWarps + kEpiWarps);
constexpr int kSlabsPerGroup = 4;
constexpr int kSlices = 4;        // streaming warps per slab
constexpr int kMaxPairs = 4;      // up to 8 orders per branch
constexpr int kBatch = 4;         // macro steps whose loads are issued together
constexpr int kMaxGroups = 128;   // groups one CTA may own (metadata table size)
constexpr int kMetaInts = 2 + 4 * kMaxPairs;   // nchunks, branch, then (order, row0) per chunk
constexpr long long kWaitLimitCycles = 4000000000ll;

struct Params {
  ForwardArgs f;
  int nms;           // macro steps: ceil(I_pad / (4 * codes per 16-byte chunk))
  int kblocks;       // I_pad / 128
  int pk;            // packed bytes of one row of one 128-code block
  int shift;         // 8 - b
  int slabs_per_branch;   // padded to a multiple of kSlabsPerGroup
  int groups;
  int xs_bytes;
  int np;            // pairs of orders per slab the partial-sum buffers are sized for
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait; false when the CTA is aborting (this wait or another one ran out).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status) {
  if (mbar_try(bar, parity)) return true;
  const long long t0 = clock64();
  while (true) {
#pragma unroll 1
    for (int i = 0; i < 16; ++i)
      if (mbar_try(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > kWaitLimitCycles) {
      *abort_flag = 1;
      raise_status(status, PIPE_ERR_TIMEOUT);
      return false;
    }
  }
}

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

// One batch of a streaming warp: kBatch macro steps of one pair of one slab.
struct Batch {
  int gi;        // index into the CTA's own group list (-1: none)
  int q;         // pair
  int ms0;       // first macro step
};

template <int BITS, int NT>
__global__ void __launch_bounds__(kThreads, 1) stream_forward_kernel(const Params p) {
  constexpr int CHK = 128 / BITS;        // codes per 16-byte chunk
  constexpr int NMMA = CHK / 8;          // MMAs per macro step
  const int RED_INTS = kSlabsPerGroup * kSlices * p.np * 32 * 4 * NT;   // one buffer of partial sums
  extern __shared__ uint4 smem_u4[];
  int* red = reinterpret_cast<int*>(smem_u4);                    // [2][slab][slice][pair][lane][4*NT]
  int* meta = red + 2 * RED_INTS;                                // [own slabs][kMetaInts]
  const int my_groups_ = (p.groups - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
  float* cstab = reinterpret_cast<float*>(meta + my_groups_ * kSlabsPerGroup * kMetaInts);   // [own slabs][2*np][8] s_k * lambda_x
  float* biastab = cstab + my_groups_ * kSlabsPerGroup * 2 * p.np * 8;                        // [own slabs][8]
  __shared__ uint64_t bars[4];   // full[2] empty[2]
  __shared__ int abort_flag_s;
  volatile int* abort_flag = &abort_flag_s;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gid = lane >> 2, tig = lane & 3;
  const int I = p.f.I;
  const int my_groups = (p.groups - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
  const uint32_t bar0 = smem_u32(bars);
  const uint32_t full0 = bar0, empty0 = bar0 + 16;

  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    for (int b = 0; b < 2; ++b) {
      mbar_init(full0 + 8u * b, kStreamWarps);
      mbar_init(empty0 + 8u * b, kEpiWarps);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // ---- metadata of every slab this CTA owns: which orders keep its group, where its 8 rows start
  for (int e = threadIdx.x; e < my_groups * kSlabsPerGroup; e += kThreads) {
    const int gi = e / kSlabsPerGroup, sl = e % kSlabsPerGroup;
    const int grp = blockIdx.x + gi * gridDim.x;
    const int slab = grp * kSlabsPerGroup + sl;
    const int branch = slab / p.slabs_per_branch;
    const int c0 = (slab - branch * p.slabs_per_branch) * 8;
    int* m = meta + e * kMetaInts;
    int nchunks = 0;
    if (c0 < p.f.O) {
      const BranchArgs& br = p.f.branch[branch];
      const int j = c0 / p.f.g;
      for (int k = br.k_begin; k < br.k_end; ++k) {
        const int32_t* cum = p.f.order[k].cum;
        const int lo = __ldg(cum + j), hi = __ldg(cum + j + 1);
        if (hi > lo) {
          m[2 + 2 * nchunks] = k;
          m[3 + 2 * nchunks] = lo * p.f.g + c0 % p.f.g;
          ++nchunks;
        }
      }
    }
    m[0] = c0 < p.f.O ? nchunks : -1;   // -1: padding slab, nothing to store
    m[1] = branch;
  }
  __syncthreads();
  // ---- scale products s_k * lambda_x of every row this CTA will finish, and its bias values
  for (int e = threadIdx.x; e < my_groups * kSlabsPerGroup * 2 * p.np * 8; e += kThreads) {
    const int r = e & 7, ci = (e >> 3) % (2 * p.np), slab_i = (e >> 3) / (2 * p.np);
    const int* m = meta + slab_i * kMetaInts;
    float v = 0.f;
    if (ci < m[0]) {
      const BranchArgs& br = p.f.branch[m[1]];
      v = __fmul_rn(__ldg(p.f.order[m[2 + 2 * ci]].scales + m[3 + 2 * ci] + r), __ldg(br.sx));
    }
    cstab[e] = v;
  }
  for (int e = threadIdx.x; e < my_groups * kSlabsPerGroup * 8; e += kThreads) {
    const int r = e & 7, slab_i = e >> 3;
    const int* m = meta + slab_i * kMetaInts;
    float v = 0.f;
    if (m[0] >= 0 && p.f.bias && p.f.branch[m[1]].add_bias) {
      const int gi = slab_i / kSlabsPerGroup, sl = slab_i % kSlabsPerGroup;
      const int slab = (blockIdx.x + gi * gridDim.x) * kSlabsPerGroup + sl;
      v = __ldg(p.f.bias + (slab - m[1] * p.slabs_per_branch) * 8 + r);
    }
    biastab[e] = v;
  }
  __syncthreads();

  if (warp < kStreamWarps) {
    // ================================================================== streaming warps
    const int sl = warp / kSlices, slice = warp % kSlices;
    const int per = (p.nms + kSlices - 1) / kSlices;
    const int ms_begin = min(slice * per, p.nms), ms_end = min(ms_begin + per, p.nms);
    const bool has_range = ms_begin < ms_end;

    auto pairs_of = [&](int gi) {
      const int nch = meta[(gi * kSlabsPerGroup + sl) * kMetaInts];
      return nch > 0 ? (nch + 1) >> 1 : 0;
    };
    // first batch at or after (gi, q = 0)
    auto first_batch = [&](int gi) {
      Batch b{-1, 0, 0};
      if (!has_range) return b;
      while (gi < my_groups && pairs_of(gi) == 0) ++gi;
      if (gi < my_groups) b = Batch{gi, 0, ms_begin};
      return b;
    };
    auto next_batch = [&](const Batch& c) {
      if (c.ms0 + kBatch < ms_end) return Batch{c.gi, c.q, c.ms0 + kBatch};
      if (c.q + 1 < pairs_of(c.gi)) return Batch{c.gi, c.q + 1, ms_begin};
      return first_batch(c.gi + 1);
    };
    auto issue = [&](const Batch& b, uint4 (&wa)[kBatch], uint4 (&wb)[kBatch]) {
      if (b.gi < 0) return;
      const int* m = meta + (b.gi * kSlabsPerGroup + sl) * kMetaInts;
      const int nch = m[0];
      const int k_a = m[2 + 4 * b.q], row_a = m[3 + 4 * b.q];
      const bool has_b = 2 * b.q + 1 < nch;
      const int k_b = has_b ? m[4 + 4 * b.q] : k_a;
      const int row_b = has_b ? m[5 + 4 * b.q] : row_a;
      const uint8_t* base_a = p.f.order[k_a].kcodes + static_cast<size_t>(row_a + gid) * p.pk;
      const uint8_t* base_b = p.f.order[k_b].kcodes + static_cast<size_t>(row_b + gid) * p.pk;
      const size_t blk_a = static_cast<size_t>(p.f.order[k_a].rows) * p.pk;
      const size_t blk_b = static_cast<size_t>(p.f.order[k_b].rows) * p.pk;
#pragma unroll
      for (int s = 0; s < kBatch; ++s) {
        const int ms = b.ms0 + s;
        wa[s] = make_uint4(0, 0, 0, 0);
        wb[s] = make_uint4(0, 0, 0, 0);
        // this thread's chunk starts at reduction offset ms*4*CHK + tig*CHK
        const int kcode = ms * 4 * CHK + tig * CHK;
        const int kb = kcode >> 7;
        if (ms < ms_end && kb < p.kblocks) {
          const int inblk = ((kcode & 127) * BITS) >> 3;
          wa[s] = __ldg(reinterpret_cast<const uint4*>(base_a + kb * blk_a + inblk));
          if (has_b) wb[s] = __ldg(reinterpret_cast<const uint4*>(base_b + kb * blk_b + inblk));
        }
      }
    };

    uint4 na[kBatch], nb[kBatch];
    Batch nxt = first_batch(0);
    issue(nxt, na, nb);

    for (int gi = 0; gi < my_groups; ++gi) {
      const int* m = meta + (gi * kSlabsPerGroup + sl) * kMetaInts;
      const int branch = meta[(gi * kSlabsPerGroup) * kMetaInts + 1];   // the group's branch (slab 0 of the group)
      const BranchArgs& br = p.f.branch[branch];
      // this thread's activation rows (token gid of each 8-token tile); aligned rows take 16-byte loads
      const int8_t* xrow[NT];
      bool xok[NT];
#pragma unroll
      for (int t = 0; t < NT; ++t) {
        xok[t] = gid + 8 * t < p.f.T;
        xrow[t] = br.xq + static_cast<int64_t>(xok[t] ? gid + 8 * t : 0) * p.f.ldxq;
      }
      const int nch = m[0];
      const int npairs = nch > 0 ? (nch + 1) >> 1 : 0;
      const int buf = gi & 1;
      // the epilogue warps must have drained this buffer (group gi - 2)
      if (!mbar_wait(empty0 + 8u * buf, ((gi >> 1) & 1) ^ 1, abort_flag, p.f.status)) break;
      int* dst_base = red + buf * RED_INTS + ((sl * kSlices + slice) * p.np * 32 + lane) * (4 * NT);
      for (int q = 0; q < npairs; ++q) {
        int acc[NT][4];
#pragma unroll
        for (int t = 0; t < NT; ++t)
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[t][e] = 0;
        if (has_range) {
          for (int ms0 = ms_begin; ms0 < ms_end; ms0 += kBatch) {
            // the loads of this batch were issued one batch ago; issue the next batch now
            uint4 wa[kBatch], wb[kBatch];
#pragma unroll
            for (int s = 0; s < kBatch; ++s) {
              wa[s] = na[s];
              wb[s] = nb[s];
            }
            nxt = next_batch(Batch{gi, q, ms0});
            issue(nxt, na, nb);
#pragma unroll
            for (int s = 0; s < kBatch; ++s) {
              const int ms = ms0 + s;
              if (ms >= ms_end) break;
              uint32_t ra[16], rb[16];
              unpack_chunk<BITS>(wa[s], ra);
              unpack_chunk<BITS>(wb[s], rb);
              // B fragments: CHK consecutive activation codes of this thread's token, from
              // reduction offset ms*4*CHK + tig*CHK (register 2m covers 8m..8m+3, 2m+1 covers 8m+4..8m+7)
              const int kx = ms * 4 * CHK + tig * CHK;
#pragma unroll
              for (int t = 0; t < NT; ++t) {
                uint32_t xb[2 * NMMA];
#pragma unroll
                for (int v = 0; v < NMMA / 2; ++v) {
                  uint4 xv = make_uint4(0, 0, 0, 0);
                  if (xok[t]) {
                    const int k16 = kx + 16 * v;
                    if (k16 < I) xv = __ldg(reinterpret_cast<const uint4*>(xrow[t] + k16));   // I % 16 == 0 (host check)
                  }
                  xb[4 * v] = xv.x; xb[4 * v + 1] = xv.y; xb[4 * v + 2] = xv.z; xb[4 * v + 3] = xv.w;
                }
#pragma unroll
                for (int mm = 0; mm < NMMA; ++mm)
                  // tile rows 0-7: first order of the pair, rows 8-15: second order
                  mma_s8(acc[t], ra[2 * mm], rb[2 * mm], ra[2 * mm + 1], rb[2 * mm + 1], xb[2 * mm], xb[2 * mm + 1]);
              }
            }
          }
        }
        int* dst = dst_base + q * 32 * (4 * NT);
#pragma unroll
        for (int t = 0; t < NT; ++t)
#pragma unroll
          for (int e = 0; e < 4; ++e) dst[t * 4 + e] = acc[t][e];
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(full0 + 8u * buf);
    }
  } else {
    // ================================================================== epilogue warps (one per slab)
    const int sl = warp - kStreamWarps;
    for (int gi = 0; gi < my_groups; ++gi) {
      const int* m = meta + (gi * kSlabsPerGroup + sl) * kMetaInts;
      const int nch = m[0];
      const int branch = m[1];
      const int npairs = nch > 0 ? (nch + 1) >> 1 : 0;
      const int buf = gi & 1;
      const int grp = blockIdx.x + gi * gridDim.x;
      const int slab = grp * kSlabsPerGroup + sl;
      const int c = (slab - branch * p.slabs_per_branch) * 8 + gid;   // this thread's output channel
      const float* cs_slab = cstab + (gi * kSlabsPerGroup + sl) * 2 * p.np * 8;
      const float bv = biastab[(gi * kSlabsPerGroup + sl) * 8 + gid];
      const bool bias = nch >= 0 && p.f.bias && p.f.branch[branch].add_bias;
      if (!mbar_wait(full0 + 8u * buf, (gi >> 1) & 1, abort_flag, p.f.status)) break;
      if (nch >= 0) {
        const BranchArgs& br = p.f.branch[branch];
        float y[NT][2];
#pragma unroll
        for (int t = 0; t < NT; ++t) y[t][0] = y[t][1] = 0.f;
#pragma unroll
        for (int q = 0; q < kMaxPairs; ++q) {
          if (q >= npairs) break;
          int acc[NT][4];
#pragma unroll
          for (int t = 0; t < NT; ++t)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[t][e] = 0;
#pragma unroll
          for (int s = 0; s < kSlices; ++s) {
            const int* src = red + buf * RED_INTS + (((sl * kSlices + s) * p.np + q) * 32 + lane) * (4 * NT);
#pragma unroll
            for (int t = 0; t < NT; ++t)
#pragma unroll
              for (int e = 0; e < 4; ++e) acc[t][e] += src[t * 4 + e];
          }
          // accumulator registers 0,1: tile row gid (first order of the pair); 2,3: tile row gid + 8
          // (second order); columns 2*tig, 2*tig + 1 of token tile t.  Ascending order.
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            const int ci = 2 * q + half;
            if (ci >= nch) break;
            const float cs = cs_slab[ci * 8 + gid];
            const int row = m[3 + 2 * ci] + gid, roff = p.f.order[m[2 + 2 * ci]].row_off;
#pragma unroll
            for (int t = 0; t < NT; ++t)
#pragma unroll
              for (int e = 0; e < 2; ++e) {
                const int a = acc[t][2 * half + e] >> p.shift;   // exact: the sum carries a factor 2^shift
                y[t][e] = __fmaf_rn(__int2float_rn(a), cs, y[t][e]);
                const int tok = 8 * t + 2 * tig + e;
                if (p.f.partials && tok < p.f.T)
                  p.f.partials[static_cast<int64_t>(tok) * p.f.total_rows + roff + row] = a;
              }
          }
        }
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
      __syncwarp();
      if (lane == 0) mbar_arrive(empty0 + 8u * buf);
    }
  }
}

}  // namespace st

static pipe_status launch_stream(const ForwardArgs& a, cudaStream_t stream) {
  using namespace st;
  if (a.T > 16 || a.g % 8 != 0) return PIPE_ERR_UNSUPPORTED;
  // activation fragments are fetched with 16-byte loads
  if (a.I % 16 != 0 || a.ldxq % 16 != 0) return PIPE_ERR_UNSUPPORTED;
  for (int m = 0; m < a.num_branches; ++m)
    if (reinterpret_cast<uintptr_t>(a.branch[m].xq) & 15) return PIPE_ERR_UNSUPPORTED;
  int max_cluster = 0;
  for (int m = 0; m < a.num_branches; ++m) max_cluster = max(max_cluster, a.branch[m].k_end - a.branch[m].k_begin);
  if (max_cluster > 2 * kMaxPairs) return PIPE_ERR_UNSUPPORTED;
  Params p;
  p.f = a;
  const int nt = a.T <= 8 ? 1 : 2;
  const int chk = 128 / a.bits;
  p.kblocks = ceil_div(a.I, 128);
  p.nms = ceil_div(p.kblocks * 128, 4 * chk);
  p.pk = 128 * a.bits / 8;
  p.shift = 8 - a.bits;
  // groups of slabs must not straddle branches: pad every branch to a multiple of the group size
  p.slabs_per_branch = round_up(a.O / 8, kSlabsPerGroup);
  p.groups = p.slabs_per_branch * a.num_branches / kSlabsPerGroup;
  p.xs_bytes = 0;
  int dev = 0, smem_max = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return PIPE_ERR_CUDA;
  cudaDeviceGetAttribute(&smem_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int grid = p.groups < sms ? p.groups : sms;
  const int own = ceil_div(p.groups, grid);
  if (own > kMaxGroups) return PIPE_ERR_UNSUPPORTED;
  p.np = (max_cluster + 1) / 2;
  const int red_bytes = 2 * kSlabsPerGroup * kSlices * p.np * 32 * 4 * nt * 4;
  const int meta_bytes = own * kSlabsPerGroup * (kMetaInts + 2 * p.np * 8 + 8) * 4;
  const int dyn = red_bytes + meta_bytes;
  if (dyn + 1024 > smem_max) return PIPE_ERR_UNSUPPORTED;

  void (*kern)(const Params) = nullptr;
  if (a.bits == 8) kern = nt == 1 ? stream_forward_kernel<8, 1> : stream_forward_kernel<8, 2>;
  else if (a.bits == 4) kern = nt == 1 ? stream_forward_kernel<4, 1> : stream_forward_kernel<4, 2>;
  else kern = nt == 1 ? stream_forward_kernel<2, 1> : stream_forward_kernel<2, 2>;
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
