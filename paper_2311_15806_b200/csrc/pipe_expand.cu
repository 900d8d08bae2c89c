// pipe_expand_weights: residual expansion of a weight matrix (Sec. 3.1, Eq. 2-3 and the masked
// form), with the per-channel symmetric quantizer of Eq. 1.
//
// Per order: [group select, orders >= 2] -> one fused pass over the kept rows that (order 1: finds the
// row maximum,) divides, rounds, packs both code layouts, updates the residual with one FMA per
// element and leaves the next order's row absmax behind.  All kernels are
// HBM-bound streaming passes: 128-bit loads, warp-shuffle reductions, one block per row.
#include <cstring>
#include <mutex>

#include "pipe_common.cuh"

namespace pipe {

constexpr int kRowThreads = 256;

__device__ __forceinline__ uint32_t warp_max_u32(uint32_t v) {
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, d));
  return v;
}

// Max over the block of an unsigned value; result valid in every thread.
__device__ __forceinline__ uint32_t block_max_u32(uint32_t v) {
  __shared__ uint32_t part[32];
  __shared__ uint32_t total;
  v = warp_max_u32(v);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) part[warp] = v;
  __syncthreads();
  if (warp == 0) {
    uint32_t w = lane < (blockDim.x + 31) / 32 ? part[lane] : 0u;
    w = warp_max_u32(w);
    if (lane == 0) total = w;
  }
  __syncthreads();
  const uint32_t r = total;
  __syncthreads();
  return r;
}

// |v| as an ordered unsigned key: for finite floats the order of the keys is the order of the
// magnitudes, and every Inf/NaN maps to a key >= 0x7f800000.
__device__ __forceinline__ uint32_t abs_key(float v) { return __float_as_uint(v) & 0x7fffffffu; }

// score[j] = max over the g rows of group j of a[] ; one thread per group.
__global__ void group_score_kernel(const float* __restrict__ a, int G, int g, float* __restrict__ score) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= G) return;
  float m = 0.f;
  for (int u = 0; u < g; ++u) m = fmaxf(m, a[static_cast<int64_t>(j) * g + u]);
  score[j] = m;
}

// keep[j] = 1 iff fewer than n_keep groups precede j in the order (score descending, index
// ascending).  Scores are non-negative finite floats, so the comparison is exact and the
// result does not depend on any reduction order.
template <typename S>
__global__ void group_rank_kernel(const S* __restrict__ score, int G, int n_keep, int32_t* __restrict__ keep) {
  // one warp per group: its lanes share the G comparisons (a count, so the order of the additions does not matter)
  const int j = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (j >= G) return;
  const S sj = score[j];
  int rank = 0;
  for (int t = lane; t < G; t += 32) {
    const S si = score[t];
    rank += (si > sj) || (si == sj && t < j);
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) rank += __shfl_xor_sync(0xffffffffu, rank, d);
  if (lane == 0) keep[j] = rank < n_keep ? 1 : 0;
}

// Second score of the structured mask (PIPE_SCORE_L2): the squared Euclidean norm of the group's residual rows in
// binary64, with the order of the additions fixed as include/pipe.h states it so that the kept lists can be compared
// bit for bit: one warp per row, lane l sums the squares of the elements l, l + 32, ... in ascending order (a square
// of a binary32 value is exact in binary64), then the 32 partial sums are added as a tree with offsets 16, 8, 4, 2, 1.
__global__ void __launch_bounds__(256) row_sumsq_kernel(const float* __restrict__ r, int64_t ld, int O, int I, double* __restrict__ rowsq) {
  const int o = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (o >= O) return;
  const float* row = r + static_cast<int64_t>(o) * ld;
  double s = 0.0;
  for (int i = lane; i < I; i += 32) {
    const double v = static_cast<double>(row[i]);
    s = __dadd_rn(s, __dmul_rn(v, v));
  }
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) s = __dadd_rn(s, __shfl_down_sync(0xffffffffu, s, off));
  if (lane == 0) rowsq[o] = s;
}

// score[j] = sum over the group's rows, ascending, of rowsq; one thread per group.
__global__ void group_score_l2_kernel(const double* __restrict__ rowsq, int G, int g, double* __restrict__ score) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= G) return;
  double s = 0.0;
  for (int u = 0; u < g; ++u) s = __dadd_rn(s, rowsq[static_cast<int64_t>(j) * g + u]);
  score[j] = s;
}

// Unstructured mask (pipe_layer_desc::keep_elems): per row, the magnitude key of the n-th largest entry of the
// residual and the index up to which entries EQUAL to it are kept (ties go to the lower index).  One block per row:
// a radix select over the four bytes of the key, then a bisection on the index among the ties.  An entry i of the
// row is kept iff key_i > thr, or key_i == thr and i <= tie_cut.
__global__ void __launch_bounds__(256) row_topn_kernel(const float* __restrict__ r, int64_t ld, int I, int n,
                                                       uint32_t* __restrict__ thr_out, int32_t* __restrict__ cut_out) {
  __shared__ int hist[256];
  __shared__ uint32_t sh_prefix;
  __shared__ int sh_remaining, sh_count;
  const float* row = r + static_cast<int64_t>(blockIdx.x) * ld;
  uint32_t prefix = 0, mask = 0;
  int remaining = n;
  for (int shift = 24; shift >= 0; shift -= 8) {
    hist[threadIdx.x] = 0;
    __syncthreads();
    for (int i = threadIdx.x; i < I; i += blockDim.x) {
      const uint32_t k = abs_key(row[i]);
      if ((k & mask) == prefix) atomicAdd(&hist[(k >> shift) & 0xffu], 1);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      int b = 255, rem = remaining;
      while (b > 0 && hist[b] < rem) rem -= hist[b--];   // the bin that holds the rem-th largest of the candidates
      sh_prefix = prefix | (static_cast<uint32_t>(b) << shift);
      sh_remaining = rem;
    }
    __syncthreads();
    prefix = sh_prefix;
    remaining = sh_remaining;
    mask |= 0xffu << shift;
    __syncthreads();
  }
  // `remaining` of the entries equal to prefix are kept: the smallest index c such that #{i <= c : key_i == prefix} = remaining
  int lo = 0, hi = I - 1;
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (threadIdx.x == 0) sh_count = 0;
    __syncthreads();
    int c = 0;
    for (int i = threadIdx.x; i <= mid; i += blockDim.x) c += abs_key(row[i]) == prefix;
    if (c) atomicAdd(&sh_count, c);
    __syncthreads();
    const int total = sh_count;
    __syncthreads();
    if (total >= remaining) hi = mid;
    else lo = mid + 1;
  }
  if (threadIdx.x == 0) {
    thr_out[blockIdx.x] = prefix;
    cut_out[blockIdx.x] = lo;
  }
}

// Exclusive prefix sum of keep[] -> cum[0..G], and the ascending list of kept groups.
// keep == nullptr means "all groups kept".  Single block of 1024 threads.
__global__ void __launch_bounds__(1024) group_compact_kernel(const int32_t* __restrict__ keep, int G,
                                                             int32_t* __restrict__ cum, int32_t* __restrict__ kept) {
  __shared__ int32_t chunk_sum[1024];
  const int per = (G + blockDim.x - 1) / blockDim.x;
  const int b = threadIdx.x * per, e = min(G, b + per);
  int32_t s = 0;
  for (int j = b; j < e; ++j) s += keep ? keep[j] : 1;
  chunk_sum[threadIdx.x] = s;
  __syncthreads();
  // inclusive Hillis-Steele scan over the chunk sums
  for (int d = 1; d < blockDim.x; d <<= 1) {
    int32_t v = threadIdx.x >= d ? chunk_sum[threadIdx.x - d] : 0;
    __syncthreads();
    chunk_sum[threadIdx.x] += v;
    __syncthreads();
  }
  int32_t run = threadIdx.x == 0 ? 0 : chunk_sum[threadIdx.x - 1];
  for (int j = b; j < e; ++j) {
    cum[j] = run;
    if (!keep || keep[j]) kept[run++] = j;
  }
  if (threadIdx.x == blockDim.x - 1) cum[G] = chunk_sum[blockDim.x - 1];
}

// Group selection of one order in ONE block, for layers of up to kFusedGroups groups: scores, ranks and
// the compacted list stay in shared memory (three tiny launches less per sparse order).  Same rule and
// same exact comparisons as the three kernels above.
constexpr int kFusedGroups = 512;   // one group per thread; a power of two (the sorting network's size)
__global__ void __launch_bounds__(kFusedGroups) group_select_kernel(const float* __restrict__ a, int G, int g, int n_keep,
                                                            int32_t* __restrict__ cum, int32_t* __restrict__ kept) {
  // Rank = position in the order (score descending, index ascending), found by sorting the keys
  // (score bits, ~index) in descending order: scores are non-negative floats, whose order is the order of their bit
  // patterns, so the keys are distinct integers and the sorted order is unique (a bitonic network of 45 rounds over
  // the 512 slots; slots beyond G hold the smallest key and end up last).
  __shared__ unsigned long long key[kFusedGroups];
  __shared__ int32_t flag[kFusedGroups];
  __shared__ int32_t chunk_sum[kFusedGroups];
  const int tid = threadIdx.x;
  {
    unsigned long long kv = 0ull;
    if (tid < G) {
      // the group's row maxima: independent loads (four at a time where the rows allow vector loads)
      const float* rows = a + static_cast<int64_t>(tid) * g;
      float m0 = 0.f, m1 = 0.f, m2 = 0.f, m3 = 0.f;
      int u = 0;
      if ((g & 3) == 0 && (reinterpret_cast<uintptr_t>(rows) & 15) == 0) {
#pragma unroll 4
        for (; u < g; u += 4) {
          const float4 v = *reinterpret_cast<const float4*>(rows + u);
          m0 = fmaxf(m0, v.x);
          m1 = fmaxf(m1, v.y);
          m2 = fmaxf(m2, v.z);
          m3 = fmaxf(m3, v.w);
        }
      }
#pragma unroll 4
      for (; u < g; ++u) m0 = fmaxf(m0, rows[u]);
      const float m = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
      kv = (static_cast<unsigned long long>(__float_as_uint(m)) << 32) | (0xffffffffu - static_cast<uint32_t>(tid));
    }
    key[tid] = kv;
  }
  __syncthreads();
  for (int k = 2; k <= kFusedGroups; k <<= 1) {
    for (int j = k >> 1; j > 0; j >>= 1) {
      const int other = tid ^ j;
      if (other > tid) {
        const unsigned long long x = key[tid], y = key[other];
        const bool descending = (tid & k) == 0;
        if (descending ? x < y : x > y) {
          key[tid] = y;
          key[other] = x;
        }
      }
      __syncthreads();
    }
  }
  if (tid < G) flag[0xffffffffu - static_cast<uint32_t>(key[tid])] = tid < n_keep ? 1 : 0;
  __syncthreads();
  const int per = (G + blockDim.x - 1) / blockDim.x;
  const int b = threadIdx.x * per, e = min(G, b + per);
  int32_t sum = 0;
  for (int j = b; j < e; ++j) sum += flag[j];
  chunk_sum[threadIdx.x] = sum;
  __syncthreads();
  for (int d = 1; d < blockDim.x; d <<= 1) {
    int32_t v = threadIdx.x >= d ? chunk_sum[threadIdx.x - d] : 0;
    __syncthreads();
    chunk_sum[threadIdx.x] += v;
    __syncthreads();
  }
  int32_t run = threadIdx.x == 0 ? 0 : chunk_sum[threadIdx.x - 1];
  for (int j = b; j < e; ++j) {
    cum[j] = run;
    if (flag[j]) kept[run++] = j;
  }
  if (threadIdx.x == blockDim.x - 1) cum[G] = chunk_sum[blockDim.x - 1];
}

// Pack 16 codes (each already in [-qmax, qmax]) into the canonical and the kernel layout.
// canonical: field e at bit e*b of the stream; kernel: see include/pipe.h.
template <int BITS>
__device__ __forceinline__ void pack16(const int (&q)[16], uint32_t (&canon)[4], uint32_t (&kern)[4]) {
  if (BITS == 8) {
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      uint32_t v = 0;
#pragma unroll
      for (int e = 0; e < 4; ++e) v |= (static_cast<uint32_t>(q[4 * w + e]) & 0xffu) << (8 * e);
      canon[w] = v;
      kern[w] = v;
    }
  } else if (BITS == 4) {
#pragma unroll
    for (int w = 0; w < 2; ++w) {
      uint32_t c = 0, k = 0;
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const uint32_t f = static_cast<uint32_t>(q[8 * w + e]) & 0xfu;
        c |= f << (4 * e);
        const int h = e >> 2, j = e & 3;  // code 4h+j -> nibble 2j+h
        k |= f << (4 * (2 * j + h));
      }
      canon[w] = c;
      kern[w] = k;
    }
  } else {
    uint32_t c = 0, k = 0;
#pragma unroll
    for (int e = 0; e < 16; ++e) {
      const uint32_t f = static_cast<uint32_t>(q[e]) & 0x3u;
      c |= f << (2 * e);
      const int h = e >> 2, j = e & 3;  // code 4h+j -> bits 8j+2h
      k |= f << (8 * j + 2 * h);
    }
    canon[0] = c;
    kern[0] = k;
  }
}

struct QuantizeRowsArgs {
  const float* src;      // residual entering this order ([O, ld_src])
  int64_t ld_src;
  float* dst;            // residual leaving this order ([O, ld_dst]) or nullptr (last order)
  int64_t ld_dst;
  float* a;              // [O] row absmax: read (this order's), overwritten (next order's) if dst
  int first;             // order 1: the row maximum is not in a[] yet, the block finds it itself
  int* status;
  const int32_t* kept;   // [rows/g] ascending kept groups
  uint8_t* codes;        // canonical [rows, canon_row_bytes]
  uint8_t* kcodes;       // streaming layout [ceil(I/128), rows, 128*BITS/8]
  uint8_t* wcodes;       // int8 copy in the tensor-core operand layout [ceil(I/128), rows, 128] or nullptr (see pipe.h)
  int rows;              // compacted rows of this order
  float* scales;         // [rows]
  int I, g, qmax;
  int canon_row_bytes, kernel_row_bytes;
  const uint32_t* mask_thr;   // unstructured mask of this order, per ORIGINAL row (nullptr: every entry is kept):
  const int32_t* mask_cut;    // an entry is kept iff its magnitude key > thr, or == thr and its index <= cut
};

// One block per compacted row: Eq. 1 on the residual, then the residual update of Eq. 3.
template <int BITS>
__global__ void __launch_bounds__(kRowThreads, 5) quantize_rows_kernel(const QuantizeRowsArgs p) {
  const int n = blockIdx.x;
  const int o = p.kept[n / p.g] * p.g + n % p.g;
  const float* src = p.src + static_cast<int64_t>(o) * p.ld_src;
  float* dst = p.dst ? p.dst + static_cast<int64_t>(o) * p.ld_dst : nullptr;
  const float fq = static_cast<float>(p.qmax);
  float amax;
  if (p.first) {
    // order 1 (Eq. 1 on W itself): one more pass over the row, which the second pass then finds in cache
    uint32_t mk = 0;
    if ((reinterpret_cast<uintptr_t>(src) & 15) == 0) {
      const int n4 = p.I >> 2;
      const float4* r4 = reinterpret_cast<const float4*>(src);
      for (int i = threadIdx.x; i < n4; i += blockDim.x) {
        const float4 v = r4[i];
        mk = max(max(mk, abs_key(v.x)), max(abs_key(v.y), max(abs_key(v.z), abs_key(v.w))));
      }
      for (int i = (n4 << 2) + threadIdx.x; i < p.I; i += blockDim.x) mk = max(mk, abs_key(src[i]));
    } else {
      for (int i = threadIdx.x; i < p.I; i += blockDim.x) mk = max(mk, abs_key(src[i]));
    }
    mk = block_max_u32(mk);
    if (threadIdx.x == 0 && mk >= 0x7f800000u) raise_status(p.status, PIPE_ERR_NONFINITE);
    amax = __uint_as_float(mk);
  } else {
    amax = p.a[o];
  }
  const float s = __fdiv_rn(amax, fq);
  const bool masked = p.mask_thr != nullptr;
  const uint32_t mthr = masked ? p.mask_thr[o] : 0u;
  const int mcut = masked ? p.mask_cut[o] : 0;
  __syncthreads();  // every thread has read a[o] before thread 0 overwrites it at the end
  if (threadIdx.x == 0) p.scales[n] = s;
  uint8_t* crow = p.codes + static_cast<int64_t>(n) * p.canon_row_bytes;
  constexpr int kStepBytes = 128 * BITS / 8;  // packed bytes of one row in one 128-code reduction block
  constexpr int kChunkBytes = 16 * BITS / 8;  // bytes of 16 packed codes
  constexpr int kWords = kChunkBytes / 4;
  const int I = p.I;
  const int I_pad = p.kernel_row_bytes * 8 / BITS;
  const bool src_vec = (reinterpret_cast<uintptr_t>(src) & 15) == 0;
  const bool dst_vec = dst && (reinterpret_cast<uintptr_t>(dst) & 15) == 0;
  const bool canon_vec = (reinterpret_cast<uintptr_t>(crow) & 3) == 0;
  uint32_t m = 0;
  constexpr int CPW = 32 / BITS;   // codes per packed 32-bit word
  constexpr int LPW = CPW / 4;     // lanes that share one word when a lane holds 4 consecutive codes
  const bool lanewise = (I % CPW == 0) && src_vec && (!dst || dst_vec) && canon_vec && (p.canon_row_bytes % 4 == 0);
  if (lanewise) {
    // Lane-contiguous form: per trip a warp covers 512 consecutive elements, lane L holding the four quads at
    // offsets w * 128 + 4 L (w = 0..3), so every load and store instruction of the warp touches one contiguous
    // run.  A packed word then takes its fields from LPW neighbouring lanes; each lane shifts its four codes
    // to their places in both layouts and the lanes OR their parts together.
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int h = lane & (LPW - 1);
    for (int base = warp * 512; base < I_pad; base += nwarps * 512) {
      float4 v[4];
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const int e0 = base + w * 128 + lane * 4;
        v[w] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (e0 < I) v[w] = *reinterpret_cast<const float4*>(src + e0);   // plain load: src may alias dst
      }
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const int e0 = base + w * 128 + lane * 4;
        float x[4] = {v[w].x, v[w].y, v[w].z, v[w].w};
        uint32_t f4[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          float c = 0.f;
          bool take = s != 0.f;
          if (masked) {
            const uint32_t key = abs_key(x[j]);
            take = take && (key > mthr || (key == mthr && e0 + j <= mcut));
          }
          if (take) {
            c = rintf(__fdiv_rn(x[j], s));         // round half to even
            c = fminf(fmaxf(c, -fq), fq);
            x[j] = __fmaf_rn(-s, c, x[j]);         // exact new residual, rounded once
          }
          m = max(m, abs_key(x[j]));
          f4[j] = static_cast<uint32_t>(static_cast<int>(c));
        }
        if (dst && e0 < I) *reinterpret_cast<float4*>(dst + e0) = make_float4(x[0], x[1], x[2], x[3]);
        // The four codes as the four bytes of a word, then both packed layouts from that word with masks and shifts
        // on all four fields at once.  Canonical: field e at bit e * b of the stream (this lane's four fields are
        // e = 4 h + j); streaming layout: field 4 h + j at bit 8 j + b h (see include/pipe.h).
        const uint32_t wv = __byte_perm(__byte_perm(f4[0], f4[1], 0x0040), __byte_perm(f4[2], f4[3], 0x0040), 0x5410);
        uint32_t cc, ck;
        if (BITS == 8) {
          cc = ck = wv;
        } else if (BITS == 4) {
          const uint32_t t = wv & 0x0F0F0F0Fu;
          const uint32_t u = (t | (t >> 4)) & 0x00FF00FFu;
          cc = ((u | (u >> 8)) & 0xFFFFu) << (16 * h);
          ck = t << (4 * h);
        } else {
          const uint32_t t = wv & 0x03030303u;
          const uint32_t u = (t | (t >> 6)) & 0x000F000Fu;
          cc = ((u | (u >> 12)) & 0xFFu) << (8 * h);
          ck = t << (2 * h);
        }
#pragma unroll
        for (int d = 1; d < LPW; d <<= 1) {
          cc |= __shfl_xor_sync(0xffffffffu, cc, d);
          ck |= __shfl_xor_sync(0xffffffffu, ck, d);
        }
        if (p.wcodes && e0 < I_pad) {
          // the lane's four codes are four bytes of piece (e0 & 127) / 16 of the row's block, which is stored as piece
          // ((e0 & 127) / 16) ^ (n & 7)
          uint8_t* wdst = p.wcodes + (static_cast<int64_t>(e0 >> 7) * p.rows + n) * 128 + (((((e0 & 127) >> 4) ^ (n & 7)) << 4) | (e0 & 15));
          *reinterpret_cast<uint32_t*>(wdst) = wv;
        }
        if (h == 0 && e0 < I_pad) {
          uint8_t* kdst = p.kcodes + (static_cast<int64_t>(e0 >> 7) * p.rows + n) * kStepBytes + (e0 & 127) * BITS / 8;
          *reinterpret_cast<uint32_t*>(kdst) = ck;
          if (e0 < I) *reinterpret_cast<uint32_t*>(crow + e0 * BITS / 8) = cc;
        }
      }
    }
  } else
  for (int i0 = threadIdx.x * 16; i0 < I_pad; i0 += blockDim.x * 16) {
    float v[16];
    const bool full = i0 + 16 <= I;
    if (full && src_vec) {
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const float4 t = reinterpret_cast<const float4*>(src + i0)[w];  // plain load: src may alias dst
        v[4 * w] = t.x; v[4 * w + 1] = t.y; v[4 * w + 2] = t.z; v[4 * w + 3] = t.w;
      }
    } else {
#pragma unroll
      for (int e = 0; e < 16; ++e) v[e] = (i0 + e < I) ? src[i0 + e] : 0.f;
    }
    int q[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) {
      float c = 0.f;
      const uint32_t key = abs_key(v[e]);
      if (s != 0.f && (!masked || key > mthr || (key == mthr && i0 + e <= mcut))) {
        c = rintf(__fdiv_rn(v[e], s));           // round half to even
        c = fminf(fmaxf(c, -fq), fq);
        v[e] = __fmaf_rn(-s, c, v[e]);           // exact new residual, rounded once
      }
      q[e] = static_cast<int>(c);
      m = max(m, abs_key(v[e]));
    }
    if (dst) {
      if (full && dst_vec) {
#pragma unroll
        for (int w = 0; w < 4; ++w)
          reinterpret_cast<float4*>(dst + i0)[w] = make_float4(v[4 * w], v[4 * w + 1], v[4 * w + 2], v[4 * w + 3]);
      } else {
#pragma unroll
        for (int e = 0; e < 16; ++e)
          if (i0 + e < I) dst[i0 + e] = v[e];
      }
    }
    uint32_t canon[4], kern[4];
    pack16<BITS>(q, canon, kern);
    if (p.wcodes) {
      uint32_t wv[4];
#pragma unroll
      for (int w = 0; w < 4; ++w)
        wv[w] = (static_cast<uint32_t>(q[4 * w]) & 0xffu) | ((static_cast<uint32_t>(q[4 * w + 1]) & 0xffu) << 8) |
                ((static_cast<uint32_t>(q[4 * w + 2]) & 0xffu) << 16) | (static_cast<uint32_t>(q[4 * w + 3]) << 24);
      uint8_t* wdst = p.wcodes + (static_cast<int64_t>(i0 >> 7) * p.rows + n) * 128 + ((((i0 & 127) >> 4) ^ (n & 7)) << 4);
      *reinterpret_cast<uint4*>(wdst) = make_uint4(wv[0], wv[1], wv[2], wv[3]);
    }
    const int byte0 = i0 * BITS / 8;
    // streaming layout: reduction-block major, [i0 / 128][row][128 codes]; padded, always whole words
    uint8_t* kdst = p.kcodes + (static_cast<int64_t>(i0 >> 7) * p.rows + n) * kStepBytes + (i0 & 127) * BITS / 8;
#pragma unroll
    for (int w = 0; w < kWords; ++w) reinterpret_cast<uint32_t*>(kdst)[w] = kern[w];
    if (i0 < I) {
      if (full && canon_vec) {
#pragma unroll
        for (int w = 0; w < kWords; ++w) reinterpret_cast<uint32_t*>(crow + byte0)[w] = canon[w];
      } else {
        const int nbytes = min(kChunkBytes, p.canon_row_bytes - byte0);
        for (int bb = 0; bb < nbytes; ++bb) crow[byte0 + bb] = static_cast<uint8_t>(canon[bb >> 2] >> (8 * (bb & 3)));
      }
    }
  }
  if (dst) {
    m = block_max_u32(m);
    if (threadIdx.x == 0) p.a[o] = __uint_as_float(m);
  }
}

// Channel-block table of one cluster of orders (see pipe.h): the groups are walked from 0 and a block is closed
// when the next group would take its stacked rows beyond PIPE_BLOCK_ROWS or its channels beyond PIPE_BLOCK_CHANNELS.
// One thread block per cluster: all threads gather the rows every group stacks (kept orders of the cluster only),
// thread 0 then cuts the blocks.
constexpr int kTableSets = 2 * (PIPE_MAX_ORDERS + 1);   // channel-block tables, then decode-unit tables
struct BlockTableArgs {
  const int32_t* cum[kTableSets][8];   // prefix counts of the cluster's orders
  int nk[kTableSets];
  int32_t* out[kTableSets];
  int cap[kTableSets];
  int limit[kTableSets];   // rows a block of the cluster may stack
  int G, g;
};

constexpr int kTableChunk = 2048;
constexpr int kTableThreads = 256;

// One thread block per table.  The groups are taken in chunks: all threads gather the rows every group of the chunk
// stacks (kept orders of the cluster only) and form their running sums; the first warp then cuts the blocks.  The
// greedy rule "close the block when the next group would take it beyond the limit" needs, for a block that starts at
// group b, the first group whose running sum from b exceeds the limit (or that would be the block's max_groups + 1-th):
// the sums are non-decreasing, so the lanes test 32 candidates at a time and the first hit is the cut.
__global__ void __launch_bounds__(kTableThreads) block_table_kernel(const __grid_constant__ BlockTableArgs a) {
  __shared__ int pre_s[kTableChunk];            // inclusive running sum of the chunk's rows
  __shared__ int part_s[kTableThreads];
  const int m = blockIdx.x;
  int32_t* out = a.out[m];
  if (!out) return;
  int cur_rows = 0, cur_groups = 0, n = 0;      // (warp 0: the same in every lane)
  const int max_groups = PIPE_BLOCK_CHANNELS / a.g > 0 ? PIPE_BLOCK_CHANNELS / a.g : 1;
  const int lane = threadIdx.x & 31;
  constexpr int kPer = kTableChunk / kTableThreads;
  for (int base = 0; base < a.G; base += kTableChunk) {
    const int cnt = min(kTableChunk, a.G - base);
    // rows of this thread's kPer consecutive groups, then a scan of the threads' totals
    int r[kPer];
    int tot = 0;
#pragma unroll
    for (int u = 0; u < kPer; ++u) {
      const int j = threadIdx.x * kPer + u;
      int v = 0;
      if (j < cnt)
        for (int q = 0; q < a.nk[m]; ++q) v += (a.cum[m][q][base + j + 1] - a.cum[m][q][base + j]) * a.g;
      tot += v;
      r[u] = tot;
    }
    part_s[threadIdx.x] = tot;
    __syncthreads();
    for (int d = 1; d < kTableThreads; d <<= 1) {
      const int v = threadIdx.x >= d ? part_s[threadIdx.x - d] : 0;
      __syncthreads();
      part_s[threadIdx.x] += v;
      __syncthreads();
    }
    const int before = threadIdx.x == 0 ? 0 : part_s[threadIdx.x - 1];
#pragma unroll
    for (int u = 0; u < kPer; ++u) {
      const int j = threadIdx.x * kPer + u;
      if (j < cnt) pre_s[j] = before + r[u];
    }
    __syncthreads();
    if (threadIdx.x < 32) {
      if (base == 0 && lane == 0) out[1] = 0;
      int pos = 0, s0 = 0;   // next group of the chunk to place; running sum before it
      while (pos < cnt) {
        for (int off = 0;; off += 32) {
          const int c = pos + off + lane;
          const bool valid = c < cnt;
          const int rsum = valid ? pre_s[c] - s0 : 0;   // rows of the groups pos .. c
          const int ng = cur_groups + off + lane;       // groups of the block before c
          const bool cut = valid && ng > 0 && (cur_rows + rsum > a.limit[m] || ng + 1 > max_groups);
          const unsigned hit = __ballot_sync(0xffffffffu, cut);
          if (hit) {
            const int f = off + __ffs(hit) - 1;         // group pos + f opens the next block
            if (lane == 0 && n < a.cap[m]) out[2 + n] = base + pos + f;   // (the capacity bound holds by construction; never write past it)
            ++n;
            cur_rows = 0;
            cur_groups = 0;
            pos += f;
            s0 = pos > 0 ? pre_s[pos - 1] : 0;
            break;
          }
          if (pos + off + 32 >= cnt) {                  // the rest of the chunk joins the block under construction
            cur_rows += pre_s[cnt - 1] - s0;
            cur_groups += cnt - pos;
            pos = cnt;
            break;
          }
        }
      }
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    if (n < a.cap[m]) out[2 + n] = a.G;
    ++n;
    out[0] = n <= a.cap[m] ? n : 0;
  }
}

// Block records (layout in pipe.h): one thread block per (block of a table, table).
struct BlockRecordArgs {
  const int32_t* cum[PIPE_MAX_ORDERS + 1][8];   // prefix counts of the cluster's orders
  const float* scales[PIPE_MAX_ORDERS + 1][8];  // their row scales
  int nk[PIPE_MAX_ORDERS + 1];
  const int32_t* tbl[PIPE_MAX_ORDERS + 1];      // the channel-block table (n, b_0 .. b_n)
  uint8_t* out[PIPE_MAX_ORDERS + 1];
  int cap[PIPE_MAX_ORDERS + 1];
  int g;
  int* status;
};

__global__ void block_record_kernel(const __grid_constant__ BlockRecordArgs a) {
  const int m = blockIdx.y, cb = blockIdx.x;
  if (!a.out[m]) return;
  const int n_blocks = a.tbl[m][0];
  if (n_blocks > a.cap[m]) {   // cannot happen (the capacity is a bound on the cut); never write past it
    if (cb == 0 && threadIdx.x == 0) raise_status(a.status, PIPE_ERR_WORKSPACE);
    return;
  }
  if (cb >= n_blocks) return;
  __shared__ int rowbase_s[9], start_s[8];
  const int j0 = a.tbl[m][1 + cb], j1 = a.tbl[m][2 + cb];
  const int nk = a.nk[m];
  if (threadIdx.x == 0) {
    int rb = 0;
    for (int q = 0; q < 8; ++q) {
      rowbase_s[q] = rb;
      start_s[q] = 0;
      if (q < nk) {
        const int lo = a.cum[m][q][j0], hi = a.cum[m][q][j1];
        start_s[q] = lo * a.g;
        rb += (hi - lo) * a.g;
      }
    }
    rowbase_s[8] = rb;
  }
  __syncthreads();
  uint8_t* rec = a.out[m] + static_cast<size_t>(cb) * kRecBytes;
  int32_t* hdr = reinterpret_cast<int32_t*>(rec);
  int16_t* colmap = reinterpret_cast<int16_t*>(rec + kRecColmapOff);
  float* scale = reinterpret_cast<float*>(rec + kRecScaleOff);
  const int c0 = j0 * a.g, c1 = j1 * a.g, n_total = rowbase_s[8];
  for (int i = threadIdx.x; i < kRecHeaderInts; i += blockDim.x) {
    int v = 0;
    if (i == 0) v = c0;
    else if (i == 1) v = c1;
    else if (i == 2) v = nk;
    else if (i == 3) v = n_total;
    else if (i >= kRecRowbase && i < kRecRowbase + 8) v = rowbase_s[i - kRecRowbase];
    else if (i >= kRecStart && i < kRecStart + 8) v = start_s[i - kRecStart];
    hdr[i] = v;
  }
  const int nch = (c1 - c0) >> 3;
  for (int e = threadIdx.x; e < kRecColmapEntries; e += blockDim.x) {
    const int cc = e >> 3, q = e & 7;
    int col = -1;
    if (q < nk && cc < nch) {
      const int c = c0 + 8 * cc;
      const int j = c / a.g;
      const int lo = a.cum[m][q][j], hi = a.cum[m][q][j + 1];
      if (hi > lo) col = rowbase_s[q] + lo * a.g + c % a.g - start_s[q];
    }
    colmap[e] = static_cast<int16_t>(col);
  }
  for (int r = threadIdx.x; r < PIPE_BLOCK_ROWS; r += blockDim.x) {
    float v = 0.f;
    if (r < n_total) {
      int q = 0;
      while (q + 1 < nk && r >= rowbase_s[q + 1]) ++q;
      v = a.scales[m][q][start_s[q] + (r - rowbase_s[q])];
    }
    scale[r] = v;
  }
}

__global__ void write_header_kernel(uint32_t* hdr, pipe_layer_desc d) {
  if (threadIdx.x == 0) {
    hdr[0] = kBlobMagic;
    hdr[1] = 1;  // format version
    int32_t* o = reinterpret_cast<int32_t*>(hdr + 2);
    o[0] = d.out_features; o[1] = d.in_features; o[2] = d.weight_bits; o[3] = d.num_orders;
    o[4] = d.group_size; o[5] = d.keep_groups; o[6] = d.num_branches;
    for (int m = 0; m < PIPE_MAX_ORDERS; ++m) o[7 + m] = d.branch_orders[m];
  }
}

}  // namespace pipe

using namespace pipe;

extern "C" pipe_status pipe_expand_weights(const pipe_layer_desc* desc, const float* d_W, int64_t ldw, void* d_blob,
                                           size_t blob_bytes, void* d_ws, size_t ws_bytes, void* stream) {
  LayerInfo L;
  pipe_status st = resolve_layer(desc, &L);
  if (st != PIPE_OK) return st;
  if (!d_W || !d_blob || !d_ws) return PIPE_ERR_INVALID_ARG;
  if (ldw < L.I) return PIPE_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(d_W) & 3) || (reinterpret_cast<uintptr_t>(d_blob) & (PIPE_BLOB_ALIGN - 1)) ||
      (reinterpret_cast<uintptr_t>(d_ws) & 255))
    return PIPE_ERR_ALIGNMENT;
  if (blob_bytes < L.lay.blob_bytes || ws_bytes < L.lay.expand_ws_bytes) return PIPE_ERR_WORKSPACE;
  int* status = device_status_word();
  if (!status) return PIPE_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);

  uint8_t* ws = static_cast<uint8_t*>(d_ws);
  const int64_t I4 = round_up(L.I, 4);
  float* resid = reinterpret_cast<float*>(ws);
  uint64_t off = round_up<uint64_t>(static_cast<uint64_t>(L.O) * I4 * 4, 256);
  float* a = reinterpret_cast<float*>(ws + off);
  off += round_up<uint64_t>(static_cast<uint64_t>(L.O) * 4, 256);
  float* score = reinterpret_cast<float*>(ws + off);          // G doubles for the L2 score, G floats otherwise
  double* score64 = reinterpret_cast<double*>(ws + off);
  off += round_up<uint64_t>(static_cast<uint64_t>(L.G) * 8, 256);
  int32_t* keep = reinterpret_cast<int32_t*>(ws + off);
  off += round_up<uint64_t>(static_cast<uint64_t>(L.G) * 4, 256);
  double* rowsq = nullptr;
  if (L.score_mode == PIPE_SCORE_L2) {
    rowsq = reinterpret_cast<double*>(ws + off);
    off += round_up<uint64_t>(static_cast<uint64_t>(L.O) * 8, 256);
  }
  uint32_t* mask_thr = nullptr;
  int32_t* mask_cut = nullptr;
  if (L.keep_elems > 0) {
    mask_thr = reinterpret_cast<uint32_t*>(ws + off);
    off += round_up<uint64_t>(static_cast<uint64_t>(L.O) * 4, 256);
    mask_cut = reinterpret_cast<int32_t*>(ws + off);
    off += round_up<uint64_t>(static_cast<uint64_t>(L.O) * 4, 256);
  }
  uint8_t* blob = static_cast<uint8_t*>(d_blob);

  write_header_kernel<<<1, 32, 0, s>>>(reinterpret_cast<uint32_t*>(blob), *desc);
  count_launch(1);
  for (int k = 0; k < L.K; ++k) {
    int32_t* kept = reinterpret_cast<int32_t*>(blob + L.lay.kept_off[k]);
    int32_t* cum = reinterpret_cast<int32_t*>(blob + L.lay.cum_off[k]);
    const bool dense = (k == 0) || (L.n_keep == L.G);
    if (!dense && L.G <= kFusedGroups && L.score_mode == PIPE_SCORE_MAXABS) {
      group_select_kernel<<<1, kFusedGroups, 0, s>>>(a, L.G, L.g, L.n_keep, cum, kept);
      count_launch(1);
    } else {
      if (!dense && L.score_mode == PIPE_SCORE_L2) {
        // (a sparse order is never the first, so the current residual is in the workspace)
        row_sumsq_kernel<<<ceil_div(L.O, 8), 256, 0, s>>>(resid, I4, L.O, L.I, rowsq);
        group_score_l2_kernel<<<ceil_div(L.G, 256), 256, 0, s>>>(rowsq, L.G, L.g, score64);
        group_rank_kernel<double><<<ceil_div(L.G, 8), 256, 0, s>>>(score64, L.G, L.n_keep, keep);
        count_launch(3);
      } else if (!dense) {
        group_score_kernel<<<ceil_div(L.G, 256), 256, 0, s>>>(a, L.G, L.g, score);
        group_rank_kernel<float><<<ceil_div(L.G, 8), 256, 0, s>>>(score, L.G, L.n_keep, keep);
        count_launch(2);
      }
      group_compact_kernel<<<1, 1024, 0, s>>>(dense ? nullptr : keep, L.G, cum, kept);
      count_launch(1);
    }
    QuantizeRowsArgs q;
    q.src = (k == 0) ? d_W : resid;
    q.ld_src = (k == 0) ? ldw : I4;
    q.dst = (k + 1 < L.K) ? resid : nullptr;
    q.ld_dst = I4;
    q.a = a;
    q.first = (k == 0) ? 1 : 0;
    q.status = status;
    q.kept = kept;
    q.codes = blob + L.lay.codes_off[k];
    q.kcodes = blob + L.lay.kcodes_off[k];
    q.wcodes = L.lay.wcodes_off[k] ? blob + L.lay.wcodes_off[k] : nullptr;
    q.scales = reinterpret_cast<float*>(blob + L.lay.scales_off[k]);
    q.I = L.I; q.g = L.g; q.qmax = L.qmax;
    q.canon_row_bytes = L.lay.canon_row_bytes;
    q.kernel_row_bytes = L.lay.kernel_row_bytes;
    q.rows = L.lay.rows[k];
    q.mask_thr = nullptr;
    q.mask_cut = nullptr;
    if (L.keep_elems > 0 && k > 0) {
      row_topn_kernel<<<L.O, 256, 0, s>>>(resid, I4, L.I, L.keep_elems, mask_thr, mask_cut);
      count_launch(1);
      q.mask_thr = mask_thr;
      q.mask_cut = mask_cut;
    }
    const int rows = L.lay.rows[k];
    if (L.bits == 8) quantize_rows_kernel<8><<<rows, kRowThreads, 0, s>>>(q);
    else if (L.bits == 4) quantize_rows_kernel<4><<<rows, kRowThreads, 0, s>>>(q);
    else quantize_rows_kernel<2><<<rows, kRowThreads, 0, s>>>(q);
    count_launch(1);
  }
  {
    // channel-block tables (entries 0 .. M) and decode-unit tables (entries M + 1 .. 2 M + 1: the same cut with the
    // layout's row limits) in one launch, one thread block per table
    BlockTableArgs t;
    std::memset(&t, 0, sizeof(t));
    t.G = L.G;
    t.g = L.g;
    bool any = false, any_blk = false;
    for (int m = 0; m <= L.M; ++m) {
      const int k0 = (m < L.M) ? L.branch_begin[m] : 0, k1 = (m < L.M) ? L.branch_begin[m + 1] : L.K;
      if (L.lay.blk_off[m] != 0) {
        t.nk[m] = k1 - k0;
        for (int q = 0; q < k1 - k0; ++q) t.cum[m][q] = reinterpret_cast<const int32_t*>(blob + L.lay.cum_off[k0 + q]);
        t.out[m] = reinterpret_cast<int32_t*>(blob + L.lay.blk_off[m]);
        t.cap[m] = L.lay.blk_cap[m];
        // even blocks: the fewest blocks that could hold the cluster's rows, their mean size plus one group of slack
        int64_t R = 0;
        for (int k = k0; k < k1; ++k) R += L.lay.rows[k];
        t.limit[m] = block_row_limit(R, L.O, k1 - k0, L.g);
        any = any_blk = true;
      }
      if (L.lay.dec_off[m] != 0) {
        const int e = L.M + 1 + m;
        t.nk[e] = k1 - k0;
        for (int q = 0; q < k1 - k0; ++q) t.cum[e][q] = reinterpret_cast<const int32_t*>(blob + L.lay.cum_off[k0 + q]);
        t.out[e] = reinterpret_cast<int32_t*>(blob + L.lay.dec_off[m]);
        t.cap[e] = L.G;
        t.limit[e] = L.lay.dec_limit[m];
        any = true;
      }
    }
    if (any) {
      block_table_kernel<<<2 * (L.M + 1), kTableThreads, 0, s>>>(t);
      count_launch(1);
    }
    if (any_blk) {
      // the records of the blocks just cut
      BlockRecordArgs r;
      std::memset(&r, 0, sizeof(r));
      r.g = L.g;
      r.status = status;
      int max_cap = 0;
      for (int m = 0; m <= L.M; ++m) {
        if (L.lay.rec_off[m] == 0) continue;
        const int k0 = (m < L.M) ? L.branch_begin[m] : 0, k1 = (m < L.M) ? L.branch_begin[m + 1] : L.K;
        r.nk[m] = k1 - k0;
        for (int q = 0; q < k1 - k0; ++q) {
          r.cum[m][q] = reinterpret_cast<const int32_t*>(blob + L.lay.cum_off[k0 + q]);
          r.scales[m][q] = reinterpret_cast<const float*>(blob + L.lay.scales_off[k0 + q]);
        }
        r.tbl[m] = reinterpret_cast<const int32_t*>(blob + L.lay.blk_off[m]);
        r.out[m] = blob + L.lay.rec_off[m];
        r.cap[m] = L.lay.rec_cap[m];
        max_cap = max_cap > r.cap[m] ? max_cap : r.cap[m];
      }
      if (max_cap > 0) {
        block_record_kernel<<<dim3(max_cap, L.M + 1), 256, 0, s>>>(r);
        count_launch(1);
      }
    }
  }
  mark_expansion(s);   // a forward call that follows on this stream must not read the blob ahead of its dependency wait
  return launch_status();
}

// ------------------------------------------------------------------------------------------------
// pipe_expand_weights_static: the same expansion for callers that cannot allocate device memory.
// Its workspace is the fixed array below, which is part of the library image: every GPU that
// loads the library holds PIPE_STATIC_SCRATCH_BYTES for it until the process exits.
namespace {

static __device__ __align__(256) unsigned char g_expand_scratch[PIPE_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
void* g_scratch_addr[kMaxDevices] = {nullptr};

// Device address of the array on the current device.  In host code the name g_expand_scratch is
// only a handle for the runtime, not an address a kernel could use; the address has to be asked
// for, once per device, while that device is current.
pipe_status static_scratch(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return PIPE_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_expand_scratch) != cudaSuccess || !p) return PIPE_ERR_CUDA;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return PIPE_OK;
}

}  // namespace

extern "C" pipe_status pipe_expand_weights_static(const pipe_layer_desc* desc, const float* d_W, int64_t ldw,
                                                  void* d_blob, size_t blob_bytes, void* stream) {
  LayerInfo L;
  pipe_status st = resolve_layer(desc, &L);
  if (st != PIPE_OK) return st;
  // the layer's workspace (fp32 residual + per-row and per-group arrays) must fit the fixed array
  if (L.lay.expand_ws_bytes > static_cast<uint64_t>(PIPE_STATIC_SCRATCH_BYTES)) return PIPE_ERR_WORKSPACE;
  void* scratch = nullptr;
  st = static_scratch(&scratch);
  if (st != PIPE_OK) return st;
  // Nothing in the workspace has to start at zero: the residual, the row maxima, the group scores
  // and the keep flags are all written by this call before it reads them, so what an earlier
  // call left behind is simply overwritten.
  return pipe_expand_weights(desc, d_W, ldw, d_blob, blob_bytes, scratch, PIPE_STATIC_SCRATCH_BYTES, stream);
}
