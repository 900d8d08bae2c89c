// Small-token kernel of the expanded layer (Appendix B, Eq. 9; Sec. 3.2 for the branches), T <= 16.
//
// With a handful of tokens the layer is bound by streaming the packed weight codes from HBM once,
// so the kernel is built around the byte stream.  A "slab" is 8 consecutive output channels of
// one branch; in every order of the branch that keeps the slab's group the slab is 8 consecutive
// compacted rows.  Every CTA (one per SM) owns one contiguous range of slabs.  Because the
// streaming section of the codes is reduction-block-major, the rows a CTA needs from one order
// and one 128-code reduction block are ONE contiguous run, which a producer warp brings into a
// deep ring of shared-memory stages with bulk asynchronous copies (a stage = one reduction block
// of every order of the branch for up to 32 slabs, plus the matching 16 x 128-byte tile of the
// quantized activations as a swizzled TMA box).  Nothing on the load path costs registers, and the
// ring keeps far more bytes in flight than the bandwidth-delay product of the memory system.
//
// 16 consumer warps form 4 groups; group j handles the stages j, j + 4, ... (so a stage is read by 4
// warps, each of which covers up to 5 slabs of it: enough independent work per visit to hide the
// latency of the barrier wait, the shared-memory loads and the chain of dependent MMAs).  A warp
// reads its slabs' 8 rows from the stage, widens sub-byte codes with the shift-and-mask layout and
// feeds warp-level integer MMAs (mma.sync m16n8k32: weights as the 16-row operand -- two orders of
// the slab, ascending, share a tile -- tokens as the 8-column operand).  At the end of a pass the
// four groups add their exact int32 sums in a small shared-memory array, and the fixed-order fp32
// epilogue runs once per slab.  Every mbarrier wait is bounded.
#include <mutex>

#include "pipe_common.cuh"

namespace pipe {

namespace st {

constexpr int kConsWarps = 16;
constexpr int kProdWarps = 4;
constexpr int kGroups = 4;                       // consumer groups = slices of the reduction axis
constexpr int kGroupWarps = kConsWarps / kGroups;
constexpr int kThreads = 32 * (kConsWarps + kProdWarps);
constexpr int kMaxOrd = 8;          // orders per branch
constexpr int kMaxPasses = 32;      // passes (<= 32 slabs of one branch) a CTA may need
constexpr int kMaxDepth = 16;
constexpr int kXTile = 16 * 128;    // 16 token rows x 128 reduction bytes
constexpr long long kWaitLimitCycles = 4000000000ll;

struct Params {
  CUtensorMap tmap_x[PIPE_MAX_ORDERS];   // per branch input: [T rows, I bytes], box 128 x 16, 128-byte swizzle
  ForwardArgs f;
  int kblocks;            // reduction blocks of 128 codes
  int pk;                 // packed bytes of one row of one reduction block
  int shift;              // 8 - b
  int slabs_per_branch;   // O / 8
  int total_slabs;
  int pass_slabs;         // slabs per pass: warps of a group * slabs per warp
  int depth, stage_bytes;
  int kbps;               // reduction blocks per stage (2 for 2-bit codes, else 1)
  int nstages;            // stages per pass
  int nkmax;              // most orders any branch has
  int own_max;            // most slabs any CTA owns
  int prefetch;           // the expanded layer is not being written by the launch before: weights may be fetched ahead of the dependency wait
  uint32_t split_mask;    // summed ensemble on one shared input, run as ONE cluster of all orders: bit k marks the order (k > 0)
                          // that opens the next predictor, whose chain the epilogue starts from zero
  int ctas_per_branch;    // every branch has its own CTAs, so no CTA's range crosses a branch boundary
};

struct Pass {
  int branch, lb, le;                 // local slab range [lb, le) of the CTA's own slabs
  int seg_row0[kMaxOrd], seg_rows[kMaxOrd], seg_off[kMaxOrd];
  int wbytes;                         // weight bytes of one reduction block of this pass
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
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

__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar)
      : "memory");
}
// Ordinary loads (not volatile asm), so that the compiler may schedule them between the MMAs; the
// barrier wait before them is a volatile asm with a memory clobber, which they cannot cross.
__device__ __forceinline__ uint4 lds128(const uint8_t* stage, uint32_t off) {
  return *reinterpret_cast<const uint4*>(stage + off);
}

__device__ __forceinline__ void mma_s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                       uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// int8 lanes (times 2^(8-b)) of MMA number mm of a 16-byte packed chunk: r0 covers the chunk's
// reduction offsets 8mm..8mm+3, r1 covers 8mm+4..8mm+7 (see the streaming layout).
template <int BITS>
__device__ __forceinline__ void frag(const uint4& w, int mm, uint32_t& r0, uint32_t& r1) {
  const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
  if (BITS == 8) {
    r0 = ww[2 * mm];
    r1 = ww[2 * mm + 1];
  } else if (BITS == 4) {
    r0 = (ww[mm] << 4) & 0xF0F0F0F0u;
    r1 = ww[mm] & 0xF0F0F0F0u;
  } else {
    const uint32_t x = ww[mm >> 1];
    const int h = 2 * (mm & 1);
    r0 = (x << (6 - 2 * h)) & 0xC0C0C0C0u;
    r1 = (x << (4 - 2 * h)) & 0xC0C0C0C0u;
  }
}

// Number of compacted rows of an order before channel c of the branch (c a multiple of 8, c <= O).
__device__ __forceinline__ int rows_before(const int32_t* cum, int c, int O, int g) {
  if (c >= O) return __ldg(cum + O / g) * g;
  const int j = c / g;
  const int lo = __ldg(cum + j), hi = __ldg(cum + j + 1);
  return lo * g + (hi > lo ? c - j * g : 0);
}

// FULL != 0: a consumer warp has FULL slab slots per pass and (nearly) every one of them holds a slab (the host knows:
// one pass, FULL = ceil(slabs of a CTA / warps of a group)): the loop over a warp's slabs then runs without its per-slab
// branches -- an absent chunk takes part with zero weights -- so that the slabs' load-and-MMA chains are one block the
// compiler may interleave (cfg4a T = 1, five slabs per warp: 17.6 -> 16.8 us; cfg4b T = 1, two: 21.2 -> 19.4 us; with the
// slots of the general kernel, five, a launch with two slabs per warp would do 2.5 times its work that way).
template <int BITS, int NT, int NP, bool SUMMED, int FULL>
__global__ void __launch_bounds__(kThreads, 1) stream_forward_kernel(const __grid_constant__ Params p) {
  constexpr int SPW = FULL ? FULL : ((NP * NT <= 2) ? 5 : (NP * NT == 4 ? 2 : 1));   // slabs per consumer warp and pass
  constexpr int CHK = 128 / BITS;               // codes per 16-byte chunk
  constexpr int KBPS = (BITS == 2) ? 2 : 1;     // reduction blocks per stage
  constexpr int MS = KBPS * 128 / (4 * CHK);    // macro steps (4 chunks per row of 8 lanes x 4) per stage
  constexpr int XCH = CHK / 16;                 // 16-byte activation chunks per macro step and token
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t bars[2 * kMaxDepth + 2];  // full[depth] empty[depth] sums_ready sums_free
  __shared__ Pass passes[kMaxPasses];
  __shared__ int abort_flag_s;
  volatile int* abort_flag = &abort_flag_s;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gid = lane >> 2, tig = lane & 3;
  const uint32_t stage0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* tables = smem_raw + (stage0 - smem_u32(smem_raw)) + static_cast<size_t>(p.depth) * p.stage_bytes;
  int* slabmeta = reinterpret_cast<int*>(tables);                                   // [own][nkmax] first row or -1
  float* cstab = reinterpret_cast<float*>(slabmeta + p.own_max * p.nkmax);          // [own][nkmax][8] s_k * lambda_x
  float* biastab = cstab + p.own_max * p.nkmax * 8;                                 // [own][8]
  int* chunktab = reinterpret_cast<int*>(biastab + p.own_max * 8);                  // [warp][SPW][1 + 3 * nkmax]
  int* sums = chunktab + kConsWarps * SPW * (1 + 3 * p.nkmax);                          // [pass slab][NP][NT * 4][32 lanes]
  const uint8_t* stage_gen = smem_raw + (stage0 - smem_u32(smem_raw));
  const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8u * kMaxDepth;
  const uint32_t sums_ready = empty0 + 8u * kMaxDepth, sums_free = sums_ready + 8u;
  const int depth = p.depth;

  // this CTA's slabs: [s0, s0 + cnt), all of one branch
  const int my_branch = static_cast<int>(blockIdx.x) / p.ctas_per_branch, cib = static_cast<int>(blockIdx.x) % p.ctas_per_branch;
  const int base = p.slabs_per_branch / p.ctas_per_branch, rem = p.slabs_per_branch % p.ctas_per_branch;
  const int s0 = my_branch * p.slabs_per_branch + cib * base + min(cib, rem);
  const int cnt = base + (cib < rem ? 1 : 0);

  // A launch of this kernel that follows in the stream may be brought onto the SMs as they become free: its CTAs
  // then exist when this launch's last CTA ends, instead of being launched only then (a chain of small-token layers
  // otherwise pays a launch gap and a cold start per layer).  Until the launch before it is complete such a CTA
  // touches nothing that launch may have written: with p.prefetch (the host knows that the expanded layer is not
  // being written: its last call on this stream was no expansion) it builds its tables and fills its whole ring
  // with WEIGHTS first, which belong to the layer alone, and waits only then, before the first access to
  // activations, steps, bias or outputs; without it, it waits before its first access to global memory.
  // Its own dependents start at once in the first case (the layer before was complete, or past this same point, when
  // this CTA started, so no expansion queued earlier is still running beside them) and after the wait in the second.
  if (p.prefetch) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    for (int s = 0; s < depth; ++s) {
      mbar_init(full0 + 8u * s, 1);
      mbar_init(empty0 + 8u * s, kGroupWarps);   // slot s is only ever read by group s % kGroups
    }
    mbar_init(sums_ready, kConsWarps);
    mbar_init(sums_free, kConsWarps);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // passes: pieces of at most pass_slabs slabs of the CTA's range (which lies in one branch)
  const int npass = min((cnt + p.pass_slabs - 1) / p.pass_slabs, kMaxPasses);
  for (int e = threadIdx.x; e < p.pass_slabs * NP * NT * 4 * 32; e += kThreads) sums[e] = 0;
  if (!p.prefetch) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  }
  // ---- which orders keep each own slab, and where its 8 rows start
  for (int e = threadIdx.x; e < cnt * p.nkmax; e += kThreads) {
    const int li = e / p.nkmax, ko = e % p.nkmax;
    const int slab = s0 + li;
    const int branch = slab / p.slabs_per_branch;
    const int c0 = (slab - branch * p.slabs_per_branch) * 8;
    const BranchArgs& br = p.f.branch[branch];
    int row0 = -1;
    if (br.k_begin + ko < br.k_end) {
      const int32_t* cum = p.f.order[br.k_begin + ko].cum;
      const int j = c0 / p.f.g;
      const int lo = __ldg(cum + j), hi = __ldg(cum + j + 1);
      if (hi > lo) row0 = lo * p.f.g + c0 % p.f.g;
    }
    slabmeta[e] = row0;
  }
  // ---- the contiguous run of rows every pass needs from every order (the last threads take this, so that
  // its loads run beside those above)
  for (int e = kThreads - 1 - threadIdx.x; e < npass * kMaxOrd; e += kThreads) {
    const int pi = e / kMaxOrd, ko = e % kMaxOrd;
    Pass& P = passes[pi];
    const BranchArgs& br = p.f.branch[my_branch];
    const int lb = pi * p.pass_slabs, le = min(cnt, lb + p.pass_slabs);
    int r0 = 0, rows = 0;
    if (br.k_begin + ko < br.k_end) {
      const int32_t* cum = p.f.order[br.k_begin + ko].cum;
      const int cb = (s0 + lb - my_branch * p.slabs_per_branch) * 8, ce = (s0 + le - my_branch * p.slabs_per_branch) * 8;
      r0 = rows_before(cum, cb, p.f.O, p.f.g);
      rows = rows_before(cum, ce, p.f.O, p.f.g) - r0;
    }
    P.seg_row0[ko] = r0;
    P.seg_rows[ko] = rows;
    if (ko == 0) {
      P.branch = my_branch;
      P.lb = lb;
      P.le = le;
    }
  }
  __syncthreads();
  if (threadIdx.x < npass) {
    Pass& P = passes[threadIdx.x];
    int off = KBPS * kXTile;
    int wb = 0;
    for (int ko = 0; ko < kMaxOrd; ++ko) {
      P.seg_off[ko] = off;
      off += KBPS * P.seg_rows[ko] * p.pk;
      wb += P.seg_rows[ko] * p.pk;
    }
    P.wbytes = wb;
  }
  __syncthreads();
  const uint32_t total_stages = static_cast<uint32_t>(npass) * p.nstages;

  if (warp >= kConsWarps) {
    // ================================================================== producer warps
    // A copy instruction keeps its issuing thread busy for a hundred cycles or more, but the
    // copies of different lanes of ONE warp instruction, and of different warps, overlap.  So each
    // producer warp issues stages in batches: lane = (stage of the batch, job), a job being one
    // copy of the stage (the activation tile or one order's rows, per reduction block); job-0
    // lanes first wait until the consumers have released their slot, then all lanes issue in
    // step.  Producer warp j owns the batches j, j + W, ... and with them a FIXED subset of the
    // ring's slots (the ring is cut to W batches), so the uses of a slot are issued in order by
    // one warp and the barrier a lane waits for is at most one phase behind.
    constexpr int kJobLanes = 4;
    const uint32_t SB = static_cast<uint32_t>(depth) / kProdWarps;   // depth = SB * kProdWarps (host)
    const int st_in_batch = lane / kJobLanes, job0 = lane % kJobLanes;
    for (uint32_t it0 = (warp - kConsWarps) * SB; it0 < total_stages; it0 += SB * kProdWarps) {
      const uint32_t it = it0 + st_in_batch;
      const bool valid = static_cast<uint32_t>(st_in_batch) < SB && it < total_stages;
      const uint32_t use = valid ? it / depth : 0, slot = valid ? it - use * depth : 0;
      const int pi = valid ? it / p.nstages : 0, ks = valid ? it - pi * p.nstages : 0;
      const Pass& P = passes[pi];
      const BranchArgs& br = p.f.branch[P.branch];
      const int nk = br.k_end - br.k_begin;
      const uint32_t sbase = stage0 + slot * p.stage_bytes;
      const uint32_t bar = full0 + 8u * slot;
      if (valid && job0 == 0) {
        if (mbar_wait(empty0 + 8u * slot, (use & 1u) ^ 1u, abort_flag, p.f.status)) {
          int nkb = 0;
#pragma unroll
          for (int kbs = 0; kbs < KBPS; ++kbs) nkb += (ks * KBPS + kbs < p.kblocks) ? 1 : 0;
          mbar_expect_tx(bar, static_cast<uint32_t>(nkb * (kXTile + P.wbytes)));
        }
      }
      __syncwarp();
      if (*abort_flag) break;
      // jobs of a stage: per reduction block, the activation tile and then one run of rows per order
      // (what: 0 all of them, 1 the weights only, 2 the activation tiles only)
      const int njobs = KBPS * (1 + nk);
      auto issue_jobs = [&](int what) {
        for (int j0 = 0; j0 < KBPS * (1 + p.nkmax); j0 += kJobLanes) {   // same trip count in every lane; lanes without a job idle
          const int j = j0 + job0;
          if (valid && j < njobs) {
            const int kbs = j / (1 + nk), idx = j - kbs * (1 + nk);
            const int kb = ks * KBPS + kbs;
            if (kb < p.kblocks) {
              if (idx == 0) {
                // activations: token rows beyond T and reduction bytes beyond I come back as zeros
                if (what != 1) tma_load_2d(sbase + kbs * kXTile, &p.tmap_x[P.branch], kb * 128, 0, bar);
              } else if (what != 2 && P.seg_rows[idx - 1] > 0) {
                const int ko = idx - 1;
                const OrderView& ov = p.f.order[br.k_begin + ko];
                const uint8_t* src = ov.kcodes + (static_cast<size_t>(kb) * ov.rows + P.seg_row0[ko]) * p.pk;
                bulk_load(sbase + P.seg_off[ko] + kbs * P.seg_rows[ko] * p.pk, src, static_cast<uint32_t>(P.seg_rows[ko] * p.pk), bar);
              }
            }
          }
          __syncwarp();
        }
      };
      if (p.prefetch && it0 < static_cast<uint32_t>(depth)) {
        // the first use of the ring: its weights go ahead of the wait for the launch before, its activation tiles after
        issue_jobs(1);
        asm volatile("griddepcontrol.wait;" ::: "memory");
        issue_jobs(2);
      } else {
        issue_jobs(0);
      }
    }
    __syncwarp();
    // no copy may still be writing into this CTA's shared memory when it exits
    if (warp == kConsWarps && lane == 0) {
      for (uint32_t j = (total_stages > static_cast<uint32_t>(depth) ? total_stages - depth : 0); j < total_stages; ++j) {
        const long long t0 = clock64();
        while (!mbar_try(full0 + 8u * (j % depth), (j / depth) & 1) && clock64() - t0 < kWaitLimitCycles) {
        }
      }
    }
  } else {
    // ================================================================== consumer warps
    if (p.prefetch) asm volatile("griddepcontrol.wait;" ::: "memory");   // (the steps and the bias are the caller's data)
    // scale products s_k * lambda_x and bias of every own slab (needed at the end of a pass only;
    // the loads overlap the first copies)
    for (int e = threadIdx.x; e < cnt * p.nkmax * 8; e += 32 * kConsWarps) {
      const int r = e & 7, ko = (e >> 3) % p.nkmax, li = (e >> 3) / p.nkmax;
      const int branch = (s0 + li) / p.slabs_per_branch;
      const BranchArgs& br = p.f.branch[branch];
      const int row0 = slabmeta[li * p.nkmax + ko];
      float v = 0.f;
      if (row0 >= 0) v = __fmul_rn(__ldg(p.f.order[br.k_begin + ko].scales + row0 + r), __ldg(br.sx));
      cstab[e] = v;
    }
    for (int e = threadIdx.x; e < cnt * 8; e += 32 * kConsWarps) {
      const int r = e & 7, li = e >> 3;
      const int branch = (s0 + li) / p.slabs_per_branch;
      float v = 0.f;
      if (p.f.bias && p.f.branch[branch].add_bias) v = __ldg(p.f.bias + (s0 + li - branch * p.slabs_per_branch) * 8 + r);
      biastab[e] = v;
    }
    asm volatile("bar.sync 1, %0;" ::"r"(32 * kConsWarps) : "memory");   // every consumer warp arrives here unconditionally

    const int centries = 1 + 3 * p.nkmax;
    const int grp = warp / kGroupWarps, wg = warp % kGroupWarps;
    bool ok = true;
    for (int pi = 0; pi < npass && ok; ++pi) {
      const Pass& P = passes[pi];
      const BranchArgs& br = p.f.branch[P.branch];
      const int nk = br.k_end - br.k_begin;
      const int nsl = P.le - P.lb;
      // the sums of the previous pass have been read and cleared by every warp
      if (pi > 0 && !mbar_wait(sums_free, (pi - 1) & 1, abort_flag, p.f.status)) break;
      // This warp's slabs in every stage it visits: wg, wg + 4, ...  Their kept orders, ascending: (byte offset
      // of the 8 rows in a stage, bytes between the reduction blocks of a stage), in a table private to the warp.
      int* mychunks = chunktab + warp * SPW * centries;
      __syncwarp();
      if (lane < SPW) {
        int* ct = mychunks + lane * centries;
        const int sl = wg + kGroupWarps * lane;
        int n = 0;
        if (sl < nsl) {
          for (int ko = 0; ko < nk; ++ko) {
            const int row0 = slabmeta[(P.lb + sl) * p.nkmax + ko];
            if (row0 < 0) continue;
            ct[2 + 3 * n] = P.seg_off[ko] + (row0 - P.seg_row0[ko]) * p.pk;
            ct[3 + 3 * n] = P.seg_rows[ko] * p.pk;
            ++n;
          }
        }
        ct[0] = n;
      }
      __syncwarp();
      int nchunks[SPW];
      uint32_t woff[SPW][2 * NP], wstr[SPW][2 * NP];
#pragma unroll
      for (int s = 0; s < SPW; ++s) {
        nchunks[s] = mychunks[s * centries];
#pragma unroll
        for (int ci = 0; ci < 2 * NP; ++ci) {
          woff[s][ci] = ci < nchunks[s] ? mychunks[s * centries + 2 + 3 * ci] : 0;
          wstr[s][ci] = ci < nchunks[s] ? mychunks[s * centries + 3 + 3 * ci] : 0;
        }
      }
      int acc[SPW][NP][NT][4];
#pragma unroll
      for (int s = 0; s < SPW; ++s)
#pragma unroll
        for (int q = 0; q < NP; ++q)
#pragma unroll
          for (int t = 0; t < NT; ++t)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[s][q][t][e] = 0;

      // stages of this pass that belong to this warp's group
      const uint32_t it_begin = static_cast<uint32_t>(pi) * p.nstages, it_end = it_begin + p.nstages;
      uint32_t it = it_begin + ((grp + kGroups - it_begin % kGroups) % kGroups);
      for (; it < it_end; it += kGroups) {
        const uint32_t use = it / depth, slot = it - use * depth;
        const int ks = it - it_begin;
        if (!mbar_wait(full0 + 8u * slot, use & 1u, abort_flag, p.f.status)) {
          ok = false;
          break;
        }
        const uint8_t* sgen = stage_gen + static_cast<size_t>(slot) * p.stage_bytes;
#pragma unroll
        for (int ms = 0; ms < MS; ++ms) {
          // this lane's chunk: CHK codes from reduction offset kc of the stage
          const int kc = ms * 4 * CHK + tig * CHK;
          const int kbs = kc >> 7, within = kc & 127;
          // A stage's later blocks may lie beyond the reduction axis.  With 2-bit codes that differs from lane
          // to lane, and the MMAs below are warp-wide instructions that every lane must execute: such a lane
          // contributes zero weights instead of leaving the loop (its activation words are stale but finite
          // integers, and zero times anything is zero).
          const bool live = ks * KBPS + kbs < p.kblocks;
          const uint32_t wbyte = static_cast<uint32_t>(gid * p.pk + ((within * BITS) >> 3));
          uint4 xv[XCH][NT];
#pragma unroll
          for (int v = 0; v < XCH; ++v)
#pragma unroll
            for (int t = 0; t < NT; ++t) {
              const int r = gid + 8 * t;
              const int c16 = (within >> 4) + v;
              xv[v][t] = lds128(sgen, kbs * kXTile + r * 128 + ((c16 ^ (r & 7)) << 4));
            }
#pragma unroll
          for (int s = 0; s < SPW; ++s) {
#pragma unroll
            for (int q = 0; q < NP; ++q) {
              uint4 wa = make_uint4(0, 0, 0, 0), wb = make_uint4(0, 0, 0, 0);
              if constexpr (FULL) {
                // (an absent chunk, or a block beyond the reduction axis, reads some valid address of the stage and is
                // replaced by zero weights)
                wa = lds128(sgen, woff[s][2 * q] + kbs * wstr[s][2 * q] + wbyte);
                wb = lds128(sgen, woff[s][2 * q + 1] + kbs * wstr[s][2 * q + 1] + wbyte);
                const bool ha = live && 2 * q < nchunks[s], hb = live && 2 * q + 1 < nchunks[s];
                wa = ha ? wa : make_uint4(0, 0, 0, 0);
                wb = hb ? wb : make_uint4(0, 0, 0, 0);
              } else {
                if (2 * q >= nchunks[s]) continue;
                if (live) wa = lds128(sgen, woff[s][2 * q] + kbs * wstr[s][2 * q] + wbyte);
                if (live && 2 * q + 1 < nchunks[s]) wb = lds128(sgen, woff[s][2 * q + 1] + kbs * wstr[s][2 * q + 1] + wbyte);
              }
#pragma unroll
              for (int mm = 0; mm < 2 * XCH; ++mm) {
                uint32_t a0, a1, b0, b1;
                frag<BITS>(wa, mm, a0, a1);
                frag<BITS>(wb, mm, b0, b1);
#pragma unroll
                for (int t = 0; t < NT; ++t) {
                  const uint32_t xw[4] = {xv[mm >> 1][t].x, xv[mm >> 1][t].y, xv[mm >> 1][t].z, xv[mm >> 1][t].w};
                  // tile rows 0-7: first order of the pair, rows 8-15: second order
                  mma_s8(acc[s][q][t], a0, b0, a1, b1, xw[2 * (mm & 1)], xw[2 * (mm & 1) + 1]);
                }
              }
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty0 + 8u * slot);
      }
      if (!ok) break;
      // ---- the four groups add their exact partial sums
#pragma unroll
      for (int s = 0; s < SPW; ++s) {
        const int sl = wg + kGroupWarps * s;
        if (sl >= nsl) continue;
#pragma unroll
        for (int q = 0; q < NP; ++q) {
          if (2 * q >= nchunks[s]) continue;
#pragma unroll
          for (int t = 0; t < NT; ++t)
#pragma unroll
            for (int e = 0; e < 4; ++e) atomicAdd(sums + ((sl * NP + q) * NT * 4 + t * 4 + e) * 32 + lane, acc[s][q][t][e]);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(sums_ready);
      if (!mbar_wait(sums_ready, pi & 1, abort_flag, p.f.status)) break;
      // ---- fixed-order epilogue, one warp per slab: accumulator registers 0,1 belong to tile row gid (first
      // order of the pair), 2,3 to row gid + 8 (second order); columns 2*tig, 2*tig + 1 of token tile t
      for (int sl = warp; sl < nsl; sl += kConsWarps) {
        const int li = P.lb + sl;
        // kept orders of the slab, ascending (at most 2 * NP)
        int kos[2 * NP];
        int nch = 0;
#pragma unroll
        for (int ko = 0; ko < kMaxOrd; ++ko)
          if (ko < nk && slabmeta[li * p.nkmax + ko] >= 0) {
#pragma unroll
            for (int ci = 0; ci < 2 * NP; ++ci)
              if (ci == nch) kos[ci] = ko;
            ++nch;
          }
        const int c = (s0 + li - P.branch * p.slabs_per_branch) * 8 + gid;   // this thread's output channel
        float y[NT][2];
#pragma unroll
        for (int t = 0; t < NT; ++t) y[t][0] = y[t][1] = 0.f;
        // Summed ensemble on a shared input (split_mask != 0): every predictor's chain starts from zero, the bias closes
        // the first one, the chains are added in ascending predictor order -- the additions one launch per predictor
        // summing into y would make, in the same order.
        float ysum[NT][2];
        bool first_chain = true;
        int next_order = 1;   // orders below this one have had their predictor boundaries handled
        const float bv = biastab[li * 8 + gid];
        auto close_chain = [&]() {
#pragma unroll
          for (int t = 0; t < NT; ++t)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              if (first_chain) ysum[t][e] = (p.f.bias && br.add_bias) ? __fadd_rn(y[t][e], bv) : y[t][e];
              else ysum[t][e] = __fadd_rn(ysum[t][e], y[t][e]);
              y[t][e] = 0.f;
            }
          first_chain = false;
        };
        auto close_up_to = [&](int ko) {   // the boundaries at orders next_order .. ko
          for (; next_order <= ko; ++next_order)
            if ((p.split_mask >> next_order) & 1u) close_chain();
        };
#pragma unroll
        for (int q = 0; q < NP; ++q) {
          if (2 * q >= nch) continue;
          int a4[NT][4];
#pragma unroll
          for (int t = 0; t < NT; ++t)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              int* cell = sums + ((sl * NP + q) * NT * 4 + t * 4 + e) * 32 + lane;
              a4[t][e] = *cell;
              *cell = 0;   // ready for the next pass
            }
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            const int ci = 2 * q + half;
            if (ci >= nch) continue;
            const int ko = kos[ci];
            if constexpr (SUMMED) close_up_to(ko);
            const float cs = cstab[(li * p.nkmax + ko) * 8 + gid];
            const int row = slabmeta[li * p.nkmax + ko] + gid, roff = p.f.order[br.k_begin + ko].row_off;
#pragma unroll
            for (int t = 0; t < NT; ++t)
#pragma unroll
              for (int e = 0; e < 2; ++e) {
                const int a = a4[t][2 * half + e] >> p.shift;   // exact: the sum carries a factor 2^shift
                y[t][e] = __fmaf_rn(__int2float_rn(a), cs, y[t][e]);
                const int tok = 8 * t + 2 * tig + e;
                if (p.f.partials && tok < p.f.T) p.f.partials[static_cast<int64_t>(tok) * p.f.total_rows + roff + row] = a;
              }
          }
        }
        if constexpr (SUMMED) {
          close_up_to(nk - 1);
          close_chain();
#pragma unroll
          for (int t = 0; t < NT; ++t) y[t][0] = ysum[t][0], y[t][1] = ysum[t][1];
        }
        const bool bias = p.f.bias && br.add_bias && !SUMMED;   // (a summed ensemble has added it inside the chain)
#pragma unroll
        for (int t = 0; t < NT; ++t)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int tok = 8 * t + 2 * tig + e;
            if (tok >= p.f.T) continue;
            float v = y[t][e];
            if (bias) v = __fadd_rn(v, bv);
            if (p.f.q8_out) {
              // inner layer of a branch: sigma, then the next layer's input quantizer (Sec. 3.2)
              v = apply_activation(v, p.f.relu);
              const float os = __ldg(br.out_scale);
              if (!(os >= 0.f && os < __uint_as_float(0x7f800000u))) raise_status(p.f.status, PIPE_ERR_INVALID_ARG);
              br.yq[static_cast<int64_t>(tok) * p.f.ldyq + c] = static_cast<int8_t>(quant_lane_exact(v, os));
              continue;
            }
            float* dst = br.y + static_cast<int64_t>(tok) * p.f.ldy + c;
            if (br.accumulate) v = __fadd_rn(*dst, v);
            *dst = v;
          }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(sums_free);
    }
  }
}

}  // namespace st

namespace st {

// What a launch has to ask the runtime, asked once per device (and once per kernel instantiation): the device's
// shared memory and SM count, an instantiation's static shared memory, and the largest dynamic shared memory its
// attribute has been raised to.
struct KernelInfo {
  const void* fn = nullptr;
  int fixed = 0, dyn_set = 0;
};
struct DeviceCache {
  std::mutex mu;
  bool ready = false;
  int smem_max = 0, sms = 0, n = 0;
  KernelInfo k[64];
};

static bool kernel_info(void (*kern)(const Params), int dyn_wanted_or_0, int* smem_max, int* sms, int* fixed) {
  constexpr int kMaxDevices = 64;
  static DeviceCache cache[kMaxDevices];
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return false;
  DeviceCache& c = cache[dev];
  std::lock_guard<std::mutex> lock(c.mu);
  if (!c.ready) {
    if (cudaDeviceGetAttribute(&c.smem_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) return false;
    if (cudaDeviceGetAttribute(&c.sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return false;
    c.ready = true;
  }
  KernelInfo* ki = nullptr;
  for (int i = 0; i < c.n; ++i)
    if (c.k[i].fn == reinterpret_cast<const void*>(kern)) ki = &c.k[i];
  if (!ki) {
    if (c.n >= 64) return false;
    cudaFuncAttributes fattr;
    if (cudaFuncGetAttributes(&fattr, kern) != cudaSuccess) return false;
    ki = &c.k[c.n++];
    ki->fn = reinterpret_cast<const void*>(kern);
    ki->fixed = static_cast<int>(fattr.sharedSizeBytes);
  }
  if (dyn_wanted_or_0 > ki->dyn_set) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn_wanted_or_0) != cudaSuccess) return false;
    ki->dyn_set = dyn_wanted_or_0;
  }
  *smem_max = c.smem_max;
  *sms = c.sms;
  *fixed = ki->fixed;
  return true;
}

}  // namespace st

static pipe_status launch_stream(const ForwardArgs& a, cudaStream_t stream, uint32_t split_mask = 0) {
  using namespace st;
  if (a.T > 16 || a.g % 8 != 0 || a.O % 8 != 0) return PIPE_ERR_UNSUPPORTED;
  if (a.ldxq % 16 != 0) return PIPE_ERR_UNSUPPORTED;   // tensor-map row pitch
  for (int m = 0; m < a.num_branches; ++m)
    if (reinterpret_cast<uintptr_t>(a.branch[m].xq) & 15) return PIPE_ERR_UNSUPPORTED;
  int max_cluster = 0;
  for (int m = 0; m < a.num_branches; ++m) max_cluster = max(max_cluster, a.branch[m].k_end - a.branch[m].k_begin);
  if (max_cluster > kMaxOrd) return PIPE_ERR_UNSUPPORTED;
  Params p;
  p.f = a;
  p.prefetch = a.blob_settled ? 1 : 0;
  p.split_mask = split_mask;
  const int nt = a.T <= 8 ? 1 : 2;
  const int np = max_cluster <= 2 ? 1 : (max_cluster <= 4 ? 2 : 4);
  const int spw = (np * nt <= 2) ? 5 : (np * nt == 4 ? 2 : 1);
  p.kblocks = ceil_div(a.I, 128);
  p.pk = 128 * a.bits / 8;
  p.shift = 8 - a.bits;
  p.kbps = a.bits == 2 ? 2 : 1;
  p.nstages = ceil_div(p.kblocks, p.kbps);
  p.nkmax = max_cluster;
  p.slabs_per_branch = a.O / 8;
  p.total_slabs = p.slabs_per_branch * a.num_branches;
  p.pass_slabs = kGroupWarps * spw;
  // (the kernel instantiation depends only on bits, tokens and orders, all known here)
  void (*kern)(const Params) = nullptr;
#define PIPE_ST_PICK(B, S)                                                                     \
  if (nt == 1) kern = np == 1 ? stream_forward_kernel<B, 1, 1, S, 0> : (np == 2 ? stream_forward_kernel<B, 1, 2, S, 0> : stream_forward_kernel<B, 1, 4, S, 0>); \
  else kern = np == 1 ? stream_forward_kernel<B, 2, 1, S, 0> : (np == 2 ? stream_forward_kernel<B, 2, 2, S, 0> : stream_forward_kernel<B, 2, 4, S, 0>);
  if (split_mask == 0) {
    if (a.bits == 8) { PIPE_ST_PICK(8, false) } else if (a.bits == 4) { PIPE_ST_PICK(4, false) } else { PIPE_ST_PICK(2, false) }
  } else {   // a summed ensemble on a shared input: the epilogue that closes the predictors' chains
    if (a.bits == 8) { PIPE_ST_PICK(8, true) } else if (a.bits == 4) { PIPE_ST_PICK(4, true) } else { PIPE_ST_PICK(2, true) }
  }
#undef PIPE_ST_PICK
  // the same kernel without per-slab branches, by slab slots per warp (one order pair; up to 8 tokens: 2 to 5 slots,
  // 9 to 16 tokens: 2 or 3 -- more would spill)
  auto full_kernel = [&](int slots) -> void (*)(const Params) {
    if (split_mask != 0 || np != 1) return nullptr;
#define PIPE_ST_FULL(B)                                                                                       \
  if (nt == 1) {                                                                                              \
    if (slots == 2) return stream_forward_kernel<B, 1, 1, false, 2>;                                          \
    if (slots == 3) return stream_forward_kernel<B, 1, 1, false, 3>;                                          \
    if (slots == 4) return stream_forward_kernel<B, 1, 1, false, 4>;                                          \
    if (slots == 5) return stream_forward_kernel<B, 1, 1, false, 5>;                                          \
  } else {                                                                                                    \
    if (slots == 2) return stream_forward_kernel<B, 2, 1, false, 2>;                                          \
    if (slots == 3) return stream_forward_kernel<B, 2, 1, false, 3>;                                          \
  }
    if (a.bits == 8) { PIPE_ST_FULL(8) } else if (a.bits == 4) { PIPE_ST_FULL(4) } else { PIPE_ST_FULL(2) }
#undef PIPE_ST_FULL
    return nullptr;
  };
  int smem_max = 0, sms = 0, fixed = 0;
  if (!kernel_info(kern, 0, &smem_max, &sms, &fixed)) return PIPE_ERR_CUDA;
  p.ctas_per_branch = sms / a.num_branches;
  if (p.ctas_per_branch < 1) return PIPE_ERR_UNSUPPORTED;
  if (p.ctas_per_branch > p.slabs_per_branch) p.ctas_per_branch = p.slabs_per_branch;
  const int grid = p.ctas_per_branch * a.num_branches;
  p.own_max = ceil_div(p.slabs_per_branch, p.ctas_per_branch);
  // one pass whose slab slots are (nearly) all taken: the kernel without per-slab branches, with just the slots it needs
  {
    const int slots = ceil_div(p.own_max, kGroupWarps);
    void (*kern_full)(const Params) = (p.own_max > kGroupWarps) ? full_kernel(slots) : nullptr;
    if (kern_full) {
      kern = kern_full;
      p.pass_slabs = kGroupWarps * slots;
      if (!kernel_info(kern, 0, &smem_max, &sms, &fixed)) return PIPE_ERR_CUDA;
    }
  }
  // passes a CTA may need: its range cut into pieces of pass_slabs
  if (ceil_div(p.own_max, p.pass_slabs) > kMaxPasses) return PIPE_ERR_UNSUPPORTED;
  // a stage holds one reduction block (two for 2-bit codes) of every order for the slabs of a pass, all kept
  const int pass_cap = p.pass_slabs < p.own_max ? p.pass_slabs : p.own_max;
  p.stage_bytes = round_up(p.kbps * (kXTile + pass_cap * 8 * max_cluster * p.pk), 1024);
  const int table_bytes = p.own_max * (max_cluster * 4 + max_cluster * 32 + 32) + kConsWarps * spw * (1 + 3 * max_cluster) * 4 +
                          p.pass_slabs * np * nt * 4 * 32 * 4;
  const int avail = smem_max - fixed - 1024 - round_up(table_bytes, 16);
  p.depth = avail / p.stage_bytes;
  if (p.depth > kMaxDepth) p.depth = kMaxDepth;
  // no more ring than the stages a CTA will ever fill
  const int most_stages = ceil_div(p.own_max, p.pass_slabs) * p.nstages;
  if (p.depth > round_up(most_stages, kProdWarps)) p.depth = round_up(most_stages, kProdWarps);
  p.depth -= p.depth % kProdWarps;   // every producer warp owns depth / kProdWarps slots
  if (p.depth < kProdWarps) return PIPE_ERR_UNSUPPORTED;
  const int dyn = 1024 + p.depth * p.stage_bytes + round_up(table_bytes, 16);
  for (int m = 0; m < a.num_branches; ++m)
    if (!make_tensor_map_2d_u8(&p.tmap_x[m], a.branch[m].xq, static_cast<uint64_t>(a.I), static_cast<uint64_t>(a.T),
                               static_cast<uint64_t>(a.ldxq), 128, 16, true))
      return PIPE_ERR_CUDA;
  if (!kernel_info(kern, dyn, &smem_max, &sms, &fixed)) return PIPE_ERR_CUDA;
  // (programmatic stream serialization: see the kernel's first lines)
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.gridDim = dim3(grid, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = dyn;
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, kern, p) != cudaSuccess) return PIPE_ERR_CUDA;
  count_launch(1);
  return launch_status();
}

pipe_status forward_stream(const ForwardArgs& a, cudaStream_t stream) {
  if (a.T == 0) return PIPE_OK;
  const bool sum_mode = a.num_branches > 1 && a.branch[1].accumulate;
  if (!sum_mode) return launch_stream(a, stream);
  // predictors that share input and step: one launch on the cluster of all orders, the chains added in registers
  if (!a.q8_out) {
    bool shared = true;
    for (int m = 1; m < a.num_branches; ++m)
      shared = shared && a.branch[m].xq == a.branch[0].xq && a.branch[m].sx == a.branch[0].sx &&
               a.branch[m].k_begin == a.branch[m - 1].k_end && a.branch[m].y == a.branch[0].y;
    const int k0 = a.branch[0].k_begin, k1 = a.branch[a.num_branches - 1].k_end;
    if (shared && k0 == 0) {
      ForwardArgs one = a;
      one.num_branches = 1;
      one.branch[0] = a.branch[0];
      one.branch[0].k_end = k1;
      one.branch[0].accumulate = 0;
      uint32_t split = 0;
      for (int m = 1; m < a.num_branches; ++m) split |= 1u << a.branch[m].k_begin;
      const pipe_status st = launch_stream(one, stream, split);
      if (st != PIPE_ERR_UNSUPPORTED) return st;
    }
  }
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
