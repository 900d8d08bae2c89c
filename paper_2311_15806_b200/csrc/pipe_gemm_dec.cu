// Small-token (T <= 16) tensor-core kernel of the expanded layer (Appendix B, Eq. 9; Sec. 3.2 for the branches):
// every packed weight is streamed from HBM exactly once and the whole call is bound by that stream.
//
// A UNIT is a run of channel groups of one branch whose stacked rows over the branch's orders fit 256 accumulator
// columns (the decode-unit tables of the blob, about one unit per SM); c CTAs (a cluster; c = 1 for wide layers)
// share a unit's reduction axis when whole units would be too narrow for the MMA.  For its part of the axis a CTA
// runs, per reduction block of 128 lanes:
//   warp 0      producer: bulk copies of the unit's packed rows -- one contiguous run per order, the streaming
//               layout being reduction-block-major -- and one tensor load of the 16 x 128-byte activation tile into a
//               deep ring of PACKED stages (they carry the bytes in flight that hide the HBM latency)
//   warps 4-11  unpack, two groups that take alternate blocks, four warps per block: packed stage -> int8 rows of the
//               swizzled B tile of an MMA stage (shift and mask, as in the other kernels)
//   warp 2      MMA issuer: tcgen05.mma kind::i8 with M = 64 (the tokens; only the first 16 rows of the A window are
//               loaded, what the other rows produce is never read), N = stacked rows, K = 32; owner of the tensor
//               memory (256 columns)
//   warp 12     (TMEM lane quarter 0) after the last MMA: the accumulators of the 16 token lanes go to shared memory
//               as [column][token]
// then, with the CTAs of a cluster adding their exact integer sums through distributed shared memory, all warps of
// the cluster's first CTA run the fixed-order fp32 epilogue, one (token, channel) per thread.
// Every wait is bounded.
#include "pipe_tc_common.cuh"

namespace pipe {

namespace dec {

using namespace tcc;

constexpr int kMaxTok = 16;
constexpr int kKStep = 128;
constexpr int kMaxN = 256;
constexpr int kMaxClusterOrders = 8;
constexpr int kUnpackWarps = 8;     // two groups of four
constexpr int kGroupWarps = 4;
constexpr int kFirstUnpackWarp = 4;
constexpr int kDrainWarp = 12;      // warp % 4 == 0: may read TMEM lanes 0..31
constexpr int kThreads = 32 * 13;
constexpr int kXBytes = kMaxTok * kKStep;          // 2 KiB: the loaded rows of the A window
constexpr int kBBytes = kMaxN * kKStep;            // 32 KiB
constexpr int kMmaStageBytes = kBBytes;            // an MMA stage is the widened B tile; the A window (64 rows, of
                                                   // which 16 are loaded) starts at the activation tile of the packed stage
constexpr int kMmaStages = 3;
constexpr int kMaxPackedStages = 8;
constexpr int kTmemCols = 256;
constexpr int kColmapEntries = kMaxClusterOrders * (PIPE_BLOCK_CHANNELS / 8);

struct Params {
  CUtensorMap tmap_x[PIPE_MAX_ORDERS];
  ForwardArgs f;
  int kblocks, split;
  int pk;                 // packed bytes of a row of a block
  int packed_stage_bytes; // activation tile + kMaxN * pk
  int packed_stages;
  int shift;
  const uint8_t* kbase;
  uint32_t koff[PIPE_MAX_ORDERS];
};

struct Unit {
  int m, k0, nk, c0, c1, n_total;
  int start[kMaxClusterOrders], rowbase[kMaxClusterOrders + 1];
};

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}

__device__ __forceinline__ void mma_i8_m64(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, bool accumulate) {
  mma_i8(d_tmem, adesc, bdesc, idesc, accumulate);
}

__device__ __forceinline__ void decode_unit(const Params& p, const int* unit_base, int unit, Unit& u) {
  int m = 0;
  while (m + 1 < p.f.num_branches && unit >= unit_base[m + 1]) ++m;
  const int cb = unit - unit_base[m];
  const BranchArgs& br = p.f.branch[m];
  u.m = m;
  u.k0 = br.k_begin;
  u.nk = br.k_end - br.k_begin;
  const int j0 = __ldg(br.dec + 1 + cb), j1 = __ldg(br.dec + 2 + cb);
  u.c0 = j0 * p.f.g;
  u.c1 = j1 * p.f.g;
  int rb = 0;
#pragma unroll
  for (int ko = 0; ko < kMaxClusterOrders; ++ko) {
    u.rowbase[ko] = rb;
    u.start[ko] = 0;
    if (ko < u.nk) {
      const int32_t* cum = p.f.order[u.k0 + ko].cum;
      const int lo = __ldg(cum + j0), hi = __ldg(cum + j1);
      u.start[ko] = lo * p.f.g;
      rb += (hi - lo) * p.f.g;
    }
  }
  u.rowbase[kMaxClusterOrders] = rb;
  u.n_total = rb;
}

template <int BITS, bool Q8>
__global__ void __launch_bounds__(kThreads, 1) dec_forward_kernel(const __grid_constant__ Params p) {
  constexpr int CPR = BITS;                // 16-byte chunks per packed row per block: 4 (int4), 2 (ternary)
  constexpr int RPI = 32 / CPR;            // rows per unpack item: 8, 16
  constexpr int PK = kKStep * BITS / 8;
  constexpr int OUT_PER_CHUNK = 8 / BITS;
  constexpr int ITEMS = kMaxN / RPI / kGroupWarps;   // items a warp may hold: 8, 4
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t pk_full[kMaxPackedStages], pk_empty[kMaxPackedStages];
  __shared__ uint64_t full[kMmaStages], done[kMmaStages], tfull_bar;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag_s;
  __shared__ int unit_base_s[PIPE_MAX_ORDERS + 1];
  __shared__ __align__(16) int16_t colmap[kColmapEntries];
  __shared__ __align__(16) float cscale[kMaxN];
  __shared__ __align__(16) int32_t accs[kMaxN][kMaxTok];   // [stacked row][token]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t mma_stage0 = smem_base;                                   // kMmaStages x {x tile, B tile}
  const uint32_t packed0 = smem_base + kMmaStages * kMmaStageBytes;        // packed_stages x packed rows
  uint8_t* mma_gen = smem_gen;
  uint8_t* packed_gen = smem_gen + kMmaStages * kMmaStageBytes;
  const int rank = static_cast<int>(cluster_rank());
  const int split = p.split;
  const int cluster_id = static_cast<int>(blockIdx.x) / split, num_clusters = static_cast<int>(gridDim.x) / split;

  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    int acc = 0;
    for (int m = 0; m < p.f.num_branches; ++m) {
      unit_base_s[m] = acc;
      acc += __ldg(p.f.branch[m].dec);
    }
    unit_base_s[p.f.num_branches] = acc;
    for (int s = 0; s < kMaxPackedStages; ++s) {
      mbar_init(smem_u32(&pk_full[s]), 1);
      mbar_init(smem_u32(&pk_empty[s]), kGroupWarps + 1);   // the unpack warps have read the rows, the MMAs the tokens
    }
    for (int s = 0; s < kMmaStages; ++s) {
      mbar_init(smem_u32(&full[s]), kGroupWarps);
      mbar_init(smem_u32(&done[s]), 1);
    }
    mbar_init(smem_u32(&tfull_bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 2) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = tmem_base_slot;
  const int num_units = unit_base_s[p.f.num_branches];
  volatile int* abort_flag = &abort_flag_s;
  // this CTA's share of the reduction axis
  const int kb_begin = static_cast<int>(static_cast<int64_t>(p.kblocks) * rank / split);
  const int kb_end = static_cast<int>(static_cast<int64_t>(p.kblocks) * (rank + 1) / split);
  const int nkb = kb_end - kb_begin;
  const int my_units = cluster_id < num_units ? (num_units - cluster_id + num_clusters - 1) / num_clusters : 0;

  // Block counters run on across the units of a CTA: block q (0, 1, ...) uses packed stage q % P and MMA stage q % 3.
  uint32_t ucount = 0;
  for (int unit = cluster_id; unit < num_units; unit += num_clusters, ++ucount) {
    Unit u;
    decode_unit(p, unit_base_s, unit, u);
    const BranchArgs& br = p.f.branch[u.m];
    const uint32_t q0 = ucount * static_cast<uint32_t>(nkb);   // first block counter of this unit
    const int n_mma = u.n_total > 0 ? (u.n_total + 15) & ~15 : 16;   // (a unit whose groups are all pruned still runs an MMA of the smallest shape)

    if (warp == 0) {
      // ---------------------------------------------------------------- weight producer
      // lane q < nk: the run of order q -- first 16-byte chunk at block 0, step per block, bytes, offset in the stage
      uint32_t run_off = 0, run_stp = 0, run_bytes = 0, run_dst = 0;
      {
        int lo = 0, hi = 0, st = 0;
#pragma unroll
        for (int q = 0; q < kMaxClusterOrders; ++q)
          if (q == lane) {
            lo = u.rowbase[q];
            hi = u.rowbase[q + 1];
            st = u.start[q];
          }
        if (lane < u.nk && hi > lo) {
          const uint32_t pk16 = PK >> 4;
          run_off = p.koff[u.k0 + lane] + static_cast<uint32_t>(st) * pk16;
          run_stp = static_cast<uint32_t>(p.f.order[u.k0 + lane].rows) * pk16;
          run_bytes = static_cast<uint32_t>(hi - lo) * PK;
          run_dst = static_cast<uint32_t>(lo) * PK;
        }
      }
      bool ok = true;
      for (int i = 0; i < nkb && ok; ++i) {
        const uint32_t q = q0 + i;
        const uint32_t ps = q % p.packed_stages, use = q / p.packed_stages;
        if (!mbar_wait(smem_u32(&pk_empty[ps]), (use & 1) ^ 1, abort_flag, p.f.status)) { ok = false; break; }
        if (lane == 0) {
          mbar_expect_tx(smem_u32(&pk_full[ps]), kXBytes + static_cast<uint32_t>(u.n_total) * PK);
          // the tokens' tile of this block; rows beyond T read zeros
          tma_load_2d(packed0 + ps * p.packed_stage_bytes, &p.tmap_x[u.m], (kb_begin + i) * kKStep, 0, smem_u32(&pk_full[ps]));
        }
        __syncwarp();
        if (run_bytes != 0) {
          const uint8_t* src = p.kbase + (static_cast<size_t>(run_off + static_cast<uint32_t>(kb_begin + i) * run_stp) << 4);
          asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                           packed0 + ps * p.packed_stage_bytes + kXBytes + run_dst),
                       "l"(src), "r"(run_bytes), "r"(smem_u32(&pk_full[ps]))
                       : "memory");
        }
        __syncwarp();
      }
    } else if (warp == 2) {
      // ---------------------------------------------------------------- MMA issuer
      if (lane == 0) {
        const uint32_t idesc = idesc_i8(64, n_mma);
        bool ok = true;
        for (int i = 0; i < nkb; ++i) {
          const uint32_t q = q0 + i;
          const uint32_t s = q % kMmaStages, use = q / kMmaStages;
          if (!mbar_wait(smem_u32(&full[s]), use & 1, abort_flag, p.f.status)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t ps = q % p.packed_stages;
          const uint64_t adesc = smem_desc_sw128(packed0 + ps * p.packed_stage_bytes);
          const uint64_t bdesc = smem_desc_sw128(mma_stage0 + s * kMmaStageBytes);
#pragma unroll
          for (int k = 0; k < kKStep / 32; ++k)
            mma_i8_m64(tmem_base, adesc + static_cast<uint64_t>(k * 2), bdesc + static_cast<uint64_t>(k * 2), idesc, (i | k) != 0);
          mma_commit(smem_u32(&done[s]));
          mma_commit(smem_u32(&pk_empty[ps]));
        }
        if (ok) mma_commit(smem_u32(&tfull_bar));
      }
    } else if (warp >= kFirstUnpackWarp && warp < kFirstUnpackWarp + kUnpackWarps) {
      // ---------------------------------------------------------------- unpack
      const int uw = warp - kFirstUnpackWarp, grp = uw / kGroupWarps, wg = uw % kGroupWarps;
      const int lr = lane / CPR, lc = lane % CPR;
      const int sw = lr & 7;
      const uint32_t out_lane = static_cast<uint32_t>((lr >> 3) * 1024 + (lr & 7) * 128);
      const int n_items = (u.n_total + RPI - 1) / RPI;   // items of the block; this warp takes wg, wg + 4, ...
      // (a unit's first block may belong to either group: the parity follows the running block counter)
      for (int i = 0; i < nkb; ++i) {
        const uint32_t q = q0 + i;
        if (static_cast<int>(q & 1u) != grp) continue;
        const uint32_t ps = q % p.packed_stages, puse = q / p.packed_stages;
        const uint32_t s = q % kMmaStages, use = q / kMmaStages;
        if (!mbar_wait(smem_u32(&pk_full[ps]), puse & 1, abort_flag, p.f.status)) break;
        uint4 w[ITEMS];
        const uint4* pk_in = reinterpret_cast<const uint4*>(packed_gen + static_cast<size_t>(ps) * p.packed_stage_bytes + kXBytes) + lane;
#pragma unroll
        for (int j = 0; j < ITEMS; ++j) {
          const int item = wg + kGroupWarps * j;
          if (item < n_items) w[j] = pk_in[item * 32];
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&pk_empty[ps]));   // the packed stage may be refilled
        if (!mbar_wait(smem_u32(&done[s]), (use & 1) ^ 1, abort_flag, p.f.status)) break;
        uint8_t* bt = mma_gen + static_cast<size_t>(s) * kMmaStageBytes;
#pragma unroll
        for (int j = 0; j < ITEMS; ++j) {
          const int item = wg + kGroupWarps * j;
          if (item >= n_items) continue;
          uint8_t* row = bt + item * (RPI >> 3) * 1024 + out_lane;
          const int c0 = lc * OUT_PER_CHUNK;
          if (BITS == 4) {
            const uint32_t m4 = 0xF0F0F0F0u;
            const uint4 v0 = make_uint4((w[j].x << 4) & m4, w[j].x & m4, (w[j].y << 4) & m4, w[j].y & m4);
            const uint4 v1 = make_uint4((w[j].z << 4) & m4, w[j].z & m4, (w[j].w << 4) & m4, w[j].w & m4);
            *reinterpret_cast<uint4*>(row + ((c0 ^ sw) << 4)) = v0;
            *reinterpret_cast<uint4*>(row + (((c0 + 1) ^ sw) << 4)) = v1;
          } else {
            const uint32_t m2c = 0xC0C0C0C0u;
            const uint32_t ww[4] = {w[j].x, w[j].y, w[j].z, w[j].w};
#pragma unroll
            for (int h = 0; h < 4; ++h) {
              const uint4 v = make_uint4((ww[h] << 6) & m2c, (ww[h] << 4) & m2c, (ww[h] << 2) & m2c, ww[h] & m2c);
              *reinterpret_cast<uint4*>(row + (((c0 + h) ^ sw) << 4)) = v;
            }
          }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&full[s]));
      }
    } else if (warp == 3) {
      // ---------------------------------------------------------------- tables of the unit (first CTA of the cluster)
      if (rank == 0) {
        const float sx = __ldg(br.sx);
        const int nch = (u.c1 - u.c0) >> 3;
        for (int e = lane; e < kMaxClusterOrders * nch; e += 32) {
          const int cc = e / kMaxClusterOrders, ko = e % kMaxClusterOrders;
          int col = -1;
          if (ko < u.nk) {
            int rb = 0, st = 0;
#pragma unroll
            for (int q = 0; q < kMaxClusterOrders; ++q)
              if (q == ko) {
                rb = u.rowbase[q];
                st = u.start[q];
              }
            const int32_t* cum = p.f.order[u.k0 + ko].cum;
            const int c = u.c0 + 8 * cc;
            const int j = c / p.f.g;
            const int lo = __ldg(cum + j), hi = __ldg(cum + j + 1);
            if (hi > lo) col = rb + lo * p.f.g + c % p.f.g - st;
          }
          colmap[e] = static_cast<int16_t>(col);
        }
        for (int r = lane; r < u.n_total; r += 32) {
          int rb = 0, st = u.start[0];
          const float* sc = p.f.order[u.k0].scales;
#pragma unroll
          for (int q = 1; q < kMaxClusterOrders; ++q)
            if (q < u.nk && r >= u.rowbase[q]) {
              rb = u.rowbase[q];
              st = u.start[q];
              sc = p.f.order[u.k0 + q].scales;
            }
          cscale[r] = __fmul_rn(__ldg(sc + st + (r - rb)), sx);
        }
      }
    } else if (warp == kDrainWarp) {
      // ---------------------------------------------------------------- accumulators -> shared memory
      if (mbar_wait(smem_u32(&tfull_bar), ucount & 1, abort_flag, p.f.status)) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        for (int c = 0; c < n_mma; c += 16) {
          int v[16];
          // TMEM lanes 0..31 of this warp's quarter; lanes 0..15 hold the tokens
          asm volatile(
              "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
              : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
                "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
              : "r"(tmem_base + c)
              : "memory");
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
          if (lane < kMaxTok) {
#pragma unroll
            for (int e = 0; e < 16; ++e) accs[c + e][lane] = v[e] >> p.shift;   // exact: the sums carry a factor 2^shift
          }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      }
    }

    // ------------------------------------------------------------------ reduction over the cluster and epilogue
    __syncthreads();
    if (split > 1) cluster_sync_all();   // every CTA's integer sums are in its shared memory
    if (rank == 0 && !*abort_flag) {
      const int nch = (u.c1 - u.c0) >> 3;
      const int nchan = u.c1 - u.c0;
      const bool add_bias = br.add_bias && p.f.bias;
      float ostep = 0.f;
      if constexpr (Q8) {
        ostep = __ldg(br.out_scale);
        if (!(ostep >= 0.f && ostep < __uint_as_float(0x7f800000u)) && threadIdx.x == 0) raise_status(p.f.status, PIPE_ERR_INVALID_ARG);
      }
      // one (token, channel) per thread and trip, channels fastest
      for (int idx = threadIdx.x; idx < nchan * kMaxTok; idx += kThreads) {
        const int t = idx / nchan, ch = idx - t * nchan;
        if (t >= p.f.T) continue;
        const int cc = ch >> 3, e = ch & 7;
        float y = 0.f;
#pragma unroll
        for (int ko = 0; ko < kMaxClusterOrders; ++ko) {
          if (ko >= u.nk) break;
          const int col = colmap[cc * kMaxClusterOrders + ko];
          if (col < 0) continue;
          int a = accs[col + e][t];
          for (int r = 1; r < split; ++r) {
            int other;
            const uint32_t addr = map_to_cta(smem_u32(&accs[col + e][t]), static_cast<uint32_t>(r));
            asm volatile("ld.shared::cluster.s32 %0, [%1];" : "=r"(other) : "r"(addr));
            a += other;
          }
          y = __fmaf_rn(__int2float_rn(a), cscale[col + e], y);
          if (p.f.partials) {
            int rb = 0, st = 0;
#pragma unroll
            for (int q = 0; q < kMaxClusterOrders; ++q)
              if (q == ko) {
                rb = u.rowbase[q];
                st = u.start[q];
              }
            p.f.partials[static_cast<int64_t>(t) * p.f.total_rows + p.f.order[u.k0 + ko].row_off + (col + e - rb + st)] = a;
          }
        }
        const int c = u.c0 + ch;
        if (add_bias) y = __fadd_rn(y, __ldg(p.f.bias + c));
        if constexpr (Q8) {
          y = apply_activation(y, p.f.relu);
          br.yq[static_cast<int64_t>(t) * p.f.ldyq + c] = static_cast<int8_t>(quant_lane_exact(y, ostep));
        } else {
          float* dst = br.y + static_cast<int64_t>(t) * p.f.ldy + c;
          *dst = br.accumulate ? __fadd_rn(*dst, y) : y;
        }
      }
      (void)nch;
    }
    // the peers' sums have been read (and this CTA's tables and sums may be overwritten by its next unit)
    if (split > 1) cluster_sync_all();
    __syncthreads();
  }
  (void)my_units;

  // ---------------------------------------------------------------------- teardown
  // after an abort, bulk copies may still be in flight into this CTA's shared memory: give them a bounded time
  if (*abort_flag && threadIdx.x == 0) {
    const long long t0 = clock64();
    while (clock64() - t0 < 20000000ll) {
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 2) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

struct DeviceSetup {
  int smem_max = 0, sms = 0, fixed = 0;
  pipe_status status = PIPE_ERR_CUDA;
};

template <typename K>
static bool prepare_kernel(K kern, int dyn) {
  return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn) == cudaSuccess &&
         cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess;
}

static const DeviceSetup& device_setup() {
  constexpr int kMaxDevices = 64;
  static DeviceSetup setups[kMaxDevices];
  static std::once_flag once[kMaxDevices];
  static const DeviceSetup bad;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return bad;
  std::call_once(once[dev], [dev] {
    DeviceSetup& d = setups[dev];
    if (cudaDeviceGetAttribute(&d.smem_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) return;
    if (cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return;
    cudaFuncAttributes fa;
    if (cudaFuncGetAttributes(&fa, dec_forward_kernel<4, false>) != cudaSuccess) return;
    d.fixed = static_cast<int>(fa.sharedSizeBytes);
    const int dyn = d.smem_max - d.fixed;
    if (!prepare_kernel(dec_forward_kernel<4, false>, dyn) || !prepare_kernel(dec_forward_kernel<4, true>, dyn) ||
        !prepare_kernel(dec_forward_kernel<2, false>, dyn) || !prepare_kernel(dec_forward_kernel<2, true>, dyn))
      return;
    d.status = PIPE_OK;
  });
  return setups[dev];
}

}  // namespace dec

static pipe_status launch_dec(const ForwardArgs& a, cudaStream_t stream) {
  using namespace dec;
  if (a.T > kMaxTok || a.conv_on) return PIPE_ERR_UNSUPPORTED;
  if (a.bits == 8) return PIPE_ERR_UNSUPPORTED;   // int8 rows need no widening; the weight-streaming kernel takes them
  if (a.decode_split < 1 || a.decode_split > 4) return PIPE_ERR_UNSUPPORTED;
  if (a.g % 8 != 0 || (a.bits == 2 && a.g % 16 != 0)) return PIPE_ERR_UNSUPPORTED;
  if (a.ldxq % 16 != 0) return PIPE_ERR_UNSUPPORTED;
  for (int m = 0; m < a.num_branches; ++m) {
    if (!a.branch[m].dec || a.branch[m].zp) return PIPE_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(a.branch[m].xq) & 15) return PIPE_ERR_UNSUPPORTED;
    if (a.branch[m].k_end - a.branch[m].k_begin > kMaxClusterOrders) return PIPE_ERR_UNSUPPORTED;
  }
  const DeviceSetup& ds = device_setup();
  if (ds.status != PIPE_OK) return ds.status;

  Params p;
  p.f = a;
  p.kblocks = ceil_div(a.I, kKStep);
  p.split = a.decode_split < p.kblocks ? a.decode_split : 1;
  p.pk = kKStep * a.bits / 8;
  p.packed_stage_bytes = kXBytes + kMaxN * p.pk;
  p.shift = 8 - a.bits;
  const int room = ds.smem_max - ds.fixed - 1024 - kMmaStages * kMmaStageBytes;
  p.packed_stages = room / p.packed_stage_bytes;
  if (p.packed_stages > kMaxPackedStages) p.packed_stages = kMaxPackedStages;
  if (p.packed_stages < 2) return PIPE_ERR_UNSUPPORTED;
  p.packed_stages &= ~1;   // an even count: a stage then always belongs to the same unpack group
  const int dyn = 1024 + kMmaStages * kMmaStageBytes + p.packed_stages * p.packed_stage_bytes;
  int k_lo = PIPE_MAX_ORDERS, k_hi = 0;
  for (int m = 0; m < a.num_branches; ++m) {
    k_lo = min(k_lo, a.branch[m].k_begin);
    k_hi = max(k_hi, a.branch[m].k_end);
  }
  const uint8_t* kbase = a.order[k_lo].kcodes;
  for (int k = k_lo; k < k_hi; ++k) kbase = a.order[k].kcodes < kbase ? a.order[k].kcodes : kbase;
  p.kbase = kbase;
  for (int k = k_lo; k < k_hi; ++k) {
    const uint64_t d = static_cast<uint64_t>(a.order[k].kcodes - kbase);
    const uint64_t end = (d + static_cast<uint64_t>(a.order[k].rows) * a.kernel_row_bytes) >> 4;
    if ((d & 15) || end >= 0xffffffffull) return PIPE_ERR_UNSUPPORTED;
    p.koff[k] = static_cast<uint32_t>(d >> 4);
  }
  for (int m = 0; m < a.num_branches; ++m)
    if (!make_map_2d(&p.tmap_x[m], a.branch[m].xq, static_cast<uint64_t>(a.I), static_cast<uint64_t>(a.T),
                     static_cast<uint64_t>(a.ldxq), kKStep, kMaxTok, CU_TENSOR_MAP_SWIZZLE_128B))
      return PIPE_ERR_CUDA;

  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = p.split;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.gridDim = dim3((ds.sms / p.split) * p.split, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = dyn;
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e;
  if (a.bits == 4) e = a.q8_out ? cudaLaunchKernelEx(&cfg, dec_forward_kernel<4, true>, p) : cudaLaunchKernelEx(&cfg, dec_forward_kernel<4, false>, p);
  else e = a.q8_out ? cudaLaunchKernelEx(&cfg, dec_forward_kernel<2, true>, p) : cudaLaunchKernelEx(&cfg, dec_forward_kernel<2, false>, p);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return PIPE_ERR_UNSUPPORTED;   // e.g. this cluster size cannot be co-scheduled here: another kernel takes the call
  }
  count_launch(1);
  return launch_status();
}

pipe_status forward_decode_tc(const ForwardArgs& a, cudaStream_t stream) {
  if (a.T == 0) return PIPE_OK;
  const bool sum_mode = a.num_branches > 1 && a.branch[1].accumulate;
  if (!sum_mode) return launch_dec(a, stream);
  // Summed ensemble: one launch per branch, in order, so that y = ((y_1 + y_2) + ...) is formed in a fixed order
  // (each branch then runs under the plan that was laid out for all of them, which only costs balance).
  for (int m = 0; m < a.num_branches; ++m) {
    ForwardArgs one = a;
    one.num_branches = 1;
    one.branch[0] = a.branch[m];
    pipe_status st = launch_dec(one, stream);
    if (st != PIPE_OK) return st;
  }
  return PIPE_OK;
}

}  // namespace pipe
