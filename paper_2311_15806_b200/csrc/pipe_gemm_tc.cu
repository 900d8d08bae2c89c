// tcgen05 tensor-core kernel of the expanded layer (Appendix B, Eq. 9; Sec. 3.2 for the branches).
//
// One persistent CTA per SM walks tiles (branch, block of BN output channels, 128 tokens).
// For a tile, the rows of ALL orders of the branch that fall into the channel block are stacked
// into one int8 B operand (order 1: BN rows; a sparse order: only its kept rows, found through
// the prefix counts), so one chain of tcgen05.mma kind::i8 instructions (M = 128 tokens,
// N = stacked rows, K = 32) fills one int32 accumulator region per order in TMEM while the
// activation tile is staged once per reduction step.  Three shared-memory rings decouple the
// latencies: activation tiles (TMA, 128B swizzle), packed weight rows (one bulk copy per order and
// reduction block: the streaming layout is reduction-block major, so the rows of a tile are
// contiguous), and unpacked int8 B tiles.  Warp roles:
//   warp 0      producer of the activation ring (TMA tensor loads)
//   warp 10     producer of the packed-weight ring (bulk copies)
//   warps 2-5   unpack: packed int8/int4/ternary rows -> int8 lanes in the swizzled B tile
//               (shift + mask only; sub-byte codes arrive multiplied by 2^(8-b))
//   warp 1      MMA issuer (one lane), owns the TMEM allocation (2 x 256 columns, double buffered)
//   warps 6-9   epilogue: tcgen05.ld the accumulators of each order, shift back, scale by
//               s_k * lambda_x and add in ascending order with one FMA per term, store fp32
// Every wait on an mbarrier is bounded; on expiry the CTA raises PIPE_ERR_TIMEOUT, all roles
// leave their loops, outstanding copies are drained, TMEM is freed and the kernel returns.
#include <cuda.h>

#include <mutex>

#include "pipe_common.cuh"

namespace pipe {

namespace tc {

constexpr int kTileM = 128;          // tokens per tile
constexpr int kKStep = 128;          // reduction bytes (int8 lanes) per stage
constexpr int kMaxN = 256;           // stacked weight rows per tile
constexpr int kMaxClusterOrders = 8;
constexpr int kThreads = 352;
constexpr int kUnpackThreads = 128;
constexpr int kEpiThreads = 128;
constexpr int kABytes = kTileM * kKStep;       // 16 KiB
constexpr int kBtBytes = kMaxN * kKStep;       // 32 KiB
constexpr int kTmemCols = 512;
constexpr int kAccCols = 256;
constexpr int kMaxRing = 8;
constexpr int kBtRing = 2;
constexpr uint64_t kWaitLimitNs = 1000000000ull;  // 1 s per wait

struct Params {
  CUtensorMap tmap_a[PIPE_MAX_ORDERS];  // one per branch input
  ForwardArgs f;
  int BN, ncb, ntt, num_tiles, kblocks;
  int na, ns;             // depth of the activation ring and of the packed-weight ring
  int pk;                 // packed bytes of one row of one reduction block (128*b/8)
  int stg_bytes;          // one packed-weight stage: kMaxN * pk
  int a_off, s_off, bt_off;  // ring offsets in dynamic shared memory (1 KiB aligned)
  int shift;              // 8 - b
};

struct TileMeta {
  int m, cb, tt;
  int nk;                              // orders in this branch
  int k0;                              // first order
  int start[kMaxClusterOrders];        // first compacted row of the channel block in order k
  int n[kMaxClusterOrders];            // rows of order k in the block
  int rowbase[kMaxClusterOrders + 1];  // row offset of order k in the stacked B tile / accumulator
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
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

// Bounded wait.  Returns false when the CTA is aborting (this wait or another one expired).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status) {
  if (mbar_try(bar, parity)) return true;
  const uint64_t t0 = global_ns();
  while (true) {
    if (mbar_try(bar, parity)) return true;
    if (*abort_flag) return false;
    if (global_ns() - t0 > kWaitLimitNs) {
      *abort_flag = 1;
      raise_status(status, PIPE_ERR_TIMEOUT);
      return false;
    }
  }
}

// After the last issue: wait (bounded) until the copies of the last `depth` ring slots have landed,
// so that no copy is still writing into this CTA's shared memory when it exits.
__device__ __forceinline__ void drain_ring(uint32_t full0, uint32_t issued, int depth) {
  for (uint32_t j = (issued > static_cast<uint32_t>(depth) ? issued - depth : 0); j < issued; ++j) {
    const int s = j % depth;
    const uint32_t ph = (j / depth) & 1;
    const uint64_t t0 = global_ns();
    while (!mbar_try(full0 + 8u * s, ph) && global_ns() - t0 < kWaitLimitNs) {
    }
  }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar)
      : "memory");
}

// Contiguous global -> shared copy (both addresses 16-byte aligned, size a multiple of 16).
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar)
               : "memory");
}

// Shared-memory matrix descriptor of a K-major int8 tile whose rows are 128 bytes, stored as
// 8-row atoms of 1024 bytes with the 128-byte swizzle (the layout TMA writes with SWIZZLE_128B).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((addr & 0x3FFFFu) >> 4);  // start address
  d |= static_cast<uint64_t>(1) << 16;                 // leading byte offset (unused for swizzled K-major)
  d |= static_cast<uint64_t>(1024 >> 4) << 32;         // stride byte offset: next 8-row atom
  d |= static_cast<uint64_t>(1) << 46;                 // descriptor version of this architecture
  d |= static_cast<uint64_t>(2) << 61;                 // 128-byte swizzle
  return d;
}

// Instruction descriptor: D = int32, A and B = signed int8, both K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t idesc_i8(int n) {
  return (2u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(kTileM >> 4) << 24);
}

__device__ __forceinline__ void mma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, bool accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.u32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate ? 1u : 0u)
      : "memory");
}

__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld8(uint32_t taddr, int (&v)[8]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
               : "r"(taddr)
               : "memory");
}

__device__ __forceinline__ void decode_tile(const Params& p, int tile, TileMeta& t) {
  t.tt = tile % p.ntt;
  const int rest = tile / p.ntt;
  t.cb = rest % p.ncb;
  t.m = rest / p.ncb;
  const BranchArgs& br = p.f.branch[t.m];
  t.k0 = br.k_begin;
  t.nk = br.k_end - br.k_begin;
  const int c0 = t.cb * p.BN;
  const int c1 = min(c0 + p.BN, p.f.O);
  const int j0 = c0 / p.f.g, j1 = c1 / p.f.g;
  int rb = 0;
#pragma unroll
  for (int ko = 0; ko < kMaxClusterOrders; ++ko) {
    t.rowbase[ko] = rb;
    if (ko < t.nk) {
      const int32_t* cum = p.f.order[t.k0 + ko].cum;
      const int lo = __ldg(cum + j0), hi = __ldg(cum + j1);
      t.start[ko] = lo * p.f.g;
      t.n[ko] = (hi - lo) * p.f.g;
      rb += t.n[ko];
    } else {
      t.start[ko] = 0;
      t.n[ko] = 0;
    }
  }
  t.rowbase[kMaxClusterOrders] = rb;
}

struct Rings {
  uint32_t a_full0, a_empty0, s_full0, s_empty0, bt_ready0, bt_empty0, tfull0, tempty0;  // barrier i is 8*i bytes on
  uint32_t a0, s0, bt0;   // shared addresses of slot 0 of each ring
  uint8_t* s_gen;         // generic addresses of slot 0 of the packed-weight and B-tile rings
  uint8_t* bt_gen;
  volatile int* abort_flag;
};

// Unpack role (128 threads): for every reduction block turn the packed weight rows of the tile
// into the 128B-swizzled int8 B tile.  Work items are (stacked row, 16-byte chunk); which items a
// thread owns depends only on the tile, so their offsets are computed once per tile.
template <int BITS>
__device__ __forceinline__ void unpack_role(const Params& p, const Rings& g, int ut) {
  constexpr int CPR = BITS;              // 16-byte chunks per packed row per block: 8, 4, 2
  constexpr int CPR_LOG = (BITS == 8) ? 3 : (BITS == 4 ? 2 : 1);
  constexpr int ITEMS = 2 * CPR;         // kMaxN * CPR / kUnpackThreads
  constexpr int OUT_PER_CHUNK = 8 / BITS;  // 16-byte vectors written per chunk read
  constexpr int PK = 128 * BITS / 8;
  uint32_t it = 0;
  for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x) {
    TileMeta t;
    decode_tile(p, tile, t);
    const int n_total = t.rowbase[kMaxClusterOrders];
    int src_off[ITEMS], dst_off0[ITEMS], sw16[ITEMS];
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) {
      const int idx = ut + i * kUnpackThreads;
      const int r = idx >> CPR_LOG, c = idx & (CPR - 1);
      src_off[i] = (r < n_total) ? r * PK + c * 16 : -1;
      dst_off0[i] = (r >> 3) * 1024 + (r & 7) * 128;
      sw16[i] = ((c * OUT_PER_CHUNK) << 8) | (r & 7);
    }
    for (int kb = 0; kb < p.kblocks; ++kb, ++it) {
      const int ss = it % p.ns, bs = it % kBtRing;
      const uint32_t sph = (it / p.ns) & 1, bph = (it / kBtRing) & 1;
      if (!mbar_wait(g.s_full0 + 8u * ss, sph, g.abort_flag, p.f.status)) return;
      const uint8_t* stage = g.s_gen + static_cast<size_t>(ss) * p.stg_bytes;
      uint4 w[ITEMS];
#pragma unroll
      for (int i = 0; i < ITEMS; ++i)
        if (src_off[i] >= 0) w[i] = *reinterpret_cast<const uint4*>(stage + src_off[i]);
      if (!mbar_wait(g.bt_empty0 + 8u * bs, bph ^ 1, g.abort_flag, p.f.status)) return;
      uint8_t* bt = g.bt_gen + static_cast<size_t>(bs) * kBtBytes;
#pragma unroll
      for (int i = 0; i < ITEMS; ++i) {
        if (src_off[i] < 0) continue;
        uint8_t* row = bt + dst_off0[i];
        const int c0 = sw16[i] >> 8, sw = sw16[i] & 7;
        if (BITS == 8) {
          *reinterpret_cast<uint4*>(row + ((c0 ^ sw) << 4)) = w[i];
        } else if (BITS == 4) {
          const uint32_t m4 = 0xF0F0F0F0u;
          const uint4 v0 = make_uint4((w[i].x << 4) & m4, w[i].x & m4, (w[i].y << 4) & m4, w[i].y & m4);
          const uint4 v1 = make_uint4((w[i].z << 4) & m4, w[i].z & m4, (w[i].w << 4) & m4, w[i].w & m4);
          *reinterpret_cast<uint4*>(row + ((c0 ^ sw) << 4)) = v0;
          *reinterpret_cast<uint4*>(row + (((c0 + 1) ^ sw) << 4)) = v1;
        } else {
          const uint32_t m2 = 0xC0C0C0C0u;
          const uint32_t ww[4] = {w[i].x, w[i].y, w[i].z, w[i].w};
#pragma unroll
          for (int h = 0; h < 4; ++h) {
            const uint4 v = make_uint4((ww[h] << 6) & m2, (ww[h] << 4) & m2, (ww[h] << 2) & m2, ww[h] & m2);
            *reinterpret_cast<uint4*>(row + (((c0 + h) ^ sw) << 4)) = v;
          }
        }
      }
      mbar_arrive(g.s_empty0 + 8u * ss);   // the packed rows are in registers / already consumed
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic writes -> visible to the MMA's reads
      mbar_arrive(g.bt_ready0 + 8u * bs);
    }
  }
}

struct EpiCtx {
  uint32_t tmem_base, tfull0, tempty0;
  volatile int* abort_flag;
  int warp, lane;
  int16_t* colmap;
  int32_t* crowmap;
  float* cscale;
};

// Epilogue role (4 warps, one TMEM lane quarter each; a lane owns one token row of the tile).
// NKMAX = most orders a branch may have at this channel-block width (NKMAX * BN = 256).
// Before the accumulators are ready the warp prepares, from the prefix counts, where each
// (order, 8-channel chunk) sits in the accumulator and the products s_k * lambda_x of all stacked
// rows, so that the drain loop has no dependent global loads.
template <int NKMAX>
__device__ __forceinline__ void epilogue_role(const Params& p, const EpiCtx& x) {
  constexpr int NCH = 32 / NKMAX;   // 8-channel chunks per channel block (BN / 8)
  constexpr int CH = 8 / NKMAX;     // chunks drained per iteration (64 accumulator registers)
  const int q = x.warp & 3;         // TMEM lane quarter this warp may read
  const int lane = x.lane;
  const int row_in_tile = q * 32 + lane;
  uint32_t tcount = 0;
  const bool y_vec = (p.f.ldy % 4 == 0);
  for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x, ++tcount) {
    TileMeta t;
    decode_tile(p, tile, t);
    const BranchArgs& br = p.f.branch[t.m];
    const int buf = tcount & 1;
    const uint32_t aph = (tcount >> 1) & 1;
    const float sx = __ldg(br.sx);
    const int c0 = t.cb * p.BN;
    const int c1 = min(c0 + p.BN, p.f.O);
    const int nch = (c1 - c0) >> 3;
    const int n_total = t.rowbase[kMaxClusterOrders];
    __syncwarp();
    {
      const int ko = lane / NCH, cc = lane % NCH;
      int col = -1, crow = 0;
      if (ko < t.nk && cc < nch) {
        int rb = 0, st = 0;
        const int32_t* cum = nullptr;
#pragma unroll
        for (int u = 0; u < NKMAX; ++u)
          if (u == ko) {
            rb = t.rowbase[u];
            st = t.start[u];
            cum = p.f.order[t.k0 + u].cum;
          }
        const int c = c0 + 8 * cc;
        const int j = c / p.f.g;
        const int lo = __ldg(cum + j), hi = __ldg(cum + j + 1);
        if (hi > lo) {
          crow = lo * p.f.g + c % p.f.g;
          col = rb + crow - st;
        }
      }
      x.colmap[lane] = static_cast<int16_t>(col);
      x.crowmap[lane] = crow;
      for (int r = lane; r < n_total; r += 32) {
        int rb = 0, st = t.start[0];
        const float* sc = p.f.order[t.k0].scales;
#pragma unroll
        for (int u = 1; u < NKMAX; ++u)
          if (u < t.nk && r >= t.rowbase[u]) {
            rb = t.rowbase[u];
            st = t.start[u];
            sc = p.f.order[t.k0 + u].scales;
          }
        x.cscale[r] = __fmul_rn(__ldg(sc + st + (r - rb)), sx);
      }
    }
    __syncwarp();
    if (!mbar_wait(x.tfull0 + 8u * buf, aph, x.abort_flag, p.f.status)) break;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const int64_t tok = static_cast<int64_t>(t.tt) * kTileM + row_in_tile;
    const bool tok_ok = tok < p.f.T;
    const uint32_t tbase = x.tmem_base + (static_cast<uint32_t>(q * 32) << 16) + buf * kAccCols;
    float* yrow = br.y + tok * p.f.ldy;
    const bool vec_ok = y_vec && ((reinterpret_cast<uintptr_t>(br.y) & 15) == 0);
    for (int cg = 0; cg < nch; cg += CH) {
      int acc[CH][NKMAX][8];
      int cols[CH][NKMAX];
#pragma unroll
      for (int u = 0; u < CH; ++u)
#pragma unroll
        for (int ko = 0; ko < NKMAX; ++ko) {
          cols[u][ko] = (cg + u < nch) ? x.colmap[ko * NCH + cg + u] : -1;
          if (cols[u][ko] >= 0) tmem_ld8(tbase + cols[u][ko], acc[u][ko]);
        }
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
      for (int u = 0; u < CH; ++u) {
        if (cg + u >= nch) continue;
        const int c = c0 + 8 * (cg + u);
        float y[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) y[e] = 0.f;
#pragma unroll
        for (int ko = 0; ko < NKMAX; ++ko) {
          if (cols[u][ko] < 0) continue;
          const float* cs = x.cscale + cols[u][ko];
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const int a = acc[u][ko][e] >> p.shift;  // exact: the accumulator holds 2^shift times the sum
            acc[u][ko][e] = a;
            y[e] = __fmaf_rn(__int2float_rn(a), cs[e], y[e]);
          }
          if (p.f.partials && tok_ok) {
            int32_t* prow = p.f.partials + tok * p.f.total_rows + p.f.order[t.k0 + ko].row_off + x.crowmap[ko * NCH + cg + u];
#pragma unroll
            for (int e = 0; e < 8; ++e) prow[e] = acc[u][ko][e];
          }
        }
        if (tok_ok) {
          if (br.add_bias && p.f.bias) {
#pragma unroll
            for (int e = 0; e < 8; ++e) y[e] = __fadd_rn(y[e], __ldg(p.f.bias + c + e));
          }
          if (br.accumulate) {
#pragma unroll
            for (int e = 0; e < 8; ++e) y[e] = __fadd_rn(yrow[c + e], y[e]);
          }
          if (vec_ok) {
            *reinterpret_cast<float4*>(yrow + c) = make_float4(y[0], y[1], y[2], y[3]);
            *reinterpret_cast<float4*>(yrow + c + 4) = make_float4(y[4], y[5], y[6], y[7]);
          } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) yrow[c + e] = y[e];
          }
        }
      }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    mbar_arrive(x.tempty0 + 8u * buf);
  }
}

__global__ void __launch_bounds__(kThreads, 1) tc_forward_kernel(const __grid_constant__ Params p) {
  extern __shared__ uint8_t smem_raw[];
  // a_full[8] a_empty[8] s_full[8] s_empty[8] bt_ready[2] bt_empty[2] tmem_full[2] tmem_empty[2]
  __shared__ uint64_t bars[4 * kMaxRing + 8];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag_s;
  __shared__ int16_t epi_colmap[4][32];     // per epilogue warp: accumulator column of (order, 8-channel chunk) or -1
  __shared__ int32_t epi_crowmap[4][32];    // ... and its compacted row in that order
  __shared__ float epi_cscale[4][kMaxN];    // per epilogue warp: s_k * lambda_x of every stacked row

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar0 = smem_u32(bars);
  Rings g;
  g.a_full0 = bar0;
  g.a_empty0 = bar0 + 8u * kMaxRing;
  g.s_full0 = bar0 + 8u * 2 * kMaxRing;
  g.s_empty0 = bar0 + 8u * 3 * kMaxRing;
  g.bt_ready0 = bar0 + 8u * 4 * kMaxRing;
  g.bt_empty0 = g.bt_ready0 + 8u * 2;
  g.tfull0 = g.bt_ready0 + 8u * 4;
  g.tempty0 = g.bt_ready0 + 8u * 6;
  g.a0 = smem_base + p.a_off;
  g.s0 = smem_base + p.s_off;
  g.bt0 = smem_base + p.bt_off;
  g.s_gen = smem_gen + p.s_off;
  g.bt_gen = smem_gen + p.bt_off;
  g.abort_flag = &abort_flag_s;

  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    for (int s = 0; s < kMaxRing; ++s) {
      mbar_init(g.a_full0 + 8u * s, 1);
      mbar_init(g.a_empty0 + 8u * s, 1);
      mbar_init(g.s_full0 + 8u * s, 1);
      mbar_init(g.s_empty0 + 8u * s, kUnpackThreads);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(g.bt_ready0 + 8u * b, kUnpackThreads);
      mbar_init(g.bt_empty0 + 8u * b, 1);
      mbar_init(g.tfull0 + 8u * b, 1);
      mbar_init(g.tempty0 + 8u * b, kEpiThreads);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = tmem_base_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ activation producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < p.num_tiles; tile += gridDim.x) {
        const int tt = tile % p.ntt;
        const int m = tile / p.ntt / p.ncb;
        for (int kb = 0; kb < p.kblocks; ++kb, ++it) {
          const int s = it % p.na;
          const uint32_t ph = (it / p.na) & 1;
          if (!mbar_wait(g.a_empty0 + 8u * s, ph ^ 1, g.abort_flag, p.f.status)) { ok = false; break; }
          mbar_expect_tx(g.a_full0 + 8u * s, kABytes);
          tma_load_2d(g.a0 + s * kABytes, &p.tmap_a[m], kb * kKStep, tt * kTileM, g.a_full0 + 8u * s);
        }
      }
      drain_ring(g.a_full0, it, p.na);
    }
  } else if (warp == 10) {
    // ------------------------------------------------------------------ packed-weight producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < p.num_tiles; tile += gridDim.x) {
        TileMeta t;
        decode_tile(p, tile, t);
        const uint32_t tx = static_cast<uint32_t>(t.rowbase[kMaxClusterOrders]) * p.pk;
        for (int kb = 0; kb < p.kblocks; ++kb, ++it) {
          const int s = it % p.ns;
          const uint32_t ph = (it / p.ns) & 1;
          if (!mbar_wait(g.s_empty0 + 8u * s, ph ^ 1, g.abort_flag, p.f.status)) { ok = false; break; }
          mbar_expect_tx(g.s_full0 + 8u * s, tx);
#pragma unroll
          for (int ko = 0; ko < kMaxClusterOrders; ++ko) {
            if (ko < t.nk && t.n[ko] > 0) {
              const OrderView& ov = p.f.order[t.k0 + ko];
              const uint8_t* src = ov.kcodes + (static_cast<size_t>(kb) * ov.rows + t.start[ko]) * p.pk;
              bulk_load(g.s0 + s * p.stg_bytes + t.rowbase[ko] * p.pk, src, static_cast<uint32_t>(t.n[ko]) * p.pk,
                        g.s_full0 + 8u * s);
            }
          }
        }
      }
      drain_ring(g.s_full0, it, p.ns);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < p.num_tiles; tile += gridDim.x, ++tcount) {
        TileMeta t;
        decode_tile(p, tile, t);
        const int buf = tcount & 1;
        const uint32_t aph = (tcount >> 1) & 1;
        if (!mbar_wait(g.tempty0 + 8u * buf, aph ^ 1, g.abort_flag, p.f.status)) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        int n = (t.rowbase[kMaxClusterOrders] + 15) & ~15;
        if (n < 16) n = 16;
        const uint32_t idesc = idesc_i8(n);
        const uint32_t d_tmem = tmem_base + buf * kAccCols;
        for (int kb = 0; kb < p.kblocks; ++kb, ++it) {
          const int as = it % p.na, bs = it % kBtRing;
          const uint32_t aphs = (it / p.na) & 1, bph = (it / kBtRing) & 1;
          if (!mbar_wait(g.a_full0 + 8u * as, aphs, g.abort_flag, p.f.status)) { ok = false; break; }
          if (!mbar_wait(g.bt_ready0 + 8u * bs, bph, g.abort_flag, p.f.status)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint64_t adesc = smem_desc_sw128(g.a0 + as * kABytes);
          const uint64_t bdesc = smem_desc_sw128(g.bt0 + bs * kBtBytes);
#pragma unroll
          for (int k = 0; k < kKStep / 32; ++k)
            mma_i8(d_tmem, adesc + static_cast<uint64_t>(k * 2), bdesc + static_cast<uint64_t>(k * 2), idesc, (kb | k) != 0);
          mma_commit(g.a_empty0 + 8u * as);
          mma_commit(g.bt_empty0 + 8u * bs);
        }
        if (ok) mma_commit(g.tfull0 + 8u * buf);
      }
    }
  } else if (warp < 6) {
    // ------------------------------------------------------------------ unpack warps
    const int ut = threadIdx.x - 64;
    if (p.f.bits == 8) unpack_role<8>(p, g, ut);
    else if (p.f.bits == 4) unpack_role<4>(p, g, ut);
    else unpack_role<2>(p, g, ut);
  } else {
    // ------------------------------------------------------------------ epilogue warps
    EpiCtx e;
    e.tmem_base = tmem_base;
    e.tfull0 = g.tfull0;
    e.tempty0 = g.tempty0;
    e.abort_flag = g.abort_flag;
    e.warp = warp;
    e.lane = lane;
    e.colmap = epi_colmap[warp - 6];
    e.crowmap = epi_crowmap[warp - 6];
    e.cscale = epi_cscale[warp - 6];
    if (p.BN == 128) epilogue_role<2>(p, e);
    else if (p.BN == 64) epilogue_role<4>(p, e);
    else epilogue_role<8>(p, e);
  }

  // ---------------------------------------------------------------------- teardown
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// ---------------------------------------------------------------------------------------------
using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeFn encode_fn() {
  static std::once_flag once;
  static EncodeFn fn = nullptr;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeFn>(p);
  });
  return fn;
}

static bool make_map_2d(CUtensorMap* map, const void* base, uint64_t inner_bytes, uint64_t rows, uint64_t pitch_bytes,
                        uint32_t box_inner, uint32_t box_rows, CUtensorMapSwizzle swz) {
  EncodeFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {inner_bytes, rows};
  const cuuint64_t strides[1] = {pitch_bytes};
  const cuuint32_t box[2] = {box_inner, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace tc

static pipe_status launch_tc(const ForwardArgs& a, cudaStream_t stream) {
  using namespace tc;
  static Params p;  // large; filled per call under the lock
  static std::mutex mu;
  std::lock_guard<std::mutex> lock(mu);

  int max_cluster = 0;
  for (int m = 0; m < a.num_branches; ++m) max_cluster = max(max_cluster, a.branch[m].k_end - a.branch[m].k_begin);
  if (max_cluster > kMaxClusterOrders) return PIPE_ERR_UNSUPPORTED;
  const int BN = max_cluster <= 2 ? 128 : (max_cluster <= 4 ? 64 : 32);
  if (a.g % 8 != 0 || a.g > BN || BN % a.g != 0) return PIPE_ERR_UNSUPPORTED;
  if (a.ldxq % 16 != 0) return PIPE_ERR_UNSUPPORTED;
  for (int m = 0; m < a.num_branches; ++m) {
    if (reinterpret_cast<uintptr_t>(a.branch[m].xq) & 15) return PIPE_ERR_UNSUPPORTED;
  }
  if (a.T > (1ll << 30)) return PIPE_ERR_UNSUPPORTED;

  p.f = a;
  p.BN = BN;
  p.ncb = ceil_div(a.O, BN);
  p.ntt = static_cast<int>(ceil_div<int64_t>(a.T, kTileM));
  const int64_t tiles = static_cast<int64_t>(p.ncb) * p.ntt * a.num_branches;
  if (tiles > INT32_MAX) return PIPE_ERR_UNSUPPORTED;
  p.num_tiles = static_cast<int>(tiles);
  p.kblocks = ceil_div(a.I, kKStep);
  p.pk = kKStep * a.bits / 8;
  p.stg_bytes = kMaxN * p.pk;
  p.shift = 8 - a.bits;
  int dev = 0, smem_max = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return PIPE_ERR_CUDA;
  cudaDeviceGetAttribute(&smem_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  // dynamic shared memory: B-tile ring (2 x 32 KiB), packed-weight ring (<= 64 KiB), the rest for activations
  int budget = smem_max - 8192 - 1024 - kBtRing * kBtBytes;  // static shared, alignment slack
  p.ns = 65536 / p.stg_bytes;
  if (p.ns > 6) p.ns = 6;
  if (p.ns < 2) p.ns = 2;
  budget -= p.ns * p.stg_bytes;
  p.na = budget / kABytes;
  if (p.na > kMaxRing) p.na = kMaxRing;
  if (p.na < 2) return PIPE_ERR_UNSUPPORTED;
  p.a_off = 0;
  p.bt_off = p.na * kABytes;
  p.s_off = p.bt_off + kBtRing * kBtBytes;
  const int dyn_smem = p.s_off + p.ns * p.stg_bytes + 1024;

  for (int m = 0; m < a.num_branches; ++m) {
    if (!make_map_2d(&p.tmap_a[m], a.branch[m].xq, static_cast<uint64_t>(a.I), static_cast<uint64_t>(a.T),
                     static_cast<uint64_t>(a.ldxq), kKStep, kTileM, CU_TENSOR_MAP_SWIZZLE_128B))
      return PIPE_ERR_CUDA;
  }
  static int attr_bytes = 0;
  if (attr_bytes < dyn_smem) {
    if (cudaFuncSetAttribute(tc_forward_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn_smem) != cudaSuccess)
      return PIPE_ERR_CUDA;
    attr_bytes = dyn_smem;
  }
  const int grid = p.num_tiles < sms ? p.num_tiles : sms;
  tc_forward_kernel<<<grid, kThreads, dyn_smem, stream>>>(p);
  count_launch(1);
  return launch_status();
}

pipe_status forward_tcgen05(const ForwardArgs& a, cudaStream_t stream) {
  if (a.T == 0) return PIPE_OK;
  const bool sum_mode = a.num_branches > 1 && a.branch[1].accumulate;
  if (!sum_mode) return launch_tc(a, stream);
  // Summed ensemble: one launch per branch, in order, so that y = ((y_1 + y_2) + ...) is formed
  // by the same thread in a fixed order.
  for (int m = 0; m < a.num_branches; ++m) {
    ForwardArgs one = a;
    one.num_branches = 1;
    one.branch[0] = a.branch[m];
    pipe_status st = launch_tc(one, stream);
    if (st != PIPE_OK) return st;
  }
  return PIPE_OK;
}

}  // namespace pipe
