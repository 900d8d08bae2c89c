// tcgen05 tensor-core kernel of the expanded layer (Appendix B, Eq. 9; Sec. 3.2 for the branches).
//
// One persistent CTA per SM walks tiles (branch, block of BN output channels, 128 tokens).
// For a tile, the rows of ALL orders of the branch that fall into the channel block are stacked
// into one int8 B operand (order 1: BN rows; a sparse order: only its kept rows, found through
// the prefix counts), so one chain of tcgen05.mma kind::i8 instructions (M = 128 tokens,
// N = stacked rows, K = 32) fills one int32 accumulator region per order in TMEM while the
// activation tile is staged once per reduction step.  A ring of stages {activation tile, B tile}
// in shared memory decouples the roles:
//   warp 0      activation producer: TMA tensor loads (128B swizzle), several lanes issue in turn
//   warps 2-7   unpack: read the packed int8/int4/ternary rows of the tile straight from the
//               reduction-block-major streaming layout (coalesced 16-byte loads, prefetched one
//               step ahead in registers) and write int8 lanes into the swizzled B tile
//               (shift + mask only; sub-byte codes arrive multiplied by 2^(8-b))
//   warp 1      MMA issuer (one lane), owns the TMEM allocation (2 x 256 columns, double buffered);
//               one tcgen05.commit per step releases the stage to both producers
//   warps 8-15  epilogue: tcgen05.ld the accumulators of each order, shift back, scale by
//               s_k * lambda_x and add in ascending order with one FMA per term, store fp32
// Barrier operations cost their issuing thread on the order of a hundred cycles each, so every
// role touches as few barriers per step as possible and ring positions are advanced without
// divisions.  Every wait on an mbarrier is bounded; on expiry the CTA raises PIPE_ERR_TIMEOUT, all
// roles leave their loops, outstanding copies are drained, TMEM is freed and the kernel returns.
#include "pipe_tc_common.cuh"

namespace pipe {

namespace tc {

constexpr int kTileM = 128;          // tokens per tile
constexpr int kKStep = 128;          // reduction bytes (int8 lanes) per stage
constexpr int kMaxN = 256;           // stacked weight rows per tile
constexpr int kMaxClusterOrders = 8;
// 2 + 6 + 8 = 16 warps: four per scheduler, so every thread may hold 128 registers and neither the unpack
// nor the epilogue role spills; measured faster than 8 unpack warps at 96 registers on every workload.
constexpr int kUnpackWarps = 6;
constexpr int kEpiWarps = 8;
constexpr int kThreads = 32 * (2 + kUnpackWarps + kEpiWarps);
constexpr int kUnpackThreads = 32 * kUnpackWarps;
constexpr int kABytes = kTileM * kKStep;       // 16 KiB per token tile
constexpr int kBtBytes = kMaxN * kKStep;       // 32 KiB
constexpr int kMaxTokTiles = 2;                // token tiles that share one B tile
constexpr int kTmemCols = 512;
constexpr int kMaxRing = 4;
constexpr int kALanes = 4;   // lanes of the activation producer warp that issue copies
using namespace tcc;

struct Params {
  CUtensorMap tmap_a[PIPE_MAX_ORDERS];  // one per branch input
  ForwardArgs f;
  int BN, ncb, ntt, num_tiles, kblocks;   // ntt: token-tile groups
  int tpt;                // token tiles (128 tokens each) per CTA tile: 1 or 2; they share every B tile
  int ntok_tiles;         // token tiles in total
  int a_bytes;            // activation bytes per stage: tpt * 16 KiB
  int stage_bytes;        // a_bytes + 32 KiB
  int nbuf;               // accumulator buffers in TMEM: 2 (epilogue overlaps the next tile) or 1
  int buf_stride;         // TMEM columns between buffers
  int acc_stride;         // TMEM columns between the accumulators of the token tiles of one buffer
  int nkmax;              // most orders any branch has
  int depth;              // stages in the ring
  int pk;                 // packed bytes of one row of one reduction block (128*b/8)
  int shift;              // 8 - b
  int conv_pw, conv_pp, conv_np, conv_chunks;   // patches per image row / per image / in total; 128-channel chunks per tap
  const uint8_t* kbase;   // lowest address of the streaming-layout sections (16-byte aligned)
  uint32_t koff[PIPE_MAX_ORDERS];  // (kcodes of order k - kbase) / 16
};

struct TileMeta {
  int m, cb, tt;                       // branch, channel block, token-tile group
  int nk;                              // orders in this branch
  int k0;                              // first order
  int start[kMaxClusterOrders];        // first compacted row of the channel block in order k
  int n[kMaxClusterOrders];            // rows of order k in the block
  int rowbase[kMaxClusterOrders + 1];  // row offset of order k in the stacked B tile / accumulator
};

// Implicit convolution: a token tile is two 8 x 8 pixel patches (64 rows each); patch p lies in
// image p / pp at patch coordinates ((p % pp) / pw, (p % pp) % pw).
__device__ __forceinline__ void patch_origin(const Params& p, int patch, int& n, int& h0, int& w0);

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

__device__ __forceinline__ void patch_origin(const Params& p, int patch, int& n, int& h0, int& w0) {
  n = patch / p.conv_pp;
  const int rem = patch - n * p.conv_pp;
  h0 = (rem / p.conv_pw) * 8;
  w0 = (rem % p.conv_pw) * 8;
}

struct Rings {
  uint32_t a_full0, bt_ready0, done0, tfull0, tempty0;  // barrier i of a family is 8*i bytes on
  uint32_t stage0;        // shared address of stage 0 (activation tile, then B tile)
  uint8_t* stage_gen;     // generic address of stage 0
  volatile int* abort_flag;
};

// Per-tile placement of one unpack work item (stacked row r, 16-byte chunk c of its packed row):
// offset of the chunk in the streaming layout at reduction block 0 and its step per block, both
// in 16-byte units relative to Params::kbase; 0xffffffff marks an item beyond the tile's rows.
__device__ __forceinline__ void place_item(const Params& p, int k0, int nk, const int (&start)[kMaxClusterOrders],
                                           const int (&rowbase)[kMaxClusterOrders + 1], int r, int c, uint32_t& off,
                                           uint32_t& step) {
  if (r >= rowbase[kMaxClusterOrders]) {
    off = 0xffffffffu;
    step = 0;
    return;
  }
  int rb = 0, st = start[0], ko = 0;
#pragma unroll
  for (int q = 1; q < kMaxClusterOrders; ++q)
    if (q < nk && r >= rowbase[q]) {
      rb = rowbase[q];
      st = start[q];
      ko = q;
    }
  const OrderView& ov = p.f.order[k0 + ko];
  const uint32_t pk16 = static_cast<uint32_t>(p.pk) >> 4;
  off = p.koff[k0 + ko] + static_cast<uint32_t>(st + r - rb) * pk16 + static_cast<uint32_t>(c);
  step = static_cast<uint32_t>(ov.rows) * pk16;
}

// Unpack role.  Work items are (stacked row, 16-byte chunk); a thread owns the same item indices
// in every tile.  A load cursor runs two reduction steps ahead of the step being written (also
// across tile boundaries): the packed chunks travel global memory (L2-resident, fully coalesced)
// -> registers -> swizzled B tile, and a step never waits for the latency of its own loads.
template <int BITS>
__device__ __forceinline__ void unpack_role(const Params& p, const Rings& g, int ut) {
  constexpr int CPR = BITS;              // 16-byte chunks per packed row per block: 8, 4, 2
  constexpr int CPR_LOG = (BITS == 8) ? 3 : (BITS == 4 ? 2 : 1);
  constexpr int ITEMS = (kMaxN * CPR + kUnpackThreads - 1) / kUnpackThreads;   // items past the last row are masked
  constexpr int OUT_PER_CHUNK = 8 / BITS;  // 16-byte vectors written per chunk read
  constexpr int AHEAD = (BITS == 8) ? 1 : 2;   // int8 rows carry 8 chunks per thread: one step ahead only
  const uint4* kb16 = reinterpret_cast<const uint4*>(p.kbase);
  const uint32_t depth = p.depth;
  const int r0 = ut >> CPR_LOG, c_item = ut & (CPR - 1);   // item i: row r0 + i * (threads / CPR), chunk c_item
  const int sw = r0 & 7;                                   // the row step between items is a multiple of 8
  const int my_tiles = (p.num_tiles - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
  if (my_tiles <= 0) return;
  const uint32_t total_steps = static_cast<uint32_t>(my_tiles) * p.kblocks;

  // ---- load cursor
  uint32_t off[ITEMS], stp[ITEMS];
  int cur_tile = blockIdx.x, cur_kb = 0;
  uint32_t issued = 0;
  TileMeta tn;   // metadata of the tile after the cursor's tile, fetched when the cursor enters a tile
  {
    TileMeta t;
    decode_tile(p, cur_tile, t);
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) {
      const int idx = ut + i * kUnpackThreads;
      place_item(p, t.k0, t.nk, t.start, t.rowbase, idx >> CPR_LOG, idx & (CPR - 1), off[i], stp[i]);
    }
    const int nt = cur_tile + gridDim.x;
    decode_tile(p, nt < p.num_tiles ? nt : cur_tile, tn);
  }
  auto fetch = [&](uint4 (&w)[ITEMS], uint32_t& mask) {
    mask = 0;
    if (issued >= total_steps) return;
#pragma unroll
    for (int i = 0; i < ITEMS; ++i)
      if (off[i] != 0xffffffffu) {
        w[i] = __ldg(kb16 + off[i]);
        mask |= 1u << i;
      }
    ++issued;
    if (++cur_kb < p.kblocks) {
#pragma unroll
      for (int i = 0; i < ITEMS; ++i)
        if (off[i] != 0xffffffffu) off[i] += stp[i];
    } else if (issued < total_steps) {
      cur_kb = 0;
      cur_tile += gridDim.x;
#pragma unroll
      for (int i = 0; i < ITEMS; ++i) {
        const int idx = ut + i * kUnpackThreads;
        place_item(p, tn.k0, tn.nk, tn.start, tn.rowbase, idx >> CPR_LOG, idx & (CPR - 1), off[i], stp[i]);
      }
      const int nt = cur_tile + gridDim.x;
      decode_tile(p, nt < p.num_tiles ? nt : cur_tile, tn);
    }
  };

  uint4 q1[ITEMS], q2[ITEMS];
  uint32_t m1 = 0, m2 = 0;
  fetch(q1, m1);
  if (AHEAD == 2) fetch(q2, m2);

  RingPos rp{0, 0};
  for (uint32_t it = 0; it < total_steps; ++it, rp.advance(1, depth)) {
    uint4 w[ITEMS];
    const uint32_t mask = m1;
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) w[i] = q1[i];
    if (AHEAD == 2) {
#pragma unroll
      for (int i = 0; i < ITEMS; ++i) q1[i] = q2[i];
      m1 = m2;
      fetch(q2, m2);
    } else {
      fetch(q1, m1);
    }
    if (!mbar_wait(g.done0 + 8u * rp.slot, rp.phase ^ 1, g.abort_flag, p.f.status)) return;
    uint8_t* bt = g.stage_gen + static_cast<size_t>(rp.slot) * p.stage_bytes + p.a_bytes;
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) {
      if (!((mask >> i) & 1u)) continue;
      const int r = r0 + i * (kUnpackThreads >> CPR_LOG);
      uint8_t* row = bt + (r >> 3) * 1024 + (r & 7) * 128;
      const int c0 = c_item * OUT_PER_CHUNK;
      if (BITS == 8) {
        *reinterpret_cast<uint4*>(row + ((c0 ^ sw) << 4)) = w[i];
      } else if (BITS == 4) {
        const uint32_t m4 = 0xF0F0F0F0u;
        const uint4 v0 = make_uint4((w[i].x << 4) & m4, w[i].x & m4, (w[i].y << 4) & m4, w[i].y & m4);
        const uint4 v1 = make_uint4((w[i].z << 4) & m4, w[i].z & m4, (w[i].w << 4) & m4, w[i].w & m4);
        *reinterpret_cast<uint4*>(row + ((c0 ^ sw) << 4)) = v0;
        *reinterpret_cast<uint4*>(row + (((c0 + 1) ^ sw) << 4)) = v1;
      } else {
        const uint32_t m2c = 0xC0C0C0C0u;
        const uint32_t ww[4] = {w[i].x, w[i].y, w[i].z, w[i].w};
#pragma unroll
        for (int h = 0; h < 4; ++h) {
          const uint4 v = make_uint4((ww[h] << 6) & m2c, (ww[h] << 4) & m2c, (ww[h] << 2) & m2c, ww[h] & m2c);
          *reinterpret_cast<uint4*>(row + (((c0 + h) ^ sw) << 4)) = v;
        }
      }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic writes -> visible to the MMA's reads
    __syncwarp();
    if ((ut & 31) == 0) mbar_arrive(g.bt_ready0 + 8u * rp.slot);   // one arrival per warp
  }
}

struct EpiCtx {
  uint32_t tmem_base, tfull0, tempty0;
  volatile int* abort_flag;
  int warp, lane;
  int jt;            // token tile of the group this warp drains
  int part, nparts;  // share of the 16-channel groups this warp drains (two warps split a lone token tile)
  int16_t* colmap;
  float* cscale;
  float* stg;        // 32 rows x 16 floats, swizzled
};

// Epilogue role (8 warps, one TMEM lane quarter each; a lane owns one token row of a token tile).
// With two token tiles per CTA tile each tile has its own four warps; a lone token tile is split
// by channel groups between the two warps of a lane quarter.
// NKMAX bounds the orders of a branch (2, 4 or 8); the channel block is BN = 8 * nch_max channels.
// Before the accumulators are ready the warp prepares, from the prefix counts, where each
// (order, 8-channel chunk) sits in the accumulator and the products s_k * lambda_x of all stacked
// rows, so that the drain loop has no dependent global loads.
// A lane computes 16 channels of its own token row at a time; the 32 x 16 block is then turned
// through shared memory so that each store instruction writes 64 contiguous bytes of 8 rows
// (a lane writing its own row directly would emit 32 separate 16-byte pieces per instruction,
// which is what bounds the drain otherwise).
template <int NKMAX, bool PARTIALS, bool Q8>
__device__ __forceinline__ void epilogue_role(const Params& p, const EpiCtx& x) {
  constexpr int CH = (NKMAX <= 2) ? 2 : 1;   // chunks per batch of accumulator loads
  const int q = x.warp & 3;                  // TMEM lane quarter this warp may read
  const int lane = x.lane;
  uint32_t tcount = 0;
  const bool y_vec = (p.f.ldy % 4 == 0);
  const int wsw = (lane >> 1) & 3;           // swizzle of this lane's row in the staging block
  // store phase: this lane writes channel quad sj of rows sr0, sr0 + 8, sr0 + 16, sr0 + 24
  const int sr0 = lane >> 2, spp = lane & 3;
  const int sj = spp ^ ((sr0 >> 1) & 3);     // the same for all four rows (they differ by multiples of 8)
  const uint32_t stg_w = smem_u32(x.stg) + static_cast<uint32_t>(lane * 64);
  const uint32_t stg_r = smem_u32(x.stg) + static_cast<uint32_t>(sr0 * 64 + spp * 16);
  const uint32_t colmap_s = smem_u32(x.colmap), cscale_s = smem_u32(x.cscale);
  for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x, ++tcount) {
    TileMeta t;
    decode_tile(p, tile, t);
    const BranchArgs& br = p.f.branch[t.m];
    const int buf = (p.nbuf == 2) ? (tcount & 1) : 0;
    const uint32_t aph = ((p.nbuf == 2) ? (tcount >> 1) : tcount) & 1;
    const float sx = __ldg(br.sx);
    const int c0 = t.cb * p.BN;
    const int c1 = min(c0 + p.BN, p.f.O);
    const int nch = (c1 - c0) >> 3;
    const int n_total = t.rowbase[kMaxClusterOrders];
    __syncwarp();
    {
      // accumulator column of (8-channel chunk, order), or -1: entry [chunk][order]
      for (int e = lane; e < NKMAX * 16; e += 32) {
        const int cc = e / NKMAX, ko = e % NKMAX;
        int col = -1;
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
          if (hi > lo) col = rb + lo * p.f.g + c % p.f.g - st;
        }
        x.colmap[e] = static_cast<int16_t>(col);
      }
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
    // Token of row r (0..31) of this warp: tok_base + r for a matrix of tokens; for the implicit
    // convolution the warp holds half of an 8 x 8 pixel patch (4 image rows of 8 pixels).
    const int ttile = t.tt * p.tpt + x.jt;
    bool tile_ok = ttile < p.ntok_tiles;
    int64_t tok_base = static_cast<int64_t>(ttile) * kTileM + q * 32;
    int eh = 4, ew = 8;
    if (p.f.conv_on) {
      const int patch = 2 * ttile + (q >> 1);
      int n, h0, w0;
      patch_origin(p, patch, n, h0, w0);
      tok_base = (static_cast<int64_t>(n) * p.f.cHo + h0 + (q & 1) * 4) * p.f.cWo + w0;
      tile_ok = patch < p.conv_np;
      eh = p.f.cHo - (h0 + (q & 1) * 4);   // rows (of 8 pixels) and pixels of this half patch that lie inside the output
      ew = p.f.cWo - w0;
    }
    auto token_of = [&](int r) -> int64_t { return p.f.conv_on ? tok_base + (r >> 3) * p.f.cWo + (r & 7) : tok_base + r; };
    // a patch on the right or lower edge of the output may hang over it
    auto inside = [&](int r) -> bool { return (r >> 3) < eh && (r & 7) < ew; };
    const int64_t tok_own = token_of(lane);
    const bool own_ok = tile_ok && (p.f.conv_on ? inside(lane) : tok_own < p.f.T);
    float* srow[4];        // the four rows this lane stores, at channel c0 + 4 * sj
    uint32_t srow_ok = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int64_t tok = token_of(sr0 + 8 * i);
      srow[i] = Q8 ? nullptr : br.y + tok * p.f.ldy + c0 + 4 * sj;
      if (tile_ok && (p.f.conv_on ? inside(sr0 + 8 * i) : tok < p.f.T)) srow_ok |= 1u << i;
    }
    const bool vec_ok = y_vec && ((reinterpret_cast<uintptr_t>(br.y) & 15) == 0);
    // Fused inner-layer epilogue.  A lane's 16 channels become 16 bytes, which it stores itself: at one byte
    // per output a row piece is half a sector however the block is turned, so the staging block is free and
    // holds the bias of the tile's channels instead.
    float ostep = 0.f, orcp = 0.f;
    bool ofast = false;
    int8_t* qrow = nullptr;      // this lane's output row at channel c0
    int qalign = 0;              // 16, 4 or 1: widest store every piece of the row allows
    if constexpr (Q8) {
      ostep = __ldg(br.out_scale);
      ofast = quant_step_is_fast(ostep);
      orcp = ofast ? __frcp_rn(ostep) : 0.f;
      if (!(ostep >= 0.f && ostep < __uint_as_float(0x7f800000u)) && lane == 0) raise_status(p.f.status, PIPE_ERR_INVALID_ARG);
      qrow = br.yq + tok_own * p.f.ldyq + c0;
      const uintptr_t bits = reinterpret_cast<uintptr_t>(br.yq) | static_cast<uintptr_t>(p.f.ldyq);
      qalign = (bits & 15) == 0 ? 16 : ((bits & 3) == 0 ? 4 : 1);
      for (int c = lane; c < p.BN; c += 32) x.stg[c] = (br.add_bias && p.f.bias && c0 + c < p.f.O) ? __ldg(p.f.bias + c0 + c) : 0.f;
    }
    const bool add_bias = br.add_bias && p.f.bias;
    const float* bias_q = add_bias ? p.f.bias + c0 + 4 * sj : nullptr;
    const int ngrp = (nch + 1) >> 1;
    __syncwarp();
    if (!mbar_wait(x.tfull0 + 8u * buf, aph, x.abort_flag, p.f.status)) break;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tbase = x.tmem_base + (static_cast<uint32_t>(q * 32) << 16) + buf * p.buf_stride + x.jt * p.acc_stride;
    for (int grp = x.part; grp < ngrp && tile_ok; grp += x.nparts) {
      // bias of this lane's channel quad: needed in the store phase only, so its latency is hidden
      const bool quad_ok = 2 * grp + (sj >> 1) < nch;
      float4 bq = make_float4(0.f, 0.f, 0.f, 0.f);
      if (!Q8 && add_bias && quad_ok) {
        const float* bp = bias_q + 16 * grp;
        bq = make_float4(__ldg(bp), __ldg(bp + 1), __ldg(bp + 2), __ldg(bp + 3));
      }
      // ---- this lane's row: 16 channels into the staging block (as 16 codes into registers for the fused epilogue)
      uint32_t packed[4] = {0u, 0u, 0u, 0u};
#pragma unroll
      for (int sub = 0; sub < 2; sub += CH) {
        int acc[CH][NKMAX][8];
        int cols[CH][NKMAX];
        {
          // CH * NKMAX int16 entries, contiguous
          constexpr int W = CH * NKMAX / 2;   // 32-bit words: 2, 2 or 4
          uint32_t cw[W];
          const uint32_t addr = colmap_s + static_cast<uint32_t>((2 * grp + sub) * NKMAX * 2);
          if constexpr (W == 2) {
            asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(cw[0]), "=r"(cw[1]) : "r"(addr));
          } else {
            asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(cw[0]), "=r"(cw[1]), "=r"(cw[2]), "=r"(cw[3]) : "r"(addr));
          }
#pragma unroll
          for (int u = 0; u < CH; ++u)
#pragma unroll
            for (int ko = 0; ko < NKMAX; ++ko) {
              const int idx = u * NKMAX + ko;
              cols[u][ko] = static_cast<int16_t>((cw[idx >> 1] >> (16 * (idx & 1))) & 0xffffu);
            }
        }
#pragma unroll
        for (int u = 0; u < CH; ++u)
#pragma unroll
          for (int ko = 0; ko < NKMAX; ++ko)
            if (cols[u][ko] >= 0) tmem_ld8(tbase + cols[u][ko], acc[u][ko]);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int u = 0; u < CH; ++u) {
          const int chunk = 2 * grp + sub + u;
          if (chunk >= nch) continue;
          float y[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) y[e] = 0.f;
#pragma unroll
          for (int ko = 0; ko < NKMAX; ++ko) {
            if (cols[u][ko] < 0) continue;
            float cs[8];
            const uint32_t ca = cscale_s + static_cast<uint32_t>(cols[u][ko] * 4);
            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(cs[0]), "=f"(cs[1]), "=f"(cs[2]), "=f"(cs[3]) : "r"(ca));
            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(cs[4]), "=f"(cs[5]), "=f"(cs[6]), "=f"(cs[7]) : "r"(ca + 16));
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const int a = acc[u][ko][e] >> p.shift;  // exact: the accumulator holds 2^shift times the sum
              acc[u][ko][e] = a;
              y[e] = __fmaf_rn(__int2float_rn(a), cs[e], y[e]);
            }
            if (PARTIALS && own_ok) {
              const int crow = cols[u][ko] - t.rowbase[ko] + t.start[ko];   // compacted row of the chunk's first channel
              int32_t* prow = p.f.partials + tok_own * p.f.total_rows + p.f.order[t.k0 + ko].row_off + crow;
#pragma unroll
              for (int e = 0; e < 8; ++e) prow[e] = acc[u][ko][e];
            }
          }
          if constexpr (Q8) {
            // bias last, sigma, then Q of the next layer (Sec. 3.2): eight codes of this lane's own row
            float bv[8];
            const uint32_t ba = smem_u32(x.stg) + static_cast<uint32_t>(chunk * 32);
            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(bv[0]), "=f"(bv[1]), "=f"(bv[2]), "=f"(bv[3]) : "r"(ba));
            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(bv[4]), "=f"(bv[5]), "=f"(bv[6]), "=f"(bv[7]) : "r"(ba + 16));
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              if (add_bias) y[e] = __fadd_rn(y[e], bv[e]);
              if (p.f.relu == 1) y[e] = fmaxf(y[e], 0.f);
              else if (p.f.relu) y[e] = apply_activation(y[e], p.f.relu);
            }
            float uu[8];
            float edge = ofast ? 0.f : 1.f;
#pragma unroll
            for (int e = 0; e < 8; ++e) uu[e] = quant_magic(y[e], orcp, edge);
            uint32_t w0 = pack4_low_bytes(uu[0], uu[1], uu[2], uu[3]), w1 = pack4_low_bytes(uu[4], uu[5], uu[6], uu[7]);
            if (edge >= 0.5f) {   // some estimate sits on a rounding boundary (or the step has no usable reciprocal)
              w0 = quant4(make_float4(y[0], y[1], y[2], y[3]), ostep, orcp, false);
              w1 = quant4(make_float4(y[4], y[5], y[6], y[7]), ostep, orcp, false);
            }
            packed[2 * (sub + u)] = w0;
            packed[2 * (sub + u) + 1] = w1;
            continue;
          }
          const int j0 = 2 * (sub + u);
          asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(stg_w + static_cast<uint32_t>((j0 ^ wsw) << 4)), "f"(y[0]),
                       "f"(y[1]), "f"(y[2]), "f"(y[3])
                       : "memory");
          asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(stg_w + static_cast<uint32_t>(((j0 + 1) ^ wsw) << 4)), "f"(y[4]),
                       "f"(y[5]), "f"(y[6]), "f"(y[7])
                       : "memory");
        }
      }
      if constexpr (Q8) {
        if (own_ok) {
          int8_t* dq = qrow + 16 * grp;
          const int nw = (2 * grp + 1 < nch) ? 4 : 2;   // a tile's last group may hold eight channels only
          if (qalign == 16 && nw == 4) {
            *reinterpret_cast<uint4*>(dq) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
          } else if (qalign >= 4) {
#pragma unroll
            for (int w = 0; w < 4; ++w)
              if (w < nw) reinterpret_cast<uint32_t*>(dq)[w] = packed[w];
          } else {
#pragma unroll
            for (int w = 0; w < 4; ++w)
              if (w < nw) {
#pragma unroll
                for (int b = 0; b < 4; ++b) dq[4 * w + b] = static_cast<int8_t>(packed[w] >> (8 * b));
              }
          }
        }
        continue;
      }
      __syncwarp();
      // ---- 8 rows x 64 bytes per store instruction; the bias joins here, after the whole chain
      if (quad_ok) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          if (!((srow_ok >> i) & 1u)) continue;
          float4 v;
          asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(stg_r + static_cast<uint32_t>(i * 8 * 64)));
          if (add_bias) v = make_float4(__fadd_rn(v.x, bq.x), __fadd_rn(v.y, bq.y), __fadd_rn(v.z, bq.z), __fadd_rn(v.w, bq.w));
          float* dst = srow[i] + 16 * grp;
          if (vec_ok) {
            if (br.accumulate) {
              const float4 o = *reinterpret_cast<const float4*>(dst);
              v = make_float4(__fadd_rn(o.x, v.x), __fadd_rn(o.y, v.y), __fadd_rn(o.z, v.z), __fadd_rn(o.w, v.w));
            }
            *reinterpret_cast<float4*>(dst) = v;
          } else {
            if (br.accumulate) v = make_float4(__fadd_rn(dst[0], v.x), __fadd_rn(dst[1], v.y), __fadd_rn(dst[2], v.z), __fadd_rn(dst[3], v.w));
            dst[0] = v.x, dst[1] = v.y, dst[2] = v.z, dst[3] = v.w;
          }
        }
      }
      __syncwarp();
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncwarp();
    if (lane == 0) mbar_arrive(x.tempty0 + 8u * buf);   // one arrival per warp
  }
}

// Q8: the fused inner-layer epilogue (activation function and the next layer's input quantizer) replaces the fp32 store.
template <bool Q8>
__global__ void __launch_bounds__(kThreads, 1) tc_forward_kernel(const __grid_constant__ Params p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t bars[3 * kMaxRing + 4];  // a_full[4] bt_ready[4] done[4] tmem_full[2] tmem_empty[2]
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag_s;
  __shared__ __align__(16) int16_t epi_colmap[kEpiWarps][128];    // per epilogue warp: accumulator column of (order, 8-channel chunk) or -1
  __shared__ __align__(16) float epi_cscale[kEpiWarps][kMaxN];    // per epilogue warp: s_k * lambda_x of every stacked row
  __shared__ __align__(16) float epi_stage[kEpiWarps][32 * 16];   // per epilogue warp: 32 token rows x 16 channels

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bar0 = smem_u32(bars);
  Rings g;
  g.a_full0 = bar0;
  g.bt_ready0 = bar0 + 8u * kMaxRing;
  g.done0 = bar0 + 8u * 2 * kMaxRing;
  g.tfull0 = bar0 + 8u * 3 * kMaxRing;
  g.tempty0 = g.tfull0 + 8u * 2;
  g.stage0 = smem_base;
  g.stage_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  g.abort_flag = &abort_flag_s;

  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    for (int s = 0; s < kMaxRing; ++s) {
      mbar_init(g.a_full0 + 8u * s, 1);
      mbar_init(g.bt_ready0 + 8u * s, kUnpackThreads / 32);
      mbar_init(g.done0 + 8u * s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(g.tfull0 + 8u * b, 1);
      mbar_init(g.tempty0 + 8u * b, kEpiWarps);
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
  const uint32_t depth = p.depth;

  if (warp == 0) {
    // ------------------------------------------------------------------ activation producer
    // A copy instruction occupies its issuing thread for several hundred cycles, but copies issued
    // by different lanes overlap.  Lane j owns the steps j, j + P, ...; every step has its own
    // barrier pair, so the lanes need no order among themselves -- PROVIDED P does not exceed the
    // ring depth N: a lane that issued step it - P has seen step it - P - N consumed, hence
    // (consumption is in order) step it - 2N as well, so when it waits for the slot of step `it`
    // that slot's barrier is at most one phase behind and the parity wait cannot be satisfied by
    // a stale phase.
    const int my_tiles = (p.num_tiles - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x);
    const uint32_t total_steps = static_cast<uint32_t>(my_tiles) * p.kblocks;
    const uint32_t P = min(static_cast<uint32_t>(kALanes), depth);
    // The boxes of one step of the implicit convolution (2 * tpt patches) are issued by as many lanes side by
    // side: one lane issuing them in turn would deliver the step a thousand cycles later.
    const uint32_t nb = p.f.conv_on ? 2u * p.tpt : 1u;
    const uint32_t sl = static_cast<uint32_t>(lane) / nb, hb = static_cast<uint32_t>(lane) % nb;
    if (sl < P) {
      RingPos rp{sl, 0};
      int tile = blockIdx.x, kb = sl;
      for (uint32_t it = sl; it < total_steps; it += P, rp.advance(P, depth), kb += P) {
        while (kb >= p.kblocks) {
          kb -= p.kblocks;
          tile += gridDim.x;
        }
        const int tt = tile % p.ntt;
        const int m = tile / p.ntt / p.ncb;
        if (!mbar_wait(g.done0 + 8u * rp.slot, rp.phase ^ 1, g.abort_flag, p.f.status)) break;
        // (a box of another lane may land before this: the transaction count may run ahead of the expectation,
        // and the phase cannot complete before the one pending arrival, which is this instruction)
        if (hb == 0) mbar_expect_tx(g.a_full0 + 8u * rp.slot, p.a_bytes);
        if (!p.f.conv_on) {
          // one box of tpt * 128 token rows; rows beyond T read zeros
          tma_load_2d(g.stage0 + rp.slot * p.stage_bytes, &p.tmap_a[m], kb * kKStep, tt * p.tpt * kTileM, g.a_full0 + 8u * rp.slot);
        } else {
          // reduction block kb = (filter tap, 128-channel chunk); the tap shifts the patch window
          const int tap = kb / p.conv_chunks, chunk = kb - tap * p.conv_chunks;
          const int dh = tap / p.f.ckw - p.f.cph, dw = tap % p.f.ckw - p.f.cpw;
          const int half = static_cast<int>(hb);
          int n, h0, w0;
          patch_origin(p, 2 * p.tpt * tt + half, n, h0, w0);   // a patch index beyond the last one reads zeros (n >= N)
          tma_load_4d(g.stage0 + rp.slot * p.stage_bytes + half * (kABytes / 2), &p.tmap_a[m], chunk * kKStep, p.f.csw * w0 + dw, p.f.csh * h0 + dh,
                      n, g.a_full0 + 8u * rp.slot);
        }
      }
    }
    __syncwarp();
    if (lane == 0) drain_ring(g.a_full0, total_steps, p.depth);
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      RingPos rp{0, 0};
      const uint64_t adesc0 = smem_desc_sw128(g.stage0), bdesc0 = smem_desc_sw128(g.stage0 + p.a_bytes);
      uint32_t tcount = 0;
      bool ok = true;
      // stacked rows of a tile (the only tile metadata this role needs); fetched one tile ahead
      auto stacked_rows = [&](int tile) {
        const int cb = (tile / p.ntt) % p.ncb, m = tile / p.ntt / p.ncb;
        const BranchArgs& br = p.f.branch[m];
        const int c0 = cb * p.BN, c1 = min(c0 + p.BN, p.f.O);
        const int j0 = c0 / p.f.g, j1 = c1 / p.f.g;
        int n = 0;
        for (int k = br.k_begin; k < br.k_end; ++k) {
          const int32_t* cum = p.f.order[k].cum;
          n += (__ldg(cum + j1) - __ldg(cum + j0)) * p.f.g;
        }
        return n;
      };
      int n_next = blockIdx.x < p.num_tiles ? stacked_rows(blockIdx.x) : 0;
      for (int tile = blockIdx.x; ok && tile < p.num_tiles; tile += gridDim.x, ++tcount) {
        const int n_total = n_next;
        if (tile + static_cast<int>(gridDim.x) < p.num_tiles) n_next = stacked_rows(tile + gridDim.x);
        const int buf = (p.nbuf == 2) ? (tcount & 1) : 0;
        const uint32_t aph = ((p.nbuf == 2) ? (tcount >> 1) : tcount) & 1;
        // token tiles of this group that exist (the last group may hold one only)
        const int jn = min(p.tpt, p.ntok_tiles - (tile % p.ntt) * p.tpt);
        if (!mbar_wait(g.tempty0 + 8u * buf, aph ^ 1, g.abort_flag, p.f.status)) { ok = false; break; }
        int n = (n_total + 15) & ~15;
        if (n < 16) n = 16;
        const uint32_t idesc = idesc_i8(kTileM, n);
        const uint32_t d_tmem = tmem_base + buf * p.buf_stride;
        for (int kb = 0; kb < p.kblocks; ++kb, rp.advance(1, depth)) {
          // both barriers are polled before either result is tested so that the two polls overlap
          const bool r1 = mbar_try(g.a_full0 + 8u * rp.slot, rp.phase);
          const bool r2 = mbar_try(g.bt_ready0 + 8u * rp.slot, rp.phase);
          if (!r1 && !mbar_wait(g.a_full0 + 8u * rp.slot, rp.phase, g.abort_flag, p.f.status)) { ok = false; break; }
          if (!r2 && !mbar_wait(g.bt_ready0 + 8u * rp.slot, rp.phase, g.abort_flag, p.f.status)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint64_t so = static_cast<uint64_t>(rp.slot * (p.stage_bytes >> 4));
          const uint64_t adesc = adesc0 + so, bdesc = bdesc0 + so;
          for (int j = 0; j < jn; ++j) {
#pragma unroll
            for (int k = 0; k < kKStep / 32; ++k)
              mma_i8(d_tmem + j * p.acc_stride, adesc + static_cast<uint64_t>(j * (kABytes >> 4) + k * 2),
                     bdesc + static_cast<uint64_t>(k * 2), idesc, (kb | k) != 0);
          }
          mma_commit(g.done0 + 8u * rp.slot);   // frees the stage for the activation producer AND the unpack warps
        }
        if (ok) mma_commit(g.tfull0 + 8u * buf);
      }
    }
  } else if (warp < 2 + kUnpackWarps) {
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
    const int ew = warp - 2 - kUnpackWarps;
    e.jt = (p.tpt == 2) ? (ew >> 2) : 0;
    e.part = (p.tpt == 2) ? 0 : (ew >> 2);
    e.nparts = (p.tpt == 2) ? 1 : 2;
    e.colmap = epi_colmap[ew];
    e.cscale = epi_cscale[ew];
    e.stg = epi_stage[ew];
    if (p.f.partials) {   // verification output: every integer accumulator is also written out
      if (p.nkmax <= 2) epilogue_role<2, true, Q8>(p, e);
      else if (p.nkmax <= 4) epilogue_role<4, true, Q8>(p, e);
      else epilogue_role<8, true, Q8>(p, e);
    } else {
      if (p.nkmax <= 2) epilogue_role<2, false, Q8>(p, e);
      else if (p.nkmax <= 4) epilogue_role<4, false, Q8>(p, e);
      else epilogue_role<8, false, Q8>(p, e);
    }
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
}  // namespace tc

// A tensor map depends on the address, the shape and the box only, and a decoding loop presents the same few
// activation buffers call after call: the last encodings of a host thread are kept (encoding one costs the host about
// as much as the rest of a small-token forward call).
bool make_tensor_map_2d_u8(CUtensorMap* map, const void* base, uint64_t inner_bytes, uint64_t rows, uint64_t pitch_bytes,
                           uint32_t box_inner, uint32_t box_rows, bool swizzle128) {
  struct Entry {
    const void* base = nullptr;
    uint64_t inner = 0, rows = 0, pitch = 0;
    uint32_t box_inner = 0, box_rows = 0;
    bool swz = false, valid = false;
    CUtensorMap map;
  };
  constexpr int kEntries = 8;
  thread_local Entry cache[kEntries];
  thread_local int next = 0;
  for (int i = 0; i < kEntries; ++i) {
    const Entry& e = cache[i];
    if (e.valid && e.base == base && e.inner == inner_bytes && e.rows == rows && e.pitch == pitch_bytes && e.box_inner == box_inner &&
        e.box_rows == box_rows && e.swz == swizzle128) {
      *map = e.map;
      return true;
    }
  }
  if (!tcc::make_map_2d(map, base, inner_bytes, rows, pitch_bytes, box_inner, box_rows,
                        swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE))
    return false;
  Entry& e = cache[next];
  next = (next + 1) % kEntries;
  e.base = base, e.inner = inner_bytes, e.rows = rows, e.pitch = pitch_bytes, e.box_inner = box_inner, e.box_rows = box_rows;
  e.swz = swizzle128, e.valid = true, e.map = *map;
  return true;
}

namespace tc {

// Asked of the runtime once per device: shared memory, SM count, the kernels' static shared memory; the dynamic
// shared-memory attribute of both instantiations is raised to everything the device allows then.
struct DeviceSetup {
  int smem_max = 0, sms = 0, fixed = 0;
  pipe_status status = PIPE_ERR_CUDA;
};

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
    cudaFuncAttributes f0, f1;
    if (cudaFuncGetAttributes(&f0, tc_forward_kernel<false>) != cudaSuccess) return;
    if (cudaFuncGetAttributes(&f1, tc_forward_kernel<true>) != cudaSuccess) return;
    d.fixed = static_cast<int>(f0.sharedSizeBytes > f1.sharedSizeBytes ? f0.sharedSizeBytes : f1.sharedSizeBytes);
    const int dyn = d.smem_max - d.fixed;
    if (cudaFuncSetAttribute(tc_forward_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn) != cudaSuccess) return;
    if (cudaFuncSetAttribute(tc_forward_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn) != cudaSuccess) return;
    d.status = PIPE_OK;
  });
  return setups[dev];
}

}  // namespace tc

static pipe_status launch_tc(const ForwardArgs& a, cudaStream_t stream) {
  using namespace tc;
  const DeviceSetup& ds = device_setup();
  if (ds.status != PIPE_OK) return ds.status;
  const int smem_max = ds.smem_max, sms = ds.sms;
  Params p;

  int max_cluster = 0;
  for (int m = 0; m < a.num_branches; ++m) max_cluster = max(max_cluster, a.branch[m].k_end - a.branch[m].k_begin);
  if (max_cluster > kMaxClusterOrders) return PIPE_ERR_UNSUPPORTED;
  // Widest channel block whose stacked rows fit the 256 accumulator columns in the worst case:
  // order 1 contributes BN rows, a sparse order at most min(BN, rows it keeps in the whole layer).
  int BN = 0, worst_rows = 0;
  for (int cand = 128; cand >= 32 && BN == 0; cand >>= 1) {
    int worst = 0;
    for (int m = 0; m < a.num_branches; ++m) {
      int w = 0;
      for (int k = a.branch[m].k_begin; k < a.branch[m].k_end; ++k) w += min(cand, a.order[k].rows);
      worst = max(worst, w);
    }
    if (worst <= kMaxN && a.g <= cand && cand % a.g == 0) BN = cand, worst_rows = worst;
  }
  if (a.g % 8 != 0 || BN == 0) return PIPE_ERR_UNSUPPORTED;
  if (a.ldxq % 16 != 0) return PIPE_ERR_UNSUPPORTED;
  if (a.conv_on && a.cC % kKStep != 0) return PIPE_ERR_UNSUPPORTED;
  for (int m = 0; m < a.num_branches; ++m) {
    if (reinterpret_cast<uintptr_t>(a.branch[m].xq) & 15) return PIPE_ERR_UNSUPPORTED;
  }
  if (a.T > (1ll << 30)) return PIPE_ERR_UNSUPPORTED;

  p.f = a;
  p.BN = BN;
  p.nkmax = max_cluster;
  p.ncb = ceil_div(a.O, BN);
  p.ntok_tiles = static_cast<int>(ceil_div<int64_t>(a.T, kTileM));
  p.conv_pw = p.conv_pp = p.conv_np = p.conv_chunks = 1;
  if (a.conv_on) {
    p.conv_pw = ceil_div(a.cWo, 8);
    p.conv_pp = ceil_div(a.cHo, 8) * p.conv_pw;
    p.conv_np = p.conv_pp * a.cN;
    p.conv_chunks = a.cC / kKStep;
    p.ntok_tiles = ceil_div(p.conv_np, 2);
  }
  // Two token tiles per CTA tile halve the unpack work per multiply-accumulate; worth it once the
  // paired tiles still give every SM a tile.
  p.tpt = (static_cast<int64_t>(p.ncb) * ceil_div(p.ntok_tiles, 2) * a.num_branches >= sms) ? 2 : 1;
  p.ntt = ceil_div(p.ntok_tiles, p.tpt);
  p.a_bytes = p.tpt * kABytes;
  p.stage_bytes = p.a_bytes + kBtBytes;
  if (p.tpt == 1) {
    p.nbuf = 2, p.buf_stride = 256, p.acc_stride = 0;
  } else if (worst_rows <= 128) {
    p.nbuf = 2, p.buf_stride = 256, p.acc_stride = 128;
  } else {
    p.nbuf = 1, p.buf_stride = 0, p.acc_stride = 256;
  }
  const int64_t tiles = static_cast<int64_t>(p.ncb) * p.ntt * a.num_branches;
  if (tiles > INT32_MAX) return PIPE_ERR_UNSUPPORTED;
  p.num_tiles = static_cast<int>(tiles);
  p.kblocks = ceil_div(a.I, kKStep);
  p.pk = kKStep * a.bits / 8;
  p.shift = 8 - a.bits;
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
  p.depth = (smem_max - ds.fixed - 1024) / p.stage_bytes;  // static shared, alignment slack
  if (p.depth > kMaxRing) p.depth = kMaxRing;
  if (p.depth < 2) return PIPE_ERR_UNSUPPORTED;
  const int dyn_smem = p.depth * p.stage_bytes + 1024;

  if (a.conv_on) {
    for (int m = 0; m < a.num_branches; ++m)
      if (!make_map_nhwc(&p.tmap_a[m], a.branch[m].xq, a.cN, a.cH, a.cW, a.cC, a.csh, a.csw)) return PIPE_ERR_CUDA;
  } else
  for (int m = 0; m < a.num_branches; ++m) {
    if (!make_map_2d(&p.tmap_a[m], a.branch[m].xq, static_cast<uint64_t>(a.I), static_cast<uint64_t>(a.T),
                     static_cast<uint64_t>(a.ldxq), kKStep, p.tpt * kTileM, CU_TENSOR_MAP_SWIZZLE_128B))
      return PIPE_ERR_CUDA;
  }
  const int which = a.q8_out ? 1 : 0;
  const int grid = p.num_tiles < sms ? p.num_tiles : sms;
  if (which) tc_forward_kernel<true><<<grid, kThreads, dyn_smem, stream>>>(p);
  else tc_forward_kernel<false><<<grid, kThreads, dyn_smem, stream>>>(p);
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
