// Two-SM form of the tcgen05 kernel of the expanded layer (Appendix B, Eq. 9; Sec. 3.2 for the branches).
//
// CTAs run as clusters of two (one SM pair).  A pair walks tiles (branch, block of BN output channels,
// 256 tokens): each CTA stages the 128 token rows that will land in ITS tensor memory and unpacks HALF
// of the stacked weight rows of the tile (the rows of all orders of the branch in the channel block,
// see the one-SM kernel), and one thread of the pair's first CTA issues tcgen05.mma.cta_group::2
// (M = 256 over the two SMs, N = stacked rows, K = 32), which reads both halves of B.  Compared with
// the one-SM kernel this halves the unpack work and the B-tile traffic per multiply-accumulate and
// leaves room for two accumulator buffers of up to 256 columns per SM, so the epilogue of a tile
// always overlaps the MMAs of the next.  Roles per CTA:
//   warp 0      activation producer: one tensor load per step (two patch boxes for the implicit convolution),
//               whose completion is counted on the FIRST CTA's stage barrier (cta_group::2 form of the copy)
//   warps 2-7   unpack half of the B tile; every warp signals the first CTA's "B in place" barrier itself
//   warp 1      first CTA: MMA issuer (one lane); both: owner of the tensor-memory allocation.
//               tcgen05.commit with a two-CTA multicast returns a stage to the producers of both
//               CTAs and hands the accumulators to the epilogue warps of both
//   warps 8-15  epilogue of the CTA's own 128 token rows (as in the one-SM kernel); every warp signals the
//               first CTA's "accumulators drained" barrier itself
// Every barrier the MMA issuer waits on therefore lives in the first CTA and counts both CTAs' arrivals; no
// thread forwards signals, and no two lanes of a warp ever spin on different barriers (lanes of one warp that
// poll different barriers take turns, which is what made an earlier relay-lane design latency-bound).
// Every mbarrier wait is bounded; the pair leaves through a cluster barrier so that neither CTA's
// shared memory or barriers disappear while its peer may still signal them.
#include "pipe_tc_common.cuh"

namespace pipe {

namespace tc2 {

constexpr int kTileM = 128;          // tokens per tile
constexpr int kKStep = 128;          // reduction bytes (int8 lanes) per block: one row of a swizzled operand tile
constexpr int kSub = 2;              // reduction blocks per ring stage: every barrier operation, proxy fence and
                                     // commit is paid once per stage, and each costs its thread on the order of a
                                     // hundred cycles, so a stage carries two blocks (eight MMAs)
constexpr int kMaxN = 256;           // stacked weight rows per tile
constexpr int kMaxClusterOrders = 8;
constexpr int kUnpackWarps = 6;   // 16 warps per CTA: 128 registers per thread (see the one-SM kernel)
constexpr int kEpiWarps = 8;
constexpr int kThreads = 32 * (2 + kUnpackWarps + kEpiWarps);
constexpr int kABytes = kTileM * kKStep;       // 16 KiB per token tile and reduction block
constexpr int kBtBytes = (kMaxN / 2) * kKStep;   // 16 KiB per block: this CTA's half of the stacked rows
constexpr int kStageBytes = kSub * (kABytes + kBtBytes);   // [kSub activation tiles][kSub B tiles]
constexpr int kStageBOff = kSub * kABytes;
constexpr int kTmemCols = 512;
constexpr int kAccCols = 256;
constexpr int kMaxRing = 3;
constexpr int kRecBufs = 3;    // copies of block records in shared memory (this tile, the next, the one before)
constexpr int kTileRing = 8;   // tiles whose stacked-row count the unpack warps keep for the MMA issuer (they are at
                               // most a ring of stages, i.e. three tiles, ahead of it)
using namespace tcc;

struct Params {
  CUtensorMap tmap_a[PIPE_MAX_ORDERS];  // one per branch input
  CUtensorMap tmap_y[PIPE_MAX_ORDERS];  // one per branch output (fp32), valid where y_tma has the branch's bit
  uint32_t y_tma;                       // branches whose fp32 output the epilogue may write with tensor stores
  ForwardArgs f;
  int ntt, kblocks;       // ntt: pairs of token tiles; kblocks: reduction blocks of 128 lanes
  int ksteps;             // ring stages per tile: ceil(kblocks / kSub)
  int blocks_fastest;     // tile order inside a branch, see locate_tile
  int ntok_tiles;         // token tiles (128 tokens) in total
  int nkmax;              // most orders any branch has
  int depth;              // stages in the ring
  int pk;                 // packed bytes of one row of one reduction block (128*b/8)
  int shift;              // 8 - b
  int direct;             // the weights come from the layer's int8 copy in the operand layout (bits reads 8, shift 0)
  uint32_t split_mask;    // summed ensemble on one shared input, run as ONE cluster of all orders: bit k is set where
                          // order k (k > 0) opens the next predictor, whose chain the epilogue starts from zero
  int conv_pw, conv_pp, conv_np, conv_chunks;   // patches per image row / per image / in total; 128-channel chunks per tap
  const uint8_t* kbase;   // lowest address of the streaming-layout sections (16-byte aligned)
  uint32_t koff[PIPE_MAX_ORDERS];  // (kcodes of order k - kbase) / 16
};

struct TileMeta {
  int m, cb, tt;                       // branch, channel block of the branch's table, token-tile group
  int c0, c1;                          // the block's output channels [c0, c1)
  int nk;                              // orders in this branch
  int k0;                              // first order
  int start[kMaxClusterOrders];        // first compacted row of the channel block in order k
  int n[kMaxClusterOrders];            // rows of order k in the block
  int rowbase[kMaxClusterOrders + 1];  // row offset of order k in the stacked B tile / accumulator
};

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Address of the same shared-memory location in the CTA of the given cluster rank.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
// Arrival on a barrier of the pair's first CTA (cluster address; the first CTA uses it for its own barriers
// too).  The default semantics (release at CTA scope) are enough and are what is used: the signal tells the MMA
// issuer that this warp's share of the stage is in place, and what reads that share is this SM's own tensor
// core, for which the writers' proxy fence (before the arrival, in program order) has already made it visible.
// A release at cluster scope makes the arriving thread wait for all of its memory operations in flight, the
// prefetch loads of later steps included, and more than doubles the time of a reduction step.
__device__ __forceinline__ void mbar_arrive_lead(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// One lane of a converged warp (the form the compiler recognises as "one thread of a uniform warp").
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
  return pred != 0;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Tensor loads of a CTA pair: the bytes land in the issuing CTA's shared memory, the completion is counted on a
// barrier of the pair's FIRST CTA (cluster address), where the MMA issuer waits for both CTAs' tiles.
__device__ __forceinline__ void tma_pair_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t lead_bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(lead_bar)
      : "memory");
}
__device__ __forceinline__ void tma_pair_load_4d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, uint32_t lead_bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(lead_bar)
      : "memory");
}

// Tensor stores of the epilogue (shared memory -> global, one bulk group per store).
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(reinterpret_cast<uint64_t>(map)),
               "r"(src), "r"(c0), "r"(c1)
               : "memory");
}
__device__ __forceinline__ void tma_store_4d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2, int c3) {
  asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];" ::"l"(
                   reinterpret_cast<uint64_t>(map)),
               "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
               : "memory");
}

// Implicit convolution: a token tile is two 8 x 8 pixel patches (64 rows each); patch p lies in
// image p / pp at patch coordinates ((p % pp) / pw, (p % pp) % pw).
__device__ __forceinline__ void patch_origin(const Params& p, int patch, int& n, int& h0, int& w0);

__device__ __forceinline__ void mma_i8_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, bool accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.u32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate ? 1u : 0u)
      : "memory");
}

// Arrives, once the MMAs issued so far have completed in both SMs, on the barrier at this
// shared-memory offset in BOTH CTAs of the pair.
__device__ __forceinline__ void mma_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
               "h"(static_cast<uint16_t>(3))
               : "memory");
}

// Tiles are numbered branch by branch.  Inside a branch either the token-tile pairs of a channel block lie next to
// each other (the pairs working at the same time then read the same weight rows and sweep the activations once per
// block) or the channel blocks of a token-tile pair do (they share the activation tiles and sweep the weights once per
// pair): Params::blocks_fastest picks the second order when the activations are too large to stay in L2.
// tile_base[m] is the number of tiles of the branches before m; the block counts come from the blob's channel-block
// tables and are known on the device only.
__device__ __forceinline__ void locate_tile(const Params& p, const int* tile_base, int tile, int& m, int& cb, int& tt) {
  m = 0;
  while (m + 1 < p.f.num_branches && tile >= tile_base[m + 1]) ++m;
  const int rest = tile - tile_base[m];
  if (p.blocks_fastest) {
    const int nblk = (tile_base[m + 1] - tile_base[m]) / p.ntt;
    tt = rest / nblk;
    cb = rest - tt * nblk;
  } else {
    cb = rest / p.ntt;
    tt = rest - cb * p.ntt;
  }
}

__device__ __forceinline__ void decode_tile(const Params& p, const int* tile_base, int tile, TileMeta& t) {
  locate_tile(p, tile_base, tile, t.m, t.cb, t.tt);
  const BranchArgs& br = p.f.branch[t.m];
  t.k0 = br.k_begin;
  t.nk = br.k_end - br.k_begin;
  const int j0 = __ldg(br.blk + 1 + t.cb), j1 = __ldg(br.blk + 2 + t.cb);
  t.c0 = j0 * p.f.g;
  t.c1 = j1 * p.f.g;
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

// Rows of the MMA's B operand for a tile that stacks n_total rows: each CTA of the pair holds half of them, and a
// half must be a whole number of unpack items (8 rows; 16 rows of 2-bit codes), so the count is rounded up to 16
// (32); the accumulator columns of the padding rows are never read.
__device__ __forceinline__ int pair_mma_rows(int n_total, int bits) {
  const int q = bits == 2 ? 32 : 16;
  const int n = (n_total + q - 1) / q * q;
  return n < q ? q : n;
}

struct Rings {
  uint32_t full0, done0, tfull0, tempty0;  // barrier i of a family is 8*i bytes on
  uint32_t full_lead0, tempty_lead0;       // the same barriers in the pair's first CTA (cluster addresses)
  int rank, pair, npairs;                  // this CTA's rank in the pair; tiles go round the pairs
  const int* tile_base;                    // shared memory: tiles before each branch, then the total
  int num_tiles;
  volatile int* ntot;                      // shared memory: stacked rows of this pair's tile i at [i % kTileRing]
  uint32_t stage0;        // shared address of stage 0 (activation tile, then B tile)
  uint8_t* stage_gen;     // generic address of stage 0
  volatile int* abort_flag;
};

// Unpack role: ONE WARP PER REDUCTION BLOCK.  The blocks of the pair's tiles form one sequence (two block
// positions per ring stage; a tile with an odd block count ends with an empty position); unpack warp w of this CTA
// takes the positions w, w + W, w + 2W, ... -- with W = 6 = stages x positions per stage that is always the same
// block slot of the ring -- and writes this CTA's half of the stacked rows of that block by itself, so that W blocks
// are in work at a time and the fixed costs of a block (barrier waits, proxy fence, arrival, position bookkeeping:
// several hundred cycles of dependent instructions) are paid by one warp per block instead of by every warp for
// every block.
// Sub-byte codes: as soon as the slot is free the warp brings the packed rows of its half tile -- at most one
// contiguous run per order, because the streaming layout is reduction-block-major -- into the END of the slot with
// bulk copies (the copy engine sustains far more bytes in flight than a warp's own loads, which stalled at issue
// when six warps each had 8 KiB outstanding), reads them into registers, and only then overwrites the slot with the
// widened rows; nothing else is staged.  A lane's item i is the 16-byte chunk 32 i + lane of those packed rows
// (RPI = 32 / CPR rows per item).
// int8 codes need no widening and fill the slot exactly; they are loaded through registers.
template <int BITS>
__device__ __forceinline__ void unpack_role(const Params& p, const Rings& g, int uw, int lane, uint32_t pkbar) {
  constexpr int CPR = BITS;                // 16-byte chunks per packed row per block: 8, 4, 2
  constexpr int RPI = 32 / CPR;            // rows per item: 4, 8, 16
  constexpr int ITEMS = (kMaxN / 2) / RPI; // items of a full half tile: 32, 16, 8
  constexpr int PASS = ITEMS > 16 ? 16 : ITEMS;   // items held in registers at a time
  constexpr int OUT_PER_CHUNK = 8 / BITS;  // 16-byte vectors written per chunk read
  constexpr int PK = kKStep * BITS / 8;    // packed bytes of a row of a block
  constexpr int kPackedOff = kBtBytes - (kMaxN / 2) * PK;   // sub-byte codes: where the packed rows land in the slot
  const uint4* kb16 = reinterpret_cast<const uint4*>(p.kbase);
  const int my_tiles = (g.num_tiles - g.pair + g.npairs - 1) / g.npairs;
  if (my_tiles <= 0) return;
  const int slots_per_tile = kSub * p.ksteps;
  const uint32_t total_slots = static_cast<uint32_t>(my_tiles) * slots_per_tile;
  // this lane's place inside an item: row (lane / CPR) of the item's RPI rows, chunk (lane % CPR) of that row
  const int lr = lane / CPR, lc = lane % CPR;
  const int sw = lr & 7;
  const uint32_t out_lane = static_cast<uint32_t>((lr >> 3) * 1024 + (lr & 7) * 128);

  // With W = stages x positions per stage the warp always works on the same block slot, so the barrier of that
  // slot's packed rows is this warp's alone and its phase is simply the parity of the warp's uses so far.
  uint32_t pk_phase = 0;
  int tile_i = -1;                         // index (0, 1, ...) of the tile whose placement the lanes hold
  // lane q < 8: the run of order q inside this CTA's half tile -- offset of its first chunk at block 0 and step per
  // block (16-byte units relative to kbase), bytes, and byte offset inside the packed rows of the half tile
  uint32_t run_off = 0, run_stp = 0, run_bytes = 0, run_dst = 0;
  int n_items = 0, mine = 0;               // items / rows of this CTA's half tile that exist
  int kbs = uw, ti = 0;                    // block position inside the tile, tile index
  while (kbs >= slots_per_tile) {
    kbs -= slots_per_tile;
    ++ti;
  }
  for (uint32_t pos = uw; pos < total_slots; pos += kUnpackWarps) {
    if (ti != tile_i) {
      tile_i = ti;
      TileMeta t;
      decode_tile(p, g.tile_base, g.pair + ti * g.npairs, t);
      const int n_total = t.rowbase[kMaxClusterOrders];
      // for the MMA issuer, which learns of it through the stage barrier this warp arrives on below
      if (lane == 0) g.ntot[ti % kTileRing] = n_total;
      const int half = pair_mma_rows(n_total, BITS) >> 1;
      const int h0 = g.rank * half;
      mine = max(0, min(half, n_total - h0));   // rows of this CTA's half that exist
      n_items = (mine + RPI - 1) / RPI;
      run_bytes = 0;
      int lo = 0, hi = 0, st = 0, ko = 0;
#pragma unroll
      for (int q = 0; q < kMaxClusterOrders; ++q)
        if (q == lane) {
          lo = t.rowbase[q];
          hi = t.rowbase[q + 1];
          st = t.start[q];
          ko = q;
        }
      if (lane < t.nk) {
        const int a = max(lo, h0), b = min(hi, h0 + mine);
        if (a < b) {
          const uint32_t pk16 = PK >> 4;
          run_off = p.koff[t.k0 + ko] + static_cast<uint32_t>(st + a - lo) * pk16;
          run_stp = static_cast<uint32_t>(p.f.order[t.k0 + ko].rows) * pk16;
          run_bytes = static_cast<uint32_t>(b - a) * PK;
          run_dst = static_cast<uint32_t>(a - h0) * PK;
        }
      }
    }
    const uint32_t gs = static_cast<uint32_t>(ti) * p.ksteps + static_cast<uint32_t>(kbs / kSub);   // stage number
    const uint32_t slot = gs % p.depth, use = gs / p.depth;
    const int sub = kbs % kSub;
    const bool real = kbs < p.kblocks && mine > 0;     // false: the empty position behind an odd block count
    const uint32_t bt_off = slot * kStageBytes + kStageBOff + sub * kBtBytes;
    uint8_t* bt = g.stage_gen + bt_off;
    bool through_registers = false;
    if constexpr (BITS == 8) through_registers = !p.direct;
    if (through_registers) {
      if constexpr (BITS == 8) {
#pragma unroll
      for (int pass = 0; pass < ITEMS / PASS; ++pass) {
        uint4 w[PASS];
        if (real) {
#pragma unroll
          for (int i = 0; i < PASS; ++i) {
            const int item = i + PASS * pass;
            // the run that holds the item's first row
            const int byte0 = item * RPI * PK;
            uint32_t src = 0;
#pragma unroll
            for (int q = 0; q < kMaxClusterOrders; ++q) {
              const uint32_t ro = __shfl_sync(0xffffffffu, run_off + static_cast<uint32_t>(kbs) * run_stp, q);
              const uint32_t rd = __shfl_sync(0xffffffffu, run_dst, q), rbts = __shfl_sync(0xffffffffu, run_bytes, q);
              if (static_cast<uint32_t>(byte0) >= rd && static_cast<uint32_t>(byte0) < rd + rbts) src = ro + ((byte0 - rd) >> 4);
            }
            if (item < n_items) w[i] = __ldg(kb16 + src + lane);
          }
        }
        // the stage is free once the MMAs of its previous use have completed (first pass of the block only)
        if (pass == 0 && !mbar_wait(g.done0 + 8u * slot, (use & 1) ^ 1, g.abort_flag, p.f.status)) return;
        if (real) {
#pragma unroll
          for (int i = 0; i < PASS; ++i) {
            const int item = i + PASS * pass;
            if (item >= n_items) continue;
            const int row0 = item * RPI;   // rows row0 + lr; the item's parity moves the row inside its 8-row atom
            uint8_t* row = bt + (row0 >> 3) * 1024 + (row0 & 7) * 128 + out_lane;
            *reinterpret_cast<uint4*>(row + ((lc ^ ((row0 + lr) & 7)) << 4)) = w[i];
          }
        }
      }
      }
    } else {
      // (int8 rows in the operand layout -- the layer's int8 copy -- are complete when their copies have landed)
      // everything the copies need is prepared before the wait for the slot: what follows the wait is on the
      // critical path of the ring (the barrier of the packed rows belongs to this warp alone, so its byte count can
      // be posted while the slot is still being read)
      const uint32_t bar = pkbar + 8u * (slot * kSub + sub);
      const uint8_t* src = p.kbase + (static_cast<size_t>(run_off + static_cast<uint32_t>(kbs) * run_stp) << 4);
      const uint32_t dst = g.stage0 + bt_off + kPackedOff + run_dst;
      if (real && lane == 0) mbar_expect_tx(bar, static_cast<uint32_t>(mine) * PK);
      if (!mbar_wait(g.done0 + 8u * slot, (use & 1) ^ 1, g.abort_flag, p.f.status)) return;
      if (real) {
        if (run_bytes != 0) {
          asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst), "l"(src),
                       "r"(run_bytes), "r"(bar)
                       : "memory");
        }
        __syncwarp();
        if (!mbar_wait(bar, pk_phase, g.abort_flag, p.f.status)) {
          // leaving with a copy possibly in flight: give it a bounded time to land in this CTA's shared memory
          const long long t0 = clock64();
          while (!mbar_try(bar, pk_phase) && clock64() - t0 < 20000000ll) {
          }
          return;
        }
        pk_phase ^= 1u;
        // Two passes over half of the items each, as a loop (half the registers and half the code of one pass over
        // all of them: the instruction footprint of the warps that share an SM partition is what the inner loops
        // of this kernel are most sensitive to).  The widened rows of the first half lie in the part of the slot
        // that holds no packed bytes; those of the second half cover the packed rows of both, all of which are in
        // registers (or used up) once every lane has loaded its share of the second half.
        if constexpr (BITS != 8) {
        const uint4* pk_in = reinterpret_cast<const uint4*>(bt + kPackedOff) + lane;
#pragma unroll 1
        for (int half = 0; half < 2; ++half) {
        constexpr int HI = ITEMS / 2;
        const int ibase = half * HI;
        uint4 w[HI];
#pragma unroll
        for (int i = 0; i < HI; ++i)
          if (ibase + i < n_items) w[i] = pk_in[(ibase + i) * 32];
        __syncwarp();   // every lane holds its packed chunks before any lane overwrites them
#pragma unroll
        for (int i = 0; i < HI; ++i) {
          if (ibase + i >= n_items) continue;
          uint8_t* row = bt + (ibase + i) * (RPI >> 3) * 1024 + out_lane;   // rows (ibase + i) * RPI + lr (RPI is 8 or 16)
          const int c0 = lc * OUT_PER_CHUNK;
          if (BITS == 4) {
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
        }
        }
      }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic writes -> visible to the MMA's reads
    __syncwarp();
    if (lane == 0) mbar_arrive_lead(g.full_lead0 + 8u * slot);   // one arrival per block position, on the first CTA's barrier
    kbs += kUnpackWarps;
    while (kbs >= slots_per_tile) {
      kbs -= slots_per_tile;
      ++ti;
    }
  }
}

struct EpiCtx {
  uint32_t tmem_base, tfull0, tempty0;
  uint32_t recbar0;   // kRecBufs barriers: the block record of the tile has landed
  uint32_t rec0;      // shared address of the first record copy
  uint32_t prebar0;   // kRecBufs barriers: the scale products of the tile are complete
  float* cfold;       // [kRecBufs][kMaxN]: s_k * lambda_x of every stacked row of the tile
  const float* sx_s;  // shared memory: lambda_x of every branch (and, behind them, the output steps of the fused epilogue)
  volatile int* abort_flag;
  int warp, lane;
  int rank, pair, npairs;
  const int* tile_base;
  int num_tiles;
  uint32_t tempty_lead0;   // the accumulator-released barriers of the pair's first CTA (cluster address)
  int part, nparts;  // share of the 16-channel groups this warp drains (two warps per lane quarter)
  float* stg;        // 32 rows x 16 floats, swizzled
  uint32_t zero_s;   // shared address of eight zero floats
};

// Epilogue role (8 warps, one TMEM lane quarter each; a lane owns one token row of a token tile).
// The CTA drains the 128 token rows held by its own tensor memory; the channel groups are split
// between the two warps of a lane quarter.
// NKMAX bounds the orders of a branch (2, 4 or 8); the channel block is BN = 8 * nch_max channels.
// Where each (order, 8-channel chunk) sits in the accumulator and the scale of every stacked row come from the
// block's record in the blob (written by the expansion), which one lane of the CTA fetches with a bulk copy one
// tile ahead into one of three copies; the epilogue itself does no dependent global load.
// A lane computes 16 channels of its own token row at a time; the 32 x 16 block is then turned
// through shared memory so that each store instruction writes 64 contiguous bytes of 8 rows
// (a lane writing its own row directly would emit 32 separate 16-byte pieces per instruction,
// which is what bounds the drain otherwise).
// Q8: the fused inner-layer epilogue (activation function and the next layer's input quantizer, see the one-SM
// kernel) replaces the fp32 store; a lane then stores the 16 codes of its own row itself and the staging block holds
// the bias of the tile's channels.
// SUMMED: the tile stacks the orders of ALL predictors of an ensemble whose predictors share one input and whose
// outputs are summed after the layer (Sec. 3.2): every predictor's chain starts from zero, the bias closes the first
// one, and the chains are added in ascending predictor order in this thread -- the same additions, in the same
// order, as one launch per predictor summing into y, without the read-modify-write of y.
template <int NKMAX, bool PARTIALS, bool Q8, bool SUMMED, bool SHORT_K>
__device__ __forceinline__ void epilogue_role(const Params& p, const EpiCtx& x) {
  constexpr int CH = (NKMAX <= 2) ? 2 : 1;   // chunks per batch of accumulator loads
  // STRAIGHT: the chain of a chunk without branches (see below).  It trades some arithmetic on pruned (chunk, order)
  // pairs for a loop body the compiler can interleave freely, which pays where the drain paces the layer -- a short
  // reduction axis (cfg3a 49.3 -> 46.1 us) -- and costs a percent where it does not, so the host picks it by the axis.
  constexpr bool STRAIGHT = SHORT_K && !PARTIALS && NKMAX <= 2;
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
  const bool bias_vec = (reinterpret_cast<uintptr_t>(p.f.bias) & 15) == 0;
  bool stg_busy = false;   // a tensor store of this warp may still be reading the staging block
  const bool rec_issuer = (x.warp == 2 + kUnpackWarps) && lane == 0;   // the lane that fetches the block records
  // Record of the pair's tile number tc (tile index `tile`) into copy tc % kRecBufs.
  auto fetch_record = [&](uint32_t tc, int tile) {
    int m, cb, tt;
    locate_tile(p, x.tile_base, tile, m, cb, tt);
    const uint8_t* src = p.f.branch[m].rec + static_cast<size_t>(cb) * kRecBytes;
    const uint32_t bar = x.recbar0 + 8u * (tc % kRecBufs);
    mbar_expect_tx(bar, kRecBytes);
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     x.rec0 + (tc % kRecBufs) * kRecBytes),
                 "l"(src), "r"(kRecBytes), "r"(bar)
                 : "memory");
  };
  if (rec_issuer) {
    if (x.pair < x.num_tiles) fetch_record(0, x.pair);
    if (x.pair + x.npairs < x.num_tiles) fetch_record(1, x.pair + x.npairs);
  }
  for (int tile = x.pair; tile < x.num_tiles; tile += x.npairs, ++tcount) {
    struct { int m, cb, tt, k0; } t;
    locate_tile(p, x.tile_base, tile, t.m, t.cb, t.tt);
    const BranchArgs& br = p.f.branch[t.m];
    t.k0 = br.k_begin;
    const int buf = tcount & 1;
    const uint32_t aph = (tcount >> 1) & 1;
    const float sx = x.sx_s[t.m];
    const uint32_t rec_s = x.rec0 + (tcount % kRecBufs) * kRecBytes;
    if (!mbar_wait(x.recbar0 + 8u * (tcount % kRecBufs), (tcount / kRecBufs) & 1, x.abort_flag, p.f.status)) break;
    int c0, c1;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(c0), "=r"(c1) : "r"(rec_s));
    const int nch = (c1 - c0) >> 3;       // at most PIPE_BLOCK_CHANNELS / 8
    const uint32_t colmap_s = rec_s + kRecColmapOff;
    // The products c = s_k * lambda_x of the tile's stacked rows, once per CTA instead of once per token row.
    float* cf = x.cfold + (tcount % kRecBufs) * kMaxN;
    {
      const int et = (x.warp - 2 - kUnpackWarps) * 32 + lane;   // this thread among the epilogue threads
      for (int r = et; r < kMaxN; r += 32 * kEpiWarps) {
        float sc;
        asm volatile("ld.shared.f32 %0, [%1];" : "=f"(sc) : "r"(rec_s + kRecScaleOff + 4u * r));
        cf[r] = __fmul_rn(sc, sx);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(x.prebar0 + 8u * (tcount % kRecBufs));
      if (!mbar_wait(x.prebar0 + 8u * (tcount % kRecBufs), (tcount / kRecBufs) & 1, x.abort_flag, p.f.status)) break;
    }
    const uint32_t cscale_s = smem_u32(cf);
    // The accumulators hold 2^(8-b) times the sums; float(2^(8-b) a) = 2^(8-b) float(a) exactly, so the shift is
    // taken as a multiplication by 2^-(8-b) after the conversion (exact for every int32, and on the pipe with the
    // most issue slots); only the verification output needs the shifted integers themselves.
    const float unshift = __int_as_float((127 - p.shift) << 23);
    // Token of row r (0..31) of this warp: tok_base + r for a matrix of tokens; for the implicit
    // convolution the warp holds half of an 8 x 8 pixel patch (4 image rows of 8 pixels).
    const int ttile = 2 * t.tt + x.rank;
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
    // Tensor stores (one per full 16-channel group, issued by one lane, straight from the staging block) where the
    // host found the output eligible: they leave the warp with neither the second pass over the staging block nor
    // the store instructions, and rows beyond T -- for a convolution, pixels beyond the image -- are clipped by
    // the copy engine.  A sum into y keeps the path through registers, which alone adds in binary32 round-to-nearest.
    const bool tma_out = !Q8 && ((p.y_tma >> t.m) & 1u) && !br.accumulate && tile_ok;
    int ty1 = static_cast<int>(tok_base), ty2 = 0, ty3 = 0;   // coordinates behind the channel: token, or (x, y, image)
    if (p.f.conv_on) {
      const int patch = 2 * ttile + (q >> 1);
      patch_origin(p, patch, ty3, ty2, ty1);
      ty2 += (q & 1) * 4;
    }
    float ostep = 0.f, orcp = 0.f;
    bool ofast = false;
    int8_t* qrow = nullptr;      // this lane's output row at channel c0
    int qalign = 0;              // 16, 4 or 1: widest store every piece of the row allows
    if constexpr (Q8) {
      ostep = x.sx_s[PIPE_MAX_ORDERS + t.m];
      ofast = quant_step_is_fast(ostep);
      orcp = ofast ? __frcp_rn(ostep) : 0.f;
      if (!(ostep >= 0.f && ostep < __uint_as_float(0x7f800000u)) && lane == 0) raise_status(p.f.status, PIPE_ERR_INVALID_ARG);
      qrow = br.yq + tok_own * p.f.ldyq + c0;
      // the block starts at a multiple of 8 channels; 16-byte stores need the row piece aligned as well
      const uintptr_t bits = reinterpret_cast<uintptr_t>(br.yq) | static_cast<uintptr_t>(p.f.ldyq) | static_cast<uintptr_t>(c0);
      qalign = (bits & 15) == 0 ? 16 : ((bits & 3) == 0 ? 4 : 1);
      for (int c = lane; c < c1 - c0; c += 32) x.stg[c] = (br.add_bias && p.f.bias) ? __ldg(p.f.bias + c0 + c) : 0.f;
    }
    const bool add_bias = !SUMMED && br.add_bias && p.f.bias;   // (a summed ensemble adds it inside the chain)
    const float* bias_q = add_bias ? p.f.bias + c0 + 4 * sj : nullptr;
    const int ngrp = (nch + 1) >> 1;
    __syncwarp();
    if (!mbar_wait(x.tfull0 + 8u * buf, aph, x.abort_flag, p.f.status)) break;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    // The record of the NEXT tile goes into the copy the tile before the last one used: the accumulators just handed
    // over were computed after every epilogue warp of the pair had finished that tile.
    if (rec_issuer && tcount >= 1 && tile + x.npairs < x.num_tiles) fetch_record(tcount + 1, tile + x.npairs);
    const uint32_t tbase = x.tmem_base + (static_cast<uint32_t>(q * 32) << 16) + buf * kAccCols;
    for (int grp = x.part; grp < ngrp && tile_ok; grp += x.nparts) {
      // bias of this lane's channel quad: needed in the store phase only, so its latency is hidden
      const bool quad_ok = 2 * grp + (sj >> 1) < nch;
      float4 bq = make_float4(0.f, 0.f, 0.f, 0.f);
      if (!Q8 && add_bias && quad_ok && !(tma_out && 2 * grp + 1 < nch)) {
        const float* bp = bias_q + 16 * grp;
        bq = make_float4(__ldg(bp), __ldg(bp + 1), __ldg(bp + 2), __ldg(bp + 3));
      }
      // ---- this lane's row: 16 channels into the staging block (as 16 codes into registers for the fused epilogue)
      const bool use_tma = tma_out && 2 * grp + 1 < nch;
      uint32_t packed[4] = {0u, 0u, 0u, 0u};
#pragma unroll
      for (int sub = 0; sub < 2; sub += CH) {
        int acc[CH][NKMAX][8];
        int cols[CH][NKMAX];
#pragma unroll
        for (int u = 0; u < CH; ++u) {
          // the chunk's eight int16 entries (one per order of a cluster), of which the first NKMAX can be present
          constexpr int W = NKMAX / 2;   // 32-bit words: 1, 2 or 4
          uint32_t cw[W];
          const uint32_t addr = colmap_s + static_cast<uint32_t>((2 * grp + sub + u) * 16);
          if constexpr (W == 1) {
            asm volatile("ld.shared.u32 %0, [%1];" : "=r"(cw[0]) : "r"(addr));
          } else if constexpr (W == 2) {
            asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(cw[0]), "=r"(cw[1]) : "r"(addr));
          } else {
            asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(cw[0]), "=r"(cw[1]), "=r"(cw[2]), "=r"(cw[3]) : "r"(addr));
          }
#pragma unroll
          for (int ko = 0; ko < NKMAX; ++ko) cols[u][ko] = static_cast<int16_t>((cw[ko >> 1] >> (16 * (ko & 1))) & 0xffffu);
        }
#pragma unroll
        for (int u = 0; u < CH; ++u)
#pragma unroll
          for (int ko = 0; ko < NKMAX; ++ko) {
            if constexpr (STRAIGHT) tmem_ld8(tbase + (cols[u][ko] >= 0 ? cols[u][ko] : 0), acc[u][ko]);
            else if (cols[u][ko] >= 0) tmem_ld8(tbase + cols[u][ko], acc[u][ko]);
          }
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int u = 0; u < CH; ++u) {
          const int chunk = 2 * grp + sub + u;
          if (chunk >= nch) continue;
          float y[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) y[e] = 0.f;
          float ysum[8];          // SUMMED: the predictors closed so far
          bool first_chain = true;
          // closes the running predictor's chain: the bias ends the first one, the others are added to the sum
          auto close_chain = [&]() {
            if (first_chain) {
              if (p.f.bias) {
                const float* bp = p.f.bias + c0 + 8 * chunk;
#pragma unroll
                for (int e = 0; e < 8; ++e) y[e] = __fadd_rn(y[e], __ldg(bp + e));
              }
#pragma unroll
              for (int e = 0; e < 8; ++e) ysum[e] = y[e];
              first_chain = false;
            } else {
#pragma unroll
              for (int e = 0; e < 8; ++e) ysum[e] = __fadd_rn(ysum[e], y[e]);
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) y[e] = 0.f;
          };
#pragma unroll
          for (int ko = 0; ko < NKMAX; ++ko) {
            if constexpr (SUMMED) {
              if (ko > 0 && ((p.split_mask >> ko) & 1u)) close_chain();
            }
            if constexpr (!STRAIGHT) {
              if (cols[u][ko] < 0) continue;
            }
            float cs[8];
            // (STRAIGHT: an order that pruned the chunk's group takes part with the scale 0 and whatever integers column 0
            // holds -- finite, times zero, added to a y that is never -0: the same bits, and no branch in the chain)
            const uint32_t ca = (STRAIGHT && cols[u][ko] < 0) ? x.zero_s : cscale_s + static_cast<uint32_t>(cols[u][ko] * 4);
            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(cs[0]), "=f"(cs[1]), "=f"(cs[2]), "=f"(cs[3]) : "r"(ca));
            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(cs[4]), "=f"(cs[5]), "=f"(cs[6]), "=f"(cs[7]) : "r"(ca + 16));
            if constexpr (PARTIALS) {
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                const int a = acc[u][ko][e] >> p.shift;  // exact: the accumulator holds 2^shift times the sum
                acc[u][ko][e] = a;
                y[e] = __fmaf_rn(__int2float_rn(a), cs[e], y[e]);
              }
            } else {
#pragma unroll
              for (int e = 0; e < 8; ++e) y[e] = __fmaf_rn(__fmul_rn(__int2float_rn(acc[u][ko][e]), unshift), cs[e], y[e]);
            }
            if (PARTIALS && own_ok) {
              int rb_ko, st_ko;   // the order's first row in the stacked block and in its own compacted rows
              asm volatile("ld.shared.u32 %0, [%1];" : "=r"(rb_ko) : "r"(rec_s + 4u * (kRecRowbase + ko)));
              asm volatile("ld.shared.u32 %0, [%1];" : "=r"(st_ko) : "r"(rec_s + 4u * (kRecStart + ko)));
              const int crow = cols[u][ko] - rb_ko + st_ko;   // compacted row of the chunk's first channel
              int32_t* prow = p.f.partials + tok_own * p.f.total_rows + p.f.order[t.k0 + ko].row_off + crow;
#pragma unroll
              for (int e = 0; e < 8; ++e) prow[e] = acc[u][ko][e];
            }
          }
          if constexpr (SUMMED) {
            close_chain();
#pragma unroll
            for (int e = 0; e < 8; ++e) y[e] = ysum[e];
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
          if (use_tma && add_bias) {
            // tensor stores: the bias of this lane's own channels joins before the staging block (the same addition,
            // after the whole chain, as on the other path)
            const float* bp = p.f.bias + c0 + 8 * chunk;
            float bo[8];
            if (bias_vec) {
              const float4 b0 = __ldg(reinterpret_cast<const float4*>(bp)), b1 = __ldg(reinterpret_cast<const float4*>(bp) + 1);
              bo[0] = b0.x, bo[1] = b0.y, bo[2] = b0.z, bo[3] = b0.w, bo[4] = b1.x, bo[5] = b1.y, bo[6] = b1.z, bo[7] = b1.w;
            } else {
#pragma unroll
              for (int e = 0; e < 8; ++e) bo[e] = __ldg(bp + e);
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) y[e] = __fadd_rn(y[e], bo[e]);
          }
          if (sub + u == 0 && stg_busy) {
            // the tensor store of the group before must have read the staging block
            if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
            __syncwarp();
            stg_busy = false;
          }
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
      if (use_tma) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the staging block, for the copy engine
        __syncwarp();
        if (lane == 0) {
          const int cch = c0 + 16 * grp;
          if (p.f.conv_on) tma_store_4d(&p.tmap_y[t.m], smem_u32(x.stg), cch, ty1, ty2, ty3);
          else tma_store_2d(&p.tmap_y[t.m], smem_u32(x.stg), cch, ty1);
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
        stg_busy = true;
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
    if (lane == 0) mbar_arrive_lead(x.tempty_lead0 + 8u * buf);   // one arrival per warp, on the first CTA's barrier
  }
  // the warp's tensor stores are complete before it leaves (the staging block is read, the rows are written)
  if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  __syncwarp();
}

template <bool Q8, bool SUMMED, bool SHORT_K>
__global__ void __launch_bounds__(kThreads, 1) tc2_forward_kernel(const __grid_constant__ Params p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t bars[2 * kMaxRing + 4];  // full[3] done[3] tmem_full[2] tmem_empty[2]
  __shared__ uint64_t pk_bars[kMaxRing * kSub];   // "packed rows have landed", one per block slot of the ring
  __shared__ uint64_t rec_bars[kRecBufs];         // "block record landed", one per copy
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag_s;
  __shared__ int tile_base_s[PIPE_MAX_ORDERS + 1];   // tiles before each branch, then the total
  __shared__ int ntot_s[kTileRing];
  __shared__ __align__(16) uint8_t tile_recs[kRecBufs][kRecBytes];   // block records of the tiles in the epilogue's hands
  __shared__ __align__(16) float cfold_s[kRecBufs][kMaxN];            // s_k * lambda_x of the stacked rows of those tiles
  __shared__ uint64_t pre_bars[kRecBufs];
  __shared__ __align__(16) float zero8_s[8];
  __shared__ float sx_s[2 * PIPE_MAX_ORDERS];                        // lambda_x of every branch, then the fused epilogue's output steps
  __shared__ __align__(1024) float epi_stage[kEpiWarps][32 * 16];   // per epilogue warp: 32 token rows x 16 channels (the
                                                                    // source of tensor stores with the 64-byte swizzle)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bar0 = smem_u32(bars);
  Rings g;
  g.full0 = bar0;
  g.done0 = bar0 + 8u * kMaxRing;
  g.tfull0 = bar0 + 8u * 2 * kMaxRing;
  g.tempty0 = g.tfull0 + 8u * 2;
  g.rank = static_cast<int>(cluster_rank());
  g.pair = static_cast<int>(blockIdx.x >> 1);
  g.npairs = static_cast<int>(gridDim.x >> 1);
  g.full_lead0 = map_to_cta(g.full0, 0);
  g.tempty_lead0 = map_to_cta(g.tempty0, 0);
  g.stage0 = smem_base;
  g.stage_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  g.abort_flag = &abort_flag_s;
  g.ntot = ntot_s;

  // A launch that follows in the stream may be brought onto the SMs as they become free (its CTAs then exist when this
  // launch's last pair ends).  This kernel waits here, before its first access to global memory, until the launch
  // before it is complete, and lets its own dependents start only after that: a dependent that reads weights ahead
  // of ITS wait (the weight-streaming kernel) then never runs beside an expansion queued before this launch.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (threadIdx.x >= 32 && threadIdx.x < 32 + 2 * PIPE_MAX_ORDERS) {
    // (inputs of this launch: written before it started)
    const int i = threadIdx.x - 32, m = i % PIPE_MAX_ORDERS;
    float v = 0.f;
    if (m < p.f.num_branches) {
      if (i < PIPE_MAX_ORDERS) v = __ldg(p.f.branch[m].sx);
      else if (Q8) v = __ldg(p.f.branch[m].out_scale);
    }
    sx_s[i] = v;
  }
  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    for (int i = 0; i < 8; ++i) zero8_s[i] = 0.f;
    int acc = 0;
    for (int m = 0; m < p.f.num_branches; ++m) {
      tile_base_s[m] = acc;
      acc += __ldg(p.f.branch[m].blk) * p.ntt;   // blocks of the branch's table x token-tile pairs
    }
    tile_base_s[p.f.num_branches] = acc;
    // The MMA issuer sits in the pair's first CTA, so the barriers it waits on live there and count the
    // arrivals of BOTH CTAs: "stage full" = the first CTA's producer (which posts the bytes of both CTAs'
    // activation tiles) + one unpack warp per block position and CTA; "accumulators drained" = every epilogue warp of the
    // pair.  The same barriers of the second CTA are initialised but never used.
    for (int s = 0; s < kMaxRing; ++s) {
      mbar_init(g.full0 + 8u * s, 1 + 2 * kSub);
      mbar_init(g.done0 + 8u * s, 1);
    }
    for (int s = 0; s < kMaxRing * kSub; ++s) mbar_init(smem_u32(&pk_bars[s]), 1);
    for (int b = 0; b < kRecBufs; ++b) {
      mbar_init(smem_u32(&rec_bars[b]), 1);
      mbar_init(smem_u32(&pre_bars[b]), kEpiWarps);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(g.tfull0 + 8u * b, 1);
      mbar_init(g.tempty0 + 8u * b, 2 * kEpiWarps);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync_all();   // both CTAs' barriers are initialised before either signals the other
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = tmem_base_slot;
  const uint32_t depth = p.depth;
  g.tile_base = tile_base_s;
  g.num_tiles = tile_base_s[p.f.num_branches];
  const int my_tiles = (g.num_tiles - g.pair + g.npairs - 1) / g.npairs;
  const uint32_t total_steps = static_cast<uint32_t>(my_tiles > 0 ? my_tiles : 0) * p.ksteps;   // ring stages

  if (warp == 0) {
    // ------------------------------------------------------------------ activation producer
    // One lane per copy of a stage (per reduction block one box for a matrix of tokens, two patch boxes for the
    // implicit convolution); the lanes run the same loop on the same barriers, so the warp stays converged.  The
    // completion of both CTAs' copies is counted on the FIRST CTA's stage barrier, whose expected byte count
    // (both tiles) that CTA's lane 0 posts; a copy of the second CTA may land before that, which only lets the
    // transaction count run ahead of the expectation while the barrier's one arrival is still pending.
    const int per_block = p.f.conv_on ? 2 : 1;        // copies per reduction block
    const int sub = lane / per_block, half = lane % per_block;
    if (lane < kSub * per_block) {
      RingPos rp{0, 0};
      // Everything a copy needs is worked out before the wait for its stage (what follows that wait is on the critical
      // path of the ring): the tile's place once per tile, the filter tap of a reduction block by stepping, not by
      // dividing.
      int tile = g.pair - g.npairs, ks = p.ksteps;
      int m = 0, ttile = 0;
      int pn = 0, ph0 = 0, pw0 = 0;     // convolution: image and origin of this lane's patch of the tile
      int chunk = 0, th = 0, tw = 0;    // convolution: 128-channel chunk and filter tap (row, column) of block kb
      for (uint32_t it = 0; it < total_steps; ++it, rp.advance(1, depth), ++ks) {
        if (ks == p.ksteps) {
          ks = 0;
          tile += g.npairs;
          int cb, tt;
          locate_tile(p, g.tile_base, tile, m, cb, tt);
          ttile = 2 * tt + g.rank;   // this CTA's 128 token rows of the pair's tile
          if (p.f.conv_on) {
            patch_origin(p, 2 * ttile + half, pn, ph0, pw0);   // a patch index beyond the last one reads zeros (n >= N)
            const int tap = sub / p.conv_chunks;
            chunk = sub - tap * p.conv_chunks;
            th = tap / p.f.ckw;
            tw = tap - th * p.f.ckw;
          }
        }
        const int nsub = min(kSub, p.kblocks - ks * kSub);   // the last stage of a tile may hold one block only
        const int kb = ks * kSub + sub;
        const uint32_t bar = g.full_lead0 + 8u * rp.slot;
        const uint32_t dst = g.stage0 + rp.slot * kStageBytes + sub * kABytes + (p.f.conv_on ? half * (kABytes / 2) : 0);
        // reduction block kb = (filter tap, 128-channel chunk); the tap shifts the patch window
        const int c0 = p.f.conv_on ? chunk * kKStep : kb * kKStep;
        const int c1 = p.f.conv_on ? p.f.csw * pw0 + tw - p.f.cpw : ttile * kTileM;
        const int c2 = p.f.csh * ph0 + th - p.f.cph;
        if (p.f.conv_on) {   // block kb + kSub, for the next stage
          chunk += kSub;
          while (chunk >= p.conv_chunks) {
            chunk -= p.conv_chunks;
            if (++tw == p.f.ckw) {
              tw = 0;
              ++th;
            }
          }
        }
        // (the byte count of the stage barrier must NOT be posted ahead of this wait: the producer runs up to a ring
        // ahead of the MMAs, so the barrier's phase of the slot's use before may still be collecting its arrivals,
        // and an early arrival would be counted into that phase)
        if (!mbar_wait(g.done0 + 8u * rp.slot, rp.phase ^ 1, g.abort_flag, p.f.status)) break;
        if (g.rank == 0 && lane == 0) mbar_expect_tx(g.full0 + 8u * rp.slot, 2 * nsub * kABytes);
        if (sub >= nsub) continue;
        if (!p.f.conv_on) tma_pair_load_2d(dst, &p.tmap_a[m], c0, c1, bar);   // rows beyond T read zeros
        else tma_pair_load_4d(dst, &p.tmap_a[m], c0, c1, c2, pn, bar);
      }
    }
    __syncwarp();
    // (Every issued copy is consumed by an MMA before the accumulators of its tile are handed over, so on the
    // normal path nothing is in flight here.  After an abort the first CTA gives the copies of both CTAs a
    // bounded time to land before the pair leaves through the cluster barrier below.)
    if (lane == 0 && g.rank == 0 && *g.abort_flag) drain_ring(g.full0, total_steps, p.depth, 20000000ll);
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (first CTA of the pair)
    // The whole warp runs the loop and its waits; one elected lane issues.  Everything the loop computes is then the same in
    // all lanes, which lets the compiler keep the descriptors in the warp's uniform registers, where the MMA
    // instruction takes them from: a loop run by one lane of a diverged warp moves every descriptor there
    // instruction by instruction, and this thread's instruction count is what paces a layer with a short reduction
    // axis.
    if (g.rank == 0) {
      RingPos rp{0, 0};
      // (the address field of a descriptor is its low 14 bits, in 16-byte units: offsets inside the ring never carry
      // out of it, so only the low word changes from MMA to MMA)
      const uint64_t adesc0 = smem_desc_sw128(g.stage0), bdesc0 = smem_desc_sw128(g.stage0 + kStageBOff);
      const uint32_t a_lo = static_cast<uint32_t>(adesc0), a_hi = static_cast<uint32_t>(adesc0 >> 32);
      const uint32_t b_lo = static_cast<uint32_t>(bdesc0), b_hi = static_cast<uint32_t>(bdesc0 >> 32);
      uint32_t tcount = 0;
      bool ok = true;
      // The stacked rows of a tile (the only tile metadata this role needs) come from the unpack warps, which decode
      // every tile anyway: a global load here, two dependent levels of them, would stall the one thread that feeds
      // the tensor core for thousands of cycles per tile.
      for (int tile = g.pair; ok && tile < g.num_tiles; tile += g.npairs, ++tcount) {
        const int buf = tcount & 1;
        const uint32_t aph = (tcount >> 1) & 1;
        if (!mbar_wait<true>(g.tempty0 + 8u * buf, aph ^ 1, g.abort_flag, p.f.status)) { ok = false; break; }
        uint32_t idesc = 0;
        const uint32_t d_tmem = tmem_base + buf * kAccCols;
        for (int ks = 0; ks < p.ksteps; ++ks, rp.advance(1, depth)) {
          // (a plain wait: these threads read none of the stage's bytes themselves -- the tensor cores of the two SMs
          // do, for which the writers' proxy fences and the copies' own completion have made them visible)
          if (!mbar_wait(g.full0 + 8u * rp.slot, rp.phase, g.abort_flag, p.f.status)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          // (written by an unpack warp of this CTA before its arrival on the barrier just waited for)
          if (ks == 0) idesc = idesc_i8(2 * kTileM, pair_mma_rows(g.ntot[tcount % kTileRing], p.f.bits));
          const uint32_t so = rp.slot * (kStageBytes >> 4);
          const int nsub = min(kSub, p.kblocks - ks * kSub);
          if (elect_one()) {
            for (int sub = 0; sub < nsub; ++sub) {
              const uint32_t al = a_lo + so + static_cast<uint32_t>(sub * (kABytes >> 4));
              const uint32_t bl = b_lo + so + static_cast<uint32_t>(sub * (kBtBytes >> 4));
#pragma unroll
              for (int k = 0; k < kKStep / 32; ++k)
                mma_i8_pair(d_tmem, (static_cast<uint64_t>(a_hi) << 32) | (al + 2u * k), (static_cast<uint64_t>(b_hi) << 32) | (bl + 2u * k), idesc,
                            (ks | sub | k) != 0);
            }
            mma_commit_pair(g.done0 + 8u * rp.slot);   // frees the stage for the producers of both CTAs
          }
          __syncwarp();
        }
        if (ok && elect_one()) mma_commit_pair(g.tfull0 + 8u * buf);
        __syncwarp();
      }
    }
  } else if (warp < 2 + kUnpackWarps) {
    // ------------------------------------------------------------------ unpack warps
    if (p.f.bits == 8) unpack_role<8>(p, g, warp - 2, lane, smem_u32(pk_bars));
    else if (p.f.bits == 4) unpack_role<4>(p, g, warp - 2, lane, smem_u32(pk_bars));
    else unpack_role<2>(p, g, warp - 2, lane, smem_u32(pk_bars));
  } else {
    // ------------------------------------------------------------------ epilogue warps
    EpiCtx e;
    e.tmem_base = tmem_base;
    e.tfull0 = g.tfull0;
    e.tempty0 = g.tempty0;
    e.recbar0 = smem_u32(rec_bars);
    e.rec0 = smem_u32(tile_recs);
    e.prebar0 = smem_u32(pre_bars);
    e.cfold = &cfold_s[0][0];
    e.sx_s = sx_s;
    e.tempty_lead0 = g.tempty_lead0;
    e.rank = g.rank;
    e.pair = g.pair;
    e.npairs = g.npairs;
    e.tile_base = g.tile_base;
    e.num_tiles = g.num_tiles;
    e.abort_flag = g.abort_flag;
    e.warp = warp;
    e.lane = lane;
    const int ew = warp - 2 - kUnpackWarps;
    e.part = ew >> 2;
    e.nparts = kEpiWarps / 4;
    e.stg = epi_stage[ew];
    e.zero_s = smem_u32(zero8_s);
    if (p.f.partials) {   // verification output: every integer accumulator is also written out
      if (p.nkmax <= 2) epilogue_role<2, true, Q8, SUMMED, SHORT_K>(p, e);
      else if (p.nkmax <= 4) epilogue_role<4, true, Q8, SUMMED, SHORT_K>(p, e);
      else epilogue_role<8, true, Q8, SUMMED, SHORT_K>(p, e);
    } else {
      if (p.nkmax <= 2) epilogue_role<2, false, Q8, SUMMED, SHORT_K>(p, e);
      else if (p.nkmax <= 4) epilogue_role<4, false, Q8, SUMMED, SHORT_K>(p, e);
      else epilogue_role<8, false, Q8, SUMMED, SHORT_K>(p, e);
    }
  }

  // ---------------------------------------------------------------------- teardown
  // Neither CTA may free its tensor memory or leave while the peer can still signal its barriers or
  // the pair's MMAs can still read its shared memory: both meet at a cluster barrier first.
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// ---------------------------------------------------------------------------------------------
}  // namespace tc2

namespace tc2 {

// What a launch needs to know about the current device, asked once per device: the ring depth that fits its
// shared memory, the dynamic shared memory to request (the attribute is set on both instantiations then) and how
// many CTA pairs can be resident.
struct DeviceSetup {
  int depth = 0, dyn_smem = 0, max_pairs = 0;
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
    int smem_max = 0, sms = 0;
    if (cudaDeviceGetAttribute(&smem_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) return;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return;
    cudaFuncAttributes f0, f1, f2;
    if (cudaFuncGetAttributes(&f0, tc2_forward_kernel<false, false, false>) != cudaSuccess) return;
    if (cudaFuncGetAttributes(&f1, tc2_forward_kernel<true, false, false>) != cudaSuccess) return;
    if (cudaFuncGetAttributes(&f2, tc2_forward_kernel<false, true, false>) != cudaSuccess) return;
    size_t fixed_b = f0.sharedSizeBytes > f1.sharedSizeBytes ? f0.sharedSizeBytes : f1.sharedSizeBytes;
    fixed_b = fixed_b > f2.sharedSizeBytes ? fixed_b : f2.sharedSizeBytes;
    const int fixed = static_cast<int>(fixed_b);
    d.depth = (smem_max - fixed - 1024) / kStageBytes;   // static shared memory, alignment slack
    if (d.depth > kMaxRing) d.depth = kMaxRing;
    d.status = PIPE_ERR_UNSUPPORTED;
    if (d.depth * kSub != kUnpackWarps) return;   // every unpack warp owns one block slot of the ring
    d.dyn_smem = d.depth * kStageBytes + 1024;
    d.status = PIPE_ERR_CUDA;
    if (cudaFuncSetAttribute(tc2_forward_kernel<false, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, d.dyn_smem) != cudaSuccess) return;
    if (cudaFuncSetAttribute(tc2_forward_kernel<true, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, d.dyn_smem) != cudaSuccess) return;
    if (cudaFuncSetAttribute(tc2_forward_kernel<false, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, d.dyn_smem) != cudaSuccess) return;
    if (cudaFuncSetAttribute(tc2_forward_kernel<false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, d.dyn_smem) != cudaSuccess) return;
    if (cudaFuncSetAttribute(tc2_forward_kernel<true, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, d.dyn_smem) != cudaSuccess) return;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.gridDim = dim3(sms & ~1, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = d.dyn_smem;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    d.status = PIPE_ERR_UNSUPPORTED;
    if (cudaOccupancyMaxActiveClusters(&n, tc2_forward_kernel<false, false, false>, &cfg) != cudaSuccess || n < 1) return;
    d.max_pairs = n < sms / 2 ? n : sms / 2;
    d.status = PIPE_OK;
  });
  return setups[dev];
}

}  // namespace tc2

static pipe_status launch_tc2(const ForwardArgs& a, cudaStream_t stream, uint32_t split_mask = 0) {
  using namespace tc2;
  const DeviceSetup& ds = device_setup();
  if (ds.status != PIPE_OK) return ds.status;
  Params p;

  int max_cluster = 0;
  for (int m = 0; m < a.num_branches; ++m) max_cluster = max(max_cluster, a.branch[m].k_end - a.branch[m].k_begin);
  if (max_cluster > kMaxClusterOrders) return PIPE_ERR_UNSUPPORTED;
  // every branch needs the channel-block table of its cluster of orders (written by the expansion)
  for (int m = 0; m < a.num_branches; ++m)
    if (!a.branch[m].blk || !a.branch[m].rec) return PIPE_ERR_UNSUPPORTED;
  if (a.g % 8 != 0) return PIPE_ERR_UNSUPPORTED;
  int k_lo = PIPE_MAX_ORDERS, k_hi = 0;
  for (int m = 0; m < a.num_branches; ++m) {
    k_lo = min(k_lo, a.branch[m].k_begin);
    k_hi = max(k_hi, a.branch[m].k_end);
  }
  bool direct = true;   // every order of the call has its int8 copy
  for (int k = k_lo; k < k_hi; ++k) direct = direct && a.order[k].wcodes != nullptr;
  if (!direct && a.bits == 2 && a.g % 16 != 0) return PIPE_ERR_UNSUPPORTED;   // an unpack item is 16 rows of 2-bit codes and must lie in one order
  if (a.ldxq % 16 != 0) return PIPE_ERR_UNSUPPORTED;
  if (a.conv_on && a.cC % kKStep != 0) return PIPE_ERR_UNSUPPORTED;
  for (int m = 0; m < a.num_branches; ++m) {
    if (reinterpret_cast<uintptr_t>(a.branch[m].xq) & 15) return PIPE_ERR_UNSUPPORTED;
  }
  if (a.T > (1ll << 30)) return PIPE_ERR_UNSUPPORTED;

  p.f = a;
  p.direct = direct ? 1 : 0;
  p.split_mask = split_mask;
  const int row_bytes = direct ? round_up(a.I, kKStep) : a.kernel_row_bytes;   // bytes of a row over all reduction blocks
  if (direct) p.f.bits = 8;   // the kernel then treats the layer as one of int8 codes
  p.nkmax = max_cluster;
  p.ntok_tiles = static_cast<int>(ceil_div<int64_t>(a.T, kTileM));
  p.conv_pw = p.conv_pp = p.conv_np = p.conv_chunks = 1;
  if (a.conv_on) {
    p.conv_pw = ceil_div(a.cWo, 8);
    p.conv_pp = ceil_div(a.cHo, 8) * p.conv_pw;
    p.conv_np = p.conv_pp * a.cN;
    p.conv_chunks = a.cC / kKStep;
    p.ntok_tiles = ceil_div(p.conv_np, 2);
  }
  // (a single token tile: the second CTA of a pair then stages zeros and stores nothing, but still unpacks its half of
  // every block, which is what such a launch spends its time on)
  if (p.ntok_tiles == 1 && kernel_choice() == 0) {
    // ... unless the whole layer is a handful of blocks: then nothing is there to share and the one-SM kernel's shorter
    // set-up wins (a forced choice of this kernel still takes the launch)
    int64_t rows = 0;
    for (int m = 0; m < a.num_branches; ++m)
      for (int k = a.branch[m].k_begin; k < a.branch[m].k_end; ++k) rows += a.order[k].rows;
    if (rows <= 4 * PIPE_BLOCK_ROWS) return PIPE_ERR_UNSUPPORTED;
  }
  p.ntt = ceil_div(p.ntok_tiles, 2);
  // the tile count is known on the device only (block counts of the tables); a table never has more blocks than groups
  if (static_cast<int64_t>(a.G) * p.ntt * a.num_branches > INT32_MAX) return PIPE_ERR_UNSUPPORTED;
  p.kblocks = ceil_div(a.I, kKStep);
  p.ksteps = ceil_div(p.kblocks, kSub);
  {
    // bytes one branch sweeps in either order: its activations, or the packed rows of its orders
    const int64_t x_bytes = a.conv_on ? static_cast<int64_t>(a.cN) * a.cH * a.cW * a.cC : a.T * static_cast<int64_t>(a.I);
    int64_t w_bytes = 0;
    for (int k = a.branch[0].k_begin; k < a.branch[0].k_end; ++k) w_bytes += static_cast<int64_t>(a.order[k].rows) * row_bytes;
    // (sweeping the activations once per channel block is the better order while they stay in L2 beside the outputs
    // streaming through it -- the pairs working together then share one weight block -- so the other order is taken
    // only for activations of tens of megabytes)
    p.blocks_fastest = (x_bytes > w_bytes && x_bytes > (48ll << 20)) ? 1 : 0;
  }
  p.pk = kKStep * p.f.bits / 8;
  p.shift = 8 - p.f.bits;

  auto section = [&](int k) { return direct ? a.order[k].wcodes : a.order[k].kcodes; };
  const uint8_t* kbase = section(k_lo);
  for (int k = k_lo; k < k_hi; ++k) kbase = section(k) < kbase ? section(k) : kbase;
  p.kbase = kbase;
  for (int k = k_lo; k < k_hi; ++k) {
    const uint64_t d = static_cast<uint64_t>(section(k) - kbase);
    const uint64_t end = (d + static_cast<uint64_t>(a.order[k].rows) * row_bytes) >> 4;
    if ((d & 15) || end >= 0xffffffffull) return PIPE_ERR_UNSUPPORTED;
    p.koff[k] = static_cast<uint32_t>(d >> 4);
  }
  p.depth = ds.depth;

  if (a.conv_on) {
    for (int m = 0; m < a.num_branches; ++m)
      if (!make_map_nhwc(&p.tmap_a[m], a.branch[m].xq, a.cN, a.cH, a.cW, a.cC, a.csh, a.csw)) return PIPE_ERR_CUDA;
  } else
  for (int m = 0; m < a.num_branches; ++m) {
    if (!make_map_2d(&p.tmap_a[m], a.branch[m].xq, static_cast<uint64_t>(a.I), static_cast<uint64_t>(a.T),
                     static_cast<uint64_t>(a.ldxq), kKStep, kTileM, CU_TENSOR_MAP_SWIZZLE_128B))
      return PIPE_ERR_CUDA;
  }
  // fp32 outputs that tensor stores can write: 16-byte aligned rows of at least one box
  p.y_tma = 0;
  if (!a.q8_out && a.ldy % 4 == 0 && a.O >= 16) {
    for (int m = 0; m < a.num_branches; ++m) {
      const float* y = a.branch[m].y;
      if (!y || (reinterpret_cast<uintptr_t>(y) & 15) || a.branch[m].accumulate) continue;
      const bool ok = a.conv_on ? make_map_out_nhwc(&p.tmap_y[m], y, a.cN, a.cHo, a.cWo, static_cast<uint64_t>(a.O), static_cast<uint64_t>(a.ldy))
                                : make_map_out_2d(&p.tmap_y[m], y, static_cast<uint64_t>(a.O), static_cast<uint64_t>(a.T), static_cast<uint64_t>(a.ldy));
      if (ok) p.y_tma |= 1u << m;
    }
  }
  // one cluster of two CTAs per SM pair; the tiles (counted on the device) go round all resident pairs
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see the kernel's first lines
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.gridDim = dim3(2 * ds.max_pairs, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = ds.dyn_smem;
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  // (a reduction axis of at most 8 blocks: the drain paces the layer, see STRAIGHT in the epilogue)
  const bool short_k = p.kblocks <= 8;
  const cudaError_t e = a.q8_out    ? (short_k ? cudaLaunchKernelEx(&cfg, tc2_forward_kernel<true, false, true>, p)
                                               : cudaLaunchKernelEx(&cfg, tc2_forward_kernel<true, false, false>, p))
                        : split_mask ? cudaLaunchKernelEx(&cfg, tc2_forward_kernel<false, true, false>, p)
                        : short_k    ? cudaLaunchKernelEx(&cfg, tc2_forward_kernel<false, false, true>, p)
                                     : cudaLaunchKernelEx(&cfg, tc2_forward_kernel<false, false, false>, p);
  if (e != cudaSuccess) return PIPE_ERR_CUDA;
  count_launch(1);
  return launch_status();
}

pipe_status forward_tcgen05_pair(const ForwardArgs& a, cudaStream_t stream) {
  if (a.T == 0) return PIPE_OK;
  const bool sum_mode = a.num_branches > 1 && a.branch[1].accumulate;
  if (!sum_mode) return launch_tc2(a, stream);
  // Predictors that share one input (the first layer of an ensemble, Sec. 3.2): ONE launch on the cluster of all
  // orders -- the activations are staged once, the MMAs run at the width of the whole cluster, and the epilogue
  // closes each predictor's chain and adds them in ascending order in registers.
  if (a.sum_blk && a.sum_rec && !a.q8_out) {
    bool shared = true;
    for (int m = 1; m < a.num_branches; ++m)
      shared = shared && a.branch[m].xq == a.branch[0].xq && a.branch[m].sx == a.branch[0].sx &&
               a.branch[m].k_begin == a.branch[m - 1].k_end && a.branch[m].y == a.branch[0].y;
    const int k0 = a.branch[0].k_begin, k1 = a.branch[a.num_branches - 1].k_end;
    if (shared && k1 - k0 <= tc2::kMaxClusterOrders) {
      ForwardArgs one = a;
      one.num_branches = 1;
      one.branch[0] = a.branch[0];
      one.branch[0].k_end = k1;
      one.branch[0].blk = a.sum_blk;
      one.branch[0].rec = a.sum_rec;
      one.branch[0].accumulate = 0;
      uint32_t split = 0;
      for (int m = 1; m < a.num_branches; ++m) split |= 1u << (a.branch[m].k_begin - k0);
      const pipe_status st = launch_tc2(one, stream, split);
      if (st != PIPE_ERR_UNSUPPORTED) return st;
    }
  }
  // Summed ensemble: one launch per branch, in order, so that y = ((y_1 + y_2) + ...) is formed
  // by the same thread in a fixed order.
  for (int m = 0; m < a.num_branches; ++m) {
    ForwardArgs one = a;
    one.num_branches = 1;
    one.branch[0] = a.branch[m];
    pipe_status st = launch_tc2(one, stream);
    if (st != PIPE_OK) return st;
  }
  return PIPE_OK;
}

}  // namespace pipe
