// Device and host helpers shared by the tcgen05 kernels of libpipe (one-SM kernel, SM-pair kernel, decode
// kernel, diagnostics): mbarrier operations with bounded waits, TMA tensor loads, the shared-memory matrix
// descriptor and the instruction descriptor of tcgen05.mma kind::i8, accumulator loads, the conversion-free
// re-quantization of the fused inner-layer epilogue, and tensor-map encoding through the runtime's
// driver-entry-point query.  The descriptor encodings, the 128-byte swizzle and the tensor-map call are fixed by
// the hardware interface.
#pragma once

#include <cuda.h>

#include <mutex>

#include "pipe_common.cuh"

namespace pipe {
namespace tcc {

constexpr long long kWaitLimitCycles = 4000000000ll;  // about 2 s per wait at the maximum SM clock

// Position in a ring of `depth` slots: slot index and phase parity, advanced without divisions.
struct RingPos {
  uint32_t slot, phase;
  __device__ __forceinline__ void advance(uint32_t by, uint32_t depth) {  // by <= depth
    slot += by;
    if (slot >= depth) {
      slot -= depth;
      phase ^= 1u;
    }
  }
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

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
// For barriers that the other CTA of a pair signals: the wait acquires at cluster scope.
__device__ __forceinline__ bool mbar_try_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}

// Bounded wait.  Returns false when the CTA is aborting (this wait or another one expired).
// The bound is counted in SM cycles; the abort flag and the clock are looked at only every few
// polls so that a barrier that completes soon is seen with little delay.
// SLEEP_NS > 0: a wait that is expected to last long (an epilogue warp waiting for a whole tile's MMAs) backs off
// between polls, so that its polling does not take shared-memory and issue slots from the warps that feed the MMAs.
template <bool CLUSTER = false, int SLEEP_NS = 0>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status,
                                          long long limit = kWaitLimitCycles) {
  if (CLUSTER ? mbar_try_cluster(bar, parity) : mbar_try(bar, parity)) return true;
  const long long t0 = clock64();
  while (true) {
#pragma unroll 1
    for (int i = 0; i < 16; ++i) {
      if (CLUSTER ? mbar_try_cluster(bar, parity) : mbar_try(bar, parity)) return true;
      if (SLEEP_NS > 0) __nanosleep(SLEEP_NS);
    }
    if (*abort_flag) return false;
    if (clock64() - t0 > limit) {
      *abort_flag = 1;
      raise_status(status, PIPE_ERR_TIMEOUT);
      return false;
    }
  }
}

// After the last issue: wait (bounded) until the copies of the last `depth` ring slots have landed,
// so that no copy is still writing into this CTA's shared memory when it exits.
__device__ __forceinline__ void drain_ring(uint32_t full0, uint32_t issued, int depth, long long limit = kWaitLimitCycles) {
  for (uint32_t j = (issued > static_cast<uint32_t>(depth) ? issued - depth : 0); j < issued; ++j) {
    const int s = j % depth;
    const uint32_t ph = (j / depth) & 1;
    const long long t0 = clock64();
    while (!mbar_try(full0 + 8u * s, ph) && clock64() - t0 < limit) {
    }
  }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar)
      : "memory");
}

// Four-dimensional tile of an NHWC tensor (coordinates innermost first: channel, x, y, image);
// coordinates outside the tensor read zeros, which is the convolution's padding.
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar)
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

// Instruction descriptor: D = int32, A and B = signed int8, both K-major, M = m (128, or 256 over an SM pair), N = n.
__device__ __forceinline__ uint32_t idesc_i8(int m, int n) {
  return (2u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(m >> 4) << 24);
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

// The code clamp(rne(v / s)) of the fused inner-layer epilogue without a conversion instruction: the estimate
// t = v * rn(1 / s), clamped to +-127 (a t beyond 127 has a true quotient above 126.9999, whose code is 127),
// is added to 1.5 * 2^23, where the spacing of binary32 is one, so the addition itself rounds to the nearest
// integer, ties to even, and leaves the code in the low byte of the sum.  `edge` collects the largest
// |t - code| + |t| * 2^-21: at 0.5 or more an estimate lies so close to a rounding boundary that the IEEE
// quotient, which defines the code, may round the other way, and the caller divides.
__device__ __forceinline__ float quant_magic(float v, float r, float& edge) {
  const float t = fminf(fmaxf(__fmul_rn(v, r), -127.f), 127.f);
  const float u = __fadd_rn(t, 12582912.f);
  const float d = __fsub_rn(t, __fsub_rn(u, 12582912.f));
  edge = fmaxf(edge, __fmaf_rn(fabsf(t), 4.76837158203125e-07f, fabsf(d)));
  return u;
}

__device__ __forceinline__ uint32_t pack4_low_bytes(float a, float b, float c, float d) {
  const uint32_t ab = __byte_perm(__float_as_uint(a), __float_as_uint(b), 0x0040);
  const uint32_t cd = __byte_perm(__float_as_uint(c), __float_as_uint(d), 0x0040);
  return __byte_perm(ab, cd, 0x5410);
}

// ---------------------------------------------------------------------------------------------
using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeFn encode_fn() {
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

inline bool make_map_2d(CUtensorMap* map, const void* base, uint64_t inner_bytes, uint64_t rows, uint64_t pitch_bytes,
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

// NHWC int8 tensor as a 4-D map; one box = 128 channels x 8 x 8 pixels of one image (64 rows of 128 bytes).
inline bool make_map_nhwc(CUtensorMap* map, const void* base, int N, int H, int W, int C, int sh, int sw) {
  EncodeFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[4] = {static_cast<cuuint64_t>(C), static_cast<cuuint64_t>(W), static_cast<cuuint64_t>(H),
                              static_cast<cuuint64_t>(N)};
  const cuuint64_t strides[3] = {static_cast<cuuint64_t>(C), static_cast<cuuint64_t>(W) * C,
                                 static_cast<cuuint64_t>(H) * W * C};
  // 8 x 8 pixels at the convolution's stride: the box spans 8 * stride positions and the copy takes every
  // stride-th of them
  const cuuint32_t box[4] = {128, static_cast<cuuint32_t>(8 * sw), static_cast<cuuint32_t>(8 * sh), 1};
  const cuuint32_t estr[4] = {1, static_cast<cuuint32_t>(sw), static_cast<cuuint32_t>(sh), 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// fp32 output [rows, channels] with a row pitch: one box = 16 channels x 32 rows (64-byte rows, 64-byte swizzle).
inline bool make_map_out_2d(CUtensorMap* map, const float* base, uint64_t channels, uint64_t rows, uint64_t pitch_elems) {
  EncodeFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {channels, rows};
  const cuuint64_t strides[1] = {pitch_elems * 4};
  const cuuint32_t box[2] = {16, 32};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// fp32 output of a convolution, pixels in NHW order with a pixel pitch: one box = 16 channels x 8 pixels x 4 image
// rows of one image (half of an 8 x 8 patch); what hangs over the right or lower edge of the image is not written.
inline bool make_map_out_nhwc(CUtensorMap* map, const float* base, int N, int Ho, int Wo, uint64_t channels, uint64_t pitch_elems) {
  EncodeFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[4] = {channels, static_cast<cuuint64_t>(Wo), static_cast<cuuint64_t>(Ho), static_cast<cuuint64_t>(N)};
  const cuuint64_t strides[3] = {pitch_elems * 4, pitch_elems * 4 * Wo, pitch_elems * 4 * Wo * Ho};
  const cuuint32_t box[4] = {16, 8, 4, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<float*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace tcc
}  // namespace pipe
