// Diagnostic and test-only entry points (include/pipe_diag.h): the issue-rate probe of the integer tensor
// pipe and a kernel whose only job is to let a bounded wait run out.
#include "pipe_diag.h"
#include "pipe_tc_common.cuh"

namespace pipe {
namespace diag {

using namespace tcc;

constexpr int kProbeThreads = 128;
constexpr int kProbeABytes = 128 * 128;   // 128 rows x 128 reduction bytes
constexpr int kProbeBBytes = 256 * 128;
constexpr int kProbeBatch = 64;           // instructions per commit

// PAIR: clusters of two CTAs, the first CTA of a pair issues tcgen05.mma.cta_group::2 (M = 256 over both SMs, each
// CTA holding its 128 rows of A and half of the n_cols rows of B).
template <bool PAIR>
__global__ void __launch_bounds__(kProbeThreads, 1) mma_i8_rate_kernel(int n_cols, long long mma_per_cta, int* status) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t bars[2];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag_s;
  const int warp = threadIdx.x >> 5;
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  // operands: a fixed pseudo-random byte pattern (the pipe's rate does not depend on the values; its power does)
  for (int i = threadIdx.x; i < (kProbeABytes + kProbeBBytes) / 4; i += kProbeThreads) {
    uint32_t v = static_cast<uint32_t>(i) * 2654435761u + 0x9e3779b9u * (blockIdx.x + 1);
    v ^= v >> 15;
    v *= 2246822519u;
    v ^= v >> 13;
    reinterpret_cast<uint32_t*>(gen)[i] = v;
  }
  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    mbar_init(smem_u32(&bars[0]), 1);
    mbar_init(smem_u32(&bars[1]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (warp == 0) {
    if (PAIR) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(512) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(512) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  uint32_t rank = 0;
  if (PAIR) {
    // both CTAs' operands and tensor memory are in place before the first instruction of the pair
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = tmem_base_slot;
  if (threadIdx.x == 0 && rank == 0) {
    const uint64_t adesc = smem_desc_sw128(base), bdesc = smem_desc_sw128(base + kProbeABytes);
    const uint32_t idesc = idesc_i8(PAIR ? 256 : 128, n_cols);
    long long issued = 0;
    uint32_t batch = 0;
    bool ok = true;
    while (ok && issued < mma_per_cta) {
      // at most two batches in flight: before batch b is issued, batch b - 2 has completed
      if (batch >= 2 && !mbar_wait(smem_u32(&bars[batch & 1]), ((batch >> 1) - 1) & 1, &abort_flag_s, status)) { ok = false; break; }
      const int nb = static_cast<int>(min(static_cast<long long>(kProbeBatch), mma_per_cta - issued));
      for (int i = 0; i < nb; ++i) {
        const uint64_t ks = static_cast<uint64_t>((i & 3) * 2);   // the four 32-byte slices of the 128-byte rows
        if (PAIR) {
          const uint32_t acc = (issued + i) >= 2 ? 1u : 0u;
          asm volatile(
              "{\n\t.reg .pred p;\n\t"
              "setp.ne.u32 p, %4, 0;\n\t"
              "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_base + (i & 1) * 256),
              "l"(adesc + ks), "l"(bdesc + ks), "r"(idesc), "r"(acc)
              : "memory");
        } else {
          mma_i8(tmem_base + (i & 1) * 256, adesc + ks, bdesc + ks, idesc, (issued + i) >= 2);
        }
      }
      if (PAIR) {
        asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&bars[batch & 1])) : "memory");
      } else {
        mma_commit(smem_u32(&bars[batch & 1]));
      }
      issued += nb;
      ++batch;
    }
    // all batches done before tensor memory is freed
    for (uint32_t b = (batch >= 2 ? batch - 2 : 0); ok && b < batch; ++b)
      if (!mbar_wait(smem_u32(&bars[b & 1]), (b >> 1) & 1, &abort_flag_s, status)) ok = false;
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  // the second CTA's shared memory and tensor memory stay in place until the first CTA's instructions are done
  if (PAIR) asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
  if (warp == 0) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (PAIR) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
}

__global__ void bounded_wait_kernel(long long limit_cycles, int* status) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag_s;
  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    // phase 0 of this barrier never completes: there is no arrival anywhere in this kernel
    mbar_wait(smem_u32(&bar), 0, &abort_flag_s, status, limit_cycles);
  }
}

}  // namespace diag
}  // namespace pipe

using namespace pipe;

extern "C" pipe_status pipe_diag_mma_i8_rate(int32_t n_cols, int64_t mma_per_cta, int32_t cta_pairs, double* h_ops_per_launch,
                                             void* stream) {
  if (!h_ops_per_launch || n_cols < 16 || n_cols > 256 || n_cols % 16 != 0 || mma_per_cta < 1 || mma_per_cta > (1ll << 40))
    return PIPE_ERR_INVALID_ARG;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return PIPE_ERR_CUDA;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) return PIPE_ERR_CUDA;
  int* status = device_status_word();
  if (!status) return PIPE_ERR_CUDA;
  const int dyn = diag::kProbeABytes + diag::kProbeBBytes + 1024;
  if (cta_pairs) {
    if (cudaFuncSetAttribute(diag::mma_i8_rate_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn) != cudaSuccess)
      return PIPE_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.gridDim = dim3(sms & ~1, 1, 1);
    cfg.blockDim = dim3(diag::kProbeThreads, 1, 1);
    cfg.dynamicSmemBytes = dyn;
    cfg.stream = static_cast<cudaStream_t>(stream);
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int pairs = 0;
    if (cudaOccupancyMaxActiveClusters(&pairs, diag::mma_i8_rate_kernel<true>, &cfg) != cudaSuccess || pairs < 1) return PIPE_ERR_UNSUPPORTED;
    if (2 * pairs < static_cast<int>(cfg.gridDim.x)) cfg.gridDim = dim3(2 * pairs, 1, 1);
    if (cudaLaunchKernelEx(&cfg, diag::mma_i8_rate_kernel<true>, n_cols, static_cast<long long>(mma_per_cta), status) != cudaSuccess)
      return PIPE_ERR_CUDA;
    count_launch(1);
    // one instruction of a pair is M = 256: mma_per_cta instructions per PAIR
    *h_ops_per_launch = 2.0 * 256.0 * n_cols * 32.0 * static_cast<double>(mma_per_cta) * (cfg.gridDim.x / 2);
    return launch_status();
  }
  if (cudaFuncSetAttribute(diag::mma_i8_rate_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn) != cudaSuccess)
    return PIPE_ERR_CUDA;
  diag::mma_i8_rate_kernel<false><<<sms, diag::kProbeThreads, dyn, static_cast<cudaStream_t>(stream)>>>(n_cols, mma_per_cta, status);
  count_launch(1);
  *h_ops_per_launch = 2.0 * 128.0 * n_cols * 32.0 * static_cast<double>(mma_per_cta) * sms;
  return launch_status();
}

extern "C" pipe_status pipe_diag_bounded_wait(int64_t limit_cycles, void* stream) {
  if (limit_cycles < 1 || limit_cycles > (1ll << 31)) return PIPE_ERR_INVALID_ARG;
  int* status = device_status_word();
  if (!status) return PIPE_ERR_CUDA;
  diag::bounded_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(limit_cycles, status);
  count_launch(1);
  return launch_status();
}
