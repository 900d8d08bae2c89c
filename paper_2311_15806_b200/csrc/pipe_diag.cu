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
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = tmem_base_slot;
  if (threadIdx.x == 0) {
    const uint64_t adesc = smem_desc_sw128(base), bdesc = smem_desc_sw128(base + kProbeABytes);
    const uint32_t idesc = idesc_i8(128, n_cols);
    long long issued = 0;
    uint32_t batch = 0;
    bool ok = true;
    while (ok && issued < mma_per_cta) {
      // at most two batches in flight: before batch b is issued, batch b - 2 has completed
      if (batch >= 2 && !mbar_wait(smem_u32(&bars[batch & 1]), ((batch >> 1) - 1) & 1, &abort_flag_s, status)) { ok = false; break; }
      const int nb = static_cast<int>(min(static_cast<long long>(kProbeBatch), mma_per_cta - issued));
      for (int i = 0; i < nb; ++i) {
        const uint64_t ks = static_cast<uint64_t>((i & 3) * 2);   // the four 32-byte slices of the 128-byte rows
        mma_i8(tmem_base + (i & 1) * 256, adesc + ks, bdesc + ks, idesc, (issued + i) >= 2);
      }
      mma_commit(smem_u32(&bars[batch & 1]));
      issued += nb;
      ++batch;
    }
    // all batches done before tensor memory is freed
    for (uint32_t b = (batch >= 2 ? batch - 2 : 0); ok && b < batch; ++b)
      if (!mbar_wait(smem_u32(&bars[b & 1]), (b >> 1) & 1, &abort_flag_s, status)) ok = false;
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
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

extern "C" pipe_status pipe_diag_mma_i8_rate(int32_t n_cols, int64_t mma_per_cta, double* h_ops_per_launch, void* stream) {
  if (!h_ops_per_launch || n_cols < 16 || n_cols > 256 || n_cols % 16 != 0 || mma_per_cta < 1 || mma_per_cta > (1ll << 40))
    return PIPE_ERR_INVALID_ARG;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return PIPE_ERR_CUDA;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) return PIPE_ERR_CUDA;
  int* status = device_status_word();
  if (!status) return PIPE_ERR_CUDA;
  const int dyn = diag::kProbeABytes + diag::kProbeBBytes + 1024;
  if (cudaFuncSetAttribute(diag::mma_i8_rate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn) != cudaSuccess)
    return PIPE_ERR_CUDA;
  diag::mma_i8_rate_kernel<<<sms, diag::kProbeThreads, dyn, static_cast<cudaStream_t>(stream)>>>(n_cols, mma_per_cta, status);
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
