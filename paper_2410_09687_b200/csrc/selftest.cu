// Self-test of the bounded device-side wait: the expiry branch that no healthy run ever takes.
//
// Every mbarrier wait in the TMA / tcgen05 kernels goes through mbar_wait, which gives up after a time limit,
// raises the CTA's abort flag and the device status flag, and lets the kernel drain and return.  This kernel
// takes exactly that path on purpose and harmlessly: one warp waits on a barrier that nothing ever arms,
// with nothing in flight, under a limit given in microseconds.
#include "ptx.cuh"

namespace moin {

constexpr int kSelftestSite = 99;

__global__ void __launch_bounds__(64) bounded_wait_probe_kernel(DeviceStatus* status, unsigned long long limit_ns,
                                                                int* result) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_flag;
  const uint32_t b = smem_u32(&bar);
  if (threadIdx.x == 0) {
    mbar_init(b, 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const unsigned long long t0 = global_ns();
  bool ok = true;
  if (threadIdx.x == 0) ok = mbar_wait(b, 0u, &abort_flag, status, kSelftestSite, limit_ns);   // the waiter that runs out
  __syncthreads();
  // a second waiter, as the other roles of a pipeline would be: it must leave through the abort flag
  bool ok2 = true;
  if (threadIdx.x == 32) ok2 = mbar_wait(b, 0u, &abort_flag, status, kSelftestSite + 1, 1000ull * limit_ns);
  __syncthreads();
  if (threadIdx.x == 0) {
    result[0] = ok ? 1 : 0;                                // 0: the wait gave up, as it should
    result[2] = (int)((global_ns() - t0) / 1000ull);       // microseconds spent
  }
  if (threadIdx.x == 32) result[1] = ok2 ? 1 : 0;          // 0: left because the CTA was aborting
}

}  // namespace moin

using namespace moin;

extern "C" moin_status moin_selftest_bounded_wait(int32_t limit_us, int32_t* result, moin_stream stream) {
  if (!result || limit_us < 1 || limit_us > 1000000) return MOIN_ERR_INVALID_ARG;
  HostState* hs;
  moin_status st = host_state(&hs);
  if (st) return st;
  bounded_wait_probe_kernel<<<1, 64, 0, (cudaStream_t)stream>>>(hs->status, 1000ull * (unsigned long long)limit_us, result);
  return record_cuda(cudaGetLastError());
}
