// Self-test of the bounded waits (not part of the public header): a kernel that waits on a barrier
// nobody ever arrives on, through the same wait routines the tensor-core kernels use, with a limit
// given by the caller.  The wait must give up, record its code in the device status word and let the
// kernel return, so that the context stays usable; rocs_last_device_status then reports
// ROCS_ERR_TIMEOUT.  Nothing here faults, traps or spins without a bound.
#include "rocs_internal.h"
#include "sm100_ptx.cuh"

namespace rocs {
namespace {

using namespace ptx;

constexpr uint32_t kStatusSelftest = 0x700;

__global__ void wait_expires_kernel(uint32_t* status, uint64_t limit_ns, int flavour, uint32_t* gave_up) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ AbortFlag abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag.v = 0;
    fence_mbar_init();
  }
  __syncthreads();
  bool ok;
  if (flavour == 0)
    ok = mbar_wait(&bar, 0, &abort_flag, status, kStatusSelftest | 1, limit_ns);
  else if (flavour == 1)
    ok = mbar_wait_paced(&bar, 0, &abort_flag, status, kStatusSelftest | 2, limit_ns);
  else
    ok = mbar_wait_paced(smem_u32(&bar), 0, &abort_flag, status, kStatusSelftest | 3, limit_ns);
  if (!ok) atomicAdd(gave_up, 1u);  // every waiting thread leaves through the abort path
}

}  // namespace
}  // namespace rocs

// flavour 0: hinted wait of the GEMM kernels, 1: paced wait, 2: paced wait on a shared-memory address.
// gave_up_dev (device, zeroed by the caller) counts the threads that returned through the abort path.
extern "C" rocs_status_t rocs_selftest_wait_expires(int flavour, uint32_t limit_us, uint32_t* gave_up_dev,
                                                    void* stream) {
  if (flavour < 0 || flavour > 2 || limit_us == 0 || limit_us > 1000000u || !gave_up_dev) return ROCS_ERR_INVALID_ARG;
  uint32_t* status = rocs::device_status_word();
  if (!status) return ROCS_ERR_CUDA;
  rocs::wait_expires_kernel<<<1, 64, 0, (cudaStream_t)stream>>>(status, (uint64_t)limit_us * 1000ull, flavour,
                                                               gave_up_dev);
  ROCS_CUDA_TRY(cudaGetLastError());
  return ROCS_OK;
}
