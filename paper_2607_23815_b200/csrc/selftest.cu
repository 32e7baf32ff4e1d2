// Test surface: a tiny kernel that lets a bounded device-side wait run out on purpose.
//
// Every mbarrier wait of the tensor-core kernel gives up after a time limit, raises the CTA's abort flag, lets the
// other roles leave at their next wait, lets copies in flight land, frees the CTA's tensor memory and records
// KV_ERR_TIMEOUT.  In a healthy run none of that code executes.  This kernel walks the same exit path with the same
// primitives on one CTA and a limit chosen by the caller: one warp waits on a barrier that nobody will ever
// complete, another is parked on a second such barrier with a much longer limit and must be released by the abort
// flag, a third has a real bulk copy in flight.  Nothing faults, traps or spins without bound; the kernel ends
// normally and the device stays usable.
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace kvattn {
using namespace ptx;

struct __align__(128) SelftestSmem {
  unsigned char buf[256];
  unsigned long long bar_copy, bar_dead, bar_parked;
  uint32_t tmem_base;
  int abort_flag;
};

// trace[0]: the bulk copy landed (1); trace[1]: lanes of the waiting warp that gave up; trace[2]: the parked warp left
// because of the flag, before its own limit (1); trace[3]: nanoseconds the waiting warp spent.
__global__ void __launch_bounds__(128, 1) bounded_wait_selftest_kernel(int* status, const unsigned char* src,
                                                                      unsigned long long limit_ns, int* trace) {
  __shared__ SelftestSmem sm;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abortp = &sm.abort_flag;
  if (threadIdx.x == 0) {
    sm.abort_flag = 0;
    mbar_init(smem_u32(&sm.bar_copy), 1);
    mbar_init(smem_u32(&sm.bar_dead), 1);
    mbar_init(smem_u32(&sm.bar_parked), 1);
    fence_mbar_init();
  }
  if (warp == 0) {
    tmem_alloc(smem_u32(&sm.tmem_base), 32);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  if (warp == 1) {
    if (lane == 0) {
      mbar_arrive_expect_tx(smem_u32(&sm.bar_copy), 256);
      bulk_g2s(smem_u32(sm.buf), src, 256, smem_u32(&sm.bar_copy));
      // copies in flight are given time to land before the CTA's shared memory goes away (bounded on its own,
      // whatever the flag says)
      int never = 0;
      const bool landed = mbar_wait_limit(smem_u32(&sm.bar_copy), 0, &never, 100000000ull);
      trace[0] = landed ? 1 : 0;
    }
  } else if (warp == 2) {
    const uint64_t t0 = globaltimer_ns();
    const bool got = mbar_wait_limit(smem_u32(&sm.bar_dead), 0, abortp, limit_ns);  // nobody arrives on this one
    const unsigned gave_up = __ballot_sync(0xffffffffu, !got);
    if (lane == 0) {
      trace[1] = __popc(gave_up);
      trace[3] = (int)min((unsigned long long)(globaltimer_ns() - t0), 0x7fffffffull);
    }
  } else if (warp == 3) {
    const uint64_t t0 = globaltimer_ns();
    const bool got = mbar_wait_limit(smem_u32(&sm.bar_parked), 0, abortp, 64 * limit_ns);
    const uint64_t dt = globaltimer_ns() - t0;
    const bool by_flag = !got && dt < 32 * limit_ns;
    if (lane == 0) trace[2] = __all_sync(0x1u, by_flag) ? 1 : 0;
  }
  tc_fence_before_sync();
  __syncthreads();
  if (threadIdx.x == 0 && sm.abort_flag != 0) report(status, KV_ERR_TIMEOUT);
  if (warp == 0) tmem_dealloc(sm.tmem_base, 32);
}

}  // namespace kvattn

using namespace kvattn;

extern "C" kv_status_t kvattn_selftest_bounded_wait(kv_pool_t* p, unsigned long long limit_ns, int* trace, void* stream) {
  if (p == nullptr || trace == nullptr || limit_ns == 0 || limit_ns > 100000000ull) return KV_ERR_INVALID;
  if (!on_pool_device(p)) return KV_ERR_INVALID;
  bounded_wait_selftest_kernel<<<1, 128, 0, (cudaStream_t)stream>>>(p->d_status, (const unsigned char*)p->k_base, limit_ns,
                                                                    trace);
  count_launch();
  KV_CUDA_OK(cudaGetLastError());
  return KV_OK;
}
