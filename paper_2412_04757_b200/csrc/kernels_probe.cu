// Test kernel for the bounded device-side waits of the tensor-core kernels (tc_util.cuh): it exercises, on purpose
// and safely, the path that a production kernel takes only when something upstream of it never arrives.
//
// One CTA of two warps.  Lane 0 of warp 0 waits on an mbarrier that nothing ever completes, with a short limit: the
// wait gives up, raises the CTA's abort flag and returns false.  Lane 0 of warp 1 waits on the same barrier with the
// context's normal limit and is released by the abort flag.  Both then meet at the CTA barrier and the status word
// gets LTRI_ETIMEOUT, as at the end of k_attn_tc / k_map_tc / k_score_tc.  Nothing traps, faults or spins without
// bound: the longest possible run is the context's normal limit (about a second).
#include "common.cuh"
#include "tc_util.cuh"

namespace ltri {

using namespace tc;

__global__ void __launch_bounds__(64) k_wait_probe(DevCtx c, long long short_limit) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int s_abort;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    s_abort = 0;
    mbar_init(smem_addr(&bar), 1);
    fence_mbar_init();
  }
  __syncthreads();
  if (lane == 0) {
    const long long t0 = clock64();
    const bool done = mbar_wait(smem_addr(&bar), 0, &s_abort, warp == 0 ? short_limit : c.wait_limit);
    const long long waited = clock64() - t0;
    // cycles each waiter spent, for the host to look at (saturated to 31 bits); a wait that "succeeded" reports -1
    c.status[2 + warp] = done ? -1 : (int)(waited > 0x7fffffffll ? 0x7fffffffll : waited);
  }
  __syncthreads();
  if (threadIdx.x == 0 && s_abort) set_status(c, -6, 9000);
}

cudaError_t launch_wait_probe(const DevCtx& c, long long short_limit, cudaStream_t s) {
  k_wait_probe<<<1, 64, 0, s>>>(c, short_limit);
  return cudaGetLastError();
}

}  // namespace ltri
