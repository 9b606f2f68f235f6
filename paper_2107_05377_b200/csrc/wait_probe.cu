// The bounded wait of the tensor-core kernels, exercised in miniature: what a pipeline role does when the barrier
// it waits on never completes.  Every mbarrier wait of gemm_bf16_tcgen05, the GEMM + LayerNorm cluster kernels and
// the tensor-memory attention kernels goes through mbar_wait (tc_ptx.cuh): it polls, looks at the CTA's abort flag
// and at %globaltimer every 256 polls, and after the limit raises the flag and returns false; the other roles see
// the flag at their next look and leave their loops too, and the CTA reports kFlagWaitTimeout in the status word.
// This kernel runs that protocol with two warps and two barriers and a limit of the caller's choosing (the
// kernels' own is 4 s), so that a test can make a wait run out in milliseconds: no barrier is ever left waiting
// for longer than the limits given, nothing faults, and the context stays usable.
//
//   warp 0 ("consumer"): waits on barrier A with `limit_ns`
//   warp 1 ("producer"): waits on barrier B with 64 * limit_ns - in the failing case it can only leave early
//                        because warp 0 raised the abort flag
//   arrive != 0: thread 0 arrives on both barriers first, the waits succeed at once and no flag is raised.

#include "tc_ptx.cuh"

namespace mt {
namespace {

struct WaitProbeParams {
  unsigned long long limit_ns;
  int arrive;
  uint32_t* status;
  unsigned long long* waited_ns;   // [2]
  int* ok_out;                     // [2]
};

__global__ void __launch_bounds__(64) wait_probe_kernel(const WaitProbeParams p) {
  const unsigned long long limit_ns = p.limit_ns;
  const int arrive = p.arrive;
  uint32_t* status = p.status;
  unsigned long long* waited_ns = p.waited_ns;
  int* ok_out = p.ok_out;
  __shared__ __align__(8) unsigned long long bars[2];
  __shared__ int abort_flag_s;
  volatile int* abort_flag = &abort_flag_s;
  const uint32_t bar_a = smem_u32(&bars[0]);
  const uint32_t bar_b = smem_u32(&bars[1]);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    mbar_init(bar_a, 1);
    mbar_init(bar_b, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (arrive != 0) {
      mbar_arrive(bar_a);
      mbar_arrive(bar_b);
    }
  }
  __syncthreads();
  grid_dependency_wait();
  grid_launch_dependents();
  const unsigned long long t0 = global_timer_ns();
  const bool ok = warp == 0 ? mbar_wait_for(bar_a, 0, abort_flag, limit_ns)
                            : mbar_wait_for(bar_b, 0, abort_flag, 64 * limit_ns);
  const unsigned long long t1 = global_timer_ns();
  if (lane == 0) {
    ok_out[warp] = ok ? 1 : 0;
    waited_ns[warp] = t1 - t0;
  }
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag && status != nullptr) atomicOr(status, kFlagWaitTimeout);
}

}  // namespace

cudaError_t launch_wait_probe(unsigned long long limit_ns, int arrive, uint32_t* status, unsigned long long* waited_ns,
                              int* ok_out, cudaStream_t stream) {
  WaitProbeParams p;
  p.limit_ns = limit_ns; p.arrive = arrive; p.status = status; p.waited_ns = waited_ns; p.ok_out = ok_out;
  return launch_kernel(wait_probe_kernel, dim3(1), dim3(64), 0, stream, p);
}

}  // namespace mt
