// Self-test of the bounded waits.  The tensor-core kernels promise that a wait which cannot
// complete ends with ELITEKV_ERR_TIMEOUT in the status word instead of a hang.  Nothing in a
// healthy run makes a wait run out, so this stand-alone kernel does: it waits, with the very
// helpers the kernels use but a short probe limit, on a barrier that nobody arrives on.  No
// copy, no tensor memory, no MMA is involved; the block records what happened and returns.
#include "tc_ptx.cuh"

namespace {

constexpr int kSelfThreads = 128;

__global__ void __launch_bounds__(kSelfThreads)
bounded_wait_selftest_kernel(unsigned limit, int32_t* status) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int s_abort, s_seen[3];
  __shared__ int s_verdict[2];
  const int warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    s_abort = 0;
    s_seen[0] = s_seen[1] = s_seen[2] = 0;
  }
  __syncthreads();
  volatile int* abort_flag = &s_abort;
  const uint32_t b = smem_u32(&bar);
  // (1) one thread, test_wait probes
  if (threadIdx.x == 0) {
    const bool ok = mbar_spin(b, 0, abort_flag, 1, limit);
    s_seen[0] = (!ok && s_abort == 1) ? 1 : 0;
    s_abort = 0;
  }
  __syncthreads();
  // (2) a whole warp, warp-uniform outcome
  if (warp == 1) {
    const bool ok = warp_wait(b, 0, abort_flag, 2, limit);
    const bool agree = __all_sync(0xffffffffu, !ok);
    __syncwarp();
    if ((threadIdx.x & 31) == 0) {
      s_seen[1] = (agree && s_abort == 2) ? 1 : 0;
      s_abort = 0;
    }
  }
  __syncthreads();
  // (3) a group with a polling leader: every thread must get the leader's outcome
  {
    unsigned turn = 0;
    const bool ok = mbar_wait_group(b, 0, abort_flag, s_verdict, turn, threadIdx.x == 0, 1, kSelfThreads, 3, limit);
    const int gave_up = __syncthreads_and(!ok);
    if (threadIdx.x == 0) s_seen[2] = (gave_up && s_abort == 3) ? 1 : 0;
  }
  __syncthreads();
  if (threadIdx.x == 0) ekv_record(status, ELITEKV_ERR_TIMEOUT, s_seen[0] | (s_seen[1] << 1) | (s_seen[2] << 2), (int)limit);
}

}  // namespace

extern "C" int elitekv_selftest_bounded_wait(const elitekv_layer* L, uint32_t poll_limit, elitekv_stream_t stream) {
  if (!L || poll_limit == 0 || poll_limit > (1u << 20)) return ELITEKV_ERR_INVALID_ARG;
  bounded_wait_selftest_kernel<<<1, kSelfThreads, 0, (cudaStream_t)stream>>>(poll_limit, L->d_status);
  EKV_CUDA_OK(cudaGetLastError());
  return ELITEKV_OK;
}
