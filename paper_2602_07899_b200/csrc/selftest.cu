// Diagnostics: the error path of the bounded barrier waits, exercised without a fault or a hang; and the guard
// words that a debugging caller can have placed between the regions of a workspace.
//
// Every wait inside the tensor-core kernels gives up after a cycle limit, records TLQ_ERR_TIMEOUT in the
// workspace header and lets the kernel finish.  In a correct run that path is never taken, so this file
// provides the one safe way to take it: a single warp waits, with a caller-chosen short limit, on a barrier
// that by construction nobody arrives on.  The wait expires, the status word is written, the kernel returns
// normally and the context stays usable.  Nothing here touches tensor memory or issues a copy.
#include "common.cuh"
#include "umma.cuh"

namespace tlq {

__global__ void bounded_wait_selftest_kernel(WorkspaceHeader* hdr, long long limit_cycles) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    ptx::mbar_init(ptx::smem_u32(&bar), 1);
    abort_flag = 0;
    ptx::fence_barrier_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    // phase 0 of a barrier that expects one arrival and gets none
    if (!ptx::mbar_wait(ptx::smem_u32(&bar), 0u, &abort_flag, limit_cycles)) {
      hdr->where = 99;
      hdr->status = TLQ_ERR_TIMEOUT;
    }
  }
  __syncthreads();
  // the second lane sees the flag the first one left behind: how the other roles of a CTA learn of a timeout
  if (threadIdx.x == 1 && abort_flag != 0) hdr->selftest = 1;
}

int launch_bounded_wait_selftest(WorkspaceHeader* hdr, long long limit_cycles, cudaStream_t st) {
  bounded_wait_selftest_kernel<<<1, 32, 0, st>>>(hdr, limit_cycles);
  return after_launch();
}

// ---------------------------------------------------------------------------------------------- workspace guard words
// One CTA per guard, one thread per 32-bit word.
__device__ __forceinline__ uint32_t guard_word(int guard, int word) {
  return 0xC5A5D00Du ^ ((uint32_t)guard * 0x9E3779B9u) ^ ((uint32_t)word * 0x85EBCA6Bu);
}

__global__ void canary_fill_kernel(uint8_t* base, const GuardList guards) {
  const int g = blockIdx.x;
  reinterpret_cast<uint32_t*>(base + guards.off[g])[threadIdx.x] = guard_word(g, threadIdx.x);
}

__global__ void canary_check_kernel(const uint8_t* base, const GuardList guards, WorkspaceHeader* hdr) {
  const int g = blockIdx.x;
  const uint32_t v = __ldcg(reinterpret_cast<const uint32_t*>(base + guards.off[g]) + threadIdx.x);
  if (v != guard_word(g, threadIdx.x) && atomicCAS(&hdr->status, TLQ_OK, TLQ_ERR_OVERRUN) == TLQ_OK)
    hdr->where = 100 + g;
}

int launch_canary_fill(void* workspace, const GuardList& guards, cudaStream_t st) {
  if (guards.n <= 0) return TLQ_OK;
  canary_fill_kernel<<<guards.n, (unsigned)(kGuardBytes / 4), 0, st>>>(reinterpret_cast<uint8_t*>(workspace), guards);
  return after_launch();
}

int launch_canary_check(const void* workspace, const GuardList& guards, WorkspaceHeader* hdr, cudaStream_t st) {
  if (guards.n <= 0) return TLQ_OK;
  canary_check_kernel<<<guards.n, (unsigned)(kGuardBytes / 4), 0, st>>>(reinterpret_cast<const uint8_t*>(workspace),
                                                                        guards, hdr);
  return after_launch();
}

}  // namespace tlq
