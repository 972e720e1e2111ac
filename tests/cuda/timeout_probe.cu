// Test-only kernels (their own small library, not part of libddd.so): the bounded waits of the
// tensor-core kernels made to run out on purpose, in the one way that touches nothing else - a
// barrier nobody arrives at and a counter nobody raises, no copies and no tensor memory in
// flight.  Each wait must give up after its limit, record DDD_ERR_TIMEOUT and let the kernel end
// normally, so that the context stays usable.
#include "tc_ptx.cuh"

using namespace ddd;
using namespace ddd::tc;

__global__ void mbarrier_wait_runs_out(int* status, int* result, unsigned long long limit_ns) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  // nobody ever arrives: phase 0 never completes
  const unsigned long long t0 = global_timer();
  const bool ok = mbar_wait(smem_u32(&bar), 0u, &abort_flag, status, true, limit_ns);
  const unsigned long long t1 = global_timer();
  if (threadIdx.x == 0) {
    result[0] = ok ? 1 : 0;
    result[1] = abort_flag;
    result[2] = (int)((t1 - t0) / 1000ull);       // microseconds spent waiting
  }
}

__global__ void grid_wait_runs_out(int* status, int* result, int* counter, int* abort_word, unsigned long long limit_ns) {
  // block 0 waits for two arrivals at a counter that only ever receives one; the other blocks watch the abort word
  if (threadIdx.x != 0) return;
  bool ok;
  if (blockIdx.x == 0) {
    atomicAdd(counter, 1);
    ok = grid_wait(counter, 2, abort_word, status, limit_ns);
  } else {
    ok = grid_wait(counter, 1 << 30, abort_word, status, 50ull * limit_ns);    // ends through the abort word
  }
  result[blockIdx.x] = ok ? 1 : 0;
}

extern "C" int probe_mbarrier_timeout(int* status, int* result, double limit_ms, void* stream) {
  mbarrier_wait_runs_out<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(status, result,
                                                                           (unsigned long long)(limit_ms * 1e6));
  return cudaGetLastError() == cudaSuccess ? 0 : -4;
}

extern "C" int probe_grid_timeout(int* status, int* result, int* counter, int* abort_word, int blocks, double limit_ms,
                                  void* stream) {
  grid_wait_runs_out<<<blocks, 32, 0, static_cast<cudaStream_t>(stream)>>>(status, result, counter, abort_word,
                                                                           (unsigned long long)(limit_ms * 1e6));
  return cudaGetLastError() == cudaSuccess ? 0 : -4;
}
