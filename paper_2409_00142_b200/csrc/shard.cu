// Vocabulary-parallel LM head: the pieces one rank adds around the kernels of a pass when it owns
// only a slice [v0, v0 + Vl) of the vocabulary.  After the LM-head kernel has left one partial per
// thread block, shard_reduce_kernel folds them into ONE record per beam row - the slice's
// (max, sum-exp) and its k best (logit, token) keys - and stores that record into slot `slot` of
// every destination buffer it is given (the rank's own and, over NVLink, its peers'), then raises
// a flag word beside each.  A record set [slots][R][k] keys + [slots][R] (max, sum-exp) has exactly
// the layout the select kernel merges, so the pass ends with the ordinary select / gate / draft
// step on every rank, reading `slots` partials instead of one per thread block.
#include "ddd_common.cuh"
#include "tree_device.cuh"

namespace ddd {

namespace {

constexpr unsigned long long kFlagWaitNs = 2000000000ull;

struct ShardDst {
  unsigned long long* keys[DDD_MAX_SHARDS];   // [slots][R][k] of each destination
  float2* ms[DDD_MAX_SHARDS];                 // [slots][R]
  int* flags[DDD_MAX_SHARDS];                 // [slots] or nullptr
  int n;
};

__device__ __forceinline__ unsigned long long shard_timer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

// One block per beam row.  Every warp folds a share of the thread blocks' lists into a wide list,
// the 16 results are merged pairwise; warp 0 adds up (max, sum-exp) in a fixed order.  Rows that
// take no part in this pass are skipped (nobody reads their records).  The last block to finish
// raises the flags, also when drafting has already stopped, so that a peer never waits in vain.
__global__ void __launch_bounds__(kWideThreads) shard_reduce_kernel(const Params p, const int d, const int slot,
                                                                    const ShardDst dst, const int flag_value,
                                                                    int* done_counter) {
  __shared__ unsigned long long buf[kWideWarps * kWideK];
  const int r = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int k = p.k, nc = p.lm_ctas, R = p.R;
  const bool live = *p.n_active != 0 && row_live(p, r, d, 0);
  if (live) {
    unsigned long long acc[4] = {0ull, 0ull, 0ull, 0ull};
    for (int c = warp; c < nc; c += kWideWarps) {
      unsigned long long t[4];
      wide_load(t, p.part_key + ((size_t)c * R + r) * k, k);
      wide_merge(acc, t);
    }
    block_merge_lists(acc, buf);
    if (warp == 0) {
      float M = neg_inf();
      for (int c = lane; c < nc; c += 32) M = fmaxf(M, p.part_ms[(size_t)c * R + r].x);
      M = ordered_to_float(__reduce_max_sync(kFullMask, float_to_ordered(M)));
      float S = 0.f;
      for (int c = lane; c < nc; c += 32) {
        const float2 ms = p.part_ms[(size_t)c * R + r];
        if (ms.y > 0.f) S += ms.y * expf(ms.x - M);
      }
      S = warp_sum(S);
      for (int i = 0; i < dst.n; ++i) {
        wide_store(acc, dst.keys[i] + ((size_t)slot * R + r) * k, k);
        if (lane == 0) dst.ms[i][(size_t)slot * R + r] = make_float2(M, S);
      }
    }
  }
  // last block out: every record of this rank is on its way, raise the flags
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence_system();
    if (atomicAdd(done_counter, 1) == (int)gridDim.x - 1) {
      *done_counter = 0;
      __threadfence_system();
      for (int i = 0; i < dst.n; ++i)
        if (dst.flags[i]) {
          asm volatile("st.release.sys.global.b32 [%0], %1;" ::"l"(dst.flags[i] + slot), "r"(flag_value) : "memory");
        }
    }
  }
}

// Waits (bounded) until every slot's flag shows this pass; a wait that runs out is reported
// through the device status and the pass goes on with whatever the records hold.
__global__ void shard_wait_kernel(const int* flags, const int slots, const int flag_value, int* dev_status) {
  const int g = threadIdx.x;
  if (g >= slots) return;
  const unsigned long long t0 = shard_timer();
  for (unsigned it = 0;; ++it) {
    int v;
    asm volatile("ld.acquire.sys.global.b32 %0, [%1];" : "=r"(v) : "l"(flags + g) : "memory");
    if (v == flag_value) return;
    if ((it & 63u) == 63u && shard_timer() - t0 > kFlagWaitNs) {
      atomicCAS(dev_status, DDD_OK, DDD_ERR_TIMEOUT);
      return;
    }
  }
}

}  // namespace

cudaError_t launch_shard_reduce(const Params& p, int d, int slot, int slots, void* const* records,
                                int32_t* const* flags, int n_dst, int flag_value, int* done_counter, cudaStream_t st) {
  ShardDst dst = {};
  dst.n = n_dst;
  for (int i = 0; i < n_dst; ++i) {
    unsigned char* base = static_cast<unsigned char*>(records[i]);
    dst.keys[i] = reinterpret_cast<unsigned long long*>(base);
    dst.ms[i] = reinterpret_cast<float2*>(base + (size_t)slots * p.R * p.k * sizeof(unsigned long long));
    dst.flags[i] = flags ? flags[i] : nullptr;
  }
  shard_reduce_kernel<<<p.R, kWideThreads, 0, st>>>(p, d, slot, dst, flag_value, done_counter);
  return cudaGetLastError();
}

cudaError_t launch_shard_wait(const int* flags, int slots, int flag_value, int* dev_status, cudaStream_t st) {
  shard_wait_kernel<<<1, 32, 0, st>>>(flags, slots, flag_value, dev_status);
  return cudaGetLastError();
}

}  // namespace ddd
