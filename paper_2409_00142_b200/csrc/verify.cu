// Verification-side helpers for a finished draft tree: the root-to-leaf path table the target
// model's tree attention is usually unpacked with, and the greedy (temperature 0) acceptance
// walk (Section 1: the target verifies the whole tree in one call and accepts a draft token
// when it equals its own choice).  Pure index work on the rows ddd_draft emitted.
#include "ddd_common.cuh"

namespace {

using namespace ddd;

constexpr int kVerifyThreads = 1024;   // one thread per output row (T <= DDD_MAX_TOTAL + 1)

// One block per sequence.
__global__ void __launch_bounds__(kVerifyThreads)
verify_greedy_kernel(const int T, const int max_depth, const int* __restrict__ n_out,
                     const int* __restrict__ token, const int* __restrict__ parent,
                     const int* __restrict__ target_argmax, ddd_verify_output out) {
  __shared__ int s_parent[kVerifyThreads];
  __shared__ int s_token[kVerifyThreads];
  __shared__ int s_has_child[kVerifyThreads];
  __shared__ int s_warp_total[kVerifyThreads / 32];
  __shared__ int s_next;
  __shared__ int s_bad;

  const int b = blockIdx.x, i = threadIdx.x;
  const int warp = i >> 5, lane = i & 31;
  const int L = max_depth + 1;
  int n = n_out[b];
  n = n < 0 ? 0 : (n > T ? T : n);
  const bool row = i < n;

  s_parent[i] = (row && i > 0) ? parent[(size_t)b * T + i] : -1;   // the root has no parent, whatever is stored
  s_token[i] = row ? token[(size_t)b * T + i] : -1;
  s_has_child[i] = 0;
  if (i == 0) s_bad = 0;
  __syncthreads();
  // A well-formed tree has parent[0] = -1 and 0 <= parent[i] < i for every other row.
  if (row && i > 0) {
    const int p = s_parent[i];
    if (p >= 0 && p < i) s_has_child[p] = 1;
    else s_bad = 1;
  }
  __syncthreads();
  const bool bad = s_bad != 0 || n == 0;

  // ---- leaves in ascending row order: block-wide exclusive scan of the leaf flags
  const bool leaf = row && !bad && !s_has_child[i];
  const unsigned ballot = __ballot_sync(kFullMask, leaf);
  if (lane == 0) s_warp_total[warp] = __popc(ballot);
  __syncthreads();
  if (warp == 0) {
    const int t = s_warp_total[lane];
    int incl = t;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int u = __shfl_up_sync(kFullMask, incl, o);
      if (lane >= o) incl += u;
    }
    s_warp_total[lane] = incl - t;
    if (lane == 31) s_next = incl;   // total number of leaves, read below before its reuse
  }
  __syncthreads();
  const int n_leaves = s_next;
  const int slot = s_warp_total[warp] + __popc(ballot & ((1u << lane) - 1u));
  int* paths = out.leaf_paths + (size_t)b * T * L;
  if (leaf) {
    int len = 0;
    for (int r = i; r >= 0 && len <= L; r = s_parent[r]) ++len;   // rows on the path, root included
    int* dst = paths + (size_t)slot * L;
    if (len <= L) {
      int r = i;
      for (int j = len - 1; j >= 0; --j, r = s_parent[r]) dst[j] = r;
      for (int j = len; j < L; ++j) dst[j] = -1;
    } else {   // deeper than max_depth: not a tree this configuration can have produced
      for (int j = 0; j < L; ++j) dst[j] = -1;
      s_bad = 1;
    }
  }
  // unused path rows
  for (int e = n_leaves * L + i; e < T * L; e += kVerifyThreads) paths[e] = -1;
  __syncthreads();

  // ---- greedy walk: from the root, step to the child whose token is the target's choice
  int cur = 0, accepted = 0;
  int* acc_rows = out.accepted_rows + (size_t)b * max_depth;
  const bool walk = !bad && s_bad == 0;
  while (walk && accepted < max_depth) {
    const int want = target_argmax[(size_t)b * T + cur];
    if (i == 0) s_next = kVerifyThreads;
    __syncthreads();
    if (row && i > 0 && s_parent[i] == cur && s_token[i] == want) atomicMin(&s_next, i);
    __syncthreads();
    const int nxt = s_next;
    __syncthreads();
    if (nxt >= kVerifyThreads) break;
    if (i == 0) acc_rows[accepted] = nxt;
    cur = nxt;
    ++accepted;
  }
  for (int j = accepted + i; j < max_depth; j += kVerifyThreads) acc_rows[j] = -1;
  if (i == 0) {
    const bool ok = walk && s_bad == 0;
    out.n_accepted[b] = ok ? accepted : 0;
    out.next_token[b] = ok ? target_argmax[(size_t)b * T + cur] : -1;
    out.n_leaves[b] = ok ? n_leaves : 0;
    if (!ok) atomicExch(out.status, DDD_ERR_INVALID_ARG);
  }
}

__global__ void verify_clear_status_kernel(int* status) { *status = DDD_OK; }

}  // namespace

extern "C" int ddd_verify_greedy(int32_t batch, int32_t t_rows, int32_t max_depth, const int32_t* n_out,
                                 const int32_t* token, const int32_t* parent, const int32_t* target_argmax,
                                 const ddd_verify_output* out, void* cuda_stream) {
  if (!n_out || !token || !parent || !target_argmax || !out) return DDD_ERR_INVALID_ARG;
  if (!out->n_accepted || !out->accepted_rows || !out->next_token || !out->n_leaves || !out->leaf_paths ||
      !out->status)
    return DDD_ERR_INVALID_ARG;
  if (batch < 1 || t_rows < 1 || t_rows > DDD_MAX_TOTAL + 1 || max_depth < 1 || max_depth > DDD_MAX_DEPTH)
    return DDD_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  verify_clear_status_kernel<<<1, 1, 0, st>>>(out->status);
  if (cudaGetLastError() != cudaSuccess) return DDD_ERR_CUDA;
  verify_greedy_kernel<<<batch, kVerifyThreads, 0, st>>>(t_rows, max_depth, n_out, token, parent, target_argmax,
                                                         *out);
  if (cudaGetLastError() != cudaSuccess) return DDD_ERR_CUDA;
  return DDD_OK;
}
