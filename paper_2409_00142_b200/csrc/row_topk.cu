// Per-row top-k and log-sum-exp over logits held in global memory (Section 1: "the draft model
// produces the top w most probable tokens"; Algorithm 1, "Run draft model on beam").  Used for wide
// beams (33..128), where the LM-head kernel writes its scaled logits out instead of keeping a
// sorted list per row and tile (lm_head_tc.cu, DENSE).  One block of 1024 threads per beam row:
//   1. one pass over the row: every thread keeps the largest of its (strided) logits and the
//      online max / sum exp(z - max) of all of them; the block's (max, sum exp) is the row's;
//   2. a floor under the row's k-th best logit from the 1024 thread maxima: the smallest, over the
//      32 warps, of the warp's j-th largest (j = k / 32 rounded up) has k logits of different threads
//      at or above it; a few warp maxima and ballots, where a histogram over all V logits piles them
//      into the few bins their exponents share (measured: 42 us per row that way, nearly all of it
//      atomic conflicts) and a radix select over the 1024 maxima alone still cost 10 us;
//   3. a second pass (the row is in L1 by now) gathers the logits at or above the floor, a few hundred,
//      and each is placed by counting the better ones: the row's list comes out sorted without a sort.
// More than 1024 logits at or above the floor (many equal ones) take the slow exact way: a radix
// select over the whole row, then the ties with the lowest tokens.  The row's record - k (logit,
// token) keys in descending order, then (max, sum exp) - goes where the select kernel expects the
// single partial of a row.  A planted column arrives as -inf and takes no part (the select kernel
// puts it back).
#include "ddd_common.cuh"
#include "lm_head_tc.cuh"
#include "tree_device.cuh"

namespace ddd {

namespace {

constexpr int kTopkThreads = 1024;
constexpr int kTopkBins = 2048;
constexpr int kTopkCand = 1024;      // candidates the counting step takes

struct RadixResult {
  uint32_t key;    // the need-th largest key
  int rest;        // how many of the entries equal to it are among the `need` largest
  int ties;        // how many entries equal it
};

// The need-th largest of n keys (key_at(i), 0 = no entry), by three histogram levels of 11 + 11 + 10
// bits.  Called by the whole block; hist [kTopkBins] and ctl [4] are shared scratch.  need >= 1 and
// at least `need` entries exist.
template <typename KeyAt>
__device__ RadixResult radix_select(const KeyAt key_at, const int n, const int need, int* hist, int* ctl) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint32_t known = 0u;
  if (tid == 0) { ctl[0] = 0; ctl[1] = need; ctl[2] = 0; }
  for (int level = 0; level < 3; ++level) {
    const int shift = level == 0 ? 21 : (level == 1 ? 10 : 0);
    const uint32_t mask = level == 2 ? 0x3FFu : 0x7FFu;
    for (int i = tid; i < kTopkBins; i += kTopkThreads) hist[i] = 0;
    __syncthreads();
    const uint32_t prefix = (uint32_t)ctl[0];
    for (int i = tid; i < n; i += kTopkThreads) {
      const uint32_t key = key_at(i);
      if (key != 0u && (key & known) == prefix) atomicAdd(&hist[(key >> shift) & mask], 1);
    }
    __syncthreads();
    if (warp == 0) {
      // lane l owns bins 64 l .. 64 l + 63; find the bin of the want-th largest key
      const int want = ctl[1];
      const int per = kTopkBins / 32;
      int mine = 0;
      for (int i = 0; i < per; ++i) mine += hist[per * lane + i];
      int above = mine;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_down_sync(kFullMask, above, o);
        if (lane + o < 32) above += t;
      }
      above -= mine;                                         // keys in higher lanes' bins
      if (above < want && want <= above + mine) {            // exactly one lane
        int rem = want - above, bin = per - 1;
        for (; bin > 0; --bin) {
          const int c = hist[per * lane + bin];
          if (c >= rem) break;
          rem -= c;
        }
        ctl[0] = (int)(prefix | ((uint32_t)(per * lane + bin) << shift));
        ctl[1] = rem;
        ctl[2] = hist[per * lane + bin];
      }
    }
    known |= mask << shift;
    __syncthreads();
  }
  RadixResult res;
  res.key = (uint32_t)ctl[0];
  res.rest = ctl[1];
  res.ties = ctl[2];
  __syncthreads();
  return res;
}

__global__ void __launch_bounds__(kTopkThreads) row_topk_kernel(const Params p, const int d,
                                                                const float* __restrict__ logits, const size_t ldl,
                                                                unsigned long long* __restrict__ rec_keys,
                                                                float2* __restrict__ rec_ms) {
  const int r = blockIdx.x;
  if (*p.n_active == 0 || !row_live(p, r, d, 0)) return;     // the same for the whole block
  const float* z = logits + (size_t)r * ldl;
  const int V = p.Vl, k = p.k;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  __shared__ int hist[kTopkBins];
  __shared__ uint32_t tmax[kTopkThreads];
  __shared__ unsigned long long cand[kTopkCand];
  __shared__ float red_m[32], red_s[32];
  __shared__ int red_n[32];
  __shared__ uint32_t warp_floor[32];
  __shared__ int warp_tot[32];
  __shared__ int ctl[4];
  __shared__ int s_need, s_count;

  // Both passes over the row fetch four 16-byte pieces per thread and step before they look at any
  // of them: with one scalar load in flight per thread a pass is bound by the latency of L2, not by
  // its bandwidth (measured: 33 us per row against 19, before the floor got cheaper).
  const int V4 = V >> 2;
  const float4* z4 = reinterpret_cast<const float4*>(z);          // rows start on 128-byte boundaries
  auto for_each = [&](auto&& body) {                               // body(values[16], tokens of the four pieces)
    for (int i0 = tid; i0 < V4; i0 += 4 * kTopkThreads) {
      float4 q[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + u * kTopkThreads;
        q[u] = i < V4 ? z4[i] : make_float4(neg_inf(), neg_inf(), neg_inf(), neg_inf());
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const float x[4] = {q[u].x, q[u].y, q[u].z, q[u].w};
        body(x, 4 * (i0 + u * kTopkThreads));
      }
    }
    if (tid < V - 4 * V4) {                                        // up to three logits behind the last whole piece
      const float x[4] = {z[4 * V4 + tid], neg_inf(), neg_inf(), neg_inf()};
      body(x, 4 * V4 + tid);
    }
  };
  // ---- 1. one pass: thread maximum, online max / sum exp, number of entries
  float m = neg_inf(), s = 0.f;
  int n_valid = 0;
  for_each([&](const float (&x)[4], int) {
    const float bm = fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3]));
    if (bm == neg_inf()) return;
    if (bm > m) { s *= __expf(m - bm); m = bm; }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      n_valid += x[j] != neg_inf() ? 1 : 0;
      s += __expf(x[j] - m);                                       // exp(-inf) = 0
    }
  });
  tmax[tid] = n_valid ? float_to_ordered(m) : 0u;
  {
    const float wm = ordered_to_float(__reduce_max_sync(kFullMask, float_to_ordered(m)));
    const float ws = warp_sum(s > 0.f ? s * __expf(m - wm) : 0.f);
    const int wn = __reduce_add_sync(kFullMask, n_valid);
    if (lane == 0) { red_m[warp] = wm; red_s[warp] = ws; red_n[warp] = wn; }
  }
  if (tid == 0) s_count = 0;
  __syncthreads();
  if (warp == 0) {                 // 32 warps' results, one per lane
    const float M = ordered_to_float(__reduce_max_sync(kFullMask, float_to_ordered(red_m[lane])));
    const float S = warp_sum(red_s[lane] > 0.f ? red_s[lane] * __expf(red_m[lane] - M) : 0.f);
    const int n = __reduce_add_sync(kFullMask, red_n[lane]);
    if (lane == 0) {
      rec_ms[r] = make_float2(M, S);
      s_need = n < k ? n : k;
    }
  }
  __syncthreads();
  const int need = s_need;                 // entries the list will hold
  if (need == 0) {
    if (tid < k) rec_keys[(size_t)r * k + tid] = 0ull;
    return;
  }
  // ---- 2. the floor: every warp's j-th largest thread maximum, j = need / 32 rounded up, has j logits
  // of that warp at or above it, so the smallest of the 32 has at least need (everything counts
  // where a warp holds fewer than j entries)
  {
    const int j = (need + 31) / 32;
    uint32_t cur = tmax[tid], jth = 0u;
    for (int t = 0; t < j; ++t) {
      jth = __reduce_max_sync(kFullMask, cur);
      const unsigned who = __ballot_sync(kFullMask, cur == jth);
      if (lane == __ffs(who) - 1) cur = 0u;
    }
    if (lane == 0) warp_floor[warp] = jth;
  }
  __syncthreads();
  uint32_t floor_key = warp_floor[0];
  for (int w = 1; w < kTopkThreads / 32; ++w) floor_key = min(floor_key, warp_floor[w]);
  if (floor_key == 0u) floor_key = 1u;
  // ---- 3. the logits at or above it
  const float floor_z = floor_key == 1u ? neg_inf() : ordered_to_float(floor_key);
  for_each([&](const float (&x)[4], int tok0) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (x[j] != neg_inf() && x[j] >= floor_z) {
        const int at = atomicAdd(&s_count, 1);
        if (at < kTopkCand) cand[at] = make_key(x[j], (uint32_t)(tok0 + j + p.v0));
      }
    }
  });
  __syncthreads();
  const int count = s_count;
  if (count <= kTopkCand) {
    // place of a candidate = number of better ones (keys are distinct: score, then lower token first)
    for (int e = tid; e < count; e += kTopkThreads) {
      const unsigned long long mine = cand[e];
      int place = 0;
      for (int j = 0; j < count; ++j) place += cand[j] > mine ? 1 : 0;
      if (place < k) rec_keys[(size_t)r * k + place] = mine;
    }
    if (tid >= need && tid < k) rec_keys[(size_t)r * k + tid] = 0ull;
    return;
  }
  // ---- the slow exact way
  __syncthreads();
  if (tid == 0) s_count = 0;
  const RadixResult kth = radix_select([&](int i) { const float x = z[i]; return x == neg_inf() ? 0u : float_to_ordered(x); },
                                       V, need, hist, ctl);
  const bool all_ties = kth.ties == kth.rest;
  for (int v = tid; v < V; v += kTopkThreads) {
    const float x = z[v];
    if (x == neg_inf()) continue;
    const uint32_t key = float_to_ordered(x);
    if (key > kth.key || (all_ties && key == kth.key)) cand[atomicAdd(&s_count, 1)] = make_key(x, (uint32_t)(v + p.v0));
  }
  if (!all_ties) {
    // only the lowest tokens among the ties: each thread counts the ties of a contiguous run of
    // tokens, a prefix sum gives the rank of its first one
    const int chunk = (V + kTopkThreads - 1) / kTopkThreads;
    const int lo = min(V, tid * chunk), hi = min(V, lo + chunk);
    int n_eq = 0;
    for (int v = lo; v < hi; ++v) n_eq += (z[v] != neg_inf() && float_to_ordered(z[v]) == kth.key) ? 1 : 0;
    int total;
    int before = block_exclusive_scan<kTopkThreads, BlockSync>(n_eq, warp_tot, &total, tid);
    for (int v = lo; v < hi && before < kth.rest; ++v) {
      const float x = z[v];
      if (x != neg_inf() && float_to_ordered(x) == kth.key) {
        cand[atomicAdd(&s_count, 1)] = make_key(x, (uint32_t)(v + p.v0));
        ++before;
      }
    }
  }
  __syncthreads();
  if (warp == 0) {                           // at most need <= 128 keys: sorted by one warp
    unsigned long long list[4];
    wide_load(list, cand, s_count);
    wide_sort(list);
    wide_store(list, rec_keys + (size_t)r * k, k);
  }
}

}  // namespace

cudaError_t launch_row_topk(const Params& p, int d, const float* logits, size_t ldl, void* record, cudaStream_t st) {
  unsigned long long* keys = static_cast<unsigned long long*>(record);
  float2* ms = reinterpret_cast<float2*>(static_cast<unsigned char*>(record) + (size_t)p.R * p.k * sizeof(unsigned long long));
  row_topk_kernel<<<p.R, kTopkThreads, 0, st>>>(p, d, logits, ldl, keys, ms);
  return cudaGetLastError();
}

}  // namespace ddd
