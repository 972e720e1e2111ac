// Kernels around the LM head: draft initialisation and the per-pass select / gate / draft step,
// which for a sequence that stops at that pass ends with the rerank and the bit-packed tree
// mask (tree_device.cuh).  One cluster of eight thread blocks per sequence.
#include <cooperative_groups.h>

#include "ddd_common.cuh"
#include "tree_device.cuh"

namespace cg = cooperative_groups;

namespace ddd {

namespace {

// Threads per block of the select kernel: the serial section of a narrow beam is a chain of
// round trips, which smaller blocks get through sooner (-2.4 us per draft at width 10, stop
// depth 2); wide beams have the work for 1024 threads (width 32: -1.2 us per pass).
constexpr int kSelThreadsNarrow = 512, kSelThreadsWide = 1024;
constexpr int kSelWideFromK = 17;
constexpr int kSelCluster = 8;      // thread blocks (one cluster) working on one sequence

// ---------------------------------------------------------------------------- init
// Resets the per-draft state and loads the root: tree node 0, beam slot 0 and hidden row b*k.
template <typename T>
__global__ void init_kernel(const Params p, const T* __restrict__ root_hidden,
                            const int* __restrict__ root_token, const int* __restrict__ root_pos) {
  griddep_launch_dependents();   // the first LM-head pass may start streaming W while this runs
  const int b = blockIdx.x;
  T* dst = static_cast<T*>(p.hbuf[0]) + (size_t)b * p.k * p.Hd;
  const T* src = root_hidden + (size_t)b * p.Hd;
  for (int j = threadIdx.x; j < p.Hd; j += blockDim.x) dst[j] = src[j];
  if (threadIdx.x == 0) {
    const int tok = root_token[b];
    p.tree_token[(size_t)b * p.Nn] = tok;
    p.tree_parent[(size_t)b * p.Nn] = -1;
    p.tree_cum[(size_t)b * p.Nn] = 0.f;
    p.beam_node[b * p.k] = 0;
    p.beam_tok[b * p.k] = tok;
    p.beam_cum[b * p.k] = 0.f;
    const bool tok_ok = tok >= 0 && tok < p.V;
    p.row_plant[b * p.k] = (p.plant_next && tok_ok) ? p.plant_next[tok] : -1;
    p.active[b] = 1;
    p.stop_depth[b] = 0;
    p.root_pos[b] = root_pos[b];
    if (b == 0) {
      *p.n_active = p.B;
      *p.dev_status = DDD_OK;
    }
  }
}

// ---------------------------------------------------------------------------- select / gate / step
// Same result when the lists do not fit in shared memory: pick the k blocks with the best
// first keys, then walk their sorted lists in a k-way merge straight from global memory
// (lane j owns one list).
__device__ __forceinline__ unsigned long long merge_row_kway(const Params& p, int r, int k, int nc,
                                                             const unsigned long long* first_s) {
  const int lane = threadIdx.x & 31;
  unsigned long long prev = ~0ull, cur = 0ull, nxt = 0ull;
  int my_cta = -1;
  for (int j = 0; j < k; ++j) {
    unsigned long long best = 0ull;
    int best_c = -1;
    for (int c = lane; c < nc; c += 32) {
      const unsigned long long key = first_s[c];
      if (key < prev && key > best) { best = key; best_c = c; }
    }
    const unsigned long long wk = warp_max_key(best);
    if (wk == 0ull) break;
    const unsigned owner = __ballot_sync(kFullMask, best == wk);
    const int win_c = __shfl_sync(kFullMask, best_c, __ffs(owner) - 1);
    if (lane == j) { cur = wk; my_cta = win_c; }
    prev = wk;
  }
  const unsigned long long* my_list = my_cta >= 0 ? p.part_key + ((size_t)my_cta * p.R + r) * k : nullptr;
  int pos = 1;
  if (my_list && pos < k) nxt = my_list[pos];
  unsigned long long res = 0ull;
  for (int j = 0; j < k; ++j) {
    const unsigned long long wk = warp_max_key(cur);
    if (wk == 0ull) break;
    if (lane == j) res = wk;
    if (cur == wk) {
      cur = nxt;
      ++pos;
      nxt = (my_list && pos < k) ? my_list[pos] : 0ull;
    }
  }
  return res;
}

// Synthetic draft step for the k new beam rows of one sequence, by all blocks of the cluster:
//   h_child = round( u / sqrt(mean(u^2) + eps) ),  u = h_parent + E[token]
// The rounding to the storage type is a quantisation decision, so everything before it is done
// in fp64 and the result is rounded once, directly from fp64: an fp32 evaluation would flip
// about one element in 10^5 to the neighbouring bf16 value, and one such flip moves a logit by
// up to a few 1e-3.  Work is cut into 16-byte chunks dealt round-robin to the cluster's
// threads; a warp's 32 chunks lie in one row (the caller checks that a row has a multiple of
// 32 chunks).  Every warp sends its partial sum of squares to all blocks through distributed
// shared memory, and each block adds a row's partials in the same fixed order.
// kBatch: chunks a thread has in flight at once (two loads each).  A narrow beam has one or two
// chunks per thread in all; with a wide one (100 rows: 12.5 chunks per thread) the step is bound by the
// latency of those loads, so more of them go out together (measured at width 100: 25 us with 2, see below).
template <typename T, int kBatch>
__device__ void draft_step_cluster(const Params& p, int b, int d, const int* sel_flat, const int* sel_tok,
                                   double* row_part /* [k][slots] */, double* row_inv /* [k] */) {
  cg::cluster_group cluster = cg::this_cluster();
  constexpr int N = Chunk<T>::N;
  const int k = p.k, lane = threadIdx.x & 31;
  const int cpr = p.Hd / N;            // chunks per row
  const int slots = cpr / 32;          // warp-sized groups of chunks per row
  const int total = k * cpr;
  const int first = (int)cluster.block_rank() * (int)blockDim.x + (int)threadIdx.x;
  const int stride = kSelCluster * (int)blockDim.x;
  const uint4* Hsrc = reinterpret_cast<const uint4*>(p.hbuf[(d - 1) & 1]);
  const uint4* Esrc = reinterpret_cast<const uint4*>(p.E);
  uint4* Hdst = reinterpret_cast<uint4*>(p.hbuf[d & 1]);
  auto locate = [&](int q, size_t& hs, size_t& es, size_t& hd, int& row) {
    row = q / cpr;
    const int col = q - row * cpr;
    const int tok = sel_tok[row];
    hs = (size_t)(b * k + sel_flat[row] / k) * cpr + col;
    es = (size_t)(tok >= 0 && tok < p.V ? tok : 0) * cpr + col;
    hd = (size_t)(b * k + row) * cpr + col;
  };
  // pass 1: sum of squares per row.  The chunks of the first round (usually all there are)
  // stay in registers for pass 2.
  uint4 hv0[kBatch], ev0[kBatch];
  for (int q0 = first; q0 - lane < total; q0 += kBatch * stride) {
    uint4 hv[kBatch], ev[kBatch];
#pragma unroll
    for (int i = 0; i < kBatch; ++i) {
      const int q = q0 + i * stride;
      if (q < total) {
        size_t hs, es, hd;
        int row;
        locate(q, hs, es, hd, row);
        hv[i] = Hsrc[hs];
        ev[i] = Esrc[es];
        if (q0 == first) { hv0[i] = hv[i]; ev0[i] = ev[i]; }
      }
    }
#pragma unroll
    for (int i = 0; i < kBatch; ++i) {
      const int q = q0 + i * stride;
      if (q - lane >= total) continue;          // whole warp past the end (total is a multiple of 32)
      double u[N];
      Chunk<T>::sum(hv[i], ev[i], u);
      double ss = 0.0;
#pragma unroll
      for (int e = 0; e < N; ++e) ss = fma(u[e], u[e], ss);
      ss = warp_sum_f64(ss);
      const int row = q / cpr;
      const int slot = row * slots + (q - row * cpr) / 32;
      if (lane < kSelCluster) cluster.map_shared_rank(row_part, lane)[slot] = ss;
    }
  }
  cluster.sync();
  for (int row = (int)threadIdx.x; row < k; row += (int)blockDim.x) {
    double ss = 0.0;
    for (int j = 0; j < slots; ++j) ss += row_part[row * slots + j];
    row_inv[row] = 1.0 / sqrt(ss / (double)p.Hd + (double)p.eps);
  }
  __syncthreads();
  // pass 2: scale, round once, store (later rounds re-read their inputs from the caches)
  for (int q0 = first; q0 - lane < total; q0 += kBatch * stride) {
    uint4 hv[kBatch], ev[kBatch];
    size_t dst[kBatch];
    int rows[kBatch];
#pragma unroll
    for (int i = 0; i < kBatch; ++i) {
      const int q = q0 + i * stride;
      rows[i] = -1;
      if (q < total) {
        size_t hs, es;
        locate(q, hs, es, dst[i], rows[i]);
        if (q0 == first) { hv[i] = hv0[i]; ev[i] = ev0[i]; }
        else { hv[i] = Hsrc[hs]; ev[i] = Esrc[es]; }
      }
    }
#pragma unroll
    for (int i = 0; i < kBatch; ++i) {
      if (rows[i] < 0) continue;
      double u[N];
      Chunk<T>::sum(hv[i], ev[i], u);
      const double inv = row_inv[rows[i]];
#pragma unroll
      for (int e = 0; e < N; ++e) u[e] *= inv;
      Hdst[dst[i]] = Chunk<T>::round(u);
    }
  }
}

// The same step with one warp per row (run by one block), for hidden sizes whose rows are not
// a whole number of 32-chunk groups.
template <typename T>
__device__ void draft_step_warp(const Params& p, int b, int d, const int* sel_flat, const int* sel_tok) {
  constexpr int N = Chunk<T>::N;
  const int k = p.k, lane = threadIdx.x & 31;
  const int cpr = p.Hd / N;
  for (int row = (int)(threadIdx.x >> 5); row < k; row += (int)(blockDim.x >> 5)) {
    const int tok = sel_tok[row];
    const uint4* hp = reinterpret_cast<const uint4*>(p.hbuf[(d - 1) & 1]) + (size_t)(b * k + sel_flat[row] / k) * cpr;
    const uint4* e = reinterpret_cast<const uint4*>(p.E) + (size_t)(tok >= 0 && tok < p.V ? tok : 0) * cpr;
    uint4* out = reinterpret_cast<uint4*>(p.hbuf[d & 1]) + (size_t)(b * k + row) * cpr;
    double ss = 0.0;
    for (int c = lane; c < cpr; c += 32) {
      double u[N];
      Chunk<T>::sum(hp[c], e[c], u);
#pragma unroll
      for (int i = 0; i < N; ++i) ss = fma(u[i], u[i], ss);
    }
    ss = warp_sum_f64(ss);
    const double inv = 1.0 / sqrt(ss / (double)p.Hd + (double)p.eps);
    for (int c = lane; c < cpr; c += 32) {
      double u[N];
      Chunk<T>::sum(hp[c], e[c], u);
#pragma unroll
      for (int i = 0; i < N; ++i) u[i] *= inv;
      out[c] = Chunk<T>::round(u);
    }
  }
}

// Called by every block of the cluster (the choice below is the same in all of them).
template <typename T, int kBatch = 2>
__device__ void draft_step(const Params& p, int b, int d, const int* sel_flat, const int* sel_tok, double* row_part,
                           double* row_inv) {
  const int cpr = p.Hd / Chunk<T>::N;
  if (cpr % 32 == 0 && cpr / 32 <= 64)
    draft_step_cluster<T, kBatch>(p, b, d, sel_flat, sel_tok, row_part, row_inv);
  else if (cg::this_cluster().block_rank() == 0)
    draft_step_warp<T>(p, b, d, sel_flat, sel_tok);
}

// 8-byte asynchronous copy global -> shared (both 8-byte aligned); completes at cp.async.wait_group.
__device__ __forceinline__ void async_copy_8(void* dst_shared, const void* src_global) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8;"
               ::"r"((uint32_t)__cvta_generic_to_shared(dst_shared)), "l"(src_global) : "memory");
}

// One cluster of kSelCluster blocks per sequence.  Beam row pr is merged by block pr % 8
// (warp pr / 8), which first copies that row's partial lists into its shared memory; the
// candidates go to block 0 through distributed shared memory, block 0 picks the new beam and
// takes the stop decision, and all blocks share the draft step.
// Dynamic shared memory per block, for its rows_max = ceil(k / 8) rows: the blocks' key lists
// [rows_max][nc][k] (or only their first keys [rows_max][nc] when the lists do not fit),
// their (max, sum-exp) [rows_max][nc], and the rows' planted columns [rows_max].
template <int kSelThreads>
__global__ void __launch_bounds__(kSelThreads) select_gate_step_kernel(const Params p, const DraftIO io,
                                                                       const int d, const int lists_in_smem,
                                                                       const cudaGraphConditionalHandle cond,
                                                                       const int set_cond) {
  // Wait for the LM-head pass, then let the next pass start: it streams W into shared memory
  // while this kernel works and reads the new hidden rows only after this kernel has finished.
  // (That burst slows this kernel's own few loads by 2-3 us each; releasing the next pass
  // later was measured and lost more than it won.)
  griddep_wait();
  griddep_launch_dependents();
  cg::cluster_group cluster = cg::this_cluster();
  const int crank = (int)cluster.block_rank();
  const int b = blockIdx.x / kSelCluster;
  if (p.active[b] == 0) return;                               // same decision in the whole cluster
  // First half of a split cluster barrier: a block may only write into another block's shared
  // memory once that block is known to have started.  Everyone arrives here, at once; the wait
  // sits just before the first remote store (phase 1), by which time all arrivals are long in,
  // so it costs next to nothing.
  asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int k = p.k, nc = p.lm_ctas, R = p.R;
  const int P = (d == 1) ? 1 : k;                            // beam rows of this sequence in pass d
  const int base = (d == 1) ? 1 : 1 + k + (d - 2) * k * k;   // node id of candidate (0, 0)
  const int rows_max = (k + kSelCluster - 1) / kSelCluster;
  const int n_mine = P > crank ? (P - crank + kSelCluster - 1) / kSelCluster : 0;   // rows of this block
  const int kl = lists_in_smem ? k : 1;                       // keys kept per (row, LM-head block)

  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned long long* keys_s = reinterpret_cast<unsigned long long*>(smem_raw);              // [rows_max][nc][kl]
  float2* ms_s = reinterpret_cast<float2*>(keys_s + (size_t)rows_max * nc * kl);              // [rows_max][nc]
  int* plant_s = reinterpret_cast<int*>(ms_s + (size_t)rows_max * nc);                        // [rows_max]
  // candidate (p, c) of this pass at [p * k + c]: score bits in the upper word, token (-1 = none)
  // in the lower; one 8-byte store per block of the cluster carries it there
  __shared__ unsigned long long cand_rec[kNarrowK * kNarrowK];
  auto cand_key_of = [&](int idx) -> unsigned long long {     // selection key: score, ties to the lower index
    const unsigned long long rec = cand_rec[idx];
    return (int)(uint32_t)rec >= 0 ? make_key(__uint_as_float((uint32_t)(rec >> 32)), (uint32_t)idx) : 0ull;
  };
  __shared__ int sel_flat[kNarrowK];
  __shared__ int sel_tok[kNarrowK];
  __shared__ double row_part[kNarrowK * 64];
  __shared__ double row_inv[kNarrowK];
  __shared__ int s_stop;
  __shared__ bool s_last;
  __shared__ float beam_cum_s[kNarrowK / kSelCluster];
  __shared__ int beam_node_s[kNarrowK / kSelCluster];

  // ---- phase 0: the block fetches everything phase 1 needs for its rows in one round trip.
  // The copies go from global to shared memory asynchronously (a warp copies one LM-head block's
  // list per step: lane q takes the q-th key), so all of them are in flight together however
  // many rows the block owns: a round trip to memory costs this lone block a microsecond or
  // two, and loads through registers would have to go in several batches.
  {
    constexpr int kW = kSelThreads / 32;
    for (int j = 0; j < n_mine; ++j) {
      const int r = b * k + crank + kSelCluster * j;
      for (int c = warp; c < nc; c += kW) {
        const size_t slot = (size_t)c * R + r;
        if (lane < kl) async_copy_8(&keys_s[((size_t)j * nc + c) * kl + lane], &p.part_key[slot * k + lane]);
        if (lane == 31) async_copy_8(&ms_s[(size_t)j * nc + c], &p.part_ms[slot]);
      }
    }
    // the few scalars phase 1 needs ride along
    if (warp == 0 && lane < n_mine) {
      const int r = b * k + crank + kSelCluster * lane;
      plant_s[lane] = p.row_plant[r];
      beam_cum_s[lane] = p.beam_cum[r];
      beam_node_s[lane] = p.beam_node[r];
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
  }
  __syncthreads();

  // ---- phase 1: per beam row of this block, warp j merges the top-k lists while warp j + 4
  //      adds up the log-sum-exp of the same row
  __shared__ float lse_s[kNarrowK / kSelCluster];
  __shared__ unsigned long long plant_key_s[kNarrowK / kSelCluster];
  constexpr int kRowsPerBlock = kNarrowK / kSelCluster;
  unsigned long long res = 0ull;
  if (warp < n_mine) {
    const int r = b * k + crank + kSelCluster * warp;
    const unsigned long long* my_keys = keys_s + (size_t)warp * nc * kl;
    if (!lists_in_smem) res = merge_row_kway(p, r, k, nc, my_keys);
    else if (nc <= 160) res = merge_row_heads<5>(k, nc, my_keys);
    else res = merge_row_heads<10>(k, nc, my_keys);      // the host keeps nc <= 320 on this path
  } else if (warp >= kRowsPerBlock && warp < kRowsPerBlock + n_mine) {
    const int j = warp - kRowsPerBlock;
    const float2* my_ms = ms_s + (size_t)j * nc;
    // log-sum-exp over all blocks (fixed lane-strided order, then a butterfly: deterministic)
    float M = neg_inf();
    for (int c = lane; c < nc; c += 32) M = fmaxf(M, my_ms[c].x);
    M = ordered_to_float(__reduce_max_sync(kFullMask, float_to_ordered(M)));
    float S = 0.f;
    for (int c = lane; c < nc; c += 32) {
      const float2 ms = my_ms[c];
      if (ms.y > 0.f) S += ms.y * expf(ms.x - M);
    }
    S = warp_sum(S);
    // planted column: its logit is (max of the others) + delta and it was left out of the partials
    const int pc = plant_s[j];
    unsigned long long plant_key = 0ull;
    if (pc >= 0) {
      const float zc = M + p.plant_delta;
      const float M2 = fmaxf(M, zc);
      S = S * expf(M - M2) + expf(zc - M2);
      M = M2;
      plant_key = make_key(zc, (uint32_t)pc);
    }
    if (lane == 0) {
      lse_s[j] = M + logf(S);
      plant_key_s[j] = plant_key;
    }
  }
  __syncthreads();
  asm volatile("barrier.cluster.wait.aligned;" ::: "memory");   // every block of the cluster is running
  unsigned long long node_rec = 0ull;
  int node_flat = -1;
  float node_lse = 0.f;
  if (warp < n_mine) {
    const int pr = crank + kSelCluster * warp;
    const float lse = lse_s[warp];
    const unsigned long long plant_key = plant_key_s[warp];
    // insert the planted candidate into the sorted result
    if (plant_key != 0ull) {
      const int ins = __popc(__ballot_sync(kFullMask, lane < k && res > plant_key));
      const unsigned long long up = __shfl_up_sync(kFullMask, res, 1);
      if (lane == ins) res = plant_key;
      else if (lane > ins) res = up;
    }
    if (lane < k) {
      const float lp = (res != 0ull) ? fminf(key_value(res) - lse, 0.f) : neg_inf();
      const int tok = (res != 0ull) ? (int)key_index(res) : -1;
      const float cand = beam_cum_s[warp] + lp;
      const int flat = pr * k + lane;
      // every block of the cluster gets the candidates of all rows
      node_rec = ((unsigned long long)__float_as_uint(cand) << 32) | (uint32_t)tok;
      for (int rk = 0; rk < kSelCluster; ++rk) cluster.map_shared_rank(cand_rec, rk)[flat] = node_rec;
      node_flat = flat;
    }
    node_lse = lse;
  }
  cluster.sync();       // the last time a block touches another block's shared memory before the draft step
  // The new tree nodes go to global memory only now: the barrier above has release semantics,
  // and with these stores ahead of it every block waited for them to reach L2 under the next
  // pass's W burst.  (A sequence that stops meets at one more barrier before its rerank.)
  if (node_flat >= 0) {
    const size_t node = (size_t)b * p.Nn + base + node_flat;
    p.tree_token[node] = (int)(uint32_t)node_rec;
    p.tree_parent[node] = beam_node_s[warp];
    p.tree_cum[node] = __uint_as_float((uint32_t)(node_rec >> 32));
  }
  if (warp < n_mine && lane == 0 && io.trace.row_lse)
    io.trace.row_lse[((size_t)b * p.n + (d - 1)) * k + crank + kSelCluster * warp] = node_lse;

  // ---- phase 2: warp 0 of every block picks the new beam, evaluates Eq. 1 and takes the stop
  //      decision (same inputs, same result everywhere; block 0 records it)
  if (warp == 0) {
    const int n_cand = P * k;
    unsigned long long mine = 0ull;
    if (n_cand <= 128) {
      unsigned long long ck[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) ck[i] = lane + 32 * i < n_cand ? cand_key_of(lane + 32 * i) : 0ull;
      for (int j = 0; j < k; ++j) {
        unsigned long long best = ck[0];
#pragma unroll
        for (int i = 1; i < 4; ++i) best = ck[i] > best ? ck[i] : best;
        const unsigned long long wk = warp_max_key(best);
        if (lane == j) mine = wk;
        if (wk == 0ull) break;
#pragma unroll
        for (int i = 0; i < 4; ++i)
          if (ck[i] == wk) ck[i] = 0ull;
      }
    } else {
      // more candidates than fit four per lane: the k candidates of a beam row are already in
      // descending key order (same parent score, log-probabilities descending, ties by lower
      // index), so lane p walks row p and the beam is a k-way merge of the P <= 32 rows
      int pos = 0;
      unsigned long long head = lane < P ? cand_key_of(lane * k) : 0ull;
      for (int j = 0; j < k; ++j) {
        const unsigned long long wk = warp_max_key(head);
        if (lane == j) mine = wk;
        if (wk == 0ull) break;
        if (head == wk) {                   // keys are unique: exactly one lane
          ++pos;
          head = pos < k ? cand_key_of(lane * k + pos) : 0ull;
        }
      }
    }
    const bool have = lane < k && mine != 0ull;
    const int flat = have ? (int)key_index(mine) : 0;
    const float cum = have ? __uint_as_float((uint32_t)(cand_rec[flat] >> 32)) : neg_inf();
    const float M = __shfl_sync(kFullMask, cum, 0);           // sorted descending: entry 0 is the max
    const float sum = warp_sum(have ? expf(cum - M) : 0.f);
    const float H = M + logf(sum);
    bool stop = (d == p.n);
    if (!stop && ((p.check_mask >> (d - 1)) & 1u)) stop = H < p.x;
    const int tok = lane < k ? (int)(uint32_t)cand_rec[flat] : -1;
    if (lane < k) {
      sel_flat[lane] = flat;
      sel_tok[lane] = tok;
    }
    if (lane == 0) s_stop = stop ? 1 : 0;
    __syncwarp();
    if (crank == 0) {
      // block 0 keeps the books in global memory (the other warps of the cluster go on meanwhile)
      if (lane < k) {
        p.beam_node[b * k + lane] = base + flat;
        p.beam_tok[b * k + lane] = tok;
        p.beam_cum[b * k + lane] = cum;
        p.row_plant[b * k + lane] = (p.plant_next && tok >= 0 && tok < p.V) ? p.plant_next[tok] : -1;
        if (io.trace.beam_sel) io.trace.beam_sel[((size_t)b * p.n + (d - 1)) * k + lane] = flat;
      }
      if (lane == 0) {
        io.out.H_trace[(size_t)b * p.n + (d - 1)] = H;
        if (stop) {
          p.stop_depth[b] = d;
          p.active[b] = 0;
          s_last = atomicSub(p.n_active, 1) == 1;
        }
      }
    }
  }
  __syncthreads();
  // In a captured draft the passes after this one sit behind a conditional node (default: skip);
  // a sequence that goes on switches them on.
  if (set_cond && !s_stop && crank == 0 && threadIdx.x == 0) cudaGraphSetConditional(cond, 1);
  if (s_stop) {             // every block takes this branch alike
    // the sequence is finished: block 0 goes on to the rerank and the mask once the nodes the other
    // blocks appended in this pass are visible to it
    cluster.sync();
    if (crank == 0) rerank_mask_block<kSelThreads, true>(p, io, b, d, s_last, smem_raw);
    return;
  }

  // ---- phase 3: synthetic draft step for the k new beam rows
  if (p.dtype == DDD_DTYPE_BF16)
    draft_step<__nv_bfloat16>(p, b, d, sel_flat, sel_tok, row_part, row_inv);
  else
    draft_step<float>(p, b, d, sel_flat, sel_tok, row_part, row_inv);
}


// ---------------------------------------------------------------------------- wide beams (width 33..128)
// The same pass for beams too wide for one key per lane.  Every list here - a thread block's
// partial top-k of a row, a row's k candidates, the new beam - is a sorted wide list (four keys
// per lane, ddd_common.cuh), and every choice is a merge of sorted lists: the warps of a block
// each fold a share of the lists into one, the 16 results meet in shared memory and are merged
// pairwise in four rounds.
// Dynamic shared memory: candidate records [k*k], merge buffers [16][128], partial sums of squares
// of the draft step [k][slots]; after a stop the same memory serves the rerank.
// The best k of n candidate records (score bits << 32 | token, token < 0 = no candidate) of a
// sequence, as a sorted wide list in warp 0's `acc` (keys: score, then lower candidate index).
// Merging the P sorted rows of 128-key lists took 22 us at width 100; here every thread keeps
// the best score among its share of the candidates, the smallest over the 16 warps of the
// warp's j-th largest thread maximum (j = k / 16 rounded up) has k candidates at or above it,
// those are gathered (a few hundred) and each is placed by counting the better ones.  Returns
// false, with nothing changed, when more than kPickCap candidates reach the floor (equal
// scores).  Called by the whole block; scratch: kWideWarps * kWideK 8-byte words.
constexpr int kPickCap = 1024;
__device__ bool pick_beam_by_floor(const unsigned long long* cand_rec, const int n, const int k,
                                   unsigned long long* scratch, unsigned long long (&acc)[4]) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  unsigned long long* gathered = scratch;                            // [kPickCap]
  unsigned long long* chosen = scratch + kPickCap;                   // [kWideK]
  uint32_t* warp_floor = reinterpret_cast<uint32_t*>(chosen + kWideK);   // [kWideWarps]
  int* count_s = reinterpret_cast<int*>(warp_floor + kWideWarps);
  uint32_t best = 0u;
  for (int f = tid; f < n; f += kWideThreads) {
    const unsigned long long rec = cand_rec[f];
    if ((int)(uint32_t)rec >= 0) best = max(best, float_to_ordered(__uint_as_float((uint32_t)(rec >> 32))));
  }
  {
    const int j = (k + kWideWarps - 1) / kWideWarps;
    uint32_t cur = best, jth = 0u;
    for (int t = 0; t < j; ++t) {
      jth = __reduce_max_sync(kFullMask, cur);
      const unsigned who = __ballot_sync(kFullMask, cur == jth);
      if (lane == __ffs(who) - 1) cur = 0u;
    }
    if (lane == 0) warp_floor[warp] = jth;
  }
  if (tid == 0) *count_s = 0;
  if (tid < kWideK) chosen[tid] = 0ull;
  __syncthreads();
  uint32_t floor_o = warp_floor[0];
  for (int w = 1; w < kWideWarps; ++w) floor_o = min(floor_o, warp_floor[w]);
  // a warp with fewer than j candidates says nothing: then everything counts
  for (int f = tid; f < n; f += kWideThreads) {
    const unsigned long long rec = cand_rec[f];
    if ((int)(uint32_t)rec < 0) continue;
    const float score = __uint_as_float((uint32_t)(rec >> 32));
    if (float_to_ordered(score) < floor_o) continue;
    const int at = atomicAdd(count_s, 1);
    if (at < kPickCap) gathered[at] = make_key(score, (uint32_t)f);
  }
  __syncthreads();
  const int count = *count_s;
  if (count > kPickCap) {
    __syncthreads();
    return false;
  }
  for (int e = tid; e < count; e += kWideThreads) {
    const unsigned long long mine = gathered[e];
    int place = 0;
    for (int i = 0; i < count; ++i) place += gathered[i] > mine ? 1 : 0;
    if (place < k) chosen[place] = mine;
  }
  __syncthreads();
  if (warp == 0) wide_load(acc, chosen, k);
  __syncthreads();
  return true;
}

__global__ void __launch_bounds__(kWideThreads) select_gate_step_wide_kernel(const Params p, const DraftIO io,
                                                                             const int d, const int part_slots,
                                                                             const cudaGraphConditionalHandle cond,
                                                                             const int set_cond) {
  griddep_wait();
  griddep_launch_dependents();
  cg::cluster_group cluster = cg::this_cluster();
  const int crank = (int)cluster.block_rank();
  const int b = blockIdx.x / kSelCluster;
  if (p.active[b] == 0) return;                               // same decision in the whole cluster
  // split cluster barrier: remote shared-memory stores below need every block of the cluster running
  asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int k = p.k, nc = p.lm_ctas, R = p.R;
  const int P = (d == 1) ? 1 : k;
  const int base = (d == 1) ? 1 : 1 + k + (d - 2) * k * k;

  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned long long* cand_rec = reinterpret_cast<unsigned long long*>(smem_raw);           // [k * k]
  unsigned long long* buf = cand_rec + (size_t)k * k;                                       // [16][128]
  double* row_part = reinterpret_cast<double*>(buf + kWideWarps * kWideK);                  // [k][part_slots]
  __shared__ int sel_flat[kWideK];
  __shared__ int sel_tok[kWideK];
  __shared__ double row_inv[kWideK];
  __shared__ int s_stop;
  __shared__ bool s_last;
  (void)part_slots;

  // ---- phase 1: merge the partial lists of this block's beam rows
  // What a warp does with a row's merged list acc and the row's (max, sum-exp) over all partials:
  // planted column, log-sum-exp, the k candidates to every block of the cluster, the tree nodes.
  auto finish_row = [&](const int pr, unsigned long long (&acc)[4], float M, float S) {
    const int r = b * k + pr;
    const int pc = p.row_plant[r];
    if (pc >= 0) {          // planted column: (max of the others) + delta; it was left out of the partials
      const float zc = M + p.plant_delta;
      const float M2 = fmaxf(M, zc);
      S = S * expf(M - M2) + expf(zc - M2);
      M = M2;
      unsigned long long one[4] = {lane == 0 ? make_key(zc, (uint32_t)pc) : 0ull, 0ull, 0ull, 0ull};
      wide_merge(acc, one);
    }
    const float lse = M + logf(S);
    const float cum0 = p.beam_cum[r];
    const int parent_node = p.beam_node[r];
#pragma unroll
    for (int s4 = 0; s4 < 4; ++s4) {
      const int e = 4 * lane + s4;
      if (e >= k) continue;
      const unsigned long long key = acc[s4];
      const float lp = key != 0ull ? fminf(key_value(key) - lse, 0.f) : neg_inf();
      const int tok = key != 0ull ? (int)key_index(key) : -1;
      const float cand = cum0 + lp;
      const int flat = pr * k + e;
      const unsigned long long rec = ((unsigned long long)__float_as_uint(cand) << 32) | (uint32_t)tok;
      cluster.map_shared_rank(cand_rec, 0)[flat] = rec;          // block 0 of the cluster picks the beam
      const size_t node = (size_t)b * p.Nn + base + flat;
      p.tree_token[node] = tok;
      p.tree_parent[node] = parent_node;
      p.tree_cum[node] = cand;
    }
    if (lane == 0 && io.trace.row_lse) io.trace.row_lse[((size_t)b * p.n + (d - 1)) * k + pr] = lse;
  };
  bool waited = false;
  if (nc == 1) {
    // one partial per row (the per-block partials were folded by a kernel of their own, or there is
    // one record set slot): nothing to merge, a warp per row, all rows of the block at once
    asm volatile("barrier.cluster.wait.aligned;" ::: "memory");
    waited = true;
    for (int pr = crank + kSelCluster * warp; pr < P; pr += kSelCluster * kWideWarps) {
      const int r = b * k + pr;
      unsigned long long acc[4];
      wide_load(acc, p.part_key + (size_t)r * k, k);
      const float2 ms = p.part_ms[r];
      finish_row(pr, acc, ms.x, ms.y);
    }
  } else {
    for (int pr = crank; pr < P; pr += kSelCluster) {
      const int r = b * k + pr;
      unsigned long long acc[4] = {0ull, 0ull, 0ull, 0ull};
      for (int c = warp; c < nc; c += kWideWarps) {
        unsigned long long t[4];
        wide_load(t, p.part_key + ((size_t)c * R + r) * k, k);
        wide_merge(acc, t);
      }
      block_merge_lists(acc, buf);
      if (!waited) {
        asm volatile("barrier.cluster.wait.aligned;" ::: "memory");
        waited = true;
      }
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
        finish_row(pr, acc, M, S);
      }
      __syncthreads();
    }
  }
  if (!waited) asm volatile("barrier.cluster.wait.aligned;" ::: "memory");
  cluster.sync();
  // The candidates and the tree nodes of all rows are in place.  The draft step is a kernel of
  // its own, so nothing is left for the other blocks: block 0 picks the beam, takes the stop
  // decision, keeps the books and reranks at a stop.
  if (crank != 0) return;

  // ---- phase 2: the new beam = best k of the P * k candidates
  {
    unsigned long long acc[4] = {0ull, 0ull, 0ull, 0ull};
    if (!pick_beam_by_floor(cand_rec, P * k, k, buf, acc)) {
      // many equal scores: merge the P sorted candidate rows instead
      for (int row = warp; row < P; row += kWideWarps) {
        unsigned long long t[4];
#pragma unroll
        for (int s4 = 0; s4 < 4; ++s4) {
          const int e = 4 * lane + s4;
          t[s4] = 0ull;
          if (e < k) {
            const unsigned long long rec = cand_rec[row * k + e];
            if ((int)(uint32_t)rec >= 0) t[s4] = make_key(__uint_as_float((uint32_t)(rec >> 32)), (uint32_t)(row * k + e));
          }
        }
        wide_merge(acc, t);
      }
      block_merge_lists(acc, buf);
    }
    if (warp == 0) {
      float cum[4];
      int flat[4], tok[4];
      float part = 0.f;
      const float M = key_value(wide_element(acc, 0));          // sorted descending: entry 0 is the maximum
#pragma unroll
      for (int s4 = 0; s4 < 4; ++s4) {
        const int e = 4 * lane + s4;
        const bool have = e < k && acc[s4] != 0ull;
        flat[s4] = have ? (int)key_index(acc[s4]) : 0;
        cum[s4] = have ? key_value(acc[s4]) : neg_inf();
        tok[s4] = e < k ? (int)(uint32_t)cand_rec[flat[s4]] : -1;
        if (have) part += expf(cum[s4] - M);
        if (e < k) {
          sel_flat[e] = flat[s4];
          sel_tok[e] = tok[s4];
        }
      }
      const float H = M + logf(warp_sum(part));
      bool stop = (d == p.n);
      if (!stop && ((p.check_mask >> (d - 1)) & 1u)) stop = H < p.x;
      if (lane == 0) s_stop = stop ? 1 : 0;
      __syncwarp();
      if (crank == 0) {
#pragma unroll
        for (int s4 = 0; s4 < 4; ++s4) {
          const int e = 4 * lane + s4;
          if (e >= k) continue;
          p.beam_node[b * k + e] = base + flat[s4];
          p.beam_tok[b * k + e] = tok[s4];
          p.beam_cum[b * k + e] = cum[s4];
          p.row_plant[b * k + e] = (p.plant_next && tok[s4] >= 0 && tok[s4] < p.V) ? p.plant_next[tok[s4]] : -1;
          if (io.trace.beam_sel) io.trace.beam_sel[((size_t)b * p.n + (d - 1)) * k + e] = flat[s4];
        }
        if (lane == 0) {
          io.out.H_trace[(size_t)b * p.n + (d - 1)] = H;
          if (stop) {
            p.stop_depth[b] = d;
            p.active[b] = 0;
            s_last = atomicSub(p.n_active, 1) == 1;
          }
        }
      }
    }
  }
  __syncthreads();
  if (set_cond && !s_stop && crank == 0 && threadIdx.x == 0) cudaGraphSetConditional(cond, 1);
  if (s_stop) {
    // the nodes the other blocks appended in this pass were written before the cluster barrier above
    if (p.Nn * 6 <= 160 * 1024) rerank_mask_block<kWideThreads, true>(p, io, b, d, s_last, smem_raw);
    else rerank_mask_block<kWideThreads, false>(p, io, b, d, s_last, smem_raw);
    return;
  }
  // the draft step of the k new rows is a kernel of its own behind this one (draft_rows_kernel)
  (void)row_part;
  (void)row_inv;
  (void)sel_tok;
}

// The synthetic draft step of a wide beam, one block per new beam row (Algorithm 1, "Run draft model on
// beam"; here h = round(u / sqrt(mean(u^2) + eps)), u = h_parent + E[token], in fp64).  Inside the
// select kernel the step had the eight SMs of a sequence's cluster: at width 100 its 100 rows of
// fp64 conversions and sums took 25 us of the kernel's 43; as B * k blocks it has the whole device.
// The row's token and parent come from the beam state the select kernel has just written.
constexpr int kRowThreads = 256;
template <typename T>
__global__ void __launch_bounds__(kRowThreads) draft_rows_kernel(const Params p, const int d) {
  griddep_wait();
  griddep_launch_dependents();
  constexpr int N = Chunk<T>::N;
  const int k = p.k, r = blockIdx.x, b = r / k;
  if (d >= p.n || p.active[b] == 0) return;          // no step after the last pass or after a stop
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int base = (d == 1) ? 1 : 1 + k + (d - 2) * k * k;
  const int parent_slot = (p.beam_node[r] - base) / k;
  const int tok = p.beam_tok[r];
  const int cpr = p.Hd / N;
  const uint4* hp = reinterpret_cast<const uint4*>(p.hbuf[(d - 1) & 1]) + (size_t)(b * k + parent_slot) * cpr;
  const uint4* er = reinterpret_cast<const uint4*>(p.E) + (size_t)(tok >= 0 && tok < p.V ? tok : 0) * cpr;
  uint4* out = reinterpret_cast<uint4*>(p.hbuf[d & 1]) + (size_t)r * cpr;
  __shared__ double red[kRowThreads / 32];
  double ss = 0.0;
  for (int q = threadIdx.x; q < cpr; q += kRowThreads) {
    double u[N];
    Chunk<T>::sum(hp[q], er[q], u);
#pragma unroll
    for (int e = 0; e < N; ++e) ss = fma(u[e], u[e], ss);
  }
  ss = warp_sum_f64(ss);
  if (lane == 0) red[warp] = ss;
  __syncthreads();
  double total = 0.0;
  for (int w = 0; w < kRowThreads / 32; ++w) total += red[w];
  const double inv = 1.0 / sqrt(total / (double)p.Hd + (double)p.eps);
  for (int q = threadIdx.x; q < cpr; q += kRowThreads) {
    double u[N];
    Chunk<T>::sum(hp[q], er[q], u);
#pragma unroll
    for (int e = 0; e < N; ++e) u[e] *= inv;
    out[q] = Chunk<T>::round(u);
  }
}

// Can the partial lists of a block's rows live in its shared memory?  (Host and device agree
// through the kernel argument.)
size_t select_smem_bytes(const Params& p, bool lists) {
  const size_t rows_max = (p.k + kSelCluster - 1) / kSelCluster;
  const size_t kl = lists ? p.k : 1;
  return rows_max * p.lm_ctas * (kl * sizeof(unsigned long long) + sizeof(float2)) + rows_max * sizeof(int);
}
bool select_lists_in_smem(const Params& p) {
  return p.lm_ctas <= 320 && select_smem_bytes(p, true) <= 160 * 1024;
}
bool is_wide(const Params& p) { return p.k > kNarrowK; }
// the rerank keeps 32-bit keys and 16-bit row numbers of all tree nodes in shared memory; trees too
// large for that (wide beams) keep only the row numbers there and read the scores from global memory
size_t rerank_smem(const Params& p) {
  const size_t both = (size_t)p.Nn * (sizeof(uint32_t) + sizeof(short));
  return (!is_wide(p) || both <= 160 * 1024) ? both : (size_t)p.Nn * sizeof(short);
}
int wide_part_slots(const Params& p) {
  const int cpr = p.Hd / (p.dtype == DDD_DTYPE_BF16 ? 8 : 4);
  return (cpr % 32 == 0 && cpr / 32 <= 64) ? cpr / 32 : 0;
}
size_t wide_select_smem(const Params& p) {
  return ((size_t)p.k * p.k + kWideWarps * kWideK) * sizeof(unsigned long long) +
         (size_t)p.k * wide_part_slots(p) * sizeof(double);
}
// the select kernel's dynamic shared memory also serves the rerank that follows a stop
size_t select_smem(const Params& p) {
  const size_t a = is_wide(p) ? wide_select_smem(p) : select_smem_bytes(p, select_lists_in_smem(p)), b = rerank_smem(p);
  return a > b ? a : b;
}

}  // namespace

// ---------------------------------------------------------------------------- launchers
cudaError_t prepare_tree(const Params& p) {
  // static + dynamic shared memory of the select kernel must fit one block's limit
  cudaFuncAttributes fa;
  const bool wide = p.k >= kSelWideFromK;
  cudaError_t e = is_wide(p) ? cudaFuncGetAttributes(&fa, select_gate_step_wide_kernel)
                  : wide     ? cudaFuncGetAttributes(&fa, select_gate_step_kernel<kSelThreadsWide>)
                             : cudaFuncGetAttributes(&fa, select_gate_step_kernel<kSelThreadsNarrow>);
  if (e != cudaSuccess) return e;
  int dev = 0, limit = 0;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&limit, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev)) != cudaSuccess) return e;
  if (fa.sharedSizeBytes + select_smem(p) > (size_t)limit) return cudaErrorInvalidValue;
  if (is_wide(p)) return allow_max_dynamic_smem(select_gate_step_wide_kernel);
  return wide ? allow_max_dynamic_smem(select_gate_step_kernel<kSelThreadsWide>)
              : allow_max_dynamic_smem(select_gate_step_kernel<kSelThreadsNarrow>);
}

cudaError_t launch_init(const Params& p, const DraftIO&, const void* root_hidden, const int* root_token,
                        const int* root_pos, cudaStream_t st) {
  if (p.dtype == DDD_DTYPE_FP32)
    init_kernel<float><<<p.B, 256, 0, st>>>(p, static_cast<const float*>(root_hidden), root_token, root_pos);
  else
    init_kernel<__nv_bfloat16><<<p.B, 256, 0, st>>>(p, static_cast<const __nv_bfloat16*>(root_hidden),
                                                    root_token, root_pos);
  return cudaGetLastError();
}

cudaError_t launch_select(const Params& p, const DraftIO& io, int d, bool pdl, cudaGraphConditionalHandle cond,
                          bool set_cond, cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(p.B * kSelCluster), 1, 1);
  const bool wide = p.k >= kSelWideFromK;
  cfg.blockDim = dim3(is_wide(p) ? kWideThreads : wide ? kSelThreadsWide : kSelThreadsNarrow, 1, 1);
  cfg.dynamicSmemBytes = select_smem(p);
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = kSelCluster;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 2 : 1;
  const int lists = select_lists_in_smem(p) ? 1 : 0, sc = set_cond ? 1 : 0;
  if (is_wide(p)) {
    cudaError_t e = cudaLaunchKernelEx(&cfg, select_gate_step_wide_kernel, p, io, d, wide_part_slots(p), cond, sc);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t rows = {};
    rows.gridDim = dim3((unsigned)p.R, 1, 1);
    rows.blockDim = dim3(kRowThreads, 1, 1);
    rows.stream = st;
    rows.attrs = attr + 1;                    // the programmatic-serialisation attribute alone
    rows.numAttrs = pdl ? 1 : 0;
    if (p.dtype == DDD_DTYPE_BF16) return cudaLaunchKernelEx(&rows, draft_rows_kernel<__nv_bfloat16>, p, d);
    return cudaLaunchKernelEx(&rows, draft_rows_kernel<float>, p, d);
  }
  if (wide) return cudaLaunchKernelEx(&cfg, select_gate_step_kernel<kSelThreadsWide>, p, io, d, lists, cond, sc);
  return cudaLaunchKernelEx(&cfg, select_gate_step_kernel<kSelThreadsNarrow>, p, io, d, lists, cond, sc);
}

}  // namespace ddd
