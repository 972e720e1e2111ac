// Device code shared by the kernels that finish a pass (tree_kernels.cu, and the tail of the
// tensor-core LM-head kernel): merging of the per-block partial lists, the fp64 pieces of the
// synthetic draft step, and the rerank with the ancestor mask.
#pragma once

#include "ddd_common.cuh"

namespace ddd {

__device__ __forceinline__ double warp_sum_f64(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFullMask, v, o);
  return v;
}

// fp64 -> bf16 bit pattern with one round-to-nearest-even step (normal range): keep the top
// 7 explicit mantissa bits of the double, then the narrowing conversions are exact.
__device__ __forceinline__ uint32_t f64_to_bf16_bits(double y) {
  unsigned long long bits = (unsigned long long)__double_as_longlong(y);
  const unsigned long long lsb = (bits >> 45) & 1ull;
  bits += ((1ull << 44) - 1ull) + lsb;
  bits &= ~((1ull << 45) - 1ull);
  const float f = (float)__longlong_as_double((long long)bits);
  return __float_as_uint(f) >> 16;
}

// Loads issued by one thread are batched (a few independent loads, then their use): a single
// block runs this kernel between two LM-head passes, so its time is made of memory round
// trips, and a loop that loads and uses one value per iteration pays one trip per iteration.
// Merge of one beam row's per-block partial lists when all of them are in shared memory
// (keys_s[c * k + q] = q-th best key of block c, descending, 0 = empty): a k-way merge in
// which every lane keeps the heads of its NL lists (blocks lane, lane + 32, ...) in registers.
// One round = best head of the lane, maximum over the warp, the owning lane steps that list.
// Lane j returns the j-th best key (0 if there is none).
template <int NL>
__device__ __forceinline__ unsigned long long merge_row_heads(int k, int nc, const unsigned long long* keys_s) {
  const int lane = threadIdx.x & 31;
  unsigned long long head[NL];
  int pos[NL];
#pragma unroll
  for (int i = 0; i < NL; ++i) {
    const int c = lane + 32 * i;
    head[i] = c < nc ? keys_s[(size_t)c * k] : 0ull;
    pos[i] = 0;
  }
  unsigned long long res = 0ull;
  for (int j = 0; j < k; ++j) {
    unsigned long long best = head[0];
#pragma unroll
    for (int i = 1; i < NL; ++i) best = head[i] > best ? head[i] : best;
    const unsigned long long wk = warp_max_key(best);
    if (wk == 0ull) break;
    if (lane == j) res = wk;
    if (best == wk) {                      // keys are unique: one lane, one list
#pragma unroll
      for (int i = 0; i < NL; ++i) {
        if (head[i] == wk) {
          ++pos[i];
          head[i] = pos[i] < k ? keys_s[(size_t)(lane + 32 * i) * k + pos[i]] : 0ull;
        }
      }
    }
  }
  return res;
}


// Blocks that work on wide lists (ddd_common.cuh) have 16 warps.
constexpr int kWideThreads = 512;
constexpr int kWideWarps = kWideThreads / 32;

// Tree of pairwise merges over the warps' lists in buf [kWideWarps][kWideK]; the result ends up
// in warp 0's registers (and in buf[0]).  All threads of the block call this.
__device__ __forceinline__ void block_merge_lists(unsigned long long (&acc)[4], unsigned long long* buf) {
  const int warp = threadIdx.x >> 5;
  wide_store(acc, buf + warp * kWideK, kWideK);
  __syncthreads();
  for (int half = kWideWarps / 2; half >= 1; half >>= 1) {
    if (warp < half) {
      unsigned long long other[4];
      wide_load(other, buf + (warp + half) * kWideK, kWideK);
      wide_merge(acc, other);
      wide_store(acc, buf + warp * kWideK, kWideK);
    }
    __syncthreads();
  }
}


// 8 (bf16) or 4 (fp32) consecutive elements of h_parent + E[token], formed in fp64.
template <typename T>
struct Chunk;
template <>
struct Chunk<__nv_bfloat16> {
  static constexpr int N = 8;
  typedef uint4 Raw;
  __device__ static void sum(const uint4& a, const uint4& c, double (&u)[8]) {
    const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, cw[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      u[2 * q] = (double)__uint_as_float(aw[q] << 16) + (double)__uint_as_float(cw[q] << 16);
      u[2 * q + 1] = (double)__uint_as_float(aw[q] & 0xFFFF0000u) + (double)__uint_as_float(cw[q] & 0xFFFF0000u);
    }
  }
  __device__ static uint4 round(const double (&y)[8]) {
    uint32_t w[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) w[q] = f64_to_bf16_bits(y[2 * q]) | (f64_to_bf16_bits(y[2 * q + 1]) << 16);
    return make_uint4(w[0], w[1], w[2], w[3]);
  }
};
template <>
struct Chunk<float> {
  static constexpr int N = 4;
  typedef uint4 Raw;
  __device__ static void sum(const uint4& a, const uint4& c, double (&u)[4]) {
    u[0] = (double)__uint_as_float(a.x) + (double)__uint_as_float(c.x);
    u[1] = (double)__uint_as_float(a.y) + (double)__uint_as_float(c.y);
    u[2] = (double)__uint_as_float(a.z) + (double)__uint_as_float(c.z);
    u[3] = (double)__uint_as_float(a.w) + (double)__uint_as_float(c.w);
  }
  __device__ static uint4 round(const double (&y)[4]) {
    return make_uint4(__float_as_uint(__double2float_rn(y[0])), __float_as_uint(__double2float_rn(y[1])),
                      __float_as_uint(__double2float_rn(y[2])), __float_as_uint(__double2float_rn(y[3])));
  }
};


// ---------------------------------------------------------------------------- rerank + mask
__device__ __forceinline__ int node_depth(int id, int k) {
  if (id == 0) return 0;
  if (id <= k) return 1;
  return 2 + (id - 1 - k) / (k * k);
}

// Block-wide exclusive prefix sum of one int per thread (THREADS threads).
// Sync::sync() is the barrier of the THREADS threads that call this together (a whole block, or
// a group of warps on a named barrier); tid is the caller's index in that group.
struct BlockSync {
  __device__ static __forceinline__ void sync() { __syncthreads(); }
};
template <int THREADS, typename Sync>
__device__ int block_exclusive_scan(int v, int* warp_tot /* [32] shared */, int* total, const int tid) {
  const int lane = tid & 31, warp = tid >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(kFullMask, inc, o);
    if (lane >= o) inc += t;
  }
  Sync::sync();                 // protect warp_tot from its previous use
  if (lane == 31) warp_tot[warp] = inc;
  Sync::sync();
  int offset = 0, tot = 0;
  for (int w = 0; w < THREADS / 32; ++w) {
    const int t = warp_tot[w];
    if (w < warp) offset += t;
    tot += t;
  }
  *total = tot;
  return offset + inc - v;
}

// Final step of a sequence, run by one block of THREADS threads right after the pass at
// which the sequence stopped (D): keep the m best nodes, emit the rows and the ancestor mask.
// smem_raw: ordered cum keys [Nn] (32 bit), then selection flags / output rows [Nn] (16 bit).  `last` says that this
// was the last sequence of the batch still drafting: that block also reports the device status.
// KEYS_IN_SMEM false: the tree is too large to keep its keys in shared memory; they are formed from
// the scores in global memory each time (smem_raw then holds only the 16-bit rows).
// The group's scratch: hist [256], warp_tot [32], two words (prefix, remaining), all 32-bit, and
// out_parent [T] 16-bit; `cap` = node slots smem_raw has room for (at least N + 1).
constexpr int kRerankScratchInts = 256 + 32 + 2;
template <int THREADS, bool KEYS_IN_SMEM, typename Sync>
__device__ void rerank_mask_impl(const Params& p, const DraftIO& io, const int b, const int D, const bool last,
                                 const int tid, unsigned char* smem_raw, const int cap, int* scratch,
                                 short* out_parent) {
  const int k = p.k, T = p.T;
  const int N = (D >= 1) ? k + (D - 1) * k * k : 0;     // generated non-root nodes
  uint32_t* key_s = reinterpret_cast<uint32_t*>(smem_raw);         // key of node id i+1 at [i]
  short* slot_of = reinterpret_cast<short*>(KEYS_IN_SMEM ? smem_raw + (size_t)cap * sizeof(uint32_t) : smem_raw);
                                                                    // output row of node id (< 1024), -1 = dropped
  int* hist = scratch;
  int* warp_tot = scratch + 256;
  uint32_t& s_prefix = *reinterpret_cast<uint32_t*>(scratch + 288);
  int& s_remaining = scratch[289];

  const float* cum = p.tree_cum + (size_t)b * p.Nn;
  const int* tparent = p.tree_parent + (size_t)b * p.Nn;
  const int* ttoken = p.tree_token + (size_t)b * p.Nn;
  auto key = [&](int i) -> uint32_t { return KEYS_IN_SMEM ? key_s[i] : float_to_ordered(cum[i + 1]); };
  if (KEYS_IN_SMEM)
    for (int i = tid; i < N; i += THREADS) key_s[i] = float_to_ordered(cum[i + 1]);
  const int m_eff = min(p.m, N);
  if (tid == 0) { s_prefix = 0u; s_remaining = m_eff; }
  Sync::sync();

  int n_selected;
  if (KEYS_IN_SMEM && N <= THREADS) {
    // ---- few nodes (a draft that stopped early: the common case): a node is ranked by counting the
    // nodes that come before it in (score descending, node id ascending) order, the count shared
    // between as many threads as the block has per node (a power of two inside one warp); the
    // kept nodes' rows follow from a ballot per warp.  Four barriers against the thirty-odd of the
    // radix path, and no loop over the nodes longer than N / (threads per node).
    int tpn = 1;
    while (tpn < 32 && 2 * tpn * N <= THREADS) tpn *= 2;
    const int node = tid / tpn, part = tid - node * tpn;
    const uint32_t mine = node < N ? key_s[node] : 0u;
    int rank = 0;
    for (int j = part; j < N; j += tpn) {
      const uint32_t q = key_s[j];
      rank += (q > mine || (q == mine && j < node)) ? 1 : 0;
    }
    for (int o = tpn >> 1; o > 0; o >>= 1) rank += __shfl_xor_sync(kFullMask, rank, o);
    if (node < N && part == 0) slot_of[node + 1] = rank < m_eff ? 1 : 0;
    Sync::sync();
    // thread t now speaks for node t: rows are dealt out in node order
    const bool sel = tid < N && slot_of[tid + 1] != 0;
    const unsigned warp_sel = __ballot_sync(kFullMask, sel);
    if ((tid & 31) == 0) warp_tot[tid >> 5] = __popc(warp_sel);
    Sync::sync();
    int before = __popc(warp_sel & ((1u << (tid & 31)) - 1u)), total = 0;
    for (int w = 0; w * 32 < N; ++w) {
      const int c = warp_tot[w];
      total += c;
      before += w < (tid >> 5) ? c : 0;
    }
    n_selected = total;
    if (tid < N) slot_of[tid + 1] = sel ? (short)(1 + before) : (short)-1;
    if (tid == 0) slot_of[0] = 0;
    Sync::sync();
  } else {
    // ---- radix select: value of the m_eff-th largest key and how many of its ties to keep
    uint32_t known_mask = 0u;
    for (int pass = 3; pass >= 0 && m_eff > 0; --pass) {
      const int shift = 8 * pass;
      for (int i = tid; i < 256; i += THREADS) hist[i] = 0;
      Sync::sync();
      const uint32_t prefix = s_prefix;
      for (int i = tid; i < N; i += THREADS) {
        const uint32_t q = key(i);
        if ((q & known_mask) == prefix) atomicAdd(&hist[(q >> shift) & 0xFF], 1);
      }
      Sync::sync();
      if (tid < 32) {
        // warp 0 finds the bin holding the `remaining`-th largest key: lane l owns bins 8l .. 8l+7
        const int remaining = s_remaining;
        int local[8], mine = 0;
  #pragma unroll
        for (int i = 0; i < 8; ++i) { local[i] = hist[8 * tid + i]; mine += local[i]; }
        int above = mine;                                   // suffix sum over lanes >= tid ...
  #pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int t = __shfl_down_sync(kFullMask, above, o);
          if (tid + o < 32) above += t;
        }
        above -= mine;                                      // ... made exclusive: keys in higher lanes' bins
        if (above < remaining && remaining <= above + mine) {   // exactly one lane
          int rem = remaining - above, bin = 7;
          for (; bin > 0; --bin) {
            if (local[bin] >= rem) break;
            rem -= local[bin];
          }
          s_prefix = prefix | ((uint32_t)(8 * tid + bin) << shift);
          s_remaining = rem;
        }
      }
      known_mask |= 0xFFu << shift;
      Sync::sync();
    }
    const uint32_t thr = s_prefix;
    const int keep_ties = s_remaining;      // among keys equal to thr, the lowest node ids win

    // ---- selection flags in node-id order; each thread owns a contiguous chunk of ids
    const int chunk = (N + THREADS - 1) / THREADS;
    const int lo = min(N, tid * chunk), hi = min(N, lo + chunk);
    int n_eq = 0;
    for (int i = lo; i < hi; ++i) n_eq += (key(i) == thr);
    int tot_unused;
    int eq_before = block_exclusive_scan<THREADS, Sync>(n_eq, warp_tot, &tot_unused, tid);
    int n_sel = 0;
    for (int i = lo; i < hi; ++i) {
      const uint32_t q = key(i);
      bool sel = false;
      if (m_eff > 0) {
        if (q > thr) sel = true;
        else if (q == thr) sel = (eq_before++ < keep_ties);
      }
      slot_of[i + 1] = sel ? 1 : 0;
      n_sel += sel;
    }
    int sel_before = block_exclusive_scan<THREADS, Sync>(n_sel, warp_tot, &n_selected, tid);
    for (int i = lo; i < hi; ++i) {
      const bool sel = slot_of[i + 1] != 0;
      slot_of[i + 1] = sel ? (short)(1 + sel_before) : (short)-1;
      sel_before += sel;
    }
    if (tid == 0) slot_of[0] = 0;
    Sync::sync();

  }

  // ---- emit rows: the root, then the kept nodes in ascending node id
  const int n_out = 1 + n_selected;
  const size_t ob = (size_t)b * T;
  for (int id = tid; id <= N; id += THREADS) {
    const int slot = slot_of[id];
    if (slot < 0 || slot >= T) continue;
    const int dep = node_depth(id, k);
    const int par = (id == 0) ? -1 : slot_of[tparent[id]];
    out_parent[slot] = par;
    io.out.token[ob + slot] = ttoken[id];
    io.out.parent[ob + slot] = par;
    io.out.depth[ob + slot] = dep;
    io.out.position[ob + slot] = p.root_pos[b] + dep;
    io.out.cum[ob + slot] = cum[id];
    if (io.trace.node_id) io.trace.node_id[ob + slot] = id;
  }
  for (int slot = n_out + tid; slot < T; slot += THREADS) {
    io.out.token[ob + slot] = -1;
    io.out.parent[ob + slot] = -1;
    io.out.depth[ob + slot] = -1;
    io.out.position[ob + slot] = -1;
    io.out.cum[ob + slot] = 0.f;
    if (io.trace.node_id) io.trace.node_id[ob + slot] = -1;
  }
  if (tid == 0) {
    io.out.n_out[b] = n_out;
    io.out.stop_depth[b] = D;
    if (last) *io.out.status = *reinterpret_cast<volatile int*>(p.dev_status);
  }
  Sync::sync();

  // ---- ancestor mask: row i has bit j set iff j is i or an ancestor of i
  for (int slot = tid; slot < T; slot += THREADS) {
    uint32_t* row = io.out.mask + (ob + slot) * p.W32;
    for (int w = 0; w < p.W32; ++w) {
      uint32_t bits = 0u;
      if (slot < n_out) {
        int a = slot;
        for (int guard = 0; a >= 0 && guard <= DDD_MAX_DEPTH; ++guard) {
          if ((a >> 5) == w) bits |= 1u << (a & 31);
          a = out_parent[a];
        }
      }
      row[w] = bits;
    }
  }
  // copy the generated tree for replay, if asked for
  if (io.trace.tree_token) {
    for (int id = tid; id < p.Nn; id += THREADS) {
      const bool gen = id <= N;
      const size_t o = (size_t)b * p.Nn + id;
      io.trace.tree_token[o] = gen ? ttoken[id] : -1;
      if (io.trace.tree_parent) io.trace.tree_parent[o] = gen ? tparent[id] : -1;
      if (io.trace.tree_cum) io.trace.tree_cum[o] = gen ? cum[id] : 0.f;
    }
  }
}

// The same for a whole thread block with its own static scratch (the kernels that end a sequence's
// last pass, and rerank_kernel).
template <int THREADS, bool KEYS_IN_SMEM>
__device__ void rerank_mask_block(const Params& p, const DraftIO& io, const int b, const int D, const bool last,
                                  unsigned char* smem_raw) {
  __shared__ int scratch[kRerankScratchInts];
  __shared__ short out_parent[DDD_MAX_TOTAL + 1];
  rerank_mask_impl<THREADS, KEYS_IN_SMEM, BlockSync>(p, io, b, D, last, (int)threadIdx.x, smem_raw, p.Nn, scratch,
                                                     out_parent);
}


}  // namespace ddd
