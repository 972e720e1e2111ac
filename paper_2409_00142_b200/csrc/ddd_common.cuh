// Shared device-side definitions of the draft-tree kernels: the parameter block, the
// order-preserving 64-bit (score, index) keys used by every top-k, and the per-row
// tile update (online max / sum-exp and running top-k) used by both LM-head kernels.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ddd.h"

namespace ddd {

constexpr int kMaxLmCtas = 512;   // upper bound on LM-head thread blocks (sizes the partial buffers)
constexpr int kTile = 128;        // vocab rows handled per epilogue tile
constexpr unsigned kFullMask = 0xFFFFFFFFu;

// Everything a kernel needs that does not change between drafts.
struct Params {
  int B, Hd, V, k, n, m, dtype;
  int Vl, v0;         // rows of W this handle streams and the token id of its first row (V, 0 unless
                      // the handle owns a slice of a vocabulary-parallel LM head)
  int R;              // B * k beam rows
  int Nn;             // node slots per sequence: 1 + k + (n-1) k^2
  int T, W32;         // output rows per sequence (m + 1) and mask words per row
  float x;            // threshold
  uint32_t check_mask;
  float s, eps, plant_delta;
  const void* W;
  const void* E;
  const float* bias;
  const int* plant_next;
  void* hbuf[2];                  // [R][Hd] hidden rows, double-buffered by pass parity
  unsigned long long* part_key;   // [lm_ctas][R][k] per-block top-k keys, descending, 0 = empty
  float2* part_ms;                // [lm_ctas][R]    per-block (max, sum exp(z - max))
  int lm_ctas;
  int* tree_token;                // [B][Nn]
  int* tree_parent;               // [B][Nn] node id
  float* tree_cum;                // [B][Nn]
  int* beam_node;                 // [B][k]
  int* beam_tok;                  // [B][k]
  float* beam_cum;                // [B][k]
  int* row_plant;                 // [R] planted column of each beam row, -1 = none
  int* active;                    // [B]
  int* n_active;                  // [1]
  int* stop_depth;                // [B]
  int* root_pos;                  // [B] copy of the caller's root positions
  int* dev_status;                // [1] first error recorded by a kernel during this draft
  int* lm_ticket;                 // [1] arrival counter of the tensor-core LM-head blocks
};

// Per-draft pointers (caller-owned device memory).
struct DraftIO {
  ddd_output out;
  ddd_trace trace;
};

// ---------------------------------------------------------------------------- keys
// Maps a float to a uint32 whose unsigned order equals the float order (-inf lowest).
__device__ __forceinline__ uint32_t float_to_ordered(float f) {
  uint32_t u = __float_as_uint(f + 0.0f);   // +0.0f turns -0 into +0
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float ordered_to_float(uint32_t o) {
  uint32_t u = (o & 0x80000000u) ? (o & 0x7FFFFFFFu) : ~o;
  return __uint_as_float(u);
}
// Larger key <=> larger value, ties broken towards the smaller index.  Key 0 means "empty".
__device__ __forceinline__ unsigned long long make_key(float v, uint32_t idx) {
  return ((unsigned long long)float_to_ordered(v) << 32) | (unsigned long long)(0xFFFFFFFFu - idx);
}
__device__ __forceinline__ float key_value(unsigned long long key) {
  return ordered_to_float((uint32_t)(key >> 32));
}
__device__ __forceinline__ uint32_t key_index(unsigned long long key) {
  return 0xFFFFFFFFu - (uint32_t)key;
}

// Maximum of one 64-bit key per lane over the warp (two 32-bit redux steps).
__device__ __forceinline__ unsigned long long warp_max_key(unsigned long long key) {
  const uint32_t hi = (uint32_t)(key >> 32);
  const uint32_t mhi = __reduce_max_sync(kFullMask, hi);
  const uint32_t lo = (hi == mhi) ? (uint32_t)key : 0u;
  const uint32_t mlo = __reduce_max_sync(kFullMask, lo);
  return ((unsigned long long)mhi << 32) | mlo;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFullMask, v, o);
  return v;
}

// Programmatic dependent launch: a kernel launched with the attribute below may start while
// its predecessor in the stream is still running; griddep_wait() blocks until that predecessor
// has completed and its writes are visible, griddep_launch_dependents() lets the successor
// start.  Both are no-ops for kernels launched the ordinary way.
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

__device__ __forceinline__ float neg_inf() { return __uint_as_float(0xFF800000u); }

// Is beam row r part of pass d?  Pass 1 has one row per sequence (the root, slot 0).
__device__ __forceinline__ bool row_live(const Params& p, int r, int d, int force_all) {
  if (force_all) return true;
  const int b = r / p.k, i = r - b * p.k;
  return p.active[b] != 0 && (d > 1 || i == 0);
}

// ---------------------------------------------------------------------------- per-row tile update
// One warp folds kTile logits of one beam row (tokens tok0 .. tok0 + kTile - 1, -inf where
// the column does not exist or is excluded) into that row's running state:
//   (m, s)    online max and sum exp(z - m), identical in all lanes
//   list_key  lane j < k holds the j-th best (logit, token) key seen so far, 0 = empty
// Tiles must be fed in ascending token order: on equal logits an entry already in the list
// (lower token) beats any entry of the new tile, and inside the tile lane / slot order is
// token order, so ties resolve to the lower token with 32-bit compares only.
__device__ __forceinline__ void row_tile_update(const float* zrow, int tok0, int k, float& m, float& s,
                                                unsigned long long& list_key) {
  const int lane = threadIdx.x & 31;
  const float4 z4 = *reinterpret_cast<const float4*>(zrow + 4 * lane);
  const float z[4] = {z4.x, z4.y, z4.z, z4.w};
  const float lm = fmaxf(fmaxf(z[0], z[1]), fmaxf(z[2], z[3]));
  const float mt = ordered_to_float(__reduce_max_sync(kFullMask, float_to_ordered(lm)));
  if (mt == neg_inf()) return;   // nothing valid in this tile (uniform across the warp)

  float ls = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) ls += __expf(z[i] - mt);
  const float st = warp_sum(ls);
  if (mt > m) {
    s = s * __expf(m - mt) + st;
    m = mt;
  } else {
    s += st * __expf(mt - m);
  }

  // ordered 32-bit scores; 0 marks "no entry" (a real score is never 0: even -inf maps above it)
  uint32_t o[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) o[i] = (z[i] == neg_inf()) ? 0u : float_to_ordered(z[i]);
  uint32_t carry_o = (uint32_t)(list_key >> 32);
  uint32_t carry_tok = key_index(list_key);
  // Nothing to do unless some entry beats the current k-th best (0 while the list is not full).
  const uint32_t kth = __shfl_sync(kFullMask, carry_o, k - 1);
  const uint32_t tile_best = max(max(o[0], o[1]), max(o[2], o[3]));
  if (!__any_sync(kFullMask, tile_best > kth)) return;

  // Insert the tile's entries that beat the k-th best, best first.  An entry goes behind every
  // list entry with a score at least as high (the older, lower token wins ties) and pushes the
  // rest down one lane; the loop ends when the best entry left in the tile no longer beats the
  // k-th best, after at most k insertions.
  uint32_t kth_now = kth;
  for (int j = 0; j < k; ++j) {
    const uint32_t best = max(max(o[0], o[1]), max(o[2], o[3]));
    const uint32_t top = __reduce_max_sync(kFullMask, best);
    if (top <= kth_now) break;                  // uniform; top > 0 here
    const unsigned in_tile = __ballot_sync(kFullMask, best == top);
    const int src = __ffs(in_tile) - 1;         // lowest lane, then lowest slot: the lowest token
    int slot = 3;
    if (o[2] == top) slot = 2;
    if (o[1] == top) slot = 1;
    if (o[0] == top) slot = 0;
    const uint32_t win_tok = __shfl_sync(kFullMask, (uint32_t)(tok0 + 4 * lane + slot), src);
    if (lane == src) {
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (i == slot) o[i] = 0u;
    }
    const int ins = __popc(__ballot_sync(kFullMask, lane < k && carry_o >= top));
    const uint32_t up_o = __shfl_up_sync(kFullMask, carry_o, 1);
    const uint32_t up_tok = __shfl_up_sync(kFullMask, carry_tok, 1);
    if (lane == ins) { carry_o = top; carry_tok = win_tok; }
    else if (lane > ins) { carry_o = up_o; carry_tok = up_tok; }
    kth_now = __shfl_sync(kFullMask, carry_o, k - 1);
  }
  list_key = (lane < k && carry_o) ? (((unsigned long long)carry_o << 32) | (unsigned long long)(0xFFFFFFFFu - carry_tok))
                                   : 0ull;
}

// ---------------------------------------------------------------------------- wide lists (beam width 33..128)
// A warp holds a list of 128 keys, four per lane: element e sits in lane e / 4, register e % 4.
// Lists are kept sorted descending (position e = e-th best, 0 = empty at the end).  Everything a
// wide beam needs - a row's running top-k, the merge of the thread blocks' partial lists, the
// choice of the new beam among k sorted candidate rows - is built from two operations on such
// lists: sort 128 keys, and merge two sorted lists keeping the best 128.
constexpr int kWideK = 128;        // capacity of a wide list
constexpr int kNarrowK = 32;       // beams up to this width keep one key per lane

__device__ __forceinline__ unsigned long long shfl_xor_key(unsigned long long v, int mask) {
  return __shfl_xor_sync(kFullMask, v, mask);
}
// One compare-exchange step of a bitonic network at distance j (a power of two, 1..64) inside
// blocks of size k2 (descending where bit k2 of the element index is clear).
__device__ __forceinline__ void bitonic_step(unsigned long long (&v)[4], int j, int k2) {
  const int lane = threadIdx.x & 31;
  if (j >= 4) {
    const int lm = j >> 2;
    const bool lower = (lane & lm) == 0;
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      const unsigned long long o = shfl_xor_key(v[s], lm);
      const bool desc = ((4 * lane + s) & k2) == 0;
      const bool keep_max = lower == desc;
      v[s] = keep_max ? (v[s] > o ? v[s] : o) : (v[s] < o ? v[s] : o);
    }
  } else {
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      if ((s & j) == 0) {
        const int t = s | j;
        const bool desc = ((4 * lane + s) & k2) == 0;
        const unsigned long long a = v[s], b = v[t];
        const unsigned long long hi = a > b ? a : b, lo = a > b ? b : a;
        v[s] = desc ? hi : lo;
        v[t] = desc ? lo : hi;
      }
    }
  }
}
// Sorts the warp's 128 keys descending.
__device__ __forceinline__ void wide_sort(unsigned long long (&v)[4]) {
  for (int k2 = 2; k2 <= kWideK; k2 <<= 1)
    for (int j = k2 >> 1; j > 0; j >>= 1) bitonic_step(v, j, k2);
}
// a, b sorted descending -> a = the best 128 of both, sorted descending.
__device__ __forceinline__ void wide_merge(unsigned long long (&a)[4], const unsigned long long (&b)[4]) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int s = 0; s < 4; ++s) {
    // element e of the reversed b is element 127 - e: lane 31 - lane, register 3 - s
    const unsigned long long r = __shfl_sync(kFullMask, b[3 - s], 31 - lane);
    a[s] = a[s] > r ? a[s] : r;                 // bitonic: first rising part of one, falling part of the other
  }
  for (int j = kWideK >> 1; j > 0; j >>= 1) bitonic_step(a, j, kWideK);
}
// Element e of a wide list (uniform e): broadcast from its lane.
__device__ __forceinline__ unsigned long long wide_element(const unsigned long long (&v)[4], int e) {
  unsigned long long x = v[0];
  const int s = e & 3;
  if (s == 1) x = v[1];
  if (s == 2) x = v[2];
  if (s == 3) x = v[3];
  return __shfl_sync(kFullMask, x, e >> 2);
}
// Loads / stores the first `count` elements of a list laid out densely in memory (8-byte aligned).
__device__ __forceinline__ void wide_load(unsigned long long (&v)[4], const unsigned long long* src, int count) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int s = 0; s < 4; ++s) v[s] = (4 * lane + s < count) ? src[4 * lane + s] : 0ull;
}
__device__ __forceinline__ void wide_store(const unsigned long long (&v)[4], unsigned long long* dst, int count) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int s = 0; s < 4; ++s)
    if (4 * lane + s < count) dst[4 * lane + s] = v[s];
}

// The per-row tile update for wide beams: same contract as row_tile_update, with the row's list
// held as a wide list.  A tile's 128 logits arrive four per lane in token order, which is the
// list layout, so the tile is sorted as it stands and merged in.
__device__ __forceinline__ void row_tile_update_wide(const float* zrow, int tok0, int k, float& m, float& s,
                                                     unsigned long long (&list)[4]) {
  const int lane = threadIdx.x & 31;
  const float4 z4 = *reinterpret_cast<const float4*>(zrow + 4 * lane);
  const float z[4] = {z4.x, z4.y, z4.z, z4.w};
  const float lm = fmaxf(fmaxf(z[0], z[1]), fmaxf(z[2], z[3]));
  const float mt = ordered_to_float(__reduce_max_sync(kFullMask, float_to_ordered(lm)));
  if (mt == neg_inf()) return;
  float ls = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) ls += __expf(z[i] - mt);
  const float st = warp_sum(ls);
  if (mt > m) {
    s = s * __expf(m - mt) + st;
    m = mt;
  } else {
    s += st * __expf(mt - m);
  }
  unsigned long long t[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) t[i] = (z[i] == neg_inf()) ? 0ull : make_key(z[i], (uint32_t)(tok0 + 4 * lane + i));
  // nothing to do unless some entry beats the current k-th best (0 while the list is not full)
  const unsigned long long kth = wide_element(list, k - 1);
  const unsigned long long best = max(max(t[0], t[1]), max(t[2], t[3]));
  if (!__any_sync(kFullMask, best > kth)) return;
  wide_sort(t);
  wide_merge(list, t);
}

// ---------------------------------------------------------------------------- launchers (host)
// Lets a kernel use as much dynamic shared memory as the device allows.  The limit is a
// property of the function, shared by every handle of the process, so it is set to the
// maximum rather than to one handle's need (a later, smaller handle would otherwise lower it
// under an earlier one).
template <typename Kernel>
inline cudaError_t allow_max_dynamic_smem(Kernel kernel) {
  int dev = 0, optin = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  cudaFuncAttributes fa;
  if (e == cudaSuccess) e = cudaFuncGetAttributes(&fa, kernel);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, optin - (int)fa.sharedSizeBytes);
}

// Each returns the cudaError_t of its launch / attribute call.
cudaError_t prepare_simt(const Params& p);
cudaError_t prepare_tree(const Params& p);
cudaError_t launch_init(const Params& p, const DraftIO& io, const void* root_hidden, const int* root_token,
                        const int* root_pos, cudaStream_t st);
cudaError_t launch_lm_head_simt(const Params& p, int d, int force_all, int ctas, cudaStream_t st);
// pdl: launch with programmatic stream serialisation (the kernel may start before its
// predecessor has finished and synchronises with it through griddep_wait()).
// set_cond: a sequence that continues after pass d sets the graph conditional `cond` to 1.
cudaError_t launch_select(const Params& p, const DraftIO& io, int d, bool pdl, cudaGraphConditionalHandle cond,
                          bool set_cond, cudaStream_t st);

// Vocabulary-parallel pieces (shard.cu): fold this rank's per-block partials of pass d into one
// record per row, stored into slot `slot` of each of the n_dst record sets (flags raised beside
// them if given); wait for the flags of all slots.
cudaError_t launch_shard_reduce(const Params& p, int d, int slot, int slots, void* const* records,
                                int32_t* const* flags, int n_dst, int flag_value, int* done_counter, cudaStream_t st);
cudaError_t launch_shard_wait(const int* flags, int slots, int flag_value, int* dev_status, cudaStream_t st);

}  // namespace ddd
