// One persistent kernel per draft (launch mode DDD_LAUNCH_FUSED).
//
// Every pass of Algorithm 1 - LM head, log-softmax statistics, per-row top-k, merge, beam choice,
// Eq. 1 and the gate, draft step - runs inside ONE launch of one thread block per SM (all of them
// resident at once: checked at ddd_create; launched as a programmatic dependent of the kernel
// before it, see launch_draft_fused).  The blocks never leave between passes, so the two kernel boundaries per pass of the other launch
// modes become two grid-wide hand-overs through counters in global memory, and a draft that
// stops after d passes has launched nothing for the passes it does not run:
//
//   warp 0      producer: streams this block's vocabulary range of the packed W through the
//               shared-memory ring, pass after pass without a break; the W of the next pass goes
//               into the ring while the tree work of this pass is still going on, only the hidden
//               rows wait for it
//   warp 1      issues tcgen05.mma into two tensor-memory accumulators
//   warps 2-17  epilogue of every tile (scale, bias, online max / sum-exp, running top-k), then
//               the tree work of the pass
//
// Tree work of pass d.  Once every block has published its partials (hand-over 1), the new beam
// row i of sequence b belongs to block (b k + i) mod G.  Each of those blocks merges the partial
// lists of the sequence's rows and picks the new beam by itself - the same inputs give the same
// result everywhere, which saves a hand-over - and then runs the draft step of its own row: 512
// threads, one 16-byte chunk each, fp64, one rounding.  The block of row 0 also keeps the books
// (tree nodes, beam state, trace, stop).  Blocks without a row go straight to hand-over 2, after
// which the producers fetch the new hidden rows and the next pass runs.  The beam state is kept
// twice, by pass parity: a block may still read the old beam while the book-keeper writes the new.
// After the last pass the blocks that kept a sequence's books rerank its tree and write the rows
// and the mask (in the epilogue's transpose buffer; a tree too large for it goes to rerank_kernel).
//
// With many beam rows (48 or more, two tiles per block) the instantiation <true> feeds both tiles
// of a block from one fetch of the hidden rows and replaces the per-tile top-k of the epilogue by a
// floor per row that the blocks agree on (floor_epilogue below).
//
// Every wait is bounded.  A wait that runs out records DDD_ERR_TIMEOUT, raises a grid-wide abort
// word that ends every other wait, and each block drains its copies, frees its tensor memory and
// returns; the last block out resets the counters.
#include "draft_fused.cuh"
#include "tc_ptx.cuh"
#include "tree_device.cuh"

namespace ddd {

namespace {

using namespace tc;

constexpr int kTreeOverZt = kChunkCols * kTile * 4;     // smallest transpose buffer of the epilogue (8 KB)
constexpr int kMaxStoppedPerBlock = 8;                  // sequences one block may keep the books of
constexpr int kL2AheadKBlocks = 16;                     // K-blocks of W requested into L2 ahead of a pass

struct TreeSmem {
  int cand, lse, sel_flat, sel_tok, sel_cum, red, misc, total;
};
__host__ __device__ inline TreeSmem tree_smem(int k) {
  TreeSmem t;
  int off = 0;
  t.cand = off; off += k * k * 8;            // candidate records of one sequence
  t.lse = off; off += kNarrowK * 4;
  t.sel_flat = off; off += kNarrowK * 4;
  t.sel_tok = off; off += kNarrowK * 4;
  t.sel_cum = off; off += kNarrowK * 4;
  off = (off + 7) / 8 * 8;
  t.red = off; off += 64 * 8;                // partial sums of squares of one row
  t.misc = off; off += 16;                   // stop flag, H
  t.total = off;
  return t;
}

// One arrival of this block at a hand-over: the caller has synchronised the threads whose writes
// the other blocks are to see.
__device__ __forceinline__ void grid_arrive(int* counter) {
  asm volatile("fence.proxy.async;" ::: "memory");     // the hidden rows are read by tensor copies elsewhere
  __threadfence();
  atomicAdd(counter, 1);
}

// Merge of one beam row's partial lists by one warp.  The warp is alone on the critical path, so
// what counts is the number of dependent instructions and of loads of lines that another SM has
// just written (those cost about three times an ordinary L2 hit).  Hence the layout: this path
// keeps its partials position-major, fkey [R][k][kFusedMaxCtas] and fms [R][kFusedMaxCtas], so that
// the heads of all blocks' lists are one contiguous run, the second entries the next, and a lane
// fetches the first two entries of the lists of blocks lane, lane + 32, ... with coalesced loads
// in a single round trip.  A round of the k-way merge is then a lane-local maximum, one 32-bit
// warp maximum and a ballot, with no load in it; only a list that gives more than two entries
// to the result is read again (two more entries per round trip).  Scores are compared as
// order-preserving 32-bit integers; equal scores resolve to the lower block, which holds the
// lower tokens, and inside a list equal scores already stand in ascending token order.
// Lane j returns the j-th best key; (M, S) = the row's merged max and sum-exp, in all lanes.
constexpr int kFusedMaxCtas = 160;     // partial lists per row: five per lane
constexpr uint32_t kNotLoaded = 0xFFFFFFFFu;
constexpr int kFloorQueue = 512;       // entries a block can pick up above the rows' floors in one pass
// scratch of the floor epilogue: [6][n_pad] floats, then the queue (8-byte keys, 2-byte rows)
__host__ __device__ inline int floor_queue_offset(int n_pad) { return (6 * n_pad * 4 + 7) / 8 * 8; }
__host__ __device__ inline int floor_scratch_bytes(int n_pad) { return floor_queue_offset(n_pad) + kFloorQueue * 10; }

__device__ __forceinline__ unsigned long long merge_row_soa(const unsigned long long* __restrict__ keys,
                                                            const float2* __restrict__ msrow, int nc, int k,
                                                            float& M, float& S) {
  const int lane = threadIdx.x & 31;
  constexpr int NL = kFusedMaxCtas / 32;
  uint32_t s0[NL], s1[NL], t0[NL], t1[NL];
  int used[NL];
  float2 ms[NL];
#pragma unroll
  for (int q = 0; q < NL; ++q) {
    const int c = lane + 32 * q;
    unsigned long long k0 = 0ull, k1 = 0ull;
    ms[q] = make_float2(neg_inf(), 0.f);
    if (c < nc) {
      k0 = __ldcg(keys + c);
      if (k > 1) k1 = __ldcg(keys + kFusedMaxCtas + c);
      ms[q] = __ldcg(msrow + c);
    }
    s0[q] = (uint32_t)(k0 >> 32); t0[q] = key_index(k0);
    s1[q] = (uint32_t)(k1 >> 32); t1[q] = key_index(k1);
    used[q] = 0;
  }
  M = neg_inf();
#pragma unroll
  for (int q = 0; q < NL; ++q) M = fmaxf(M, ms[q].x);
  M = ordered_to_float(__reduce_max_sync(kFullMask, float_to_ordered(M)));
  S = 0.f;
#pragma unroll
  for (int q = 0; q < NL; ++q)
    if (ms[q].y > 0.f) S += ms[q].y * expf(ms[q].x - M);
  S = warp_sum(S);

  unsigned long long res = 0ull;
  for (int j = 0; j < k; ++j) {
    // a list whose two fetched entries are used up and which has more: fetch the next two
    bool need = false;
#pragma unroll
    for (int q = 0; q < NL; ++q) need |= s0[q] == kNotLoaded;
    if (__any_sync(kFullMask, need)) {
#pragma unroll
      for (int q = 0; q < NL; ++q) {
        if (s0[q] == kNotLoaded) {
          const int c = lane + 32 * q;
          const unsigned long long k0 = __ldcg(keys + (size_t)used[q] * kFusedMaxCtas + c);
          const unsigned long long k1 = used[q] + 1 < k ? __ldcg(keys + (size_t)(used[q] + 1) * kFusedMaxCtas + c) : 0ull;
          s0[q] = (uint32_t)(k0 >> 32); t0[q] = key_index(k0);
          s1[q] = (uint32_t)(k1 >> 32); t1[q] = key_index(k1);
        }
      }
    }
    uint32_t best = s0[0];
    int bq = 0;
#pragma unroll
    for (int q = 1; q < NL; ++q)
      if (s0[q] > best) { best = s0[q]; bq = q; }      // strictly greater: the lower block wins a tie
    const uint32_t top = __reduce_max_sync(kFullMask, best);
    if (top == 0u) break;                              // nothing left anywhere (uniform)
    const unsigned owners = __ballot_sync(kFullMask, best == top);
    int src = __ffs(owners) - 1;
    if (owners & (owners - 1u))                        // equal scores in several lanes: the lowest block
      src = (int)__reduce_min_sync(kFullMask, best == top ? (unsigned)(lane + 32 * bq) : 0x7FFFFFFFu) & 31;
    uint32_t tok = t0[0];
#pragma unroll
    for (int q = 1; q < NL; ++q)
      if (q == bq) tok = t0[q];
    tok = __shfl_sync(kFullMask, tok, src);
    if (lane == j) res = ((unsigned long long)top << 32) | (unsigned long long)(0xFFFFFFFFu - tok);
    if (lane == src) {
#pragma unroll
      for (int q = 0; q < NL; ++q) {
        if (q == bq) {
          ++used[q];
          s0[q] = s1[q];
          t0[q] = t1[q];
          s1[q] = used[q] + 1 < k ? kNotLoaded : 0u;
        }
      }
    }
  }
  return res;
}

struct EpiSync {      // the 16 epilogue warps on their named barrier
  __device__ static __forceinline__ void sync() { epilogue_barrier(); }
};

__device__ __forceinline__ void rerank_in_epilogue(const Params& p, const DraftIO& io, int b, int D, int et,
                                                bool keys_in_smem, unsigned char* rr, int cap, int* scratch,
                                                short* out_parent) {
  if (keys_in_smem) rerank_mask_impl<kEpiThreads, true, EpiSync>(p, io, b, D, false, et, rr, cap, scratch, out_parent);
  else rerank_mask_impl<kEpiThreads, false, EpiSync>(p, io, b, D, false, et, rr, cap, scratch, out_parent);
}

// ---------------------------------------------------------------------------- kernel
// MANY: the instantiation for many beam rows (fa.pair != 0: both tiles of a block per stage, the
// floor epilogue, a sequence's rows on its own blocks).  The other one is kept as it was measured
// before that mode existed: the serial section of a pass is a chain of single-warp steps, and
// the same source with one more branch in it has come out 1.5 us per pass slower on the 7B shape.
template <bool MANY>
__global__ void __launch_bounds__(kTcThreads, 1)
draft_fused_kernel(const Params p, const FusedArgs fa, const __grid_constant__ CUtensorMap map_h0,
                   const __grid_constant__ CUtensorMap map_h1) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_dyn) + 1023u) & ~static_cast<uintptr_t>(1023u));
  const int stages = fa.stages, ksub = fa.ksub, n_pad = fa.n_pad, cpg = fa.cpg;
  // pair mode: a block's two tiles share every stage, so the hidden rows cross from L2 once per pass
  // instead of once per tile (what bounds a pass with many beam rows is L2 -> SM traffic)
  const int pair = fa.pair;
  const bool use_floor = MANY && fa.floor;
  const SmemPlan sp = smem_plan(stages, ksub, n_pad, p.R, p.k, cpg, pair ? pair : 4);
  const TreeSmem ts = tree_smem(p.k);
  // The tree work's scratch lies over the epilogue's transpose buffer, which is idle between the
  // last tile of a pass and the first of the next (behind everything else where it is too large).
  unsigned char* tree_base = ts.total <= kTreeOverZt ? smem + sp.zt : smem + ((sp.total + 7) / 8 * 8);
  float* zt = reinterpret_cast<float*>(smem + sp.zt);
  unsigned long long* st_key = reinterpret_cast<unsigned long long*>(smem + sp.key);
  float2* st_ms = reinterpret_cast<float2*>(smem + sp.ms);
  int* s_plant = reinterpret_cast<int*>(smem + sp.plant);
  int* s_live = reinterpret_cast<int*>(smem + sp.live);
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem + sp.bars);
  uint32_t* tmem_ptr = reinterpret_cast<uint32_t*>(smem + sp.tmem_ptr);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + sp.abort_flag);
  unsigned long long* cand_s = reinterpret_cast<unsigned long long*>(tree_base + ts.cand);
  float* lse_s = reinterpret_cast<float*>(tree_base + ts.lse);
  int* sel_flat = reinterpret_cast<int*>(tree_base + ts.sel_flat);
  int* sel_tok = reinterpret_cast<int*>(tree_base + ts.sel_tok);
  float* sel_cum = reinterpret_cast<float*>(tree_base + ts.sel_cum);
  double* red_s = reinterpret_cast<double*>(tree_base + ts.red);
  volatile int* s_misc = reinterpret_cast<volatile int*>(tree_base + ts.misc);    // [0] stop, [1] H bits
  __shared__ int s_pass_state[2];      // what the producer learnt at hand-over 2: pass number to run, or 0 = leave
  __shared__ __align__(8) unsigned long long s_bar_spare;   // end of the MMAs when the block gives up
  __shared__ int s_stopped[kMaxStoppedPerBlock];            // sequences of this block's books that stopped in this pass
  __shared__ int s_nstopped;
  __shared__ int s_queue_n;                                 // entries in the queue of the floor epilogue

  const uint32_t a_base = smem_u32(smem + sp.a), b_base = smem_u32(smem + sp.b);
  const uint32_t b_bytes = (uint32_t)n_pad * kBlockK * 2;
  const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8u * stages;
  const uint32_t bar_tfull = bar_empty + 8u * stages, bar_tempty = bar_tfull + 16u;
  const uint32_t bar_pass = bar_tempty + 16u;      // the plan's fifth word: "the producer knows how the draft goes on"
  const uint32_t bar_spare = smem_u32(&s_bar_spare);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = (int)gridDim.x, bid = (int)blockIdx.x;
  const int k = p.k, R = p.R;
  int* const cnt_partials = fa.sync + 0;     // hand-over 1: partials of a pass published
  int* const cnt_hidden = fa.sync + 1;       // hand-over 2: state and hidden rows of the next pass written
  int* const abort_word = fa.sync + 2;
  int* const exit_ticket = fa.sync + 3;
  int* const cnt_floor = fa.sync + 4;        // floor hand-over: every block's row maxima are recorded

  // this block's contiguous range of 32-row units (fixed: block i always covers the same rows)
  const int n_units = (p.Vl + kUnitRows - 1) / kUnitRows;
  const int base_units = n_units / G, rem_units = n_units % G;
  const int my_units = base_units + (bid < rem_units ? 1 : 0);
  const int unit0 = bid * base_units + (bid < rem_units ? bid : rem_units);
  const int n_tiles = (my_units + 3) / 4;
  const int num_kb = p.Hd / (kBlockK * ksub);
  const uint32_t a_kblock = (uint32_t)(pair ? pair : 4) * kUnitBytes;     // bytes of W per K-block of a stage
  const uint32_t a_stage = (uint32_t)ksub * a_kblock, b_stage = (uint32_t)ksub * b_bytes;
  const int total_iters = pair ? num_kb : n_tiles * num_kb;         // pipeline steps per pass
  const int prefill = total_iters < stages ? total_iters : stages;

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(bar_full + 8u * s, 1);
      mbar_init(bar_empty + 8u * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_tfull + 8u * a, 1);
      mbar_init(bar_tempty + 8u * a, 4);
    }
    mbar_init(bar_pass, 1);
    mbar_init(bar_spare, 1);
    *abort_flag = 0;
    s_pass_state[0] = s_pass_state[1] = 0;
    s_nstopped = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_ptr)), "r"((uint32_t)fa.tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // Nothing above touches what the kernel before this one in the stream may still be using, so a
  // draft launched as a programmatic dependent sets itself up on every SM the previous draft has
  // left (all but the one that still picks the beam and reranks) and waits here for its end.
  griddep_launch_dependents();
  griddep_wait();
  // ---- start of a draft: per-sequence state and the root rows (version 0 of the beam state)
  for (int b = bid; b < p.B; b += G) {
    const uint4* src = reinterpret_cast<const uint4*>(static_cast<const unsigned char*>(fa.root_hidden) +
                                                      (size_t)b * p.Hd * 2);
    uint4* dst = reinterpret_cast<uint4*>(static_cast<unsigned char*>(p.hbuf[0]) + (size_t)b * k * p.Hd * 2);
    for (int j = threadIdx.x; j < p.Hd / 8; j += kTcThreads) dst[j] = src[j];
    if (threadIdx.x == 0) {
      const int tok = fa.root_token[b];
      p.tree_token[(size_t)b * p.Nn] = tok;
      p.tree_parent[(size_t)b * p.Nn] = -1;
      p.tree_cum[(size_t)b * p.Nn] = 0.f;
      fa.beam_node[b * k] = 0;
      fa.beam_cum[b * k] = 0.f;
      fa.row_plant[b * k] = (p.plant_next && tok >= 0 && tok < p.V) ? p.plant_next[tok] : -1;
      p.active[b] = 1;
      p.stop_depth[b] = 0;
      p.root_pos[b] = fa.root_pos[b];
    }
  }
  if (bid == 0 && threadIdx.x == 0) {
    *p.n_active = p.B;
    *p.dev_status = DDD_OK;
  }
  if (use_floor && threadIdx.x < kNarrowK)      // group maxima of the rows this block looks after: none yet
    for (int r = bid; r < R; r += G) fa.gmax[r * kNarrowK + threadIdx.x] = 0u;
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_ptr;
  if (threadIdx.x == 0) grid_arrive(cnt_hidden);     // instance 0 of hand-over 2

  if (warp == 0) {
    // ======================================================================= producer
    unsigned long long evict_first = 0ull;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(evict_first));
    uint32_t itg = 0;                // pipeline steps issued since the start of the draft
    bool ok = true;
    auto issue_w = [&](int i, int stage) {
      // step i of a pass: tile t, K-group kb - or, in pair mode, K-group i of all the block's units
      const int t = pair ? 0 : i / num_kb, kb = pair ? i : i - t * num_kb;
      const int nu = pair ? my_units : min(4, my_units - 4 * t);
      const uint32_t full = bar_full + 8u * stage;
      if (lane == 0) mbar_expect_tx(full, (uint32_t)ksub * ((uint32_t)nu * kUnitBytes + b_bytes));
      __syncwarp();
      const unsigned char* src = fa.w_packed + ((size_t)(kb * ksub) * n_units + (size_t)(unit0 + 4 * t)) * kUnitBytes;
      const uint32_t dst = a_base + (uint32_t)stage * a_stage;
      if (lane < ksub)
        bulk_load_hint(dst + (uint32_t)lane * a_kblock, src + (size_t)lane * n_units * kUnitBytes,
                       (uint32_t)nu * kUnitBytes, full, evict_first);
    };
    auto issue_h = [&](const CUtensorMap* map, int i, int stage) {
      if (lane == ksub)
        tma_load_3d(b_base + (uint32_t)stage * b_stage, map, bar_full + 8u * stage, 0, 0, (i % num_kb) * ksub);
    };
    auto wait_stage_free = [&](uint32_t it) -> bool {
      const uint32_t fill = it / (uint32_t)stages;
      if (fill == 0) return true;
      return __all_sync(kFullMask, mbar_wait(bar_empty + 8u * (it % stages), (fill - 1u) & 1u, abort_flag, p.dev_status));
    };
    for (int d = 1; d <= p.n; ++d) {
      const CUtensorMap* map = ((d - 1) & 1) ? &map_h1 : &map_h0;
      const uint32_t it0 = itg;
      // W of the first steps of this pass: it depends on nothing, so it is fetched while the tree
      // work of the previous pass is still going on elsewhere
      int issued_w = 0;
      for (; issued_w < prefill && ok; ++issued_w) {
        ok = wait_stage_free(itg);
        if (!ok) break;
        issue_w(issued_w, (int)(itg % stages));
        ++itg;
      }
      // HBM is nearly idle while the tree work of the previous pass goes on: ask L2 for the K-blocks
      // of the first tile that follow the ring.  Measured on the 7B shape: 16 K-blocks (256 KB per
      // block, 38 MB in all) take 0.9 us off a pass, 24 already lose again (the burst delays the
      // loads of the tree work), and pass 1 has no tree work to hide behind.
      if (ok && d > 1) {
        const int nu0 = pair ? my_units : min(4, my_units);
        const int kb_first = prefill * ksub;
        const int kb_last = min(p.Hd / kBlockK, kb_first + kL2AheadKBlocks);
        for (int kb64 = kb_first + lane; kb64 < kb_last; kb64 += 32)
          l2_prefetch(fa.w_packed + ((size_t)kb64 * n_units + (size_t)unit0) * kUnitBytes, (uint32_t)nu0 * kUnitBytes);
      }
      // hand-over 2 of the previous pass: hidden rows and state of this pass are in place
      int go = 0;
      if (ok) {
        if (lane == 0) {
          go = grid_wait(cnt_hidden, d * G, abort_word, p.dev_status) ? 1 : -1;
          if (go == 1 && d > 1 && *reinterpret_cast<volatile const int*>(p.n_active) == 0) go = 0;
        }
        go = __shfl_sync(kFullMask, go, 0);
      } else {
        go = -1;
      }
      if (lane == 0) {
        if (go < 0) *abort_flag = 1;
        s_pass_state[(d - 1) & 1] = go == 1 ? d : 0;
        mbar_arrive(bar_pass);                       // tells the other warps of the block
      }
      __syncwarp();
      asm volatile("fence.proxy.async;" ::: "memory");
      // the hidden rows of the steps already holding W (on a stop they are fetched all the same:
      // a stage's barrier only completes, and its copies only end, once both parts have landed)
      for (int i = 0; i < issued_w; ++i) issue_h(map, i, (int)((it0 + i) % stages));
      __syncwarp();
      if (go != 1) {
        for (int i = 0; i < issued_w; ++i) {
          const uint32_t it = it0 + i;
          mbar_wait(bar_full + 8u * (it % stages), (it / stages) & 1u, abort_flag, p.dev_status, false);
        }
        __syncwarp();
        break;
      }
      for (int i = prefill; i < total_iters; ++i) {
        ok = wait_stage_free(itg);
        if (!ok) break;
        issue_w(i, (int)(itg % stages));
        issue_h(map, i, (int)(itg % stages));
        __syncwarp();
        ++itg;
      }
      if (!ok) {
        // gave up in mid-pass: wait (bounded) until every copy already issued has landed
        for (uint32_t it = (itg > (uint32_t)stages ? itg - stages : 0u); it < itg; ++it)
          mbar_wait(bar_full + 8u * (it % stages), (it / stages) & 1u, abort_flag, p.dev_status, false);
        __syncwarp();
        break;
      }
    }
  } else if (warp == 1) {
    // ======================================================================= MMA issuer
    const uint32_t idesc = make_instr_desc(n_pad);
    uint32_t itg = 0, tg = 0;
    bool ok = true;
    for (int d = 1; d <= p.n && ok; ++d) {
      ok = __all_sync(kFullMask, mbar_wait(bar_pass, (uint32_t)(d - 1) & 1u, abort_flag, p.dev_status));
      if (!ok || s_pass_state[(d - 1) & 1] == 0) break;
      if (pair) {
        // both tiles at once: accumulator 0 takes units 0-3, accumulator 1 units 4-7, every stage feeds both
        for (int a2 = 0; a2 < 2 && ok; ++a2)
          ok = __all_sync(kFullMask, mbar_wait(bar_tempty + 8u * a2, (((tg + a2) >> 1) & 1u) ^ 1u, abort_flag, p.dev_status));
        if (!ok) break;
        tc_fence_after();
        for (int kb = 0; kb < num_kb; ++kb, ++itg) {
          const int stage = (int)(itg % stages);
          ok = __all_sync(kFullMask, mbar_wait(bar_full + 8u * stage, (itg / stages) & 1u, abort_flag, p.dev_status));
          if (!ok) break;
          tc_fence_after();
          if (lane == 0) {
            for (int kk = 0; kk < ksub; ++kk) {
              const uint32_t a_addr = a_base + (uint32_t)stage * a_stage + (uint32_t)kk * a_kblock;
              const uint32_t b_addr = b_base + (uint32_t)stage * b_stage + (uint32_t)kk * b_bytes;
#pragma unroll
              for (int k4 = 0; k4 < kBlockK / kUmmaK; ++k4) {
                const unsigned long long bd = make_smem_desc(b_addr + k4 * kUmmaK * 2);
                const uint32_t accum = (kb | kk | k4) != 0 ? 1u : 0u;
                tc_mma_bf16(tmem_base, make_smem_desc(a_addr + k4 * kUmmaK * 2), bd, idesc, accum);
                tc_mma_bf16(tmem_base + (uint32_t)n_pad, make_smem_desc(a_addr + kABytes + k4 * kUmmaK * 2), bd, idesc, accum);
              }
            }
            tc_commit(bar_empty + 8u * stage);
          }
          __syncwarp();
        }
        if (ok && lane == 0) {
          tc_commit(bar_tfull);
          tc_commit(bar_tfull + 8u);
        }
        __syncwarp();
        tg += 2;
        continue;
      }
      for (int t = 0; t < n_tiles && ok; ++t, ++tg) {
        const int acc = (int)(tg & 1u);
        ok = __all_sync(kFullMask, mbar_wait(bar_tempty + 8u * acc, ((tg >> 1) & 1u) ^ 1u, abort_flag, p.dev_status));
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * n_pad);
        for (int kb = 0; kb < num_kb; ++kb, ++itg) {
          const int stage = (int)(itg % stages);
          ok = __all_sync(kFullMask, mbar_wait(bar_full + 8u * stage, (itg / stages) & 1u, abort_flag, p.dev_status));
          if (!ok) break;
          tc_fence_after();
          if (lane == 0) {
            for (int kk = 0; kk < ksub; ++kk) {
              const uint32_t a_addr = a_base + (uint32_t)stage * a_stage + (uint32_t)kk * kABytes;
              const uint32_t b_addr = b_base + (uint32_t)stage * b_stage + (uint32_t)kk * b_bytes;
#pragma unroll
              for (int k4 = 0; k4 < kBlockK / kUmmaK; ++k4)
                tc_mma_bf16(d_tmem, make_smem_desc(a_addr + k4 * kUmmaK * 2), make_smem_desc(b_addr + k4 * kUmmaK * 2),
                            idesc, (kb | kk | k4) != 0 ? 1u : 0u);
            }
            tc_commit(bar_empty + 8u * stage);
          }
          __syncwarp();
        }
        if (ok && lane == 0) tc_commit(bar_tfull + 8u * acc);
        __syncwarp();
      }
    }
    if (!ok) {
      // make sure no MMA is still running before tensor memory is released
      if (lane == 0) tc_commit(bar_spare);
      __syncwarp();
      mbar_wait(bar_spare, 0u, abort_flag, p.dev_status, false);
      __syncwarp();
    }
  } else {
    // ======================================================================= epilogue, then tree work
    const int quarter = warp & 3;
    const int ew = warp - 2, et = (int)threadIdx.x - 64;
    const int lw = ew >> 2;
    const int n_chunks = (R + kChunkCols - 1) / kChunkCols;
    const int cpr = p.Hd / 8;                      // 16-byte chunks per hidden row
    const bool row_by_block = (cpr % 32 == 0) && (cpr / 32 <= 64);
    uint32_t tg = 0;
    bool ok = true;
    // The new beam rows this block looks after (merge, beam, gate, draft step), in ascending order,
    // -1 behind the last.  Up to one row per block they are dealt out cyclically.  With more rows than
    // blocks a block's rows should belong to one sequence, whose lists it then merges once: sequence
    // b gets blocks b * bps .. b * bps + bps - 1, row i < bps goes to block i of them, the others
    // are dealt out from the far end (row 0's block also keeps the sequence's books).
    const int bps = (MANY && R > G && p.B <= G) ? G / p.B : 0;
    auto owned_row = [&](const int j) -> int {
      if (bps == 0) {
        const int r = bid + j * G;
        return r < R ? r : -1;
      }
      const int b = bid / bps, q = bid - b * bps;
      if (b >= p.B) return -1;
      const int i = j == 0 ? q : 2 * bps - 1 - q + (j - 1) * bps;
      return i < k ? b * k + i : -1;
    };
    // The epilogue of a pass whose two accumulators (tile 0: units 0-3, tile 1: the rest) finish
    // together.  A logit below the k-th best of its row over the whole vocabulary is of no use
    // to anyone, and a floor under that k-th best is cheap: the blocks fall into k groups (block
    // mod k), every group records the largest logit any of its blocks holds for the row (one atomic
    // maximum per row and block), and the smallest of the k group maxima has k entries of k
    // different blocks at or above it.  Steps, each over the 2 x n_chunks chunks of 16 beam rows
    // dealt to the 16 warps (warp = one 32-lane quarter of tensor memory, every fourth chunk):
    //   1. the largest logit per row: warp maxima, then the block's over its 8 quarter-tiles;
    //      published with the atomic maximum, and the block arrives at the floor hand-over
    //   2. sum exp(z - block maximum) per row, under the other blocks' way to the hand-over
    //   3. wait for the hand-over (bounded), floor per row = minimum over the k groups
    //   4. logits at or above the floor go to a queue in shared memory, the rest is dropped
    //   5. the queue (tens of entries) is sorted into the rows' lists by counting
    // Returns 1: lists and (max, sum) of this pass are in st_key / st_ms; 0: the queue ran over
    // (a floor that says nothing, e.g. k groups of which one holds no valid entry): nothing is
    // lost, the accumulators are still there and the tile loop does the pass; -1: a wait ran out.
    unsigned char* const fl_base = smem + sp.zt;
    float* const fl_part = reinterpret_cast<float*>(fl_base);                       // [4][n_pad] per quarter of the 128 lanes
    float* const fl_max = fl_part + 4 * n_pad;                                      // [n_pad] block maximum
    float* const fl_floor = fl_max + n_pad;                                         // [n_pad] floor of the row
    unsigned long long* const fl_qkey = reinterpret_cast<unsigned long long*>(fl_base + floor_queue_offset(n_pad));
    short* const fl_qrow = reinterpret_cast<short*>(fl_qkey + kFloorQueue);
    auto floor_epilogue = [&](const int d) -> int {
      for (int a2 = 0; a2 < 2; ++a2)
        if (!epilogue_all(mbar_wait(bar_tfull + 8u * a2, (tg >> 1) & 1u, abort_flag, p.dev_status, false))) return -1;
      tc_fence_after();
      if (et == 0) s_queue_n = 0;
      // This thread's vocabulary row in either tile.  The work is instruction-bound (80 logits per
      // thread and step), so the common case - the warp's 32 rows all exist and no column is
      // planted - is one multiply-add per logit; anything else takes the checked form.
      const bool plants = p.plant_next != nullptr;
      int tok_t[2];
      float bias_t[2];
      bool valid_t[2], plain_t[2], none_t[2];
#pragma unroll
      for (int t = 0; t < 2; ++t) {
        const int rows = min(4, my_units - 4 * t) * kUnitRows;
        const int vrow = quarter * 32 + lane;
        const int v = (unit0 + 4 * t) * kUnitRows + vrow;
        valid_t[t] = vrow < rows && v < p.Vl;
        bias_t[t] = (valid_t[t] && p.bias) ? p.bias[v] : 0.f;
        tok_t[t] = v + p.v0;
        plain_t[t] = !plants && __all_sync(kFullMask, valid_t[t]);
        none_t[t] = !__any_sync(kFullMask, valid_t[t]);
      }
      // logits of 8 beam rows (columns c0 .. c0 + 7) of tile t, -inf where there is none; padded
      // columns hold whatever the zero rows behind the last beam row give and are never looked at
      auto load8 = [&](const int t, const int c0, float (&zv)[8]) {
        if (none_t[t]) {
#pragma unroll
          for (int c = 0; c < 8; ++c) zv[c] = neg_inf();
          return;
        }
        float accv[8];
        tc_load_8cols(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(t * n_pad + c0), accv);
        if (plain_t[t]) {
#pragma unroll
          for (int c = 0; c < 8; ++c) zv[c] = fmaf(accv[c], p.s, bias_t[t]);
        } else {
#pragma unroll
          for (int c = 0; c < 8; ++c)
            zv[c] = (valid_t[t] && s_plant[min(c0 + c, R - 1)] != tok_t[t]) ? fmaf(accv[c], p.s, bias_t[t]) : neg_inf();
        }
      };
      // One value per column over the warp's 32 lanes, 8 columns at once: the first three steps
      // halve the columns a lane still holds; lane l ends with column l / 4.
      auto fold8 = [&](float (&e)[8], auto op) -> float {
        float v4[4], v2[2];
        const bool b16 = lane & 16, b8 = lane & 8, b4 = lane & 4;
#pragma unroll
        for (int j = 0; j < 4; ++j) v4[j] = op(b16 ? e[j + 4] : e[j], __shfl_xor_sync(kFullMask, b16 ? e[j] : e[j + 4], 16));
#pragma unroll
        for (int j = 0; j < 2; ++j) v2[j] = op(b8 ? v4[j + 2] : v4[j], __shfl_xor_sync(kFullMask, b8 ? v4[j] : v4[j + 2], 8));
        float v1 = op(b4 ? v2[1] : v2[0], __shfl_xor_sync(kFullMask, b4 ? v2[0] : v2[1], 4));
        v1 = op(v1, __shfl_xor_sync(kFullMask, v1, 2));
        return op(v1, __shfl_xor_sync(kFullMask, v1, 1));
      };
      const int col = lane >> 2;
      const int n_eights = n_pad / 8;
      // ---- 1. maxima (both tiles hold the same beam rows: joined before the lanes are)
      for (int hc = lw; hc < n_eights; hc += 4) {
        const int c0 = hc * 8;
        float z0[8], z1[8];
        load8(0, c0, z0);
        load8(1, c0, z1);
#pragma unroll
        for (int c = 0; c < 8; ++c) z0[c] = fmaxf(z0[c], z1[c]);
        const float mx = fold8(z0, [](float x, float y) { return fmaxf(x, y); });
        if (!(lane & 3)) fl_part[quarter * n_pad + c0 + col] = mx;
      }
      epilogue_barrier();
      if (et < n_pad) {
        const float M = fmaxf(fmaxf(fl_part[et], fl_part[n_pad + et]), fmaxf(fl_part[2 * n_pad + et], fl_part[3 * n_pad + et]));
        const bool live = et < R && s_live[et];
        if (live && M != neg_inf()) atomicMax(fa.gmax + et * kNarrowK + bid % k, float_to_ordered(M));
        fl_max[et] = M == neg_inf() ? 0.f : M;         // reference of the exponentials; the row's maximum if it has one
        if (et < R) st_ms[et].x = M;
      }
      epilogue_barrier();
      if (et == 0) grid_arrive(cnt_floor);
      // ---- 2. sums, while the other blocks find their way to the hand-over
      for (int hc = lw; hc < n_eights; hc += 4) {
        const int c0 = hc * 8;
        float z0[8], z1[8];
        load8(0, c0, z0);
        load8(1, c0, z1);
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const float M = fl_max[c0 + c];
          z0[c] = __expf(z0[c] - M) + __expf(z1[c] - M);
        }
        const float sum = fold8(z0, [](float x, float y) { return x + y; });
        if (!(lane & 3)) fl_part[quarter * n_pad + c0 + col] = sum;
      }
      // ---- 3. the floor: the smallest of the k group maxima, one warp per row
      bool w_ok = true;
      if (et == 0) w_ok = grid_wait(cnt_floor, d * G, abort_word, p.dev_status);
      if (!epilogue_all(w_ok)) return -1;
      {
        uint32_t g[16];                                // n_pad <= 256: at most 16 rows per warp, all loads in flight at once
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int r = ew + j * kEpiWarps;
          g[j] = 0xFFFFFFFFu;
          if (r < R && lane < k && s_live[r]) g[j] = __ldcg(fa.gmax + r * kNarrowK + lane);
        }
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int r = ew + j * kEpiWarps;
          if (r >= n_pad) break;
          const uint32_t fl = __reduce_min_sync(kFullMask, g[j]);
          // rows that are not drafting, and padded columns, keep nothing; a group without any entry says nothing
          if (lane == 0)
            fl_floor[r] = fl == 0xFFFFFFFFu ? __int_as_float(0x7F800000) : (fl == 0u ? -3.4028234664e38f : ordered_to_float(fl));
        }
      }
      if (et < R) {
        const float S = (fl_part[et] + fl_part[n_pad + et]) + (fl_part[2 * n_pad + et] + fl_part[3 * n_pad + et]);
        st_ms[et].y = st_ms[et].x == neg_inf() ? 0.f : S;
      }
      epilogue_barrier();
      // ---- 4. what lies at or above the floor
      for (int hc = lw; hc < n_eights; hc += 4) {
        const int c0 = hc * 8;
        float z0[8], z1[8], fl[8];
        load8(0, c0, z0);
        load8(1, c0, z1);
        bool any = false;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          fl[c] = fl_floor[c0 + c];
          any |= z0[c] >= fl[c];
          any |= z1[c] >= fl[c];
        }
        if (any) {
#pragma unroll
          for (int c = 0; c < 8; ++c) {
#pragma unroll
            for (int t = 0; t < 2; ++t) {
              const float z = t ? z1[c] : z0[c];
              if (z >= fl[c]) {
                const int at = atomicAdd(&s_queue_n, 1);
                if (at < kFloorQueue) {
                  fl_qkey[at] = make_key(z, (uint32_t)tok_t[t]);
                  fl_qrow[at] = (short)(c0 + c);
                }
              }
            }
          }
        }
      }
      tc_fence_before();
      epilogue_barrier();
      const int n_q = s_queue_n;
      if (n_q > kFloorQueue) {
        // start over with the tile loop: its running state as at the start of the pass
        for (int r = et; r < R; r += kEpiThreads) st_ms[r] = make_float2(neg_inf(), 0.f);
        epilogue_barrier();
        return 0;
      }
      if (ew < 4 && lane == 0) {                      // both accumulators may be overwritten
        mbar_arrive(bar_tempty);
        mbar_arrive(bar_tempty + 8u);
      }
      // ---- 5. the lists: entry e goes to place (number of better entries of its row)
      for (int e = et; e < n_q; e += kEpiThreads) {
        const unsigned long long key = fl_qkey[e];
        const int r = fl_qrow[e];
        int place = 0;
        for (int o = 0; o < n_q; ++o) place += (fl_qrow[o] == r && fl_qkey[o] > key) ? 1 : 0;
        if (place < k) st_key[r * k + place] = key;
      }
      epilogue_barrier();
      return 1;
    };
    for (int d = 1; d <= p.n; ++d) {
      ok = epilogue_all(mbar_wait(bar_pass, (uint32_t)(d - 1) & 1u, abort_flag, p.dev_status, false));
      if (!ok || s_pass_state[(d - 1) & 1] == 0) break;
      const int par_in = (d - 1) & 1, par_out = d & 1;
      // ---- per-row flags and running state of this pass
      for (int r = et; r < R; r += kEpiThreads) {
        s_plant[r] = fa.row_plant[par_in * R + r];
        s_live[r] = row_live(p, r, d, 0) ? 1 : 0;
        st_ms[r] = make_float2(neg_inf(), 0.f);
      }
      for (int i = et; i < R * k; i += kEpiThreads) st_key[i] = 0ull;
      epilogue_barrier();
      // ---- many beam rows, both tiles fed together: nothing runs beside this epilogue, and a top-k
      // per row and tile would cost it 40 us.  So the blocks first agree on a floor per row below which
      // no logit can reach the row's k best anywhere (see floor_epilogue), then only pick up what
      // lies above it: a fraction of an entry per row and block.
      bool lists_done = false;
      if constexpr (MANY) {
        if (use_floor) {
          int state = floor_epilogue(d);
          if (state < 0) { ok = false; break; }
          lists_done = state == 1;
          if (lists_done) tg += 2;
        }
      }
      // ---- the tiles of this block's vocabulary range
      for (int t = 0; t < n_tiles && ok && !lists_done; ++t, ++tg) {
        const int acc = (int)(tg & 1u);
        const int rows = min(4, my_units - 4 * t) * kUnitRows;
        const int row0 = (unit0 + 4 * t) * kUnitRows;
        ok = epilogue_all(mbar_wait(bar_tfull + 8u * acc, (tg >> 1) & 1u, abort_flag, p.dev_status, false));
        if (!ok) break;
        tc_fence_after();
        const int vrow = quarter * 32 + lane;
        const int v = row0 + vrow;
        const bool v_ok = vrow < rows && v < p.Vl;
        const float bias = (v_ok && p.bias) ? p.bias[v] : 0.f;
        for (int g0 = 0; g0 < n_chunks; g0 += cpg) {
          const int ch = g0 + lw;
          if (lw < cpg && ch < n_chunks) {
            const int c0 = ch * kChunkCols;
            float accv[16];
            tc_load_16cols(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * n_pad + c0), accv);
#pragma unroll
            for (int c = 0; c < kChunkCols; ++c) {
              const int r = c0 + c;
              float z = neg_inf();
              if (v_ok && r < R && s_plant[r] != v + p.v0) z = fmaf(accv[c], p.s, bias);
              zt[(lw * kChunkCols + c) * kTile + vrow] = z;
            }
            tc_fence_before();
          }
          epilogue_barrier();
          if (g0 + cpg >= n_chunks && ew < 4 && lane == 0) mbar_arrive(bar_tempty + 8u * acc);
          for (int rr = ew; rr < cpg * kChunkCols; rr += kEpiWarps) {
            const int r = g0 * kChunkCols + rr;
            if (r >= R || !s_live[r]) continue;
            float2 ms = st_ms[r];
            unsigned long long key = lane < k ? st_key[r * k + lane] : 0ull;
            row_tile_update(zt + rr * kTile, row0 + p.v0, k, ms.x, ms.y, key);
            if (lane < k) st_key[r * k + lane] = key;
            if (lane == 0) st_ms[r] = ms;
          }
          epilogue_barrier();
        }
      }
      if (!ok) break;
      // ---- publish this block's partials: hand-over 1
      for (int r = ew; r < R; r += kEpiWarps) {
        if (!s_live[r]) continue;
        // a list is read up to its first empty entry: nothing behind that one needs to be written
        if (lane < k && (!MANY || lane == 0 || st_key[r * k + lane - 1] != 0ull))
          fa.fkey[((size_t)r * k + lane) * kFusedMaxCtas + bid] = st_key[r * k + lane];
        if (lane == 0) fa.fms[(size_t)r * kFusedMaxCtas + bid] = st_ms[r];
      }
      epilogue_barrier();
      if (et == 0) grid_arrive(cnt_partials);

      // ---- tree work: the new beam rows this block owns
      const int P = (d == 1) ? 1 : k;
      const int base = (d == 1) ? 1 : 1 + k + (d - 2) * k * k;
      // The books of sequence b after this pass: all P * k candidates become tree nodes, the new
      // beam state is written for the next pass (the other parity), a stop is recorded.  Called by
      // all epilogue threads of the block that owns the sequence's row 0; none of it is waited for
      // until the hand-over at the end of the pass.
      auto keep_books = [&](const int b) {
        // this block keeps the sequence's books
        for (int flat = et; flat < P * k; flat += kEpiThreads) {
          const unsigned long long rec = cand_s[flat];
          const size_t node = (size_t)b * p.Nn + base + flat;
          p.tree_token[node] = (int)(uint32_t)rec;
          p.tree_parent[node] = fa.beam_node[par_in * R + b * k + flat / k];
          p.tree_cum[node] = __uint_as_float((uint32_t)(rec >> 32));
        }
        if (et < k) {
          const int tok = sel_tok[et];
          fa.beam_node[par_out * R + b * k + et] = base + sel_flat[et];
          fa.beam_cum[par_out * R + b * k + et] = sel_cum[et];
          fa.row_plant[par_out * R + b * k + et] = (p.plant_next && tok >= 0 && tok < p.V) ? p.plant_next[tok] : -1;
          if (fa.io.trace.beam_sel) fa.io.trace.beam_sel[((size_t)b * p.n + (d - 1)) * k + et] = sel_flat[et];
        }
        if (et < P && fa.io.trace.row_lse) fa.io.trace.row_lse[((size_t)b * p.n + (d - 1)) * k + et] = lse_s[et];
        if (et == 0) {
          fa.io.out.H_trace[(size_t)b * p.n + (d - 1)] = __int_as_float(s_misc[1]);
          if (s_misc[0]) {
            p.stop_depth[b] = d;
            p.active[b] = 0;
            atomicSub(p.n_active, 1);
            if (s_nstopped < kMaxStoppedPerBlock) s_stopped[s_nstopped++] = b;
          }
        }
      };
      bool waited = false;
      int cur_b = -1;
      for (int own = 0, r_new = bid; (MANY ? (r_new = owned_row(own)) >= 0 : r_new < R) && ok; ++own, r_new += MANY ? 0 : G) {
        const int b = r_new / k, i = r_new - b * k;
        if (!s_live[b * k]) continue;                 // sequence not drafting in this pass
        if (d == p.n && i != 0) continue;             // after the last pass there is no draft step
        if (!waited) {
          bool w_ok = true;
          if (et == 0) w_ok = grid_wait(cnt_partials, d * G, abort_word, p.dev_status);
          ok = epilogue_all(w_ok);
          waited = true;
          if (!ok) break;
          // every block has published, so none reads this pass's group maxima any more: clear those
          // of this block's rows for the next pass (ordered before it by hand-over 2)
          if (use_floor && et < kNarrowK)
            for (int j = 0, r; (r = owned_row(j)) >= 0; ++j) fa.gmax[r * kNarrowK + et] = 0u;
        }
        if (b != cur_b) {
          cur_b = b;
          // merge the partial lists of the sequence's rows, one warp per row
          for (int pr = ew; pr < P; pr += kEpiWarps) {
            const int r = b * k + pr;
            float M, S;
            unsigned long long res = merge_row_soa(fa.fkey + (size_t)r * k * kFusedMaxCtas,
                                                   fa.fms + (size_t)r * kFusedMaxCtas, G, k, M, S);
            const int pc = s_plant[r];
            if (pc >= 0) {      // planted column: (max of the others) + delta; it was left out of the partials
              const float zc = M + p.plant_delta;
              const float M2 = fmaxf(M, zc);
              S = S * expf(M - M2) + expf(zc - M2);
              M = M2;
              const unsigned long long plant_key = make_key(zc, (uint32_t)pc);
              const int ins = __popc(__ballot_sync(kFullMask, lane < k && res > plant_key));
              const unsigned long long up = __shfl_up_sync(kFullMask, res, 1);
              if (lane == ins) res = plant_key;
              else if (lane > ins) res = up;
            }
            const float lse = M + logf(S);
            if (lane < k) {
              const float lp = (res != 0ull) ? fminf(key_value(res) - lse, 0.f) : neg_inf();
              const int tok = (res != 0ull) ? (int)key_index(res) : -1;
              const float cand = fa.beam_cum[par_in * R + r] + lp;
              cand_s[pr * k + lane] = ((unsigned long long)__float_as_uint(cand) << 32) | (uint32_t)tok;
            }
            if (lane == 0) lse_s[pr] = lse;
          }
          epilogue_barrier();
          // While one warp picks the beam, idle warps ask L2 for the embedding rows of this block's
          // share of the candidates (the k blocks of a sequence cover all k * k between them), so that
          // the draft step's gather finds them there: -1.2 us per pass on the 7B shape.
          if (ew >= 12 && d < p.n) {
            const int n_cand = P * k;
            for (int flat = i + k * ((ew - 12) * 32 + lane); flat < n_cand; flat += k * 128) {
              const int tokc = (int)(uint32_t)cand_s[flat];
              if (tokc >= 0 && tokc < p.V)
                l2_prefetch(static_cast<const unsigned char*>(p.E) + (size_t)tokc * p.Hd * 2, (uint32_t)p.Hd * 2);
            }
          }
          // the new beam, Eq. 1 and the gate
          if (ew == 0) {
            // The k candidates of a beam row are already in descending order (same parent score,
            // log-probabilities descending, ties by lower index), so lane p walks row p and the beam
            // is a k-way merge of the P <= 32 rows: one 32-bit warp maximum and a ballot per entry.
            // Equal scores go to the lower row, then the lower position: the lower candidate index.
            int pos = 0;
            int mine_flat = -1;
            for (int j = 0; j < k; ++j) {
              uint32_t hs = 0u;
              if (lane < P && pos < k) {
                const unsigned long long rec = cand_s[lane * k + pos];
                if ((int)(uint32_t)rec >= 0) hs = float_to_ordered(__uint_as_float((uint32_t)(rec >> 32)));
              }
              const uint32_t top = __reduce_max_sync(kFullMask, hs);
              if (top == 0u) break;
              const int src = __ffs(__ballot_sync(kFullMask, hs == top)) - 1;
              const int flat_j = src * k + __shfl_sync(kFullMask, pos, src);
              if (lane == j) mine_flat = flat_j;
              if (lane == src) ++pos;
            }
            const unsigned long long mine = mine_flat >= 0 ? 1ull : 0ull;
            const bool have = lane < k && mine != 0ull;
            const int flat = have ? mine_flat : 0;
            const float cum = have ? __uint_as_float((uint32_t)(cand_s[flat] >> 32)) : neg_inf();
            const float M = __shfl_sync(kFullMask, cum, 0);
            const float sum = warp_sum(have ? expf(cum - M) : 0.f);
            const float H = M + logf(sum);
            bool stop = (d == p.n);
            if (!stop && ((p.check_mask >> (d - 1)) & 1u)) stop = H < p.x;
            if (lane < k) {
              sel_flat[lane] = flat;
              sel_tok[lane] = (int)(uint32_t)cand_s[flat];
              sel_cum[lane] = cum;
            }
            if (lane == 0) {
              s_misc[0] = stop ? 1 : 0;
              s_misc[1] = __float_as_int(H);
            }
          }
          epilogue_barrier();
        }
        if (s_misc[0]) {                               // the sequence stops here: no draft step
          if (i == 0) keep_books(b);
          continue;
        }
        // ---- draft step of new beam row i: h = round(u / sqrt(mean(u^2) + eps)), u = h_parent + E[token]
        {
          // MANY: a block with a second row of the same sequence takes both at once, half of the
          // threads each: the step is a chain of round trips that 256 threads get through as fast as 512
          int i2 = -1;
          if constexpr (MANY) {
            const int r2 = owned_row(own + 1);
            if (r2 >= 0 && r2 / k == b && row_by_block && 2 * (cpr / 32) <= 64) {
              i2 = r2 - b * k;
              ++own;
            }
          }
          const int tpr = (MANY && i2 >= 0) ? kEpiThreads / 2 : kEpiThreads;       // threads per row
          const int second = (MANY && et >= tpr) ? 1 : 0;
          const int lt = MANY ? et - second * tpr : et;                            // this thread's index among its row's
          const int my_i = second ? i2 : i;
          const int tok = sel_tok[my_i];
          const uint4* hp = reinterpret_cast<const uint4*>(p.hbuf[par_in]) + (size_t)(b * k + sel_flat[my_i] / k) * cpr;
          const uint4* er = reinterpret_cast<const uint4*>(p.E) + (size_t)(tok >= 0 && tok < p.V ? tok : 0) * cpr;
          uint4* out = reinterpret_cast<uint4*>(p.hbuf[par_out]) + (size_t)(b * k + my_i) * cpr;
          if (row_by_block) {
            // chunk q belongs to thread q mod 512 (256); a warp's 32 chunks form one partial sum (slot q / 32)
            const int slots = cpr / 32;
            double* const red_row = MANY ? red_s + second * slots : red_s;
            uint4 hv0 = make_uint4(0, 0, 0, 0), ev0 = hv0;
            if (lt - lane < cpr) { hv0 = hp[lt]; ev0 = er[lt]; }     // in flight while the books are kept
            if (i == 0) keep_books(b);
            for (int q = lt; q - lane < cpr; q += tpr) {
              uint4 hv = hv0, ev = ev0;
              if (q != lt) { hv = hp[q]; ev = er[q]; }
              double u[8];
              Chunk<__nv_bfloat16>::sum(hv, ev, u);
              double ss = 0.0;
#pragma unroll
              for (int e = 0; e < 8; ++e) ss = fma(u[e], u[e], ss);
              ss = warp_sum_f64(ss);
              if (lane == 0) red_row[q / 32] = ss;
            }
            epilogue_barrier();
            double ss = 0.0;
            for (int j = 0; j < slots; ++j) ss += red_row[j];
            const double inv = 1.0 / sqrt(ss / (double)p.Hd + (double)p.eps);
            for (int q = lt; q < cpr; q += tpr) {
              uint4 hv = hv0, ev = ev0;
              if (q != lt) { hv = hp[q]; ev = er[q]; }
              double u[8];
              Chunk<__nv_bfloat16>::sum(hv, ev, u);
#pragma unroll
              for (int e = 0; e < 8; ++e) u[e] *= inv;
              out[q] = Chunk<__nv_bfloat16>::round(u);
            }
            epilogue_barrier();                          // red_s is reused by the block's next row
          } else {
            if (i == 0) keep_books(b);
            if (ew == 0) {
            // rows that are not a whole number of 32-chunk groups: one warp does the row
            double ss = 0.0;
            for (int c = lane; c < cpr; c += 32) {
              double u[8];
              Chunk<__nv_bfloat16>::sum(hp[c], er[c], u);
#pragma unroll
              for (int e = 0; e < 8; ++e) ss = fma(u[e], u[e], ss);
            }
            ss = warp_sum_f64(ss);
            const double inv = 1.0 / sqrt(ss / (double)p.Hd + (double)p.eps);
            for (int c = lane; c < cpr; c += 32) {
              double u[8];
              Chunk<__nv_bfloat16>::sum(hp[c], er[c], u);
#pragma unroll
              for (int e = 0; e < 8; ++e) u[e] *= inv;
              out[c] = Chunk<__nv_bfloat16>::round(u);
            }
            }
          }
        }
      }
      if (!ok) break;
      // ---- hand-over 2: this block's share of the next pass's state and hidden rows is written
      epilogue_barrier();
      if (et == 0) grid_arrive(cnt_hidden);
    }
    // ---- the sequences whose books this block kept are finished here, after the last pass, where
    // nobody waits for it: rerank to m nodes, rows, parents, positions, mask.  The transpose buffer
    // is free now and holds keys, rows and scratch.
    if (ok && fa.rerank_inside) {
      epilogue_barrier();
      const int cap = p.Nn;
      unsigned char* rr = smem + sp.zt;
      const size_t node_bytes = (size_t)cap * (fa.rerank_inside == 1 ? 6 : 2);
      int* scratch = reinterpret_cast<int*>(rr + ((node_bytes + 7) / 8) * 8);
      short* out_parent = reinterpret_cast<short*>(scratch + kRerankScratchInts);
      const int n_stopped = s_nstopped;
      for (int q = 0; q < n_stopped; ++q) {
        const int b = s_stopped[q];
        rerank_in_epilogue(p, fa.io, b, p.stop_depth[b], et, fa.rerank_inside == 1, rr, cap, scratch, out_parent);
        epilogue_barrier();
      }
    }
    if (!ok && et == 0) *abort_flag = 1;
  }

  // ---- teardown: everyone meets, the MMAs are known to have ended (every accumulator that was
  // committed has been read, or the block gave up after bounded waits), tensor memory is freed;
  // the last block out resets the hand-over counters for the next draft
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) {
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)fa.tmem_cols)
                 : "memory");
  }
  if (threadIdx.x == 0) {
    if (*abort_flag) atomicExch(abort_word, 1);
    __threadfence();
    if (atomicAdd(exit_ticket, 1) == G - 1) {
      if (fa.rerank_inside) *fa.io.out.status = *reinterpret_cast<volatile int*>(p.dev_status);
      atomicExch(cnt_partials, 0);
      atomicExch(cnt_hidden, 0);
      if (MANY) atomicExch(cnt_floor, 0);
      atomicExch(abort_word, 0);
      atomicExch(exit_ticket, 0);
      __threadfence();
    }
  }
}

// The rerank and the mask of every sequence, after the draft: one block per sequence.
__global__ void __launch_bounds__(1024) rerank_kernel(const Params p, const DraftIO io, const int keys_in_smem) {
  griddep_wait();
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int b = blockIdx.x;
  const int D = p.stop_depth[b];
  if (keys_in_smem) rerank_mask_block<1024, true>(p, io, b, D, b == 0, smem_raw);
  else rerank_mask_block<1024, false>(p, io, b, D, b == 0, smem_raw);
}

size_t rerank_kernel_smem(const Params& p, bool* keys_in_smem) {
  const size_t both = (size_t)p.Nn * (sizeof(uint32_t) + sizeof(short));
  *keys_in_smem = both <= 160 * 1024;
  return *keys_in_smem ? both : (size_t)p.Nn * sizeof(short);
}

}  // namespace

int fused_extra_smem(int k) {
  const int t = tree_smem(k).total;
  return t <= kTreeOverZt ? 0 : t + 8;
}

bool fused_supported(const Params& p) {
  return p.dtype == DDD_DTYPE_BF16 && p.Hd % kBlockK == 0 && p.k <= kNarrowK && p.lm_ctas <= kFusedMaxCtas;
}

int fused_stage_units(const Params& p, int sm_count) {
  const int n_units = (p.Vl + kUnitRows - 1) / kUnitRows;
  const int ctas = sm_count < n_units ? sm_count : n_units;
  const int lo = n_units / ctas, hi = lo + (n_units % ctas ? 1 : 0);
  const bool pair = p.R >= 48 && lo >= 5 && hi <= 8 && 2 * ((p.R + 15) / 16 * 16) <= 512;
  return pair ? hi : 4;
}

// Can the rerank run inside the draft kernel, in the epilogue's transpose buffer?  1: with the
// tree's keys in shared memory, 2: keys read from global memory, 0: no (rerank_kernel follows).
int fused_rerank_mode(const Params& p, const TcPlan& plan) {
  const size_t room = (size_t)plan.epi_chunks * kChunkCols * kTile * 4;
  const size_t fixed = 8 + kRerankScratchInts * sizeof(int) + (size_t)p.T * sizeof(short);
  if ((size_t)p.R > (size_t)kMaxStoppedPerBlock * plan.ctas) return 0;
  if ((size_t)p.Nn * 6 + fixed <= room) return 1;
  if ((size_t)p.Nn * 2 + fixed <= room) return 2;
  return 0;
}

int fused_pass_kind(const Params& p, const TcPlan& plan) {
  if (plan.a_units <= 4) return 0;
  // the floor epilogue: its scratch lies in the transpose buffer, and k groups of blocks need k blocks
  const bool floor = plan.ctas >= p.k && floor_scratch_bytes(plan.n_pad) <= plan.epi_chunks * kChunkCols * kTile * 4;
  return floor ? 2 : 1;
}

int fused_prepare(const Params& p, const TcPlan& plan) {
  if (!fused_supported(p)) return DDD_ERR_UNSUPPORTED;
  if (allow_max_dynamic_smem(draft_fused_kernel<false>) != cudaSuccess) return DDD_ERR_CUDA;
  if (allow_max_dynamic_smem(draft_fused_kernel<true>) != cudaSuccess) return DDD_ERR_CUDA;
  if (allow_max_dynamic_smem(rerank_kernel) != cudaSuccess) return DDD_ERR_CUDA;
  // every block must be resident at once: the blocks wait for one another
  int per_sm = 0, dev = 0, sms = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, plan.a_units > 4 ? draft_fused_kernel<true> : draft_fused_kernel<false>,
                                                    kTcThreads, plan.smem) != cudaSuccess ||
      cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return DDD_ERR_CUDA;
  if (per_sm < 1 || plan.ctas > per_sm * sms) return DDD_ERR_UNSUPPORTED;
  bool keys;
  cudaFuncAttributes fattr;
  if (cudaFuncGetAttributes(&fattr, rerank_kernel) != cudaSuccess) return DDD_ERR_CUDA;
  if (rerank_kernel_smem(p, &keys) + fattr.sharedSizeBytes > (size_t)kSmemLimit) return DDD_ERR_UNSUPPORTED;
  return DDD_OK;
}

cudaError_t launch_draft_fused(const Params& p, const TcPlan& plan, const FusedArgs& fa_in, bool cooperative,
                               cudaStream_t st) {
  FusedArgs fa = fa_in;
  fa.w_packed = plan.w_packed;
  fa.n_pad = plan.n_pad;
  fa.stages = plan.stages;
  fa.ksub = plan.ksub;
  fa.cpg = plan.epi_chunks;
  fa.pair = plan.a_units > 4 ? plan.a_units : 0;
  fa.floor = fused_pass_kind(p, plan) == 2 ? 1 : 0;
  fa.rerank_inside = fused_rerank_mode(p, plan);
  fa.tmem_cols = plan.tmem_cols;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)plan.ctas, 1, 1);
  cfg.blockDim = dim3(kTcThreads, 1, 1);
  cfg.dynamicSmemBytes = plan.smem;
  cfg.stream = st;
  // The blocks wait for one another, so all of them must be resident at once.  fused_prepare has
  // checked that the device has room for them, and a draft kernel holds a whole SM per block, so on
  // a device that runs nothing else they are: blocks of the next draft move in as those of this one
  // leave (programmatic dependent launch: 3 us per draft at stop depth 2) and wait for its end.
  // Under other long-running work a block may come late; the others' waits are bounded and end
  // in DDD_ERR_TIMEOUT.  A cooperative launch (all blocks at once, or not at all) excludes that and
  // the overlap with it.
  cudaLaunchAttribute attr[1];
  if (cooperative) {
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
  } else {
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
  }
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = fa.pair ? cudaLaunchKernelEx(&cfg, draft_fused_kernel<true>, p, fa, plan.map_h[0], plan.map_h[1])
                          : cudaLaunchKernelEx(&cfg, draft_fused_kernel<false>, p, fa, plan.map_h[0], plan.map_h[1]);
  if (e != cudaSuccess || fa.rerank_inside) return e;
  // rerank + mask: started early (programmatic dependent launch), waits on the device for the draft
  bool keys;
  cudaLaunchConfig_t rc = {};
  rc.gridDim = dim3((unsigned)p.B, 1, 1);
  rc.blockDim = dim3(1024, 1, 1);
  rc.dynamicSmemBytes = rerank_kernel_smem(p, &keys);
  rc.stream = st;
  cudaLaunchAttribute rattr[1];
  rattr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  rattr[0].val.programmaticStreamSerializationAllowed = 1;
  rc.attrs = rattr;
  rc.numAttrs = 1;
  return cudaLaunchKernelEx(&rc, rerank_kernel, p, fa.io, keys ? 1 : 0);
}

}  // namespace ddd
