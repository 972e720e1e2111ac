// LM-head pass on the sm_100a tensor cores.
//
// logits[v][r] = sum_j W[v][j] h[r][j] is computed "swap-AB": the 128 vocab rows of a W
// tile are the M operand, the (few) beam rows are the N operand, so one tcgen05.mma of
// M = 128, N = 16..256 keeps every vocab row in its own tensor-memory lane and every beam
// row in its own column.  The pass is bound by streaming W from HBM once; everything else
// hides under that stream:
//   warp 0     TMA producer: W comes from a copy that ddd_create packs once into the exact
//              shared-memory image the MMA wants - pre-swizzled 4 KB chunks of 32 vocab rows x
//              64 hidden elements, ordered [K-block][32-row unit] - so the rows of one MMA tile
//              and one K-block are a single contiguous run fetched by one plain bulk copy
//              (cp.async.bulk); the matching slice of h comes through a 3-D tensor map; both
//              land in a ring of shared-memory stages.  Issuing a copy costs the thread a few
//              hundred cycles, so stages are made of few, large copies
//   warp 1     issues tcgen05.mma into one of two tensor-memory accumulators
//   warps 2-17 epilogue: four of them tcgen05.ld the finished accumulator, apply scale and bias
//              and transpose it through shared memory; then every warp folds one beam row's
//              128 values into that row's online max / sum-exp and running top-k
// Each thread block owns a contiguous range of vocab rows (a multiple of 32) and publishes
// one partial (max, sum-exp, top-k list) per beam row; logits never reach global memory
// (except for beams wider than 32, see DENSE below).
// Every wait is bounded: when one runs out the block records DDD_ERR_TIMEOUT, drains what
// it has in flight, frees its tensor memory and returns.
#include "lm_head_tc.cuh"
#include "tc_ptx.cuh"

namespace ddd {

namespace {

using namespace tc;

// ---------------------------------------------------------------------------- kernel
// DENSE: the instantiation for wide beams (33..128) on an unsliced vocabulary.  There the sorted
// 128-key list per row and tile would cost the epilogue more than the stream (the pass took 77-117 us
// at widths 50-100 against 42), and R * V logits are little beside V * Hd weights (5 % at 100 rows), so
// this form writes the scaled logits to `logits` [R][ldl] (fp32, -inf for a planted column) and
// leaves the top-k and the log-sum-exp of every row to row_topk_kernel (row_topk.cu); it keeps no
// lists, so the ring gets the shared memory they took.
template <bool DENSE>
__global__ void __launch_bounds__(kTcThreads, 1)
lm_head_tc_kernel(const Params p, const unsigned char* __restrict__ w_packed,
                  const __grid_constant__ CUtensorMap map_h, const int d, const int force_all,
                  const int n_pad, const int stages, const int tmem_cols, const int ksub, const int cpg,
                  float* __restrict__ logits, const size_t ldl) {
  // The kernel may have been launched while the select kernel of the previous pass is still
  // running (programmatic dependent launch).  Until griddep_wait() below it touches nothing
  // that kernel writes, except for one speculative look at the activity counter: if drafting
  // had already stopped before that kernel, there is nothing to prefetch (pass 1 always runs).
  const bool spec_active = force_all || d == 1 || *reinterpret_cast<volatile const int*>(p.n_active) != 0;
  __shared__ int s_ticket;
  if (threadIdx.x == 0) {
    // arrival counter, reset by the last block to arrive; a successor kernel can only start once
    // every block of this one has passed griddep_launch_dependents() below, i.e. after the reset
    const int t = atomicAdd(p.lm_ticket, 1);
    if (t == (int)gridDim.x - 1) {
      atomicExch(p.lm_ticket, 0);
      __threadfence();
    }
    s_ticket = t % (int)gridDim.x;
  }
  __syncthreads();

  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_dyn) + 1023u) & ~static_cast<uintptr_t>(1023u));
  const SmemPlan sp = smem_plan(stages, ksub, n_pad, p.R, DENSE ? 0 : p.k, cpg);
  float* zt = reinterpret_cast<float*>(smem + sp.zt);
  unsigned long long* st_key = reinterpret_cast<unsigned long long*>(smem + sp.key);
  float2* st_ms = reinterpret_cast<float2*>(smem + sp.ms);
  int* s_plant = reinterpret_cast<int*>(smem + sp.plant);
  int* s_live = reinterpret_cast<int*>(smem + sp.live);
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem + sp.bars);
  uint32_t* tmem_ptr = reinterpret_cast<uint32_t*>(smem + sp.tmem_ptr);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + sp.abort_flag);

  const uint32_t a_base = smem_u32(smem + sp.a), b_base = smem_u32(smem + sp.b);
  const uint32_t b_bytes = (uint32_t)n_pad * kBlockK * 2;
  const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8u * stages;
  const uint32_t bar_tfull = bar_empty + 8u * stages, bar_tempty = bar_tfull + 16u;
  const uint32_t bar_spare = bar_tempty + 16u;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // this block's contiguous range of 32-row units
  const int n_units = (p.Vl + kUnitRows - 1) / kUnitRows;    // W, bias: local rows; tokens: v0 + local row
  const int base_units = n_units / (int)gridDim.x, rem_units = n_units % (int)gridDim.x;
  // Vocab ranges are handed out in arrival order: the larger ranges go to the blocks that
  // start first, and the blocks that could only start after the previous select kernel left
  // its SMs get the smaller ones.  Range (and partial-result slot) `bid` always covers the
  // same rows, so the result does not depend on which block took it.
  const int bid = s_ticket;
  const int my_units = base_units + (bid < rem_units ? 1 : 0);
  const int unit0 = bid * base_units + (bid < rem_units ? bid : rem_units);
  // MMA tiles: up to four consecutive units, counted from the start of the block's range.
  const int n_tiles = (my_units + 3) / 4;
  const int num_kb = p.Hd / (kBlockK * ksub);      // stages per tile; each holds ksub K-blocks of 64
  const uint32_t a_stage = (uint32_t)ksub * kABytes, b_stage = (uint32_t)ksub * b_bytes;

  // One (tile, K-group) step of the pipeline: which packed chunk it reads and where it lands.
  const int total_iters = n_tiles * num_kb;
  const int prefill = total_iters < stages ? total_iters : stages;
  // Both are called by all 32 lanes of warp 0.  Issuing a copy occupies the issuing thread for a
  // few hundred cycles whatever its size, so the copies of a stage go out from different lanes in
  // one warp-wide instruction: lane kk sends K-block kk of W, lane ksub the h slice.
  unsigned long long evict_first = 0ull;
  auto issue_w = [&](int it, int stage) {
    const int t = it / num_kb, kb = it - t * num_kb;
    const int nu = min(4, my_units - 4 * t);
    const uint32_t full = bar_full + 8u * stage;
    if (lane == 0) mbar_expect_tx(full, (uint32_t)ksub * ((uint32_t)nu * kUnitBytes + b_bytes));   // W and h bytes
    __syncwarp();
    // W: for each 64-element K-block the tile's units are one contiguous run of the packed copy
    const unsigned char* src = w_packed + ((size_t)(kb * ksub) * n_units + (size_t)(unit0 + 4 * t)) * kUnitBytes;
    const uint32_t dst = a_base + (uint32_t)stage * a_stage;
    if (lane < ksub)
      bulk_load_hint(dst + (uint32_t)lane * kABytes, src + (size_t)lane * n_units * kUnitBytes, (uint32_t)nu * kUnitBytes,
                     full, evict_first);
  };
  auto issue_h = [&](int it, int stage) {
    // h: ksub K-blocks of all beam rows in one tensor copy
    if (lane == ksub)
      tma_load_3d(b_base + (uint32_t)stage * b_stage, &map_h, bar_full + 8u * stage, 0, 0, (it % num_kb) * ksub);
  };

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(bar_full + 8u * s, 1);
      mbar_init(bar_empty + 8u * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_tfull + 8u * a, 1);
      mbar_init(bar_tempty + 8u * a, 4);     // one arrival per epilogue warp
    }
    mbar_init(bar_spare, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncwarp();
  if (warp == 0) {
    // W does not depend on the previous kernel: fill the ring with it right away.
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(evict_first));
    if (spec_active)
      for (int it = 0; it < prefill; ++it) issue_w(it, it);
  }
  __syncwarp();
  // While the previous kernel is still at work HBM is idle: one more thread asks L2 for the part
  // of W that follows the ring (first tile, in the order the pipeline will want it), about as
  // much as the memory system can deliver before the wait below returns.
  if (spec_active && threadIdx.x == 64) {
    const int nu0 = min(4, my_units);
    const int kb_first = prefill * ksub;
    const int kb_last = min(p.Hd / kBlockK, kb_first + kL2PrefetchBytes / (nu0 * kUnitBytes));
    for (int kb64 = kb_first; kb64 < kb_last; ++kb64)
      l2_prefetch(w_packed + ((size_t)kb64 * n_units + (size_t)unit0) * kUnitBytes, (uint32_t)nu0 * kUnitBytes);
  }

  // ---- from here on the previous kernel's results (hidden rows, row flags, counters) are needed
  griddep_wait();
  griddep_launch_dependents();
  if (!force_all && *p.n_active == 0) {
    // every sequence has stopped: complete and await the copies already in flight, then leave
    if (spec_active && warp == 0) {
      for (int it = 0; it < prefill; ++it) issue_h(it, it);
      __syncwarp();
      for (int it = 0; it < prefill; ++it) mbar_wait(bar_full + 8u * it, 0u, abort_flag, p.dev_status, false);
    }
    return;
  }
  if (warp == 0) {
    if (!spec_active)
      for (int it = 0; it < prefill; ++it) issue_w(it, it);
    for (int it = 0; it < prefill; ++it) issue_h(it, it);
  }
  __syncwarp();
  if (warp == 1) {   // tensor-memory allocation is a warp-wide operation
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_ptr)), "r"((uint32_t)tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // per-row flags and running state
  for (int r = threadIdx.x; r < p.R; r += kTcThreads) {
    s_plant[r] = p.row_plant[r];
    s_live[r] = row_live(p, r, d, force_all) ? 1 : 0;
    st_ms[r] = make_float2(neg_inf(), 0.f);
  }
  const int kst = DENSE ? 0 : key_stride(p.k);
  for (int i = threadIdx.x; i < p.R * kst; i += kTcThreads) st_key[i] = 0ull;
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_ptr;

  // Warps 0 and 1 run their loops with all 32 lanes (every lane waits, lane 0 issues), so that
  // each warp stays converged for the block-wide barriers and the warp-wide tcgen05 calls.
  if (warp == 0) {
    // ======================================================================= TMA producer
    int stage = prefill % stages, issued = prefill;
    uint32_t phase = (prefill == stages) ? 1u : 0u;
    bool ok = true;
    for (int it = prefill; it < total_iters; ++it) {
      ok = __all_sync(kFullMask, mbar_wait(bar_empty + 8u * stage, phase ^ 1u, abort_flag, p.dev_status));
      if (!ok) break;
      issue_w(it, stage);
      issue_h(it, stage);
      __syncwarp();
      ++issued;
      if (++stage == stages) { stage = 0; phase ^= 1u; }
    }
    if (!ok) {
      // gave up: wait (bounded) until every copy already issued has landed
      for (int s = 0; s < stages; ++s) {
        const int fills = (issued + stages - 1 - s) / stages;
        if (fills > 0) mbar_wait(bar_full + 8u * s, (uint32_t)((fills - 1) & 1), abort_flag, p.dev_status, false);
      }
      __syncwarp();
    }
  } else if (warp == 1) {
    // ======================================================================= MMA issuer
    const uint32_t idesc = make_instr_desc(n_pad);
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int t = 0; t < n_tiles && ok; ++t) {
      const int acc = t & 1;
      const uint32_t acc_phase = (uint32_t)(t >> 1) & 1u;
      ok = __all_sync(kFullMask, mbar_wait(bar_tempty + 8u * acc, acc_phase ^ 1u, abort_flag, p.dev_status));
      if (!ok) break;
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + (uint32_t)(acc * n_pad);
      for (int kb = 0; kb < num_kb; ++kb) {
        ok = __all_sync(kFullMask, mbar_wait(bar_full + 8u * stage, phase, abort_flag, p.dev_status));
        if (!ok) break;
        tc_fence_after();
        if (lane == 0) {
          for (int kk = 0; kk < ksub; ++kk) {
            const uint32_t a_addr = a_base + (uint32_t)stage * a_stage + (uint32_t)kk * kABytes;
            const uint32_t b_addr = b_base + (uint32_t)stage * b_stage + (uint32_t)kk * b_bytes;
#pragma unroll
            for (int k4 = 0; k4 < kBlockK / kUmmaK; ++k4) {
              tc_mma_bf16(d_tmem, make_smem_desc(a_addr + k4 * kUmmaK * 2),
                          make_smem_desc(b_addr + k4 * kUmmaK * 2), idesc, (kb | kk | k4) != 0 ? 1u : 0u);
            }
          }
          tc_commit(bar_empty + 8u * stage);     // frees the stage once these MMAs have read it
        }
        __syncwarp();
        if (++stage == stages) { stage = 0; phase ^= 1u; }
      }
      if (ok && lane == 0) tc_commit(bar_tfull + 8u * acc);   // accumulator complete
      __syncwarp();
    }
    if (!ok) {
      // make sure no MMA is still running before tensor memory is released
      if (lane == 0) tc_commit(bar_spare);
      __syncwarp();
      mbar_wait(bar_spare, 0u, abort_flag, p.dev_status, false);
      __syncwarp();
    }
  } else {
    // ======================================================================= epilogue
    // Warp ew reads lane quarter ew % 4 of chunk ew / 4 of the current group of chunks, so up to
    // 64 beam rows leave tensor memory between two barriers; then every warp folds the rows r
    // with r % kEpiWarps == ew.
    const int quarter = warp & 3;            // tensor-memory lanes this warp may read
    const int ew = warp - 2;
    const int lw = ew >> 2;                  // chunk of the group this warp loads
    const int n_chunks = (p.R + kChunkCols - 1) / kChunkCols;
    bool ok = true;
    for (int t = 0; t < n_tiles && ok; ++t) {
      const int acc = t & 1;
      const uint32_t acc_phase = (uint32_t)(t >> 1) & 1u;
      const int rows = min(4, my_units - 4 * t) * kUnitRows;
      const int row0 = (unit0 + 4 * t) * kUnitRows;
      // All epilogue warps must leave this wait together (they share named barrier 1 below).
      ok = epilogue_all(mbar_wait(bar_tfull + 8u * acc, acc_phase, abort_flag, p.dev_status, false));
      if (!ok) break;
      tc_fence_after();
      const int vrow = quarter * 32 + lane;
      const int v = row0 + vrow;
      const bool v_ok = vrow < rows && v < p.Vl;
      const float bias = (v_ok && p.bias) ? p.bias[v] : 0.f;
      if constexpr (DENSE) {
        // chunk ch of 16 beam rows by warp (quarter, ch mod 4): a warp's store is 32 consecutive logits of one row
        for (int ch = lw; ch < n_chunks; ch += kEpiWarps / 4) {
          const int c0 = ch * kChunkCols;
          float accv[16];
          tc_load_16cols(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * n_pad + c0), accv);
#pragma unroll
          for (int c = 0; c < kChunkCols; ++c) {
            const int r = c0 + c;
            if (v_ok && r < p.R && s_live[r])
              logits[(size_t)r * ldl + v] = s_plant[r] != v + p.v0 ? fmaf(accv[c], p.s, bias) : neg_inf();
          }
        }
        tc_fence_before();
        epilogue_barrier();
        if (ew < 4 && lane == 0) mbar_arrive(bar_tempty + 8u * acc);
        continue;
      }
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
            if (v_ok && r < p.R && s_plant[r] != v + p.v0) z = fmaf(accv[c], p.s, bias);
            zt[(lw * kChunkCols + c) * kTile + vrow] = z;
          }
          tc_fence_before();
        }
        epilogue_barrier();
        if (g0 + cpg >= n_chunks && ew < 4 && lane == 0) {
          // every warp has read its part of the accumulator: hand it back to the MMA warp
          mbar_arrive(bar_tempty + 8u * acc);
        }
        for (int rr = ew; rr < cpg * kChunkCols; rr += kEpiWarps) {
          const int r = g0 * kChunkCols + rr;
          if (r >= p.R || !s_live[r]) continue;
          float2 ms = st_ms[r];
          if (p.k <= kNarrowK) {
            unsigned long long key = lane < p.k ? st_key[r * p.k + lane] : 0ull;
            row_tile_update(zt + rr * kTile, row0 + p.v0, p.k, ms.x, ms.y, key);
            if (lane < p.k) st_key[r * p.k + lane] = key;
          } else {
            unsigned long long list[4];
            wide_load(list, st_key + r * kst, kst);
            row_tile_update_wide(zt + rr * kTile, row0 + p.v0, p.k, ms.x, ms.y, list);
            wide_store(list, st_key + r * kst, kst);
          }
          if (lane == 0) st_ms[r] = ms;
        }
        epilogue_barrier();
      }
    }
    // publish this block's partial results (each row by its owning warp)
    if (ok && !DENSE) {
      for (int r = ew; r < p.R; r += kEpiWarps) {
        if (!s_live[r]) continue;
        const size_t slot = (size_t)bid * p.R + r;
        for (int e = lane; e < p.k; e += 32) p.part_key[slot * p.k + e] = st_key[r * kst + e];
        if (lane == 0) p.part_ms[slot] = st_ms[r];
      }
    }
  }

  // ---- teardown: everyone meets, then the allocating warp frees tensor memory.  Warps 0 and 1
  // ran single-lane loops: reconverge them first, the block barrier counts whole warps.
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) {
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)tmem_cols)
                 : "memory");
  }
}

// ---------------------------------------------------------------------------- one-time repack of W
// Packed layout: 4 KB chunks, chunk number kb * n_units + u holds rows 32u .. 32u+31 of K-block
// kb (hidden elements 64 kb .. 64 kb + 63), 128 bytes per row, with the 16-byte pieces of each
// row permuted by the 128-byte swizzle (piece c of row r sits at piece c ^ (r & 7)).  A run of
// consecutive chunks is byte for byte the shared-memory image of a K-major SWIZZLE_128B
// operand, so the LM-head kernel fetches any run of units with one plain bulk copy.  Rows past
// V are zero.
__global__ void __launch_bounds__(256) pack_w_kernel(const __nv_bfloat16* __restrict__ W, unsigned char* __restrict__ out,
                                                     int V, int Hd, int n_units) {
  const size_t chunk = blockIdx.x;                 // kb * n_units + u
  const int kb = (int)(chunk / n_units), u = (int)(chunk % n_units);
  uint4* dst = reinterpret_cast<uint4*>(out + chunk * kUnitBytes);
  const int r = threadIdx.x >> 3, c = threadIdx.x & 7;     // 32 rows x 8 pieces of 16 bytes
  const int v = u * kUnitRows + r;
  uint4 val = make_uint4(0u, 0u, 0u, 0u);
  if (v < V) val = *reinterpret_cast<const uint4*>(W + (size_t)v * Hd + kb * kBlockK + c * 8);
  dst[r * 8 + (c ^ (r & 7))] = val;
}

// ---------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn) return fn;
  void* ptr = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || !ptr)
    return nullptr;
  fn = reinterpret_cast<EncodeTiledFn>(ptr);
  return fn;
}

// The hidden rows [rows][cols] bf16 (cols contiguous) seen as a 3-D tensor {64 columns, rows,
// cols / 64 K-blocks}: one box of 64 x box_rows x box_kb lands as box_kb consecutive K-major,
// 128-byte-swizzled operand tiles.  Out-of-range rows read as zero.
bool encode_hidden_3d(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows,
                      uint32_t box_kb) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[3] = {(cuuint64_t)kBlockK, rows, cols / kBlockK};
  const cuuint64_t strides[2] = {cols * 2, (cuuint64_t)kBlockK * 2};
  const cuuint32_t box[3] = {(cuuint32_t)kBlockK, box_rows, box_kb};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

size_t tc_packed_bytes(int vocab, int hidden) {
  const size_t units = ((size_t)vocab + kUnitRows - 1) / kUnitRows;
  return units * kUnitRows * (size_t)hidden * 2;
}

int tc_plan_create(const Params& p, int sm_count, void* w_packed, TcPlan* plan, int extra_smem, int a_units, bool dense) {
  if (p.dtype != DDD_DTYPE_BF16 || p.Hd % kBlockK != 0) return DDD_ERR_UNSUPPORTED;
  const int n_pad = (p.R + 15) / 16 * 16;
  if (n_pad > 256) return DDD_ERR_UNSUPPORTED;
  int cols = 32;
  while (cols < 2 * n_pad) cols *= 2;
  if (cols > 512) return DDD_ERR_UNSUPPORTED;
  const int n_units = (p.Vl + kUnitRows - 1) / kUnitRows;
  int ctas = sm_count < n_units ? sm_count : n_units;
  if (ctas > kMaxLmCtas) ctas = kMaxLmCtas;
  // K-blocks per stage: as many as still leave a ring of two stages, at most 4.  A pipeline step
  // has a fixed cost of about half a microsecond (barrier round trip, copy issue), so few large
  // stages win over many small ones: measured with 32 and 64 beam rows, two stages of four
  // K-blocks beat five of two by 5-7 %.
  // The epilogue takes up to four chunks of 16 beam rows out of tensor memory between two
  // barriers, 8 KB of shared memory each; it gives way to the stage size when both do not fit.
  int ksub = 4, cpg = epi_group(p.R);
  auto fits = [&](int st, int ks, int cg) {
    return smem_plan(st, ks, n_pad, p.R, dense ? 0 : p.k, cg, a_units).total + extra_smem + 1024 <= kSmemLimit;
  };
  for (;;) {
    if (p.Hd % (kBlockK * ksub) == 0 && fits(2, ksub, cpg)) break;
    if (cpg > 1) { cpg /= 2; continue; }
    if (ksub == 1) break;
    ksub /= 2;
    cpg = epi_group(p.R);
  }
  int stages = 0;
  for (int s = 8; s >= 2; --s) {
    if (fits(s, ksub, cpg)) { stages = s; break; }
  }
  if (a_units > 4) {
    // Both tiles of a block fed per stage (many beam rows): what bounds the pass there is the bytes
    // a block has in flight, all stages but the one being multiplied.  So stages of one K-block,
    // as many as fit beside the smallest epilogue buffer, then the largest buffer that still fits.
    ksub = 1;
    cpg = 1;
    stages = 0;
    for (int s = 8; s >= 2; --s) {
      if (fits(s, 1, 1)) { stages = s; break; }
    }
    while (stages && cpg * 2 <= epi_group(p.R) && fits(stages, 1, cpg * 2)) cpg *= 2;
  }
  if (stages == 0) return DDD_ERR_UNSUPPORTED;
  plan->ksub = ksub;
  plan->ctas = ctas;
  plan->n_pad = n_pad;
  plan->stages = stages;
  plan->tmem_cols = cols;
  plan->epi_chunks = cpg;
  plan->smem = (size_t)smem_plan(stages, ksub, n_pad, p.R, dense ? 0 : p.k, cpg, a_units).total + extra_smem + 1024;
  plan->a_units = a_units;
  plan->dense = dense;
  plan->w_packed = static_cast<unsigned char*>(w_packed);
  {
    const size_t chunks = tc_packed_bytes(p.Vl, p.Hd) / kUnitBytes;
    pack_w_kernel<<<(unsigned)chunks, 256>>>(static_cast<const __nv_bfloat16*>(p.W), plan->w_packed, p.Vl, p.Hd,
                                             n_units);
    if (cudaGetLastError() != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) return DDD_ERR_CUDA;
  }
  for (int i = 0; i < 2; ++i)
    if (!encode_hidden_3d(&plan->map_h[i], p.hbuf[i], (uint64_t)p.R, (uint64_t)p.Hd, (uint32_t)n_pad, (uint32_t)ksub))
      return DDD_ERR_CUDA;
  if (allow_max_dynamic_smem(lm_head_tc_kernel<false>) != cudaSuccess) return DDD_ERR_CUDA;
  if (allow_max_dynamic_smem(lm_head_tc_kernel<true>) != cudaSuccess) return DDD_ERR_CUDA;
  return DDD_OK;
}

cudaError_t launch_lm_head_tc(const Params& p, const TcPlan& plan, int d, int force_all, bool pdl, cudaStream_t st,
                              float* logits, size_t ldl) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)plan.ctas, 1, 1);
  cfg.blockDim = dim3(kTcThreads, 1, 1);
  cfg.dynamicSmemBytes = plan.smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  if (plan.dense) {
    if (!logits) return cudaErrorInvalidValue;
    return cudaLaunchKernelEx(&cfg, lm_head_tc_kernel<true>, p, (const unsigned char*)plan.w_packed, plan.map_h[(d - 1) & 1],
                              d, force_all, plan.n_pad, plan.stages, plan.tmem_cols, plan.ksub, plan.epi_chunks, logits, ldl);
  }
  return cudaLaunchKernelEx(&cfg, lm_head_tc_kernel<false>, p, (const unsigned char*)plan.w_packed, plan.map_h[(d - 1) & 1],
                            d, force_all, plan.n_pad, plan.stages, plan.tmem_cols, plan.ksub, plan.epi_chunks,
                            static_cast<float*>(nullptr), (size_t)0);
}

}  // namespace ddd
