// Host interface of the tensor-core LM-head kernel (lm_head_tc.cu).
#pragma once

#include <cuda.h>

#include "ddd_common.cuh"

namespace ddd {

struct TcPlan {
  unsigned char* w_packed; // W re-laid out as pre-swizzled 16 KB chunks [tile of 128 rows][K-block of 64]
  CUtensorMap map_h[2];   // hidden rows [R][Hd] bf16 of each pass parity: box 64 x n_pad
  int ctas;               // persistent thread blocks, one per SM at most
  int n_pad;              // MMA N: beam rows rounded up to a multiple of 16
  int stages;             // depth of the shared-memory ring
  int ksub;               // 64-element K-blocks per stage
  int epi_chunks;         // 16-row accumulator chunks the epilogue unloads per barrier pair (1..4)
  int tmem_cols;          // allocated tensor-memory columns (power of two)
  int a_units;            // 32-row units of W per K-block of a stage (4 = one tile; 5-8: both tiles of a block, see draft_fused.cu)
  size_t smem;            // dynamic shared memory per block
  bool dense;             // sized for the form that writes the logits out (no per-row lists in shared memory)
};

// Bytes of the packed copy of W (vocab rounded up to whole 128-row tiles).
size_t tc_packed_bytes(int vocab, int hidden);
// Packs W into `w_packed` (device, 1024-byte aligned, tc_packed_bytes), encodes the tensor maps of
// the hidden buffers and sizes the pipeline.  Synchronises the device.  Returns a DDD_* code.
// extra_smem: bytes kept free behind the pipeline's own shared memory (for a kernel that does more than the pass).
// dense: size the pipeline for the form that writes the logits to global memory (wide beams; see lm_head_tc.cu).
int tc_plan_create(const Params& p, int sm_count, void* w_packed, TcPlan* plan, int extra_smem = 0, int a_units = 4,
                   bool dense = false);
// pdl: launch with programmatic stream serialisation (see griddep_wait in ddd_common.cuh).
// logits / ldl: with a plan sized `dense`, where the scaled logits go ([R][ldl] fp32); else ignored.
cudaError_t launch_lm_head_tc(const Params& p, const TcPlan& plan, int d, int force_all, bool pdl, cudaStream_t st,
                              float* logits = nullptr, size_t ldl = 0);

// row_topk.cu: the record of every live row of pass d ([R][k] keys, then [R] (max, sum exp)) from its logits [R][ldl].
cudaError_t launch_row_topk(const Params& p, int d, const float* logits, size_t ldl, void* record, cudaStream_t st);

}  // namespace ddd
