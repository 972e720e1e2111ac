// Host interface of the tensor-core LM-head kernel (lm_head_tc.cu).
#pragma once

#include <cuda.h>

#include "ddd_common.cuh"

namespace ddd {

struct TcPlan {
  CUtensorMap map_w;      // W [V][Hd] bf16: box of 64 hidden elements x 32 vocab rows, 128-byte swizzle
  CUtensorMap map_h[2];   // hidden rows [R][Hd] bf16 of each pass parity: box 64 x n_pad
  int ctas;               // persistent thread blocks, one per SM at most
  int n_pad;              // MMA N: beam rows rounded up to a multiple of 16
  int stages;             // depth of the shared-memory ring
  int tmem_cols;          // allocated tensor-memory columns (power of two)
  size_t smem;            // dynamic shared memory per block
};

// Encodes the tensor maps and sizes the pipeline.  Returns a DDD_* code.
int tc_plan_create(const Params& p, int sm_count, TcPlan* plan);
cudaError_t launch_lm_head_tc(const Params& p, const TcPlan& plan, int d, int force_all, cudaStream_t st);

}  // namespace ddd
