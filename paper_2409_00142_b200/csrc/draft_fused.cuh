// Host interface of the one-kernel-per-draft path (draft_fused.cu).
#pragma once

#include "ddd_common.cuh"
#include "lm_head_tc.cuh"

namespace ddd {

// What the persistent kernel needs beyond Params: the caller's root and output pointers of this
// draft and the state that only this path keeps (all device pointers into the workspace).
struct FusedArgs {
  const unsigned char* w_packed;
  const void* root_hidden;
  const int* root_token;
  const int* root_pos;
  DraftIO io;
  float* beam_cum;      // [2][R] summed log-probability of the beam, by pass parity
  int* beam_node;       // [2][R] tree node of each beam entry
  int* row_plant;       // [2][R] planted column of each beam row, -1 = none
  int* sync;            // [5] hand-over counters (partials, hidden rows), abort word, exit ticket, floor hand-over
  unsigned int* gmax;   // [R][32] largest logit of the row in each group of blocks (ordered score), see floor
  unsigned long long* fkey;   // [R][k][160] per-block top-k keys, position-major (entry j of all blocks together)
  float2* fms;                // [R][160]    per-block (max, sum exp(z - max))
  int n_pad, stages, ksub, cpg, tmem_cols;
  int rerank_inside;    // the rerank runs inside the draft kernel (1: keys in shared memory, 2: from global memory)
  int pair;             // 0, or the 32-row units of W per K-block of a stage (5-8) when both tiles of a block
                        // share each stage (one fetch of the hidden rows per pass)
  int floor;            // pair mode: the blocks agree on a floor per row before they pick their k best
};

// Shared memory the tree work needs behind the LM-head pipeline's own.
int fused_extra_smem(int k);
// 32-row units of W per K-block of a stage: 4 (one tile), or the most a block owns (5 to 8) where a block
// should feed both of its tiles from one fetch of the hidden rows.  That needs every block to own exactly
// two tiles and pays off once the hidden rows weigh: from 48 beam rows.
int fused_stage_units(const Params& p, int sm_count);
// Can this configuration run as one kernel (bf16, tensor-core kernel, beam width up to 32)?
bool fused_supported(const Params& p);
// Checks that all blocks fit on the device at once and sets the kernels' attributes.  DDD_* code.
int fused_prepare(const Params& p, const TcPlan& plan);
int fused_rerank_mode(const Params& p, const TcPlan& plan);
// 0: tile after tile, 1: both tiles of a block per stage, 2: as 1 with a floor per row agreed between the blocks.
int fused_pass_kind(const Params& p, const TcPlan& plan);
// Enqueues the draft kernel and, where the rerank does not fit inside it, the rerank kernel behind it.
// cooperative: launch with the cooperative attribute instead of as a programmatic dependent of the kernel before it.
cudaError_t launch_draft_fused(const Params& p, const TcPlan& plan, const FusedArgs& fa, bool cooperative, cudaStream_t st);

}  // namespace ddd
