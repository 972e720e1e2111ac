/*
 * ddd.h - C ABI of the Dynamic Depth Decoding draft-tree library (single GPU, sm_100a).
 *
 * One call of ddd_draft runs Algorithm 1 of the paper ("Dynamic Depth Decoding") for a
 * batch of B independent sequences, entirely on the device and without a host
 * synchronisation between draft-model calls:
 *
 *   for pass d = 1 .. n:                              (Algorithm 1, the for-loop; n = max_depth)
 *     logits  = s * h W^T + bias   for the beam rows  (Section 1: the draft model ends in the
 *                                                      target's LM head; "Run draft model on beam")
 *     logprob = log-softmax(logits), clamped to <= 0  (Section 2: draft output goes through logsoftmax)
 *     per-row top-k tokens; candidate score = parent's logprobsum + logprob
 *                                                     (Section 1: sum of logprobs ranks token sequences;
 *                                                      Algorithm 1: logprobsum update)
 *     new beam = top-k of the k*k candidates          (Algorithm 1: "produce the new beam")
 *     H = log sum_i exp(logprobsum[i])                (Eq. 1)
 *     stop if d == n, or if step d is in S and H < x  (Algorithm 1: "if step in S", "if H < x: break")
 *     h_child = RMSNorm(h_parent + E[token])          (stands in for the trained draft head of Section 1)
 *   rerank: keep the m best tree nodes by logprobsum, emit tokens, parents, depths, position
 *   ids and a bit-packed ancestor mask                (Section 1: the tree goes to the target model
 *                                                      with an adjusted attention mask)
 *
 * Conventions
 *   - Every pointer argument says whether it is a HOST or a DEVICE pointer.  The library
 *     never allocates device memory: weights, workspace, inputs and outputs are allocated by
 *     the caller and only borrowed.  E, bias, plant_next and the workspace must stay valid
 *     and unchanged until ddd_destroy.  So must W for the CUDA-core kernel (DDD_LM_HEAD_SIMT,
 *     every fp32 handle); a handle on the tensor-core kernel reads W only inside ddd_create,
 *     which packs it into the workspace, and the caller may free or reuse W afterwards.
 *   - All functions return DDD_OK (0) or a negative DDD_ERR_* code; nothing throws, traps or
 *     aborts.  ddd_strerror maps a code to a static string.
 *   - ddd_draft only enqueues work on the given stream.  Outputs are valid once that stream
 *     has been synchronised.  Problems found on the device (a bounded wait that ran out)
 *     are reported through ddd_output.status, never as a fault.
 *   - One draft in flight per handle; a handle is not thread-safe.
 *   - The library reads two environment variables.  DDD_DEBUG: if it is set (to anything), a
 *     failed CUDA call is described on stderr before DDD_ERR_CUDA is returned.
 *     DDD_FUSED_COOPERATIVE: see DDD_LAUNCH_FUSED.  Nothing else about its behaviour depends
 *     on the environment.
 */
#ifndef DDD_H_
#define DDD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ddd_handle ddd_handle; /* opaque */

enum {
  DDD_OK = 0,
  DDD_ERR_INVALID_ARG = -1, /* NULL pointer, size out of range, unknown enum value          */
  DDD_ERR_ALIGNMENT = -2,   /* a pointer is not aligned as documented                        */
  DDD_ERR_WORKSPACE = -3,   /* workspace smaller than ddd_workspace_bytes()                  */
  DDD_ERR_CUDA = -4,        /* a CUDA runtime / driver call failed                           */
  DDD_ERR_TIMEOUT = -5,     /* device status: a bounded wait inside a kernel ran out         */
  DDD_ERR_UNSUPPORTED = -6  /* valid request this build cannot serve (e.g. kernel / dtype)   */
};

enum { DDD_DTYPE_FP32 = 0, DDD_DTYPE_BF16 = 1 };

/* Which LM-head kernel runs a pass.  AUTO picks TCGEN05 for bf16 and SIMT for fp32. */
enum { DDD_LM_HEAD_AUTO = 0, DDD_LM_HEAD_SIMT = 1, DDD_LM_HEAD_TCGEN05 = 2 };

/* How a draft is enqueued.  STREAM launches kernel by kernel, each allowed to start while its
 * predecessor still runs (programmatic dependent launch; they synchronise on the device).
 * GRAPH replays one captured CUDA graph per draft, in which the passes are cut into groups (after
 * checked steps: passes 1-3, 4-5, 6-8, 9-12, ... when every step is checked) and every group
 * but the first sits behind a conditional node that only a still-drafting sequence switches
 * on, so that a draft that stops early launches little that has nothing to do.  PLAIN launches
 * kernel by kernel in ordinary stream order, one after the other: the slowest, and the one
 * profilers can follow.  FUSED runs the whole draft as ONE persistent kernel of one thread block
 * per SM that loops over the passes itself and hands over between them
 * through counters in global memory; the rerank and the mask run inside it too where the tree
 * fits the kernel's spare shared memory, else in one small kernel behind it:
 * the fastest, for bf16 handles on the tensor-core kernel with a beam of at most 32
 * (ddd_create returns DDD_ERR_UNSUPPORTED otherwise, also where the device cannot hold all
 * blocks at once).  Its blocks wait for one another, a whole SM each, so nothing else should
 * run on the device meanwhile: a block kept off its SM by other work for longer than the
 * waits' limit (2 s) ends the draft with DDD_ERR_TIMEOUT in ddd_output.status, never in a hang.
 * The kernel is launched as a programmatic dependent of the kernel before it in the stream:
 * blocks of the next draft set themselves up on the SMs that those of the running draft have
 * left, and wait for its end before they touch anything the two share.  With
 * DDD_FUSED_COOPERATIVE set in the environment it is a cooperative launch instead (all blocks
 * resident at once or the launch fails; no overlap between drafts). */
enum { DDD_LAUNCH_STREAM = 0, DDD_LAUNCH_GRAPH = 1, DDD_LAUNCH_PLAIN = 2, DDD_LAUNCH_FUSED = 3 };

#define DDD_MAX_K 128         /* beam width limit (the paper's appendix table goes to 100) */
#define DDD_MAX_DEPTH 32      /* check_mask has one bit per step                   */
#define DDD_MAX_TOTAL 1023    /* m limit (output rows = m + 1)                     */
#define DDD_MAX_ROWS 256      /* B * k limit                                       */
#define DDD_MAX_NODES 98304   /* 1 + k + (n-1) k^2 limit                           */
#define DDD_MAX_SHARDS 16      /* slices of a vocabulary-parallel LM head           */
#define DDD_CHECK_EVERY_STEP 0xFFFFFFFFu

/* Parameters of Algorithm 1 (n, w, S, x) and the tensor shapes. */
typedef struct {
  int32_t batch;        /* B >= 1 independent sequences                                           */
  int32_t hidden;       /* Hd, multiple of 8 (multiple of 64 for the TCGEN05 kernel)              */
  int32_t vocab;        /* V > k                                                                  */
  int32_t k;            /* beam width w, 1..DDD_MAX_K (beams wider than 32 take a slower, sort-based path;
                           a configuration whose per-row lists do not fit on chip, e.g. 256 rows of
                           width 128, is refused with DDD_ERR_UNSUPPORTED)                        */
  int32_t max_depth;    /* n: maximum number of draft-model calls, 1..DDD_MAX_DEPTH               */
  int32_t total_tokens; /* m: draft nodes kept by the rerank (the root is extra), 1..DDD_MAX_TOTAL */
  int32_t dtype;        /* DDD_DTYPE_*: storage type of W, E and every hidden state               */
  float threshold;      /* x: after a checked step, drafting continues iff H >= x                 */
  uint32_t check_mask;  /* S: bit (s-1) set <=> the heuristic is checked after step s             */
  float logit_scale;    /* s in logits = s * h W^T + bias                                         */
  float rms_eps;        /* eps inside the square root of RMSNorm                                  */
  float plant_delta;    /* see plant_next in ddd_create                                           */
  int32_t device;       /* CUDA device ordinal                                                    */
  int32_t lm_head_kernel; /* DDD_LM_HEAD_*                                                        */
  int32_t launch_mode;    /* DDD_LAUNCH_*                                                         */
  int32_t vocab_begin;    /* first token id of the slice of W this handle owns, and                      */
  int32_t vocab_count;    /* its number of rows; 0, 0 = the whole vocabulary (see ddd_shard_* below)      */
} ddd_config;

/*
 * Results of one draft.  With T = total_tokens + 1 and W32 = ceil(T / 32), per sequence b:
 *   n_out[b]        rows used: 1 + min(m, N), N = k + (D-1) k^2 nodes generated in D passes
 *   stop_depth[b]   D: number of draft-model calls made (1..n)
 *   row 0 is the root; rows 1..n_out-1 are the kept nodes in ascending generation order,
 *   so a parent always precedes its children.  Rows >= n_out hold token = parent = depth =
 *   position = -1, cum = 0 and an all-zero mask row.
 *   token[b][i], parent[b][i] (row index of the parent, -1 for the root), depth[b][i],
 *   position[b][i] = root_pos[b] + depth, cum[b][i] = summed logprob of the path (root 0)
 *   mask[b][i][w]   bit j of row i (word j / 32, bit j % 32, LSB first) is set iff row j is
 *                   row i itself or one of its ancestors
 *   H_trace[b][d-1] Eq. 1 evaluated after pass d, for every pass that ran (others untouched)
 *   status[0]       DDD_OK, or the first DDD_ERR_* a kernel recorded during this draft
 * Every field is required and is a DEVICE pointer for ddd_draft, a HOST pointer for
 * ddd_draft_host.  Layout is dense row-major in the index order shown.
 */
typedef struct {
  int32_t *n_out;      /* [B]         */
  int32_t *stop_depth; /* [B]         */
  int32_t *token;      /* [B][T]      */
  int32_t *parent;     /* [B][T]      */
  int32_t *depth;      /* [B][T]      */
  int32_t *position;   /* [B][T]      */
  float *cum;          /* [B][T]      */
  uint32_t *mask;      /* [B][T][W32] */
  float *H_trace;      /* [B][n]      */
  int32_t *status;     /* [1]         */
} ddd_output;

/*
 * Optional record of the search itself (all DEVICE pointers, each may be NULL), used to
 * replay the decisions in another implementation.  Nn = 1 + k + (n-1) k^2 node slots per
 * sequence; node 0 is the root, pass 1 creates nodes 1..k, pass d >= 2 creates node
 * 1 + k + (d-2) k^2 + p k + c for the c-th best token of beam row p.
 *   node_id[b][i]      tree node shown in output row i (-1 beyond n_out)
 *   tree_token[b][j], tree_parent[b][j] (node id), tree_cum[b][j]   for generated nodes
 *   beam_sel[b][d-1][i] candidate index p k + c that became beam entry i after pass d
 *   row_lse[b][d-1][p]  logsumexp of the logits of beam row p in pass d
 */
typedef struct {
  int32_t *node_id;     /* [B][T]    */
  int32_t *tree_token;  /* [B][Nn]   */
  int32_t *tree_parent; /* [B][Nn]   */
  float *tree_cum;      /* [B][Nn]   */
  int32_t *beam_sel;    /* [B][n][k] */
  float *row_lse;       /* [B][n][k] */
} ddd_trace;

/*
 * Bytes of device workspace a handle with this configuration needs (0 if the configuration
 * is invalid).  Pure host function; makes no CUDA call.
 */
size_t ddd_workspace_bytes(const ddd_config *cfg /* HOST */);

/*
 * Creates a handle.  (Algorithm 1's Require line: n, w, S, x arrive in cfg.)
 *   W           DEVICE [V][Hd], row-major (hidden contiguous), cfg->dtype, 16-byte aligned:
 *               the LM head, logits[r][v] = s * sum_j W[v][j] h[r][j] + bias[v]
 *   E           DEVICE [V][Hd], same layout and type: embedding rows for the draft step
 *   bias        DEVICE [V] fp32 or NULL
 *   plant_next  DEVICE [V] int32 or NULL.  If given and c = plant_next[t] >= 0 for the last
 *               token t of a beam row, that row's logit of column c is replaced by
 *               (maximum of the row's other logits) + plant_delta before the log-softmax.
 *   workspace   DEVICE, 256-byte aligned, at least ddd_workspace_bytes(cfg) bytes; its
 *               contents are owned by the handle until ddd_destroy.
 * Makes cfg->device current, creates no stream, allocates no device memory.
 * Errors: INVALID_ARG, ALIGNMENT, WORKSPACE, UNSUPPORTED, CUDA.  *out is NULL on error.
 */
int ddd_create(const ddd_config *cfg /* HOST */, const void *W, const void *E, const float *bias,
               const int32_t *plant_next, void *workspace, size_t workspace_bytes,
               ddd_handle **out /* HOST */);

/*
 * Enqueues one draft of the whole batch on `cuda_stream` (a cudaStream_t; NULL = the legacy
 * default stream) and returns without waiting.  (Algorithm 1, all lines; then the rerank.)
 *   root_hidden DEVICE [B][Hd], cfg->dtype, 16-byte aligned: hidden state fed to pass 1
 *   root_token  DEVICE [B] int32: last accepted token of each sequence (tree node 0)
 *   root_pos    DEVICE [B] int32: its position id
 *   out         HOST struct of DEVICE pointers, all required
 *   trace       HOST struct of DEVICE pointers or NULL
 * In DDD_LAUNCH_GRAPH mode everything after the first kernel is replayed from a captured CUDA
 * graph, which is reused while the out / trace pointers and the stream stay the same and is
 * re-captured when they change (the root_* pointers may change freely).  Graph mode needs a
 * non-default stream; with NULL the kernels are enqueued one by one.
 * Errors: INVALID_ARG, ALIGNMENT, CUDA.
 */
int ddd_draft(ddd_handle *h, const void *root_hidden, const int32_t *root_token,
              const int32_t *root_pos, const ddd_output *out, const ddd_trace *trace,
              void *cuda_stream);

/*
 * The same draft the way the paper runs it (Section 2, Section 3.4 "Strict"): after every
 * LM-head pass the HOST synchronises the stream, reads how many sequences are still drafting
 * and only then launches the next pass.  Arguments and results are those of ddd_draft (DEVICE
 * buffers); the call returns after the last pass has been enqueued, with *passes_run (HOST, may be
 * NULL) = number of passes launched.  It exists to measure what the device-resident gate of
 * ddd_draft saves; results are identical.  Errors: INVALID_ARG, ALIGNMENT, CUDA.
 */
int ddd_draft_host_gated(ddd_handle *h, const void *root_hidden, const int32_t *root_token,
                         const int32_t *root_pos, const ddd_output *out, const ddd_trace *trace,
                         void *cuda_stream, int32_t *passes_run);

/*
 * Same draft with HOST buffers: copies the inputs to staging space inside the workspace,
 * runs the draft, copies every ddd_output field back and synchronises the stream before
 * returning.  All pointers (inputs and the fields of `out`) are HOST pointers of ordinary or
 * pinned memory: the call packs them into one pinned buffer of its own (allocated on the first
 * call), so there is one copy in each direction.  In DDD_LAUNCH_GRAPH mode with a non-default
 * stream the whole call is a single graph launch (input copy, first kernel, passes, output
 * copy), captured on the first call per stream.  Returns the device status (e.g.
 * DDD_ERR_TIMEOUT) if the draft itself reported one.
 */
int ddd_draft_host(ddd_handle *h, const void *root_hidden, const int32_t *root_token,
                   const int32_t *root_pos, const ddd_output *out, void *cuda_stream);

/*
 * Enqueues ONE LM-head pass (logits, online max / sum-exp and per-row top-k partials, the
 * kernel that streams W) over all B*k beam rows currently held by the handle, for timing
 * and profiling that kernel alone.  It reads the hidden rows left by the last draft and
 * writes only workspace scratch.  (Section 1: the draft model call; Algorithm 1 "Run draft
 * model on beam".)  Errors: INVALID_ARG, CUDA.
 */
int ddd_lm_head_pass(ddd_handle *h, void *cuda_stream);

/*
 * ddd_launches_per_draft: kernels one ddd_draft launches when a sequence of the batch needs
 * `passes_needed` LM-head passes (its largest stop depth).  Outside graph mode every pass is
 * launched (kernels of passes after the stop exit at once); in graph mode the passes up to the
 * end of the group that holds pass `passes_needed` are launched.
 * ddd_lm_head_blocks: thread blocks of the LM-head kernel.
 * ddd_fused_pass_kind: how a DDD_LAUNCH_FUSED handle runs a pass on this device: 0 = a block walks
 * its 128-row tiles one after the other, 1 = both tiles of a block are fed from one fetch of the
 * hidden rows (48 beam rows or more, five to eight 32-row units of the vocabulary per block),
 * 2 = as 1, and the blocks agree on a lower bound of every row's k-th best logit before they
 * pick their k best; handles of other launch modes give 0.  Results do not depend on it
 * (scores agree to rounding): it exists for tests and benchmarks that want to know which path ran.
 * Pure host queries; negative on a NULL handle.
 */
int ddd_launches_per_draft(const ddd_handle *h, int32_t passes_needed);
int ddd_lm_head_blocks(const ddd_handle *h);
int ddd_fused_pass_kind(const ddd_handle *h);

/*
 * One LM-head pass that allocates nothing.  (The paper has no counterpart: this exists for
 * integration, not for the method.)  For `rows` hidden rows it computes
 * logits = logit_scale * h W^T + bias, the log-softmax of every row, and the row's k best
 * tokens with their log-probabilities - the same arithmetic as one pass of ddd_draft - but it
 * needs no handle and no caller workspace.  It is meant for callers that cannot obtain device
 * memory at call time: code living inside another library's callback or plug-in interface
 * that is handed fixed buffers only, a process whose device memory belongs to a framework pool
 * it must not call into, or a latency-critical loop where cudaMalloc (which may synchronise
 * the device) is unacceptable.  Its scratch space, the per-block partial results, is a fixed
 * array of 2,162,688 bytes inside the library's device image; every GPU that loads the
 * library holds it until the process exits.
 *   W            DEVICE [vocab][hidden], dtype DDD_DTYPE_*, 16-byte aligned
 *   bias         DEVICE [vocab] fp32 or NULL
 *   hidden_rows  DEVICE [rows][hidden], same dtype, 16-byte aligned
 *   out_token    DEVICE [rows][k] int32, best first (ties: lower token id)
 *   out_logprob  DEVICE [rows][k] fp32, clamped to <= 0
 *   out_lse      DEVICE [rows] fp32 logsumexp of the row's logits
 * Limits: 1 <= rows <= 32, 1 <= k <= 32, hidden a multiple of 8, vocab > k.  Sizes
 * beyond these do not fit the fixed scratch and return DDD_ERR_INVALID_ARG; misaligned W or
 * hidden_rows return DDD_ERR_ALIGNMENT.  Works on the device that is current in the calling
 * thread and only enqueues two kernels on `cuda_stream`; it calls no allocating routine.
 * The first call on each device looks up the scratch array's device address (a one-time
 * set-up under a lock); make that first call before starting any stream capture.
 * All calls share the one scratch array: it keeps whatever the previous call left, which is
 * harmless because every slot that is read is rewritten first, but two calls whose kernels
 * overlap on the GPU (different streams, or different threads) race.  Serialise them.
 */
int ddd_lm_head_topk_noalloc(const void *W, const float *bias, const void *hidden_rows, int32_t dtype,
                             int32_t rows, int32_t hidden, int32_t vocab, int32_t k, float logit_scale,
                             int32_t *out_token, float *out_logprob, float *out_lse, void *cuda_stream);

/*
 * Vocabulary-parallel LM head.  (The paper runs on one GPU - Section 3.1, Setup - and has no
 * counterpart; this splits the one step of Algorithm 1 that streams the LM-head matrix.)
 * G ranks, one handle each, created with vocab_begin / vocab_count set: such a handle takes as W
 * only the rows [vocab_begin, vocab_begin + vocab_count) of the LM head (DEVICE
 * [vocab_count][Hd]) and as bias the matching slice ([vocab_count] or NULL); E, plant_next and
 * cfg->vocab stay those of the whole vocabulary, and token ids everywhere are global.  Every rank
 * keeps the whole tree state and runs the same select / gate / draft step; only the LM-head pass
 * is split.  A pass d = 1..n is three steps on every rank:
 *   ddd_shard_lm_head  streams the rank's slice and folds the result into one record per beam row:
 *                      the slice's (max, sum-exp) and its k best (logit, token) pairs.  The record
 *                      goes to slot `slot` of each of the n_dst record sets listed in records_dst:
 *                      the rank's own and, through peer pointers, those of the other ranks (or
 *                      only its own, if the caller moves records itself, e.g. with an all-gather).
 *                      If flags_dst is given, flags_dst[i][slot] is set to a value that names this
 *                      draft and pass once the records are on their way.
 *   (exchange)         whatever carries the other ranks' records into this rank's record set
 *   ddd_shard_select   merges the `slots` records of a record set, in slot order, and runs the
 *                      ordinary select / gate / draft step of pass d; with `flags` given it first
 *                      waits, bounded, until all of them name this draft and pass (a wait that
 *                      runs out sets status to DDD_ERR_TIMEOUT; nothing hangs).
 * A record set is ddd_shard_records_bytes(cfg, slots) bytes, 16-byte aligned; flags are `slots`
 * int32 words, zero before the first draft.  Use two record sets and flag arrays, alternating by
 * the parity of d: a rank may already be writing pass d + 1 while a slower peer still reads pass d.
 * ddd_shard_begin starts a draft (resets the state, loads the root; every rank passes the same
 * inputs) and must be called the same number of times on every rank, since the flag values count
 * drafts.  After a sequence has stopped, the calls of later passes do nothing for it; once all have
 * stopped they do nothing at all but still raise their flags, so the simplest caller enqueues all
 * n passes.  Results land in `out` / `trace` of ddd_shard_begin on every rank alike.  Per-slice
 * sums are added up per rank and then across ranks, so scores may differ from an unsharded draft
 * in the last bits (not in the tokens, unless two scores tie to within those bits).
 * ddd_draft* on a handle that owns a slice return DDD_ERR_INVALID_ARG.  A handle that owns the
 * whole vocabulary may use these calls with slots = 1: a one-slice run.
 * Errors: INVALID_ARG (d, slot, slots, n_dst out of range, NULL pointers), ALIGNMENT, CUDA.
 */
size_t ddd_shard_records_bytes(const ddd_config *cfg /* HOST */, int32_t slots);
int ddd_shard_begin(ddd_handle *h, const void *root_hidden, const int32_t *root_token, const int32_t *root_pos,
                    const ddd_output *out, const ddd_trace *trace, void *cuda_stream);
int ddd_shard_lm_head(ddd_handle *h, int32_t d, int32_t slot, int32_t slots,
                      void *const *records_dst /* HOST array of n_dst DEVICE pointers */,
                      int32_t *const *flags_dst /* HOST array of n_dst DEVICE pointers, or NULL */,
                      int32_t n_dst, void *cuda_stream);
int ddd_shard_select(ddd_handle *h, int32_t d, const void *records /* DEVICE */, int32_t slots,
                     const int32_t *flags /* DEVICE [slots] or NULL */, void *cuda_stream);

/*
 * What the verification step needs from a finished tree.  With T = t_rows and L = max_depth + 1,
 * per sequence b (all DEVICE pointers, all required):
 *   n_accepted[b]        draft tokens the greedy walk accepted (0..max_depth)
 *   accepted_rows[b][j]  output row of the j-th accepted token, j < n_accepted; -1 after that
 *   next_token[b]        the target's token after the last accepted row (the token that is
 *                        always gained, even when no draft token is accepted)
 *   n_leaves[b]          rows of the tree without a child among the emitted rows
 *   leaf_paths[b][l][j]  for the l-th leaf in ascending row order, the rows from the root
 *                        (j = 0, always row 0) down to the leaf; -1 after the leaf and in
 *                        the rows l >= n_leaves
 *   status[0]            DDD_OK, or DDD_ERR_INVALID_ARG if some sequence's rows were not a tree
 *                        (a parent index not below its child's, or a path longer than L); that
 *                        sequence then reports 0 accepted, next_token -1 and 0 leaves
 */
typedef struct {
  int32_t *n_accepted;    /* [B]            */
  int32_t *accepted_rows; /* [B][max_depth] */
  int32_t *next_token;    /* [B]            */
  int32_t *n_leaves;      /* [B]            */
  int32_t *leaf_paths;    /* [B][T][L]      */
  int32_t *status;        /* [1]            */
} ddd_verify_output;

/*
 * Greedy acceptance walk and leaf-path table over the rows ddd_draft emitted.  (Section 1: the
 * target model verifies the tree in one call; at temperature 0 a draft token is accepted when it
 * is the target's own choice after its parent, which makes acceptance a walk from the root.)
 *   n_out, token, parent   DEVICE, as in ddd_output ([B], [B][T], [B][T]); row 0 is the root
 *   target_argmax          DEVICE [B][T] int32: the target's choice of next token after row i
 *                          (its argmax at that row's position under the tree mask); rows
 *                          >= n_out are ignored
 * The walk starts at row 0 and moves to the child of the current row whose token equals
 * target_argmax of the current row (the lowest such row, should siblings repeat a token) until
 * there is none.  Needs no handle and no workspace; enqueues two small kernels on `cuda_stream`
 * and returns without waiting.  Limits: 1 <= t_rows <= DDD_MAX_TOTAL + 1, 1 <= max_depth <=
 * DDD_MAX_DEPTH, batch >= 1.  Errors: INVALID_ARG, CUDA.
 */
int ddd_verify_greedy(int32_t batch, int32_t t_rows, int32_t max_depth, const int32_t *n_out,
                      const int32_t *token, const int32_t *parent, const int32_t *target_argmax,
                      const ddd_verify_output *out /* HOST struct */, void *cuda_stream);

/* Releases host state (and the captured graph).  Device memory stays with the caller. */
int ddd_destroy(ddd_handle *h);

/* Static description of a DDD_* code. */
const char *ddd_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* DDD_H_ */
