// Host side of the C ABI declared in ddd.h: argument checking, workspace carving, the
// launch sequence of one draft (optionally replayed from a CUDA graph) and the host-buffer
// variant.  No device memory is allocated here; the only allocation is a small pinned host
// bounce buffer used by ddd_draft_host.
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "ddd_common.cuh"
#include "draft_fused.cuh"
#include "lm_head_tc.cuh"

using namespace ddd;

namespace {

// Clears the sticky CUDA error; with DDD_DEBUG set in the environment, says what it was.
void note_cuda_error(int line) {
  const cudaError_t e = cudaGetLastError();
  static const bool verbose = std::getenv("DDD_DEBUG") != nullptr;
  if (verbose) std::fprintf(stderr, "[ddd] CUDA failure near ddd_api.cu:%d: %s\n", line, cudaGetErrorString(e));
}

constexpr size_t kAlign = 256;
size_t align_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }

struct Layout {
  size_t hbuf[2], part_key, part_ms, tree_token, tree_parent, tree_cum, beam_node, beam_tok, beam_cum,
      row_plant, active, stop_depth, root_pos, n_active, dev_status, lm_ticket, shard_counter, fused_sync,
      fused_beam_cum, fused_beam_node, fused_row_plant, fused_key, fused_ms, fused_gmax, wide_records, wide_logits, wide_ldl, w_packed;
  // staging for ddd_draft_host: inputs, then the packed output block
  size_t in_hidden, in_token, in_pos, out_block;
  size_t o_n_out, o_stop, o_token, o_parent, o_depth, o_position, o_cum, o_mask, o_H, o_status, out_bytes;
  size_t in_bytes;   // in_hidden .. in_pos are contiguous: one copy
  size_t total;
};

int validate(const ddd_config* c) {
  if (!c) return DDD_ERR_INVALID_ARG;
  if (c->batch < 1 || c->hidden < 8 || c->vocab < 2) return DDD_ERR_INVALID_ARG;
  if (c->hidden % 8 != 0) return DDD_ERR_INVALID_ARG;
  if (c->k < 1 || c->k > DDD_MAX_K || c->vocab <= c->k) return DDD_ERR_INVALID_ARG;
  if (c->max_depth < 1 || c->max_depth > DDD_MAX_DEPTH) return DDD_ERR_INVALID_ARG;
  if (c->total_tokens < 1 || c->total_tokens > DDD_MAX_TOTAL) return DDD_ERR_INVALID_ARG;
  if (c->dtype != DDD_DTYPE_FP32 && c->dtype != DDD_DTYPE_BF16) return DDD_ERR_INVALID_ARG;
  if ((long long)c->batch * c->k > DDD_MAX_ROWS) return DDD_ERR_INVALID_ARG;
  const long long nn = 1 + (long long)c->k + (long long)(c->max_depth - 1) * c->k * c->k;
  if (nn > DDD_MAX_NODES) return DDD_ERR_INVALID_ARG;
  if (!(c->logit_scale == c->logit_scale) || !(c->threshold == c->threshold)) return DDD_ERR_INVALID_ARG;
  if (!(c->rms_eps >= 0.f)) return DDD_ERR_INVALID_ARG;
  if (c->device < 0) return DDD_ERR_INVALID_ARG;
  if (c->lm_head_kernel < DDD_LM_HEAD_AUTO || c->lm_head_kernel > DDD_LM_HEAD_TCGEN05) return DDD_ERR_INVALID_ARG;
  if (c->launch_mode < DDD_LAUNCH_STREAM || c->launch_mode > DDD_LAUNCH_FUSED) return DDD_ERR_INVALID_ARG;
  if (c->vocab_count == 0 ? c->vocab_begin != 0
                          : (c->vocab_begin < 0 || c->vocab_count < 1 ||
                             (long long)c->vocab_begin + c->vocab_count > c->vocab))
    return DDD_ERR_INVALID_ARG;
  if (c->lm_head_kernel == DDD_LM_HEAD_TCGEN05 && (c->dtype != DDD_DTYPE_BF16 || c->hidden % 64 != 0))
    return DDD_ERR_UNSUPPORTED;
  return DDD_OK;
}

Layout make_layout(const ddd_config* c) {
  Layout L{};
  const size_t elt = c->dtype == DDD_DTYPE_FP32 ? 4 : 2;
  const size_t B = c->batch, k = c->k, R = B * k, n = c->max_depth, T = c->total_tokens + 1;
  const size_t W32 = (T + 31) / 32, Nn = 1 + k + (n - 1) * k * k;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
  L.hbuf[0] = take(R * c->hidden * elt);
  L.hbuf[1] = take(R * c->hidden * elt);
  L.part_key = take((size_t)kMaxLmCtas * R * k * 8);
  L.part_ms = take((size_t)kMaxLmCtas * R * 8);
  L.tree_token = take(B * Nn * 4);
  L.tree_parent = take(B * Nn * 4);
  L.tree_cum = take(B * Nn * 4);
  L.beam_node = take(R * 4);
  L.beam_tok = take(R * 4);
  L.beam_cum = take(R * 4);
  L.row_plant = take(R * 4);
  L.active = take(B * 4);
  L.stop_depth = take(B * 4);
  L.root_pos = take(B * 4);
  L.n_active = take(4);
  L.dev_status = take(4);
  L.lm_ticket = take(8);
  L.shard_counter = take(8);
  L.fused_sync = take(32);
  L.fused_beam_cum = take(2 * R * 4);
  L.fused_beam_node = take(2 * R * 4);
  L.fused_row_plant = take(2 * R * 4);
  const bool may_fuse = c->launch_mode == DDD_LAUNCH_FUSED && k <= 32;
  L.fused_key = take(may_fuse ? R * k * 160 * 8 : 0);
  L.fused_ms = take(may_fuse ? R * 160 * 8 : 0);
  L.fused_gmax = take(may_fuse ? R * 32 * 4 : 0);
  L.wide_records = take(k > 32 ? R * (k + 1) * 8 : 0);      // beams wider than 32: one folded partial per row
  // ... and, on the tensor-core kernel with an unsliced vocabulary, the logits of a pass [R][ldl] fp32
  const bool wide_dense = k > 32 && c->vocab_count == 0 && c->dtype == DDD_DTYPE_BF16 && c->hidden % 64 == 0 &&
                          c->lm_head_kernel != DDD_LM_HEAD_SIMT;
  L.wide_ldl = (size_t)(c->vocab + 31) / 32 * 32;
  L.wide_logits = take(wide_dense ? R * L.wide_ldl * 4 : 0);
  // packed copy of W for the tensor-core kernel (kept 1024-byte aligned relative to the base)
  off = (off + 1023) / 1024 * 1024;
  const bool tc_possible = c->dtype == DDD_DTYPE_BF16 && c->hidden % 64 == 0 && c->lm_head_kernel != DDD_LM_HEAD_SIMT;
  L.w_packed = take(tc_possible ? tc_packed_bytes(c->vocab_count ? c->vocab_count : c->vocab, c->hidden) : 0);
  // host-variant staging: inputs packed back to back (each 16-byte aligned), one output block
  L.in_hidden = take(0);
  size_t in = 0;
  auto in_take = [&](size_t bytes) { size_t o = in; in = (in + bytes + 15) / 16 * 16; return o; };
  const size_t ih = in_take(B * c->hidden * elt), it = in_take(B * 4), ip = in_take(B * 4);
  L.in_bytes = in;
  L.in_token = L.in_hidden + it;
  L.in_pos = L.in_hidden + ip;
  (void)ih;
  take(in);
  L.out_block = take(0);
  size_t o = 0;
  auto o_take = [&](size_t bytes) { size_t r = o; o = (o + bytes + 15) / 16 * 16; return r; };
  L.o_n_out = o_take(B * 4);
  L.o_stop = o_take(B * 4);
  L.o_token = o_take(B * T * 4);
  L.o_parent = o_take(B * T * 4);
  L.o_depth = o_take(B * T * 4);
  L.o_position = o_take(B * T * 4);
  L.o_cum = o_take(B * T * 4);
  L.o_mask = o_take(B * T * W32 * 4);
  L.o_H = o_take(B * n * 4);
  L.o_status = o_take(4);
  L.out_bytes = o;
  take(o);
  L.total = off;
  return L;
}

constexpr int kFirstBoundary = 3;    // first pass after which a captured draft may end early
constexpr int kMaxGraphLevels = 4;   // nested IF nodes of a captured draft

struct GraphKey {
  ddd_output out;
  ddd_trace trace;
  cudaStream_t stream;
};

}  // namespace

struct ddd_handle {
  ddd_config cfg;
  Params p;
  Layout L;
  unsigned char* ws;
  int sm_count;
  int lm_kind;     // DDD_LM_HEAD_SIMT or DDD_LM_HEAD_TCGEN05
  TcPlan tc;
  // graph cache (one entry)
  cudaGraphExec_t exec;
  cudaGraphExec_t exec_host;    // ddd_draft_host's graph: input copy, init, passes, output copy
  cudaStream_t host_stream;     // stream exec_host was captured on
  GraphKey key;
  bool have_graph;
  bool use_pdl;    // programmatic dependent launch between the kernels of a draft
  bool graph_pdl;  // whether the captured graph uses it
  int bounds[kMaxGraphLevels];   // passes after which a captured draft may end early (IF nodes), ascending
  int n_bounds;
  int graph_bounds;   // how many of them the captured graph has
  // pinned host bounce buffer for ddd_draft_host
  unsigned char* bounce;
  size_t bounce_bytes;
  // vocabulary-parallel drafting: output pointers of the draft in progress, drafts begun so far
  DraftIO shard_io;
  bool shard_open;
  int shard_epoch;
  int* shard_counter;
};

namespace {

cudaError_t launch_lm_head(const ddd_handle* h, int d, int force_all, bool pdl, cudaStream_t st) {
  if (h->lm_kind == DDD_LM_HEAD_TCGEN05)
    return launch_lm_head_tc(h->p, h->tc, d, force_all, pdl, st,
                             h->tc.dense ? reinterpret_cast<float*>(h->ws + h->L.wide_logits) : nullptr, h->L.wide_ldl);
  return launch_lm_head_simt(h->p, d, force_all, h->p.lm_ctas, st);
}

// Everything after the init kernel: it depends on the output pointers only, so a captured
// graph of it can be replayed for any root.
// With pdl every kernel after the init kernel is launched with programmatic stream
// serialisation: it may start while its predecessor runs and waits for it on the device.
// Passes first..last are enqueued; the select kernel of pass `cond_pass` (0 = none) switches
// the graph conditional `cond` on if its sequence goes on.
// `after_kernel`: the first LM-head launch directly follows a kernel of this library in the same
// stream or capture (the init kernel), so it may be a programmatic dependent too.
cudaError_t enqueue_passes(const ddd_handle* h, const DraftIO& io, bool pdl, int first, int last,
                           cudaGraphConditionalHandle cond, int cond_pass, cudaStream_t st,
                           bool after_kernel = false) {
  cudaError_t e = cudaSuccess;
  // Beams wider than 32: a kernel of one block per beam row folds the per-block partials into one
  // list per row first (the select kernel's eight blocks per sequence would otherwise merge
  // k x 148 lists one row after the other), and the select kernel reads that one partial.
  const bool wide = h->p.k > 32;
  Params q = h->p;
  void* rec = h->ws + h->L.wide_records;
  if (wide) {
    q.part_key = reinterpret_cast<unsigned long long*>(rec);
    q.part_ms = reinterpret_cast<float2*>(h->ws + h->L.wide_records + (size_t)q.R * q.k * sizeof(unsigned long long));
    q.lm_ctas = 1;
  }
  for (int d = first; d <= last && e == cudaSuccess; ++d) {
    e = launch_lm_head(h, d, 0, pdl && (d > first || after_kernel), st);
    if (e == cudaSuccess && wide) {
      // the record of a row: from its logits where the LM-head kernel wrote them out, else folded from the blocks' lists
      if (h->lm_kind == DDD_LM_HEAD_TCGEN05 && h->tc.dense)
        e = launch_row_topk(h->p, d, reinterpret_cast<const float*>(h->ws + h->L.wide_logits), h->L.wide_ldl, rec, st);
      else
        e = launch_shard_reduce(h->p, d, 0, 1, &rec, nullptr, 1, 0, h->shard_counter, st);
    }
    if (e == cudaSuccess) e = launch_select(wide ? q : h->p, io, d, pdl, cond, d == cond_pass, st);
  }
  return e;
}

// Where a captured draft may end early.  A pass that has nothing left to do still costs two
// kernel launches (about 4 us), and most drafts stop long before pass n, so the passes are cut
// into groups: group 0 (passes 1..b1) always runs, every later group sits in the body of an IF
// node that only a sequence still drafting after the previous group switches on; the bodies
// nest.  Boundaries are put after checked steps only (nothing can stop elsewhere), the first
// not before pass 3, the groups growing by one pass each (3, 5, 8, 12 when every step is
// checked), at most kMaxGraphLevels of them: entering an IF body costs about as much as two to
// three idle passes, so a deep draft should not cross many.  None at all when the threshold is so
// low that drafting always runs to pass n.

int graph_boundaries(const ddd_config& cfg, int* bounds /* [kMaxGraphLevels] */) {
  const int n = cfg.max_depth;
  int count = 0;
  if (n <= kFirstBoundary + 1) return 0;
  if (!(cfg.threshold > -1e30f)) return 0;   // no finite H is below such a threshold: fixed-depth drafting
  int want = kFirstBoundary, gap = 2;
  for (int d = kFirstBoundary; d < n && count < kMaxGraphLevels; ++d) {
    if (d < want || !((cfg.check_mask >> (d - 1)) & 1u)) continue;
    bounds[count++] = d;
    want = d + gap;
    ++gap;
  }
  return count;
}

struct CaptureLog {
  int step = 0;   // which call failed first, for the diagnostic
  bool good(cudaError_t e, int id) {
    if (e != cudaSuccess && step == 0) step = id;
    return e == cudaSuccess;
  }
};

// Captures group `level` (passes first..bounds[level], or first..n for the last group) into
// `graph`, followed by the IF node that guards the next group.
// With `host_wrap` the top level also holds what ddd_draft_host puts around a draft: the copy of
// the packed inputs from the pinned bounce buffer, the init kernel on the staged inputs, and,
// last, the copy of the packed results back to the bounce buffer.
bool capture_level(ddd_handle* h, const DraftIO& io, bool pdl, cudaStream_t st, cudaGraph_t graph,
                   const int* bounds, int n_bounds, int level, int first, CaptureLog& log, bool host_wrap) {
  const int n = h->p.n;
  const bool has_if = level < n_bounds;
  const int last = has_if ? bounds[level] : n;
  const int id = 10 * level;
  cudaGraphConditionalHandle cond = 0;
  cudaGraph_t body = nullptr;
  bool ok = true;
  if (has_if) ok = log.good(cudaGraphConditionalHandleCreate(&cond, graph, 0, cudaGraphCondAssignDefault), id + 2);
  bool capturing = false;
  if (ok) {
    ok = log.good(cudaStreamBeginCaptureToGraph(st, graph, nullptr, nullptr, 0, cudaStreamCaptureModeThreadLocal),
                  id + 3);
    capturing = ok;
  }
  const bool wrap = host_wrap && level == 0;
  if (ok && wrap) {
    const Layout& L = h->L;
    ok = log.good(cudaMemcpyAsync(h->ws + L.in_hidden, h->bounce, L.in_bytes, cudaMemcpyHostToDevice, st), id + 1) &&
         log.good(launch_init(h->p, io, h->ws + L.in_hidden, reinterpret_cast<const int*>(h->ws + L.in_token),
                              reinterpret_cast<const int*>(h->ws + L.in_pos), st), id + 1);
  }
  if (ok) ok = log.good(enqueue_passes(h, io, pdl, first, last, cond, has_if ? last : 0, st, wrap), id + 4);
  if (ok && has_if) {
    // splice the IF node in behind the captured passes
    cudaStreamCaptureStatus status;
    const cudaGraphNode_t* deps = nullptr;
    size_t n_deps = 0;
    ok = log.good(cudaStreamGetCaptureInfo(st, &status, nullptr, nullptr, &deps, &n_deps), id + 5) &&
         status == cudaStreamCaptureStatusActive;
    cudaGraphNode_t node = nullptr;
    if (ok) {
      cudaGraphNodeParams np = {};
      np.type = cudaGraphNodeTypeConditional;
      np.conditional.handle = cond;
      np.conditional.type = cudaGraphCondTypeIf;
      np.conditional.size = 1;
      ok = log.good(cudaGraphAddNode(&node, graph, deps, n_deps, &np), id + 6);
      if (ok) body = np.conditional.phGraph_out[0];
    }
    if (ok) ok = log.good(cudaStreamUpdateCaptureDependencies(st, &node, 1, cudaStreamSetCaptureDependencies), id + 7);
  }
  if (ok && wrap)
    ok = log.good(cudaMemcpyAsync(h->bounce, h->ws + h->L.out_block, h->L.out_bytes, cudaMemcpyDeviceToHost, st), id + 8);
  if (capturing) {
    cudaGraph_t done = nullptr;
    if (!log.good(cudaStreamEndCapture(st, &done), id + 9)) ok = false;
  }
  if (ok && body) ok = capture_level(h, io, pdl, st, body, bounds, n_bounds, level + 1, last + 1, log, host_wrap);
  return ok;
}

// Captures everything after the init kernel into h->exec, with IF nodes after the first
// `n_bounds` boundaries.  Returns false (and leaves no graph) on any failure.
bool capture_graph(ddd_handle* h, const DraftIO& io, bool pdl, int n_bounds, cudaStream_t st,
                   bool host_wrap = false) {
  cudaGraph_t graph = nullptr;
  cudaGraphExec_t* exec = host_wrap ? &h->exec_host : &h->exec;
  CaptureLog log;
  bool ok = log.good(cudaGraphCreate(&graph, 0), 1);
  if (ok) ok = capture_level(h, io, pdl, st, graph, h->bounds, n_bounds, 0, 1, log, host_wrap);
  if (ok) ok = log.good(cudaGraphInstantiate(exec, graph, 0), 99);
  if (graph) cudaGraphDestroy(graph);
  if (!ok) {
    note_cuda_error(1000 + log.step);   // 1000 + 10 * group + index of the capture step that failed
    *exec = nullptr;
    return false;
  }
  if (!host_wrap) {
    h->graph_pdl = pdl;
    h->graph_bounds = n_bounds;
  }
  return true;
}

// Tries the capture with programmatic dependent launches and nested IF nodes first, then with a
// single IF node, then as a plain stream-ordered sequence.
bool capture_with_fallbacks(ddd_handle* h, const DraftIO& io, cudaStream_t st, bool host_wrap) {
  const int one = h->n_bounds < 1 ? h->n_bounds : 1;
  return (h->use_pdl && capture_graph(h, io, true, h->n_bounds, st, host_wrap)) ||
         (h->use_pdl && one != h->n_bounds && capture_graph(h, io, true, one, st, host_wrap)) ||
         capture_graph(h, io, false, one, st, host_wrap);
}

bool aligned16(const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15u) == 0; }

}  // namespace

extern "C" {

size_t ddd_workspace_bytes(const ddd_config* cfg) {
  if (validate(cfg) != DDD_OK) return 0;
  return make_layout(cfg).total;
}

int ddd_create(const ddd_config* cfg, const void* W, const void* E, const float* bias,
               const int32_t* plant_next, void* workspace, size_t workspace_bytes, ddd_handle** out) {
  if (out) *out = nullptr;
  if (!out) return DDD_ERR_INVALID_ARG;
  const int v = validate(cfg);
  if (v != DDD_OK) return v;
  if (!W || !E || !workspace) return DDD_ERR_INVALID_ARG;
  if (!aligned16(W) || !aligned16(E)) return DDD_ERR_ALIGNMENT;
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign != 0) return DDD_ERR_ALIGNMENT;
  const Layout L = make_layout(cfg);
  if (workspace_bytes < L.total) return DDD_ERR_WORKSPACE;

  if (cudaSetDevice(cfg->device) != cudaSuccess) return DDD_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, cfg->device) != cudaSuccess) return DDD_ERR_CUDA;

  ddd_handle* h = new (std::nothrow) ddd_handle();
  if (!h) return DDD_ERR_CUDA;
  h->cfg = *cfg;
  h->L = L;
  h->ws = static_cast<unsigned char*>(workspace);
  h->sm_count = prop.multiProcessorCount;
  h->have_graph = false;
  h->n_bounds = graph_boundaries(*cfg, h->bounds);
  h->graph_bounds = 0;
  h->use_pdl = cfg->launch_mode != DDD_LAUNCH_PLAIN;
  h->graph_pdl = false;
  h->exec = nullptr;
  h->exec_host = nullptr;
  h->host_stream = nullptr;
  h->bounce = nullptr;
  h->bounce_bytes = 0;
  h->shard_open = false;
  h->shard_epoch = 0;
  h->shard_counter = reinterpret_cast<int*>(h->ws + L.shard_counter);

  Params& p = h->p;
  p.B = cfg->batch; p.Hd = cfg->hidden; p.V = cfg->vocab; p.k = cfg->k; p.n = cfg->max_depth;
  p.m = cfg->total_tokens; p.dtype = cfg->dtype;
  p.Vl = cfg->vocab_count ? cfg->vocab_count : cfg->vocab;
  p.v0 = cfg->vocab_count ? cfg->vocab_begin : 0;
  p.R = p.B * p.k;
  p.Nn = 1 + p.k + (p.n - 1) * p.k * p.k;
  p.T = p.m + 1;
  p.W32 = (p.T + 31) / 32;
  p.x = cfg->threshold; p.check_mask = cfg->check_mask;
  p.s = cfg->logit_scale; p.eps = cfg->rms_eps; p.plant_delta = cfg->plant_delta;
  p.W = W; p.E = E; p.bias = bias; p.plant_next = plant_next;
  unsigned char* ws = h->ws;
  p.hbuf[0] = ws + L.hbuf[0];
  p.hbuf[1] = ws + L.hbuf[1];
  p.part_key = reinterpret_cast<unsigned long long*>(ws + L.part_key);
  p.part_ms = reinterpret_cast<float2*>(ws + L.part_ms);
  p.tree_token = reinterpret_cast<int*>(ws + L.tree_token);
  p.tree_parent = reinterpret_cast<int*>(ws + L.tree_parent);
  p.tree_cum = reinterpret_cast<float*>(ws + L.tree_cum);
  p.beam_node = reinterpret_cast<int*>(ws + L.beam_node);
  p.beam_tok = reinterpret_cast<int*>(ws + L.beam_tok);
  p.beam_cum = reinterpret_cast<float*>(ws + L.beam_cum);
  p.row_plant = reinterpret_cast<int*>(ws + L.row_plant);
  p.active = reinterpret_cast<int*>(ws + L.active);
  p.stop_depth = reinterpret_cast<int*>(ws + L.stop_depth);
  p.root_pos = reinterpret_cast<int*>(ws + L.root_pos);
  p.n_active = reinterpret_cast<int*>(ws + L.n_active);
  p.dev_status = reinterpret_cast<int*>(ws + L.dev_status);
  p.lm_ticket = reinterpret_cast<int*>(ws + L.lm_ticket);

  int rc = DDD_OK;
  // Zero the workspace once so that rows never written by a draft hold finite values.
  if (cudaMemset(ws, 0, L.total) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) rc = DDD_ERR_CUDA;
  h->lm_kind = cfg->lm_head_kernel;
  if (h->lm_kind == DDD_LM_HEAD_AUTO)
    h->lm_kind = (cfg->dtype == DDD_DTYPE_BF16 && cfg->hidden % 64 == 0) ? DDD_LM_HEAD_TCGEN05 : DDD_LM_HEAD_SIMT;
  if (rc == DDD_OK && h->lm_kind == DDD_LM_HEAD_TCGEN05) {
    if (prop.major != 10) rc = DDD_ERR_UNSUPPORTED;
    const bool fused = cfg->launch_mode == DDD_LAUNCH_FUSED;
    if (rc == DDD_OK && fused && cfg->k > 32) rc = DDD_ERR_UNSUPPORTED;
    const int a_units = fused && cfg->k <= 32 ? fused_stage_units(p, h->sm_count) : 4;
    const bool dense = cfg->k > 32 && cfg->vocab_count == 0;      // wide beams: logits out, top-k per row behind (row_topk.cu)
    if (rc == DDD_OK)
      rc = tc_plan_create(p, h->sm_count, ws + L.w_packed, &h->tc, fused ? fused_extra_smem(cfg->k) : 0, a_units, dense);
    if (rc == DDD_OK) p.lm_ctas = h->tc.ctas;
    if (rc == DDD_OK && fused) rc = fused_prepare(p, h->tc);
  } else if (rc == DDD_OK && cfg->launch_mode == DDD_LAUNCH_FUSED) {
    rc = DDD_ERR_UNSUPPORTED;            // the one-kernel draft is built on the tensor-core LM head
  } else if (rc == DDD_OK) {
    const int n_tiles = (p.Vl + kTile - 1) / kTile;
    int ctas = 2 * h->sm_count;
    if (ctas > n_tiles) ctas = n_tiles;
    if (ctas > kMaxLmCtas) ctas = kMaxLmCtas;
    p.lm_ctas = ctas;
    if (prepare_simt(p) != cudaSuccess) rc = DDD_ERR_CUDA;
  }
  if (rc == DDD_OK && prepare_tree(p) != cudaSuccess) rc = DDD_ERR_CUDA;
  if (rc != DDD_OK) {
    note_cuda_error(__LINE__);
    delete h;
    return rc;
  }
  *out = h;
  return DDD_OK;
}

int ddd_draft(ddd_handle* h, const void* root_hidden, const int32_t* root_token, const int32_t* root_pos,
              const ddd_output* out, const ddd_trace* trace, void* cuda_stream) {
  if (!h || !root_hidden || !root_token || !root_pos || !out) return DDD_ERR_INVALID_ARG;
  if (!out->n_out || !out->stop_depth || !out->token || !out->parent || !out->depth || !out->position ||
      !out->cum || !out->mask || !out->H_trace || !out->status)
    return DDD_ERR_INVALID_ARG;
  if (!aligned16(root_hidden)) return DDD_ERR_ALIGNMENT;
  if (h->cfg.vocab_count != 0) return DDD_ERR_INVALID_ARG;     // a slice cannot draft alone: ddd_shard_*
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  DraftIO io;
  io.out = *out;
  if (trace) io.trace = *trace; else std::memset(&io.trace, 0, sizeof io.trace);

  if (h->cfg.launch_mode == DDD_LAUNCH_FUSED) {
    FusedArgs fa = {};
    fa.root_hidden = root_hidden;
    fa.root_token = root_token;
    fa.root_pos = root_pos;
    fa.io = io;
    fa.beam_cum = reinterpret_cast<float*>(h->ws + h->L.fused_beam_cum);
    fa.beam_node = reinterpret_cast<int*>(h->ws + h->L.fused_beam_node);
    fa.row_plant = reinterpret_cast<int*>(h->ws + h->L.fused_row_plant);
    fa.sync = reinterpret_cast<int*>(h->ws + h->L.fused_sync);
    fa.fkey = reinterpret_cast<unsigned long long*>(h->ws + h->L.fused_key);
    fa.fms = reinterpret_cast<float2*>(h->ws + h->L.fused_ms);
    fa.gmax = reinterpret_cast<unsigned int*>(h->ws + h->L.fused_gmax);
    static const bool cooperative = std::getenv("DDD_FUSED_COOPERATIVE") != nullptr;
    if (launch_draft_fused(h->p, h->tc, fa, cooperative, st) != cudaSuccess) {
      note_cuda_error(__LINE__);
      return DDD_ERR_CUDA;
    }
    return DDD_OK;
  }
  if (h->cfg.launch_mode == DDD_LAUNCH_GRAPH && st != nullptr) {
    GraphKey key;
    std::memset(&key, 0, sizeof key);
    key.out = io.out; key.trace = io.trace; key.stream = st;
    if (!h->have_graph || std::memcmp(&key, &h->key, sizeof key) != 0) {
      if (h->exec) { cudaGraphExecDestroy(h->exec); h->exec = nullptr; }
      h->have_graph = false;
      if (!capture_with_fallbacks(h, io, st, false)) return DDD_ERR_CUDA;
      h->key = key;
      h->have_graph = true;
    }
    if (launch_init(h->p, io, root_hidden, root_token, root_pos, st) != cudaSuccess ||
        cudaGraphLaunch(h->exec, st) != cudaSuccess) {
      note_cuda_error(__LINE__);
      return DDD_ERR_CUDA;
    }
    return DDD_OK;
  }
  if (launch_init(h->p, io, root_hidden, root_token, root_pos, st) != cudaSuccess ||
      enqueue_passes(h, io, h->use_pdl, 1, h->p.n, 0, 0, st, true) != cudaSuccess) {
    note_cuda_error(__LINE__);
    return DDD_ERR_CUDA;
  }
  return DDD_OK;
}

int ddd_draft_host_gated(ddd_handle* h, const void* root_hidden, const int32_t* root_token, const int32_t* root_pos,
                         const ddd_output* out, const ddd_trace* trace, void* cuda_stream, int32_t* passes_run) {
  if (passes_run) *passes_run = 0;
  if (!h || !root_hidden || !root_token || !root_pos || !out) return DDD_ERR_INVALID_ARG;
  if (!out->n_out || !out->stop_depth || !out->token || !out->parent || !out->depth || !out->position ||
      !out->cum || !out->mask || !out->H_trace || !out->status)
    return DDD_ERR_INVALID_ARG;
  if (!aligned16(root_hidden)) return DDD_ERR_ALIGNMENT;
  if (h->cfg.vocab_count != 0) return DDD_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  DraftIO io;
  io.out = *out;
  if (trace) io.trace = *trace; else std::memset(&io.trace, 0, sizeof io.trace);
  cudaError_t e = launch_init(h->p, io, root_hidden, root_token, root_pos, st);
  int d = 1;
  for (; d <= h->p.n && e == cudaSuccess; ++d) {
    e = enqueue_passes(h, io, h->use_pdl, d, d, 0, 0, st);
    // the host decides: wait for the pass, read how many sequences are still drafting
    int still = 0;
    if (e == cudaSuccess) e = cudaMemcpyAsync(&still, h->p.n_active, sizeof still, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess || still == 0) break;
  }
  if (passes_run) *passes_run = d <= h->p.n ? d : h->p.n;
  if (e != cudaSuccess) {
    note_cuda_error(__LINE__);
    return DDD_ERR_CUDA;
  }
  return DDD_OK;
}

int ddd_draft_host(ddd_handle* h, const void* root_hidden, const int32_t* root_token, const int32_t* root_pos,
                   const ddd_output* out, void* cuda_stream) {
  if (!h || !root_hidden || !root_token || !root_pos || !out) return DDD_ERR_INVALID_ARG;
  if (!out->n_out || !out->stop_depth || !out->token || !out->parent || !out->depth || !out->position ||
      !out->cum || !out->mask || !out->H_trace || !out->status)
    return DDD_ERR_INVALID_ARG;
  if (h->cfg.vocab_count != 0) return DDD_ERR_INVALID_ARG;
  const Layout& L = h->L;
  const Params& p = h->p;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  // inputs first, results behind them (the fused mode reads and writes this buffer from the device)
  const size_t out_off = align_up(L.in_bytes);
  const size_t need = out_off + L.out_bytes;
  if (!h->bounce) {
    if (cudaMallocHost(reinterpret_cast<void**>(&h->bounce), need) != cudaSuccess) {
      note_cuda_error(__LINE__);
      return DDD_ERR_CUDA;
    }
    h->bounce_bytes = need;
  }
  const size_t elt = p.dtype == DDD_DTYPE_FP32 ? 4 : 2;
  const size_t B = p.B, T = p.T;
  // pack the inputs into pinned memory: one host-to-device copy
  std::memcpy(h->bounce, root_hidden, B * p.Hd * elt);
  std::memcpy(h->bounce + (L.in_token - L.in_hidden), root_token, B * 4);
  std::memcpy(h->bounce + (L.in_pos - L.in_hidden), root_pos, B * 4);
  unsigned char* ob = h->ws + L.out_block;
  ddd_output dev;
  dev.n_out = reinterpret_cast<int32_t*>(ob + L.o_n_out);
  dev.stop_depth = reinterpret_cast<int32_t*>(ob + L.o_stop);
  dev.token = reinterpret_cast<int32_t*>(ob + L.o_token);
  dev.parent = reinterpret_cast<int32_t*>(ob + L.o_parent);
  dev.depth = reinterpret_cast<int32_t*>(ob + L.o_depth);
  dev.position = reinterpret_cast<int32_t*>(ob + L.o_position);
  dev.cum = reinterpret_cast<float*>(ob + L.o_cum);
  dev.mask = reinterpret_cast<uint32_t*>(ob + L.o_mask);
  dev.H_trace = reinterpret_cast<float*>(ob + L.o_H);
  dev.status = reinterpret_cast<int32_t*>(ob + L.o_status);
  const unsigned char* hb = h->bounce;      // where the packed results end up
  if (h->cfg.launch_mode == DDD_LAUNCH_FUSED) {
    // Pinned host memory is addressable from the device: the persistent kernel reads the roots from
    // the bounce buffer itself (8 KB, under its first W copies) and writes the rows straight into it,
    // so the call is one kernel launch and one synchronisation, with no copy commands.
    unsigned char* hob = h->bounce + out_off;
    ddd_output direct;
    direct.n_out = reinterpret_cast<int32_t*>(hob + L.o_n_out);
    direct.stop_depth = reinterpret_cast<int32_t*>(hob + L.o_stop);
    direct.token = reinterpret_cast<int32_t*>(hob + L.o_token);
    direct.parent = reinterpret_cast<int32_t*>(hob + L.o_parent);
    direct.depth = reinterpret_cast<int32_t*>(hob + L.o_depth);
    direct.position = reinterpret_cast<int32_t*>(hob + L.o_position);
    direct.cum = reinterpret_cast<float*>(hob + L.o_cum);
    direct.mask = reinterpret_cast<uint32_t*>(hob + L.o_mask);
    direct.H_trace = reinterpret_cast<float*>(hob + L.o_H);
    direct.status = reinterpret_cast<int32_t*>(hob + L.o_status);
    const int rc = ddd_draft(h, h->bounce, reinterpret_cast<const int32_t*>(h->bounce + (L.in_token - L.in_hidden)),
                             reinterpret_cast<const int32_t*>(h->bounce + (L.in_pos - L.in_hidden)), &direct, nullptr,
                             cuda_stream);
    if (rc != DDD_OK) return rc;
    if (cudaStreamSynchronize(st) != cudaSuccess) {
      note_cuda_error(__LINE__);
      return DDD_ERR_CUDA;
    }
    hb = hob;
  } else if (h->cfg.launch_mode == DDD_LAUNCH_GRAPH && st != nullptr) {
    // the whole call is one graph launch: input copy, init kernel, the passes, output copy
    if (!h->exec_host || h->host_stream != st) {
      if (h->exec_host) { cudaGraphExecDestroy(h->exec_host); h->exec_host = nullptr; }
      DraftIO io;
      io.out = dev;
      std::memset(&io.trace, 0, sizeof io.trace);
      if (!capture_with_fallbacks(h, io, st, true)) return DDD_ERR_CUDA;
      h->host_stream = st;
    }
    if (cudaGraphLaunch(h->exec_host, st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess) {
      note_cuda_error(__LINE__);
      return DDD_ERR_CUDA;
    }
  } else {
    if (cudaMemcpyAsync(h->ws + L.in_hidden, h->bounce, L.in_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) {
      note_cuda_error(__LINE__);
      return DDD_ERR_CUDA;
    }
    const int rc = ddd_draft(h, h->ws + L.in_hidden, reinterpret_cast<const int32_t*>(h->ws + L.in_token),
                             reinterpret_cast<const int32_t*>(h->ws + L.in_pos), &dev, nullptr, cuda_stream);
    if (rc != DDD_OK) return rc;
    // one device-to-host copy of the packed results
    if (cudaMemcpyAsync(h->bounce, ob, L.out_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
      note_cuda_error(__LINE__);
      return DDD_ERR_CUDA;
    }
  }
  // scatter the packed results to the caller's arrays
  std::memcpy(out->n_out, hb + L.o_n_out, B * 4);
  std::memcpy(out->stop_depth, hb + L.o_stop, B * 4);
  std::memcpy(out->token, hb + L.o_token, B * T * 4);
  std::memcpy(out->parent, hb + L.o_parent, B * T * 4);
  std::memcpy(out->depth, hb + L.o_depth, B * T * 4);
  std::memcpy(out->position, hb + L.o_position, B * T * 4);
  std::memcpy(out->cum, hb + L.o_cum, B * T * 4);
  std::memcpy(out->mask, hb + L.o_mask, B * T * p.W32 * 4);
  std::memcpy(out->H_trace, hb + L.o_H, B * p.n * 4);
  std::memcpy(out->status, hb + L.o_status, 4);
  return out->status[0];
}

size_t ddd_shard_records_bytes(const ddd_config* cfg, int32_t slots) {
  if (validate(cfg) != DDD_OK || slots < 1 || slots > DDD_MAX_SHARDS) return 0;
  const size_t R = (size_t)cfg->batch * cfg->k;
  return (size_t)slots * R * ((size_t)cfg->k + 1) * 8;
}

int ddd_shard_begin(ddd_handle* h, const void* root_hidden, const int32_t* root_token, const int32_t* root_pos,
                    const ddd_output* out, const ddd_trace* trace, void* cuda_stream) {
  if (!h || !root_hidden || !root_token || !root_pos || !out) return DDD_ERR_INVALID_ARG;
  if (!out->n_out || !out->stop_depth || !out->token || !out->parent || !out->depth || !out->position ||
      !out->cum || !out->mask || !out->H_trace || !out->status)
    return DDD_ERR_INVALID_ARG;
  if (!aligned16(root_hidden)) return DDD_ERR_ALIGNMENT;
  h->shard_io.out = *out;
  if (trace) h->shard_io.trace = *trace; else std::memset(&h->shard_io.trace, 0, sizeof h->shard_io.trace);
  if (launch_init(h->p, h->shard_io, root_hidden, root_token, root_pos, static_cast<cudaStream_t>(cuda_stream)) !=
      cudaSuccess) {
    note_cuda_error(__LINE__);
    return DDD_ERR_CUDA;
  }
  h->shard_open = true;
  h->shard_epoch = (h->shard_epoch + 1) & 0xFFFFFF;
  return DDD_OK;
}

static int shard_flag_value(const ddd_handle* h, int d) { return h->shard_epoch * (DDD_MAX_DEPTH + 1) + d; }

int ddd_shard_lm_head(ddd_handle* h, int32_t d, int32_t slot, int32_t slots, void* const* records_dst,
                      int32_t* const* flags_dst, int32_t n_dst, void* cuda_stream) {
  if (!h || !h->shard_open || !records_dst) return DDD_ERR_INVALID_ARG;
  if (d < 1 || d > h->p.n || slots < 1 || slots > DDD_MAX_SHARDS || slot < 0 || slot >= slots) return DDD_ERR_INVALID_ARG;
  if (n_dst < 1 || n_dst > DDD_MAX_SHARDS) return DDD_ERR_INVALID_ARG;
  for (int i = 0; i < n_dst; ++i) {
    if (!records_dst[i] || (flags_dst && !flags_dst[i])) return DDD_ERR_INVALID_ARG;
    if (!aligned16(records_dst[i])) return DDD_ERR_ALIGNMENT;
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (launch_lm_head(h, d, 0, false, st) != cudaSuccess ||
      launch_shard_reduce(h->p, d, slot, slots, records_dst, flags_dst, n_dst, shard_flag_value(h, d),
                          h->shard_counter, st) != cudaSuccess) {
    note_cuda_error(__LINE__);
    return DDD_ERR_CUDA;
  }
  return DDD_OK;
}

int ddd_shard_select(ddd_handle* h, int32_t d, const void* records, int32_t slots, const int32_t* flags,
                     void* cuda_stream) {
  if (!h || !h->shard_open || !records) return DDD_ERR_INVALID_ARG;
  if (d < 1 || d > h->p.n || slots < 1 || slots > DDD_MAX_SHARDS) return DDD_ERR_INVALID_ARG;
  if (!aligned16(records)) return DDD_ERR_ALIGNMENT;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e = cudaSuccess;
  if (flags) e = launch_shard_wait(flags, slots, shard_flag_value(h, d), h->p.dev_status, st);
  // the select kernel merges `slots` partials per row from the record set instead of one per thread block
  Params q = h->p;
  unsigned char* base = static_cast<unsigned char*>(const_cast<void*>(records));
  q.part_key = reinterpret_cast<unsigned long long*>(base);
  q.part_ms = reinterpret_cast<float2*>(base + (size_t)slots * q.R * q.k * sizeof(unsigned long long));
  q.lm_ctas = slots;
  if (e == cudaSuccess) e = launch_select(q, h->shard_io, d, false, 0, false, st);
  if (e != cudaSuccess) {
    note_cuda_error(__LINE__);
    return DDD_ERR_CUDA;
  }
  return DDD_OK;
}

int ddd_lm_head_pass(ddd_handle* h, void* cuda_stream) {
  if (!h) return DDD_ERR_INVALID_ARG;
  // Pass index 2 selects the hidden buffer written by the first draft step; all rows are forced live.
  if (launch_lm_head(h, 2, 1, h->use_pdl, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) {
    note_cuda_error(__LINE__);
    return DDD_ERR_CUDA;
  }
  return DDD_OK;
}

int ddd_launches_per_draft(const ddd_handle* h, int32_t passes_needed) {
  if (!h) return DDD_ERR_INVALID_ARG;
  const int n = h->p.n;
  int passes = n;
  if (h->cfg.launch_mode == DDD_LAUNCH_FUSED)      // the draft kernel and, where the rerank does not fit in it, the rerank kernel
    return fused_rerank_mode(h->p, h->tc) ? 1 : 2;
  if (h->cfg.launch_mode == DDD_LAUNCH_GRAPH) {
    const int nb = h->have_graph ? h->graph_bounds : h->n_bounds;
    for (int j = nb - 1; j >= 0; --j)
      if (passes_needed <= h->bounds[j]) passes = h->bounds[j];   // the group that holds the last needed pass
  }
  // init, then per launched pass LM head + select; for beams wider than 32 also the kernel between them
  // that makes one record per row, and the draft step of the new rows as a kernel behind the select
  return 1 + (h->p.k > 32 ? 4 : 2) * passes;
}

int ddd_lm_head_blocks(const ddd_handle* h) {
  if (!h) return DDD_ERR_INVALID_ARG;
  return h->p.lm_ctas;
}

int ddd_fused_pass_kind(const ddd_handle* h) {
  if (!h) return DDD_ERR_INVALID_ARG;
  if (h->cfg.launch_mode != DDD_LAUNCH_FUSED) return 0;
  return fused_pass_kind(h->p, h->tc);
}

int ddd_destroy(ddd_handle* h) {
  if (!h) return DDD_ERR_INVALID_ARG;
  if (h->exec) cudaGraphExecDestroy(h->exec);
  if (h->exec_host) cudaGraphExecDestroy(h->exec_host);
  if (h->bounce) cudaFreeHost(h->bounce);
  delete h;
  return DDD_OK;
}

const char* ddd_strerror(int code) {
  switch (code) {
    case DDD_OK: return "ok";
    case DDD_ERR_INVALID_ARG: return "invalid argument";
    case DDD_ERR_ALIGNMENT: return "pointer not aligned as required";
    case DDD_ERR_WORKSPACE: return "workspace too small";
    case DDD_ERR_CUDA: return "CUDA call failed";
    case DDD_ERR_TIMEOUT: return "a bounded wait inside a kernel ran out";
    case DDD_ERR_UNSUPPORTED: return "not supported by this build or device";
    default: return "unknown error code";
  }
}

}  // extern "C"
