"""CPU parity oracle for the Dynamic Depth Decoding draft-tree path.

TEST INFRASTRUCTURE ONLY.  Only tests, the smoke check and the CPU-baseline leg
of the benchmark may import this module; the product path never does, and this
module imports nothing from the CUDA package.  Everything is fp64 on the exact
values of the stored-dtype inputs, written step by step in the order of the
paper's Algorithm 1, with no blocking, fusion or reordering.

The method is a heuristic search (a beam search with a stopping rule), so the
oracle *is* the algorithm:

  * draft-model call        - Section 1 (embedding + head + the target's LM head);
                              Algorithm 1 "Run draft model on prompt / on beam".
                              The trainable head is replaced by the synthetic
                              recurrence h_child = RMSNorm(h_parent + E[token]).
  * log-softmax             - Section 2 (draft output goes through logsoftmax).
  * beam postprocess        - Section 1 (top-k token sequences by summed logprob)
                              and Algorithm 1 "Postprocess ... to produce the new beam".
  * logprobsum update       - Algorithm 1 (add parent's logprobsum to the new logprobs).
  * heuristic H and gate    - Eq. 1 and Algorithm 1's "if H < x: break".
  * rerank / tree mask      - Section 1 (the whole tree is fed to the target with an
                              adjusted attention mask); the top-m rule is this
                              library's stated reading, the paper leaves it to EAGLE-2.
  * acceptance walk         - Section 1 (the target verifies the tree in one call; at
                              temperature 0 a draft token is accepted iff it is the
                              target's own choice after its parent) and the root-to-leaf
                              path table of the emitted tree.

Parity status: every function below is pinned by tests in tests/test_oracle_pins.py
(brute-force path enumeration, closed forms, invariants, library routines).
"""
from __future__ import annotations

import ctypes
import dataclasses
import math
import os
import subprocess
from typing import Dict, List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "_build", "libddd_ref.so")
_LIB = None


# --------------------------------------------------------------------------- build / load
def build(force: bool = False) -> str:
    """Compile oracle/lm_head_ref.c into oracle/_build/libddd_ref.so (gcc, OpenMP)."""
    src = os.path.join(_HERE, "lm_head_ref.c")
    if (not force and os.path.exists(_LIB_PATH)
            and os.path.getmtime(_LIB_PATH) >= os.path.getmtime(src)):
        return _LIB_PATH
    os.makedirs(os.path.dirname(_LIB_PATH), exist_ok=True)
    tmp = _LIB_PATH + f".{os.getpid()}.tmp"
    subprocess.run(["gcc", "-O3", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
                    "-o", tmp, src], check=True)
    os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _lib():
    global _LIB
    if _LIB is None:
        lib = ctypes.CDLL(build())
        lib.ddd_ref_logits.restype = ctypes.c_int
        lib.ddd_ref_logits.argtypes = [
            ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_int64,
            ctypes.c_void_p, ctypes.c_int, ctypes.c_double, ctypes.c_void_p, ctypes.c_void_p]
        lib.ddd_ref_num_threads.restype = ctypes.c_int
        _LIB = lib
    return _LIB


def num_threads() -> int:
    return int(_lib().ddd_ref_num_threads())


# --------------------------------------------------------------------------- storage dtypes
def _raw_matrix(t):
    """(pointer-holder ndarray, is_bf16) for a CPU torch tensor or ndarray of fp32 / bf16."""
    import torch
    if isinstance(t, np.ndarray):
        if t.dtype == np.float32:
            return np.ascontiguousarray(t), 0
        if t.dtype == np.uint16:          # raw bf16 bit patterns
            return np.ascontiguousarray(t), 1
        raise TypeError(f"unsupported ndarray dtype {t.dtype}")
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.float32:
        return t.numpy(), 0
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16), 1
    raise TypeError(f"unsupported tensor dtype {t.dtype}")


def to_f64(t) -> np.ndarray:
    """Exact widening of stored values (fp32 / bf16 / ints) to fp64."""
    import torch
    if isinstance(t, np.ndarray):
        if t.dtype == np.uint16:
            return (t.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
        return t.astype(np.float64)
    return t.detach().cpu().to(torch.float64).numpy()


def round_to_storage(y: np.ndarray, dtype: str) -> np.ndarray:
    """Round fp64 values once to the storage dtype, result held in fp64.

    bf16 keeps 8 significant bits; rounding is to nearest, ties to even, done
    directly from fp64 (normal range only - hidden states have unit RMS).
    """
    y = np.asarray(y, dtype=np.float64)
    if dtype == "fp32":
        return y.astype(np.float32).astype(np.float64)
    if dtype == "bf16":
        mant, expo = np.frexp(y)                 # y = mant * 2**expo, 0.5 <= |mant| < 1
        return np.ldexp(np.rint(mant * 256.0), expo - 8)   # np.rint: ties to even
    raise ValueError(dtype)


# --------------------------------------------------------------------------- the steps
def lm_head_logits(W, h: np.ndarray, scale: float, bias: Optional[np.ndarray]) -> np.ndarray:
    """z[r][v] = s * <W[v], h[r]> + bias[v]; sequential fp64 dots (see lm_head_ref.c)."""
    Wn, is_bf16 = _raw_matrix(W)
    vocab, hidden = Wn.shape
    h = np.asarray(h, dtype=np.float64)
    assert h.ndim == 2 and h.shape[1] == hidden
    rows = h.shape[0]
    hT = np.ascontiguousarray(h.T)
    z = np.empty((rows, vocab), dtype=np.float64)
    b = None if bias is None else np.ascontiguousarray(bias, dtype=np.float64)
    rc = _lib().ddd_ref_logits(
        Wn.ctypes.data, is_bf16, vocab, hidden, hT.ctypes.data, rows, float(scale),
        None if b is None else b.ctypes.data, z.ctypes.data)
    if rc != 0:
        raise RuntimeError(f"ddd_ref_logits failed ({rc})")
    return z


def apply_plant(z_row: np.ndarray, column: int, delta: float) -> np.ndarray:
    """Replace one logit by (max of the row's other logits) + delta."""
    z_row = z_row.copy()
    if column >= 0:
        others = np.delete(z_row, column)
        z_row[column] = others.max() + delta
    return z_row


def log_softmax_row(z_row: np.ndarray) -> np.ndarray:
    """logprob = z - (M + log sum exp(z - M)), clamped to <= 0 (Section 2)."""
    M = z_row.max()
    lse = M + math.log(np.exp(z_row - M).sum())
    return np.minimum(z_row - lse, 0.0)


def topk_desc(scores: np.ndarray, k: int) -> np.ndarray:
    """Indices of the k largest scores, order (score desc, index asc); full stable sort."""
    order = np.argsort(-np.asarray(scores, dtype=np.float64), kind="stable")
    return order[:k]


def heuristic_H(logprobsum: Sequence[float]) -> float:
    """Eq. 1: H = log sum_i exp(logprobsum[i]) over the w beam entries (max-shifted)."""
    a = np.asarray(logprobsum, dtype=np.float64)
    M = a.max()
    return float(M + math.log(np.exp(a - M).sum()))


def draft_step(h_parent: np.ndarray, e_row: np.ndarray, eps: float, dtype: str) -> np.ndarray:
    """h_child = round_to_storage( u / sqrt(mean(u^2) + eps) ),  u = h_parent + E[token]."""
    u = h_parent + e_row
    y = u / math.sqrt(float(np.mean(u * u)) + eps)
    return round_to_storage(y, dtype)


def rerank(cum: np.ndarray, m: int) -> np.ndarray:
    """Ids (ascending) of the top-min(m, N) non-root nodes by (cum desc, node id asc).

    `cum[i]` belongs to node id i+1 (node 0 is the root and is not ranked).
    """
    n = len(cum)
    chosen = topk_desc(cum, min(m, n)) + 1
    return np.sort(chosen)


def tree_mask_rows(parent_slot: Sequence[int]) -> List[int]:
    """mask[i] = mask[parent(i)] | bit i, mask[0] = bit 0 (python ints as bit sets)."""
    rows: List[int] = []
    for i, p in enumerate(parent_slot):
        rows.append((1 << i) if p < 0 else (rows[p] | (1 << i)))
    return rows


# --------------------------------------------------------------------------- admissibility (replay)
def admissible_topk(scores: np.ndarray, chosen: Sequence[int], k: int, tol: float,
                    ordered: bool = True) -> List[str]:
    """Check an externally supplied top-k against fp64 scores.

    Accepts any choice that differs from the exact one only inside +-tol bands:
      * every chosen entry scores >= (exact k-th best) - tol,
      * every entry scoring > (exact k-th best) + tol is chosen,
      * if `ordered`, the supplied order is non-increasing up to tol.
    Returns a list of violation messages (empty if admissible).
    """
    scores = np.asarray(scores, dtype=np.float64)
    chosen = [int(c) for c in chosen]
    bad: List[str] = []
    if len(chosen) != k or len(set(chosen)) != k:
        return [f"expected {k} distinct entries, got {chosen}"]
    if min(chosen) < 0 or max(chosen) >= len(scores):
        return [f"entry out of range in {chosen}"]
    kth = np.sort(scores)[::-1][k - 1]
    cs = scores[chosen]
    if (cs < kth - tol).any():
        bad.append(f"chosen entry below k-th best - tol: {cs.min()} < {kth} - {tol}")
    must = np.nonzero(scores > kth + tol)[0]
    missing = set(must.tolist()) - set(chosen)
    if missing:
        bad.append(f"entries clearly above the k-th best not chosen: {sorted(missing)[:5]}")
    if ordered and (np.diff(cs) > tol).any():
        bad.append("order is not non-increasing within tol")
    return bad


# --------------------------------------------------------------------------- results
@dataclasses.dataclass
class SequenceResult:
    stop_depth: int
    H_trace: List[float]                  # H after pass d (index d-1), every executed pass
    tree_token: np.ndarray                # [N+1] int64, node 0 = root
    tree_parent: np.ndarray               # [N+1] node id of parent, root -1
    tree_depth: np.ndarray                # [N+1]
    tree_cum: np.ndarray                  # [N+1] fp64
    beam_sel: List[List[int]]             # per pass: flat candidate indices p*k+c of the new beam
    row_lse: List[np.ndarray]             # per pass: logsumexp of each beam row's logits
    n_out: int = 0
    node_id: np.ndarray = None            # [n_out] tree node id per output slot
    token: np.ndarray = None
    parent: np.ndarray = None             # output-slot index of the parent, root -1
    depth: np.ndarray = None
    position: np.ndarray = None
    cum: np.ndarray = None
    mask: List[int] = None                # python-int bit sets, one per output slot
    violations: List[str] = dataclasses.field(default_factory=list)
    ambiguities: List[str] = dataclasses.field(default_factory=list)


@dataclasses.dataclass
class FollowSequence:
    """Decisions taken by another implementation, for replay (one sequence)."""
    stop_depth: int
    tree_token: np.ndarray                # [N+1]; row top-k tokens in its own order
    beam_sel: Sequence[Sequence[int]]     # per executed pass
    node_id: Optional[np.ndarray] = None  # reranked node ids (ascending, root first)


def first_node_of_pass(d: int, k: int) -> int:
    """Node id of candidate (p=0, c=0) generated by pass d: 1, then 1 + k + (d-2) k^2."""
    return 1 if d == 1 else 1 + k + (d - 2) * k * k


def _margin_note(scores: np.ndarray, k: int, tol: float, ordered: bool = True) -> Optional[str]:
    """Describes a near-tie that makes more than one answer acceptable, or None.

    For an ordered top-k any two neighbours among the best k+1 scores closer than tol may
    legally swap; for an unordered selection only the k-th / (k+1)-th boundary matters.
    """
    s = np.sort(np.asarray(scores, dtype=np.float64))[::-1]
    if len(s) > k and s[k - 1] - s[k] < tol:
        return f"k-th and (k+1)-th differ by {s[k - 1] - s[k]:.3e}"
    if ordered:
        gaps = -np.diff(s[:k])
        if len(gaps) and gaps.min() < tol:
            return f"two of the best k differ by {gaps.min():.3e}"
    return None


def draft(cfg, weights: Dict, root_hidden, root_token, root_pos,
          follow: Optional[Sequence[FollowSequence]] = None, tol: float = 2e-3
          ) -> List[SequenceResult]:
    """Run Algorithm 1 for every sequence of the batch; returns one result per sequence.

    `cfg` needs: batch, hidden, vocab, k, max_depth, total_tokens, dtype, threshold,
    check_mask, logit_scale, rms_eps, plant_delta.  `weights` holds W, E, bias,
    plant_next.  With `follow`, each decision of the other implementation is first
    checked for admissibility (recorded in `violations`) and then adopted, so one
    legal near-tie swap does not make everything downstream differ.
    """
    B, k, n, m = cfg.batch, cfg.k, cfg.max_depth, cfg.total_tokens
    W, E = weights["W"], weights["E"]
    bias = None if weights.get("bias") is None else to_f64(weights["bias"])
    plant_next = weights.get("plant_next")
    plant_next = None if plant_next is None else np.asarray(plant_next).astype(np.int64)
    root_hidden = to_f64(root_hidden).reshape(B, cfg.hidden)
    root_token = np.asarray(root_token).astype(np.int64).reshape(B)
    root_pos = np.asarray(root_pos).astype(np.int64).reshape(B)
    n_nodes = 1 + k + (n - 1) * k * k

    res: List[SequenceResult] = []
    for b in range(B):
        r = SequenceResult(
            stop_depth=0, H_trace=[],
            tree_token=np.full(n_nodes, -1, np.int64), tree_parent=np.full(n_nodes, -1, np.int64),
            tree_depth=np.zeros(n_nodes, np.int64), tree_cum=np.zeros(n_nodes, np.float64),
            beam_sel=[], row_lse=[])
        r.tree_token[0] = root_token[b]
        res.append(r)

    # Beam state per sequence: hidden rows, node ids, logprobsum.  Pass 1 has one row: the root.
    beam_h = [root_hidden[b:b + 1].copy() for b in range(B)]
    beam_node = [np.array([0], np.int64) for _ in range(B)]
    beam_cum = [np.array([0.0]) for _ in range(B)]
    active = [True] * B

    for d in range(1, n + 1):
        live = [b for b in range(B) if active[b]]
        if not live:
            break
        # ---- run the draft model's LM head on every live beam row (one call, rows stacked)
        rows = np.concatenate([beam_h[b] for b in live], axis=0)
        z_all = lm_head_logits(W, rows, cfg.logit_scale, bias)
        offset = 0
        for b in live:
            r = res[b]
            P = beam_h[b].shape[0]
            z = z_all[offset:offset + P]
            offset += P
            base = first_node_of_pass(d, k)
            cand = np.empty(P * k)
            lses = np.empty(P)
            for p in range(P):
                zp = z[p]
                if plant_next is not None:
                    last_tok = int(r.tree_token[beam_node[b][p]])
                    zp = apply_plant(zp, int(plant_next[last_tok]), cfg.plant_delta)
                lp = log_softmax_row(zp)
                M = zp.max()
                lses[p] = M + math.log(np.exp(zp - M).sum())
                # ---- per-beam top-k tokens
                if follow is not None:
                    ids = base + p * k + np.arange(k)
                    top = np.asarray(follow[b].tree_token[ids]).astype(np.int64)
                    for msg in admissible_topk(lp, top, k, tol):
                        r.violations.append(f"pass {d} row {p} token top-k: {msg}")
                    if r.violations:
                        top = np.clip(top, 0, cfg.vocab - 1)
                else:
                    top = topk_desc(lp, k)
                note = _margin_note(lp, k, tol)
                if note:
                    r.ambiguities.append(f"pass {d} row {p} token top-k: {note}")
                # ---- logprobsum of each candidate; every candidate becomes a tree node
                for c in range(k):
                    node = base + p * k + c
                    r.tree_token[node] = top[c]
                    r.tree_parent[node] = beam_node[b][p]
                    r.tree_depth[node] = d
                    r.tree_cum[node] = beam_cum[b][p] + lp[top[c]]
                    cand[p * k + c] = r.tree_cum[node]
            r.row_lse.append(lses)
            # ---- new beam = top-k of the P*k candidates
            if follow is not None:
                sel = np.asarray(follow[b].beam_sel[d - 1]).astype(np.int64)
                for msg in admissible_topk(cand, sel, k, tol):
                    r.violations.append(f"pass {d} beam top-k: {msg}")
                if r.violations:
                    sel = np.clip(sel, 0, P * k - 1)
            else:
                sel = topk_desc(cand, k)
            note = _margin_note(cand, k, tol)
            if note:
                r.ambiguities.append(f"pass {d} beam top-k: {note}")
            r.beam_sel.append([int(s) for s in sel])
            new_node = base + sel
            new_cum = cand[sel]
            # ---- heuristic and gate (the check after `d` draft calls, before call d+1)
            H = heuristic_H(new_cum)
            r.H_trace.append(H)
            stop = False
            if d == n:
                stop = True
            elif (cfg.check_mask >> (d - 1)) & 1:
                stop = H < cfg.threshold
                if abs(H - cfg.threshold) < tol:
                    r.ambiguities.append(f"pass {d} gate: |H - x| = {abs(H - cfg.threshold):.3e}")
                if follow is not None:
                    theirs = follow[b].stop_depth == d
                    if theirs != stop and abs(H - cfg.threshold) >= tol:
                        r.violations.append(
                            f"pass {d} gate: H={H:.6f} x={cfg.threshold} but other side "
                            f"{'stopped' if theirs else 'continued'}")
                    stop = theirs
            elif follow is not None and follow[b].stop_depth == d:
                r.violations.append(f"pass {d} gate: other side stopped at a step outside S")
            if stop:
                r.stop_depth = d
                active[b] = False
                continue
            # ---- draft step: next hidden rows of the new beam
            parent_slot = sel // k
            Etok = to_f64(E[np.asarray(r.tree_token[new_node])])
            beam_h[b] = np.stack([
                draft_step(beam_h[b][parent_slot[i]], Etok[i], cfg.rms_eps, cfg.dtype)
                for i in range(k)])
            beam_node[b] = new_node
            beam_cum[b] = new_cum

    # ---- final rerank, positions and tree mask
    for b in range(B):
        r = res[b]
        D = r.stop_depth
        N = k + (D - 1) * k * k
        cum = r.tree_cum[1:N + 1]
        if follow is not None and follow[b].node_id is not None:
            ids = np.asarray(follow[b].node_id).astype(np.int64)
            ids = ids[ids > 0]
            for msg in admissible_topk(cum, ids - 1, min(m, N), tol, ordered=False):
                r.violations.append(f"rerank: {msg}")
            if (np.diff(ids) <= 0).any():
                r.violations.append("rerank: node ids not strictly ascending")
            chosen = ids if not r.violations else rerank(cum, m)
        else:
            chosen = rerank(cum, m)
        note = _margin_note(cum, min(m, N), tol, ordered=False)
        if note:
            r.ambiguities.append(f"rerank: {note}")
        node_id = np.concatenate([[0], chosen]).astype(np.int64)
        slot_of = {int(nid): i for i, nid in enumerate(node_id)}
        r.n_out = len(node_id)
        r.node_id = node_id
        r.token = r.tree_token[node_id]
        r.parent = np.array([-1 if nid == 0 else slot_of.get(int(r.tree_parent[nid]), -2)
                             for nid in node_id], np.int64)
        if (r.parent == -2).any():
            r.violations.append("rerank: selected set is not ancestor-closed")
            r.parent[r.parent == -2] = 0
        r.depth = r.tree_depth[node_id]
        r.position = root_pos[b] + r.depth
        r.cum = r.tree_cum[node_id]
        r.mask = tree_mask_rows(r.parent)
    return res


def greedy_accept(token: Sequence[int], parent: Sequence[int], n_out: int,
                  target_argmax: Sequence[int]):
    """Section 1, verification at temperature 0.  Rows 0..n_out-1 are a tree (row 0 the root,
    parent[i] the parent's row).  target_argmax[i] is the target's choice of the token that
    follows row i.  Starting at the root, the child of the current row that carries exactly that
    token is accepted and becomes the current row; the walk ends when no child does.
    Returns (accepted rows in order, the target's token after the last accepted row)."""
    cur = 0
    accepted: List[int] = []
    while True:
        want = int(target_argmax[cur])
        nxt = -1
        for i in range(1, n_out):
            if int(parent[i]) == cur and int(token[i]) == want:
                nxt = i
                break
        if nxt < 0:
            return accepted, want
        accepted.append(nxt)
        cur = nxt


def leaf_paths(parent: Sequence[int], n_out: int) -> List[List[int]]:
    """Root-to-leaf row lists of the emitted tree, one per leaf, leaves in ascending row order.
    A leaf is a row that no emitted row names as its parent."""
    has_child = [False] * n_out
    for i in range(1, n_out):
        has_child[int(parent[i])] = True
    paths = []
    for leaf in range(n_out):
        if has_child[leaf]:
            continue
        path = []
        r = leaf
        while r >= 0:
            path.append(r)
            r = int(parent[r])
        paths.append(path[::-1])
    return paths


def mask_words(mask_rows: Sequence[int], t_max: int) -> np.ndarray:
    """Bit-packed mask [t_max][ceil(t_max/32)] uint32, bit j of row i in word j//32, LSB first."""
    w32 = (t_max + 31) // 32
    out = np.zeros((t_max, w32), np.uint32)
    for i, bits in enumerate(mask_rows):
        for w in range(w32):
            out[i, w] = (bits >> (32 * w)) & 0xFFFFFFFF
    return out
