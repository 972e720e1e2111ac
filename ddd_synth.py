"""Seeded synthetic inputs for the Dynamic Depth Decoding draft-tree path.

This module only *draws numbers*: weights, embeddings, biases, planted-token
tables and per-draft roots, each rounded to the storage dtype of the
configuration, plus random tree shapes and target choices for the verification
helpers.  It contains none of the method's arithmetic (no logits, no
softmax, no top-k, no search and no acceptance logic), so both the CPU oracle and the CUDA path can
be fed from it without sharing any computation.

The paper evaluates on MT-bench with Vicuna / LLaMA2-Chat targets and trained
EAGLE draft heads (Section 3.1).  None of that is available offline; the
configurations below stand in for it with tensors of the same shapes (hidden
4096 / 5120 / 8192, vocab 32000, plus a 128256-vocab variant) and simple,
stated value distributions.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, Optional

import numpy as np
import torch

CHECK_EVERY_STEP = 0xFFFFFFFF


@dataclasses.dataclass(frozen=True)
class DraftConfig:
    """One workload: Algorithm 1's parameters (n, w, S, x) plus tensor shapes."""

    name: str
    batch: int            # B independent sequences
    hidden: int           # Hd
    vocab: int            # V
    k: int                # beam width (the paper's w)
    max_depth: int        # maximum number of draft-model calls (the paper's n)
    total_tokens: int     # m: draft nodes kept by the final rerank (root is extra)
    dtype: str            # "fp32" or "bf16": storage type of W, E and hidden states
    threshold: float      # x: drafting continues iff H >= x
    check_mask: int = CHECK_EVERY_STEP  # bit (s-1) set <=> step s is in S
    logit_scale: float = 1.0
    rms_eps: float = 1e-6
    plant_delta: float = 0.0
    sigma_w: float = 0.02
    bias_kind: str = "none"      # "none" | "zipf"
    plant_frac: float = 0.0      # fraction of token ids that plant a confident successor
    seed: int = 0

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "fp32" else torch.bfloat16

    @property
    def n_max_nodes(self) -> int:
        """Non-root tree nodes after max_depth passes: k + (n-1) k^2."""
        return self.k + (self.max_depth - 1) * self.k * self.k

    @property
    def t_max(self) -> int:
        """Output rows per sequence: root + m."""
        return self.total_tokens + 1

    @property
    def mask_words(self) -> int:
        return (self.t_max + 31) // 32

    def replace(self, **kw) -> "DraftConfig":
        return dataclasses.replace(self, **kw)


def _scale_for_unit_rms_rows(sigma_w: float, hidden: int, target_std: float = 3.0) -> float:
    # Rows fed to the LM head have unit RMS, so a logit is a sum of `hidden`
    # products of variance sigma_w^2: choose s so that s*sigma_w*sqrt(hidden) = target.
    return target_std / (sigma_w * math.sqrt(hidden))


CONFIGS: Dict[str, DraftConfig] = {
    "tiny": DraftConfig(
        name="tiny", batch=1, hidden=256, vocab=1024, k=4, max_depth=4, total_tokens=16,
        dtype="fp32", threshold=-2.0, sigma_w=0.06, seed=0),
    "llama2_7b": DraftConfig(
        name="llama2_7b", batch=1, hidden=4096, vocab=32000, k=10, max_depth=12, total_tokens=60,
        dtype="bf16", threshold=-2.0, sigma_w=0.02,
        logit_scale=_scale_for_unit_rms_rows(0.02, 4096), seed=1),
    "vicuna_13b": DraftConfig(
        name="vicuna_13b", batch=1, hidden=5120, vocab=32000, k=10, max_depth=12, total_tokens=60,
        dtype="bf16", threshold=-2.0, sigma_w=0.02,
        logit_scale=_scale_for_unit_rms_rows(0.02, 5120),
        plant_frac=0.10, plant_delta=8.0, seed=2),
    "llama2_70b_b16": DraftConfig(
        name="llama2_70b_b16", batch=16, hidden=8192, vocab=32000, k=10, max_depth=10, total_tokens=60,
        dtype="bf16", threshold=-2.0, sigma_w=0.02,
        logit_scale=_scale_for_unit_rms_rows(0.02, 8192), seed=3),
    "llama3_8b_128k": DraftConfig(
        name="llama3_8b_128k", batch=4, hidden=4096, vocab=128256, k=16, max_depth=16, total_tokens=96,
        dtype="bf16", threshold=-3.0, sigma_w=0.02, logit_scale=1.0, bias_kind="zipf", seed=4),
}

# Thresholds the 7B-shaped workload is swept over.
LLAMA2_7B_THRESHOLDS = (-1.0, -2.0, -4.0)


def scaled_down(cfg: DraftConfig, hidden: int, vocab: int, **kw) -> DraftConfig:
    """Same distributions and search parameters on a smaller LM head.

    The logit scale is recomputed so that per-row logit std stays where the
    full-size configuration puts it.
    """
    scale = cfg.logit_scale
    if cfg.logit_scale != 1.0:
        scale = _scale_for_unit_rms_rows(cfg.sigma_w, hidden)
    return cfg.replace(name=f"{cfg.name}_h{hidden}_v{vocab}", hidden=hidden, vocab=vocab,
                       logit_scale=scale, **kw)


def _normal(rng: np.random.Generator, shape, sigma: float, dtype: torch.dtype) -> torch.Tensor:
    # Drawn in fp32 in row chunks to bound peak host memory, then rounded once
    # to the storage dtype (round-to-nearest-even, done by torch).
    rows, cols = shape
    out = torch.empty((rows, cols), dtype=dtype)
    step = max(1, (1 << 25) // max(cols, 1))
    for r0 in range(0, rows, step):
        r1 = min(rows, r0 + step)
        blk = rng.standard_normal((r1 - r0, cols), dtype=np.float32)
        if sigma != 1.0:
            blk *= np.float32(sigma)
        out[r0:r1] = torch.from_numpy(blk).to(dtype)
    return out


def make_weights(cfg: DraftConfig) -> Dict[str, Optional[torch.Tensor]]:
    """Draw W [V][Hd], E [V][Hd], bias [V] (or None) and plant_next [V] (or None).

    Everything is a CPU tensor; W and E are already in the storage dtype.
    """
    rng = np.random.default_rng([cfg.seed, 0x5EED])
    W = _normal(rng, (cfg.vocab, cfg.hidden), cfg.sigma_w, cfg.torch_dtype)
    E = _normal(rng, (cfg.vocab, cfg.hidden), 1.0, cfg.torch_dtype)
    bias = None
    if cfg.bias_kind == "zipf":
        # Zipf(1.1)-like skew over token ids: log-weight of id v is -1.1 ln(v+1).
        v = np.arange(cfg.vocab, dtype=np.float64)
        bias = torch.from_numpy((-1.1 * np.log(v + 1.0)).astype(np.float32))
    elif cfg.bias_kind != "none":
        raise ValueError(f"unknown bias_kind {cfg.bias_kind!r}")
    plant_next = None
    if cfg.plant_frac > 0.0:
        # A fixed fraction of token ids "plant" one confident successor token:
        # a row whose last token is such an id gets one logit lifted above the rest.
        chosen = rng.random(cfg.vocab) < cfg.plant_frac
        target = rng.integers(0, cfg.vocab, size=cfg.vocab, dtype=np.int64)
        table = np.where(chosen, target, -1).astype(np.int32)
        plant_next = torch.from_numpy(table)
    return {"W": W, "E": E, "bias": bias, "plant_next": plant_next}


def make_roots(cfg: DraftConfig, draft_index: int) -> Dict[str, torch.Tensor]:
    """Per-draft inputs: root hidden [B][Hd], root token [B], root position [B]."""
    rng = np.random.default_rng([cfg.seed, 0xD0A7, int(draft_index)])
    h = rng.standard_normal((cfg.batch, cfg.hidden), dtype=np.float32)
    tok = rng.integers(0, cfg.vocab, size=cfg.batch, dtype=np.int64).astype(np.int32)
    pos = rng.integers(1, 2048, size=cfg.batch, dtype=np.int64).astype(np.int32)
    return {
        "root_hidden": torch.from_numpy(h).to(cfg.torch_dtype),
        "root_token": torch.from_numpy(tok),
        "root_pos": torch.from_numpy(pos),
    }


def random_tree(rng: np.random.Generator, n_rows: int, vocab: int, max_children: int = 4):
    """A random emitted tree for the verification helpers: rows in generation order (row 0 the
    root, every parent row below its child's), the tokens of siblings distinct.
    Returns (token [n_rows], parent [n_rows]) as int64 arrays."""
    max_children = min(max_children, vocab)
    parent, token = [-1], [int(rng.integers(vocab))]
    used = {0: set()}
    for i in range(1, n_rows):
        while True:
            p = int(rng.integers(i))
            if len(used[p]) < max_children:
                break
        t = int(rng.integers(vocab))
        while t in used[p]:
            t = int(rng.integers(vocab))
        used[p].add(t)
        used[i] = set()
        parent.append(p)
        token.append(t)
    return np.array(token, dtype=np.int64), np.array(parent, dtype=np.int64)


def target_choices_along(rng: np.random.Generator, token, parent, n_rows: int, goal_row: int, vocab: int):
    """Synthetic target choices [n_rows] for a tree: along the root path of `goal_row` the target
    picks the path's next token, everywhere else a random token of the vocabulary (which may or
    may not be some child's token)."""
    target = rng.integers(vocab, size=n_rows).astype(np.int64)
    r = int(goal_row)
    while r > 0:
        target[int(parent[r])] = int(token[r])
        r = int(parent[r])
    return target


def shard_draft_indices(n_drafts: int, rank: int, world_size: int):
    """Contiguous block of draft indices owned by `rank` (replica sharding).

    Drafts are independent problems, so ranks never exchange data; the first
    `n_drafts % world_size` ranks take one extra draft.
    """
    if not (0 <= rank < world_size):
        raise ValueError("rank out of range")
    base, extra = divmod(n_drafts, world_size)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))
