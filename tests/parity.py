"""Helpers shared by the GPU parity tests: run a draft through the C ABI, replay its
decisions in the CPU oracle and compare element by element.

Tolerances (absolute): logprobs, cumulative scores, H and row logsumexp within 2e-3;
tokens, parents, depths, positions, node ids and masks bit-exact, where a choice that
differs from the oracle's own only inside a 2e-3 near-tie band is adopted by the replay.
"""
from __future__ import annotations

import numpy as np
import torch

import ddd_synth as S
from oracle import ddd_oracle as O

TOL = 2e-3


def to_device(roots, device):
    return {k: v.to(device) for k, v in roots.items()}


def run_gpu(engine, roots):
    dev = to_device(roots, engine.device)
    engine.draft(dev["root_hidden"], dev["root_token"], dev["root_pos"])
    res = engine.results()
    assert int(res["status"][0]) == 0, f"device status {int(res['status'][0])}"
    assert engine.guards_intact(), "a kernel wrote outside the workspace"
    return {k: v.numpy() for k, v in res.items()}


def follow_from_gpu(cfg, g):
    out = []
    for b in range(cfg.batch):
        D = int(g["stop_depth"][b])
        assert 1 <= D <= cfg.max_depth
        out.append(O.FollowSequence(
            stop_depth=D, tree_token=g["tree_token"][b].astype(np.int64),
            beam_sel=[g["beam_sel"][b, d].tolist() for d in range(D)],
            node_id=g["node_id"][b][: int(g["n_out"][b])].astype(np.int64)))
    return out


def mask_bits(words_row):
    bits = 0
    for w, word in enumerate(words_row):
        bits |= (int(word) & 0xFFFFFFFF) << (32 * w)
    return bits


def compare_with_oracle(cfg, weights, roots, g, strict=False):
    """Asserts parity of GPU results `g` with the oracle; returns the oracle results."""
    follow = None if strict else follow_from_gpu(cfg, g)
    ref = O.draft(cfg, weights, roots["root_hidden"], roots["root_token"], roots["root_pos"],
                  follow=follow, tol=TOL)
    k, n, T = cfg.k, cfg.max_depth, cfg.total_tokens + 1
    for b, r in enumerate(ref):
        assert not r.violations, (b, r.violations[:3])
        D = r.stop_depth
        assert int(g["stop_depth"][b]) == D, (b, int(g["stop_depth"][b]), D, r.H_trace, r.ambiguities)
        N = k + (D - 1) * k * k
        n_out = r.n_out
        assert int(g["n_out"][b]) == n_out == 1 + min(cfg.total_tokens, N)
        # the search itself
        np.testing.assert_array_equal(g["tree_token"][b][: N + 1], r.tree_token[: N + 1])
        np.testing.assert_array_equal(g["tree_parent"][b][: N + 1], r.tree_parent[: N + 1])
        np.testing.assert_allclose(g["tree_cum"][b][: N + 1], r.tree_cum[: N + 1], rtol=0, atol=TOL)
        for d in range(D):
            assert g["beam_sel"][b, d].tolist() == r.beam_sel[d]
            P = 1 if d == 0 else k
            np.testing.assert_allclose(g["row_lse"][b, d, :P], r.row_lse[d], rtol=0, atol=TOL)
        np.testing.assert_allclose(g["H_trace"][b, :D], np.array(r.H_trace), rtol=0, atol=TOL)
        # the emitted tree
        np.testing.assert_array_equal(g["node_id"][b][:n_out], r.node_id)
        np.testing.assert_array_equal(g["token"][b][:n_out], r.token)
        np.testing.assert_array_equal(g["parent"][b][:n_out], r.parent)
        np.testing.assert_array_equal(g["depth"][b][:n_out], r.depth)
        np.testing.assert_array_equal(g["position"][b][:n_out], r.position)
        np.testing.assert_allclose(g["cum"][b][:n_out], r.cum, rtol=0, atol=TOL)
        for i in range(n_out):
            assert mask_bits(g["mask"][b, i]) == r.mask[i], (b, i)
        # padding rows
        assert (g["token"][b][n_out:] == -1).all() and (g["parent"][b][n_out:] == -1).all()
        assert (g["depth"][b][n_out:] == -1).all() and (g["position"][b][n_out:] == -1).all()
        assert (g["cum"][b][n_out:] == 0).all() and (g["mask"][b][n_out:] == 0).all()
        # properties that hold at any size
        cum = g["cum"][b][:n_out]
        par = g["parent"][b][:n_out]
        assert (cum[1:] <= cum[par[1:]] + 0.0).all()          # monotone along every path
        assert (par[1:] < np.arange(1, n_out)).all()
    return ref


def strict_equal_when_unambiguous(cfg, weights, roots, g):
    """With no near-tie anywhere the oracle's own choices must equal the GPU's bit for bit."""
    ref = O.draft(cfg, weights, roots["root_hidden"], roots["root_token"], roots["root_pos"])
    checked = 0
    for b, r in enumerate(ref):
        if r.ambiguities:
            continue
        checked += 1
        D = r.stop_depth
        N = cfg.k + (D - 1) * cfg.k ** 2
        assert int(g["stop_depth"][b]) == D
        np.testing.assert_array_equal(g["tree_token"][b][: N + 1], r.tree_token[: N + 1])
        np.testing.assert_array_equal(g["node_id"][b][: r.n_out], r.node_id)
        np.testing.assert_array_equal(g["parent"][b][: r.n_out], r.parent)
        for i in range(r.n_out):
            assert mask_bits(g["mask"][b, i]) == r.mask[i]
    return checked
