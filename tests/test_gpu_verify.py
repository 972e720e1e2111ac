"""GPU parity of the verification helpers (greedy acceptance walk, leaf-path table): the CUDA
kernel behind ddd_verify_greedy against the CPU oracle, bit for bit (pure index work)."""
import numpy as np
import pytest
import torch

import ddd_synth as S
import paper_2409_00142_b200 as P
from oracle import ddd_oracle as O
from tests import parity

pytestmark = pytest.mark.gpu


def _run_abi(token, parent, n_out, target, max_depth):
    """token/parent/target: int arrays [B][T]; n_out [B].  Calls ddd_verify_greedy directly."""
    dev = torch.device("cuda", 0)
    B, T = token.shape
    i32 = torch.int32
    t = {name: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
         for name, a in (("token", token), ("parent", parent), ("n_out", n_out), ("target", target))}
    out = {
        "n_accepted": torch.full((B,), -9, dtype=i32, device=dev),
        "accepted_rows": torch.full((B, max_depth), -9, dtype=i32, device=dev),
        "next_token": torch.full((B,), -9, dtype=i32, device=dev),
        "n_leaves": torch.full((B,), -9, dtype=i32, device=dev),
        "leaf_paths": torch.full((B, T, max_depth + 1), -9, dtype=i32, device=dev),
        "status": torch.full((1,), -9, dtype=i32, device=dev),
    }
    c_out = P.DddVerifyOutput(**{name: x.data_ptr() for name, x in out.items()})
    P.ddd_verify_greedy(B, T, max_depth, t["n_out"].data_ptr(), t["token"].data_ptr(), t["parent"].data_ptr(),
                        t["target"].data_ptr(), c_out, torch.cuda.current_stream(dev).cuda_stream)
    torch.cuda.synchronize(dev)
    return {name: x.cpu().numpy() for name, x in out.items()}


def _check_against_oracle(g, token, parent, n_out, target, max_depth):
    B, T = token.shape
    assert int(g["status"][0]) == 0
    for b in range(B):
        n = int(n_out[b])
        accepted, nxt = O.greedy_accept(token[b], parent[b], n, target[b])
        assert int(g["n_accepted"][b]) == len(accepted), b
        want = np.full(max_depth, -1)
        want[: len(accepted)] = accepted
        np.testing.assert_array_equal(g["accepted_rows"][b], want)
        assert int(g["next_token"][b]) == nxt
        paths = O.leaf_paths(parent[b], n)
        assert int(g["n_leaves"][b]) == len(paths)
        table = np.full((T, max_depth + 1), -1)
        for l, path in enumerate(paths):
            table[l, : len(path)] = path
        np.testing.assert_array_equal(g["leaf_paths"][b], table)


def _depth_of(parent):
    depth = np.zeros(len(parent), dtype=np.int64)
    for i in range(1, len(parent)):
        depth[i] = depth[parent[i]] + 1
    return depth


@pytest.mark.parametrize("T,batch,vocab", [(1, 1, 8), (2, 3, 4), (61, 5, 6), (257, 4, 9), (1024, 2, 5)])
def test_random_trees_match_oracle(T, batch, vocab):
    rng = np.random.default_rng([T, batch, vocab])
    token = np.full((batch, T), -1, dtype=np.int64)
    parent = np.full((batch, T), -1, dtype=np.int64)
    target = np.zeros((batch, T), dtype=np.int64)
    n_out = np.zeros(batch, dtype=np.int64)
    max_depth = 1
    for b in range(batch):
        n = T if b == 0 else int(rng.integers(1, T + 1))           # ragged: fewer rows than T
        tok, par = S.random_tree(rng, n, vocab, max_children=3)
        token[b, :n], parent[b, :n], n_out[b] = tok, par, n
        goal = int(rng.integers(n))
        target[b, :n] = S.target_choices_along(rng, tok, par, n, goal, vocab)
        max_depth = max(max_depth, int(_depth_of(par).max()))
    max_depth = min(max_depth, 32)
    # rows deeper than the limit cannot occur in a drafted tree: rebuild those cases shallower
    for b in range(batch):
        n = int(n_out[b])
        while int(_depth_of(parent[b, :n]).max()) > max_depth:
            tok, par = S.random_tree(rng, n, vocab, max_children=3)
            token[b, :n], parent[b, :n] = tok, par
            target[b, :n] = S.target_choices_along(rng, tok, par, n, int(rng.integers(n)), vocab)
    g = _run_abi(token, parent, n_out, target, max_depth)
    _check_against_oracle(g, token, parent, n_out, target, max_depth)
    # second call into the same buffers: nothing is left over from the first
    g2 = _run_abi(token, parent, n_out, target, max_depth)
    for name in g:
        np.testing.assert_array_equal(g[name], g2[name])


def test_chain_accepts_every_token_and_nothing():
    n = 12
    token = np.arange(50, 50 + n)[None, :]
    parent = np.arange(-1, n - 1)[None, :]
    n_out = np.array([n])
    all_of_it = np.append(token[0, 1:], 999)[None, :]
    g = _run_abi(token, parent, n_out, all_of_it, n - 1)
    assert int(g["n_accepted"][0]) == n - 1 and int(g["next_token"][0]) == 999
    np.testing.assert_array_equal(g["accepted_rows"][0], np.arange(1, n))
    assert int(g["n_leaves"][0]) == 1
    np.testing.assert_array_equal(g["leaf_paths"][0, 0], np.arange(n))
    none_of_it = np.full((1, n), 7)
    g = _run_abi(token, parent, n_out, none_of_it, n - 1)
    assert int(g["n_accepted"][0]) == 0 and int(g["next_token"][0]) == 7
    _check_against_oracle(g, token, parent, n_out, none_of_it, n - 1)


def test_rows_that_are_not_a_tree_are_reported_not_walked():
    token = np.array([[5, 6, 7, 8]])
    parent = np.array([[-1, 0, 3, 1]])                  # row 2 names a later row as its parent
    g = _run_abi(token, parent, np.array([4]), np.array([[6, 8, 0, 0]]), 4)
    assert int(g["status"][0]) == -1
    assert int(g["n_accepted"][0]) == 0 and int(g["next_token"][0]) == -1 and int(g["n_leaves"][0]) == 0
    assert (g["leaf_paths"] == -1).all() and (g["accepted_rows"] == -1).all()


@pytest.mark.parametrize("name", ["tiny", "7b_small"])
def test_walk_on_drafted_trees(name):
    """The tree of a real draft (already checked against the oracle), target choices planted along
    one emitted row per sequence: engine.verify_greedy equals the oracle's walk on that tree."""
    if name == "tiny":
        cfg = S.CONFIGS["tiny"].replace(threshold=-1e30)
    else:
        cfg = S.scaled_down(S.CONFIGS["llama2_7b"], hidden=256, vocab=4096, batch=3, threshold=-6.0)
    w = S.make_weights(cfg)
    eng = P.DraftEngine(cfg, w)
    rng = np.random.default_rng(3)
    for i in range(3):
        roots = S.make_roots(cfg, i)
        g = parity.run_gpu(eng, roots)
        parity.compare_with_oracle(cfg, w, roots, g)
        B, T = cfg.batch, cfg.total_tokens + 1
        target = np.zeros((B, T), dtype=np.int64)
        for b in range(B):
            n = int(g["n_out"][b])
            goal = int(rng.integers(n))
            target[b, :n] = S.target_choices_along(rng, g["token"][b], g["parent"][b], n, goal, cfg.vocab)
        v = eng.verify_greedy(torch.from_numpy(target.astype(np.int32)).to(eng.device))
        torch.cuda.synchronize(eng.device)
        v = {k: x.cpu().numpy() for k, x in v.items()}
        _check_against_oracle(v, g["token"], g["parent"], g["n_out"], target, cfg.max_depth)
        for b in range(B):
            assert int(v["n_accepted"][b]) >= 0
    eng.close()
