"""Pins of the CPU oracle against things other than itself.

Each test checks oracle/ddd_oracle.py against a closed form, an invariant, a
library routine or a brute-force enumeration written independently here.  The
brute force below deliberately uses none of the oracle's functions.
"""
import itertools
import math
import os

import numpy as np
import pytest
import scipy.special
import torch

import ddd_synth as S
from oracle import ddd_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
NEG_INF = -1e30


def small_cfg(**kw):
    base = dict(name="t", batch=1, hidden=8, vocab=5, k=2, max_depth=3, total_tokens=6,
                dtype="fp32", threshold=NEG_INF, sigma_w=0.5, seed=11)
    base.update(kw)
    return S.DraftConfig(**base)


# ----------------------------------------------------------------------------- a1 / a2
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_logits_match_library_matmul(dtype):
    rng = np.random.default_rng(0)
    V, Hd, R = 37, 24, 5
    tdt = torch.float32 if dtype == "fp32" else torch.bfloat16
    W = torch.from_numpy(rng.standard_normal((V, Hd)).astype(np.float32)).to(tdt)
    h = rng.standard_normal((R, Hd))
    bias = rng.standard_normal(V)
    z = O.lm_head_logits(W, h, 1.75, bias)
    ref = 1.75 * (h @ W.to(torch.float64).numpy().T) + bias[None, :]
    np.testing.assert_allclose(z, ref, rtol=0, atol=1e-12)
    # transposed-operand mistake would give a different shape or values
    assert z.shape == (R, V)
    z0 = O.lm_head_logits(W, h, 1.0, None)
    np.testing.assert_allclose(z0, h @ W.to(torch.float64).numpy().T, atol=1e-12)


def test_log_softmax_invariants_and_library():
    rng = np.random.default_rng(1)
    for scale in (0.1, 3.0, 40.0):
        z = rng.standard_normal(1000) * scale
        lp = O.log_softmax_row(z)
        assert abs(np.exp(lp).sum() - 1.0) < 1e-12
        assert (lp <= 0).all()
        np.testing.assert_allclose(lp, scipy.special.log_softmax(z), atol=1e-12)
    # large offsets must not overflow (max shift)
    z = np.array([1000.0, 999.0, 998.0])
    np.testing.assert_allclose(O.log_softmax_row(z), scipy.special.log_softmax(z), atol=1e-12)


def test_round_to_storage_matches_library_casts():
    rng = np.random.default_rng(2)
    y = np.concatenate([rng.standard_normal(20000) * 1.3, [1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8,
                                                          -(1.0 + 2.0 ** -8), 0.0, 2.0 ** -20]])
    got = O.round_to_storage(y, "bf16")
    # torch cannot cast fp64->bf16 in one rounding on every build; values chosen from fp32
    y32 = y.astype(np.float32)
    want = torch.from_numpy(y32).to(torch.bfloat16).to(torch.float64).numpy()
    same_input = y32.astype(np.float64) == y
    np.testing.assert_array_equal(got[same_input], want[same_input])
    # generic values: double rounding via fp32 can differ only on a vanishing set
    assert (got != want).mean() < 1e-3
    # exact ties go to even
    assert O.round_to_storage(np.array([1.0 + 2.0 ** -8]), "bf16")[0] == 1.0
    assert O.round_to_storage(np.array([1.0 + 3 * 2.0 ** -8]), "bf16")[0] == 1.0 + 2.0 ** -6
    np.testing.assert_array_equal(O.round_to_storage(y, "fp32"), y.astype(np.float32).astype(np.float64))


def test_topk_desc_ties_and_order():
    s = np.array([1.0, 3.0, 3.0, 2.0, 3.0, -1.0])
    assert O.topk_desc(s, 4).tolist() == [1, 2, 4, 3]
    assert O.topk_desc(np.zeros(7), 3).tolist() == [0, 1, 2]


def test_plant_closed_form():
    V, delta = 50, 8.0
    z = O.apply_plant(np.zeros(V), 17, delta)
    lp = O.log_softmax_row(z)
    assert abs(lp[17] - math.log(math.exp(delta) / (math.exp(delta) + V - 1))) < 1e-12
    assert abs(lp[0] - math.log(1.0 / (math.exp(delta) + V - 1))) < 1e-12
    # the planted logit replaces, it is not added: max is over the *other* columns
    z = np.arange(10.0)
    out = O.apply_plant(z, 9, 8.0)
    assert out[9] == 8.0 + 8.0 and (out[:9] == z[:9]).all()
    assert (O.apply_plant(z, -1, 8.0) == z).all()


# ----------------------------------------------------------------------------- a7
def test_draft_step_textbook_rmsnorm():
    rng = np.random.default_rng(3)
    hp, e = rng.standard_normal(64), rng.standard_normal(64)
    y = O.draft_step(hp, e, 1e-6, "fp32")
    u = hp + e
    want = u / np.sqrt((u ** 2).mean() + 1e-6)
    np.testing.assert_allclose(y, want, rtol=1e-6)
    assert abs((y ** 2).mean() - 1.0) < 1e-4
    yb = O.draft_step(hp, e, 1e-6, "bf16")
    np.testing.assert_allclose(yb, want, rtol=2.0 ** -8)
    # eps sits inside the square root: a zero vector maps to zero, not to NaN
    assert (O.draft_step(np.zeros(8), np.zeros(8), 1e-6, "fp32") == 0).all()


def test_draft_step_gathers_the_chosen_token_row():
    # E rows are multiples of distinct unit vectors, W = 0 so every logit ties and
    # the beam takes tokens 0..k-1; the next hidden must contain exactly that row.
    cfg = small_cfg(vocab=6, hidden=6, k=3, max_depth=2)
    W = torch.zeros(6, 6)
    E = torch.eye(6) * 100.0
    root = torch.zeros(1, 6)
    res = O.draft(cfg, {"W": W, "E": E, "bias": None, "plant_next": None},
                  root, np.array([0]), np.array([0]))[0]
    assert res.tree_token[1:4].tolist() == [0, 1, 2]
    # W = 0: nothing observable from h in the logits, so test the step function directly
    for tok in range(6):
        y = O.draft_step(np.zeros(6), O.to_f64(E[tok]), 1e-6, "fp32")
        assert np.argmax(np.abs(y)) == tok and abs(y[tok] - math.sqrt(6.0)) < 1e-3


# ----------------------------------------------------------------------------- brute force
def _bf_round(y, dtype):
    t = torch.from_numpy(np.asarray(y, dtype=np.float64))
    if dtype == "fp32":
        return t.to(torch.float32).to(torch.float64).numpy()
    return t.to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()


def brute_force_paths(cfg, weights, root_hidden, depth):
    """log-probability of every token path of length 1..depth, by direct enumeration."""
    W = weights["W"].to(torch.float64).numpy()
    E = weights["E"].to(torch.float64).numpy()
    bias = 0.0 if weights["bias"] is None else weights["bias"].to(torch.float64).numpy()
    V = cfg.vocab
    table = {}
    hidden = {(): root_hidden.to(torch.float64).numpy()[0]}
    score = {(): 0.0}
    for d in range(1, depth + 1):
        for prefix in itertools.product(range(V), repeat=d - 1):
            h = hidden[prefix]
            lp = scipy.special.log_softmax(cfg.logit_scale * (W @ h) + bias)
            for t in range(V):
                path = prefix + (t,)
                score[path] = score[prefix] + lp[t]
                table[path] = score[path]
                if d < depth:
                    u = h + E[t]
                    hidden[path] = _bf_round(u / np.sqrt((u * u).mean() + cfg.rms_eps), cfg.dtype)
    return table


def node_path(res, node):
    path = []
    while node != 0:
        path.append(int(res.tree_token[node]))
        node = int(res.tree_parent[node])
    return tuple(reversed(path))


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("V,k,depth", [(4, 2, 4), (5, 3, 3), (6, 2, 3), (8, 4, 3)])
def test_tree_scores_equal_brute_force_path_table(V, k, depth, dtype):
    cfg = small_cfg(vocab=V, k=k, max_depth=depth, total_tokens=7, dtype=dtype, seed=V * 10 + k,
                    logit_scale=1.3)
    w = S.make_weights(cfg)
    r = S.make_roots(cfg, 0)
    res = O.draft(cfg, w, **r)[0]
    table = brute_force_paths(cfg, w, r["root_hidden"], depth)
    # (iv) probabilities of all V^d paths of each length sum to one
    for d in range(1, depth + 1):
        tot = sum(math.exp(v) for p, v in table.items() if len(p) == d)
        assert abs(tot - 1.0) < 1e-10
    # (i) every tree node's cumulative score is its path's log-probability
    N = k + (depth - 1) * k * k
    assert res.stop_depth == depth
    for node in range(1, N + 1):
        p = node_path(res, node)
        assert len(p) == res.tree_depth[node]
        assert abs(res.tree_cum[node] - table[p]) < 1e-9, (node, p)
        # monotone non-increasing along the path
        assert res.tree_cum[node] <= res.tree_cum[res.tree_parent[node]] + 1e-15
    # (ii) each new beam is the exact top-k among all k*V children of the previous beam
    beam_paths = [()]
    for d in range(1, depth + 1):
        children = {bp + (t,): table[bp + (t,)] for bp in beam_paths for t in range(V)}
        want = sorted(children, key=lambda p: -children[p])[:k]
        base = O.first_node_of_pass(d, k)
        got = [node_path(res, base + s) for s in res.beam_sel[d - 1]]
        assert got == want, (d, got, want)
        beam_paths = got


@pytest.mark.parametrize("V,seed", [(3, 5), (4, 6), (6, 7)])
def test_exhaustive_beam_equals_global_topk(V, seed):
    # (iii) Beam search is a heuristic, but when nothing has been pruned before depth d the beam
    # after pass d is the exact top-k of all V^d paths.  That needs k >= V^(d-1), and a row keeps
    # k <= V tokens, so depth 2 with k = V is the one instance there is: the first beam holds every
    # token, and the second is the best k of all V^2 two-token paths.
    cfg = small_cfg(vocab=V, k=V, hidden=8, max_depth=2, total_tokens=5, seed=seed, logit_scale=2.0)
    w = S.make_weights(cfg)
    r = S.make_roots(cfg, 0)
    res = O.draft(cfg, w, **r)[0]
    assert sorted(res.tree_token[1:V + 1].tolist()) == list(range(V))
    table = brute_force_paths(cfg, w, r["root_hidden"], 2)
    want = sorted((p for p in table if len(p) == 2), key=lambda p: -table[p])[:V]
    base = O.first_node_of_pass(2, V)
    got = [node_path(res, base + s) for s in res.beam_sel[1]]
    assert got == want


# ----------------------------------------------------------------------------- a6: closed forms
def uniform_weights(cfg, bias=None):
    return {"W": torch.zeros(cfg.vocab, cfg.hidden), "E": torch.randn(cfg.vocab, cfg.hidden),
            "bias": bias, "plant_next": None}


def test_uniform_closed_form_H_and_tiebreaks():
    # W = 0, no bias: every logprob is -ln V, H_d = ln k - d ln V, ties pick tokens 0..k-1.
    cfg = S.CONFIGS["tiny"].replace(threshold=NEG_INF)
    w = uniform_weights(cfg)
    r = S.make_roots(cfg, 0)
    res = O.draft(cfg, w, **r)[0]
    k, V = cfg.k, cfg.vocab
    assert res.stop_depth == cfg.max_depth
    for d, H in enumerate(res.H_trace, start=1):
        assert abs(H - (math.log(k) - d * math.log(V))) < 1e-12
    assert res.tree_token[1:k + 1].tolist() == list(range(k))
    assert res.beam_sel[0] == list(range(k))
    assert res.beam_sel[1] == list(range(k))            # lowest flat indices win the tie
    # Tiny's own threshold: H_1 = ln 4 - ln 1024 = -5.545 < -2 -> one pass only
    res = O.draft(S.CONFIGS["tiny"], w, **r)[0]
    assert res.stop_depth == 1 and res.n_out == 1 + k


def test_stop_depth_against_hand_thresholds():
    cfg0 = small_cfg(vocab=16, k=4, hidden=8, max_depth=6, total_tokens=10)
    w = uniform_weights(cfg0)
    r = S.make_roots(cfg0, 0)
    Hd = lambda d: math.log(4) - d * math.log(16)       # noqa: E731
    for d in range(1, 6):
        # threshold just below H_d: pass d survives the check, pass d+1 fails it
        x = Hd(d) - 1e-9
        res = O.draft(cfg0.replace(threshold=x), w, **r)[0]
        assert res.stop_depth == min(d + 1, 6)
        # threshold just above H_d: stop right after pass d
        res = O.draft(cfg0.replace(threshold=Hd(d) + 1e-9), w, **r)[0]
        assert res.stop_depth == d
    # equality continues (strict '<' in Algorithm 1): choose x equal to the oracle-independent
    # closed form evaluated the same way the heuristic is (max-shifted), i.e. from exact inputs
    lp = -math.log(16)
    H1 = lp + math.log(4.0)                              # max-shifted form with all terms equal
    res = O.draft(cfg0.replace(threshold=H1), w, **r)[0]
    assert res.H_trace[0] == H1
    assert res.stop_depth >= 2


def test_greedy_chain_k1():
    # W = 0, arbitrary bias, k = 1: greedy chain on argmax token; H_d = d log p_max.
    rng = np.random.default_rng(9)
    cfg = small_cfg(vocab=12, k=1, hidden=8, max_depth=5, total_tokens=8)
    bias = torch.from_numpy(rng.standard_normal(12).astype(np.float32))
    w = uniform_weights(cfg, bias)
    r = S.make_roots(cfg, 1)
    res = O.draft(cfg, w, **r)[0]
    p = scipy.special.softmax(bias.to(torch.float64).numpy())
    for d, H in enumerate(res.H_trace, start=1):
        assert abs(H - d * math.log(p.max())) < 1e-12
    assert res.n_out == 6
    assert res.token[1:].tolist() == [int(p.argmax())] * 5
    assert res.parent.tolist() == [-1, 0, 1, 2, 3, 4]
    assert res.depth.tolist() == [0, 1, 2, 3, 4, 5]
    assert res.position.tolist() == (int(r["root_pos"][0]) + np.arange(6)).tolist()
    assert res.mask == [(1 << (i + 1)) - 1 for i in range(6)]        # lower-triangular
    # stop rule: first d with d log p_max < x
    x = 2.5 * math.log(p.max())
    assert O.draft(cfg.replace(threshold=x), w, **r)[0].stop_depth == 3


def test_H_invariants_and_schedule():
    cfg = small_cfg(vocab=40, k=4, hidden=16, max_depth=8, total_tokens=20, logit_scale=2.0, seed=3)
    w = S.make_weights(cfg)
    r = S.make_roots(cfg, 0)
    res = O.draft(cfg, w, **r)[0]
    H = res.H_trace
    assert len(H) == 8 and all(h <= 1e-15 for h in H)
    assert all(H[i + 1] <= H[i] + 1e-12 for i in range(7))     # beam mass can only shrink
    # Eq. 1 by its definition
    base = O.first_node_of_pass(3, cfg.k)
    cum = [res.tree_cum[base + s] for s in res.beam_sel[2]]
    assert abs(H[2] - math.log(sum(math.exp(c) for c in cum))) < 1e-12
    # a sparser S can only delay the stop
    x = 0.5 * (H[2] + H[3])                                       # H_3 >= x > H_4
    every = O.draft(cfg.replace(threshold=x), w, **r)[0]
    assert every.stop_depth == 4
    sparse = O.draft(cfg.replace(threshold=x, check_mask=(1 << 1) | (1 << 5)), w, **r)[0]
    assert sparse.stop_depth == 6
    never = O.draft(cfg.replace(threshold=x, check_mask=0), w, **r)[0]
    assert never.stop_depth == 8
    # identical prefixes: the decisions before the stop do not depend on S
    assert every.tree_token[:20].tolist() == sparse.tree_token[:20].tolist()


def test_paper_parameter_set_from_fixture():
    vals = {}
    for line in open(os.path.join(GOLDEN, "paper_parameters.txt")):
        if line.strip() and not line.startswith("#"):
            key, v = line.split("=")
            vals[key.strip()] = v.split()
    n, w_ = int(vals["n"][0]), int(vals["w"][0])
    S_steps = [int(s) for s in vals["S"]]
    x = float(vals["x"][0])
    assert (n, w_, S_steps, x) == (11, 10, [5, 7, 9], -0.3)
    mask = sum(1 << (s - 1) for s in S_steps)
    cfg = small_cfg(vocab=64, k=w_, hidden=16, max_depth=n, total_tokens=60, threshold=x,
                    check_mask=mask, logit_scale=2.0, seed=8)
    w = S.make_weights(cfg)
    r = S.make_roots(cfg, 0)
    res = O.draft(cfg, w, **r)[0]
    free = O.draft(cfg.replace(check_mask=0), w, **r)[0]            # never checks: all H_d
    first_below = next(d for d, H in enumerate(free.H_trace, start=1) if H < x)
    assert first_below < 5
    # H already fell below -0.3 before the first check of S = {5,7,9}: stop after the 5th call
    assert res.stop_depth == 5 and res.H_trace[4] < x
    strict = sum(1 << (int(s) - 1) for s in vals["S_strict"])
    assert O.draft(cfg.replace(check_mask=strict), w, **r)[0].stop_depth == first_below
    # fixed depth like EAGLE-2: S empty, n = 6
    depth6 = int(vals["eagle2_depth"][0])
    assert O.draft(cfg.replace(check_mask=0, max_depth=depth6), w, **r)[0].stop_depth == depth6


# ----------------------------------------------------------------------------- a8 / a9
def test_rerank_plain_definition_and_invariants():
    cfg = small_cfg(vocab=30, k=3, hidden=16, max_depth=4, total_tokens=11, logit_scale=2.0, seed=4)
    w = S.make_weights(cfg)
    r = S.make_roots(cfg, 0)
    res = O.draft(cfg, w, **r)[0]
    N = cfg.k + 3 * cfg.k ** 2
    ranked = sorted(range(1, N + 1), key=lambda i: (-res.tree_cum[i], i))[:11]
    assert res.node_id.tolist() == [0] + sorted(ranked)
    assert res.n_out == 12
    chosen = set(res.node_id.tolist())
    for nid in res.node_id[1:]:
        assert int(res.tree_parent[nid]) in chosen                  # ancestor-closed
    for i in range(1, res.n_out):
        assert res.node_id[res.parent[i]] == res.tree_parent[res.node_id[i]]
        assert res.parent[i] < i
    # m >= N returns the whole tree
    big = O.draft(cfg.replace(total_tokens=1000), w, **r)[0]
    assert big.n_out == 1 + N and big.node_id.tolist() == list(range(N + 1))
    # ties: lower node id wins
    assert O.rerank(np.array([-1.0, -1.0, -1.0, -0.5]), 2).tolist() == [1, 4]


def test_mask_two_constructions_agree():
    cfg = small_cfg(vocab=50, k=4, hidden=16, max_depth=5, total_tokens=40, logit_scale=2.5, seed=6)
    w = S.make_weights(cfg)
    r = S.make_roots(cfg, 0)
    res = O.draft(cfg, w, **r)[0]
    for i in range(res.n_out):
        bits, j = 0, i
        while j >= 0:                                               # parent-pointer walk
            bits |= 1 << j
            j = int(res.parent[j])
        assert bits == res.mask[i]
        assert bin(bits).count("1") == res.depth[i] + 1
        assert bits & 1 and bits < (1 << (i + 1))
    words = O.mask_words(res.mask, cfg.t_max)
    assert words.shape == (41, 2) and words.dtype == np.uint32
    for i in range(res.n_out):
        assert int(words[i, 0]) | (int(words[i, 1]) << 32) == res.mask[i]
    assert (words[res.n_out:] == 0).all()


def test_batch_sequences_are_independent():
    cfg = small_cfg(batch=3, vocab=40, k=3, hidden=16, max_depth=5, total_tokens=12,
                    logit_scale=2.0, threshold=-1.0, seed=12)
    w = S.make_weights(cfg)
    r = S.make_roots(cfg, 0)
    both = O.draft(cfg, w, **r)
    assert len({x.stop_depth for x in both}) > 1                    # stops differ across the batch
    one = cfg.replace(batch=1)
    for b in range(3):
        solo = O.draft(one, w, r["root_hidden"][b:b + 1], r["root_token"][b:b + 1],
                       r["root_pos"][b:b + 1])[0]
        assert solo.stop_depth == both[b].stop_depth
        assert solo.node_id.tolist() == both[b].node_id.tolist()
        np.testing.assert_array_equal(solo.cum, both[b].cum)


# ----------------------------------------------------------------------------- replay mode
def _follow_from(res):
    return O.FollowSequence(stop_depth=res.stop_depth, tree_token=res.tree_token.copy(),
                            beam_sel=[list(s) for s in res.beam_sel], node_id=res.node_id.copy())


REPLAY_H = (-0.17074681981286077, -0.8118013902899263, -1.4596241337374665, -2.2107429074698577)


def _replay_case(threshold=-1.0, **kw):
    """A draft whose heuristic falls through -0.17, -0.81, -1.46, -2.21 (REPLAY_H, checked below):
    with x = -1 it stops after the third of at most four calls, so a stop one step early and one
    step late both exist."""
    cfg = small_cfg(vocab=60, k=3, hidden=16, max_depth=4, total_tokens=12, logit_scale=2.0,
                    threshold=threshold, seed=13, **kw)
    return cfg, S.make_weights(cfg), S.make_roots(cfg, 0)


def _gate_violations(res):
    return [v for v in res.violations if "gate" in v]


def test_replay_of_own_decisions_is_clean_and_detects_mistakes():
    cfg, w, r = _replay_case()
    res = O.draft(cfg, w, **r)[0]
    assert res.stop_depth == 3 and not res.ambiguities
    np.testing.assert_allclose(res.H_trace, REPLAY_H[:3], rtol=0, atol=1e-12)
    again = O.draft(cfg, w, **r, follow=[_follow_from(res)])[0]
    assert not again.violations
    np.testing.assert_array_equal(again.tree_cum, res.tree_cum)
    # a wrong token in a row's top-k is flagged
    f = _follow_from(res)
    worst = int(np.argmin(O.log_softmax_row(O.lm_head_logits(
        w["W"], O.to_f64(r["root_hidden"]), cfg.logit_scale, None)[0])))
    f.tree_token[2] = worst
    assert any("token top-k" in v for v in O.draft(cfg, w, **r, follow=[f])[0].violations)
    # a wrong member of the new beam is flagged: the worst of the k*k candidates of pass 2
    f = _follow_from(res)
    base = O.first_node_of_pass(2, cfg.k)
    cand = res.tree_cum[base:base + cfg.k * cfg.k]
    f.beam_sel[1][cfg.k - 1] = int(np.argmin(cand))
    assert int(np.argmin(cand)) not in res.beam_sel[1]
    assert any("beam top-k" in v for v in O.draft(cfg, w, **r, follow=[f])[0].violations)


def test_replay_rejects_a_stop_decision_outside_the_tolerance_band():
    """Algorithm 1 stops iff H < x at a checked step.  A replayed stop that differs from that is a
    violation unless |H - x| < tol; the heuristic values are fixed numbers here (REPLAY_H), so
    which side of the band each case lies on is known without asking the oracle."""
    tol = 2e-3
    cfg, w, r = _replay_case(-1.0)
    full = O.draft(cfg.replace(threshold=NEG_INF), w, **r)[0]          # the search itself does not depend on x
    np.testing.assert_allclose(full.H_trace, REPLAY_H, rtol=0, atol=1e-12)
    own = O.draft(cfg, w, **r)[0]
    assert own.stop_depth == 3

    def follow_stopping_at(depth):
        return O.FollowSequence(stop_depth=depth, tree_token=full.tree_token.copy(),
                                beam_sel=[list(s) for s in full.beam_sel[:depth]], node_id=None)

    # x = -1: H_2 = -0.81 >= x and H_3 = -1.46 < x, both far outside the band
    early = O.draft(cfg, w, **r, follow=[follow_stopping_at(2)])[0]
    assert _gate_violations(early) and "pass 2" in _gate_violations(early)[0]
    assert early.stop_depth == 2                                     # the decision is adopted after the check
    late = O.draft(cfg, w, **r, follow=[follow_stopping_at(4)])[0]
    assert _gate_violations(late) and "pass 3" in _gate_violations(late)[0]
    right = O.draft(cfg, w, **r, follow=[follow_stopping_at(3)])[0]
    assert not right.violations and right.stop_depth == 3
    # the same two shifts with x moved to within half the tolerance of H_3: either decision passes
    for x, own_depth in ((REPLAY_H[2] + 0.5 * tol, 3), (REPLAY_H[2] - 0.5 * tol, 4)):
        c2 = cfg.replace(threshold=x)
        assert O.draft(c2, w, **r)[0].stop_depth == own_depth
        for depth in (3, 4):
            res = O.draft(c2, w, **r, follow=[follow_stopping_at(depth)], tol=tol)[0]
            assert not res.violations, (x, depth, res.violations)
            assert res.stop_depth == depth
            assert any("gate" in a for a in res.ambiguities)
    # ... and just outside the band the shifted decision is rejected again
    for x, wrong in ((REPLAY_H[2] + 1.5 * tol, 4), (REPLAY_H[2] - 1.5 * tol, 3)):
        res = O.draft(cfg.replace(threshold=x), w, **r, follow=[follow_stopping_at(wrong)], tol=tol)[0]
        assert _gate_violations(res), (x, wrong)


def test_replay_rejects_a_stop_at_an_unchecked_step():
    # S = {3}: nothing may stop after step 2, whatever H is
    cfg, w, r = _replay_case(-0.5, check_mask=1 << 2)
    own = O.draft(cfg, w, **r)[0]
    assert own.stop_depth == 3                                       # H_1, H_2 are below x but unchecked
    # the search decisions of every pass stay available: having noted the violation the replay goes on
    f = _follow_from(O.draft(cfg.replace(threshold=NEG_INF), w, **r)[0])
    f.stop_depth, f.node_id = 2, None
    res = O.draft(cfg, w, **r, follow=[f])[0]
    assert any("pass 2" in v and "outside S" in v for v in res.violations)


def test_replay_rejects_an_inadmissible_rerank_set():
    cfg, w, r = _replay_case()
    res = O.draft(cfg, w, **r)[0]
    N = cfg.k + (res.stop_depth - 1) * cfg.k ** 2
    m = cfg.total_tokens
    cum = res.tree_cum[1:N + 1]
    order = np.argsort(-cum, kind="stable") + 1                      # node ids, best first
    kept, dropped = order[:m], order[m:]
    assert cum[kept[-1] - 1] - cum[dropped[0] - 1] > 0.05            # no near-tie at the boundary
    assert sorted(kept.tolist()) == res.node_id[1:].tolist()

    def replay(ids):
        f = _follow_from(res)
        f.node_id = np.concatenate([[0], np.asarray(ids, dtype=np.int64)])
        return [v for v in O.draft(cfg, w, **r, follow=[f])[0].violations if "rerank" in v]

    assert not replay(sorted(kept.tolist()))
    # the best node dropped for the best of the rest: something clearly above the m-th is missing
    assert any("not chosen" in v for v in replay(sorted(kept[1:].tolist() + [int(dropped[0])])))
    # the m-th swapped for the worst node of the tree: a member clearly below the m-th
    assert any("below" in v for v in replay(sorted(kept[:-1].tolist() + [int(dropped[-1])])))
    # right set, wrong order
    ids = sorted(kept.tolist())
    ids[3], ids[4] = ids[4], ids[3]
    assert any("ascending" in v for v in replay(ids))


def _one_hot_bias_case():
    """W = 0 and one token with a logit 60 above the rest: every row's best token has logprob
    -(V-1) e^-60 (about -1e-25, far inside any tolerance) and every other token -60, so the chain root ->
    a -> b -> c of best tokens has three nodes whose scores agree to 1e-24."""
    cfg = small_cfg(vocab=9, k=2, hidden=8, max_depth=3, total_tokens=2)
    bias = torch.zeros(cfg.vocab)
    bias[4] = 60.0
    return cfg, uniform_weights(cfg, bias=bias), S.make_roots(cfg, 0)


def test_replay_accepts_a_swap_inside_the_band_and_wants_an_ancestor_closed_set():
    cfg, w, r = _one_hot_bias_case()
    res = O.draft(cfg, w, **r)[0]
    k = cfg.k
    a, b, c = 1, O.first_node_of_pass(2, k), O.first_node_of_pass(3, k)
    assert res.tree_token[[a, b, c]].tolist() == [4, 4, 4]
    assert res.tree_parent[[a, b, c]].tolist() == [0, a, b]
    assert abs(res.tree_cum[c]) < 1e-20 and res.tree_cum[2] < -59
    assert res.node_id.tolist() == [0, a, b]                          # ties go to the lower node id

    def replay(ids):
        f = _follow_from(res)
        f.node_id = np.array([0] + ids, dtype=np.int64)
        return O.draft(cfg, w, **r, follow=[f])[0]

    # b and c score the same to 1e-24: by score alone {a, c} is as good as {a, b} ...
    assert not O.admissible_topk(res.tree_cum[1:], [a - 1, c - 1], 2, 2e-3, ordered=False)
    # ... but c's parent b would be missing from the emitted tree
    swapped = replay([a, c])
    assert any("ancestor-closed" in v for v in swapped.violations)
    # with room for three nodes a swap among equal scores that keeps every parent is accepted:
    # uniform logits, all nine depth-2 nodes tie, any of them may fill the last places
    cfg2 = small_cfg(vocab=7, k=3, hidden=8, max_depth=2, total_tokens=6)
    w2, r2 = uniform_weights(cfg2), S.make_roots(cfg2, 0)
    res2 = O.draft(cfg2, w2, **r2)[0]
    assert res2.node_id.tolist() == [0, 1, 2, 3, 4, 5, 6]
    f = _follow_from(res2)
    f.node_id = np.array([0, 1, 2, 3, 4, 5, 12], dtype=np.int64)
    out = O.draft(cfg2, w2, **r2, follow=[f])[0]
    assert not out.violations and out.node_id.tolist() == [0, 1, 2, 3, 4, 5, 12]
    assert out.parent.tolist() == [-1, 0, 0, 0, 1, 1, 3]
    assert any("rerank" in a_ for a_ in out.ambiguities)


def test_admissible_topk_bands():
    s = np.array([5.0, 4.0, 3.0005, 3.0, 1.0])
    assert not O.admissible_topk(s, [0, 1, 2], 3, 2e-3)
    assert not O.admissible_topk(s, [0, 1, 3], 3, 2e-3)             # inside the band
    assert O.admissible_topk(s, [0, 1, 4], 3, 2e-3)                 # clearly worse entry
    assert O.admissible_topk(s, [0, 2, 3], 3, 2e-3)                 # clearly better entry missing
    assert O.admissible_topk(s, [1, 0, 2], 3, 2e-3)                 # wrong order
    assert not O.admissible_topk(s, [1, 0, 2], 3, 2e-3, ordered=False)
    assert O.admissible_topk(s, [0, 0, 1], 3, 2e-3)                 # duplicates


# --------------------------------------------------------------------------- acceptance walk, leaf paths
def _path_to(parent, i):
    path = []
    while i >= 0:
        path.append(i)
        i = int(parent[i])
    return path[::-1]


def test_greedy_accept_against_consistency_definition():
    """Accepted rows = exactly the rows whose whole root path agrees with the target: each row on
    the path carries the token the target chose after that row's parent (Section 1)."""
    rng = np.random.default_rng(11)
    n_agree = []
    for trial in range(200):
        n_rows = int(rng.integers(1, 40))
        vocab = int(rng.integers(3, 9))          # small vocabulary: agreements are common
        token, parent = S.random_tree(rng, n_rows, vocab)
        target = rng.integers(vocab, size=n_rows)
        consistent = []
        for i in range(1, n_rows):
            path = _path_to(parent, i)
            if all(token[j] == target[parent[j]] for j in path[1:]):
                consistent.append(i)
        # sibling tokens are distinct, so the consistent rows lie on one root path
        consistent.sort(key=lambda i: len(_path_to(parent, i)))
        for a, b in zip(consistent, consistent[1:]):
            assert parent[b] == a
        accepted, nxt = O.greedy_accept(token, parent, n_rows, target)
        assert accepted == consistent
        last = accepted[-1] if accepted else 0
        assert nxt == target[last]
        n_agree.append(len(accepted))
    assert max(n_agree) >= 3 and min(n_agree) == 0          # the cases exercise both ends


def test_greedy_accept_chain_closed_form():
    """A k = 1 chain whose first j tokens match the target accepts exactly j tokens."""
    n = 9
    token = np.arange(100, 100 + n)
    parent = np.arange(-1, n - 1)
    for j in range(n):
        target = np.full(n, -7)
        target[:j] = token[1:j + 1]               # the target agrees after rows 0..j-1
        accepted, nxt = O.greedy_accept(token, parent, n, target)
        assert accepted == list(range(1, j + 1))
        assert nxt == -7
    # every draft token accepted: the bonus token is the target's choice after the last row
    target = np.append(token[1:], 555)
    accepted, nxt = O.greedy_accept(token, parent, n, target)
    assert accepted == list(range(1, n)) and nxt == 555
    # rows beyond n_out do not take part
    accepted, nxt = O.greedy_accept(token, parent, 4, target)
    assert accepted == [1, 2, 3] and nxt == token[4]


def test_leaf_paths_cover_the_tree():
    rng = np.random.default_rng(5)
    for trial in range(100):
        n_rows = int(rng.integers(1, 60))
        token, parent = S.random_tree(rng, n_rows, 50)
        paths = O.leaf_paths(parent, n_rows)
        leaves = [p[-1] for p in paths]
        assert leaves == sorted(set(range(n_rows)) - set(int(x) for x in parent[1:]))
        covered = set()
        for p in paths:
            assert p[0] == 0
            for a, b in zip(p, p[1:]):
                assert parent[b] == a
            covered.update(p)
        assert covered == set(range(n_rows))
        # the ancestor mask of a leaf (a separately pinned construction) marks exactly its path
        mask = O.tree_mask_rows(list(parent))
        for p in paths:
            assert mask[p[-1]] == sum(1 << r for r in p)


def test_acceptance_on_a_drafted_tree_follows_a_planted_path():
    """Target choices planted along one emitted row's ancestors: the walk accepts that path."""
    cfg = S.CONFIGS["tiny"].replace(batch=1, threshold=-1e30)
    w = S.make_weights(cfg)
    res = O.draft(cfg, w, **S.make_roots(cfg, 0))[0]
    n_out = res.n_out
    deepest = int(np.argmax(res.depth[:n_out]))
    path = _path_to(res.parent, deepest)
    target = np.full(n_out, cfg.vocab)            # a token no draft row can carry
    for a, b in zip(path, path[1:]):
        target[a] = res.token[b]
    accepted, nxt = O.greedy_accept(res.token, res.parent, n_out, target)
    assert accepted == path[1:] and nxt == cfg.vocab
    assert len(accepted) == res.depth[deepest]
