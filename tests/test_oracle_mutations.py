"""The pins must notice plausible mistakes: each case below plants one mistake in the CPU
oracle (never in the CUDA path) and expects a named pin from test_oracle_pins.py to fail."""
import inspect
import math

import numpy as np
import pytest

from oracle import ddd_oracle as O
from tests import test_oracle_pins as pins


def _h_mean(logprobsum):                      # Eq. 1 with a mean instead of a sum
    a = np.asarray(logprobsum, dtype=np.float64)
    return float(a.max() + math.log(np.exp(a - a.max()).mean()))


def _h_extra_term(logprobsum):                # the garbled upper bound taken literally: w + 1 terms
    a = np.append(np.asarray(logprobsum, dtype=np.float64), 0.0)
    return float(a.max() + math.log(np.exp(a - a.max()).sum()))


def _topk_high_index_first(scores, k):        # ties resolved towards the larger index
    s = np.asarray(scores, dtype=np.float64)
    return np.lexsort((-np.arange(len(s)), -s))[:k]


def _softmax_unnormalised(z_row):             # forgets the log-sum-exp
    return np.minimum(z_row - z_row.max(), 0.0)


def _step_eps_outside(h_parent, e_row, eps, dtype):
    u = h_parent + e_row
    return O.round_to_storage(u / (math.sqrt(float(np.mean(u * u))) + 1.0), dtype)


def _step_no_embedding(h_parent, e_row, eps, dtype):
    u = h_parent
    return O.round_to_storage(u / math.sqrt(float(np.mean(u * u)) + eps), dtype)


def _mask_without_self(parent_slot):
    rows = []
    for i, p in enumerate(parent_slot):
        rows.append(1 if p < 0 else (rows[p] | (1 << p)))
    return rows


def _rerank_lowest(cum, m):                   # keeps the worst nodes
    n = len(cum)
    return np.sort(O.topk_desc(-np.asarray(cum), min(m, n)) + 1)


def _plant_added(z_row, column, delta):       # adds delta to the column instead of replacing it
    z_row = z_row.copy()
    if column >= 0:
        z_row[column] += delta
    return z_row


def _logits_transposed_scale(W, h, scale, bias):   # scale applied to the bias as well
    z = ORIG["lm_head_logits"](W, h, 1.0, bias)
    return scale * z


def _accept_any_row_with_the_token(token, parent, n_out, target_argmax):   # forgets the parent link
    cur, accepted = 0, []
    while True:
        want = int(target_argmax[cur])
        nxt = next((i for i in range(cur + 1, n_out) if int(token[i]) == want), -1)
        if nxt < 0:
            return accepted, want
        accepted.append(nxt)
        cur = nxt


def _accept_one_step_only(token, parent, n_out, target_argmax):             # stops after the first match
    accepted, nxt = ORIG["greedy_accept"](token, parent, n_out, target_argmax)
    return accepted[:1], (int(target_argmax[accepted[0]]) if accepted else nxt)


def _leaf_paths_leaf_first(parent, n_out):                                  # paths not reversed
    return [p[::-1] for p in ORIG["leaf_paths"](parent, n_out)]


def _leaf_paths_every_row(parent, n_out):                                   # inner rows listed as leaves too
    out = []
    for leaf in range(n_out):
        path, r = [], leaf
        while r >= 0:
            path.append(r)
            r = int(parent[r])
        out.append(path[::-1])
    return out


ORIG = {name: getattr(O, name) for name in (
    "heuristic_H", "topk_desc", "log_softmax_row", "draft_step", "tree_mask_rows", "rerank", "apply_plant",
    "lm_head_logits", "greedy_accept", "leaf_paths")}

CASES = [
    ("heuristic_H", _h_mean, pins.test_uniform_closed_form_H_and_tiebreaks, ()),
    ("heuristic_H", _h_extra_term, pins.test_greedy_chain_k1, ()),
    ("topk_desc", _topk_high_index_first, pins.test_topk_desc_ties_and_order, ()),
    ("topk_desc", _topk_high_index_first, pins.test_uniform_closed_form_H_and_tiebreaks, ()),
    ("log_softmax_row", _softmax_unnormalised, pins.test_log_softmax_invariants_and_library, ()),
    ("log_softmax_row", _softmax_unnormalised, pins.test_tree_scores_equal_brute_force_path_table, (5, 3, 3, "fp32")),
    ("draft_step", _step_eps_outside, pins.test_draft_step_textbook_rmsnorm, ()),
    ("draft_step", _step_no_embedding, pins.test_tree_scores_equal_brute_force_path_table, (5, 3, 3, "fp32")),
    ("tree_mask_rows", _mask_without_self, pins.test_mask_two_constructions_agree, ()),
    ("rerank", _rerank_lowest, pins.test_rerank_plain_definition_and_invariants, ()),
    ("apply_plant", _plant_added, pins.test_plant_closed_form, ()),
    ("lm_head_logits", _logits_transposed_scale, pins.test_logits_match_library_matmul, ("bf16",)),
    ("greedy_accept", _accept_any_row_with_the_token, pins.test_greedy_accept_against_consistency_definition, ()),
    ("greedy_accept", _accept_one_step_only, pins.test_greedy_accept_chain_closed_form, ()),
    ("greedy_accept", _accept_one_step_only, pins.test_acceptance_on_a_drafted_tree_follows_a_planted_path, ()),
    ("leaf_paths", _leaf_paths_leaf_first, pins.test_leaf_paths_cover_the_tree, ()),
    ("leaf_paths", _leaf_paths_every_row, pins.test_leaf_paths_cover_the_tree, ()),
]


@pytest.mark.parametrize("name,mutant,pin,args", CASES,
                         ids=[f"{c[0]}:{c[1].__name__}->{c[2].__name__}" for c in CASES])
def test_pin_catches_planted_mistake(monkeypatch, name, mutant, pin, args):
    pin(*args)                                   # green on the real oracle
    monkeypatch.setattr(O, name, mutant)
    with pytest.raises(AssertionError):
        pin(*args)


def test_gate_strictness_mistake_is_caught(monkeypatch):
    # "H <= x" instead of "H < x": the equality case of the hand-threshold pin must fail.
    src = O.draft.__code__
    real = O.heuristic_H

    def nudged(logprobsum):                      # makes H a hair smaller, so that H == x turns into H < x
        return np.nextafter(real(logprobsum), -np.inf)

    pins.test_stop_depth_against_hand_thresholds()
    monkeypatch.setattr(O, "heuristic_H", nudged)
    with pytest.raises(AssertionError):
        pins.test_stop_depth_against_hand_thresholds()
    assert O.draft.__code__ is src


# ----------------------------------------------------------------------------- the replay checker
# The checks that police another implementation's decisions live inside O.draft itself, so the
# mistake is planted in its source text: one edit, recompiled in the oracle's own namespace.
def _draft_with(monkeypatch, old: str, new: str):
    src = inspect.getsource(O.draft)
    assert src.count(old) == 1, f"the oracle's replay code no longer reads {old!r}"
    scope = dict(vars(O))
    exec(compile(src.replace(old, new), "<mutated oracle draft>", "exec"), scope)
    monkeypatch.setattr(O, "draft", scope["draft"])


REPLAY_MUTANTS = [
    # the gate check never fires: any stop depth is adopted
    ("if theirs != stop and abs(H - cfg.threshold) >= tol:", "if False:",
     pins.test_replay_rejects_a_stop_decision_outside_the_tolerance_band),
    # the band is ignored: a decision inside it is rejected too
    ("if theirs != stop and abs(H - cfg.threshold) >= tol:", "if theirs != stop:",
     pins.test_replay_rejects_a_stop_decision_outside_the_tolerance_band),
    # a stop at an unchecked step goes unnoticed
    ("elif follow is not None and follow[b].stop_depth == d:", "elif False:",
     pins.test_replay_rejects_a_stop_at_an_unchecked_step),
    # the rerank set is adopted without its admissibility check
    ("for msg in admissible_topk(cum, ids - 1, min(m, N), tol, ordered=False):", "for msg in []:",
     pins.test_replay_rejects_an_inadmissible_rerank_set),
    # ... or without the order check
    ("if (np.diff(ids) <= 0).any():", "if False:", pins.test_replay_rejects_an_inadmissible_rerank_set),
    # ... or without the ancestor check
    ("if (r.parent == -2).any():", "if False:",
     pins.test_replay_accepts_a_swap_inside_the_band_and_wants_an_ancestor_closed_set),
    # the beam choice is adopted unchecked
    ("for msg in admissible_topk(cand, sel, k, tol):", "for msg in []:",
     pins.test_replay_of_own_decisions_is_clean_and_detects_mistakes),
    # the rows' token lists are adopted unchecked
    ("for msg in admissible_topk(lp, top, k, tol):", "for msg in []:",
     pins.test_replay_of_own_decisions_is_clean_and_detects_mistakes),
]


@pytest.mark.parametrize("old,new,pin", REPLAY_MUTANTS,
                         ids=[f"{i}:{m[2].__name__}" for i, m in enumerate(REPLAY_MUTANTS)])
def test_replay_checker_pins_catch_planted_mistakes(monkeypatch, old, new, pin):
    pin()
    _draft_with(monkeypatch, old, new)
    with pytest.raises(AssertionError):
        pin()


def test_admissible_topk_mistakes_are_caught(monkeypatch):
    real = O.admissible_topk
    pins.test_admissible_topk_bands()
    for broken in (lambda *a, **kw: [],                                             # accepts anything
                   lambda s, c, k, tol, ordered=True: real(s, c, k, 0.0, ordered),   # no band at all
                   lambda s, c, k, tol, ordered=True: real(s, c, k, tol, False)):    # order never checked
        monkeypatch.setattr(O, "admissible_topk", broken)
        with pytest.raises(AssertionError):
            pins.test_admissible_topk_bands()
