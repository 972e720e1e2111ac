"""GPU test of ddd_lm_head_topk_noalloc, the entry point for callers that cannot allocate
device memory (plug-ins given fixed buffers, processes whose memory is owned by a framework
pool): its scratch is a fixed array inside the library instead of a caller workspace.

Two yardsticks.  (1) The first pass of an ordinary draft computes exactly what this entry
point computes for the root rows - each row's logsumexp and its k best tokens with their
log-probabilities - so the existing ddd_draft (with its trace) is compared with it.  (2) The
CPU oracle's logits, log-softmax and top-k give the expected values directly, which also covers
the sizes at the edge of the fixed array: 32 rows, k = 32, and a vocabulary large enough that
all 256 thread blocks run and some of them walk two tiles.  Calls are always made in pairs, back
to back with different inputs, the second one smaller than the first, because every call reuses
the same scratch array and must not be affected by what the previous one left there.  This file
is named to be collected last.
"""
import numpy as np
import pytest
import torch

import ddd_synth as S
import paper_2409_00142_b200 as P
from oracle import ddd_oracle as O

pytestmark = pytest.mark.gpu
TOL = 2e-3


def first_pass_of_draft(eng, cfg, roots):
    dev = {k: v.to(eng.device) for k, v in roots.items()}
    eng.draft(dev["root_hidden"], dev["root_token"], dev["root_pos"])
    res = eng.results()
    assert int(res["status"][0]) == 0
    k = cfg.k
    return (res["tree_token"][:, 1:k + 1].numpy(), res["tree_cum"][:, 1:k + 1].numpy(),
            res["row_lse"][:, 0, 0].numpy())


def call_no_alloc(W, bias, h, k, scale, stream=None):
    """One call through the C ABI on device tensors W [V][Hd], bias [V] or None, h [rows][Hd]."""
    dev = W.device
    rows, hidden = h.shape
    vocab = W.shape[0]
    # outputs belong to the caller; the entry point itself allocates nothing
    tok = torch.full((rows, k), -7, dtype=torch.int32, device=dev)
    lp = torch.zeros((rows, k), dtype=torch.float32, device=dev)
    lse = torch.zeros(rows, dtype=torch.float32, device=dev)
    P.ddd_lm_head_topk_noalloc(
        W.data_ptr(), None if bias is None else bias.data_ptr(), h.data_ptr(),
        P.DDD_DTYPE_FP32 if W.dtype == torch.float32 else P.DDD_DTYPE_BF16, rows, hidden, vocab, k,
        float(scale), tok.data_ptr(), lp.data_ptr(), lse.data_ptr(),
        torch.cuda.current_stream(dev).cuda_stream if stream is None else stream)
    torch.cuda.synchronize(dev)
    return tok.cpu().numpy(), lp.cpu().numpy(), lse.cpu().numpy()


def no_alloc_pass(eng, cfg, roots):
    h = roots["root_hidden"].to(eng.device).contiguous()
    return call_no_alloc(eng.W, eng.bias, h, cfg.k, cfg.logit_scale, eng.stream_ptr())


def check_same(got, want):
    tok, lp, lse = got
    wtok, wlp, wlse = want
    np.testing.assert_allclose(lse, wlse, rtol=0, atol=TOL)
    np.testing.assert_allclose(lp, wlp, rtol=0, atol=TOL)
    for b in range(tok.shape[0]):
        if tok[b].tolist() == wtok[b].tolist():
            continue
        # a different order or member is only acceptable between scores closer than the tolerance
        for j in range(tok.shape[1]):
            if tok[b, j] != wtok[b, j]:
                assert abs(lp[b, j] - wlp[b, j]) < TOL
                partner = np.nonzero(wtok[b] == tok[b, j])[0]
                if len(partner):
                    assert abs(wlp[b, partner[0]] - lp[b, j]) < TOL
                else:           # a member the other side does not have: it must tie with its last one
                    assert abs(wlp[b, -1] - lp[b, j]) < TOL


def check_against_oracle(W, bias, h, k, scale, got):
    """Expected values from the oracle's own steps: logits, log-softmax, top-k (ties to the lower
    token); a choice that differs only inside a 2e-3 band is accepted, as in the parity tests."""
    tok, lp, lse = got
    z = O.lm_head_logits(W.cpu(), O.to_f64(h.cpu()), scale, None if bias is None else O.to_f64(bias.cpu()))
    exact = 0
    for r in range(h.shape[0]):
        want_lp = O.log_softmax_row(z[r])
        M = z[r].max()
        assert abs(lse[r] - (M + np.log(np.exp(z[r] - M).sum()))) < TOL, r
        assert not O.admissible_topk(want_lp, tok[r], k, TOL), (r, O.admissible_topk(want_lp, tok[r], k, TOL))
        np.testing.assert_allclose(lp[r], want_lp[tok[r]], rtol=0, atol=TOL)
        exact += tok[r].tolist() == O.topk_desc(want_lp, k).tolist()
    return exact


@pytest.mark.parametrize("case", ["fp32_tiny", "bf16_batch_bias"])
def test_no_alloc_entry_point_matches_first_pass_of_a_draft_twice_in_a_row(case):
    if case == "fp32_tiny":
        cfg = S.CONFIGS["tiny"].replace(batch=3, threshold=-1e30, max_depth=2)
    else:
        cfg = S.scaled_down(S.CONFIGS["llama3_8b_128k"], 256, 9000 + 16, max_depth=2, batch=4)
    w = S.make_weights(cfg)
    eng = P.DraftEngine(cfg, w)
    for draft_index in (0, 1):                      # two calls in a row, different inputs
        roots = S.make_roots(cfg, draft_index)
        want = first_pass_of_draft(eng, cfg, roots)
        got = no_alloc_pass(eng, cfg, roots)
        assert (got[0] >= 0).all() and (got[0] < cfg.vocab).all()
        check_same(got, want)
        h = roots["root_hidden"].to(eng.device)
        check_against_oracle(eng.W, eng.bias, h, cfg.k, cfg.logit_scale, got)
    eng.close()


def _random_case(dtype, vocab, hidden, rows, seed, with_bias):
    rng = np.random.default_rng([seed, vocab, rows])
    tdt = torch.float32 if dtype == "fp32" else torch.bfloat16
    W = torch.from_numpy((0.25 * rng.standard_normal((vocab, hidden))).astype(np.float32)).to(tdt).cuda()
    h = torch.from_numpy(rng.standard_normal((rows, hidden)).astype(np.float32)).to(tdt).cuda()
    bias = torch.from_numpy(rng.standard_normal(vocab).astype(np.float32)).cuda() if with_bias else None
    return W, bias, h


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_no_alloc_entry_point_against_the_oracle_at_the_limits_of_its_scratch(dtype):
    # First call: every limit at once.  32 rows (four chunks of eight rows, four rows per warp),
    # k = 32 (a full list per row), 40037 tokens = 313 tiles of 128 with a ragged last one, so
    # all 256 blocks run and blocks 0..56 carry their running state over a second tile.
    # Second call, right behind it: fewer rows, a narrower list, fewer blocks.  The slots of
    # the first call beyond those extents are still in the array and must not be looked at.
    big = _random_case(dtype, 40037, 64, 32, 1, with_bias=True)
    small = _random_case(dtype, 5000 + 3, 64, 5, 2, with_bias=False)
    got_big = call_no_alloc(*big, k=32, scale=1.5)
    got_small = call_no_alloc(*small, k=7, scale=0.75)
    again_big = call_no_alloc(*big, k=32, scale=1.5)
    exact = check_against_oracle(*big, 32, 1.5, got_big)
    check_against_oracle(*small, 7, 0.75, got_small)
    for a, b in zip(got_big, again_big):                # same inputs, same result, whatever ran in between
        np.testing.assert_array_equal(a, b)
    assert (got_big[0] >= 0).all() and (got_big[0] < 40037).all()
    # 11 (fp32) and 6 (bf16) of the 32 rows have no two of their best 33 scores within the tolerance:
    # there at least the list must be the oracle's own, token for token
    assert exact >= (11 if dtype == "fp32" else 6), exact


def test_no_alloc_entry_point_rejects_sizes_beyond_its_scratch():
    cfg = S.CONFIGS["tiny"]
    w = S.make_weights(cfg)
    eng = P.DraftEngine(cfg, w)
    buf = torch.zeros(64 * 64, dtype=torch.float32, device=eng.device)
    args = dict(W=eng.W.data_ptr(), bias=None, hidden_rows=eng.W.data_ptr(), dtype=P.DDD_DTYPE_FP32, rows=1,
                hidden=cfg.hidden, vocab=cfg.vocab, k=4, logit_scale=1.0, out_token=buf.data_ptr(),
                out_logprob=buf.data_ptr(), out_lse=buf.data_ptr(), stream=eng.stream_ptr())
    for bad in (dict(rows=33), dict(rows=0), dict(k=33), dict(k=0), dict(hidden=12), dict(vocab=4), dict(dtype=5)):
        with pytest.raises(P.DddError) as err:
            P.ddd_lm_head_topk_noalloc(**{**args, **bad})
        assert err.value.code == -1, bad
    with pytest.raises(P.DddError) as err:
        P.ddd_lm_head_topk_noalloc(**{**args, "W": eng.W.data_ptr() + 4})
    assert err.value.code == -2
    torch.cuda.synchronize(eng.device)
    eng.close()
