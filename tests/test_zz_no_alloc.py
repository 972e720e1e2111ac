"""GPU test of ddd_lm_head_topk_noalloc, the entry point for callers that cannot allocate
device memory (plug-ins given fixed buffers, processes whose memory is owned by a framework
pool): its scratch is a fixed array inside the library instead of a caller workspace.

The first pass of an ordinary draft computes exactly what this entry point computes for the
root rows - each row's logsumexp and its k best tokens with their log-probabilities - so the
existing ddd_draft (with its trace) is the yardstick.  Two calls are made back to back with
different inputs, because every call reuses the same scratch array and must not be affected
by what the previous one left there.  This file is named to be collected last.
"""
import numpy as np
import pytest
import torch

import ddd_synth as S
import paper_2409_00142_b200 as P

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


def no_alloc_pass(eng, cfg, roots):
    dev = eng.device
    h = roots["root_hidden"].to(dev).contiguous()
    B, k = cfg.batch, cfg.k
    # outputs belong to the caller; the entry point itself allocates nothing
    tok = torch.full((B, k), -7, dtype=torch.int32, device=dev)
    lp = torch.zeros((B, k), dtype=torch.float32, device=dev)
    lse = torch.zeros(B, dtype=torch.float32, device=dev)
    P.ddd_lm_head_topk_noalloc(
        eng.W.data_ptr(), None if eng.bias is None else eng.bias.data_ptr(), h.data_ptr(),
        P.DDD_DTYPE_FP32 if cfg.dtype == "fp32" else P.DDD_DTYPE_BF16, B, cfg.hidden, cfg.vocab, k,
        cfg.logit_scale, tok.data_ptr(), lp.data_ptr(), lse.data_ptr(), eng.stream_ptr())
    torch.cuda.synchronize(dev)
    return tok.cpu().numpy(), lp.cpu().numpy(), lse.cpu().numpy()


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
    eng.close()


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
