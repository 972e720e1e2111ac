"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the same seeded
inputs.  Small cases are compared element by element with both LM-head kernels; full-size
configurations run in the launch configuration the benchmark times (tensor-core kernel,
CUDA graph)."""
import math

import numpy as np
import pytest
import torch

import ddd_synth as S
import paper_2409_00142_b200 as P
from tests import parity

pytestmark = pytest.mark.gpu
NEG = -1e30

_weights_cache = {}


def weights_for(cfg):
    key = (cfg.seed, cfg.hidden, cfg.vocab, cfg.dtype, cfg.sigma_w, cfg.bias_kind, cfg.plant_frac)
    if key not in _weights_cache:
        if len(_weights_cache) > 2:
            _weights_cache.clear()
        _weights_cache[key] = S.make_weights(cfg)
    return _weights_cache[key]


def engine_for(cfg, kernel, mode=P.DDD_LAUNCH_STREAM):
    return P.DraftEngine(cfg, weights_for(cfg), lm_head_kernel=kernel, launch_mode=mode)


SIMT, TC = P.DDD_LM_HEAD_SIMT, P.DDD_LM_HEAD_TCGEN05


# ----------------------------------------------------------------------------- tiny (fp32)
@pytest.mark.parametrize("threshold", [-2.0, -8.0, NEG])
def test_tiny_fp32(threshold):
    cfg = S.CONFIGS["tiny"].replace(threshold=threshold)
    eng = engine_for(cfg, P.DDD_LM_HEAD_AUTO)
    checked = 0
    for i in range(4):
        roots = S.make_roots(cfg, i)
        g = parity.run_gpu(eng, roots)
        parity.compare_with_oracle(cfg, weights_for(cfg), roots, g)
        checked += parity.strict_equal_when_unambiguous(cfg, weights_for(cfg), roots, g)
    # at least one of these four drafts has no near-tie anywhere at each threshold (3, 1 and 1 of them):
    # there the oracle's own decisions, not replayed ones, must be the GPU's
    assert checked >= 1
    eng.close()


def test_uniform_logits_closed_form_on_gpu():
    # W = 0: every logprob is -ln V, ties resolve to the lowest token / candidate index,
    # H_d = ln k - d ln V exactly as the closed form says.
    cfg = S.CONFIGS["tiny"].replace(threshold=NEG)
    w = dict(weights_for(cfg))
    w["W"] = torch.zeros_like(w["W"])
    eng = P.DraftEngine(cfg, w)
    roots = S.make_roots(cfg, 0)
    g = parity.run_gpu(eng, roots)
    k, V = cfg.k, cfg.vocab
    assert int(g["stop_depth"][0]) == cfg.max_depth
    for d in range(1, cfg.max_depth + 1):
        assert abs(g["H_trace"][0, d - 1] - (math.log(k) - d * math.log(V))) < 1e-4
        assert g["beam_sel"][0, d - 1].tolist() == list(range(k))
    assert g["tree_token"][0, 1:k + 1].tolist() == list(range(k))
    parity.compare_with_oracle(cfg, w, roots, g, strict=True)
    eng.close()


# ----------------------------------------------------------------------------- scaled-down shapes
def small_cases():
    c = S.CONFIGS
    return {
        # several 128-row tiles per block plus a ragged tail (vocab not a multiple of 32)
        "7b": S.scaled_down(c["llama2_7b"], 512, 8200 - 12, threshold=-4.0),
        "13b_plant": S.scaled_down(c["vicuna_13b"], 640, 6000, threshold=-2.0, plant_frac=0.3),
        "70b_batch": S.scaled_down(c["llama2_70b_b16"], 512, 4096 + 40, threshold=-3.0),
        "128k_zipf": S.scaled_down(c["llama3_8b_128k"], 256, 20000 + 8, threshold=-3.0),
        "full_depth": S.scaled_down(c["llama2_7b"], 256, 3000, threshold=NEG),
    }


@pytest.mark.parametrize("kernel", [SIMT, TC], ids=["simt", "tcgen05"])
@pytest.mark.parametrize("case", list(small_cases()))
def test_small_shapes_match_oracle(case, kernel):
    cfg = small_cases()[case]
    eng = engine_for(cfg, kernel)
    depths = []
    for i in range(3):
        roots = S.make_roots(cfg, i)
        g = parity.run_gpu(eng, roots)
        parity.compare_with_oracle(cfg, weights_for(cfg), roots, g)
        depths += g["stop_depth"].tolist()
    if case == "70b_batch":
        assert len(set(depths)) > 1, "batched sequences should stop at different depths"
    if case == "13b_plant":
        assert max(depths) > 2, "planted tokens should keep some drafts going"
    eng.close()


def test_strict_oracle_agrees_when_no_near_ties():
    # a narrow beam leaves few neighbouring scores, so most drafts have no near-tie at all
    cfg = small_cases()["7b"].replace(k=3, max_depth=5, total_tokens=20)
    eng = engine_for(cfg, TC)
    checked = 0
    for i in range(8):
        roots = S.make_roots(cfg, 10 + i)
        g = parity.run_gpu(eng, roots)
        checked += parity.strict_equal_when_unambiguous(cfg, weights_for(cfg), roots, g)
    eng.close()
    assert checked >= 6          # seven of these eight drafts are free of near-ties


def test_check_schedule_and_paper_parameters():
    # S = {5, 7, 9}, n = 11, w = 10 (Section 3.2): stops can only happen at checked steps.
    mask = sum(1 << (s - 1) for s in (5, 7, 9))
    cfg = S.scaled_down(S.CONFIGS["llama2_7b"], 256, 4000, threshold=-0.3, max_depth=11, check_mask=mask)
    eng = engine_for(cfg, TC)
    roots = S.make_roots(cfg, 0)
    g = parity.run_gpu(eng, roots)
    assert int(g["stop_depth"][0]) in (5, 7, 9, 11)
    parity.compare_with_oracle(cfg, weights_for(cfg), roots, g)
    eng.close()


def test_k1_greedy_chain_and_k_equal_to_limit():
    base = S.scaled_down(S.CONFIGS["llama2_7b"], 256, 2048, threshold=NEG)
    for k, depth, m in ((1, 6, 4), (32, 3, 200)):
        cfg = base.replace(k=k, max_depth=depth, total_tokens=m)
        for kernel in (SIMT, TC):
            eng = engine_for(cfg, kernel)
            roots = S.make_roots(cfg, 0)
            g = parity.run_gpu(eng, roots)
            parity.compare_with_oracle(cfg, weights_for(cfg), roots, g)
            eng.close()


# ----------------------------------------------------------------------------- wide beams (the paper's appendix: up to 100)
def wide_cases():
    base = S.scaled_down(S.CONFIGS["llama2_7b"], 256, 3000 + 24, threshold=NEG, max_depth=3, total_tokens=200)
    zipf = S.scaled_down(S.CONFIGS["llama3_8b_128k"], 128, 9000 + 5, threshold=-6.0, max_depth=4, total_tokens=300)
    return {
        "k33": base.replace(k=33),                                   # first width past one key per lane
        "k50": base.replace(k=50),
        "k75_two_sequences": base.replace(k=75, batch=2, max_depth=2, threshold=-9.0),   # 150 rows in a pass
        "k100": base.replace(k=100),
        "k128": base.replace(k=128, max_depth=2),                    # the limit
        # fewer logits per row than the per-row top-k kernel has threads: every logit is a candidate
        "k40_small_vocab": S.scaled_down(S.CONFIGS["llama2_7b"], 128, 1000, threshold=NEG, max_depth=3, total_tokens=100,
                                         k=40),
        "k100_zipf": zipf.replace(k=100, batch=1),                   # winners cluster in the first vocab tiles
        # 28,737 tree nodes: more than the rerank keeps keys for in shared memory
        "k64_large_tree": S.scaled_down(S.CONFIGS["vicuna_13b"], 128, 2000, threshold=NEG, k=64, max_depth=8,
                                        total_tokens=500, plant_frac=0.2),
    }


@pytest.mark.parametrize("kernel", [SIMT, TC], ids=["simt", "tcgen05"])
@pytest.mark.parametrize("case", list(wide_cases()))
def test_wide_beams_match_oracle(case, kernel):
    cfg = wide_cases()[case]
    if kernel == SIMT and cfg.batch * cfg.k > 128:
        pytest.skip("the CUDA-core kernel keeps at most 128 wide rows in shared memory")
    eng = engine_for(cfg, kernel, P.DDD_LAUNCH_GRAPH if case == "k50" else P.DDD_LAUNCH_STREAM)
    with torch.cuda.stream(torch.cuda.Stream()):
        for i in range(2):
            roots = S.make_roots(cfg, i)
            g = parity.run_gpu(eng, roots)
            parity.compare_with_oracle(cfg, weights_for(cfg), roots, g)
    eng.close()


@pytest.mark.parametrize("k", [40, 100])
def test_wide_beams_with_equal_logits_take_the_exact_slow_ways(k):
    # W = 0 on the tensor-core path: every logit of a row is the same, so far more than 1024 of them lie
    # on the floor the per-row top-k kernel derives (it falls back to a radix select over the row and takes
    # the lowest tokens among the ties), and all k * k candidates of a pass tie as well (the select kernel
    # falls back to merging the sorted candidate rows).  The closed form: tokens 0..k-1, candidates
    # 0..k-1, H_d = ln k - d ln V.
    cfg = S.scaled_down(S.CONFIGS["llama2_7b"], 256, 3000 + 24, threshold=NEG, max_depth=3, total_tokens=120, k=k)
    w = dict(weights_for(cfg))
    w["W"] = torch.zeros_like(w["W"])
    eng = P.DraftEngine(cfg, w, lm_head_kernel=TC, launch_mode=P.DDD_LAUNCH_STREAM)
    with torch.cuda.stream(torch.cuda.Stream()):
        roots = S.make_roots(cfg, 0)
        g = parity.run_gpu(eng, roots)
    V = cfg.vocab
    assert int(g["stop_depth"][0]) == cfg.max_depth
    for d in range(1, cfg.max_depth + 1):
        assert abs(g["H_trace"][0, d - 1] - (math.log(k) - d * math.log(V))) < 1e-3
        assert g["beam_sel"][0, d - 1].tolist() == list(range(k))
    assert g["tree_token"][0, 1:k + 1].tolist() == list(range(k))
    parity.compare_with_oracle(cfg, w, roots, g, strict=True)
    eng.close()


def test_full_size_7b_at_width_100_depth_6():
    # the widest row of the paper's appendix table, in the configuration the benchmark's sweep times
    cfg = S.CONFIGS["llama2_7b"].replace(k=100, max_depth=6, threshold=NEG, total_tokens=60)
    eng = engine_for(cfg, P.DDD_LM_HEAD_AUTO, P.DDD_LAUNCH_GRAPH)
    with torch.cuda.stream(torch.cuda.Stream()):
        roots = S.make_roots(cfg, 0)
        g = parity.run_gpu(eng, roots)
    parity.compare_with_oracle(cfg, weights_for(cfg), roots, g)
    assert int(g["stop_depth"][0]) == 6 and int(g["n_out"][0]) == 61
    eng.close()


def edge_cases():
    base = S.scaled_down(S.CONFIGS["llama2_7b"], 128, 1000, threshold=NEG)
    return {
        "single_pass": base.replace(max_depth=1, total_tokens=20),                 # n = 1: no draft step at all
        "m_exceeds_tree": base.replace(k=3, max_depth=2, total_tokens=50),         # fewer nodes than m: padded rows
        "vocab_just_above_k": base.replace(vocab=40, k=8, max_depth=3, total_tokens=30),
        "odd_vocab": base.replace(vocab=1001, k=5, max_depth=3, total_tokens=25),  # not a multiple of 8 or 32
        "hidden_64": S.scaled_down(S.CONFIGS["llama2_7b"], 64, 700, threshold=NEG, k=6, max_depth=3, total_tokens=20),
        "rows_256": base.replace(batch=8, k=32, max_depth=2, total_tokens=100),    # B * k at its limit
        "mask_1024_rows": base.replace(k=32, max_depth=3, total_tokens=1023),      # widest mask: 32 words per row
        "one_token": base.replace(k=2, max_depth=4, total_tokens=1),
    }


@pytest.mark.parametrize("kernel", [SIMT, TC], ids=["simt", "tcgen05"])
@pytest.mark.parametrize("case", list(edge_cases()))
def test_edge_shapes_match_oracle(case, kernel):
    cfg = edge_cases()[case]
    eng = engine_for(cfg, kernel)
    for i in range(2):
        roots = S.make_roots(cfg, i)
        g = parity.run_gpu(eng, roots)
        parity.compare_with_oracle(cfg, weights_for(cfg), roots, g)
    eng.close()


def fused_edge_cases():
    cases = dict(edge_cases())
    base = S.scaled_down(S.CONFIGS["llama2_7b"], 128, 1000, threshold=-6.0)
    cases.update({
        "more_sequences_than_blocks": base.replace(batch=200, k=1, max_depth=5, total_tokens=4),   # 200 rows, 32 blocks
        "two_blocks_for_eight_rows": base.replace(vocab=40, k=8, max_depth=4, total_tokens=30),    # a block owns 4 rows of one sequence
        "batch_stops_apart": base.replace(batch=6, k=5, max_depth=8, total_tokens=40, threshold=-2.5),
    })
    return cases


@pytest.mark.parametrize("case", list(fused_edge_cases()))
def test_edge_shapes_in_one_persistent_kernel(case):
    cfg = fused_edge_cases()[case]
    eng = engine_for(cfg, TC, P.DDD_LAUNCH_FUSED)
    stops = set()
    for i in range(2):
        roots = S.make_roots(cfg, i)
        g = parity.run_gpu(eng, roots)
        parity.compare_with_oracle(cfg, weights_for(cfg), roots, g)
        stops.update(g["stop_depth"].tolist())
    if case == "batch_stops_apart":
        assert len(stops) > 1, stops
    eng.close()


# ----------------------------------------------------------------------------- seeded random shapes
def random_shapes():
    """Forty seeded configurations spread over the legal ranges: beam rows 1..256 (so every
    epilogue grouping and stage size of the tensor-core kernel occurs), ragged vocabularies,
    sparse and dense check schedules, planted rows, Zipf bias, both launch modes."""
    rng = np.random.default_rng(20240900)
    out = []
    while len(out) < 40:
        k = int(rng.choice([1, 2, 3, 5, 8, 10, 13, 16, 17, 24, 31, 32]))
        batch = int(rng.choice([1, 1, 2, 3, 5, 8]))
        if batch * k > 256:
            continue
        n = int(rng.integers(1, 9))
        if 1 + k + (n - 1) * k * k > 6000:
            continue
        hidden = 64 * int(rng.integers(1, 9))
        vocab = int(rng.integers(k + 1, 5000))
        m = int(rng.integers(1, 200))
        mask = int(rng.integers(0, 1 << n)) if rng.random() < 0.5 else 0xFFFFFFFF
        base = S.CONFIGS[str(rng.choice(["llama2_7b", "vicuna_13b", "llama3_8b_128k"]))]
        out.append(S.scaled_down(base, hidden, vocab, batch=batch, k=k, max_depth=n, total_tokens=m,
                                 check_mask=mask, threshold=float(rng.choice([-1.0, -3.0, -6.0, -12.0])),
                                 seed=int(rng.integers(1 << 30))))
    return out


@pytest.mark.parametrize("index", range(40))
def test_random_shapes_match_oracle(index):
    cfg = random_shapes()[index]
    kernel = SIMT if index % 5 == 4 else TC
    mode = (P.DDD_LAUNCH_STREAM, P.DDD_LAUNCH_GRAPH, P.DDD_LAUNCH_FUSED)[index % 3]
    if mode == P.DDD_LAUNCH_FUSED and kernel == SIMT:
        mode = P.DDD_LAUNCH_GRAPH
    eng = engine_for(cfg, kernel, mode)
    with torch.cuda.stream(torch.cuda.Stream()):
        for i in range(2):
            roots = S.make_roots(cfg, i)
            g = parity.run_gpu(eng, roots)
            parity.compare_with_oracle(cfg, weights_for(cfg), roots, g)
    eng.close()


# ----------------------------------------------------------------------------- launch modes
def _random_many_rows_or_wide(index):
    """Seeded random shapes for the two paths the ordinary random shapes do not reach: the many-rows
    form of the persistent kernel (48 beam rows or more, 23,700-37,800 vocabulary rows on a 148-SM
    device) for even indices, beams wider than 32 for odd ones."""
    rng = np.random.default_rng([20240900142, index])
    if index % 2 == 0:
        k = int(rng.choice([8, 10, 12, 16, 24, 32]))
        batch = int(rng.integers(max(2, -(-48 // k)), min(256 // k, max(3, 200 // k)) + 1))
        vocab = int(rng.integers(23700, 37800) // 8 * 8 + int(rng.choice([0, 8, 16, 24])))
        cfg = S.scaled_down(S.CONFIGS["llama2_70b_b16"], int(rng.choice([128, 256, 512])), vocab, batch=batch, k=k,
                            total_tokens=int(rng.integers(10, 80)), threshold=float(rng.choice([NEG, -2.0, -3.0, -4.0])),
                            max_depth=int(rng.integers(2, 6)), plant_frac=float(rng.choice([0.0, 0.0, 0.3])),
                            plant_delta=8.0, bias_kind=str(rng.choice(["none", "none", "zipf"])),
                            seed=int(rng.integers(0, 1000)))
        return cfg, P.DDD_LAUNCH_FUSED
    k = int(rng.choice([33, 40, 50, 64, 75, 100, 128]))
    batch = int(rng.integers(1, max(1, 256 // k) + 1))
    vocab = max(k + 64, int(rng.integers(600, 12000) // 8 * 8 + int(rng.choice([0, 8, 16]))))
    cfg = S.scaled_down(S.CONFIGS["llama2_7b"], int(rng.choice([128, 256])), vocab, batch=batch, k=k,
                        total_tokens=int(rng.integers(20, 300)), threshold=float(rng.choice([NEG, -6.0, -9.0])),
                        max_depth=int(rng.integers(2, 5)), plant_frac=float(rng.choice([0.0, 0.0, 0.3])), plant_delta=8.0,
                        bias_kind=str(rng.choice(["none", "none", "zipf"])), seed=int(rng.integers(0, 1000)))
    return cfg, int(rng.choice([P.DDD_LAUNCH_STREAM, P.DDD_LAUNCH_GRAPH, P.DDD_LAUNCH_PLAIN]))


@pytest.mark.parametrize("index", range(24))
def test_random_many_rows_and_wide_shapes_match_oracle(index):
    cfg, mode = _random_many_rows_or_wide(index)
    w = S.make_weights(cfg)
    eng = P.DraftEngine(cfg, w, lm_head_kernel=TC, launch_mode=mode)
    with torch.cuda.stream(torch.cuda.Stream()):
        for i in range(2):
            roots = S.make_roots(cfg, 500 + i)
            g = parity.run_gpu(eng, roots)
            parity.compare_with_oracle(cfg, w, roots, g)
    eng.close()


def test_graph_mode_host_variant_and_determinism():
    cfg = small_cases()["7b"]
    roots = S.make_roots(cfg, 1)
    eng_p = engine_for(cfg, TC, P.DDD_LAUNCH_PLAIN)
    a0 = parity.run_gpu(eng_p, roots)
    eng_p.close()
    eng_s = engine_for(cfg, TC, P.DDD_LAUNCH_STREAM)
    a = parity.run_gpu(eng_s, roots)
    a2 = parity.run_gpu(eng_s, roots)
    eng_g = engine_for(cfg, TC, P.DDD_LAUNCH_GRAPH)
    with torch.cuda.stream(torch.cuda.Stream()):
        b = parity.run_gpu(eng_g, roots)
        b2 = parity.run_gpu(eng_g, roots)           # second launch replays the captured graph
        other = S.make_roots(cfg, 2)
        c = parity.run_gpu(eng_g, other)            # new input pointers: re-captured
    for name in a:
        np.testing.assert_array_equal(a[name], a0[name], err_msg=name)    # plain launches == overlapped launches
        np.testing.assert_array_equal(a[name], a2[name], err_msg=name)    # run-to-run identical
        np.testing.assert_array_equal(a[name], b[name], err_msg=name)     # graph == stream
        np.testing.assert_array_equal(b[name], b2[name], err_msg=name)
    parity.compare_with_oracle(cfg, weights_for(cfg), other, c)
    # host-buffer entry point
    host_out = eng_s.make_host_out()
    eng_s.draft_host(roots["root_hidden"].pin_memory(), roots["root_token"].pin_memory(),
                     roots["root_pos"].pin_memory(), host_out)
    for name in host_out:
        np.testing.assert_array_equal(host_out[name].numpy(), a[name], err_msg=name)
    # in graph mode the host-buffer call is one graph launch (copies and init kernel included)
    with torch.cuda.stream(torch.cuda.Stream()):
        for r, want in ((roots, a), (other, c), (roots, a)):
            host_g = eng_g.make_host_out()
            eng_g.draft_host(r["root_hidden"].pin_memory(), r["root_token"].pin_memory(),
                             r["root_pos"].pin_memory(), host_g)
            for name in host_g:
                np.testing.assert_array_equal(host_g[name].numpy(), want[name], err_msg=name)
    assert P.ddd_launches_per_draft(eng_s.handle, 1) == 1 + 2 * cfg.max_depth
    # captured drafts end early after passes 3, 5 and 8 (every step checked, n = 12)
    assert cfg.max_depth == 12 and cfg.check_mask & 0xFFF == 0xFFF
    for needed, launched in [(1, 3), (2, 3), (3, 3), (4, 5), (5, 5), (6, 8), (8, 8), (9, 12), (12, 12)]:
        assert P.ddd_launches_per_draft(eng_g.handle, needed) == 1 + 2 * launched, needed
    assert 1 <= P.ddd_lm_head_blocks(eng_s.handle) <= 512
    eng_s.close()
    eng_g.close()


@pytest.mark.parametrize("schedule", ["every_step", "paper_5_7_9", "only_4"])
def test_captured_drafts_of_every_stop_depth_equal_stream_launches(schedule):
    # the captured graph nests its conditional groups; whatever depth a draft stops at, inside a
    # group, at its end or at n, the results are those of the kernel-by-kernel launches
    base = small_cases()["7b"]
    if schedule == "every_step":
        cfgs = [base.replace(threshold=x) for x in (-1.0, -3.0, -5.0, -7.0, -9.0, -12.0, -16.0, -22.0, NEG)]
    elif schedule == "paper_5_7_9":
        mask = sum(1 << (s - 1) for s in (5, 7, 9))
        cfgs = [base.replace(max_depth=11, check_mask=mask, threshold=x) for x in (-0.3, -9.0, -13.0, -17.0, NEG)]
    else:
        cfgs = [base.replace(max_depth=6, check_mask=1 << 3, threshold=x) for x in (-0.5, NEG)]
    seen = set()
    stream = torch.cuda.Stream()
    for cfg in cfgs:
        eng_s = engine_for(cfg, TC, P.DDD_LAUNCH_STREAM)
        eng_g = engine_for(cfg, TC, P.DDD_LAUNCH_GRAPH)
        for i in range(3):
            roots = S.make_roots(cfg, i)
            a = parity.run_gpu(eng_s, roots)
            with torch.cuda.stream(stream):
                b = parity.run_gpu(eng_g, roots)
            for name in a:
                np.testing.assert_array_equal(a[name], b[name], err_msg=f"{name} x={cfg.threshold}")
            seen.update(a["stop_depth"].tolist())
        parity.compare_with_oracle(cfg, weights_for(cfg), roots, b)
        if cfg.threshold == NEG:      # fixed-depth drafting: no conditional groups at all
            assert P.ddd_launches_per_draft(eng_g.handle, 1) == 1 + 2 * cfg.max_depth
        eng_s.close()
        eng_g.close()
    if schedule == "every_step":
        assert len(seen) >= 6 and min(seen) <= 2 and max(seen) == 12, sorted(seen)
    elif schedule == "paper_5_7_9":
        assert seen <= {5, 7, 9, 11} and len(seen) >= 2, sorted(seen)
    else:
        assert seen <= {4, 6}, sorted(seen)


# ----------------------------------------------------------------------------- one persistent kernel per draft
@pytest.mark.parametrize("case", list(small_cases()))
def test_fused_draft_equals_kernel_by_kernel_draft(case):
    # same partials, same merge order, same fp64 draft step: the one-kernel draft must give the
    # results of the kernel-by-kernel launches bit for bit, and both must match the oracle
    cfg = small_cases()[case]
    eng_s = engine_for(cfg, TC, P.DDD_LAUNCH_STREAM)
    eng_f = engine_for(cfg, TC, P.DDD_LAUNCH_FUSED)
    assert P.ddd_launches_per_draft(eng_f.handle, 1) in (1, 2)      # the rerank kernel only where it does not fit inside
    depths = set()
    for i in range(4):
        roots = S.make_roots(cfg, i)
        a = parity.run_gpu(eng_s, roots)
        b = parity.run_gpu(eng_f, roots)
        for name in a:
            if name in ("beam_sel", "row_lse", "H_trace"):
                for q in range(cfg.batch):
                    D = int(a["stop_depth"][q])
                    np.testing.assert_array_equal(a[name][q, :D], b[name][q, :D], err_msg=name)
            else:
                np.testing.assert_array_equal(a[name], b[name], err_msg=name)
        parity.compare_with_oracle(cfg, weights_for(cfg), roots, b)
        depths.update(b["stop_depth"].tolist())
    # two drafts back to back without a synchronisation in between, then the host-buffer entry point
    r0, r1 = (parity.to_device(S.make_roots(cfg, j), eng_f.device) for j in (0, 1))
    eng_f.draft(r0["root_hidden"], r0["root_token"], r0["root_pos"])
    eng_f.draft(r1["root_hidden"], r1["root_token"], r1["root_pos"])
    last = {k2: v.numpy() for k2, v in eng_f.results().items()}
    want = parity.run_gpu(eng_s, S.make_roots(cfg, 1))
    np.testing.assert_array_equal(last["token"], want["token"])
    np.testing.assert_array_equal(last["mask"], want["mask"])
    host_out = eng_f.make_host_out()
    hr = S.make_roots(cfg, 1)
    eng_f.draft_host(hr["root_hidden"].pin_memory(), hr["root_token"].pin_memory(), hr["root_pos"].pin_memory(), host_out)
    for name in host_out:
        if name == "H_trace":       # entries of passes that did not run keep whatever an earlier draft left
            for q in range(cfg.batch):
                D = int(want["stop_depth"][q])
                np.testing.assert_array_equal(host_out[name].numpy()[q, :D], want[name][q, :D])
        else:
            np.testing.assert_array_equal(host_out[name].numpy(), want[name], err_msg=name)
    eng_s.close()
    eng_f.close()
    if case == "full_depth":
        assert depths == {cfg.max_depth}


@pytest.mark.parametrize("vocab", [24000 + 8, 37000 - 3])
def test_fused_draft_with_both_tiles_of_a_block_sharing_a_stage(vocab):
    # from 48 beam rows on, and where every block owns five to eight 32-row units (two tiles), the
    # persistent kernel feeds both tiles from one fetch of the hidden rows: 751 units = 5-6 per block
    # of a 148-SM device, 1157 units = 7-8
    cfg = S.scaled_down(S.CONFIGS["llama2_70b_b16"], 256, vocab, batch=5, threshold=-3.0, max_depth=4)
    eng_s = engine_for(cfg, TC, P.DDD_LAUNCH_STREAM)
    eng_f = engine_for(cfg, TC, P.DDD_LAUNCH_FUSED)
    if torch.cuda.get_device_properties(0).multi_processor_count == 148:
        assert P.ddd_fused_pass_kind(eng_f.handle) >= 1
    for i in range(3):
        roots = S.make_roots(cfg, i)
        a = parity.run_gpu(eng_s, roots)
        b = parity.run_gpu(eng_f, roots)
        for name in ("stop_depth", "n_out", "token", "parent", "depth", "position", "mask", "node_id",
                     "tree_token", "tree_parent"):
            np.testing.assert_array_equal(a[name], b[name], err_msg=name)
        # the persistent kernel adds up a row's exp(z - max) in another order there (per quarter of a
        # tile against the block's maximum): scores agree to rounding, choices are the same
        for name in ("cum", "tree_cum"):
            np.testing.assert_allclose(a[name], b[name], rtol=0, atol=2e-5, err_msg=name)
        parity.compare_with_oracle(cfg, weights_for(cfg), roots, b)
    eng_s.close()
    eng_f.close()


def floor_cases():
    # Shapes where the persistent kernel's blocks agree on a floor per row before they pick
    # their k best (48 beam rows or more, five to eight 32-row units per block on a 148-SM device).
    base = S.CONFIGS["llama2_70b_b16"]
    return {
        # more rows than blocks: a sequence's ten rows on its own nine blocks
        "160_rows": S.scaled_down(base, 256, 32000, batch=16, threshold=-2.5, max_depth=4),
        # eight rows per sequence on seven blocks, ragged last unit
        "k8_b20": S.scaled_down(base, 256, 31000 + 8, batch=20, k=8, total_tokens=40, threshold=-2.5, max_depth=4),
        # planted columns take the checked form of the logit
        "plant": S.scaled_down(base, 256, 30000 + 8, batch=6, threshold=-3.0, max_depth=4, plant_frac=0.3,
                               plant_delta=8.0),
        # a bias that puts every winner into the first blocks: their queues fill, the others' stay empty
        "zipf_bias": S.scaled_down(base, 256, 26000, batch=5, threshold=-3.0, max_depth=3, bias_kind="zipf"),
        "k16": S.scaled_down(base, 256, 28000, batch=4, k=16, total_tokens=64, threshold=-3.0, max_depth=3),
        "k32": S.scaled_down(base, 256, 36000, batch=2, k=32, total_tokens=96, threshold=NEG, max_depth=3),
    }


@pytest.mark.parametrize("case", list(floor_cases()))
def test_fused_draft_with_a_floor_per_row(case):
    cfg = floor_cases()[case]
    eng_s = engine_for(cfg, TC, P.DDD_LAUNCH_STREAM)
    eng_f = engine_for(cfg, TC, P.DDD_LAUNCH_FUSED)
    if torch.cuda.get_device_properties(0).multi_processor_count == 148:
        assert P.ddd_fused_pass_kind(eng_f.handle) == 2
    assert P.ddd_fused_pass_kind(eng_s.handle) == 0
    for i in range(2):
        roots = S.make_roots(cfg, i)
        a = parity.run_gpu(eng_s, roots)
        b = parity.run_gpu(eng_f, roots)
        parity.compare_with_oracle(cfg, weights_for(cfg), roots, b)
        for name in ("stop_depth", "n_out", "token", "parent", "depth", "position", "mask", "tree_token", "tree_parent"):
            np.testing.assert_array_equal(a[name], b[name], err_msg=name)
        np.testing.assert_allclose(a["cum"], b["cum"], rtol=0, atol=2e-5)
    eng_s.close()
    eng_f.close()


def test_fused_draft_where_the_floor_says_nothing():
    # W = 0: all logits of a row are equal, every one of them lies on the floor, the queue of
    # each block runs over and the pass is done by the tile loop instead; the result is the
    # closed form (ties to the lowest token and candidate index)
    cfg = S.scaled_down(S.CONFIGS["llama2_70b_b16"], 256, 32000, batch=6, threshold=NEG, max_depth=3)
    w = dict(weights_for(cfg))
    w["W"] = torch.zeros_like(w["W"])
    eng = P.DraftEngine(cfg, w, lm_head_kernel=TC, launch_mode=P.DDD_LAUNCH_FUSED)
    if torch.cuda.get_device_properties(0).multi_processor_count == 148:
        assert P.ddd_fused_pass_kind(eng.handle) == 2
    roots = S.make_roots(cfg, 0)
    g = parity.run_gpu(eng, roots)
    k, V = cfg.k, cfg.vocab
    for q in range(cfg.batch):
        assert int(g["stop_depth"][q]) == cfg.max_depth
        for d in range(1, cfg.max_depth + 1):
            assert abs(g["H_trace"][q, d - 1] - (math.log(k) - d * math.log(V))) < 1e-3
            assert g["beam_sel"][q, d - 1].tolist() == list(range(k))
        assert g["tree_token"][q, 1:k + 1].tolist() == list(range(k))
    parity.compare_with_oracle(cfg, w, roots, g, strict=True)
    eng.close()


@pytest.mark.parametrize("k,n,launches", [(10, 12, 1), (10, 16, 1), (16, 16, 2)], ids=["keys_in_smem", "keys_from_global", "kernel"])
def test_fused_draft_rerank_inside_or_behind_the_kernel(k, n, launches):
    # The persistent kernel reranks in its 8 KB transpose buffer where the tree fits: 1111 nodes with
    # their keys, 1511 nodes with keys read from global memory; 3857 nodes go to the rerank kernel.
    cfg = S.scaled_down(S.CONFIGS["llama2_7b"], 256, 3000 + 8, threshold=NEG, k=k, max_depth=n, total_tokens=90)
    eng_s = engine_for(cfg, TC, P.DDD_LAUNCH_STREAM)
    eng_f = engine_for(cfg, TC, P.DDD_LAUNCH_FUSED)
    assert P.ddd_launches_per_draft(eng_f.handle, n) == launches
    for i in range(2):
        roots = S.make_roots(cfg, i)
        a = parity.run_gpu(eng_s, roots)
        b = parity.run_gpu(eng_f, roots)
        for name in a:
            np.testing.assert_array_equal(a[name], b[name], err_msg=name)
        parity.compare_with_oracle(cfg, weights_for(cfg), roots, b)
    eng_s.close()
    eng_f.close()


@pytest.mark.parametrize("mode", [P.DDD_LAUNCH_STREAM, P.DDD_LAUNCH_FUSED], ids=["stream", "fused"])
def test_w_may_be_released_after_create_on_the_tensor_core_path(mode):
    # ddd_create packs W into the workspace; nothing on the tensor-core path reads the original again
    cfg = small_cases()["7b"]
    eng = engine_for(cfg, TC, mode)
    eng.W.fill_(float("nan"))
    torch.cuda.synchronize()
    roots = S.make_roots(cfg, 2)
    g = parity.run_gpu(eng, roots)
    parity.compare_with_oracle(cfg, weights_for(cfg), roots, g)
    eng.close()


def test_fused_draft_equals_stream_draft_over_many_roots():
    # the blocks of the persistent kernel hand over through counters in global memory: a rare
    # ordering mistake would show as a run-to-run difference, so many drafts are compared bit for bit
    cfg = small_cases()["70b_batch"].replace(batch=3, max_depth=6)
    eng_s = engine_for(cfg, TC, P.DDD_LAUNCH_STREAM)
    eng_f = engine_for(cfg, TC, P.DDD_LAUNCH_FUSED)
    names = ("stop_depth", "n_out", "token", "parent", "cum", "mask")
    depths = set()
    for i in range(300):
        dev = parity.to_device(S.make_roots(cfg, 1000 + i), eng_s.device)
        eng_s.draft(dev["root_hidden"], dev["root_token"], dev["root_pos"])
        eng_f.draft(dev["root_hidden"], dev["root_token"], dev["root_pos"])
        torch.cuda.synchronize()
        assert int(eng_f.out["status"].item()) == 0
        for name in names:
            assert torch.equal(eng_s.out[name], eng_f.out[name]), (i, name)
        depths.update(eng_f.out["stop_depth"].cpu().tolist())
    assert len(depths) > 1 and eng_f.guards_intact()
    eng_s.close()
    eng_f.close()


def test_fused_mode_is_refused_where_it_cannot_run():
    base = S.scaled_down(S.CONFIGS["llama2_7b"], 256, 3000, threshold=NEG, max_depth=2, total_tokens=20)
    for cfg, kernel in ((base.replace(k=33), TC), (S.CONFIGS["tiny"], P.DDD_LM_HEAD_AUTO), (base, SIMT)):
        with pytest.raises(P.DddError) as err:
            P.DraftEngine(cfg, weights_for(cfg), lm_head_kernel=kernel, launch_mode=P.DDD_LAUNCH_FUSED)
        assert err.value.code == -6


def test_handles_of_different_sizes_coexist():
    # kernel attributes (dynamic shared memory limit) are per process: a smaller handle created
    # later must not take room away from a larger one created earlier
    big = small_cases()["128k_zipf"]
    small = big.replace(k=2, max_depth=2, total_tokens=3)
    eng_big = engine_for(big, TC)
    eng_small = engine_for(small, TC)
    roots = S.make_roots(big, 0)
    g = parity.run_gpu(eng_big, roots)
    parity.compare_with_oracle(big, weights_for(big), roots, g)
    g2 = parity.run_gpu(eng_small, S.make_roots(small, 0))
    parity.compare_with_oracle(small, weights_for(small), S.make_roots(small, 0), g2)
    eng_big.close()
    eng_small.close()


def test_host_gated_draft_equals_device_gated_draft():
    # the paper's control flow (host sync and decision after every pass) must give the same tree
    cfg = small_cases()["7b"]
    eng = engine_for(cfg, TC, P.DDD_LAUNCH_STREAM)
    for i in (0, 3):
        roots = S.make_roots(cfg, i)
        a = parity.run_gpu(eng, roots)
        dev = parity.to_device(roots, eng.device)
        passes = eng.draft_host_gated(dev["root_hidden"], dev["root_token"], dev["root_pos"])
        b = {k: v.numpy() for k, v in eng.results().items()}
        assert passes == int(a["stop_depth"].max())
        for name in a:
            np.testing.assert_array_equal(a[name], b[name], err_msg=name)
    eng.close()


def test_simt_and_tensor_core_kernels_agree():
    cfg = small_cases()["70b_batch"]
    roots = S.make_roots(cfg, 5)
    e1, e2 = engine_for(cfg, SIMT), engine_for(cfg, TC)
    a, b = parity.run_gpu(e1, roots), parity.run_gpu(e2, roots)
    np.testing.assert_array_equal(a["stop_depth"], b["stop_depth"])
    np.testing.assert_allclose(a["H_trace"], b["H_trace"], atol=2e-3)
    e1.close()
    e2.close()


# ----------------------------------------------------------------------------- full-size configurations
# (name, threshold, drafts, how many of them at least must be free of near-ties and therefore
# equal to the oracle's own, unreplayed decisions)
FULL_SIZE = [
    ("llama2_7b", -1.0, 16, 10), ("llama2_7b", -2.0, 16, 2), ("llama2_7b", -4.0, 16, 1), ("llama2_7b", NEG, 4, 0),
    ("vicuna_13b", -2.0, 16, 3), ("llama2_70b_b16", -2.0, 2, 4), ("llama3_8b_128k", -3.0, 4, 0)]


@pytest.mark.parametrize("name,threshold,n_drafts,min_strict", FULL_SIZE,
                         ids=[f"{c[0]}_x{c[1]:g}" for c in FULL_SIZE])
def test_full_size_configs_in_bench_launch_configuration(name, threshold, n_drafts, min_strict, record_property):
    cfg = S.CONFIGS[name].replace(threshold=threshold)
    eng = engine_for(cfg, P.DDD_LM_HEAD_AUTO, P.DDD_LAUNCH_FUSED)
    depths, strict = [], 0
    with torch.cuda.stream(torch.cuda.Stream()):
        for i in range(n_drafts):
            roots = S.make_roots(cfg, i)
            g = parity.run_gpu(eng, roots)
            ref = parity.compare_with_oracle(cfg, weights_for(cfg), roots, g)
            depths += g["stop_depth"].tolist()
            # A replay that met no near-tie had nothing to adopt: every decision of the GPU was
            # checked against a band that holds the oracle's own choice alone.  One draft per case
            # is also run again without any replay.
            strict += sum(1 for r in ref if not r.ambiguities)
            if i == 0:
                parity.strict_equal_when_unambiguous(cfg, weights_for(cfg), roots, g)
    eng.close()
    record_property("sequences", len(depths))
    record_property("sequences_without_near_tie", strict)
    record_property("stop_depths", sorted(set(depths)))
    assert strict >= min_strict, (strict, len(depths))
    if threshold == NEG:
        assert set(depths) == {cfg.max_depth}
    elif name in ("vicuna_13b", "llama2_70b_b16") or threshold in (-1.0, -4.0):
        assert len(set(depths)) > 1, depths       # sequences stop at different depths (7B at x = -2: all at 2)
