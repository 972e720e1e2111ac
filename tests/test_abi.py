"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol
that include/ddd.h declares, and rejects bad arguments before touching CUDA."""
import ctypes
import os
import re

import pytest

import paper_2409_00142_b200 as P

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def good_config(**kw):
    base = dict(batch=1, hidden=256, vocab=1024, k=4, max_depth=4, total_tokens=16, dtype=P.DDD_DTYPE_FP32,
                threshold=-2.0, check_mask=0xFFFFFFFF, logit_scale=1.0, rms_eps=1e-6, plant_delta=0.0,
                device=0, lm_head_kernel=P.DDD_LM_HEAD_AUTO, launch_mode=P.DDD_LAUNCH_STREAM)
    base.update(kw)
    return P.DddConfig(**base)


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "ddd.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = sorted(set(re.findall(r"\b(ddd_[a-z_]+)\s*\(", header)))
    assert declared, "no declarations found"
    lib = P.load_library()
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in ddd.h but not exported"
    assert sorted(P.exported_symbols()) == declared


def test_workspace_bytes_and_config_validation():
    assert P.ddd_workspace_bytes(good_config()) > 0
    for bad in (dict(batch=0), dict(hidden=100), dict(k=0), dict(k=129), dict(vocab=4), dict(max_depth=0),
                dict(max_depth=33), dict(total_tokens=0), dict(total_tokens=1024), dict(dtype=7),
                dict(batch=100, k=4), dict(k=64, max_depth=32, vocab=4096), dict(lm_head_kernel=9), dict(launch_mode=5),
                dict(logit_scale=float("nan")), dict(device=-1)):
        assert P.ddd_workspace_bytes(good_config(**bad)) == 0, bad
    big = P.ddd_workspace_bytes(good_config(batch=16, hidden=8192, vocab=32000, k=10, max_depth=10,
                                            total_tokens=60, dtype=P.DDD_DTYPE_BF16))
    assert big > P.ddd_workspace_bytes(good_config())


def test_workspace_of_wide_beams_holds_the_logits_where_the_lm_head_writes_them_out():
    # beams wider than 32 on the tensor-core kernel with an unsliced vocabulary: [B k][V rounded up to 32] fp32
    shape = dict(batch=1, hidden=64, vocab=3000, max_depth=3, total_tokens=30, dtype=P.DDD_DTYPE_BF16)
    logits = 100 * 3008 * 4
    packed_w = 3008 * 64 * 2            # the tensor-core kernel's own copy of W (whole 32-row units): well under the logits here

    def extra(**kw):                    # what the tensor-core path adds over the CUDA-core path
        return (P.ddd_workspace_bytes(good_config(**shape, **kw)) -
                P.ddd_workspace_bytes(good_config(**shape, **kw, lm_head_kernel=P.DDD_LM_HEAD_SIMT)))

    assert extra(k=32) == packed_w
    assert extra(k=100) == logits + packed_w
    # a slice of a vocabulary-parallel head keeps per-block lists instead
    assert extra(k=100, vocab_begin=0, vocab_count=1504) == 1504 * 64 * 2


def test_create_rejects_bad_arguments_without_a_device():
    lib = P.load_library()
    cfg = good_config()
    out = ctypes.c_void_p(123)
    ws = P.ddd_workspace_bytes(cfg)
    fake = 0x10000   # never dereferenced: every call below fails validation first
    call = lambda c, W, E, wsp, wsb: lib.ddd_create(ctypes.byref(c), W, E, None, None, wsp, wsb,  # noqa: E731
                                                   ctypes.byref(out))
    assert call(cfg, None, fake, fake, ws) == -1 and out.value is None
    assert call(cfg, fake, None, fake, ws) == -1
    assert call(cfg, fake, fake, None, ws) == -1
    assert call(cfg, fake + 4, fake, fake, ws) == -2            # W not 16-byte aligned
    assert call(cfg, fake, fake, fake + 64, ws) == -2           # workspace not 256-byte aligned
    assert call(cfg, fake, fake, fake, ws - 1) == -3            # workspace too small
    assert call(good_config(k=0), fake, fake, fake, ws) == -1
    assert call(good_config(lm_head_kernel=P.DDD_LM_HEAD_TCGEN05), fake, fake, fake, ws) == -6  # fp32 on tensor cores
    assert lib.ddd_create(ctypes.byref(cfg), fake, fake, None, None, fake, ws, None) == -1
    assert lib.ddd_draft(None, fake, fake, fake, None, None, None) == -1
    assert lib.ddd_draft_host(None, fake, fake, fake, None, None) == -1
    assert lib.ddd_draft_host_gated(None, fake, fake, fake, None, None, None, None) == -1
    assert lib.ddd_lm_head_pass(None, None) == -1
    assert lib.ddd_destroy(None) == -1
    assert lib.ddd_launches_per_draft(None, 1) < 0 and lib.ddd_lm_head_blocks(None) < 0 and lib.ddd_fused_pass_kind(None) < 0


def test_verify_greedy_rejects_bad_arguments_without_a_device():
    fake = 0x10000   # never dereferenced: every call below fails validation first
    out = P.DddVerifyOutput(**{name: fake for name, _ in P.DddVerifyOutput._fields_})
    for sizes in [(0, 4, 4), (1, 0, 4), (1, 1025, 4), (1, 4, 0), (1, 4, 33)]:
        with pytest.raises(P.DddError) as err:
            P.ddd_verify_greedy(*sizes, fake, fake, fake, fake, out, 0)
        assert err.value.code == -1, sizes
    for missing in range(4):
        ptrs = [fake] * 4
        ptrs[missing] = None
        with pytest.raises(P.DddError):
            P.ddd_verify_greedy(1, 4, 4, *ptrs, out, 0)
    with pytest.raises(P.DddError):
        P.ddd_verify_greedy(1, 4, 4, fake, fake, fake, fake, P.DddVerifyOutput(), 0)


def test_strerror_covers_every_code():
    seen = {P.ddd_strerror(c) for c in range(0, -7, -1)}
    assert len(seen) == 7 and "unknown error code" not in seen
    assert P.ddd_strerror(-99) == "unknown error code"


def test_engine_refuses_to_run_without_cuda():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    import ddd_synth as S
    cfg = S.CONFIGS["tiny"]
    with pytest.raises(RuntimeError):
        P.DraftEngine(cfg, {"W": torch.zeros(1), "E": torch.zeros(1)})
