"""ctypes binding with the same names as the C ABI (include/ddd.h), plus a small
convenience class that owns the torch buffers.  Argument marshalling only."""
from __future__ import annotations

import ctypes
import os
from typing import Dict, Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_NAME = "libddd.so"
_lib = None

DDD_DTYPE_FP32, DDD_DTYPE_BF16 = 0, 1
DDD_LM_HEAD_AUTO, DDD_LM_HEAD_SIMT, DDD_LM_HEAD_TCGEN05 = 0, 1, 2
DDD_LAUNCH_STREAM, DDD_LAUNCH_GRAPH, DDD_LAUNCH_PLAIN, DDD_LAUNCH_FUSED = 0, 1, 2, 3


class DddError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {ddd_strerror(code)} ({code})")


class DddConfig(ctypes.Structure):
    _fields_ = [
        ("batch", ctypes.c_int32), ("hidden", ctypes.c_int32), ("vocab", ctypes.c_int32),
        ("k", ctypes.c_int32), ("max_depth", ctypes.c_int32), ("total_tokens", ctypes.c_int32),
        ("dtype", ctypes.c_int32), ("threshold", ctypes.c_float), ("check_mask", ctypes.c_uint32),
        ("logit_scale", ctypes.c_float), ("rms_eps", ctypes.c_float), ("plant_delta", ctypes.c_float),
        ("device", ctypes.c_int32), ("lm_head_kernel", ctypes.c_int32), ("launch_mode", ctypes.c_int32),
        ("vocab_begin", ctypes.c_int32), ("vocab_count", ctypes.c_int32),
    ]


class DddOutput(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in (
        "n_out", "stop_depth", "token", "parent", "depth", "position", "cum", "mask", "H_trace", "status")]


class DddTrace(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in (
        "node_id", "tree_token", "tree_parent", "tree_cum", "beam_sel", "row_lse")]


class DddVerifyOutput(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in (
        "n_accepted", "accepted_rows", "next_token", "n_leaves", "leaf_paths", "status")]


def library_path() -> str:
    return os.path.join(_HERE, _LIB_NAME)


def load_library():
    """Loads libddd.so from the package directory.  There is no fallback: a missing
    library is an error (build it with `python -m paper_2409_00142_b200.build`)."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not os.path.exists(path):
        raise ImportError(f"{path} not found: the CUDA library is not built "
                          "(run `python -m paper_2409_00142_b200.build`)")
    lib = ctypes.CDLL(path)
    vp, i32p = ctypes.c_void_p, ctypes.c_void_p
    lib.ddd_workspace_bytes.restype = ctypes.c_size_t
    lib.ddd_workspace_bytes.argtypes = [ctypes.POINTER(DddConfig)]
    lib.ddd_create.restype = ctypes.c_int
    lib.ddd_create.argtypes = [ctypes.POINTER(DddConfig), vp, vp, vp, i32p, vp, ctypes.c_size_t,
                               ctypes.POINTER(ctypes.c_void_p)]
    lib.ddd_draft.restype = ctypes.c_int
    lib.ddd_draft.argtypes = [vp, vp, i32p, i32p, ctypes.POINTER(DddOutput), ctypes.POINTER(DddTrace), vp]
    lib.ddd_draft_host_gated.restype = ctypes.c_int
    lib.ddd_draft_host_gated.argtypes = [vp, vp, i32p, i32p, ctypes.POINTER(DddOutput), ctypes.POINTER(DddTrace), vp,
                                         ctypes.POINTER(ctypes.c_int32)]
    lib.ddd_draft_host.restype = ctypes.c_int
    lib.ddd_draft_host.argtypes = [vp, vp, i32p, i32p, ctypes.POINTER(DddOutput), vp]
    lib.ddd_lm_head_pass.restype = ctypes.c_int
    lib.ddd_lm_head_pass.argtypes = [vp, vp]
    lib.ddd_launches_per_draft.restype = ctypes.c_int
    lib.ddd_launches_per_draft.argtypes = [vp, ctypes.c_int32]
    lib.ddd_lm_head_blocks.restype = ctypes.c_int
    lib.ddd_lm_head_blocks.argtypes = [vp]
    lib.ddd_fused_pass_kind.restype = ctypes.c_int
    lib.ddd_fused_pass_kind.argtypes = [vp]
    lib.ddd_lm_head_topk_noalloc.restype = ctypes.c_int
    lib.ddd_lm_head_topk_noalloc.argtypes = [vp, vp, vp, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                             ctypes.c_int32, ctypes.c_int32, ctypes.c_float, vp, vp, vp, vp]
    lib.ddd_shard_records_bytes.restype = ctypes.c_size_t
    lib.ddd_shard_records_bytes.argtypes = [ctypes.POINTER(DddConfig), ctypes.c_int32]
    lib.ddd_shard_begin.restype = ctypes.c_int
    lib.ddd_shard_begin.argtypes = [vp, vp, i32p, i32p, ctypes.POINTER(DddOutput), ctypes.POINTER(DddTrace), vp]
    lib.ddd_shard_lm_head.restype = ctypes.c_int
    lib.ddd_shard_lm_head.argtypes = [vp, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                      ctypes.POINTER(ctypes.c_void_p), ctypes.POINTER(ctypes.c_void_p),
                                      ctypes.c_int32, vp]
    lib.ddd_shard_select.restype = ctypes.c_int
    lib.ddd_shard_select.argtypes = [vp, ctypes.c_int32, vp, ctypes.c_int32, vp, vp]
    lib.ddd_verify_greedy.restype = ctypes.c_int
    lib.ddd_verify_greedy.argtypes = [ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, i32p, i32p, i32p, i32p,
                                      ctypes.POINTER(DddVerifyOutput), vp]
    lib.ddd_destroy.restype = ctypes.c_int
    lib.ddd_destroy.argtypes = [vp]
    lib.ddd_strerror.restype = ctypes.c_char_p
    lib.ddd_strerror.argtypes = [ctypes.c_int]
    _lib = lib
    return lib


def exported_symbols():
    """Names this binding expects the library to export (all of include/ddd.h)."""
    return ["ddd_workspace_bytes", "ddd_create", "ddd_draft", "ddd_draft_host", "ddd_draft_host_gated", "ddd_lm_head_pass",
            "ddd_launches_per_draft", "ddd_lm_head_blocks", "ddd_fused_pass_kind", "ddd_lm_head_topk_noalloc", "ddd_verify_greedy",
            "ddd_shard_records_bytes", "ddd_shard_begin", "ddd_shard_lm_head", "ddd_shard_select",
            "ddd_destroy", "ddd_strerror"]


# ----------------------------------------------------------------------------- same-name wrappers
def ddd_strerror(code: int) -> str:
    return load_library().ddd_strerror(int(code)).decode()


def ddd_workspace_bytes(cfg: DddConfig) -> int:
    return int(load_library().ddd_workspace_bytes(ctypes.byref(cfg)))


def ddd_create(cfg: DddConfig, W: int, E: int, bias: Optional[int], plant_next: Optional[int],
               workspace: int, workspace_bytes: int) -> int:
    """Returns the handle (an integer address).  Pointer arguments are device addresses."""
    out = ctypes.c_void_p()
    rc = load_library().ddd_create(ctypes.byref(cfg), W, E, bias, plant_next, workspace, workspace_bytes,
                                   ctypes.byref(out))
    if rc != 0:
        raise DddError(rc, "ddd_create")
    return out.value


def ddd_draft(handle: int, root_hidden: int, root_token: int, root_pos: int, out: DddOutput,
              trace: Optional[DddTrace], stream: int) -> None:
    rc = load_library().ddd_draft(handle, root_hidden, root_token, root_pos, ctypes.byref(out),
                                  ctypes.byref(trace) if trace is not None else None, stream)
    if rc != 0:
        raise DddError(rc, "ddd_draft")


def ddd_draft_host_gated(handle: int, root_hidden: int, root_token: int, root_pos: int, out: DddOutput,
                         trace: Optional[DddTrace], stream: int) -> int:
    """The paper's control flow: a host synchronisation and decision after every pass.  Returns the
    number of passes launched."""
    n = ctypes.c_int32(0)
    rc = load_library().ddd_draft_host_gated(handle, root_hidden, root_token, root_pos, ctypes.byref(out),
                                             ctypes.byref(trace) if trace is not None else None, stream,
                                             ctypes.byref(n))
    if rc != 0:
        raise DddError(rc, "ddd_draft_host_gated")
    return int(n.value)


def ddd_draft_host(handle: int, root_hidden: int, root_token: int, root_pos: int, out: DddOutput,
                   stream: int) -> None:
    rc = load_library().ddd_draft_host(handle, root_hidden, root_token, root_pos, ctypes.byref(out), stream)
    if rc != 0:
        raise DddError(rc, "ddd_draft_host")


def ddd_lm_head_pass(handle: int, stream: int) -> None:
    rc = load_library().ddd_lm_head_pass(handle, stream)
    if rc != 0:
        raise DddError(rc, "ddd_lm_head_pass")


def ddd_launches_per_draft(handle: int, passes_needed: int) -> int:
    return int(load_library().ddd_launches_per_draft(handle, int(passes_needed)))


def ddd_lm_head_blocks(handle: int) -> int:
    return int(load_library().ddd_lm_head_blocks(handle))


def ddd_fused_pass_kind(handle: int) -> int:
    return int(load_library().ddd_fused_pass_kind(handle))


def ddd_lm_head_topk_noalloc(W: int, bias: Optional[int], hidden_rows: int, dtype: int, rows: int, hidden: int,
                             vocab: int, k: int, logit_scale: float, out_token: int, out_logprob: int,
                             out_lse: int, stream: int) -> None:
    """LM-head pass with top-k for callers that cannot allocate device memory: the scratch is a
    fixed array inside the library (see include/ddd.h).  All pointers are device addresses."""
    rc = load_library().ddd_lm_head_topk_noalloc(W, bias, hidden_rows, dtype, rows, hidden, vocab, k,
                                                 logit_scale, out_token, out_logprob, out_lse, stream)
    if rc != 0:
        raise DddError(rc, "ddd_lm_head_topk_noalloc")


def ddd_verify_greedy(batch: int, t_rows: int, max_depth: int, n_out: int, token: int, parent: int,
                      target_argmax: int, out: DddVerifyOutput, stream: int) -> None:
    """Greedy acceptance walk and leaf-path table of emitted trees.  Pointers are device addresses."""
    rc = load_library().ddd_verify_greedy(batch, t_rows, max_depth, n_out, token, parent, target_argmax,
                                          ctypes.byref(out), stream)
    if rc != 0:
        raise DddError(rc, "ddd_verify_greedy")


def ddd_shard_records_bytes(cfg: DddConfig, slots: int) -> int:
    return int(load_library().ddd_shard_records_bytes(ctypes.byref(cfg), int(slots)))


def ddd_shard_begin(handle: int, root_hidden: int, root_token: int, root_pos: int, out: DddOutput,
                    trace: Optional[DddTrace], stream: int) -> None:
    rc = load_library().ddd_shard_begin(handle, root_hidden, root_token, root_pos, ctypes.byref(out),
                                        ctypes.byref(trace) if trace is not None else None, stream)
    if rc != 0:
        raise DddError(rc, "ddd_shard_begin")


def ddd_shard_lm_head(handle: int, d: int, slot: int, slots: int, records_dst, flags_dst, stream: int) -> None:
    """records_dst / flags_dst: sequences of device addresses, one per destination record set
    (flags_dst may be None)."""
    n = len(records_dst)
    rec = (ctypes.c_void_p * n)(*records_dst)
    flg = None if flags_dst is None else (ctypes.c_void_p * n)(*flags_dst)
    rc = load_library().ddd_shard_lm_head(handle, d, slot, slots, rec, flg, n, stream)
    if rc != 0:
        raise DddError(rc, "ddd_shard_lm_head")


def ddd_shard_select(handle: int, d: int, records: int, slots: int, flags: Optional[int], stream: int) -> None:
    rc = load_library().ddd_shard_select(handle, d, records, slots, flags, stream)
    if rc != 0:
        raise DddError(rc, "ddd_shard_select")


def vocab_slice(vocab: int, world: int, rank: int):
    """(first token id, number of rows) of rank's slice of a vocabulary split over `world` ranks:
    whole 32-row units (the granule the tensor-core kernel streams), as even as they go, the
    ragged end with the last rank that has rows."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    units = (vocab + 31) // 32
    base, extra = divmod(units, world)
    first = rank * base + min(rank, extra)
    mine = base + (1 if rank < extra else 0)
    begin = min(first * 32, vocab)
    return begin, max(0, min((first + mine) * 32, vocab) - begin)


def ddd_destroy(handle: int) -> None:
    rc = load_library().ddd_destroy(handle)
    if rc != 0:
        raise DddError(rc, "ddd_destroy")


# ----------------------------------------------------------------------------- convenience
class DraftEngine:
    """Owns the torch buffers one handle needs: device copies of the weights, the workspace
    and one set of output / trace tensors.  All computation happens inside the library."""

    GUARD_BYTES = 4096
    GUARD_PATTERN = 0xA5

    def __init__(self, cfg, weights: Dict, device: int = 0, lm_head_kernel: int = DDD_LM_HEAD_AUTO,
                 launch_mode: int = DDD_LAUNCH_STREAM, with_trace: bool = True, vocab_slice=None):
        """vocab_slice = (begin, count): this engine owns only those rows of the LM head (one rank
        of a vocabulary-parallel head); it then drafts through the shard_* methods."""
        import torch
        load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("DraftEngine needs a CUDA device; there is no CPU path")
        self.torch = torch
        self.cfg = cfg
        self.device = torch.device("cuda", device)
        self.dtype = torch.float32 if cfg.dtype == "fp32" else torch.bfloat16
        dev = self.device
        v_begin, v_count = vocab_slice if vocab_slice is not None else (0, 0)
        if vocab_slice is not None and v_count < 1:
            raise ValueError("an empty vocabulary slice cannot have a handle")
        rows = slice(v_begin, v_begin + v_count) if v_count else slice(None)
        self.W = weights["W"][rows].to(dev, self.dtype).contiguous()
        self.E = weights["E"].to(dev, self.dtype).contiguous()
        self.bias = None if weights.get("bias") is None else weights["bias"][rows].to(dev, torch.float32).contiguous()
        pn = weights.get("plant_next")
        self.plant_next = None if pn is None else pn.to(dev, torch.int32).contiguous()
        self.c = DddConfig(
            batch=cfg.batch, hidden=cfg.hidden, vocab=cfg.vocab, k=cfg.k, max_depth=cfg.max_depth,
            total_tokens=cfg.total_tokens, dtype=DDD_DTYPE_FP32 if cfg.dtype == "fp32" else DDD_DTYPE_BF16,
            threshold=max(cfg.threshold, -3.0e38), check_mask=cfg.check_mask & 0xFFFFFFFF,
            logit_scale=cfg.logit_scale, rms_eps=cfg.rms_eps, plant_delta=cfg.plant_delta, device=device,
            lm_head_kernel=lm_head_kernel, launch_mode=launch_mode, vocab_begin=v_begin, vocab_count=v_count)
        nbytes = ddd_workspace_bytes(self.c)
        if nbytes == 0:
            raise DddError(-1, "ddd_workspace_bytes")
        # the workspace sits between two guard bands filled with a pattern: a kernel that wrote outside
        # what ddd_workspace_bytes promised shows up in guards_intact()
        guard = self.GUARD_BYTES
        self.workspace = torch.full((nbytes + 256 + 2 * guard,), self.GUARD_PATTERN, dtype=torch.uint8, device=dev)
        ws_ptr = (self.workspace.data_ptr() + guard + 255) // 256 * 256
        self._ws_offset = ws_ptr - self.workspace.data_ptr()
        self._ws_bytes = nbytes
        self.handle = ddd_create(self.c, self.W.data_ptr(), self.E.data_ptr(),
                                 None if self.bias is None else self.bias.data_ptr(),
                                 None if self.plant_next is None else self.plant_next.data_ptr(),
                                 ws_ptr, nbytes)
        B, T, n, k = cfg.batch, cfg.total_tokens + 1, cfg.max_depth, cfg.k
        W32 = (T + 31) // 32
        Nn = 1 + k + (n - 1) * k * k
        i32, f32 = torch.int32, torch.float32
        self.out = {
            "n_out": torch.zeros(B, dtype=i32, device=dev), "stop_depth": torch.zeros(B, dtype=i32, device=dev),
            "token": torch.zeros(B, T, dtype=i32, device=dev), "parent": torch.zeros(B, T, dtype=i32, device=dev),
            "depth": torch.zeros(B, T, dtype=i32, device=dev), "position": torch.zeros(B, T, dtype=i32, device=dev),
            "cum": torch.zeros(B, T, dtype=f32, device=dev), "mask": torch.zeros(B, T, W32, dtype=i32, device=dev),
            "H_trace": torch.zeros(B, n, dtype=f32, device=dev), "status": torch.zeros(1, dtype=i32, device=dev),
        }
        self.c_out = DddOutput(**{name: t.data_ptr() for name, t in self.out.items()})
        self.trace = None
        self.c_trace = None
        if with_trace:
            self.trace = {
                "node_id": torch.zeros(B, T, dtype=i32, device=dev),
                "tree_token": torch.zeros(B, Nn, dtype=i32, device=dev),
                "tree_parent": torch.zeros(B, Nn, dtype=i32, device=dev),
                "tree_cum": torch.zeros(B, Nn, dtype=f32, device=dev),
                "beam_sel": torch.zeros(B, n, k, dtype=i32, device=dev),
                "row_lse": torch.zeros(B, n, k, dtype=f32, device=dev),
            }
            self.c_trace = DddTrace(**{name: t.data_ptr() for name, t in self.trace.items()})

    def stream_ptr(self) -> int:
        return self.torch.cuda.current_stream(self.device).cuda_stream

    def draft(self, root_hidden, root_token, root_pos) -> None:
        """Enqueues one draft on torch's current stream.  Inputs must be device tensors that stay
        alive until the stream has been synchronised; results land in self.out / self.trace."""
        assert root_hidden.is_cuda and root_hidden.dtype == self.dtype and root_hidden.is_contiguous()
        assert root_token.is_cuda and root_token.dtype == self.torch.int32
        assert root_pos.is_cuda and root_pos.dtype == self.torch.int32
        ddd_draft(self.handle, root_hidden.data_ptr(), root_token.data_ptr(), root_pos.data_ptr(),
                  self.c_out, self.c_trace, self.stream_ptr())

    def draft_host_gated(self, root_hidden, root_token, root_pos) -> int:
        """Like draft(), but the host waits and decides after every pass (the paper's "Strict" flow)."""
        return ddd_draft_host_gated(self.handle, root_hidden.data_ptr(), root_token.data_ptr(), root_pos.data_ptr(),
                                    self.c_out, self.c_trace, self.stream_ptr())

    def draft_host(self, root_hidden, root_token, root_pos, host_out: Dict) -> None:
        """Host-buffer variant: CPU tensors in, CPU tensors (same names as self.out) out."""
        cached = getattr(self, "_host_out_struct", None)
        if cached is None or cached[0] is not host_out:       # marshal the ten pointers once per buffer set
            cached = (host_out, DddOutput(**{name: host_out[name].data_ptr() for name in self.out}))
            self._host_out_struct = cached
        c_out = cached[1]
        ddd_draft_host(self.handle, root_hidden.data_ptr(), root_token.data_ptr(), root_pos.data_ptr(),
                       c_out, self.stream_ptr())

    def make_host_out(self, pinned: bool = True) -> Dict:
        return {name: self.torch.zeros(t.shape, dtype=t.dtype, pin_memory=pinned) for name, t in self.out.items()}

    def verify_greedy(self, target_argmax) -> Dict:
        """Runs the acceptance walk on the tree of the last draft.  `target_argmax` is a device int32
        tensor [B][T]; returns device tensors named like the fields of ddd_verify_output."""
        torch = self.torch
        B, T, n = self.cfg.batch, self.cfg.total_tokens + 1, self.cfg.max_depth
        assert target_argmax.is_cuda and target_argmax.dtype == torch.int32 and target_argmax.is_contiguous()
        assert tuple(target_argmax.shape) == (B, T)
        if getattr(self, "verify_out", None) is None:
            i32, dev = torch.int32, self.device
            self.verify_out = {
                "n_accepted": torch.zeros(B, dtype=i32, device=dev),
                "accepted_rows": torch.zeros(B, n, dtype=i32, device=dev),
                "next_token": torch.zeros(B, dtype=i32, device=dev),
                "n_leaves": torch.zeros(B, dtype=i32, device=dev),
                "leaf_paths": torch.zeros(B, T, n + 1, dtype=i32, device=dev),
                "status": torch.zeros(1, dtype=i32, device=dev),
            }
            self.c_verify_out = DddVerifyOutput(**{name: t.data_ptr() for name, t in self.verify_out.items()})
        ddd_verify_greedy(B, T, n, self.out["n_out"].data_ptr(), self.out["token"].data_ptr(),
                          self.out["parent"].data_ptr(), target_argmax.data_ptr(), self.c_verify_out,
                          self.stream_ptr())
        return self.verify_out

    def shard_begin(self, root_hidden, root_token, root_pos) -> None:
        ddd_shard_begin(self.handle, root_hidden.data_ptr(), root_token.data_ptr(), root_pos.data_ptr(),
                        self.c_out, self.c_trace, self.stream_ptr())

    def shard_lm_head(self, d: int, slot: int, slots: int, records_dst, flags_dst=None) -> None:
        """records_dst / flags_dst: device tensors (record sets and flag arrays) to publish into."""
        ddd_shard_lm_head(self.handle, d, slot, slots, [t.data_ptr() for t in records_dst],
                          None if flags_dst is None else [t.data_ptr() for t in flags_dst], self.stream_ptr())

    def shard_select(self, d: int, records, slots: int, flags=None) -> None:
        ddd_shard_select(self.handle, d, records.data_ptr(), slots,
                         None if flags is None else flags.data_ptr(), self.stream_ptr())

    def guards_intact(self) -> bool:
        """True while the bytes just before and just after the workspace still hold their pattern."""
        before = self.workspace[:self._ws_offset]
        after = self.workspace[self._ws_offset + self._ws_bytes:]
        return bool((before == self.GUARD_PATTERN).all().item()) and bool((after == self.GUARD_PATTERN).all().item())

    def lm_head_pass(self) -> None:
        ddd_lm_head_pass(self.handle, self.stream_ptr())

    def results(self) -> Dict:
        """Synchronises and returns CPU copies of outputs (and trace)."""
        self.torch.cuda.synchronize(self.device)
        res = {name: t.cpu() for name, t in self.out.items()}
        if self.trace is not None:
            res.update({name: t.cpu() for name, t in self.trace.items()})
        return res

    def close(self) -> None:
        if getattr(self, "handle", None):
            ddd_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
