#!/usr/bin/env python
"""Benchmark of the draft-tree hot path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one batch of `--drafts-per-step` whole drafts (every expansion pass, the gate,
the draft step, the rerank and the mask) of the 7B-shaped workload, each from its own seeded
root.  `value` is drafts per second with inputs resident in HBM; `e2e` is the same metric
through ddd_draft_host with pinned host buffers.  With N > 1 (torchrun) every rank runs the
same number of drafts on its own GPU on a disjoint block of draft indices (replicas: no
data-path collective), and the time is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

import ddd_synth as S  # noqa: E402

METRIC = "drafts_per_sec"
UNIT = "drafts/s"
NEG = -1e30
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes (read + write) of one launch of the persistent draft kernel (a full-depth draft) from the
# ncu capture summarised under profiles/, valid only while the kernel source is the one that was profiled.
NCU_TRAFFIC = {"llama2_7b": {"bytes": 2942.2e6, "source_sha256_16": "f7456c78b72c5525",
                             "profile": "profiles/draft_fused_llama2_7b.md"},
               "llama2_70b_b16": {"bytes": 5131.3e6, "source_sha256_16": "f7456c78b72c5525",
                                  "profile": "profiles/draft_fused_llama2_70b_b16.md"}}
BEAM_WIDTHS = (5, 10, 20, 50, 75, 100)      # fixed-depth-6 sweep: the widths of the paper's appendix table
OTHER_WORKLOADS = ("vicuna_13b", "llama2_70b_b16", "llama3_8b_128k")
CLOCK_QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
               "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
               "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama2_7b", choices=list(S.CONFIGS))
    ap.add_argument("--threshold", type=float, default=None, help="override the workload's threshold x")
    ap.add_argument("--beam-width", type=int, default=None,
                    help="override the workload's beam width k (beyond 32: not with --launch-mode fused)")
    ap.add_argument("--max-depth", type=int, default=None, help="override the workload's maximum depth n")
    ap.add_argument("--drafts-per-step", type=int, default=1000,
                    help="distinct seeded roots drafted per step and rank (the 7B workload is stated on 1000 drafts)")
    ap.add_argument("--lm-head-reps", type=int, default=200)
    ap.add_argument("--cpu-sample", type=int, default=None, help="drafts the CPU baseline times")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--no-width-sweep", action="store_true",
                    help="skip the fixed-depth-6 drafts at the beam widths of the paper's appendix table")
    ap.add_argument("--no-other-workloads", action="store_true",
                    help="skip the short runs of the other bf16 workloads (13B-, 70B-shaped, 128k vocabulary)")
    ap.add_argument("--dist-backend", default="nccl", choices=["nccl", "gloo"],
                    help="process-group backend of a multi-rank run (gloo: host-side tests of the rank logic)")
    ap.add_argument("--launch-mode", default="fused", choices=["fused", "graph", "stream", "plain"],
                    help="fused: one persistent kernel per draft; plain: ordinary stream-ordered launches of the "
                         "kernel-by-kernel path, which a profiler's launch list can follow")
    return ap.parse_args()


def ncu_traffic(workload: str):
    import hashlib
    ent = NCU_TRAFFIC.get(workload)
    if not ent:
        return None
    digest = hashlib.sha256()
    try:
        for name in ("draft_fused.cu", "tc_ptx.cuh", "ddd_common.cuh", "tree_device.cuh"):      # the kernel and what it inlines
            with open(os.path.join(ROOT, "paper_2409_00142_b200", "csrc", name), "rb") as f:
                digest.update(f.read())
    except OSError:
        return None
    if digest.hexdigest()[:16] != ent["source_sha256_16"]:
        return None                  # kernel changed since the counters were taken
    return ent["bytes"]


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.file = None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={CLOCK_QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.file.read().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                smax.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.file.close()
        os.unlink(self.file.name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(smax), reasons=sorted(reasons), samples=len(sm))
        return out


def dist_setup(n_gpus: int, backend: str = "nccl"):
    """Joins the process group torchrun describes in the environment (none for a single process)."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        if backend == "nccl":
            dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        else:
            dist.init_process_group(backend)
    return rank, world, local


def dist_teardown(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def emit(line: dict, rank: int) -> bool:
    """Rank 0 prints the one JSON line of the run; the other ranks print nothing."""
    if rank != 0:
        return False
    print(json.dumps(line), flush=True)
    return True


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(value: float, world: int, device) -> float:
    if world == 1:
        return value
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, world: int, device) -> float:
    if world == 1:
        return value
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def timed_drafts(eng, roots_dev, steps: int, warmup: int, world: int, device):
    """Returns (ms per step as max over ranks, mean stop depth)."""
    stream = torch.cuda.current_stream(device)

    def one_step():
        for r in roots_dev:
            eng.draft(r["root_hidden"], r["root_token"], r["root_pos"])

    for _ in range(warmup):
        one_step()
    torch.cuda.synchronize(device)
    barrier(world)
    torch.cuda.synchronize(device)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        one_step()
    e1.record(stream)
    torch.cuda.synchronize(device)
    # a draft that recorded an error (a bounded wait that ran out) publishes nothing and would look fast
    assert int(eng.out["status"].item()) == 0, "device reported an error status during the timed drafts"
    barrier(world)
    ms = e0.elapsed_time(e1) / steps
    return max_over_ranks(ms, world, device), ms


def mean_stop_depth(eng, roots_dev, device):
    depths = []
    for r in roots_dev:
        eng.draft(r["root_hidden"], r["root_token"], r["root_pos"])
        torch.cuda.synchronize(device)
        assert int(eng.out["status"].item()) == 0, "device reported an error status"
        depths.append(eng.out["stop_depth"].cpu().tolist())     # one list per draft (one entry per sequence)
    return depths


def _mean(depth_lists):
    flat = [d for lst in depth_lists for d in lst]
    return sum(flat) / len(flat)


def run_reference(args):
    """The CPU oracle, as it stands, timed on the host cores on a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import ddd_oracle as O
    cfg = S.CONFIGS[args.workload]
    if args.threshold is not None:
        cfg = cfg.replace(threshold=args.threshold)
    w = S.make_weights(cfg)
    sample = args.cpu_sample or 1
    times, depths = [], []
    idx = 0
    for step in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        for _ in range(sample):
            res = O.draft(cfg, w, **S.make_roots(cfg, idx))
            depths += [r.stop_depth for r in res]
            idx += 1
        dt = time.perf_counter() - t0
        if step >= args.warmup:
            times.append(dt)
    ms = 1e3 * sum(times) / len(times)
    value = sample * cfg.batch / (ms / 1e3)
    cores = O.num_threads()
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "threshold": cfg.threshold, "drafts_per_step": sample,
                   "batch": cfg.batch, "mean_stop_depth": sum(depths) / len(depths)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"{sample} draft(s) of {cfg.name} per step, x={cfg.threshold}"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    emit(line, rank)


def stack_roots(cfg, indices):
    """The seeded roots of the given draft indices as three host tensors [n][B][Hd], [n][B], [n][B]."""
    roots = [S.make_roots(cfg, i) for i in indices]
    return {k: torch.stack([r[k] for r in roots]).contiguous() for k in ("root_hidden", "root_token", "root_pos")}


def rows_of(stacked):
    """Per-draft views (no copies) of stacked roots."""
    n = stacked["root_token"].shape[0]
    return [{k: v[i] for k, v in stacked.items()} for i in range(n)]


def time_lm_head(eng, reps: int, stream, device, flush):
    """The LM-head kernel alone, two ways.  Back to back: `reps` launches in a row, the period between
    them (each launch's set-up and first loads overlap the tail of the one before, as they overlap the
    select kernel inside a draft).  Isolated: one launch at a time behind a write of a buffer larger
    than L2, timed by its own pair of events (nothing to overlap with, cold L2)."""
    for _ in range(5):
        eng.lm_head_pass()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(reps):
        eng.lm_head_pass()
    e1.record(stream)
    torch.cuda.synchronize(device)
    period_us = 1e3 * e0.elapsed_time(e1) / reps
    n_iso = max(5, min(40, reps // 5))
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_iso)]
    for a, b in pairs:
        flush.zero_()                  # evicts W from L2 and keeps the queue busy until the launch is enqueued
        a.record(stream)
        eng.lm_head_pass()
        b.record(stream)
    torch.cuda.synchronize(device)
    iso_us = statistics.median(1e3 * a.elapsed_time(b) for a, b in pairs)
    return period_us, iso_us


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    import paper_2409_00142_b200 as P

    rank, world, local = dist_setup(args.gpus, args.dist_backend)
    device = torch.device("cuda", local)
    torch.cuda.set_device(device)
    cfg = S.CONFIGS[args.workload]
    if args.threshold is not None:
        cfg = cfg.replace(threshold=args.threshold)
    if args.beam_width is not None:
        cfg = cfg.replace(k=args.beam_width)
    if args.max_depth is not None:
        cfg = cfg.replace(max_depth=args.max_depth)
    weights = S.make_weights(cfg)
    n_per_rank = args.drafts_per_step
    my_indices = S.shard_draft_indices(n_per_rank * world, rank, world)
    roots_host = stack_roots(cfg, my_indices)
    stream = torch.cuda.Stream(device)
    mode = {"fused": P.DDD_LAUNCH_FUSED, "graph": P.DDD_LAUNCH_GRAPH, "stream": P.DDD_LAUNCH_STREAM,
            "plain": P.DDD_LAUNCH_PLAIN}[args.launch_mode]
    peak, peak_kind = measured_peak()
    elt = 4 if cfg.dtype == "fp32" else 2
    w_bytes = cfg.vocab * cfg.hidden * elt
    sub_steps = max(3, args.steps // 4)

    with torch.cuda.stream(stream):
        eng = P.DraftEngine(cfg, weights, device=local, launch_mode=mode, with_trace=False)
        dev_weights = {"W": eng.W, "E": eng.E, "bias": eng.bias, "plant_next": eng.plant_next}
        roots_dev = rows_of({k: v.to(device) for k, v in roots_host.items()})
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)      # larger than the 126 MB L2
        torch.cuda.synchronize(device)
        depth_lists = mean_stop_depth(eng, roots_dev, device)
        depth_mean = _mean(depth_lists)
        stop_depths = [max(lst) for lst in depth_lists]     # passes each draft needs

        sampler = ClockSampler(local)
        sampler.start()
        ms_step, _ = timed_drafts(eng, roots_dev, args.steps, args.warmup, world, device)
        clocks = sampler.stop()
        drafts_total = n_per_rank * world * cfg.batch
        value = drafts_total / (ms_step / 1e3)
        us_per_draft = 1e3 * ms_step / n_per_rank
        passes_mean = _mean([[d] for d in stop_depths])

        # ---- the LM-head kernel alone: CUDA events on the launching stream, W (> L2) streamed each launch
        lm_us, lm_iso_us = time_lm_head(eng, args.lm_head_reps, stream, device, flush)
        achieved = w_bytes / (lm_us * 1e-6) / 1e9

        def variant(c, launch=None, w=None):
            launch = mode if launch is None else launch
            if launch == P.DDD_LAUNCH_FUSED and c.k > 32:
                launch = P.DDD_LAUNCH_GRAPH          # beams wider than 32 run kernel by kernel
            return P.DraftEngine(c, w or dev_weights, device=local, launch_mode=launch, with_trace=False)

        # ---- fixed full depth (x = -inf): per-expansion-step time independent of where drafts stop
        extra = {}
        step_us = None
        if not args.no_sweep:
            full_roots = roots_dev[:max(1, min(len(roots_dev), 64))]
            eng_full = variant(cfg.replace(threshold=NEG))
            ms_full, _ = timed_drafts(eng_full, full_roots, sub_steps, args.warmup, world, device)
            per_draft_us = 1e3 * ms_full / len(full_roots)
            step_us = per_draft_us / cfg.max_depth
            extra["full_depth"] = {"drafts_per_sec": len(full_roots) * world * cfg.batch / (ms_full / 1e3),
                                   "us_per_draft": per_draft_us, "us_per_expansion_step": step_us,
                                   "passes": cfg.max_depth, "drafts_per_step": len(full_roots) * world}
            eng_full.close()
            if cfg.name == "llama2_7b" and args.threshold is None:
                sweep = {}
                for x in S.LLAMA2_7B_THRESHOLDS:
                    ex = variant(cfg.replace(threshold=x))
                    dm = _mean(mean_stop_depth(ex, roots_dev, device))
                    msx, _ = timed_drafts(ex, roots_dev, sub_steps, args.warmup, world, device)
                    sweep[str(x)] = {"drafts_per_sec": drafts_total / (msx / 1e3), "mean_stop_depth": dm,
                                     "drafts": n_per_rank * world}
                    ex.close()
                extra["threshold_sweep"] = sweep

        # ---- where the gate lives: the paper checks the heuristic on the host after a synchronisation
        # (Section 2; its "Strict" variants of Section 3.4 do so after every draft call); here the check
        # is on the device.  Same drafts, same results, host-gated: launch pass, synchronise, read, decide.
        if not args.no_sweep and world == 1:
            gate_roots = roots_dev[:min(len(roots_dev), 128)]

            def host_gated_rate(engine, reps):
                for r in gate_roots[:4]:
                    engine.draft_host_gated(r["root_hidden"], r["root_token"], r["root_pos"])
                torch.cuda.synchronize(device)
                t0 = time.perf_counter()
                for _ in range(reps):
                    for r in gate_roots:
                        engine.draft_host_gated(r["root_hidden"], r["root_token"], r["root_pos"])
                torch.cuda.synchronize(device)
                return reps * len(gate_roots) * cfg.batch / (time.perf_counter() - t0)

            def device_gated_rate(engine):
                ms, _ = timed_drafts(engine, gate_roots, sub_steps, args.warmup, world, device)
                return len(gate_roots) * cfg.batch / (ms / 1e3)

            reps = max(2, args.steps // 10)
            extra["gate_placement"] = {"device_gate_drafts_per_sec": device_gated_rate(eng),
                                       "host_gate_drafts_per_sec": host_gated_rate(eng, reps),
                                       "note": "host gate = stream sync + 4-byte read after every pass"}
            # the paper's own parameters (Section 3.2): n = 11, S = {5, 7, 9}, x = -0.3, w = 10, beside
            # EAGLE-2's fixed depth 6 at the same width
            pmask = sum(1 << (s_ - 1) for s_ in (5, 7, 9))
            pe = variant(cfg.replace(max_depth=11, check_mask=pmask, threshold=-0.3, k=10), mode)
            pdm = _mean(mean_stop_depth(pe, gate_roots, device))
            fixed6 = variant(cfg.replace(max_depth=6, threshold=NEG, k=10), mode)
            extra["paper_parameters"] = {"n": 11, "S": [5, 7, 9], "x": -0.3, "w": 10, "mean_stop_depth": pdm,
                                         "device_gate_drafts_per_sec": device_gated_rate(pe),
                                         "host_gate_drafts_per_sec": host_gated_rate(pe, reps),
                                         "eagle2_fixed_depth6_drafts_per_sec": device_gated_rate(fixed6)}
            pe.close()
            fixed6.close()

        # ---- beam width vs run time at fixed depth 6 (the paper's appendix reports an almost flat curve)
        if not args.no_width_sweep and not args.no_sweep and world == 1:
            sweep_w = {}
            wide_roots = roots_dev[:min(len(roots_dev), 32)]
            for kw in BEAM_WIDTHS:
                we = variant(cfg.replace(k=kw, max_depth=6, threshold=NEG, total_tokens=60), mode)
                wms, _ = timed_drafts(we, wide_roots, sub_steps, args.warmup, world, device)
                sweep_w[str(kw)] = {"us_per_draft": 1e3 * wms / len(wide_roots),
                                    "us_per_expansion_step": 1e3 * wms / len(wide_roots) / 6}
                we.close()
            extra["beam_width_sweep_depth6"] = sweep_w

        # ---- vocabulary-parallel LM head, compute side only: the G ranks' kernels of a pass (LM head over a
        # slice, fold to one record per row, select over the G records) run one after the other on this one
        # GPU; the time of a pass divided by G is what one rank computes.  No exchange is timed: one GPU.
        if not args.no_sweep and world == 1 and cfg.dtype == "bf16":
            G = 8
            vcfg = cfg.replace(threshold=NEG)
            ranks = [P.DraftEngine(vcfg, dev_weights, device=local, with_trace=False,
                                   vocab_slice=P.vocab_slice(vcfg.vocab, G, g)) for g in range(G)]
            nbytes = P.ddd_shard_records_bytes(ranks[0].c, G)
            recs = [[torch.zeros(nbytes, dtype=torch.uint8, device=device) for _ in range(2)] for _ in range(G)]
            flags = [[torch.zeros(G, dtype=torch.int32, device=device) for _ in range(2)] for _ in range(G)]

            def sharded_draft(r):
                for e in ranks:
                    e.shard_begin(r["root_hidden"], r["root_token"], r["root_pos"])
                for d in range(1, vcfg.max_depth + 1):
                    par = d & 1
                    for g, e in enumerate(ranks):
                        e.shard_lm_head(d, g, G, [recs[q][par] for q in range(G)], [flags[q][par] for q in range(G)])
                    for g, e in enumerate(ranks):
                        e.shard_select(d, recs[g][par], G, flags[g][par])

            for r in roots_dev[:2]:
                sharded_draft(r)
            torch.cuda.synchronize(device)
            # replayed from a captured graph: launched call by call from Python the 4 x G small kernels of a pass
            # would measure the host, not the device
            vp_graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(vp_graph, stream=stream):
                sharded_draft(roots_dev[0])
            vp_graph.replay()
            torch.cuda.synchronize(device)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            n_vp = 8
            e0.record(stream)
            for _ in range(n_vp):
                vp_graph.replay()
            e1.record(stream)
            torch.cuda.synchronize(device)
            del vp_graph
            assert all(int(e.out["status"].item()) == 0 for e in ranks)
            per_pass = 1e3 * e0.elapsed_time(e1) / n_vp / vcfg.max_depth
            extra["vocab_parallel"] = {
                "ranks": G, "us_per_pass_per_rank_compute": per_pass / G, "us_per_pass_all_ranks_serialised": per_pass,
                "record_bytes_per_rank_per_pass": nbytes // G,
                "note": "the ranks' kernels run back to back on one GPU; no exchange is timed (unmeasured on hardware)"}
            for e in ranks:
                e.close()
            del ranks, recs, flags

        # ---- end to end through the host-buffer entry point (pinned host memory, copies inside)
        host_out = eng.make_host_out(pinned=True)
        pinned = rows_of({k: v.pin_memory() for k, v in roots_host.items()})
        for r in pinned[:4]:
            eng.draft_host(r["root_hidden"], r["root_token"], r["root_pos"], host_out)
        torch.cuda.synchronize(device)
        barrier(world)
        t0 = time.perf_counter()
        e2e_steps = max(2, args.steps // 4)
        for _ in range(e2e_steps):
            for r in pinned:
                eng.draft_host(r["root_hidden"], r["root_token"], r["root_pos"], host_out)    # raises on a bad status
        torch.cuda.synchronize(device)
        e2e_ms = 1e3 * (time.perf_counter() - t0) / e2e_steps
        e2e_ms = max_over_ranks(e2e_ms, world, device)
        h2d = sum(v.numel() * v.element_size() for v in pinned[0].values()) * n_per_rank
        d2h = sum(v.numel() * v.element_size() for v in host_out.values()) * n_per_rank
        launches = sum(P.ddd_launches_per_draft(eng.handle, dd) for dd in stop_depths) * args.steps
        blocks = P.ddd_lm_head_blocks(eng.handle)
        eng.close()

        # ---- the other bf16 workloads, briefly: LM-head bandwidth, drafts/s at the workload's own
        # threshold, time per expansion step at full depth
        if not args.no_other_workloads and not args.no_sweep and world == 1 and args.workload == "llama2_7b":
            del eng, dev_weights, roots_dev
            others = {}
            for name in OTHER_WORKLOADS:
                oc = S.CONFIGS[name]
                ow = S.make_weights(oc)
                oe = variant(oc, mode, ow)
                odw = {"W": oe.W, "E": oe.E, "bias": oe.bias, "plant_next": oe.plant_next}
                n_o = max(4, 64 // oc.batch)
                oroots = rows_of({k: v.to(device) for k, v in stack_roots(oc, range(n_o)).items()})
                odepth = _mean(mean_stop_depth(oe, oroots, device))
                oms, _ = timed_drafts(oe, oroots, sub_steps, args.warmup, world, device)
                o_period, o_iso = time_lm_head(oe, max(20, args.lm_head_reps // 4), stream, device, flush)
                of = variant(oc.replace(threshold=NEG), mode, odw)
                ofms, _ = timed_drafts(of, oroots[:8], 3, args.warmup, world, device)
                o_bytes = oc.vocab * oc.hidden * 2
                o_step = 1e3 * ofms / len(oroots[:8]) / oc.max_depth
                others[name] = {
                    "threshold": oc.threshold, "beam_rows": oc.batch * oc.k, "mean_stop_depth": odepth,
                    "fused_pass_kind": P.ddd_fused_pass_kind(of.handle),
                    "drafts_per_sec": n_o * oc.batch / (oms / 1e3),
                    "lm_head_us_back_to_back": o_period, "lm_head_us_isolated": o_iso,
                    "lm_head_gbs": o_bytes / (o_period * 1e-6) / 1e9, "lm_head_frac": o_bytes / (o_period * 1e-6) / 1e9 / peak,
                    "us_per_expansion_step_full_depth": o_step,
                    "step_frac": o_bytes / (o_step * 1e-6) / 1e9 / peak}
                if others[name]["fused_pass_kind"]:
                    others[name]["lm_head_note"] = ("lm_head_* time the LM-head kernel of the kernel-by-kernel path; the "
                                                    "persistent kernel's pass for many beam rows is organised differently "
                                                    "(both tiles of a block per stage, a floor per row) and is timed by "
                                                    "us_per_expansion_step_full_depth")
                of.close()
                oe.close()
                del oe, of, ow, odw, oroots
                torch.cuda.empty_cache()
            extra["other_workloads"] = others

    if rank != 0:
        dist_teardown(world)
        return

    lm_head_alone = {"kernel": "lm_head_tc_kernel (one pass per launch)", "achieved": achieved, "frac": achieved / peak,
                     "us_per_launch": lm_us,
                     "us_per_launch_kind": "period of back-to-back launches (set-up and first loads overlap the predecessor)",
                     "us_per_launch_isolated": lm_iso_us, "frac_isolated": w_bytes / (lm_iso_us * 1e-6) / 1e9 / peak,
                     "algorithmic_bytes_per_launch": w_bytes, "frac_of_8TBs_nominal": achieved / 8000.0}
    # the whole draft against the same peak: W bytes of the passes a draft needs / time per draft
    draft_frac = passes_mean * w_bytes / (us_per_draft * 1e-6) / 1e9 / peak
    if args.launch_mode == "fused" and step_us is not None:
        # One launch of the persistent kernel is a whole draft, so the dominant kernel is timed on
        # full-depth drafts (x = -inf): n passes, each streaming W once.  The events bracket whole
        # drafts, i.e. they include the small rerank kernel behind every launch.
        fused_bytes = cfg.max_depth * w_bytes
        fused_us = step_us * cfg.max_depth
        fused_gbs = fused_bytes / (fused_us * 1e-6) / 1e9
        roofline = {"bound": "hbm", "achieved": fused_gbs, "peak": peak, "unit": "GB/s", "frac": fused_gbs / peak,
                    "traffic": ncu_traffic(cfg.name), "peak_kind": f"of {peak_kind}",
                    "kernel": "draft_fused_kernel (%d expansion steps per launch, full-depth drafts)" % cfg.max_depth,
                    "us_per_launch": fused_us, "algorithmic_bytes_per_launch": fused_bytes,
                    "frac_of_8TBs_nominal": fused_gbs / 8000.0, "blocks": blocks,
                    "step_frac": fused_gbs / peak, "step_frac_of_8TBs_nominal": fused_gbs / 8000.0,
                    "draft_frac": draft_frac, "lm_head_alone": lm_head_alone}
    else:
        roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                    "frac": achieved / peak, "traffic": None, "peak_kind": f"of {peak_kind}",
                    "kernel": "lm_head", "us_per_launch": lm_us,
                    "us_per_launch_kind": lm_head_alone["us_per_launch_kind"],
                    "us_per_launch_isolated": lm_iso_us, "frac_isolated": lm_head_alone["frac_isolated"],
                    "algorithmic_bytes_per_launch": w_bytes,
                    "frac_of_8TBs_nominal": achieved / 8000.0, "blocks": blocks, "draft_frac": draft_frac}
        if step_us is not None:
            # the expansion step (LM head + select / gate / draft step) at full depth: the figure the
            # 70-%-of-HBM-bandwidth target is stated on
            roofline["step_frac"] = w_bytes / (step_us * 1e-6) / 1e9 / peak
            roofline["step_frac_of_8TBs_nominal"] = w_bytes / (step_us * 1e-6) / 1e9 / 8000.0
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": cfg.dtype if cfg.dtype != "fp32" else "f32", "data": "synthetic",
        "config": {"workload": cfg.name, "batch": cfg.batch, "hidden": cfg.hidden, "vocab": cfg.vocab,
                   "k": cfg.k, "max_depth": cfg.max_depth, "total_tokens": cfg.total_tokens,
                   "threshold": cfg.threshold, "drafts_per_step": n_per_rank * world,
                   "mean_stop_depth": depth_mean, "parallelism": f"replicas{world}",
                   "l2": "inputs larger than L2: every pass streams W (%.0f MB) from HBM" % (w_bytes / 1e6),
                   "launch": args.launch_mode},
        "clocks": clocks,
        "e2e": {"value": n_per_rank * world * cfg.batch / (e2e_ms / 1e3), "unit": UNIT,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "transfer": ("ddd_draft_host: the kernel reads the roots from and writes the rows to pinned host memory"
                             if args.launch_mode == "fused" else
                             "ddd_draft_host: one copy command in each direction through a pinned bounce buffer")},
        "gpu_launches": launches,
        "gpu_launches_kind": "computed: ddd_launches_per_draft(stop depth) summed over the timed drafts",
        "us_per_draft": us_per_draft,
        "roofline": roofline,
    }
    line.update(extra)
    if not args.no_cpu_baseline and world == 1:
        from oracle import ddd_oracle as O
        # a bounded sample of the same workload: drafts until about 12 s of CPU work (or --cpu-sample drafts)
        cpu_roots = rows_of(roots_host)
        sample, t0 = 0, time.perf_counter()
        while True:
            O.draft(cfg, weights, **cpu_roots[sample % len(cpu_roots)])
            sample += 1
            dt = time.perf_counter() - t0
            if (args.cpu_sample and sample >= args.cpu_sample) or (not args.cpu_sample and (dt > 12.0 or sample >= 400)):
                break
        line["cpu_baseline"] = {"value": sample * cfg.batch / dt, "unit": UNIT, "cores": O.num_threads(),
                                "kind": "oracle",
                                "sample": f"{sample} draft(s) of {cfg.name}, x={cfg.threshold}, {dt:.1f} s"}
    emit(line, rank)
    dist_teardown(world)


if __name__ == "__main__":
    main()
