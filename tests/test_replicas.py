"""Multi-process host logic of the replica sharding (gloo, world size 2, CPU only): every
draft index is owned by exactly one rank, ranks need no data-path exchange, and the timing
reduction used by the benchmark (max over ranks) works over a process group."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import ddd_synth as S


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, n_drafts, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = list(S.shard_draft_indices(n_drafts, rank, world))
    # the per-rank inputs come from the shared seeded generator; nothing is exchanged
    cfg = S.CONFIGS["tiny"]
    roots = [S.make_roots(cfg, i) for i in mine]
    checksum = sum(float(r["root_hidden"].double().sum()) for r in roots)
    # whole-job time = max over ranks; whole-job work = sum over ranks
    t = torch.tensor([10.0 + rank], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    n = torch.tensor([float(len(mine))], dtype=torch.float64)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    gathered = [None] * world
    dist.all_gather_object(gathered, mine)
    if rank == 0:
        torch.save({"max_t": t.item(), "total": n.item(), "gathered": gathered, "checksum": checksum},
                   os.path.join(out_dir, "r0.pt"))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_replica_sharding(tmp_path):
    world, n_drafts = 2, 7
    mp.spawn(_worker, args=(world, _free_port(), n_drafts, str(tmp_path)), nprocs=world, join=True)
    res = torch.load(os.path.join(tmp_path, "r0.pt"))
    assert res["max_t"] == 11.0 and res["total"] == n_drafts
    flat = [i for part in res["gathered"] for i in part]
    assert sorted(flat) == list(range(n_drafts)) and len(set(flat)) == n_drafts
    assert [len(p) for p in res["gathered"]] == [4, 3]


def _bench_rank_worker(rank, world, port, out_dir):
    # what torchrun puts in the environment of each rank
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import contextlib
    import io
    import bench
    got_rank, got_world, local = bench.dist_setup(world, backend="gloo")
    cpu = torch.device("cpu")
    bench.barrier(got_world)
    slowest = bench.max_over_ranks(3.0 + 2.0 * got_rank, got_world, cpu)      # ms per step of this rank
    total = bench.sum_over_ranks(5.0, got_world, cpu)
    mine = list(S.shard_draft_indices(7 * got_world, got_rank, got_world))
    buf = io.StringIO()
    with contextlib.redirect_stdout(buf):
        printed = bench.emit({"value": 7 * got_world / (slowest / 1e3), "n_gpus": got_world}, got_rank)
    bench.barrier(got_world)
    bench.dist_teardown(got_world)
    torch.save({"rank": got_rank, "world": got_world, "local": local, "slowest": slowest, "total": total,
                "mine": mine, "printed": printed, "stdout": buf.getvalue()}, os.path.join(out_dir, f"b{rank}.pt"))


def test_bench_rank_logic_over_two_gloo_ranks(tmp_path):
    """bench.py's own multi-rank code: group set-up from the torchrun environment, barrier, the
    max-over-ranks time, and that rank 0 alone prints the line."""
    import json
    world = 2
    mp.spawn(_bench_rank_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    recs = [torch.load(os.path.join(tmp_path, f"b{r}.pt")) for r in range(world)]
    assert [r["rank"] for r in recs] == [0, 1] and all(r["world"] == 2 for r in recs)
    assert all(r["slowest"] == 5.0 for r in recs)            # every rank reports the slowest rank's time
    assert all(r["total"] == 10.0 for r in recs)
    assert sorted(recs[0]["mine"] + recs[1]["mine"]) == list(range(14))
    assert recs[0]["printed"] and not recs[1]["printed"] and recs[1]["stdout"] == ""
    line = json.loads(recs[0]["stdout"])
    assert line["n_gpus"] == 2 and abs(line["value"] - 14 / 5e-3) < 1e-6


def test_shard_is_a_partition_for_any_world_size():
    for n in (0, 1, 5, 32, 1000):
        for world in (1, 2, 3, 8):
            parts = [list(S.shard_draft_indices(n, r, world)) for r in range(world)]
            assert [i for p in parts for i in p] == list(range(n))
            assert max(len(p) for p in parts) - min(len(p) for p in parts) <= 1


def test_generator_is_deterministic_and_rounded_to_storage():
    cfg = S.scaled_down(S.CONFIGS["vicuna_13b"], 64, 512)
    a, b = S.make_weights(cfg), S.make_weights(cfg)
    for key in ("W", "E", "plant_next"):
        assert torch.equal(a[key], b[key])
    assert a["W"].dtype == torch.bfloat16 and a["W"].shape == (512, 64)
    frac = (a["plant_next"] >= 0).float().mean().item()
    assert 0.03 < frac < 0.2
    z = S.make_weights(S.scaled_down(S.CONFIGS["llama3_8b_128k"], 64, 512))
    assert z["bias"][0] == 0 and abs(float(z["bias"][9]) + 1.1 * 2.302585) < 1e-4
    r0, r1 = S.make_roots(cfg, 0), S.make_roots(cfg, 1)
    assert not torch.equal(r0["root_hidden"], r1["root_hidden"])
    assert torch.equal(r0["root_hidden"], S.make_roots(cfg, 0)["root_hidden"])
