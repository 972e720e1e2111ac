"""Host side of the vocabulary-parallel LM head, on CPU.  (1) The slice partition.  (2) The
protocol itself over a two-rank gloo group: each rank forms, with the oracle's own steps, the record
of its slice of the vocabulary - per row the slice's maximum logit, its sum of exponentials and its
k best (logit, token) pairs, 8 (k + 1) bytes per row - the records are all-gathered, and the merged
result must be the log-softmax, log-sum-exp and top-k of the whole vocabulary as the oracle
computes them directly, planted columns included."""
import math
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import ddd_synth as S
import paper_2409_00142_b200 as P
from oracle import ddd_oracle as O


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_vocab_slices_partition_the_vocabulary():
    for vocab in (33, 1000, 1024, 32000, 128256, 40037):
        for world in (1, 2, 3, 4, 8, 16):
            parts = [P.vocab_slice(vocab, world, r) for r in range(world)]
            pos = 0
            for begin, count in parts:
                assert begin == pos and count >= 0 and (count == 0 or begin % 32 == 0)
                pos += count
            assert pos == vocab
            counts = [c for _, c in parts if c]
            assert max(counts) - min(counts) <= 32 + (-vocab) % 32


def _slice_record(W, bias, h, scale, begin, count, k, planted):
    """(M, S, top-k logits, top-k tokens) per row over tokens [begin, begin + count), the planted
    column of each row left out (its logit depends on the maximum over ALL other tokens)."""
    z = O.lm_head_logits(W[begin:begin + count], h, scale, None if bias is None else bias[begin:begin + count])
    rows = z.shape[0]
    M, Ssum = np.full(rows, -np.inf), np.zeros(rows)
    top_z, top_t = np.full((rows, k), -np.inf), np.full((rows, k), -1, np.int64)
    for r in range(rows):
        zr = z[r].copy()
        c = planted[r]
        if begin <= c < begin + count:
            zr[c - begin] = -np.inf
        M[r] = zr.max()
        if np.isfinite(M[r]):
            Ssum[r] = np.exp(zr - M[r]).sum()
        order = O.topk_desc(zr, min(k, count))
        order = order[np.isfinite(zr[order])]
        top_z[r, :len(order)] = zr[order]
        top_t[r, :len(order)] = order + begin
    return M, Ssum, top_z, top_t


def _merge_records(records, k, planted, delta):
    """What every rank does with the gathered records, in rank order."""
    rows = records[0][0].shape[0]
    lse, toks, lps = np.zeros(rows), np.zeros((rows, k), np.int64), np.zeros((rows, k))
    for r in range(rows):
        M = max(rec[0][r] for rec in records)
        Ssum = sum(rec[1][r] * math.exp(rec[0][r] - M) for rec in records if rec[1][r] > 0)
        zs = np.concatenate([rec[2][r] for rec in records])
        ts = np.concatenate([rec[3][r] for rec in records])
        if planted[r] >= 0:
            zc = M + delta
            M2 = max(M, zc)
            Ssum = Ssum * math.exp(M - M2) + math.exp(zc - M2)
            M = M2
            zs, ts = np.append(zs, zc), np.append(ts, planted[r])
        keep = ts >= 0
        zs, ts = zs[keep], ts[keep]
        order = np.lexsort((ts, -zs))[:k]                    # logit descending, ties to the lower token
        lse[r] = M + math.log(Ssum)
        toks[r] = ts[order]
        lps[r] = np.minimum(zs[order] - lse[r], 0.0)
    return lse, toks, lps


def _rank_worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = S.scaled_down(S.CONFIGS["vicuna_13b"], 64, 1000 + 9, k=10, batch=1)
    w = S.make_weights(cfg)
    rows = 10
    rng = np.random.default_rng(5)
    h = O.to_f64(torch.from_numpy(rng.standard_normal((rows, cfg.hidden)).astype(np.float32)).to(torch.bfloat16))
    bias = rng.standard_normal(cfg.vocab)
    planted = np.array([-1, 17, -1, 999, 500, -1, 1008, -1, 3, -1])     # some in either slice, some nowhere
    begin, count = P.vocab_slice(cfg.vocab, world, rank)
    M, Ssum, top_z, top_t = _slice_record(w["W"], bias, h, cfg.logit_scale, begin, count, cfg.k, planted)
    # one record: rows x (k + 1) eight-byte words, as on the device: k (logit, token) pairs, then (max, sum)
    mine = torch.from_numpy(np.concatenate([top_z, top_t.astype(np.float64), M[:, None], Ssum[:, None]], axis=1))
    gathered = [torch.zeros_like(mine) for _ in range(world)]
    dist.all_gather(gathered, mine)
    k = cfg.k
    records = [(g[:, 2 * k].numpy(), g[:, 2 * k + 1].numpy(), g[:, :k].numpy(), g[:, k:2 * k].numpy().astype(np.int64))
               for g in gathered]
    lse, toks, lps = _merge_records(records, k, planted, cfg.plant_delta)
    torch.save({"lse": lse, "toks": toks, "lps": lps, "planted": planted, "h": h, "bias": bias,
                "bytes_per_row": 8 * (k + 1)}, os.path.join(out_dir, f"v{rank}.pt"))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_record_exchange_reproduces_the_whole_vocabulary(tmp_path):
    world = 2
    mp.spawn(_rank_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    res = [torch.load(os.path.join(tmp_path, f"v{r}.pt"), weights_only=False) for r in range(world)]
    cfg = S.scaled_down(S.CONFIGS["vicuna_13b"], 64, 1000 + 9, k=10, batch=1)
    w = S.make_weights(cfg)
    z = O.lm_head_logits(w["W"], res[0]["h"], cfg.logit_scale, res[0]["bias"])
    assert res[0]["bytes_per_row"] * 10 == 880           # the record of a 10-row pass at k = 10
    for r in range(z.shape[0]):
        zr = O.apply_plant(z[r], int(res[0]["planted"][r]), cfg.plant_delta)
        lp = O.log_softmax_row(zr)
        M = zr.max()
        for rank in range(world):
            assert abs(res[rank]["lse"][r] - (M + math.log(np.exp(zr - M).sum()))) < 1e-9
            assert res[rank]["toks"][r].tolist() == O.topk_desc(lp, cfg.k).tolist()
            np.testing.assert_allclose(res[rank]["lps"][r], lp[res[rank]["toks"][r]], rtol=0, atol=1e-9)
    for name in ("lse", "toks", "lps"):                  # both ranks hold the same merged result
        np.testing.assert_array_equal(res[0][name], res[1][name])
