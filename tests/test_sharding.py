"""Multi-GPU path on CPU: shard by request, two gloo ranks, no collective on the data path.

Each rank evaluates its shard with the oracle (the CUDA kernels need a GPU); gathering the shards
must reproduce the unsharded result exactly, because a request and its candidates are an independent
unit (Eq. 1, Eq. 11)."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

from paper_2607_27744_b200 import sharding, workloads as wl


def test_partition_covers_every_request_once_and_balances():
    cfg = wl.CONFIGS[5]
    counts = wl.candidate_counts(cfg)
    lens = wl.sequence_lengths(cfg)
    cost = sharding.request_cost(counts, lens, c_linear=1.0, c_attn=0.01, c_glm=0.5)
    for world in (2, 4, 8):
        parts = sharding.partition_requests(cost, world)
        allr = np.concatenate(parts)
        assert np.array_equal(np.sort(allr), np.arange(cfg.R))
        loads = np.array([cost[p].sum() for p in parts])
        assert loads.max() <= loads.mean() + cost.max()          # LPT bound
        assert loads.max() / loads.mean() < 1.05


def test_shard_rows_builds_local_offsets():
    off = np.array([0, 3, 3, 7, 9], np.int32)
    rows, local = sharding.shard_rows(off, np.array([0, 2]))
    assert rows.tolist() == [0, 1, 2, 3, 4, 5, 6] and local.tolist() == [0, 3, 7]
    rows, local = sharding.shard_rows(off, np.array([], np.int64))
    assert rows.size == 0 and local.tolist() == [0]


def test_replicated_global_batch_shards_into_equal_weak_scaling_pieces():
    """bench.py --gpus N builds a global batch of N copies of the configuration's requests and gives
    every rank its shard: equal-cost requests must split into N shards of the single-GPU size that
    together cover every candidate once."""
    cfg = wl.CONFIGS[2].with_(R=16)
    co = wl.cand_offsets(cfg)
    for world in (1, 2, 4, 8):
        glob = sharding.replicate_offsets(co, world)
        assert glob.size == world * cfg.R + 1 and glob[-1] == world * co[-1]
        shards = [sharding.shard_batch(glob, world, r) for r in range(world)]
        assert all(sh.requests.size == cfg.R and sh.cand_offsets[-1] == co[-1] for sh in shards)
        rows = np.concatenate([sh.cand_rows for sh in shards])
        assert np.array_equal(np.sort(rows), np.arange(glob[-1]))


def test_oversized_request_is_cut_and_every_candidate_is_scored_once():
    """One request with most of the batch's candidates cannot be balanced whole: with max_share its
    candidates go to several ranks (each with a copy of the request's own tensors), every candidate row
    is owned exactly once, and the ranks' loads are even."""
    co = wl.offsets_from_counts([5, 4000, 0, 7, 300, 12])
    so = wl.offsets_from_counts([40, 100, 7, 0, 64, 33])
    for world in (2, 4):
        whole = [sharding.shard_batch(co, world, r) for r in range(world)]
        assert max(int(s.cand_offsets[-1]) for s in whole) >= 4000           # the request cannot be balanced whole
        cut = [sharding.shard_batch(co, world, r, seq_offsets=so, max_share=0.5) for r in range(world)]
        rows = np.concatenate([s.cand_rows for s in cut])
        assert np.array_equal(np.sort(rows), np.arange(co[-1]))
        loads = np.array([int(s.cand_offsets[-1]) for s in cut])
        assert loads.max() - loads.min() <= 8
        for s in cut:
            # local offsets describe the rows, and every local request carries its own sequence
            assert s.cand_offsets[-1] == s.cand_rows.size and s.cand_offsets.size == s.requests.size + 1
            assert np.array_equal(np.diff(s.seq_offsets), np.diff(so)[s.requests])
            m = np.repeat(s.requests, np.diff(s.cand_offsets))
            assert np.array_equal(m, np.searchsorted(co, s.cand_rows, side="right") - 1)   # rows belong to their request
        assert sum(1 for s in cut if 1 in s.requests) >= 2                   # request 1 really is on several ranks


def _worker(rank, world, port, out_q, max_share=None):
    sys.path.insert(0, ROOT)
    from oracle import rocs_ref as ref
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = wl.CONFIGS[1].with_(R=7)
    co, so = wl.cand_offsets(cfg), wl.seq_offsets(cfg)
    if max_share is not None:   # one request dominates the batch
        co = wl.offsets_from_counts([3, 90, 0, 5, 2, 7, 1])
    lin, att = wl.linear_inputs(cfg, co), wl.dca_inputs(cfg, co, so)
    sh = sharding.shard_batch(co, world, rank, seq_offsets=so, c_attn=0.05, max_share=max_share)   # the helper bench.py --gpus N uses
    mine, rows, co_l, seq_rows, so_l = sh.requests, sh.cand_rows, sh.cand_offsets, sh.seq_rows, sh.seq_offsets
    y = ref.ikbo_linear(co_l, lin["XR"][mine], lin["XC"][rows], lin["W"])
    o = ref.dca_attention(co_l, so_l, att["Q"][rows], att["K"][seq_rows], att["V"][seq_rows])
    # timing reduction used by the benchmark: max over ranks
    t = torch.tensor([float(rank + 1)], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    gathered = [None] * world
    dist.all_gather_object(gathered, (rows, y, o))
    if rank == 0:
        N = int(co[-1])
        Y = np.zeros((N, cfg.d_out))
        O = np.zeros((N, 1, cfg.H, cfg.dh))
        seen = np.zeros(N, bool)
        for r_, y_, o_ in gathered:
            assert not seen[r_].any()
            seen[r_] = True
            Y[r_], O[r_] = y_, o_
        want_y = ref.ikbo_linear(co, lin["XR"], lin["XC"], lin["W"])
        want_o = ref.dca_attention(co, so, att["Q"], att["K"], att["V"])
        out_q.put((bool(seen.all()), bool(np.array_equal(Y, want_y)), bool(np.array_equal(O, want_o)), float(t.item())))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("max_share", [None, 0.5])
def test_two_gloo_ranks_reproduce_the_unsharded_result(max_share):
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000 + (0 if max_share is None else 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q, max_share)) for r in range(2)]
    for p in procs:
        p.start()
    res = q.get(timeout=180)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res == (True, True, True, 2.0)
