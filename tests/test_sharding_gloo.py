"""The N > 1 path: rows are split across ranks with no data-path collective; the optional output
gather is exercised here with two gloo ranks on CPU."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2605_02888_b200.shard import gather_rows, row_range


@pytest.mark.parametrize("B,world", [(256, 1), (256, 8), (10, 4), (3, 8), (0, 2), (1024, 3)])
def test_row_ranges_partition_the_batch(B, world):
    seen = []
    for r in range(world):
        rr = row_range(B, r, world)
        seen += list(rr)
        assert abs(len(rr) - B / world) < 1
    assert seen == list(range(B))


def _worker(rank, world, port, B, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    rows = row_range(B, rank, world)
    full_tok = torch.arange(B * 3, dtype=torch.int32).view(B, 3)
    full_h = torch.arange(B, dtype=torch.float32) * 0.5
    local = {"out_tokens": full_tok[rows.start:rows.stop].clone(), "H": full_h[rows.start:rows.stop].clone()}
    got = gather_rows(local, B)
    ok = torch.equal(got["out_tokens"], full_tok) and torch.equal(got["H"], full_h)
    q.put((rank, bool(ok)))
    dist.destroy_process_group()


@pytest.mark.parametrize("B", [7, 8])
def test_gather_rows_two_gloo_ranks(B):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, B, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
    assert res == [(0, True), (1, True)]


# ---- vocabulary shards: the two exchanges of the sharded step, two gloo ranks on CPU ----
def _exchange_worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2605_02888_b200.vocab_shard import exchange_gather, exchange_max
    B, J = 5, 7
    mine = torch.full((B, J, 4), float(rank + 1))
    allst = torch.zeros(world, B, J, 4)
    exchange_gather(allst, mine)
    ok = all(bool((allst[r] == r + 1).all()) for r in range(world))       # shard order = rank order
    w = torch.full((B, 2), 0.25 * (rank + 1), dtype=torch.float64)
    allw = torch.zeros(world, B, 2, dtype=torch.float64)
    exchange_gather(allw, w)
    ok = ok and all(bool((allw[r] == 0.25 * (r + 1)).all()) for r in range(world))
    toks = torch.full((B, 3), -1, dtype=torch.int32)
    toks[:, 0] = 11                      # accepted token, the same on every rank
    toks[rank, 1] = 100 + rank           # the fresh token of row `rank` lives on this rank
    exchange_max(toks)
    want = torch.full((B, 3), -1, dtype=torch.int32)
    want[:, 0] = 11
    for r in range(world):
        want[r, 1] = 100 + r
    ok = ok and torch.equal(toks, want)
    q.put((rank, bool(ok)))
    dist.destroy_process_group()


def test_vocab_shard_exchanges_two_gloo_ranks():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_exchange_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
    assert res == [(0, True), (1, True)]
