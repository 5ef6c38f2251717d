"""Row sharding over ranks (world size 2, gloo on CPU): the host-side logic of the N > 1 path.
The sampler call itself is stood in for by the oracle (allowed in tests); what is checked is that
shard + row_base + padding + gather reproduce the single-rank result exactly."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2606_01927_b200 import sharding, workloads as W


def test_plan_covers_rows_once_and_pads_equally():
    for B in (0, 1, 7, 8, 9, 255, 256):
        for world in (1, 2, 3, 4, 8):
            shards = sharding.plan(B, world)
            assert len({s.rows for s in shards}) == 1
            covered = [i for s in shards for i in range(s.lo, s.hi)]
            assert covered == list(range(B))
            assert all(s.hi - s.lo <= s.rows for s in shards)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    from oracle import albireo_oracle as O
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = W.random_small(77, B=9, V=600, dtype=W.BF16)        # 9 rows over 2 ranks: one padded row
        shard = sharding.plan(w.B, world)[rank]
        part = sharding.shard_workload(w, shard)
        assert part.B == shard.rows and part.row_base == shard.lo
        out = O.sample(part)
        tok = torch.from_numpy(out.tokens.astype(np.int64))
        lp = torch.from_numpy(out.logprobs.copy())
        toks = [torch.empty_like(tok) for _ in range(world)]
        lps = [torch.empty_like(lp) for _ in range(world)]
        dist.all_gather(toks, tok)
        dist.all_gather(lps, lp)
        if rank == 0:
            shards = sharding.plan(w.B, world)
            got_t = np.concatenate([sharding.unpad(t.numpy(), s) for t, s in zip(toks, shards)])
            got_l = np.concatenate([sharding.unpad(t.numpy(), s) for t, s in zip(lps, shards)])
            ref = O.sample(w)
            q.put((bool((got_t == ref.tokens).all()), bool((got_l == ref.logprobs).all()), len(got_t)))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_reproduce_the_single_rank_result():
    ctx = mp.get_context("spawn")
    q = ctx.SimpleQueue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    same_tokens, same_logprobs, n = q.get()
    assert n == 9 and same_tokens and same_logprobs
