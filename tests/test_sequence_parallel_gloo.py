"""Sequence-parallel sampling (§6.1: scatter metadata, all-to-all logits, sample local rows, gather
token ids) on 2 and 3 gloo ranks on CPU.  Step (3) is stood in for by the oracle (allowed in tests);
what is checked is the exchange layout, the batch padding (§6.2), the metadata scatter and the
gather: every rank must end up with exactly the single-worker result of the whole batch."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2606_01927_b200 import workloads as W


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _oracle_sample_fn(V):
    from oracle import albireo_oracle as O

    def fn(pieces, meta, row_base, step):
        t, rows, vs = pieces.shape
        assert t * vs == V
        x = pieces.permute(1, 0, 2).reshape(rows, V).contiguous().numpy()       # row b = its t pieces in order
        g = lambda k, dt: None if meta.get(k) is None else meta[k].numpy().astype(dt)
        hid = hoff = None
        if meta.get("history_ids") is not None:
            hoff = meta["history_offsets"].numpy().astype(np.int32)
            hid = np.ascontiguousarray(meta["history_ids"].numpy().astype(np.int32)[: max(int(hoff[-1]), 1)])
        seeds = None if meta.get("seeds") is None else meta["seeds"].numpy().view(np.uint64)
        w = W.Workload("local", rows, V, W.F32, x, temperature=g("temperature", np.float32), top_k=g("top_k", np.int32),
                       top_p=g("top_p", np.float32), min_p=g("min_p", np.float32),
                       repetition_penalty=g("repetition_penalty", np.float32),
                       presence_penalty=g("presence_penalty", np.float32),
                       frequency_penalty=g("frequency_penalty", np.float32),
                       history_ids=hid, history_offsets=hoff, seeds=seeds, step=step, row_base=row_base)
        o = O.sample(w)
        return torch.from_numpy(o.tokens.astype(np.int32)), torch.from_numpy(o.logprobs.astype(np.float32))
    return fn


def _worker(rank, world, port, s_rows, q):
    from oracle import albireo_oracle as O
    from paper_2606_01927_b200 import sequence_parallel as SP
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        V = 600 * world
        w = W.random_small(88, B=s_rows, V=V, dtype=W.F32)
        vs = V // world
        # what a tensor-parallel LM head leaves on this worker: its vocabulary shard of all rows
        local_shard = torch.from_numpy(np.ascontiguousarray(w.logits[:, rank * vs:(rank + 1) * vs]))
        lay = SP.layout(s_rows)
        assert lay.rows == -(-s_rows // world) and lay.row_base == rank * lay.rows
        meta = None
        if rank == 0:       # only the driver worker knows the requests' parameters
            meta = {f: torch.from_numpy(getattr(w, f)) for f in SP.ROW_FIELDS if f != "seeds"}
            meta["seeds"] = torch.from_numpy(w.seeds.view(np.int64))
            meta["history_ids"] = torch.from_numpy(w.history_ids)
            meta["history_offsets"] = torch.from_numpy(w.history_offsets)
        mine = SP.scatter_metadata(meta, lay, "cpu")
        lo, hi = min(s_rows, lay.row_base), min(s_rows, lay.row_base + lay.rows)
        assert (mine["temperature"][: hi - lo].numpy() == w.temperature[lo:hi]).all()
        o = w.history_offsets
        assert (mine["history_ids"][: int(o[hi] - o[lo])].numpy() == w.history_ids[o[lo]:o[hi]]).all()
        fn = _oracle_sample_fn(V)
        pieces = SP.exchange_logits(local_shard, lay)
        if hi > lo:       # piece j of my rows is columns [j vs, (j+1) vs) of the full matrix
            for j in range(world):
                assert (pieces[j, : hi - lo].numpy() == w.logits[lo:hi, j * vs:(j + 1) * vs]).all()
        tok, lp = SP.sample_step(fn, local_shard, mine, lay, step=w.step)
        ref = O.sample(w)
        ok_sp = bool((tok.numpy() == ref.tokens).all()) and bool((lp.numpy() == ref.logprobs.astype(np.float32)).all())
        # the arrangement it replaces gives the same tokens
        meta_all = None
        if rank == 0:
            meta_all = {k: v for k, v in meta.items()}
        tok2, lp2 = SP.gather_then_sample_step(fn, local_shard, meta_all, s_rows, step=w.step)
        ok_gather = bool((tok2.numpy() == ref.tokens).all())
        q.put((rank, ok_sp, ok_gather, int(tok.numel())))
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world,s_rows", [(2, 7), (2, 8), (3, 4)])
def test_sequence_parallel_steps_reproduce_the_single_worker_result(world, s_rows):
    ctx = mp.get_context("spawn")
    q = ctx.SimpleQueue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, s_rows, q)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(timeout=180)
        assert p.exitcode == 0
    got = sorted(q.get() for _ in range(world))
    assert [g[0] for g in got] == list(range(world))
    assert all(g[1] and g[2] and g[3] == s_rows for g in got)
