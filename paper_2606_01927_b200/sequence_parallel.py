"""Sequence-parallel sampling over the workers of a tensor-parallel group (section 6.1).

After the language-model head every worker holds a vocabulary shard ``[s, v / t]`` of the logits
of all ``s`` rows.  Instead of gathering them on one worker, the group
  (1) scatters the per-row sampling metadata,
  (2) exchanges logits with an all-to-all so that worker ``r`` holds all ``v`` logits of rows
      ``[r s'/t, (r+1) s'/t)`` (``s'`` = ``s`` padded to a multiple of ``t``, section 6.2),
  (3) samples its rows, and
  (4) all-gathers one (token id, log-probability) pair per row.
The all-to-all needs no packing on either side: chunk ``j`` of the send buffer is rows
``[j s'/t, (j+1) s'/t)`` of the local shard as they lie in memory, and the receive buffer
``[t, s'/t, v/t]`` is handed to the sampler as it is, which reads every row from its ``t`` pieces
(``num_segments`` of the C ABI).  Draws use the global row id, so the result does not depend on ``t``.

Only ``torch.distributed`` plumbing lives here; step (3) is a callable, in the product the CUDA
sampler (``cuda_sample_fn``).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Callable, Dict, Optional, Tuple

import torch
import torch.distributed as dist

ROW_FIELDS = ("temperature", "top_k", "top_p", "min_p", "repetition_penalty", "presence_penalty",
              "frequency_penalty", "seeds")
_FIELD_DTYPES = {"top_k": torch.int32, "seeds": torch.int64}


@dataclass(frozen=True)
class Layout:
    s: int            # real rows of the batch
    t: int            # workers
    rows: int         # rows per worker after padding
    rank: int

    @property
    def s_padded(self) -> int:
        return self.rows * self.t

    @property
    def row_base(self) -> int:
        return self.rank * self.rows


def layout(s: int, group=None) -> Layout:
    t = dist.get_world_size(group)
    return Layout(s=s, t=t, rows=-(-s // t) if s else 0, rank=dist.get_rank(group))


def exchange_logits(local_shard: torch.Tensor, lay: Layout, group=None,
                    recv: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Step (2).  ``local_shard`` is this worker's ``[s, v/t]`` vocabulary shard (contiguous).
    Returns ``[t, rows, v/t]``: piece ``j`` is vocabulary shard ``j`` of this worker's rows."""
    s, vs = local_shard.shape
    if s != lay.s or not local_shard.is_contiguous():
        raise ValueError("local_shard must be a contiguous [s, v/t] tensor")
    send = local_shard
    if lay.s_padded != s:
        # batch padding (section 6.2): the last real row is repeated; its outputs are dropped
        send = torch.empty((lay.s_padded, vs), dtype=local_shard.dtype, device=local_shard.device)
        send[:s] = local_shard
        send[s:] = local_shard[s - 1]
    if recv is None:
        recv = torch.empty((lay.t, lay.rows, vs), dtype=local_shard.dtype, device=local_shard.device)
    dist.all_to_all_single(recv.view(-1), send.view(-1), group=group)
    return recv


def scatter_metadata(meta: Optional[Dict[str, torch.Tensor]], lay: Layout, device, src: int = 0,
                     group=None) -> Dict[str, Optional[torch.Tensor]]:
    """Step (1).  On ``src``, ``meta`` maps the names of ROW_FIELDS to ``[s]`` tensors (absent or
    None: feature off) and optionally ``history_ids`` / ``history_offsets`` (CSR over the ``s``
    rows).  Every worker gets the slices of its rows (padding rows: copies of the last row's
    parameters and an empty history)."""
    is_src = lay.rank == src
    header = [None]
    if is_src:
        meta = meta or {}
        present = [f for f in ROW_FIELDS if meta.get(f) is not None]
        hist_len = None
        if meta.get("history_ids") is not None:
            off = meta["history_offsets"].to("cpu", torch.int64)
            bounds = [min(lay.s, r * lay.rows) for r in range(lay.t + 1)]
            hist_len = [int(off[bounds[r + 1]] - off[bounds[r]]) for r in range(lay.t)]
        header[0] = (present, hist_len)
    dist.broadcast_object_list(header, src=src, group=group)
    present, hist_len = header[0]
    out: Dict[str, Optional[torch.Tensor]] = {f: None for f in ROW_FIELDS}
    out["history_ids"] = out["history_offsets"] = None

    def scatter(dst, chunks):
        dist.scatter(dst, scatter_list=chunks if is_src else None, src=src, group=group)

    for f in present:
        dtype = _FIELD_DTYPES.get(f, torch.float32)
        mine = torch.empty(lay.rows, dtype=dtype, device=device)
        chunks = None
        if is_src:
            full = meta[f].to(device=device, dtype=dtype)
            if lay.s_padded != lay.s:
                full = torch.cat([full, full[-1:].expand(lay.s_padded - lay.s)])
            chunks = [c.contiguous() for c in full.view(lay.t, lay.rows)]
        scatter(mine, chunks)
        out[f] = mine
    if hist_len is not None:
        # per-row history lengths, then the ids in equal-sized (padded) chunks
        lens = torch.empty(lay.rows, dtype=torch.int32, device=device)
        cap = max(max(hist_len), 1)
        ids = torch.empty(cap, dtype=torch.int32, device=device)
        len_chunks = id_chunks = None
        if is_src:
            off = meta["history_offsets"].to(device=device, dtype=torch.int64)
            row_len = (off[1:] - off[:-1]).to(torch.int32)
            row_len = torch.cat([row_len, torch.zeros(lay.s_padded - lay.s, dtype=torch.int32, device=device)])
            len_chunks = [c.contiguous() for c in row_len.view(lay.t, lay.rows)]
            all_ids = meta["history_ids"].to(device=device, dtype=torch.int32)
            id_chunks = []
            for r in range(lay.t):
                lo = int(off[min(lay.s, r * lay.rows)])
                piece = torch.zeros(cap, dtype=torch.int32, device=device)
                piece[: hist_len[r]] = all_ids[lo: lo + hist_len[r]]
                id_chunks.append(piece)
        scatter(lens, len_chunks)
        scatter(ids, id_chunks)
        offs = torch.zeros(lay.rows + 1, dtype=torch.int32, device=device)
        offs[1:] = torch.cumsum(lens, 0)
        out["history_ids"] = ids          # the first hist_len[rank] entries are this worker's; the rest is padding
        out["history_offsets"] = offs
    return out


def gather_results(tokens: torch.Tensor, logprobs: torch.Tensor, lay: Layout, group=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Step (4): every worker gets the ``s`` tokens and log-probabilities in row order."""
    all_tok = torch.empty(lay.s_padded, dtype=tokens.dtype, device=tokens.device)
    all_lp = torch.empty(lay.s_padded, dtype=logprobs.dtype, device=logprobs.device)
    dist.all_gather_into_tensor(all_tok, tokens.contiguous(), group=group)
    dist.all_gather_into_tensor(all_lp, logprobs.contiguous(), group=group)
    return all_tok[: lay.s], all_lp[: lay.s]


SampleFn = Callable[[torch.Tensor, Dict[str, Optional[torch.Tensor]], int, int], Tuple[torch.Tensor, torch.Tensor]]


def sample_step(sample_fn: SampleFn, local_shard: torch.Tensor, meta_local: Dict[str, Optional[torch.Tensor]],
                lay: Layout, step: int, group=None, recv: Optional[torch.Tensor] = None):
    """Steps (2)-(4) for one decode iteration.  ``sample_fn(pieces, meta_local, row_base, step)``
    returns this worker's ``rows`` tokens (int32) and log-probabilities (float32)."""
    pieces = exchange_logits(local_shard, lay, group=group, recv=recv)
    tok, lp = sample_fn(pieces, meta_local, lay.row_base, step)
    return gather_results(tok, lp, lay, group=group)


def cuda_sample_fn(sampler) -> SampleFn:
    """Step (3) on the CUDA sampler (``binding.Sampler``): the pieces are read where they landed."""
    def fn(pieces, meta_local, row_base, step):
        out = sampler.albireo_sample(pieces, **meta_local, step=step, row_base=row_base)
        return out.tokens, out.logprobs
    return fn


def gather_then_sample_step(sample_fn: SampleFn, local_shard: torch.Tensor, meta_all: Dict[str, Optional[torch.Tensor]],
                            s: int, step: int, group=None, dst: int = 0):
    """The arrangement the paper replaces (section 6.1, "gather"): every shard goes to one worker,
    which samples all rows and broadcasts the tokens.  Kept as the comparison point for benchmarks;
    ``meta_all`` (all ``s`` rows) is only used on ``dst``."""
    t, rank = dist.get_world_size(group), dist.get_rank(group)
    vs = local_shard.shape[1]
    buf = torch.empty((t, s, vs), dtype=local_shard.dtype, device=local_shard.device) if rank == dst else None
    dist.gather(local_shard.contiguous(), gather_list=list(buf.unbind(0)) if rank == dst else None, dst=dst, group=group)
    tok = torch.empty(s, dtype=torch.int32, device=local_shard.device)
    lp = torch.empty(s, dtype=torch.float32, device=local_shard.device)
    if rank == dst:
        t_, l_ = sample_fn(buf, meta_all, 0, step)       # [t, s, v/t] is already "rows in pieces"
        tok.copy_(t_); lp.copy_(l_)
    dist.broadcast(tok, src=dst, group=group)
    dist.broadcast(lp, src=dst, group=group)
    return tok, lp


# ------------------------------------------------------------------ no exchange step: read the peers' shards in place

def peer_shards(s_padded: int, vs: int, dtype: torch.dtype, device, group=None):
    """Allocates this worker's ``[s', v/t]`` vocabulary shard in symmetric memory and maps every peer's.
    Returns ``(mine, peers, handle)``: the LM head writes ``mine``; ``peers[j]`` is worker ``j``'s shard
    as a tensor on this device (peer-mapped; ``peers[rank] is`` the local one); ``handle.barrier()`` is
    the cross-worker barrier.  Padding rows stay zero."""
    import torch.distributed._symmetric_memory as symm
    mine = symm.empty((s_padded, vs), dtype=dtype, device=device)
    mine.zero_()
    grp = dist.group.WORLD if group is None else group
    handle = symm.rendezvous(mine, grp)
    world = dist.get_world_size(group)
    peers = [handle.get_buffer(r, (s_padded, vs), dtype) for r in range(world)]
    return mine, peers, handle


def peer_sample_step(sampler, peers, handle, meta_local: Dict[str, Optional[torch.Tensor]], lay: Layout, step: int,
                     group=None):
    """Steps (2)-(4) with step (2) folded into step (3): the sampler reads piece ``j`` of each of its
    rows straight from worker ``j``'s shard (``segment_ptrs`` of the C ABI), so every logit crosses
    NVLink once, into the sampler's shared memory, and no exchange buffer exists.  Plain bulk copies
    from peer memory, each CTA fetching its own tiles.  The barriers make sure that every shard is complete before it is
    read and not overwritten before everybody has read it."""
    vs = peers[0].shape[1]
    handle.barrier()
    out = sampler.albireo_sample(peers[0], **meta_local, B=lay.rows, V=vs * lay.t, step=step, row_base=lay.row_base,
                                 segment_tensors=peers, segment_row_offset=lay.row_base)
    handle.barrier()
    return gather_results(out.tokens, out.logprobs, lay, group=group)
