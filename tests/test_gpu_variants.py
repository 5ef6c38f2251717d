"""Parity of the sampler's variants with the CPU oracle: binary16 logits (the paper's models are
FP16, §8.1), pre-generated Exp(1) variates (§6.2) and the early-feedback targets (§5.2)."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import albireo_oracle as O
from paper_2606_01927_b200 import workloads as W

from parity import EXCUSED_FRACTION, compare, compare_top_lists, to_host

pytestmark = pytest.mark.gpu

DBG_CAP = 128
_CORES = len(os.sched_getaffinity(0))


@pytest.fixture(scope="module")
def binding():
    from paper_2606_01927_b200 import binding as Bd
    return Bd


@pytest.fixture(scope="module")
def sampler(binding):
    s = binding.Sampler(max_rows=512, max_vocab=152064 + 64, max_history_total=1 << 21)
    yield s
    s.close()


def run(binding, sampler, w, *, flags=0, **kw):
    t = binding.workload_tensors(w, sampler.device)
    t.pop("backfill_index", None)
    out = sampler.albireo_sample(t.pop("logits"), **t, row_base=w.row_base, num_top=w.num_top,
                                 want_counts=True, dbg_cap=DBG_CAP, want_status=True, flags=flags, **kw)
    torch.cuda.synchronize()
    return to_host(out)


def check(binding, sampler, w, *, flags=0, allow_excused=0):
    ref = O.sample(w, threads=_CORES, topk_cap=DBG_CAP)
    g = run(binding, sampler, w, flags=flags)
    rep = compare(w, g, ref, dbg_cap=DBG_CAP)
    print(rep.summary())
    assert rep.ok(), rep.failures[:5]
    assert len(rep.excused) <= max(allow_excused, math.floor(EXCUSED_FRACTION * w.B)), rep.excused[:5]
    bad = compare_top_lists(w, g, ref)
    assert not bad, bad[:3]
    return g, ref


# ------------------------------------------------------------------ binary16 logits

F16_SMALL = [(201, 48, 1000, None), (202, 40, 4099, None), (203, 32, 9001, 0.5), (204, 12, 70001, None), (205, 64, 17, None)]


@pytest.mark.parametrize("seed,B,V,q", F16_SMALL)
@pytest.mark.parametrize("flags", [0, 1], ids=["auto", "general"])
def test_f16_small_mixed_parameters(binding, sampler, seed, B, V, q, flags):
    w = W.as_f16(W.random_small(seed, B=B, V=V, dtype=W.F32, quantise=q))
    w.num_top = 5
    check(binding, sampler, w, flags=flags)


@pytest.mark.parametrize("flags", [0, 1], ids=["auto", "general"])
def test_f16_degenerate_rows(binding, sampler, flags):
    V = 20000
    rng = np.random.default_rng(23)
    rows = [np.full(V, 1.5, np.float32)]                                       # all equal
    r = np.full(V, -np.inf, np.float32); r[[5, 77, 19999]] = [1.0, 1.0, 0.5]  # fewer finite than k
    rows.append(r)
    rows.append((rng.standard_normal(V) * 1e-6).astype(np.float32))            # binary16 subnormals and signed zeros
    r = rng.standard_normal(V).astype(np.float32); r[1234] += 30               # one-hot like
    rows.append(r)
    rows.append(np.round(rng.standard_normal(V) * 2).astype(np.float32))       # thousands of ties at the k-th value
    rows.append((rng.standard_normal(V) * 2000).astype(np.float32))            # near the top of the binary16 range
    x = np.stack(rows)
    n = x.shape[0]
    variants = [
        dict(temperature=np.full(n, 0.8, np.float32), top_k=np.full(n, 50, np.int32)),
        dict(temperature=np.full(n, 1.0, np.float32), top_k=np.full(n, 40, np.int32), top_p=np.full(n, 0.9, np.float32)),
        dict(temperature=np.full(n, 1.0, np.float32), min_p=np.full(n, 0.05, np.float32), top_p=np.full(n, 0.95, np.float32)),
        dict(temperature=np.full(n, 0.7, np.float32), top_p=np.full(n, 0.5, np.float32)),
        dict(temperature=np.zeros(n, np.float32)),
        dict(temperature=np.full(n, 1e-4, np.float32), top_k=np.full(n, 20, np.int32)),   # a very small temperature
    ]
    for i, kw in enumerate(variants):
        w = W.as_f16(W.Workload(f"f16deg{i}", n, V, W.F32, x, seeds=np.arange(n, dtype=np.uint64) + 3, step=9,
                                num_top=8, **kw))
        check(binding, sampler, w, flags=flags)


def test_f16_full_vocabulary_rows(binding, sampler):
    w = W.as_f16(W.config2(B=48))
    g, _ = check(binding, sampler, w)
    assert (g["row_status"] & 1).sum() == 0            # every row on the single-pass path


def test_f16_history_rows(binding, sampler):
    check(binding, sampler, W.as_f16(W.config3(B=24)))


# ------------------------------------------------------------------ pre-generated Exp(1) variates

@pytest.mark.parametrize("dtype", [W.F32, W.BF16])
@pytest.mark.parametrize("flags", [0, 1], ids=["auto", "general"])
def test_exp1_table_small(binding, sampler, dtype, flags):
    w = W.with_exp1(W.random_small(301, B=40, V=4099, dtype=dtype), seed=5)
    w.num_top = 4
    check(binding, sampler, w, flags=flags)


def test_exp1_table_full_vocabulary(binding, sampler):
    base = W.config4(B=32)
    g, ref = check(binding, sampler, W.with_exp1(base, seed=6))
    # the table, not the seeds, decides: the counter-based tokens of the same rows differ somewhere
    plain = O.sample(base, threads=_CORES)
    assert (plain.tokens != ref.tokens).any()


def test_exp1_forced_winner_and_row_stride(binding, sampler):
    w = W.with_exp1(W.random_small(302, B=16, V=2000, dtype=W.BF16, with_history=False), seed=8)
    w.temperature[:] = 1.0
    w.top_k[:] = 0
    w.top_p[:] = 1.0
    w.min_p[:] = 0.0
    forced = np.arange(16) * 100 + 7
    w.exp1[np.arange(16), forced] = np.float32(1e-35)       # -ln E = 80: beats any score gap here
    t = binding.workload_tensors(w, sampler.device)
    wide = torch.full((16, 2000 + 40), float("nan"), device=sampler.device)
    wide[:, :2000] = t.pop("exp1")
    out = sampler.albireo_sample(t.pop("logits"), **t, exp1=wide[:, :2000])
    torch.cuda.synchronize()
    assert out.tokens.cpu().tolist() == forced.tolist()


# ------------------------------------------------------------------ early feedback

@pytest.mark.parametrize("flags", [0, 1], ids=["auto", "general"])
def test_backfill_and_feedback_ring(binding, sampler, flags):
    w = W.with_backfill(W.random_small(401, B=50, V=3000, dtype=W.BF16))
    w.row_base = 1000
    ref = O.sample(w, threads=_CORES)
    dev = sampler.device
    ids_next = torch.full((w.backfill_len,), -7, dtype=torch.int32, device=dev)
    index = torch.from_numpy(w.backfill_index).to(dev)
    ring_dev = torch.full((64,), -1, dtype=torch.int64, device=dev)
    g = run(binding, sampler, w, flags=flags, backfill_ids=ids_next, backfill_index=index,
            feedback_ring=ring_dev, feedback_head=60)
    tok = g["tokens"]
    assert (tok == ref.tokens).all()
    got = ids_next.cpu().numpy()
    want = np.full(w.backfill_len, -7, dtype=np.int32)
    for b in range(w.B):
        if w.backfill_index[b] >= 0:
            want[w.backfill_index[b]] = tok[b]
    assert (got == want).all()
    ring = ring_dev.cpu().numpy()
    for b in range(w.B):
        rec = int(ring[(60 + b) % 64])
        assert rec >> 32 == 1000 + b and (rec & 0xFFFFFFFF) == tok[b]
    for slot in set(range(64)) - {(60 + b) % 64 for b in range(w.B)}:
        assert ring[slot] == -1


def test_feedback_ring_in_pinned_host_memory_and_identity_map(binding, sampler):
    w = W.random_small(402, B=20, V=3000, dtype=W.F32)
    ref = O.sample(w, threads=_CORES)
    ring = torch.full((32,), -1, dtype=torch.int64).pin_memory()
    ids_next = torch.full((w.B,), -7, dtype=torch.int32, device=sampler.device)
    g = run(binding, sampler, w, backfill_ids=ids_next, feedback_ring=ring)      # no index: row b -> slot b
    assert (g["tokens"] == ref.tokens).all()
    assert (ids_next.cpu().numpy() == ref.tokens).all()
    r = ring.numpy()
    assert [int(v) & 0xFFFFFFFF for v in r[: w.B]] == ref.tokens.tolist()
    assert [int(v) >> 32 for v in r[: w.B]] == list(range(w.B))
    assert (r[w.B:] == -1).all()


def test_backfill_index_out_of_range_is_flagged_and_skipped(binding, sampler):
    w = W.random_small(403, B=8, V=500, dtype=W.F32, with_history=False)
    ids_next = torch.full((4,), -7, dtype=torch.int32, device=sampler.device)
    index = torch.tensor([0, 1, 2, 3, 4, 100, -1, -5], dtype=torch.int32, device=sampler.device)
    g = run(binding, sampler, w, backfill_ids=ids_next, backfill_index=index)
    assert (ids_next.cpu().numpy() == g["tokens"][:4]).all()
    assert [(int(s) >> 1) & 1 for s in g["row_status"]] == [0, 0, 0, 0, 1, 1, 0, 0]


def test_variant_argument_errors(binding, sampler):
    w = W.random_small(404, B=4, V=500, dtype=W.F32, with_history=False)
    t = binding.workload_tensors(w, sampler.device)
    lg = t.pop("logits")
    n0 = sampler.launch_count()
    with pytest.raises(ValueError):
        sampler.albireo_sample(lg, **t, exp1=torch.ones((4, 500), dtype=torch.float64, device=sampler.device))
    with pytest.raises(binding.AlbireoError):
        sampler.albireo_sample(lg, **t, exp1=torch.ones((4, 400), device=sampler.device))   # row stride < V
    with pytest.raises(binding.AlbireoError):
        sampler.albireo_sample(lg, **t, feedback_ring=torch.zeros(8, dtype=torch.int64, device=sampler.device),
                               feedback_head=-1)
    assert sampler.launch_count() == n0


# ------------------------------------------------------------------ rows in pieces (sequence-parallel layout)

def pieces(logits_2d: torch.Tensor, t: int, pad_rows: int = 0, pad_cols: int = 0) -> torch.Tensor:
    """[B, V] -> the [t, B, V/t] layout an all-to-all of vocabulary shards leaves (optionally inside a
    larger allocation so that the strides are not the dense ones)."""
    B, V = logits_2d.shape
    Vs = V // t
    big = torch.zeros((t, B + pad_rows, Vs + pad_cols), dtype=logits_2d.dtype, device=logits_2d.device)
    for j in range(t):
        big[j, :B, :Vs] = logits_2d[:, j * Vs:(j + 1) * Vs]
    return big[:, :B, :Vs]


@pytest.mark.parametrize("t,dtype,V,pad", [(2, W.BF16, 8192, (0, 0)), (4, W.BF16, 152064, (0, 0)), (4, W.F32, 40000, (3, 8)),
                                           (8, W.BF16, 70016, (1, 16)), (4, W.F16, 152064, (0, 0))])
@pytest.mark.parametrize("flags", [0, 1], ids=["auto", "general"])
def test_rows_in_pieces_match_contiguous_rows(binding, sampler, t, dtype, V, pad, flags):
    base = W.random_small(500 + t, B=24, V=V, dtype=W.F32 if dtype == W.F16 else dtype)
    w = W.as_f16(base) if dtype == W.F16 else base
    w.num_top = 3
    ref = O.sample(w, threads=_CORES, topk_cap=DBG_CAP)
    tt = binding.workload_tensors(w, sampler.device)
    lg = pieces(tt.pop("logits"), t, *pad)
    out = sampler.albireo_sample(lg, **tt, num_top=w.num_top, want_counts=True, dbg_cap=DBG_CAP, want_status=True, flags=flags)
    torch.cuda.synchronize()
    g = to_host(out)
    rep = compare(w, g, ref, dbg_cap=DBG_CAP)
    print(rep.summary())
    assert rep.ok(), rep.failures[:5]
    assert len(rep.excused) <= 1
    assert not compare_top_lists(w, g, ref)


def test_rows_in_pieces_argument_errors(binding, sampler):
    w = W.random_small(510, B=4, V=4096, dtype=W.BF16, with_history=False)
    tt = binding.workload_tensors(w, sampler.device)
    lg2 = tt.pop("logits")
    n0 = sampler.launch_count()
    with pytest.raises(binding.AlbireoError):                   # pieces of 4096 / 3 elements: V not divisible
        sampler.albireo_sample(pieces(lg2[:, :4095], 3), **tt, V=4096)
    with pytest.raises(binding.AlbireoError):                   # pieces whose byte length is not a multiple of 16
        sampler.albireo_sample(pieces(lg2[:, :4088], 2, 0, 4), **tt)
    assert sampler.launch_count() == n0


def test_sequence_parallel_step_on_one_rank(binding, sampler):
    """The whole sequence-parallel step (all-to-all, sample, gather) through NCCL with a group of one:
    the collectives are trivial, the code path and the sampler's reading of the pieces are the real ones."""
    import socket
    import torch.distributed as dist
    from paper_2606_01927_b200 import sequence_parallel as SP
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=sampler.device)
    try:
        w = W.config4(B=40)
        ref = O.sample(w, threads=_CORES)
        tt = binding.workload_tensors(w, sampler.device)
        shard = tt.pop("logits")
        step = tt.pop("step")
        lay = SP.layout(w.B)
        meta = SP.scatter_metadata(tt, lay, sampler.device)
        tok, lp = SP.sample_step(SP.cuda_sample_fn(sampler), shard, meta, lay, step=step)
        torch.cuda.synchronize()
        rep = compare(w, {"tokens": tok.cpu().numpy(), "logprobs": lp.cpu().numpy()}, ref)
        print(rep.summary())
        assert rep.ok(), rep.failures[:5]
        assert not rep.excused, rep.excused
    finally:
        dist.destroy_process_group()


# ------------------------------------------------------------------ prompt / output split of the histories

@pytest.mark.parametrize("dtype", [W.F32, W.BF16])
@pytest.mark.parametrize("flags", [0, 1], ids=["auto", "general"])
def test_split_history_small(binding, sampler, dtype, flags):
    w = W.with_split_history(W.random_small(601, B=48, V=4099, dtype=dtype))
    w.num_top = 4
    check(binding, sampler, w, flags=flags)


def test_split_history_full_vocabulary_and_limits(binding, sampler):
    base = W.config3(B=24)
    w = W.with_split_history(base)
    g, ref = check(binding, sampler, w)
    # all-output split == no split, bit for bit
    w0 = W.config3(B=24)
    w0.output_start = np.zeros(w0.B, dtype=np.int32)
    a = run(binding, sampler, w0)
    b = run(binding, sampler, W.config3(B=24))
    assert (a["tokens"] == b["tokens"]).all() and (a["logprobs"] == b["logprobs"]).all()
    # out-of-range values are clamped to [0, length]
    w1 = W.config3(B=24)
    w1.output_start = np.full(w1.B, -5, dtype=np.int32)
    c = run(binding, sampler, w1)
    assert (c["tokens"] == b["tokens"]).all()
    w2 = W.config3(B=24)
    w2.output_start = np.full(w2.B, 10**6, dtype=np.int32)
    w3 = W.config3(B=24)
    w3.output_start = np.diff(w3.history_offsets).astype(np.int32)
    d, e = run(binding, sampler, w2), run(binding, sampler, w3)
    assert (d["tokens"] == e["tokens"]).all() and (d["logprobs"] == e["logprobs"]).all()


# ------------------------------------------------------------------ top-k that keeps ties

@pytest.mark.parametrize("dtype", [W.F32, W.BF16, W.F16])
@pytest.mark.parametrize("general", [0, 1], ids=["auto", "general"])
def test_topk_keep_ties(binding, sampler, dtype, general):
    base = W.random_small(701, B=48, V=9001, dtype=W.F32 if dtype == W.F16 else dtype, quantise=0.5)   # ties at every cut
    w = W.as_f16(base) if dtype == W.F16 else base
    w.topk_keep_ties = True
    w.num_top = 6
    flags = binding.FLAG_TOPK_KEEP_TIES | (binding.FLAG_FORCE_GENERAL if general else 0)
    g, ref = check(binding, sampler, w, flags=flags)
    strict = O.sample(W.random_small(701, B=48, V=9001, dtype=W.F32 if dtype == W.F16 else dtype, quantise=0.5))
    assert (ref.rows["n_topk"] > strict.rows["n_topk"]).sum() >= 5          # the mode matters on these rows
    assert (g["num_topk"] == ref.rows["n_topk"]).all()


def test_topk_keep_ties_thousands_of_ties(binding, sampler):
    rng = np.random.default_rng(71)
    x = np.round(rng.standard_normal((6, 30000)) * 2).astype(np.float32)    # ~6000 elements per distinct value
    w = W.Workload("ties", 6, 30000, W.BF16, W.f32_to_bf16_bits(x), temperature=np.full(6, 0.9, np.float32),
                   top_k=np.array([1, 5, 50, 300, 2000, 29999], np.int32), top_p=np.full(6, 0.95, np.float32),
                   seeds=np.arange(6, dtype=np.uint64), topk_keep_ties=True)
    g, ref = check(binding, sampler, w, flags=binding.FLAG_TOPK_KEEP_TIES)
    assert (g["num_topk"] == ref.rows["n_topk"]).all() and ref.rows["n_topk"][4] > 2500


# ------------------------------------------------------------------ log-probabilities relative to the full vocabulary

@pytest.mark.parametrize("dtype", [W.F32, W.BF16])
@pytest.mark.parametrize("general", [0, 1], ids=["auto", "general"])
def test_full_vocabulary_logprobs(binding, sampler, dtype, general):
    w = W.random_small(801, B=48, V=9001, dtype=dtype)
    w.logprob_full_vocab = True
    w.num_top = 5
    flags = binding.FLAG_LOGPROB_FULL_VOCAB | (binding.FLAG_FORCE_GENERAL if general else 0)
    g, ref = check(binding, sampler, w, flags=flags)
    plain = O.sample(W.random_small(801, B=48, V=9001, dtype=dtype))
    assert (plain.tokens == ref.tokens).all() and (ref.logprobs < plain.logprobs - 1e-9).sum() >= 20


def test_full_vocabulary_top_list_reaches_past_the_cuts(binding, sampler):
    """top_k below num_top, greedy rows, min-p only rows: the list is still the head of the whole row."""
    w = W.random_small(802, B=40, V=6000, dtype=W.BF16)
    w.top_k[:] = np.where(np.arange(40) % 3 == 0, 2, w.top_k)        # cuts far tighter than the list
    w.logprob_full_vocab = True
    w.num_top = 12
    for general in (0, 1):
        flags = binding.FLAG_LOGPROB_FULL_VOCAB | (binding.FLAG_FORCE_GENERAL if general else 0)
        g, ref = check(binding, sampler, w, flags=flags)
        assert (ref.top_ids >= 0).all() and (g["top_ids"] == ref.top_ids).all()
    wk = W.random_small(802, B=40, V=6000, dtype=W.BF16)
    wk.top_k[:] = np.where(np.arange(40) % 3 == 0, 2, wk.top_k)
    wk.logprob_full_vocab = True; wk.topk_keep_ties = True; wk.num_top = 12
    check(binding, sampler, wk, flags=binding.FLAG_LOGPROB_FULL_VOCAB | binding.FLAG_TOPK_KEEP_TIES)


def test_full_vocabulary_logprobs_full_size_rows(binding, sampler):
    w = W.config4(B=48)
    w.logprob_full_vocab = True
    check(binding, sampler, w, flags=binding.FLAG_LOGPROB_FULL_VOCAB)


# ------------------------------------------------------------------ programmatic dependent launch

def test_programmatic_launch_gives_the_same_results(binding, sampler):
    """Back-to-back calls launched with programmatic stream serialisation, the second reading what the
    first wrote nowhere: each equals the plain launch bit for bit, also inside a captured graph."""
    w = W.config3(B=32)
    t = binding.workload_tensors(w, sampler.device)
    lg = t.pop("logits")
    plain = sampler.albireo_sample(lg, **t, num_top=4)
    torch.cuda.synchronize()
    outs = [sampler.albireo_sample(lg, **t, num_top=4, flags=binding.FLAG_PROGRAMMATIC_LAUNCH) for _ in range(4)]
    torch.cuda.synchronize()
    for o in outs:
        assert torch.equal(o.tokens, plain.tokens) and torch.equal(o.logprobs, plain.logprobs)
        assert torch.equal(o.top_ids, plain.top_ids)
    st = torch.cuda.Stream(device=sampler.device)
    tok = torch.empty(32, dtype=torch.int32, device=sampler.device)
    lp = torch.empty(32, dtype=torch.float32, device=sampler.device)
    with torch.cuda.stream(st):
        sampler.albireo_sample(lg, **t, out_tokens=tok, out_logprobs=lp, stream=st, flags=binding.FLAG_PROGRAMMATIC_LAUNCH)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=st):
        for _ in range(3):
            sampler.albireo_sample(lg, **t, out_tokens=tok, out_logprobs=lp, stream=st, flags=binding.FLAG_PROGRAMMATIC_LAUNCH)
    tok.fill_(-9)
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(tok, plain.tokens) and torch.equal(lp, plain.logprobs)


# ------------------------------------------------------------------ pieces in buffers of their own (peer memory stand-in)

@pytest.mark.parametrize("t,dtype,V", [(2, W.BF16, 8192), (4, W.BF16, 152064), (4, W.F32, 40000), (8, W.F16, 70016)])
@pytest.mark.parametrize("flags", [0, 1], ids=["auto", "general"])
def test_pieces_in_separate_buffers(binding, sampler, t, dtype, V, flags):
    """Every piece in an allocation of its own, as if it were another worker's vocabulary shard [s, V/t]
    with this call's rows starting at row 5: the sampler reads them in place through a pointer table."""
    import ctypes as C
    base = W.random_small(900 + t, B=20, V=V, dtype=W.F32 if dtype == W.F16 else dtype)
    w = W.as_f16(base) if dtype == W.F16 else base
    w.num_top = 3
    ref = O.sample(w, threads=_CORES, topk_cap=DBG_CAP)
    tt = binding.workload_tensors(w, sampler.device)
    lg = tt.pop("logits")
    Vs, off = V // t, 5
    shards = []
    for j in range(t):
        sh = torch.zeros((off + w.B + 2, Vs), dtype=lg.dtype, device=lg.device)      # other rows before and after
        sh[off:off + w.B] = lg[:, j * Vs:(j + 1) * Vs]
        shards.append(sh)
    out = sampler.albireo_sample(shards[0], **tt, B=w.B, V=V, num_top=w.num_top, want_counts=True, dbg_cap=DBG_CAP,
                                 want_status=True, flags=flags, segment_tensors=shards, segment_row_offset=off)
    torch.cuda.synchronize()
    g = to_host(out)
    rep = compare(w, g, ref, dbg_cap=DBG_CAP)
    print(rep.summary())
    assert rep.ok(), rep.failures[:5]
    assert len(rep.excused) <= 1 and not compare_top_lists(w, g, ref)


def test_peer_shards_step_on_one_rank(binding, sampler):
    """The exchange-free sequence-parallel step through symmetric memory with a group of one: allocation,
    rendezvous, barrier, the sampler reading the (here: its own) shard through the pointer table, gather."""
    import socket
    import torch.distributed as dist
    from paper_2606_01927_b200 import sequence_parallel as SP
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=sampler.device)
    try:
        w = W.config2(B=24)
        ref = O.sample(w, threads=_CORES)
        tt = binding.workload_tensors(w, sampler.device)
        lg, step = tt.pop("logits"), tt.pop("step")
        lay = SP.layout(w.B)
        mine, peers, handle = SP.peer_shards(lay.s_padded, w.V, lg.dtype, sampler.device)
        mine[: w.B].copy_(lg)                                 # what the LM head would have written
        meta = SP.scatter_metadata(tt, lay, sampler.device)
        tok, lp = SP.peer_sample_step(sampler, peers, handle, meta, lay, step=step)
        torch.cuda.synchronize()
        assert (tok.cpu().numpy() == ref.tokens).all()
        assert np.abs(lp.cpu().numpy() - ref.logprobs).max() < 2e-5
    finally:
        dist.destroy_process_group()


# ------------------------------------------------------------------ race ties, out-of-contract parameters, history overflow

@pytest.mark.parametrize("dtype", [W.F32, W.BF16])
@pytest.mark.parametrize("flags", [0, 1], ids=["auto", "general"])
def test_race_tie_goes_to_the_lowest_id(binding, sampler, dtype, flags):
    """Equal scores with equal pre-generated variates have equal race scores: the lowest id wins, whether
    the tied ids sit in one thread's vector, in different warps' stripes or in different tiles."""
    V = 40000
    tied = [[7, 19, 33], [0, V - 1], [38000, 5, 21000, 6], [16, 17], [8191, 8192, 24575], [12345, 30000]]
    B = len(tied)
    rng = np.random.default_rng(81)
    x = (rng.standard_normal((B, V)) * 0.5 - 6.0).astype(np.float32)
    for b, ids in enumerate(tied):
        x[b, ids] = 2.0
    cuts = [dict(), dict(top_k=np.full(B, 50, np.int32)), dict(top_p=np.full(B, 0.9, np.float32)),
            dict(top_k=np.full(B, 2, np.int32))]
    for kw in cuts:
        w = W.Workload("ties", B, V, dtype, x if dtype == W.F32 else W.f32_to_bf16_bits(x),
                       temperature=np.ones(B, np.float32), seeds=np.arange(B, dtype=np.uint64), **kw)
        w.exp1 = np.full((B, V), 0.75, dtype=np.float32)
        ref = O.sample(w, threads=_CORES)
        assert ref.tokens.tolist() == [min(t) for t in tied] and (ref.rows["race_gap"] == 0.0).all()
        g = run(binding, sampler, w, flags=flags)
        assert g["tokens"].tolist() == [min(t) for t in tied], kw
        rep = compare(w, g, ref)
        assert rep.ok() and not rep.excused, (rep.failures[:3], rep.excused[:3])


@pytest.mark.parametrize("dtype", [W.F32, W.BF16])
@pytest.mark.parametrize("flags", [0, 1], ids=["auto", "general"])
def test_out_of_contract_parameters_are_flagged_and_follow_the_definition(binding, sampler, dtype, flags):
    """T < 0 and T = NaN read as greedy, r <= 0 is applied as written; such rows carry ALBIREO_ROW_BAD_PARAM,
    the other rows of the batch do not, and every row still equals the oracle's."""
    w = W.random_small(401, B=12, V=9001, dtype=dtype)
    bad_T = {1: -1.0, 4: np.nan, 7: -np.inf}
    bad_r = {2: -1.5, 4: -0.25, 9: -2.0}
    for b, v in bad_T.items():
        w.temperature[b] = v
    for b, v in bad_r.items():
        w.repetition_penalty[b] = v
    ref = O.sample(w, threads=_CORES, topk_cap=DBG_CAP)
    assert all(ref.rows["greedy"][b] == 1 for b in bad_T)
    g = run(binding, sampler, w, flags=flags)
    rep = compare(w, g, ref, dbg_cap=DBG_CAP)
    print(rep.summary())
    assert rep.ok() and not rep.excused, (rep.failures[:3], rep.excused[:3])
    flagged = (g["row_status"] & binding.ROW_BAD_PARAM) != 0
    assert flagged.tolist() == [b in bad_T or b in bad_r for b in range(w.B)]
    for b in bad_T:
        assert g["logprobs"][b] == 0.0 and g["tokens"][b] == ref.tokens[b]


@pytest.mark.parametrize("flags", [0, 1], ids=["auto", "general"])
def test_history_overflow_is_flagged_and_skips_the_penalties(binding, flags):
    """A workspace too small for a row's distinct history ids: the row is sampled without penalties and
    carries ALBIREO_ROW_HISTORY_OVERFLOW; rows whose ids fit on chip or in the workspace are untouched."""
    V, B = 30000, 5
    rng = np.random.default_rng(83)
    x = (rng.standard_normal((B, V)) * 2).astype(np.float32)
    lens = np.array([50, 9000, 0, 6000, 300], dtype=np.int64)
    off = np.zeros(B + 1, dtype=np.int64); off[1:] = np.cumsum(lens)
    ids = rng.integers(0, V, size=int(off[-1])).astype(np.int32)
    kw = dict(temperature=np.full(B, 0.9, np.float32), top_k=np.full(B, 64, np.int32),
              repetition_penalty=np.full(B, 1.3, np.float32), presence_penalty=np.full(B, 0.5, np.float32),
              frequency_penalty=np.full(B, 0.2, np.float32), seeds=np.arange(B, dtype=np.uint64) + 5)
    w = W.Workload("overflow", B, V, W.BF16, W.f32_to_bf16_bits(x), history_ids=ids,
                   history_offsets=off.astype(np.int32), **kw)
    over = [1, 3]                                  # > 2048 distinct ids each, and the workspace holds 1000 counters
    for b in over:
        assert np.unique(ids[off[b]:off[b + 1]]).size > 2048
    # what the definition gives when those rows have no history
    lens2 = lens.copy(); lens2[over] = 0
    off2 = np.zeros(B + 1, dtype=np.int64); off2[1:] = np.cumsum(lens2)
    ids2 = np.concatenate([ids[off[b]:off[b + 1]] for b in range(B) if b not in over])
    w2 = W.Workload("overflow-ref", B, V, W.BF16, w.logits, history_ids=ids2, history_offsets=off2.astype(np.int32), **kw)
    ref = O.sample(w2, threads=_CORES, topk_cap=DBG_CAP)
    full = O.sample(w, threads=_CORES)
    assert any(full.tokens[b] != ref.tokens[b] or full.logprobs[b] != ref.logprobs[b] for b in over)   # penalties matter here
    s = binding.Sampler(max_rows=B, max_vocab=V, max_history_total=1000)
    try:
        g = run(binding, s, w, flags=flags)
    finally:
        s.close()
    rep = compare(w2, g, ref, dbg_cap=DBG_CAP)
    print(rep.summary())
    assert rep.ok() and not rep.excused, (rep.failures[:3], rep.excused[:3])
    flagged = (g["row_status"] & binding.ROW_HISTORY_OVERFLOW) != 0
    assert flagged.tolist() == [b in over for b in range(B)]


# ------------------------------------------------------------------ the stream-only measurement aid

@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16, torch.float16])
def test_stream_only_reads_every_streamed_element(binding, sampler, dtype):
    """The measurement kernel really moves the rows: a +inf anywhere in the streamed part of a row shows
    in that row's word, ordinary rows give 0, and no wait expires."""
    B, V = 6, 70001                                    # several tiles and a ragged end
    g = torch.Generator(device="cpu").manual_seed(5)
    x = (torch.randn((B, V), generator=g) * 3).to(dtype)
    per_vec = 16 // x.element_size()
    where = {1: 5 * per_vec + 1, 3: V - 40 * per_vec, 4: 3 * 512 * 4 * per_vec + 7}     # first tile, last tile, a middle tile
    for b, i in where.items():
        x[b, i] = float("inf")
    xd = x.to(sampler.device)
    sink = torch.full((B,), 123, dtype=torch.int32, device=sampler.device)
    n0 = sampler.launch_count()
    sampler.albireo_stream_only(xd, sink)
    torch.cuda.synchronize()
    got = sink.cpu().numpy().astype(np.int64) & 0xFFFFFFFF
    assert not (got >> 31).any(), got                  # no expired wait
    assert [int(v > 0) for v in got] == [int(b in where) for b in range(B)], got
    assert sampler.launch_count() == n0                # (not a sampling launch)
    with pytest.raises(ValueError):
        sampler.albireo_stream_only(xd[:, :100], sink)           # not dense
    with pytest.raises(binding.AlbireoError):
        sampler.albireo_stream_only(torch.zeros((2000, 8), dtype=dtype, device=sampler.device),
                                    torch.zeros(2000, dtype=torch.int32, device=sampler.device))   # more rows than the handle allows


def test_bounded_wait_expires_and_the_context_stays_usable(binding, sampler):
    """A tile whose copy is announced but never issued: the ring's bounded wait on it runs out, every row
    reports it (bit 31), the copies in flight are waited for, the kernel returns, and the next launches --
    the stream alone and a real sampling call -- behave as if nothing had happened."""
    w = W.config1(B=8, V=32000)
    t = binding.workload_tensors(w, sampler.device)
    x = t.pop("logits")
    sink = torch.zeros(w.B, dtype=torch.int32, device=sampler.device)
    for drop in (0, 2):                                    # in the first fill of the ring, and in a refill
        sampler.albireo_stream_only(x, sink, drop_tile=drop)
        torch.cuda.synchronize()
        got = sink.cpu().numpy().astype(np.int64) & 0xFFFFFFFF
        assert ((got >> 31) == 1).all(), (drop, got)
    sampler.albireo_stream_only(x, sink)
    torch.cuda.synchronize()
    assert (sink.cpu().numpy() == 0).all()
    check(binding, sampler, w)
