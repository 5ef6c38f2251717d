"""The entry point for callers that cannot allocate device memory.

Some users of the sampler get control when allocation is off the table: every byte of the
GPU already belongs to another component's pool, or a cudaMalloc would stall the work
queued around the call, or their process forbids allocation after start-up.  They cannot
provide the workspace that `albireo_sample_init` asks for, so `albireo_sample_fixed_scratch`
keeps its only scratch (history occurrence counts for rows with very many distinct ids) in
a fixed array inside the library.  This test drives that entry point through the C ABI on
rows that really use the scratch and checks it against the CPU oracle (the rules of the parity
tests) and against the ordinary entry point (bit for bit), twice in a row, because the array is
shared and keeps the previous call's contents; the per-row status must show no overflow of the
history counts and no other fault.

The file name makes pytest collect it last, so a run that stops at the first failure has
already run everything else.
"""
import numpy as np
import pytest
import torch

from oracle import albireo_oracle as O
from paper_2606_01927_b200 import workloads as W

from parity import compare, to_host

pytestmark = pytest.mark.gpu


def _workload(seed, B=6, V=30000):
    """Rows whose histories hold far more distinct ids than the on-chip count table."""
    rng = np.random.default_rng(seed)
    x = (rng.standard_normal((B, V)) * 2).astype(np.float32)
    lens = rng.integers(6000, 22000, size=B).astype(np.int64)
    lens[0] = 0
    off = np.zeros(B + 1, dtype=np.int64)
    off[1:] = np.cumsum(lens)
    ids = rng.integers(0, V, size=int(off[-1])).astype(np.int32)
    return W.Workload(f"fixed{seed}", B, V, W.BF16, W.f32_to_bf16_bits(x),
                      temperature=np.full(B, 0.9, np.float32), top_k=np.full(B, 64, np.int32),
                      top_p=np.full(B, 0.95, np.float32),
                      repetition_penalty=np.full(B, 1.2, np.float32), presence_penalty=np.full(B, 0.4, np.float32),
                      frequency_penalty=np.full(B, 0.1, np.float32),
                      history_ids=ids, history_offsets=off.astype(np.int32),
                      seeds=np.arange(B, dtype=np.uint64) + seed, step=seed)


def test_fixed_scratch_entry_matches_the_workspace_entry_twice_in_a_row():
    from paper_2606_01927_b200 import binding
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    for call, seed in enumerate((41, 42)):            # two calls in a row, different contents
        w = _workload(seed)
        t = binding.workload_tensors(w, dev)
        logits = t.pop("logits")
        got = binding.albireo_sample_fixed_scratch(logits, **t, want_status=True, want_counts=True)
        sampler = binding.Sampler(max_rows=w.B, max_vocab=w.V, max_history_total=int(w.history_ids.size), device=dev)
        ref = sampler.albireo_sample(logits, **t, want_status=True, want_counts=True)
        torch.cuda.synchronize()
        # the per-row status: nothing but the path bit may be set (no history overflow, no timeout, ...)
        bad_bits = ~np.int32(binding.ROW_GENERAL_PATH)
        assert not (got.row_status.cpu().numpy() & bad_bits).any(), (call, got.row_status.cpu().numpy())
        assert not (ref.row_status.cpu().numpy() & bad_bits).any()
        # against the CPU oracle, by the rules of the parity tests
        rep = compare(w, to_host(got), O.sample(w, threads=4))
        print(rep.summary())
        assert rep.ok() and not rep.excused, (call, rep.failures[:3], rep.excused[:3])
        # and against the entry point with a workspace: the same kernel, so the same bits
        assert (got.tokens.cpu().numpy() == ref.tokens.cpu().numpy()).all(), call
        assert (got.logprobs.cpu().numpy().view(np.uint32) == ref.logprobs.cpu().numpy().view(np.uint32)).all(), call
        assert (got.num_kept.cpu().numpy() == ref.num_kept.cpu().numpy()).all(), call
        sampler.close()


def test_fixed_scratch_entry_rejects_sizes_beyond_its_array():
    from paper_2606_01927_b200 import binding
    dev = torch.device("cuda", 0)
    x = torch.zeros((2, 64), dtype=torch.float32, device=dev)
    ids = torch.zeros(1, dtype=torch.int32, device=dev)
    off = torch.zeros(3, dtype=torch.int32, device=dev)
    with pytest.raises(binding.AlbireoError) as e:
        binding.albireo_sample_fixed_scratch(x, history_ids=ids, history_offsets=off,
                                             history_total=binding.FIXED_MAX_HISTORY + 1)
    assert e.value.code == binding.EUNSUPPORTED and "ALBIREO_FIXED_MAX_HISTORY" in str(e.value)
