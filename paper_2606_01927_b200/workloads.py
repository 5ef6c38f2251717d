"""Seeded synthetic workloads for the batched token sampler.

This module only *generates inputs* (logits, per-row sampling parameters, token
histories, seeds).  It contains none of the sampler's arithmetic, so both the CPU
oracle's tests and the CUDA path's tests/bench may import it.

The five numbered configurations stand in for the logits an LLM decode step would
hand to the sampling task (T4, §2.1): a Gaussian bulk, a few dominant tokens, a
Zipfian prior over token ids (Qwen-2.5 sized vocabulary, Appendix A), bf16
quantisation, and the per-request penalty metadata of §3.1 / §8.1 (Workload).  The
paper's real inputs (dataset prompts through model weights) are not reproduced; only
shape, dtype and rough distribution matter to the sampling path.

Everything is numpy on the host.  bf16 logits are stored as ``uint16`` bit patterns
(round-to-nearest-even of the fp32 draw).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np

F32 = 0
BF16 = 1
F16 = 2     # IEEE binary16, the precision of the paper's models (§8.1)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest, ties to even); returns uint16 bit patterns."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (b >> np.uint32(16)) & np.uint32(1)
    r = (b + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass
class Workload:
    """One batch of sampler inputs, all host numpy arrays.

    ``None`` for a per-row array means "feature off for every row" (the C-ABI takes
    NULL there).  ``logits`` is float32 ``[B, V]`` for dtype F32 and uint16 bf16 bit
    patterns ``[B, V]`` for dtype BF16 (binary16 bit patterns for dtype F16).

    ``exp1`` switches the draw to pre-generated random numbers (the scheme of §6.2):
    a float32 ``[B, V]`` table of Exp(1) variates read instead of the counter-based
    generator.  ``backfill_index`` (int32 ``[B]``, -1 = skip) says where in the next
    iteration's input-id tensor of ``backfill_len`` entries each row's token goes
    (early feedback, §5.2).  ``output_start`` (int32 ``[B]``) splits each history into prompt
    (the first ``output_start[b]`` ids) and generated output (the rest): the repetition penalty then
    looks at both, the presence and frequency penalties at the output alone.
    ``topk_keep_ties`` switches top-k to "keep every score not below the k-th largest";
    ``logprob_full_vocab`` reports log-probabilities relative to the softmax over the whole row.
    """

    name: str
    B: int
    V: int
    dtype: int
    logits: np.ndarray
    temperature: Optional[np.ndarray] = None
    top_k: Optional[np.ndarray] = None
    top_p: Optional[np.ndarray] = None
    min_p: Optional[np.ndarray] = None
    repetition_penalty: Optional[np.ndarray] = None
    presence_penalty: Optional[np.ndarray] = None
    frequency_penalty: Optional[np.ndarray] = None
    history_ids: Optional[np.ndarray] = None
    history_offsets: Optional[np.ndarray] = None
    seeds: Optional[np.ndarray] = None
    step: int = 0
    row_base: int = 0
    num_top: int = 0
    exp1: Optional[np.ndarray] = None
    backfill_index: Optional[np.ndarray] = None
    backfill_len: int = 0
    output_start: Optional[np.ndarray] = None
    topk_keep_ties: bool = False
    logprob_full_vocab: bool = False
    notes: dict = field(default_factory=dict)

    @property
    def elem_size(self) -> int:
        return 4 if self.dtype == F32 else 2

    @property
    def logit_bytes(self) -> int:
        return self.B * self.V * self.elem_size

    @property
    def history_bytes(self) -> int:
        if self.history_ids is None:
            return 0
        return int(self.history_ids.size) * 4 + int(self.history_offsets.size) * 4

    def logits_f32(self) -> np.ndarray:
        if self.dtype == F16:
            return self.logits.view(np.float16).astype(np.float32)
        return self.logits if self.dtype == F32 else bf16_bits_to_f32(self.logits)

    def rows(self, lo: int, hi: int) -> "Workload":
        """Rows [lo, hi) as a self-contained workload whose ``row_base`` keeps the
        global row ids (used by the shard-invariance tests and the row-sharded
        multi-GPU path, §6.1)."""
        def cut(a):
            return None if a is None else np.ascontiguousarray(a[lo:hi])
        hid = hoff = None
        if self.history_ids is not None:
            o = self.history_offsets
            hid = np.ascontiguousarray(self.history_ids[o[lo]:o[hi]])
            hoff = (o[lo:hi + 1] - o[lo]).astype(np.int32)
        return Workload(
            name=f"{self.name}[{lo}:{hi}]", B=hi - lo, V=self.V, dtype=self.dtype,
            logits=np.ascontiguousarray(self.logits[lo:hi]),
            temperature=cut(self.temperature), top_k=cut(self.top_k), top_p=cut(self.top_p),
            min_p=cut(self.min_p), repetition_penalty=cut(self.repetition_penalty),
            presence_penalty=cut(self.presence_penalty), frequency_penalty=cut(self.frequency_penalty),
            history_ids=hid, history_offsets=hoff, seeds=cut(self.seeds), step=self.step,
            row_base=self.row_base + lo, num_top=self.num_top, exp1=cut(self.exp1),
            backfill_index=cut(self.backfill_index), backfill_len=self.backfill_len,
            output_start=cut(self.output_start), topk_keep_ties=self.topk_keep_ties,
            logprob_full_vocab=self.logprob_full_vocab, notes=dict(self.notes))


# --------------------------------------------------------------------------- helpers

def _rng(config_number: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(1000 + config_number))


def _full(B, value, dtype):
    return np.full(B, value, dtype=dtype)


def _zipf_cdf(V: int, s: float) -> np.ndarray:
    w = np.arange(1, V + 1, dtype=np.float64) ** (-s)
    c = np.cumsum(w)
    return c / c[-1]


def zipf_ids(rng: np.random.Generator, V: int, s: float, n: int, cdf=None) -> np.ndarray:
    """n token ids with P(id = r-1) proportional to r^-s on r in [1, V]."""
    if cdf is None:
        cdf = _zipf_cdf(V, s)
    u = rng.random(n)
    return np.minimum(np.searchsorted(cdf, u, side="left"), V - 1).astype(np.int32)


def _gauss(rng, B, V, std):
    # drawn row by row to bound peak host memory for the largest configs
    out = np.empty((B, V), dtype=np.float32)
    for b in range(B):
        out[b] = rng.standard_normal(V, dtype=np.float32) * np.float32(std)
    return out


def _zipf_bias(V: int, s: float) -> np.ndarray:
    # log of an (unnormalised) Zipf(s) pmf with rank = id + 1, shared by all rows
    return (-s * np.log(np.arange(1, V + 1, dtype=np.float64))).astype(np.float32)


def _histories(rng, B, V, lengths, s=1.2):
    cdf = _zipf_cdf(V, s)
    off = np.zeros(B + 1, dtype=np.int64)
    off[1:] = np.cumsum(lengths)
    ids = zipf_ids(rng, V, s, int(off[-1]), cdf=cdf)
    return ids, off.astype(np.int32)


# --------------------------------------------------------------------------- configs

def config1(B=8, V=32000) -> Workload:
    """fp32 logits ~ N(0, 2^2) with five +8 spikes per row; T=0.8, top_k=50."""
    rng = _rng(1)
    x = _gauss(rng, B, V, 2.0)
    for b in range(B):
        ids = rng.choice(V, size=5, replace=False)
        x[b, ids] += np.float32(8.0)
    return Workload("config1", B, V, F32, x,
                    temperature=_full(B, 0.8, np.float32), top_k=_full(B, 50, np.int32),
                    seeds=np.zeros(B, dtype=np.uint64), step=0)


def config2(B=128, V=152064, name="config2") -> Workload:
    """bf16 logits ~ N(0, 3^2) + Zipf(1.1)-ranked bias; T=0.7, top_k=40, top_p=0.9."""
    rng = _rng(2)
    x = _gauss(rng, B, V, 3.0)
    x += _zipf_bias(V, 1.1)[None, :]
    return Workload(name, B, V, BF16, f32_to_bf16_bits(x),
                    temperature=_full(B, 0.7, np.float32), top_k=_full(B, 40, np.int32),
                    top_p=_full(B, 0.9, np.float32),
                    seeds=np.arange(B, dtype=np.uint64), step=0)


def config_metric(B=256, V=152064) -> Workload:
    """The metric workload: config 2's generator and parameters at B=256."""
    return config2(B=B, V=V, name="configM")


def config3(B=256, V=128256, hist_len=2048) -> Workload:
    """bf16 N(0, 3^2) + ten spikes of U[6,10]; all three penalties from 2048-id
    Zipf(1.2) histories; T=1, min_p=0.05, top_p=0.95."""
    rng = _rng(3)
    x = _gauss(rng, B, V, 3.0)
    for b in range(B):
        ids = rng.choice(V, size=10, replace=False)
        x[b, ids] += rng.uniform(6.0, 10.0, size=10).astype(np.float32)
    hid, hoff = _histories(rng, B, V, np.full(B, hist_len, dtype=np.int64))
    return Workload("config3", B, V, BF16, f32_to_bf16_bits(x),
                    temperature=_full(B, 1.0, np.float32),
                    top_p=_full(B, 0.95, np.float32), min_p=_full(B, 0.05, np.float32),
                    repetition_penalty=_full(B, 1.1, np.float32),
                    presence_penalty=_full(B, 0.5, np.float32),
                    frequency_penalty=_full(B, 0.3, np.float32),
                    history_ids=hid, history_offsets=hoff,
                    seeds=np.arange(B, dtype=np.uint64), step=0)


def config4(B=512, V=152064, max_hist=4096) -> Workload:
    """bf16 logits as config 2; row class = b mod 4: greedy / top-k in U{1..100} /
    top-p in U[0.5,1] / min-p in U[0.01,0.2]; T in U[0.3,1.5]; histories of
    U{0..4096} ids; penalty coefficients as config 3."""
    rng = _rng(4)
    x = _gauss(rng, B, V, 3.0)
    x += _zipf_bias(V, 1.1)[None, :]
    cls = np.arange(B) % 4
    T = rng.uniform(0.3, 1.5, size=B).astype(np.float32)
    T[cls == 0] = 0.0
    top_k = np.zeros(B, dtype=np.int32)
    top_k[cls == 1] = rng.integers(1, 101, size=int((cls == 1).sum()), dtype=np.int32)
    top_p = np.ones(B, dtype=np.float32)
    top_p[cls == 2] = rng.uniform(0.5, 1.0, size=int((cls == 2).sum())).astype(np.float32)
    min_p = np.zeros(B, dtype=np.float32)
    min_p[cls == 3] = rng.uniform(0.01, 0.2, size=int((cls == 3).sum())).astype(np.float32)
    lengths = rng.integers(0, max_hist + 1, size=B).astype(np.int64)
    hid, hoff = _histories(rng, B, V, lengths)
    return Workload("config4", B, V, BF16, f32_to_bf16_bits(x),
                    temperature=T, top_k=top_k, top_p=top_p, min_p=min_p,
                    repetition_penalty=_full(B, 1.1, np.float32),
                    presence_penalty=_full(B, 0.5, np.float32),
                    frequency_penalty=_full(B, 0.3, np.float32),
                    history_ids=hid, history_offsets=hoff,
                    seeds=np.arange(B, dtype=np.uint64), step=0,
                    notes={"row_class": cls})


def config5(B=1024, V=129280, hist_len=1024) -> Workload:
    """fp32 N(0, 4^2); every 100th row near-flat (std 0.01), the next one-hot-like
    (+30 on one id); T=0.6, top_k=20, top_p=0.8; penalties as config 3 from
    1024-id histories; top-20 logprobs requested."""
    rng = _rng(5)
    x = _gauss(rng, B, V, 4.0)
    for b in range(B):
        if b % 100 == 0:
            x[b] = rng.standard_normal(V, dtype=np.float32) * np.float32(0.01)
        elif b % 100 == 1:
            x[b, int(rng.integers(0, V))] += np.float32(30.0)
    hid, hoff = _histories(rng, B, V, np.full(B, hist_len, dtype=np.int64))
    return Workload("config5", B, V, F32, x,
                    temperature=_full(B, 0.6, np.float32), top_k=_full(B, 20, np.int32),
                    top_p=_full(B, 0.8, np.float32),
                    repetition_penalty=_full(B, 1.1, np.float32),
                    presence_penalty=_full(B, 0.5, np.float32),
                    frequency_penalty=_full(B, 0.3, np.float32),
                    history_ids=hid, history_offsets=hoff,
                    seeds=np.arange(B, dtype=np.uint64), step=0, num_top=20)


CONFIGS = {
    "config1": config1, "config2": config2, "configM": config_metric,
    "config3": config3, "config4": config4, "config5": config5,
}


def make(name: str, **kw) -> Workload:
    return CONFIGS[name](**kw)


# --------------------------------------------------------------------------- small / adversarial

def random_small(seed: int, B: int, V: int, dtype: int = F32, *, std=2.0, with_history=True,
                 quantise=None) -> Workload:
    """A small mixed-parameter batch for element-by-element parity checks.

    ``quantise`` (a float step) rounds logits to multiples of that step so that
    exact ties at every cut are common.
    """
    rng = np.random.Generator(np.random.PCG64(seed))
    x = rng.standard_normal((B, V)).astype(np.float32) * np.float32(std)
    if quantise:
        x = (np.round(x / quantise) * quantise).astype(np.float32)
    T = rng.uniform(0.3, 1.5, size=B).astype(np.float32)
    T[rng.random(B) < 0.15] = 0.0
    top_k = rng.integers(1, max(2, min(V, 64)), size=B).astype(np.int32)
    top_k[rng.random(B) < 0.35] = 0
    top_p = rng.uniform(0.3, 1.0, size=B).astype(np.float32)
    top_p[rng.random(B) < 0.35] = 1.0
    min_p = rng.uniform(0.005, 0.3, size=B).astype(np.float32)
    min_p[rng.random(B) < 0.5] = 0.0
    w = Workload(f"small{seed}", B, V, dtype,
                 x if dtype == F32 else f32_to_bf16_bits(x),
                 temperature=T, top_k=top_k, top_p=top_p, min_p=min_p,
                 seeds=rng.integers(0, 2**63, size=B, dtype=np.uint64), step=int(rng.integers(0, 2**40)))
    if with_history:
        lengths = rng.integers(0, 4 * min(V, 64), size=B).astype(np.int64)
        lengths[rng.random(B) < 0.2] = 0
        hid, hoff = _histories(rng, B, V, lengths)
        # a few ids outside [0, V) which the sampler must ignore
        if hid.size:
            bad = rng.random(hid.size) < 0.01
            hid[bad] = np.where(rng.random(int(bad.sum())) < 0.5, -1, V + 3).astype(np.int32)
        w.history_ids, w.history_offsets = hid, hoff
        w.repetition_penalty = rng.uniform(0.8, 1.5, size=B).astype(np.float32)
        w.presence_penalty = rng.uniform(-0.5, 1.0, size=B).astype(np.float32)
        w.frequency_penalty = rng.uniform(-0.2, 0.5, size=B).astype(np.float32)
    return w


def as_f16(w: Workload) -> Workload:
    """The same workload with its logits rounded to binary16 (stored as uint16 bit patterns)."""
    import copy
    out = copy.copy(w)
    out.name = w.name + "_f16"
    out.dtype = F16
    out.logits = np.ascontiguousarray(w.logits_f32().astype(np.float16).view(np.uint16))
    out.notes = dict(w.notes)
    return out


def with_exp1(w: Workload, seed: int = 7) -> Workload:
    """The same workload drawing from a pre-generated ``[B, V]`` table of Exp(1) variates."""
    import copy
    out = copy.copy(w)
    out.name = w.name + "_exp1"
    rng = np.random.Generator(np.random.PCG64(seed))
    out.exp1 = rng.standard_exponential((w.B, w.V), dtype=np.float32)
    np.maximum(out.exp1, np.float32(1e-30), out=out.exp1)      # strictly positive: ln E stays finite
    out.notes = dict(w.notes)
    return out


def with_backfill(w: Workload, seed: int = 11, slack: int = 3) -> Workload:
    """The same workload with a scattered early-feedback map: row b's token goes to a distinct
    slot of a ``B + slack`` entry input-id tensor; about one row in eight is skipped (-1)."""
    import copy
    out = copy.copy(w)
    rng = np.random.Generator(np.random.PCG64(seed))
    out.backfill_len = w.B + slack
    idx = rng.permutation(out.backfill_len)[: w.B].astype(np.int32)
    idx[rng.random(w.B) < 0.125] = -1
    out.backfill_index = idx
    out.notes = dict(w.notes)
    return out


def with_split_history(w: Workload, seed: int = 13) -> Workload:
    """The same workload with every history split at a random point into prompt and output
    (a few rows all prompt, a few all output)."""
    import copy
    out = copy.copy(w)
    out.name = w.name + "_split"
    rng = np.random.Generator(np.random.PCG64(seed))
    lens = np.diff(w.history_offsets.astype(np.int64))
    start = np.floor(rng.random(w.B) * (lens + 1)).astype(np.int32)
    pick = rng.random(w.B)
    start[pick < 0.1] = 0
    start[pick > 0.9] = lens[pick > 0.9].astype(np.int32)
    out.output_start = start
    out.notes = dict(w.notes)
    return out
