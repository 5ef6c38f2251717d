"""Pins for the CPU oracle: each test ties a part of it to something other than itself
(a hand-computed example, a published known-answer vector, a closed form, a library
routine on a special case, brute force on tiny inputs, or a statistical law)."""
import json
import math
import os
from decimal import Decimal, getcontext
from fractions import Fraction

import numpy as np
import pytest
import scipy.special
import scipy.stats
import torch

from oracle import albireo_oracle as O
from paper_2606_01927_b200 import workloads as W


def one_row(x, dtype=W.F32, T=None, top_k=None, top_p=None, min_p=None, r=None, p=None, f=None,
            history=None, seed=0, step=0, row_base=0, num_top=0, B=None):
    x = np.atleast_2d(np.asarray(x))
    B = x.shape[0]
    arr = lambda v, dt: None if v is None else np.full(B, v, dtype=dt) if np.isscalar(v) else np.asarray(v, dtype=dt)
    logits = x.astype(np.float32) if dtype == W.F32 else W.f32_to_bf16_bits(x.astype(np.float32))
    hid = hoff = None
    if history is not None:
        hid = np.tile(np.asarray(history, dtype=np.int32), B)
        hoff = (np.arange(B + 1) * len(history)).astype(np.int32)
    return W.Workload("t", B, x.shape[1], dtype, np.ascontiguousarray(logits),
                      temperature=arr(T, np.float32), top_k=arr(top_k, np.int32), top_p=arr(top_p, np.float32),
                      min_p=arr(min_p, np.float32), repetition_penalty=arr(r, np.float32),
                      presence_penalty=arr(p, np.float32), frequency_penalty=arr(f, np.float32),
                      history_ids=hid, history_offsets=hoff,
                      seeds=arr(seed, np.uint64), step=step, row_base=row_base, num_top=num_top)


# ------------------------------------------------------------------ Philox

def philox_bigint(ctr, key):
    """Independent restatement with Python integers (no 32-bit types anywhere)."""
    M0, M1 = 0xD2511F53, 0xCD9E8D57
    c = list(ctr)
    k = list(key)
    mask = (1 << 32) - 1
    for _ in range(10):
        p0, p1 = M0 * c[0], M1 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k[0], p1 & mask, (p0 >> 32) ^ c[3] ^ k[1], p0 & mask]
        k = [(k[0] + 0x9E3779B9) & mask, (k[1] + 0xBB67AE85) & mask]
    return c


def test_philox_known_answer_vectors(golden_dir):
    n = 0
    for line in open(os.path.join(golden_dir, "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(t, 16) for t in line.split()]
        assert O.philox4x32_10(w[0:4], w[4:6]) == w[6:10]
        assert philox_bigint(w[0:4], w[4:6]) == w[6:10]
        n += 1
    assert n == 3


def test_philox_matches_bigint_on_random_counters():
    rng = np.random.default_rng(7)
    for _ in range(200):
        ctr = [int(v) for v in rng.integers(0, 2**32, size=4)]
        key = [int(v) for v in rng.integers(0, 2**32, size=2)]
        assert O.philox4x32_10(ctr, key) == philox_bigint(ctr, key)


def test_race_word_keying():
    # token id -> (block id>>2, word id&3); row, step and seed go to the other counter/key words
    seed, R, step = (5 << 32) | 9, 77, (3 << 32) | 11
    for tok in [0, 1, 2, 3, 4, 5, 1023, 152063]:
        blk = philox_bigint([tok >> 2, R, step & 0xFFFFFFFF, step >> 32], [seed & 0xFFFFFFFF, seed >> 32])
        assert O.race_word(seed, R, step, tok) == blk[tok & 3]


def test_exp1_map_against_high_precision():
    getcontext().prec = 60
    for w in [0, 1, 2, 1000, 2**31, 2**32 - 2, 2**32 - 1, 0x9ceaf053]:
        v = (Decimal(w) + Decimal("0.5")) / Decimal(2**32)
        ref = -(Decimal(1) - v).ln()
        got = O.exp1_from_word(w)
        assert abs(Decimal(got) - ref) <= abs(ref) * Decimal("4e-16")
    assert O.exp1_from_word(0) > 0 and math.isfinite(O.exp1_from_word(2**32 - 1))


# ------------------------------------------------------------------ worked example

@pytest.fixture(scope="module")
def worked(golden_dir):
    return json.load(open(os.path.join(golden_dir, "worked_example.json")))


def test_worked_example_scores(worked):
    x = np.array(worked["x"], dtype=np.float32)
    z = O.row_scores(x, W.F32, T=worked["temperature"], r=worked["repetition_penalty"],
                     p=worked["presence_penalty"], f=worked["frequency_penalty"], history=worked["history"])
    assert z.tolist() == worked["z"]
    xpen = O.row_scores(x, W.F32, T=1.0, r=worked["repetition_penalty"], p=worked["presence_penalty"],
                        f=worked["frequency_penalty"], history=worked["history"])
    assert xpen.tolist() == worked["x_pen"]


@pytest.mark.parametrize("case", ["A", "B", "C", "D"])
def test_worked_example_cases(worked, case):
    c = worked["cases"][case]
    for d in c["draws"]:
        w = one_row(worked["x"], T=worked["temperature"], top_k=c["top_k"], top_p=c["top_p"], min_p=c["min_p"],
                    r=worked["repetition_penalty"], p=worked["presence_penalty"], f=worked["frequency_penalty"],
                    history=worked["history"], seed=d["seed"], step=d["step"], row_base=d["row"], num_top=8)
        o = O.sample(w, topk_cap=8, kept_cap=8)
        kept = [i for i in o.kept_ids[0].tolist() if i >= 0]
        assert kept == c["kept"]
        if "topk_ids" in c:
            assert [i for i in o.topk_ids[0].tolist() if i >= 0] == c["topk_ids"]
        assert int(o.tokens[0]) == d["token"]
        assert abs(o.logprobs[0] - d["logprob"]) < 2e-10
        lps = o.top_logprobs[0][: len(kept)]
        assert np.allclose(lps, c["logprobs"], atol=2e-10, rtol=0)
        assert o.top_ids[0][: len(kept)].tolist() == kept
        assert (o.top_ids[0][len(kept):] == -1).all() and np.isneginf(o.top_logprobs[0][len(kept):]).all()
        if "S" in c:
            assert abs(o.rows["S"][0] - c["S"]) < 2e-10
        for tok, word in d.get("words", {}).items():
            assert O.race_word(d["seed"], d["row"], d["step"], int(tok)) == int(word, 16)
        if "g" in d:
            _, ids, zs, gs = O.row_shifted(w, 0, want_sorted=True)
            for tok, g in d["g"].items():
                j = ids.tolist().index(int(tok))
                assert abs(gs[j] - g) < 2e-10


def test_worked_example_full_order(worked):
    w = one_row(worked["x"], T=worked["temperature"], r=worked["repetition_penalty"],
                p=worked["presence_penalty"], f=worked["frequency_penalty"], history=worked["history"])
    _, ids, zs, _ = O.row_shifted(w, 0, want_sorted=True)
    assert ids.tolist() == worked["order"]


def test_worked_example_draw_frequencies(worked):
    """Case A over 20000 seeds: chi-square against the closed-form kept-set distribution."""
    c = worked["cases"]["A"]
    n = 20000
    x = np.tile(np.array(worked["x"], dtype=np.float32), (n, 1))
    w = one_row(x, T=worked["temperature"], top_k=c["top_k"], top_p=c["top_p"], min_p=c["min_p"],
                r=worked["repetition_penalty"], p=worked["presence_penalty"], f=worked["frequency_penalty"],
                history=worked["history"], seed=np.arange(n, dtype=np.uint64))
    o = O.sample(w)
    q = np.exp(np.array(c["logprobs"]))
    counts = np.array([(o.tokens == t).sum() for t in c["kept"]])
    assert counts.sum() == n
    chi2 = float((((counts - n * q) ** 2) / (n * q)).sum())
    assert scipy.stats.chi2.sf(chi2, len(q) - 1) > 1e-3


# ------------------------------------------------------------------ conversions and element-wise steps

def test_bf16_widening_exhaustive():
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    z = O.row_scores(bits, W.BF16)          # T=1, no penalties: z == widened logits
    ref = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float32).numpy()
    ok = ~np.isnan(ref)
    assert (z.view(np.uint32)[ok] == ref.view(np.uint32)[ok]).all()
    assert np.isnan(z[~ok]).all()


def test_identity_parameters_leave_bits_unchanged():
    rng = np.random.default_rng(3)
    x = (rng.standard_normal(4096) * 5).astype(np.float32)
    x[:4] = [0.0, -0.0, np.float32(1e-40), -np.inf]
    hist = rng.integers(0, 4096, size=3000)
    z = O.row_scores(x, W.F32, T=1.0, r=1.0, p=0.0, f=0.0, history=hist)
    assert (z.view(np.uint32) == x.view(np.uint32)).all()


def test_penalties_elementwise_fp32_semantics():
    """Each penalty step is one IEEE fp32 operation; recomputed with numpy float32 scalars
    and, separately, with exact rational arithmetic rounded once per step."""
    rng = np.random.default_rng(11)
    V = 512
    x = (rng.standard_normal(V) * 3).astype(np.float32)
    hist = rng.integers(-2, V + 2, size=700)            # includes out-of-range ids
    r, p, f, T = np.float32(1.3), np.float32(0.7), np.float32(0.15), np.float32(0.9)
    z = O.row_scores(x, W.F32, T=float(T), r=float(r), p=float(p), f=float(f), history=hist)
    cnt = np.bincount(hist[(hist >= 0) & (hist < V)], minlength=V)
    assert cnt.max() >= 3

    def rnd(fr):       # round an exact rational to fp32 (nearest even) via float64 (exact here: |fr| moderate)
        return np.float32(float(fr))

    inv_T = np.float32(1.0) / T
    for i in range(V):
        a = x[i]
        if cnt[i] > 0:
            a = a / r if a > 0 else a * r
            a = a - f * np.float32(cnt[i])
            a = a - p
        assert np.float32(a * inv_T) == z[i]
    # exact-rational cross-check on penalised entries (division is the step most easily got wrong)
    for i in np.nonzero(cnt)[0][:50]:
        a = Fraction(float(x[i]))
        a = Fraction(float(rnd(a / Fraction(float(r))))) if x[i] > 0 else Fraction(float(rnd(a * Fraction(float(r)))))
        t = rnd(Fraction(float(f)) * int(cnt[i]))
        a = Fraction(float(rnd(a - Fraction(float(t)))))
        a = Fraction(float(rnd(a - Fraction(float(p)))))
        a = rnd(a * Fraction(float(inv_T)))
        assert a == z[i]


def test_repetition_sign_branch_and_zero():
    x = np.array([2.0, -2.0, 0.0, 4.0], dtype=np.float32)
    z = O.row_scores(x, W.F32, T=1.0, r=2.0, p=0.0, f=0.0, history=[0, 1, 2])
    assert z.tolist() == [1.0, -4.0, 0.0, 4.0]


def test_order_key_is_order_preserving():
    vals = np.array([-np.inf, -3.5, -1e-40, -0.0, 0.0, 1e-40, 2.0, 2.0000002, 1e30, np.inf], dtype=np.float32)
    keys = [O.order_key(float(v)) for v in vals]
    assert keys == sorted(keys) and len(set(keys)) == len(keys)


# ------------------------------------------------------------------ order, top-k

def test_total_order_matches_lexsort_with_ties():
    rng = np.random.default_rng(5)
    for trial in range(20):
        V = int(rng.integers(2, 400))
        x = np.round(rng.standard_normal(V) * 2).astype(np.float32)      # many exact ties
        w = one_row(x, T=1.0)
        _, ids, zs, _ = O.row_shifted(w, 0, want_sorted=True)
        ref = np.lexsort((np.arange(V), -x.astype(np.float64)))
        # -0.0 sorts below +0.0 by design; avoid the case rather than model it
        if np.any(np.signbit(x) & (x == 0)):
            continue
        assert ids.tolist() == ref.tolist()


def test_topk_brute_force_tiny_vocab():
    rng = np.random.default_rng(9)
    for V in [1, 2, 3, 7, 16]:
        for trial in range(6):
            x = np.round(rng.standard_normal(V) * 1.5).astype(np.float32) + np.float32(0.25)
            prev = None
            for k in range(0, V + 2):
                w = one_row(x, T=1.0, top_k=k)
                o = O.sample(w, topk_cap=V, kept_cap=V)
                kept = [i for i in o.topk_ids[0].tolist() if i >= 0]
                # brute force: repeatedly take the largest remaining value, lowest index on ties
                want_n = V if (k <= 0 or k >= V) else k
                rest = list(range(V)); ref = []
                while len(ref) < want_n:
                    best = max(rest, key=lambda i: (x[i], -i))
                    ref.append(best); rest.remove(best)
                assert kept == ref
                if prev is not None and 0 < k < V:
                    assert set(prev) <= set(kept)          # membership monotone in k
                if 0 < k < V:
                    prev = kept


def test_topk1_is_greedy_lowest_index_argmax():
    rng = np.random.default_rng(13)
    x = np.round(rng.standard_normal((64, 300)) * 2).astype(np.float32) + np.float32(0.5)
    for kw in [dict(T=0.9, top_k=1), dict(T=0.0)]:
        o = O.sample(one_row(x, seed=np.arange(64, dtype=np.uint64), **kw))
        assert (o.tokens == np.argmax(x, axis=1)).all()
        assert (o.logprobs == 0).all() and (o.rows["n_keep"] == 1).all()


def test_greedy_ignores_other_cuts_and_scaling():
    x = np.array([[1.0, 3.0, 3.0, -1.0]], dtype=np.float32)
    o = O.sample(one_row(x, T=0.0, top_k=3, top_p=0.1, min_p=0.9))
    assert int(o.tokens[0]) == 1 and o.rows["greedy"][0] == 1


def test_minus_inf_rows_keep_only_finite():
    x = np.full((1, 10), -np.inf, dtype=np.float32)
    x[0, [2, 7, 8]] = [1.0, 2.0, 1.0]
    o = O.sample(one_row(x, T=1.0, top_k=5), topk_cap=10, kept_cap=10)
    assert o.rows["n_fin"][0] == 3 and o.rows["n_topk"][0] == 3
    assert [i for i in o.topk_ids[0].tolist() if i >= 0] == [7, 2, 8]


# ------------------------------------------------------------------ min-p / top-p / softmax

def test_no_cuts_equals_library_log_softmax():
    rng = np.random.default_rng(17)
    for dtype in (W.F32, W.BF16):
        x = (rng.standard_normal((3, 200)) * 3).astype(np.float32)
        T = 0.75
        w = one_row(x, dtype=dtype, T=T, num_top=200, seed=np.arange(3, dtype=np.uint64))
        o = O.sample(w)
        xin = w.logits_f32()
        z = (xin * (np.float32(1.0) / np.float32(T))).astype(np.float32).astype(np.float64)
        ref = scipy.special.log_softmax(z, axis=1)
        for b in range(3):
            got = np.full(200, np.nan)
            got[o.top_ids[b]] = o.top_logprobs[b]
            assert np.max(np.abs(got - ref[b])) < 1e-12
            assert abs(o.logprobs[b] - ref[b, o.tokens[b]]) < 1e-12
            assert abs(np.exp(o.top_logprobs[b]).sum() - 1.0) < 1e-12


def test_kept_probabilities_sum_to_one_under_cuts():
    w = W.random_small(21, B=64, V=500, dtype=W.BF16)
    w.num_top = 500
    o = O.sample(w)
    s = np.exp(o.top_logprobs).sum(axis=1)
    assert np.max(np.abs(s - 1.0)) < 1e-12
    assert ((o.top_ids >= 0).sum(axis=1) == o.rows["n_keep"]).all()


def test_closed_forms_flat_and_two_point():
    x = np.full((1, 12), 1.5, dtype=np.float32)
    o = O.sample(one_row(x, T=0.7, top_k=5, num_top=12))
    assert o.rows["n_keep"][0] == 5 and abs(o.logprobs[0] + math.log(5)) < 1e-12
    assert o.top_ids[0][:5].tolist() == [0, 1, 2, 3, 4]
    # two-point row: probabilities sigma(+-a/T)
    a, T = 1.25, 0.5
    x = np.array([[0.0, a]], dtype=np.float32)
    o = O.sample(one_row(x, T=T, num_top=2))
    lp = dict(zip(o.top_ids[0].tolist(), o.top_logprobs[0].tolist()))
    assert abs(lp[1] + math.log1p(math.exp(-a / T))) < 1e-12
    assert abs(lp[0] - (-a / T - math.log1p(math.exp(-a / T)))) < 1e-12


def test_top_p_definition_on_known_masses():
    # probabilities 0.5, 0.25, 0.125, 0.125 (z = ln of them, T = 1)
    q = np.array([0.5, 0.25, 0.125, 0.125])
    x = np.log(q).astype(np.float32)[None, :]
    for top_p, n in [(0.0, 1), (0.3, 1), (0.6, 2), (0.76, 3), (0.9, 4), (1.0, 4)]:
        o = O.sample(one_row(x, T=1.0, top_p=top_p))
        assert o.rows["n_keep"][0] == n, top_p
    # mass refers to the survivors of top-k: with top_k=2 the masses are 2/3, 1/3
    o = O.sample(one_row(x, T=1.0, top_k=2, top_p=0.7))
    assert o.rows["n_keep"][0] == 2
    o = O.sample(one_row(x, T=1.0, top_k=2, top_p=0.6))
    assert o.rows["n_keep"][0] == 1


def test_min_p_definition_and_floor_of_one():
    q = np.array([0.5, 0.25, 0.125, 0.125])
    x = np.log(q).astype(np.float32)[None, :]
    for min_p, n in [(0.0, 4), (0.2, 4), (0.3, 2), (0.6, 1), (1.5, 1)]:
        o = O.sample(one_row(x, T=1.0, min_p=min_p))
        assert o.rows["n_keep"][0] == n, min_p


def test_cut_monotonicity():
    rng = np.random.default_rng(23)
    x = (rng.standard_normal((1, 300)) * 2.5).astype(np.float32)
    prev = 0
    for tp in np.linspace(0.0, 1.0, 21):
        n = int(O.sample(one_row(x, T=1.0, top_p=float(tp))).rows["n_keep"][0])
        assert n >= prev; prev = n
    prev = 10**9
    for mp in np.linspace(0.001, 1.0, 21):
        n = int(O.sample(one_row(x, T=1.0, min_p=float(mp))).rows["n_keep"][0])
        assert n <= prev; prev = n
    prev = 0
    for k in range(1, 300, 13):
        n = int(O.sample(one_row(x, T=1.0, top_k=k, top_p=0.9)).rows["n_keep"][0])
        assert n >= prev; prev = n


# ------------------------------------------------------------------ race distribution

def _draw_freq_check(x, n, **params):
    V = len(x)
    w = one_row(np.tile(np.asarray(x, dtype=np.float32), (n, 1)), seed=np.arange(n, dtype=np.uint64), num_top=V, **params)
    o = O.sample(w)
    # every row has the same kept set and distribution (only seed and row id differ)
    ids = o.top_ids[0][o.top_ids[0] >= 0]
    return o, ids


def test_race_distribution_chi_square_tiny_vocab():
    rng = np.random.default_rng(29)
    n = 100_000
    for V, params in [(16, dict(T=1.0)), (16, dict(T=0.8, top_k=6)), (11, dict(T=1.2, top_p=0.8)), (5, dict(T=1.0, min_p=0.1))]:
        x = (rng.standard_normal(V) * 1.5).astype(np.float32)
        o, ids = _draw_freq_check(x, n, **params)
        # closed-form renormalised distribution over the kept ids, computed independently
        z = (x * (np.float32(1.0) / np.float32(params["T"]))).astype(np.float64)[ids]
        q = np.exp(z - z.max()); q /= q.sum()
        counts = np.array([(o.tokens == t).sum() for t in ids])
        assert counts.sum() == n
        chi2 = float((((counts - n * q) ** 2) / (n * q)).sum())
        assert scipy.stats.chi2.sf(chi2, max(1, len(ids) - 1)) > 1e-3, (V, params, chi2)


def test_race_binomial_two_tokens():
    n = 100_000
    o, ids = _draw_freq_check([0.0, 1.0], n, T=1.0)
    q1 = 1.0 / (1.0 + math.exp(-1.0))
    k = int((o.tokens == 1).sum())
    assert abs(k - n * q1) < 4.5 * math.sqrt(n * q1 * (1 - q1))


def test_single_survivor_needs_no_draw():
    x = np.array([[0.0, 9.0, 1.0]], dtype=np.float32)
    for seed in range(20):
        o = O.sample(one_row(x, T=1.0, top_p=0.5, seed=seed))
        assert int(o.tokens[0]) == 1 and o.logprobs[0] == 0 and np.isinf(o.rows["race_gap"][0])


# ------------------------------------------------------------------ shard invariance, determinism, bands

def test_shard_invariance_and_padding():
    w = W.random_small(31, B=24, V=700, dtype=W.BF16)
    full = O.sample(w)
    a, b = O.sample(w.rows(0, 10)), O.sample(w.rows(10, 24))
    assert (np.concatenate([a.tokens, b.tokens]) == full.tokens).all()
    assert (np.concatenate([a.logprobs, b.logprobs]) == full.logprobs).all()
    # different row ids must change draws for a diffuse row
    w2 = w.rows(0, 24); w2.row_base = 1000
    assert (O.sample(w2).tokens != full.tokens).any()


def test_step_and_seed_change_draws():
    x = np.zeros((1, 64), dtype=np.float32)
    toks = {int(O.sample(one_row(x, T=1.0, seed=3, step=s)).tokens[0]) for s in range(40)}
    assert len(toks) > 10
    toks = {int(O.sample(one_row(x, T=1.0, seed=s, step=(1 << 40))).tokens[0]) for s in range(40)}
    assert len(toks) > 10


def test_threads_do_not_change_results():
    w = W.random_small(37, B=40, V=900)
    a, b = O.sample(w, threads=1, topk_cap=16), O.sample(w, threads=4, topk_cap=16)
    assert (a.rows == b.rows).all() and (a.topk_ids == b.topk_ids).all()


def test_acceptable_results_on_exact_cut_boundary():
    # four equal logits, top_p = 0.5: the cumulative mass hits the target exactly after two
    x = np.zeros((1, 4), dtype=np.float32)
    w = one_row(x, T=1.0, top_p=0.5, seed=5)
    o = O.sample(w)
    assert o.rows["n_keep"][0] == 2 and o.rows["topp_margin"][0] < 1e-12
    acc = O.acceptable(w, 0)
    assert acc[0][0] == int(o.tokens[0])
    assert {a[2] for a in acc} == {2, 3}          # one element more is inside the top_p band
    # min-p exactly on an element
    x = np.log(np.array([[0.5, 0.25, 0.125, 0.125]])).astype(np.float32)
    w = one_row(x, T=1.0, min_p=0.25, seed=5)
    assert O.sample(w).rows["minp_margin"][0] < 1e-6
    assert {a[2] for a in O.acceptable(w, 0)} >= {2, 4} or {a[2] for a in O.acceptable(w, 0)} >= {1, 2}


def test_acceptable_is_just_the_primary_away_from_boundaries():
    w = W.config1(B=4, V=2000)
    o = O.sample(w)
    for b in range(4):
        acc = O.acceptable(w, b)
        assert all(a[0] == acc[0][0] and abs(a[1] - acc[0][1]) < 1e-12 for a in acc)
        assert acc[0][0] == int(o.tokens[b])


# ------------------------------------------------------------------ fp16 logits and pre-generated Exp(1) variates

def test_f16_widening_exhaustive():
    # §8.1: the paper's models run in FP16; binary16 -> fp32 is exact, checked against the library cast
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    z = O.row_scores(bits, W.F16)           # T=1, no penalties: z == widened logits
    ref = bits.view(np.float16).astype(np.float32)
    ok = ~np.isnan(ref)
    assert (z.view(np.uint32)[ok] == ref.view(np.uint32)[ok]).all()
    assert np.isnan(z[~ok]).all()


def test_f16_rows_equal_fp32_rows_of_the_same_values():
    rng = np.random.default_rng(41)
    x = (rng.standard_normal((6, 300)) * 3).astype(np.float16)
    w32 = one_row(x.astype(np.float32), T=0.8, top_k=20, top_p=0.9, seed=5)
    w16 = W.as_f16(w32)
    assert (w16.logits.view(np.float16) == x).all()
    a, b = O.sample(w32, kept_cap=20), O.sample(w16, kept_cap=20)
    assert (a.tokens == b.tokens).all() and (a.kept_ids == b.kept_ids).all()
    assert (a.logprobs == b.logprobs).all()


def test_exp1_table_brute_force_and_forced_winner():
    # §6.2 (pre-generated random numbers): token = argmax over the kept set of (z - zmax) - ln E[b, t]
    rng = np.random.default_rng(43)
    B, V = 5, 12
    x = (rng.standard_normal((B, V)) * 2).astype(np.float32)
    w = W.with_exp1(one_row(x, T=1.0, top_k=6, seed=1), seed=3)
    o = O.sample(w, kept_cap=V)
    for b in range(B):
        kept = [i for i in o.kept_ids[b].tolist() if i >= 0]
        assert len(kept) == 6
        g = {i: (float(x[b, i]) - float(x[b].max())) - math.log(float(w.exp1[b, i])) for i in kept}
        assert o.tokens[b] == max(kept, key=lambda i: (g[i], -i))
    # an almost-zero E for one kept token makes it win; the same E for a token outside the kept set changes nothing
    for b in range(B):
        kept = [i for i in o.kept_ids[b].tolist() if i >= 0]
        out_id = next(i for i in range(V) if i not in kept)
        w2 = W.with_exp1(one_row(x, T=1.0, top_k=6, seed=1), seed=3)
        w2.exp1[b, kept[-1]] = np.float32(1e-30)
        assert O.sample(w2).tokens[b] == kept[-1]
        w3 = W.with_exp1(one_row(x, T=1.0, top_k=6, seed=1), seed=3)
        w3.exp1[b, out_id] = np.float32(1e-30)
        assert O.sample(w3).tokens[b] == o.tokens[b]


def test_exp1_table_of_the_philox_variates_reproduces_the_counter_based_draw():
    rng = np.random.default_rng(47)
    B, V = 8, 64
    x = (rng.standard_normal((B, V)) * 2).astype(np.float32)
    w = one_row(x, T=0.9, top_p=0.95, seed=np.arange(B, dtype=np.uint64) + 100, step=3, row_base=5)
    ref = O.sample(w)
    tab = np.empty((B, V), dtype=np.float32)
    for b in range(B):
        for t in range(V):
            tab[b, t] = O.exp1_from_word(O.race_word(100 + b, 5 + b, 3, t))
    w.exp1 = tab
    got = O.sample(w)
    sure = ref.rows["race_gap"] > 1e-5          # fp32 rounding of E moves ln E by < 1e-7
    assert sure.sum() >= B - 1
    assert (got.tokens[sure] == ref.tokens[sure]).all()
    assert np.allclose(got.logprobs[sure], ref.logprobs[sure], atol=0, rtol=0)


def test_exp1_table_draw_frequencies():
    # P(token t) = p_t for independent Exp(1) variates (the exponential race), checked by chi-square
    V, N = 4, 4000
    x = np.log(np.array([0.4, 0.3, 0.2, 0.1], dtype=np.float64)).astype(np.float32)
    w = W.with_exp1(one_row(np.tile(x, (N, 1)), T=1.0), seed=99)
    tok = O.sample(w).tokens
    obs = np.bincount(tok, minlength=V)
    p = np.exp(x.astype(np.float64)); p /= p.sum()
    assert scipy.stats.chisquare(obs, p * N).pvalue > 1e-4


# ------------------------------------------------------------------ prompt / output split of the history

def test_split_history_elementwise_and_limits():
    """Repetition looks at prompt and output, presence and frequency at the output alone; each step
    one IEEE fp32 operation, recomputed here from the two parts' own tallies."""
    rng = np.random.default_rng(51)
    V = 400
    x = (rng.standard_normal(V) * 3).astype(np.float32)
    hist = rng.integers(-2, V + 2, size=600)
    r, p, f, T = np.float32(1.25), np.float32(0.6), np.float32(0.2), np.float32(0.8)
    inv_T = np.float32(1.0) / T
    valid = lambda h: h[(h >= 0) & (h < V)]
    for start in (0, 1, 250, 599, 600):
        z = O.row_scores(x, W.F32, T=float(T), r=float(r), p=float(p), f=float(f), history=hist, output_start=start)
        c_any = np.bincount(valid(hist), minlength=V)
        c_out = np.bincount(valid(hist[start:]), minlength=V)
        assert start != 250 or ((c_any > 0) & (c_out == 0)).sum() >= 5            # prompt-only tokens exist
        for i in range(V):
            a = x[i]
            if c_any[i] > 0:
                a = a / r if a > 0 else a * r
                a = a - f * np.float32(c_out[i])
                if c_out[i] > 0:
                    a = a - p
            assert np.float32(a * inv_T) == z[i], (start, i)
    # limits: everything output == no split; everything prompt == repetition penalty alone
    z_all_out = O.row_scores(x, W.F32, T=float(T), r=float(r), p=float(p), f=float(f), history=hist, output_start=0)
    z_plain = O.row_scores(x, W.F32, T=float(T), r=float(r), p=float(p), f=float(f), history=hist)
    assert (z_all_out.view(np.uint32) == z_plain.view(np.uint32)).all()
    z_all_prompt = O.row_scores(x, W.F32, T=float(T), r=float(r), p=float(p), f=float(f), history=hist, output_start=600)
    z_rep_only = O.row_scores(x, W.F32, T=float(T), r=float(r), p=0.0, f=0.0, history=hist)
    assert (z_all_prompt.view(np.uint32) == z_rep_only.view(np.uint32)).all()


def test_split_history_through_the_batch_entry():
    w = W.with_split_history(W.random_small(53, B=12, V=300, dtype=W.F32))
    assert w.output_start is not None and (w.output_start >= 0).all()
    got = O.sample(w, kept_cap=8)
    # the same rows one by one, each with its own split handed to the single-row score routine
    for b in range(w.B):
        o = w.history_offsets
        z = O.row_scores(w.logits[b], W.F32, T=float(w.temperature[b]) if w.temperature[b] > 0 else 1.0,
                         r=float(w.repetition_penalty[b]), p=float(w.presence_penalty[b]),
                         f=float(w.frequency_penalty[b]), history=w.history_ids[o[b]:o[b + 1]],
                         output_start=int(w.output_start[b]))
        assert got.kept_ids[b][0] == int(np.lexsort((np.arange(w.V), -z.astype(np.float64)))[0])
    # and the split matters: some row's token or logprob differs from the unsplit run
    w0 = W.random_small(53, B=12, V=300, dtype=W.F32)
    base = O.sample(w0)
    assert (base.tokens != got.tokens).any() or (base.logprobs != got.logprobs).any()


# ------------------------------------------------------------------ top-k that keeps ties

def test_topk_keep_ties_equals_masking_below_the_kth_value():
    """Keep-ties top-k is what masking every logit below the k-th largest value gives (brute force
    with numpy on quantised rows), and equals the strict top-k whenever the k-th value is unique."""
    rng = np.random.default_rng(61)
    for V in (7, 40, 300):
        for trial in range(5):
            x = (np.round(rng.standard_normal(V) * 1.5) * 0.5).astype(np.float32)      # many exact ties
            x = x + np.float32(0.0)                 # no -0.0: the order puts it below +0.0, numpy's >= does not
            for k in (1, 2, 3, V // 2, V - 1):
                if k < 1:
                    continue
                w = one_row(x, T=1.0, top_k=k)
                w.topk_keep_ties = True
                o = O.sample(w, topk_cap=V, kept_cap=V)
                kth = np.sort(x)[::-1][k - 1]
                want = sorted(np.nonzero(x >= kth)[0].tolist())
                got = sorted(i for i in o.topk_ids[0].tolist() if i >= 0)
                assert got == want and o.rows["n_topk"][0] == len(want)
                # the distribution over the kept set is the softmax of the masked row
                masked = np.where(x >= kth, x.astype(np.float64), -np.inf)
                lp = masked - scipy.special.logsumexp(masked)
                assert abs(o.logprobs[0] - lp[o.tokens[0]]) < 1e-12
                strict = O.sample(one_row(x, T=1.0, top_k=k), topk_cap=V)
                if (x >= kth).sum() == k:          # no tie reaches beyond the k-th place: same set as the strict cut
                    assert (strict.topk_ids == o.topk_ids).all() and strict.tokens[0] == o.tokens[0]
                else:
                    assert strict.rows["n_topk"][0] == k < o.rows["n_topk"][0]


def test_topk_keep_ties_leaves_greedy_and_other_cuts_alone():
    x = np.array([[2.0, 2.0, 1.0, 2.0, 0.5, 1.0]], dtype=np.float32)
    g = one_row(x, T=0.0, top_k=2); g.topk_keep_ties = True
    assert O.sample(g).tokens[0] == 0 and O.sample(g).rows["n_keep"][0] == 1       # greedy: lowest id of the maxima
    w = one_row(x, T=1.0, top_k=2, top_p=0.5); w.topk_keep_ties = True
    o = O.sample(w, kept_cap=6)
    assert o.rows["n_topk"][0] == 3                                                 # the three 2.0s
    assert [i for i in o.kept_ids[0] if i >= 0] == [0, 1]                           # top-p on their mass: 1/3 + 1/3 >= 0.5


# ------------------------------------------------------------------ log-probabilities relative to the full vocabulary

def test_full_vocabulary_logprobs_equal_library_log_softmax_whatever_the_cuts():
    rng = np.random.default_rng(67)
    B, V = 10, 500
    x = (rng.standard_normal((B, V)) * 2.5).astype(np.float32)
    x[3, ::7] = -np.inf                                     # masked entries carry no mass
    T = np.float32(0.8)
    ref = scipy.special.log_softmax((x * (np.float32(1.0) / T)).astype(np.float64), axis=1)
    base = O.sample(one_row(x, T=float(T), top_k=3, top_p=0.9, min_p=0.02, seed=4, num_top=6))
    w = one_row(x, T=float(T), top_k=3, top_p=0.9, min_p=0.02, seed=4, num_top=6)
    w.logprob_full_vocab = True
    o = O.sample(w)
    assert (o.tokens == base.tokens).all() and (o.rows["n_keep"] == base.rows["n_keep"]).all()   # the draw is untouched
    for b in range(B):
        assert abs(o.logprobs[b] - ref[b, o.tokens[b]]) < 1e-12
        # the list is the head of the whole row's order, whatever the cuts kept
        zb = (x[b] * (np.float32(1.0) / T)).astype(np.float64)
        want = np.lexsort((np.arange(V), -zb))[:6]
        assert o.top_ids[b].tolist() == want.tolist()
        for j in range(6):
            assert abs(o.top_logprobs[b, j] - ref[b, o.top_ids[b, j]]) < 1e-12
        assert o.logprobs[b] <= base.logprobs[b] + 1e-15      # the kept set's normaliser is the smaller one
    # greedy rows: the arg max under the softmax of the unscaled scores
    g = one_row(x, T=0.0)
    g.logprob_full_vocab = True
    og = O.sample(g)
    ref0 = scipy.special.log_softmax(x.astype(np.float64), axis=1)
    for b in range(B):
        assert og.tokens[b] == int(np.argmax(x[b])) and abs(og.logprobs[b] - ref0[b, og.tokens[b]]) < 1e-12


# ------------------------------------------------------------------ race ties, out-of-contract parameters, band enumeration

def test_race_tie_goes_to_the_lowest_id():
    # equal scores and equal variates give equal race scores g: the lowest id of the tied best wins,
    # wherever the tied ids sit in the sorted order and whatever id carries the (lower) rest
    V = 40
    x = np.full((3, V), -3.0, dtype=np.float32)
    tied = [[7, 19, 33], [0, 39], [38, 5, 21, 6]]
    for b, ids in enumerate(tied):
        x[b, ids] = 2.0
    w = one_row(x, T=1.0, seed=9)
    E = np.full((3, V), 0.75, dtype=np.float32)
    w.exp1 = E.copy()
    o = O.sample(w)
    assert o.tokens.tolist() == [min(t) for t in tied]
    assert (o.rows["race_gap"] == 0.0).all()
    # equal g from unequal parts: z lower by ln 2 exactly where E is halved (z = k ln 2 is not exact in fp32,
    # so build it the other way round: E' = E * exp(z' - z) in fp64, rounded once -- the tie is then only
    # near, and the winner is whichever g is larger, computed here from the same fp32 inputs)
    x2 = np.full((1, V), -30.0, dtype=np.float32)
    x2[0, [4, 9]] = [1.0, 0.5]
    w2 = one_row(x2, T=1.0, seed=9)
    E2 = np.full((1, V), 0.5, dtype=np.float32)
    E2[0, 9] = np.float32(0.5 * math.exp(-0.5))
    w2.exp1 = E2
    g4 = (1.0 - 1.0) - math.log(float(E2[0, 4]))
    g9 = (0.5 - 1.0) - math.log(float(E2[0, 9]))
    want = 4 if (g4 > g9 or (g4 == g9)) else 9
    assert O.sample(w2).tokens[0] == want
    # the tie rule does not depend on the cut that built the kept set
    w3 = one_row(x, T=1.0, top_k=2, seed=9)
    w3.exp1 = E.copy()
    assert O.sample(w3).tokens.tolist() == [7, 0, 5]


def test_negative_and_nan_temperature_mean_greedy():
    # T <= 0 is greedy; the same reading covers a negative and a NaN temperature (anything not > 0)
    rng = np.random.default_rng(71)
    x = (rng.standard_normal((6, 500)) * 3).astype(np.float32)
    x[2, [17, 300]] = x[2].max() + 1.0                      # a tie at the top: lowest id
    ref = O.sample(one_row(x, T=0.0, top_k=40, top_p=0.5, min_p=0.2, seed=3))
    for T in (-1.0, -np.inf, np.nan, -0.0):
        o = O.sample(one_row(x, T=T, top_k=40, top_p=0.5, min_p=0.2, seed=3))
        assert (o.rows["greedy"] == 1).all()
        assert o.tokens.tolist() == [int(np.argmax(r)) for r in x] == ref.tokens.tolist()
        assert (o.logprobs == 0.0).all() and (o.rows["n_keep"] == 1).all()
    assert ref.tokens[2] == 17


def test_nonpositive_repetition_penalty_is_plain_arithmetic():
    # r <= 0 is outside the method's contract; the definition is applied as written (x / r for x > 0,
    # x * r otherwise), one fp32 rounding per operation, so that both implementations agree on such rows
    rng = np.random.default_rng(72)
    V = 64
    x = (rng.standard_normal(V) * 3).astype(np.float32)
    hist = [3, 3, 10, 40, 63]
    for r in (-1.5, -0.25):
        z = O.row_scores(x, W.F32, T=1.0, r=r, history=hist)
        want = x.copy()
        for t in set(hist):
            want[t] = np.float32(x[t] / np.float32(r)) if x[t] > 0 else np.float32(x[t] * np.float32(r))
        assert (z.view(np.uint32) == want.view(np.uint32)).all()
        w = one_row(x[None], T=1.0, r=r, history=hist, top_k=5, seed=2)
        o = O.sample(w, kept_cap=5)
        order = np.lexsort((np.arange(V), -want.astype(np.float64)))
        assert o.kept_ids[0].tolist() == order[:5].tolist()


def test_shifted_cut_parameters_equal_changed_parameters():
    # the oracle's "same row, cut parameter moved" entry against the plain entry with the moved parameter
    # itself, for moves that are exact in fp32 (top_p 0.75 -> 0.5 and 0.25 -> 0.5; min_p 0.125 -> 0.25)
    rng = np.random.default_rng(73)
    x = (rng.standard_normal((8, 300)) * 2).astype(np.float32)
    for p0, dp in ((0.75, -0.25), (0.25, 0.25)):
        a = one_row(x, T=1.0, top_p=p0, seed=4)
        b = O.sample(one_row(x, T=1.0, top_p=p0 + dp, seed=4))
        for i in range(8):
            r, _, _, _ = O.row_shifted(a, i, 0.0, dp)
            assert (r["token"], r["n_keep"]) == (b.tokens[i], b.rows["n_keep"][i])
            assert r["logprob"] == b.logprobs[i]
    a = one_row(x, T=1.0, min_p=0.125, seed=4)
    b = O.sample(one_row(x, T=1.0, min_p=0.25, seed=4))
    for i in range(8):
        r, _, _, _ = O.row_shifted(a, i, math.log(2.0), 0.0)
        assert (r["token"], r["n_keep"]) == (b.tokens[i], b.rows["n_keep"][i])
    assert (b.rows["n_keep"] < O.sample(a).rows["n_keep"]).any()        # (the move does change the cut)


def test_band_enumeration_contains_every_shifted_result():
    # acceptable() enumerates the kept-prefix lengths reachable inside the bands with numpy; every result of
    # the C entry with the parameters moved to the ends (and the middle) of the bands must be among them,
    # in the ordinary and in the full-vocabulary log-probability mode
    rng = np.random.default_rng(74)
    x = np.round(rng.standard_normal((6, 400)) * 2, 1).astype(np.float32)        # many exact ties
    x[0] = 0.0                                                                    # flat row: cut on a boundary
    for full in (False, True):
        for kw in (dict(top_p=0.5), dict(min_p=float(np.exp(np.float32(-1.0)))), dict(top_p=0.9, min_p=0.05, top_k=50)):
            w = one_row(x, T=1.0, seed=6, **kw)
            w.logprob_full_vocab = full
            for b in range(6):
                acc = O.acceptable(w, b)
                prim, _, _, _ = O.row_shifted(w, b, 0.0, 0.0)
                assert (acc[0][0], acc[0][2]) == (prim["token"], prim["n_keep"]) and acc[0][1] == prim["logprob"]
                for s7 in (-O.LN_MIN_P_BAND, 0.0, O.LN_MIN_P_BAND):
                    for s8 in (-O.TOP_P_BAND, 0.0, O.TOP_P_BAND):
                        r, _, _, _ = O.row_shifted(w, b, s7 * 0.999, s8 * 0.999)
                        assert any(t == r["token"] and n == r["n_keep"] and abs(lp - r["logprob"]) < 1e-12
                                   for (t, lp, n) in acc), (full, kw, b, s7, s8)
    # full-vocabulary mode: the enumerated log-probabilities are relative to the whole row
    w = one_row(x, T=1.0, seed=6, top_p=0.5)
    w.logprob_full_vocab = True
    ls = scipy.special.log_softmax(x.astype(np.float64), axis=1)
    for b in range(6):
        for (t, lp, _) in O.acceptable(w, b):
            assert abs(lp - ls[b, t]) < 1e-12


def test_race_near_tie_band_is_relative():
    # two survivors whose race scores differ by 3e-5 at |g| ~ 20: inside the relative band (1e-5 * 20),
    # so the runner-up is acceptable; the same gap at |g| ~ 1 is outside it
    def two(z1, e0, e1):
        x = np.full((1, 8), -200.0, dtype=np.float32)
        x[0, 0], x[0, 1] = 0.0, z1
        w = one_row(x, T=1.0, top_k=2, seed=1)
        E = np.ones((1, 8), dtype=np.float32)
        E[0, 0], E[0, 1] = e0, e1
        w.exp1 = E
        return w
    w = two(0.0, math.exp(-20.0), math.exp(-20.0 + 3e-5))
    gap = O.sample(w).rows["race_gap"][0]
    assert 1e-5 < gap < 1e-4
    assert {a[0] for a in O.acceptable(w, 0)} == {0, 1}
    w = two(0.0, math.exp(-1.0), math.exp(-1.0 + 3e-5))
    assert 1e-5 < O.sample(w).rows["race_gap"][0] < 1e-4
    assert {a[0] for a in O.acceptable(w, 0)} == {0}
