"""ctypes front end of the CPU oracle (``albireo_oracle.c``) -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
module.  It shares no code with the CUDA library; the product never routes through it.

``sample`` gives the primary result of the definition for every row.  ``acceptable``
enumerates, for one row, every (token, logprob) pair the definition yields when the
two real-valued cut parameters are moved inside their backward-error bands
(ln(min_p) by <= 1e-5, top_p by <= 1e-6) and, where the two best race scores are
closer than 1e-5 x max(1, their magnitude), the runner-up token as well.  In the
full-vocabulary log-probability mode every enumerated log-probability is relative to the
whole row, as the primary result's is.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "albireo_oracle.c")
_LIB = os.path.join(_HERE, "libalbireo_oracle.so")

LN_MIN_P_BAND = 1e-5
TOP_P_BAND = 1e-6
RACE_BAND = 1e-5


class RowResult(C.Structure):
    _fields_ = [
        ("token", C.c_int32), ("n_fin", C.c_int32), ("n_topk", C.c_int32), ("n_minp", C.c_int32),
        ("n_keep", C.c_int32), ("greedy", C.c_int32),
        ("logprob", C.c_double), ("z_max", C.c_double), ("S", C.c_double),
        ("race_gap", C.c_double), ("minp_margin", C.c_double), ("topp_margin", C.c_double),
    ]


ROW_DTYPE = np.dtype([
    ("token", np.int32), ("n_fin", np.int32), ("n_topk", np.int32), ("n_minp", np.int32),
    ("n_keep", np.int32), ("greedy", np.int32),
    ("logprob", np.float64), ("z_max", np.float64), ("S", np.float64),
    ("race_gap", np.float64), ("minp_margin", np.float64), ("topp_margin", np.float64),
])
assert ROW_DTYPE.itemsize == C.sizeof(RowResult)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-std=c11", "-shared", "-fPIC",
               "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.albireo_oracle_sample.restype = C.c_int
        _lib.albireo_oracle_row_shifted.restype = C.c_int
        _lib.albireo_oracle_row_scores.restype = C.c_int
        _lib.albireo_oracle_order_key.restype = C.c_uint32
        _lib.albireo_oracle_order_key.argtypes = [C.c_float]
        _lib.albireo_oracle_exp1_from_word.restype = C.c_double
        _lib.albireo_oracle_exp1_from_word.argtypes = [C.c_uint32]
        _lib.albireo_oracle_race_word.restype = C.c_uint32
        _lib.albireo_oracle_race_word.argtypes = [C.c_uint64, C.c_uint32, C.c_uint64, C.c_int32]
    return _lib


def _ptr(a: Optional[np.ndarray], dtype):
    if a is None:
        return None
    assert a.dtype == dtype and a.flags.c_contiguous, (a.dtype, dtype)
    return a.ctypes.data_as(C.c_void_p)


def _common_args(w):
    return [
        _ptr(w.logits, np.float32 if w.dtype == 0 else np.uint16), C.c_int32(w.B), C.c_int32(w.V),
        C.c_int32(w.dtype), C.c_int64(w.V),
        _ptr(w.temperature, np.float32), _ptr(w.top_k, np.int32), _ptr(w.top_p, np.float32),
        _ptr(w.min_p, np.float32), _ptr(w.repetition_penalty, np.float32),
        _ptr(w.presence_penalty, np.float32), _ptr(w.frequency_penalty, np.float32),
        _ptr(w.history_ids, np.int32), _ptr(w.history_offsets, np.int32),
        _ptr(w.seeds, np.uint64), C.c_uint64(w.step), C.c_uint32(w.row_base),
        _ptr(getattr(w, "exp1", None), np.float32),
        _ptr(getattr(w, "output_start", None), np.int32),
        C.c_uint32((2 if getattr(w, "topk_keep_ties", False) else 0) | (4 if getattr(w, "logprob_full_vocab", False) else 0)),
    ]


@dataclass
class OracleOut:
    rows: np.ndarray                    # structured array, ROW_DTYPE, [B]
    topk_ids: Optional[np.ndarray]      # [B, topk_cap] step-6 kept ids in order, -1 padded
    kept_ids: Optional[np.ndarray]      # [B, kept_cap] final kept ids in order, -1 padded
    top_ids: Optional[np.ndarray]       # [B, num_top]
    top_logprobs: Optional[np.ndarray]  # [B, num_top] float64
    threads: int = 1

    @property
    def tokens(self):
        return self.rows["token"]

    @property
    def logprobs(self):
        return self.rows["logprob"]


def sample(w, threads: int = 1, topk_cap: int = 0, kept_cap: int = 0, rows=None) -> OracleOut:
    """Primary result for rows ``rows`` (default all) of workload ``w``.

    ``threads`` > 1 splits the rows over that many host threads (rows are
    independent, section 6.1); the arithmetic per row is unchanged.
    """
    L = lib()
    B = w.B
    out = np.zeros(B, dtype=ROW_DTYPE)
    topk = np.full((B, topk_cap), -1, dtype=np.int32) if topk_cap else None
    kept = np.full((B, kept_cap), -1, dtype=np.int32) if kept_cap else None
    nt = int(w.num_top)
    tids = np.full((B, nt), -1, dtype=np.int32) if nt else None
    tlps = np.full((B, nt), -np.inf, dtype=np.float64) if nt else None
    lo, hi = (0, B) if rows is None else rows
    common = _common_args(w)

    def run(r0, r1):
        rc = L.albireo_oracle_sample(
            *common, C.c_int32(r0), C.c_int32(r1), out.ctypes.data_as(C.c_void_p),
            C.c_int32(topk_cap), _ptr(topk, np.int32), C.c_int32(kept_cap), _ptr(kept, np.int32),
            C.c_int32(nt), _ptr(tids, np.int32), _ptr(tlps, np.float64))
        if rc != 0:
            raise RuntimeError("albireo_oracle_sample failed")

    n = hi - lo
    threads = max(1, min(int(threads), n)) if n > 0 else 1
    if threads == 1:
        if n > 0:
            run(lo, hi)
    else:
        # small contiguous chunks so uneven rows balance
        chunk = max(1, n // (threads * 4))
        spans = [(s, min(s + chunk, hi)) for s in range(lo, hi, chunk)]
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(lambda s: run(*s), spans))
    return OracleOut(out, topk, kept, tids, tlps, threads)


def row_shifted(w, b: int, ln_min_p_shift: float = 0.0, top_p_shift: float = 0.0, want_sorted=False):
    """One row with shifted cut parameters; optionally the full sorted (ids, z, g)."""
    L = lib()
    res = np.zeros(1, dtype=ROW_DTYPE)
    ids = np.empty(w.V, dtype=np.int32) if want_sorted else None
    zs = np.empty(w.V, dtype=np.float32) if want_sorted else None
    gs = np.empty(w.V, dtype=np.float64) if want_sorted else None
    rc = L.albireo_oracle_row_shifted(
        *_common_args(w), C.c_int32(b), C.c_double(ln_min_p_shift), C.c_double(top_p_shift),
        res.ctypes.data_as(C.c_void_p), _ptr(ids, np.int32), _ptr(zs, np.float32), _ptr(gs, np.float64))
    if rc != 0:
        raise RuntimeError("albireo_oracle_row_shifted failed")
    return res[0], ids, zs, gs


def row_scores(logits_row: np.ndarray, dtype: int, T=1.0, r=1.0, p=0.0, f=0.0, history=None, output_start: int = 0) -> np.ndarray:
    """Steps 1-4 (widen, penalties, temperature) of one row; returns z as float32[V]."""
    L = lib()
    V = logits_row.shape[0]
    z = np.empty(V, dtype=np.float32)
    h = None if history is None else np.ascontiguousarray(history, dtype=np.int32)
    rc = L.albireo_oracle_row_scores(
        _ptr(np.ascontiguousarray(logits_row), np.float32 if dtype == 0 else np.uint16),
        C.c_int32(V), C.c_int32(dtype), C.c_float(T), C.c_float(r), C.c_float(p), C.c_float(f),
        _ptr(h, np.int32), C.c_int32(0 if h is None else h.size), C.c_int32(output_start), z.ctypes.data_as(C.c_void_p))
    if rc != 0:
        raise RuntimeError("albireo_oracle_row_scores failed")
    return z


def philox4x32_10(ctr, key):
    L = lib()
    c = (C.c_uint32 * 4)(*[int(x) & 0xFFFFFFFF for x in ctr])
    k = (C.c_uint32 * 2)(*[int(x) & 0xFFFFFFFF for x in key])
    o = (C.c_uint32 * 4)()
    L.albireo_oracle_philox4x32_10(c, k, o)
    return [int(x) for x in o]


def order_key(z: float) -> int:
    return int(lib().albireo_oracle_order_key(C.c_float(z)))


def race_word(seed: int, R: int, step: int, token: int) -> int:
    return int(lib().albireo_oracle_race_word(C.c_uint64(seed), C.c_uint32(R), C.c_uint64(step), C.c_int32(token)))


def exp1_from_word(wd: int) -> float:
    return float(lib().albireo_oracle_exp1_from_word(C.c_uint32(wd)))


def acceptable(w, b: int):
    """All (token, logprob, n_keep) triples acceptable for row ``b``.

    The first entry is the primary result.  The rest come from moving ln(min_p) within
    +-1e-5 and top_p within +-1e-6 (every kept-prefix length reachable inside the
    bands), and from near-ties of the race (gap < 1e-5 x max(1, |score|) between the two best scores).
    """
    prim, ids, zs, gs = row_shifted(w, b, 0.0, 0.0, want_sorted=True)
    out = [(int(prim["token"]), float(prim["logprob"]), int(prim["n_keep"]))]
    if prim["greedy"]:
        return out
    d = zs.astype(np.float64) - float(prim["z_max"])
    L6 = int(prim["n_topk"])
    min_p = float(w.min_p[b]) if w.min_p is not None else 0.0
    top_p = float(w.top_p[b]) if w.top_p is not None else 1.0

    # reachable lengths after the min-p cut
    if min_p > 0.0:
        ln = float(np.log(np.float64(np.float32(min_p))))
        lo, hi = ln - LN_MIN_P_BAND, ln + LN_MIN_P_BAND
        thr = {lo, ln, hi}
        inband = d[:L6][(d[:L6] > lo) & (d[:L6] < hi)]
        for v in inband:
            thr.add(float(v))
            thr.add(float(np.nextafter(v, np.inf)))
        L7s = sorted({max(1, int(np.count_nonzero(d[:L6] >= t))) for t in thr})
    else:
        L7s = [L6]

    # the full-vocabulary mode measures probabilities against every finite score of the row
    full = bool(getattr(w, "logprob_full_vocab", False))
    S_full = float(np.sum(np.exp(d[np.isfinite(d)]))) if full else None

    def near_tie(ga, gb):
        # race scores are differences of O(1..100) terms: the band scales with their size
        return ga - gb < RACE_BAND * max(1.0, abs(ga), abs(gb))

    seen = set()
    for L7 in L7s:
        e = np.exp(d[:L7])
        if top_p < 1.0:
            # sequential running sum in sorted order, as the definition states
            Cs = np.cumsum(e)
            Sp = Cs[-1]
            def first(t):
                if t >= 1.0:
                    return L7
                j = int(np.searchsorted(Cs, t * Sp, side="left"))
                return min(L7, j + 1)
            a, c = first(top_p - TOP_P_BAND), first(top_p + TOP_P_BAND)
            L8s = range(max(1, a), c + 1)
        else:
            L8s = [L7]
        for L8 in L8s:
            if L8 in seen:
                continue
            seen.add(L8)
            g = gs[:L8]
            S = S_full if full else float(np.sum(e[:L8]))
            order = np.lexsort((ids[:L8], -g))       # best g first, ties -> lowest id
            jb = int(order[0])
            out.append((int(ids[jb]), float(d[jb] - np.log(S)), L8))
            if L8 > 1:
                j2 = int(order[1])
                if near_tie(float(g[jb]), float(g[j2])):
                    out.append((int(ids[j2]), float(d[j2] - np.log(S)), L8))
    return out
