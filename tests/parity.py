"""Comparison of the CUDA path with the CPU oracle, shared by the GPU tests.

Rules (tolerances written out here, nowhere else):
  * greedy rows: token bit-exact, logprob exactly 0 (within the logprob tolerance in the
    full-vocabulary mode, where it is not 0 by definition);
  * top-k stage: the number of ids kept is equal in every row, and for rows with an
    active top-k (1 <= k < V, or greedy) the id set is bit-exact wherever it fits the
    debug capacity;
  * logprob: |gpu - oracle| <= LOGPROB_TOL (absolute) against the primary result; the output is an
    fp32, whose spacing exceeds that once |logprob| passes about 170 (probabilities below e^-170,
    met only in top-N lists at tiny temperatures), so two fp32 spacings of the value are allowed on top
    where that spacing is above 1e-6 (|logprob| >= 16); below that the bound is the plain 2e-5;
  * token: identical to the primary result, except *excused* rows: the GPU's
    (token, logprob) matches one of the results the definition gives when ln(min_p) moves
    by <= 1e-5, top_p by <= 1e-6, or the two best race scores are closer than 1e-5 x max(1, |score|).
    Excused rows are counted; unexcused mismatches must be zero.
The final kept-set size is diagnostic only (it is ill-conditioned for diffuse rows).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from oracle import albireo_oracle as O

LOGPROB_TOL = 2e-5
# the fp32 output's own spacing is added to the tolerance only where it is no longer negligible
# beside LOGPROB_TOL (|logprob| >= 16: spacing 1.9e-6); ordinary values get the plain 2e-5
FP32_SPACING_FLOOR = 1e-6


def logprob_tol(ref):
    """Allowed |gpu - oracle| for a log-probability whose oracle value is ``ref``."""
    sp = np.spacing(np.abs(np.asarray(ref, dtype=np.float64)).astype(np.float32)).astype(np.float64)
    return LOGPROB_TOL + np.where(sp > FP32_SPACING_FLOOR, 2.0 * sp, 0.0)


EXCUSED_FRACTION = 1e-3


@dataclass
class ParityReport:
    name: str
    rows: int = 0
    token_match: int = 0
    excused: list = field(default_factory=list)
    failures: list = field(default_factory=list)
    max_dlogprob: float = 0.0
    kept_size_diff_rows: int = 0
    general_rows: int = 0

    def ok(self) -> bool:
        return not self.failures

    def summary(self) -> str:
        return (f"{self.name}: rows={self.rows} token_match={self.token_match} excused={len(self.excused)} "
                f"failures={len(self.failures)} max|dlogprob|={self.max_dlogprob:.3g} "
                f"kept_size_diff_rows={self.kept_size_diff_rows} general_path_rows={self.general_rows}")


def compare(w, gpu, oracle_out, dbg_cap: int = 0, name: str = "") -> ParityReport:
    """gpu: SampleOutputs already moved to host numpy via ``to_host``; oracle_out: OracleOut."""
    rep = ParityReport(name or w.name, rows=w.B)
    rows = oracle_out.rows
    for b in range(w.B):
        tok, lp = int(gpu["tokens"][b]), float(gpu["logprobs"][b])
        otok, olp = int(rows["token"][b]), float(rows["logprob"][b])
        if not (0 <= tok < w.V):
            rep.failures.append((b, "token out of range", tok))
            continue
        if gpu.get("num_topk") is not None and int(gpu["num_topk"][b]) != int(rows["n_topk"][b]):
            rep.failures.append((b, "top-k stage size", int(gpu["num_topk"][b]), int(rows["n_topk"][b])))
            continue
        k_b = int(w.top_k[b]) if w.top_k is not None else 0
        topk_active = bool(rows["greedy"][b]) or (1 <= k_b < w.V)
        if dbg_cap and topk_active and gpu.get("dbg_topk_ids") is not None and oracle_out.topk_ids is not None \
                and int(rows["n_topk"][b]) <= dbg_cap:
            g = np.sort(gpu["dbg_topk_ids"][b][gpu["dbg_topk_ids"][b] >= 0])
            o = np.sort(oracle_out.topk_ids[b][oracle_out.topk_ids[b] >= 0])
            if g.shape != o.shape or (g != o).any():
                rep.failures.append((b, "top-k membership", g.tolist()[:8], o.tolist()[:8]))
                continue
        if gpu.get("row_status") is not None and int(gpu["row_status"][b]) & 1:
            rep.general_rows += 1
        if gpu.get("num_kept") is not None and int(gpu["num_kept"][b]) != int(rows["n_keep"][b]):
            rep.kept_size_diff_rows += 1
        if rows["greedy"][b]:
            full = getattr(w, "logprob_full_vocab", False)      # then a greedy row's logprob is not 0 by definition
            if tok != otok or (lp != 0.0 if not full else abs(lp - olp) > logprob_tol(olp)):
                rep.failures.append((b, "greedy", tok, otok, lp))
            else:
                rep.token_match += 1
            continue
        if tok == otok and abs(lp - olp) <= logprob_tol(olp):
            rep.token_match += 1
            rep.max_dlogprob = max(rep.max_dlogprob, abs(lp - olp))
            continue
        acc = O.acceptable(w, b)
        if any(tok == t and abs(lp - l) <= logprob_tol(l) for (t, l, _) in acc[1:]):
            rep.excused.append((b, tok, otok, lp, olp))
        else:
            rep.failures.append((b, "token/logprob", tok, otok, lp, olp,
                                 float(rows["race_gap"][b]), float(rows["topp_margin"][b]),
                                 float(rows["minp_margin"][b])))
    return rep


def compare_top_lists(w, gpu, oracle_out) -> list:
    """Top-N lists: same ids in the same order and logprobs within tolerance, for rows whose
    final kept-set size agrees (otherwise the row is a cut-boundary case checked on token+logprob)."""
    bad = []
    if not w.num_top:
        return bad
    for b in range(w.B):
        if gpu.get("num_kept") is not None and int(gpu["num_kept"][b]) != int(oracle_out.rows["n_keep"][b]):
            continue
        gi, oi = gpu["top_ids"][b], oracle_out.top_ids[b]
        if (gi != oi).any():
            bad.append((b, "ids", gi.tolist(), oi.tolist()))
            continue
        m = oi >= 0
        if (np.abs(gpu["top_logprobs"][b][m].astype(np.float64) - oracle_out.top_logprobs[b][m]) > logprob_tol(oracle_out.top_logprobs[b][m])).any():
            bad.append((b, "logprobs"))
        if not np.isneginf(gpu["top_logprobs"][b][~m]).all():
            bad.append((b, "padding"))
    return bad


def to_host(out) -> dict:
    d = {}
    for k in ("tokens", "logprobs", "top_ids", "top_logprobs", "num_kept", "num_topk", "dbg_topk_ids", "row_status"):
        v = getattr(out, k)
        d[k] = None if v is None else v.detach().cpu().numpy()
    return d
