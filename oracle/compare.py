"""Parity rules between a verify implementation and the oracle (test infrastructure only).

Rules (stated once, used by the GPU tests, the smoke check and the benchmark's parity summary):
  * accept length, draft index and emitted tokens must be bit-exact, except for batch rows where
    a uniform lies within ``margin`` (1e-6) of a decision threshold of the oracle -- an
    acceptance weight, or a CDF edge of the cell the extra token was drawn from; those rows are
    counted and reported, not compared;
  * acceptance weights h and residual masses S must agree within ``rtol`` (1e-5) relative, plus
    an absolute floor that is negligible against the 2^-24 granularity of the uniforms they are
    compared with (h) or against the prefix probability a_i that scales them (S).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np


@dataclass
class ParityReport:
    rows: int = 0
    rows_compared: int = 0
    threshold_exceptions: int = 0     # rows excused by the |u - threshold| < margin rule
    exceptions_matching: int = 0      # excused rows that agree anyway
    decision_mismatches: int = 0      # rows outside the exception rule that differ
    status_mismatches: int = 0
    h_max_rel: float = 0.0
    h_violations: int = 0
    S_max_rel: float = 0.0
    S_violations: int = 0
    block_efficiency_ref: float = 0.0
    block_efficiency_got: float = 0.0
    degenerate_rows: int = 0
    detail: list = field(default_factory=list)

    @property
    def ok(self) -> bool:
        return (self.decision_mismatches == 0 and self.status_mismatches == 0
                and self.h_violations == 0 and self.S_violations == 0)

    def summary(self) -> dict:
        d = {k: v for k, v in self.__dict__.items() if k != "detail"}
        d["ok"] = self.ok
        return d


def compare(ref, tau, f, tokens, h=None, S=None, status=None, margin: float = 1e-6,
            rtol: float = 1e-5, h_atol: float = 1e-9, S_atol_rel_a: float = 1e-9) -> ParityReport:
    """ref: oracle.VerifyResult; the rest: numpy arrays from the implementation under test."""
    rep = ParityReport()
    tau, f, tokens = np.asarray(tau), np.asarray(f), np.asarray(tokens)
    B = ref.tau.shape[0]
    rep.rows = B
    valid = (ref.status & 3) == 0
    excused = valid & ((ref.margin_accept < margin) | (ref.margin_sample < margin))
    rep.threshold_exceptions = int(excused.sum())
    check = ~excused
    rep.rows_compared = int(check.sum())
    same = (tau == ref.tau) & (f == ref.f) & (tokens == ref.tokens).all(axis=1)
    bad = check & ~same
    rep.exceptions_matching = int((excused & same).sum())
    rep.decision_mismatches = int(bad.sum())
    for b in np.nonzero(bad)[0][:8]:
        rep.detail.append(("decision", int(b), int(ref.tau[b]), int(tau[b]), int(ref.f[b]), int(f[b]),
                           ref.tokens[b].tolist(), tokens[b].tolist(),
                           float(ref.margin_accept[b]), float(ref.margin_sample[b])))
    if status is not None:
        status = np.asarray(status)
        sm = (status != ref.status) & check
        rep.status_mismatches = int(sm.sum())
        for b in np.nonzero(sm)[0][:4]:
            rep.detail.append(("status", int(b), int(ref.status[b]), int(status[b])))
    rep.degenerate_rows = int(((ref.status & 4) != 0).sum())
    if valid.any():
        rep.block_efficiency_ref = float(np.mean(ref.tau[valid] + 1))
        rep.block_efficiency_got = float(np.mean(tau[valid] + 1))
    if h is not None:
        h = np.asarray(h, dtype=np.float64)
        err = np.abs(h[valid] - ref.h[valid])
        tol = rtol * np.abs(ref.h[valid]) + h_atol
        rep.h_violations = int((err > tol).sum())
        nz = np.abs(ref.h[valid]) > h_atol / rtol
        if nz.any():
            rep.h_max_rel = float((err[nz] / np.abs(ref.h[valid][nz])).max())
        for idx in np.argwhere(err > tol)[:6]:
            i = tuple(int(v) for v in idx)
            rep.detail.append(("h", i, float(ref.h[valid][i]), float(h[valid][i])))
    if S is not None:
        S = np.asarray(S, dtype=np.float64)
        a = np.exp(ref.loga[..., :-1])
        err = np.abs(S[valid] - ref.S[valid])
        tol = rtol * np.abs(ref.S[valid]) + S_atol_rel_a * a[valid]
        rep.S_violations = int((err > tol).sum())
        nz = ref.S[valid] > (S_atol_rel_a / rtol) * a[valid]
        if nz.any():
            rep.S_max_rel = float((err[nz] / ref.S[valid][nz]).max())
        for idx in np.argwhere(err > tol)[:6]:
            i = tuple(int(v) for v in idx)
            rep.detail.append(("S", i, float(ref.S[valid][i]), float(S[valid][i]), float(a[valid][i])))
    return rep
