"""Test-side helpers: tiny tree models, exhaustive enumeration of Algorithm 1's outcome law and
an independent single-draft GBV.  Everything here is written from the definitions with numpy and
plain Python; the only things taken from the oracle are the quantities under test."""
from __future__ import annotations

import itertools

import numpy as np


def np_softmax(z, T=1.0):
    s = np.asarray(z, dtype=np.float64) / T
    e = np.exp(s - s.max())
    return e / e.sum()


class TreeModel:
    """Every token prefix of length i <= gamma has its own target row; every prefix of length
    i < gamma has its own draft row.  Rows are float32 logits; probabilities are their softmax."""

    def __init__(self, V, gamma, seed, T=1.0, scale=1.5, corr=0.6):
        self.V, self.gamma, self.T = V, gamma, T
        rng = np.random.default_rng(seed)
        self.zq, self.zp = {}, {}
        for i in range(gamma + 1):
            for pre in itertools.product(range(V), repeat=i):
                zq = (scale * rng.standard_normal(V)).astype(np.float32)
                self.zq[pre] = zq
                if i < gamma:
                    zp = corr * zq + np.sqrt(1 - corr * corr) * scale * rng.standard_normal(V)
                    self.zp[pre] = zp.astype(np.float32)

    def q(self, pre):
        return np_softmax(self.zq[tuple(pre)], self.T)

    def p(self, pre):
        return np_softmax(self.zp[tuple(pre)], self.T)

    def joint(self, seq):
        """(q(seq), p(seq)) joint probabilities of a token sequence (len <= gamma)."""
        a = b = 1.0
        for i, t in enumerate(seq):
            a *= self.q(seq[:i])[t]
            b *= self.p(seq[:i])[t]
        return a, b

    def verify_inputs(self, drafts):
        """Arrays for one batch row holding the given K drafts (tuples of gamma tokens)."""
        K, g, V = len(drafts), self.gamma, self.V
        zq = np.zeros((1, K, g + 1, V), np.float32)
        zp = np.zeros((1, K, g, V), np.float32)
        tok = np.zeros((1, K, g), np.int32)
        for k, d in enumerate(drafts):
            tok[0, k] = d
            for i in range(g + 1):
                zq[0, k, i] = self.zq[tuple(d[:i])]
                if i < g:
                    zp[0, k, i] = self.zp[tuple(d[:i])]
        return zq, zp, tok


def py_scan_outcomes(bits, tok):
    """Algorithm 1's scan driven by Bernoulli outcomes instead of uniforms.
    bits[k][i-1] = 1 if the trial on sub-block (k,i) succeeds. Returns (tau, f)."""
    K, g = len(tok), len(tok[0])
    tau, f, H = 0, -1, set()
    for k in range(K):
        start = tau + 1
        stop = False
        for i in range(start, g + 1):
            blk = tuple(int(t) for t in tok[k][:i])
            if bits[k][i - 1] and blk not in H:
                tau, f = i, k
                if i == g:
                    stop = True
                    break
            else:
                H.add(blk)
        if stop:
            break
    return tau, f


def scan_law(h, tok):
    """Exact law of (tau, f) given the acceptance weights h[K][gamma] and the drafts:
    sum over all 2^(K*gamma) Bernoulli outcome vectors."""
    K, g = len(tok), len(tok[0])
    law = {}
    hv = np.asarray(h, dtype=np.float64).reshape(K, g)
    for flat in itertools.product((0, 1), repeat=K * g):
        bits = [flat[k * g:(k + 1) * g] for k in range(K)]
        pr = 1.0
        for k in range(K):
            for j in range(g):
                pr *= hv[k, j] if bits[k][j] else (1.0 - hv[k, j])
        if pr == 0.0:
            continue
        key = py_scan_outcomes(bits, tok)
        law[key] = law.get(key, 0.0) + pr
    return law


def gbv_single_draft(q_rows, p_rows, tok, eta, u_s):
    """Independent single-draft greedy block verification, written from its definition:
    nu_i = nu_{i-1} q(x_i|x^{i-1})/p(x_i|x^{i-1}), nu_0 = 1;
    alpha(x^i) = sum_x max(nu_i q(x|x^i) - p(x|x^i), 0) / sum_x max(p(x|x^i) - nu_i q(x|x^i), 0)
    for i < L, alpha(x^L) = nu_L; each sub-block is tested with its own uniform, the longest
    accepted one wins; the extra token comes from norm(max(nu_tau q - p, 0)) or from q after a
    full accept.  Probabilities above 1 mean "accept".
    q_rows: gamma+1 arrays, p_rows: gamma arrays. Returns (alpha[gamma], tau, y)."""
    g = len(tok)
    nu = [1.0]
    for i in range(g):
        nu.append(nu[-1] * q_rows[i][tok[i]] / p_rows[i][tok[i]])
    alpha = []
    for i in range(1, g):
        up = np.maximum(nu[i] * q_rows[i] - p_rows[i], 0.0).sum()
        dn = np.maximum(p_rows[i] - nu[i] * q_rows[i], 0.0).sum()
        alpha.append(1.0 if dn <= 0 else min(1.0, up / dn))
    alpha.append(min(1.0, nu[g]))
    tau = 0
    for i in range(1, g + 1):
        if eta[i - 1] < alpha[i - 1]:
            tau = i
    if tau < g:
        w = np.maximum(nu[tau] * q_rows[tau] - p_rows[tau], 0.0)
    else:
        w = q_rows[g]
    cum = np.cumsum(w)
    y = int(np.searchsorted(cum, u_s * cum[-1], side="right"))
    return np.array(alpha), tau, min(y, len(w) - 1)


def chi_square(counts, probs, min_expected=5.0):
    """Pearson chi-square of observed counts against exact cell probabilities, merging cells
    whose expectation is below min_expected. Returns (statistic, degrees of freedom)."""
    n = sum(counts.values())
    cells = sorted(probs.items(), key=lambda kv: kv[1])
    stat, dof, acc_e, acc_o = 0.0, 0, 0.0, 0.0
    for key, pr in cells:
        acc_e += pr * n
        acc_o += counts.get(key, 0)
        if acc_e >= min_expected:
            stat += (acc_o - acc_e) ** 2 / acc_e
            dof += 1
            acc_e = acc_o = 0.0
    if acc_e > 0:
        stat += (acc_o - acc_e) ** 2 / max(acc_e, 1e-300) if acc_e >= 1.0 else 0.0
        dof += 1 if acc_e >= 1.0 else 0
    unseen = [k for k in counts if k not in probs]
    assert not unseen, f"observed outcomes with zero exact probability: {unseen[:5]}"
    return stat, max(dof - 1, 1)
