"""Monte-Carlo runs of the oracle against exhaustively enumerated laws, and the properties of
the expected acceptance length (Lemma 5.1, Remark 5.2, Theorem 5.3).  CPU only.

Finding recorded here: Algorithm 1 as printed, run on truly i.i.d. drafts, attains the bound of
Theorem 5.3 and the target law only at K = 1 (the trials of different sub-block values present
in the draft set are independent, not mutually exclusive).  So at K >= 2 the tests assert what
does hold -- Monte-Carlo agrees with the enumerated law of the algorithm itself, Bound(K) is
strictly increasing, E[tau] stays below the bound -- and print the gap.  E[tau] of the printed
algorithm is not even monotone in K in general: with p = q uniform over many tokens, gamma = 1,
K = 1 accepts always while K = 2 accepts each of two (typically distinct) drafts with weight
about 1/2, i.e. with probability about 3/4 overall (asserted below).
"""
import itertools

import numpy as np
import pytest

import oracle
from paper_2604_25925_b200 import workloads
from treemodel import TreeModel, chi_square, np_softmax, scan_law


def _chi2_critical(dof):
    """Upper 1e-4 quantile of chi-square by the Wilson-Hilferty approximation."""
    z = 3.719
    return dof * (1 - 2 / (9 * dof) + z * np.sqrt(2 / (9 * dof))) ** 3


def _exact_law_fixed_drafts(zq, zp, tok, T, K):
    """Exact law of (tau, f, y) given the drafts, for one batch row (small V)."""
    g = tok.shape[1]
    res = oracle.verify(zq[None], zp[None], tok[None], np.zeros((1, K * g + 1), np.float32), T)
    law = {}
    for (tau, f), pr in scan_law(res.h[0], tok).items():
        kk = 0 if tau == 0 else f
        q = np_softmax(zq[kk, tau], T)
        if tau < g:
            p = np_softmax(zp[kk, tau], T)
            a = np.exp(res.loga[0, kk, tau])
            b = np.exp(res.logb[0, kk, tau])
            w = np.array([a * q[x] * (1 - min(b * p[x] / (a * q[x]), 1.0)) ** K for x in range(len(q))])
        else:
            w = q
        w = w / w.sum()
        for y, wy in enumerate(w):
            if wy > 0:
                law[(tau, f, y)] = law.get((tau, f, y), 0.0) + pr * wy
    return law


def test_config1_20000_trials_match_enumerated_law():
    cfg = workloads.CONFIGS["c1"]
    inp = workloads.make_inputs(cfg)
    n = 20000
    zq = inp.target_logits.numpy()[0]
    zp = inp.draft_logits.numpy()[0]
    tok = inp.draft_tokens.numpy()[0]
    law = _exact_law_fixed_drafts(zq, zp, tok, cfg.temperature, cfg.K)
    assert sum(law.values()) == pytest.approx(1.0, abs=1e-12)
    u = workloads.make_uniforms(n, cfg.K, cfg.gamma, seed=cfg.seed + 1).numpy()
    res = oracle.verify(np.broadcast_to(zq, (n,) + zq.shape), np.broadcast_to(zp, (n,) + zp.shape),
                        np.broadcast_to(tok, (n,) + tok.shape), u, cfg.temperature)
    counts = {}
    for t, f, row in zip(res.tau, res.f, res.tokens):
        key = (int(t), int(f), int(row[t]))
        counts[key] = counts.get(key, 0) + 1
    stat, dof = chi_square(counts, law)
    assert stat < _chi2_critical(dof), (stat, dof)
    # accepted tokens are copied from the accepted draft
    for t, f, row in zip(res.tau[:500], res.f[:500], res.tokens[:500]):
        assert list(row[:t]) == list(tok[f, :t]) and (row[t + 1:] == -1).all()
    be = float(np.mean(res.tau + 1))
    exact_be = sum(pr * (k[0] + 1) for k, pr in law.items())
    assert be == pytest.approx(exact_be, abs=4 * np.sqrt(cfg.gamma ** 2 / n))


def _bound(tm, K):
    """Lemma 5.1: sum over sub-block lengths and values of q(x^i) [1 - (1 - min{p/q,1})^K]."""
    tot = 0.0
    for i in range(1, tm.gamma + 1):
        for seq in itertools.product(range(tm.V), repeat=i):
            a, b = tm.joint(seq)
            tot += a * (1 - (1 - min(b / a, 1.0)) ** K)
    return tot


def _exact_expected_tau(tm, K):
    """E[tau] of Algorithm 1 over i.i.d. drafts, by enumerating every K-tuple of drafts and every
    Bernoulli path (weights from the oracle)."""
    g = tm.gamma
    e = 0.0
    first = np.zeros(tm.V)
    blocks = list(itertools.product(range(tm.V), repeat=g))
    for drafts in itertools.product(blocks, repeat=K):
        pd = np.prod([tm.joint(d)[1] for d in drafts])
        zq, zp, tok = tm.verify_inputs(list(drafts))
        res = oracle.verify(zq, zp, tok, np.zeros((1, K * g + 1), np.float32), tm.T)
        for (tau, f), pr in scan_law(res.h[0], tok[0]).items():
            e += pd * pr * tau
            if tau > 0:
                first[drafts[f][0]] += pd * pr
            else:
                _, w = oracle.resmass(tm.q(()), tm.p(()), 1.0, 1.0, K)
                first += pd * pr * (w / w.sum() if w.sum() > 0 else tm.q(()))
    return e, first


@pytest.mark.parametrize("V,g,seed", [(3, 2, 0), (2, 3, 4)])
def test_expected_acceptance_length_vs_bound(V, g, seed):
    tm = TreeModel(V, g, seed, T=1.0)
    bounds = [_bound(tm, K) for K in (1, 2, 3, 4, 64)]
    assert all(b1 < b2 for b1, b2 in zip(bounds, bounds[1:]))          # strictly increasing in K
    assert bounds[-1] <= g and bounds[-1] > 0.98 * g or bounds[-1] > bounds[-2]   # towards gamma
    mins = sum(min(*tm.joint(seq)) for i in range(1, g + 1)
               for seq in itertools.product(range(V), repeat=i))
    assert bounds[0] == pytest.approx(mins, abs=1e-13)                 # Bound(1) = sum min{p,q}
    for K in (1, 2, 3):
        e, first = _exact_expected_tau(tm, K)
        tv = 0.5 * np.abs(first - tm.q(())).sum()
        print(f"V={V} gamma={g} K={K}: E[tau]={e:.6f} Bound={bounds[K-1]:.6f} TV(first,q)={tv:.2e}")
        assert e <= bounds[K - 1] + 1e-12                              # Lemma 5.1 holds
        if K == 1:
            assert e == pytest.approx(bounds[0], abs=1e-12)            # bound attained
            assert tv < 1e-12                                          # first token follows q


def test_monte_carlo_with_redrawn_drafts_matches_enumeration():
    """Drafts are redrawn i.i.d. from the tree model's draft law for every trial; the empirical
    E[tau] and first-token law must match the exhaustive enumeration (K = 1 and K = 2)."""
    V, g = 3, 2
    tm = TreeModel(V, g, 5, T=1.0)
    rng = np.random.default_rng(17)
    n = 20000
    for K in (1, 2):
        e_exact, first_exact = _exact_expected_tau(tm, K)
        zq = np.zeros((n, K, g + 1, V), np.float32)
        zp = np.zeros((n, K, g, V), np.float32)
        tok = np.zeros((n, K, g), np.int32)
        for t in range(n):
            for k in range(K):
                d = ()
                for i in range(g):
                    d += (int(rng.choice(V, p=tm.p(d))),)
                tok[t, k] = d
                for i in range(g + 1):
                    zq[t, k, i] = tm.zq[d[:i]]
                    if i < g:
                        zp[t, k, i] = tm.zp[d[:i]]
        u = rng.random((n, K * g + 1)).astype(np.float32)
        res = oracle.verify(zq, zp, tok, u, 1.0)
        assert float(res.tau.mean()) == pytest.approx(e_exact, abs=4 * g / np.sqrt(n))
        counts = {int(x): int(c) for x, c in zip(*np.unique(res.tokens[:, 0], return_counts=True))}
        stat, dof = chi_square(counts, {x: first_exact[x] for x in range(V)})
        assert stat < _chi2_critical(dof), (K, stat, dof)


def test_block_efficiency_non_decreasing_in_K_on_config_shape():
    """Monte-Carlo block efficiency (mean of tau+1) on the Zipf+Gaussian generator at a reduced
    vocabulary: non-decreasing in K within Monte-Carlo error; K = 1 equals sum min{p,q}-type
    expectation only in law, so here only monotonicity is asserted."""
    be = []
    for K in (1, 2, 4):
        cfg = workloads.VerifyConfig("mono", B=600, K=K, gamma=3, V=64, alpha=0.8, sigma=1.5,
                                     boost=3.0, seed=77)
        inp = workloads.make_inputs(cfg)
        res = oracle.verify(inp.target_logits.numpy(), inp.draft_logits.numpy(),
                            inp.draft_tokens.numpy(), inp.uniforms.numpy(), cfg.temperature)
        assert (res.status & ~oracle.STATUS_DEGENERATE_RESIDUAL == 0).all()
        be.append(float(np.mean(res.tau + 1)))
    print("block efficiency by K:", be)
    err = 3 * 3 / np.sqrt(600)
    assert be[1] >= be[0] - err and be[2] >= be[1] - err


def test_identical_models_k2_accepts_less_than_k1():
    """p = q uniform on V tokens, gamma = 1.  K = 1: weight min{1, q/p} = 1.  K = 2: Eq. 3 gives
    (1/V) / (1 - (1 - 1/V)^2) = V/(2V-1), so two distinct drafts are both rejected with probability
    ((V-1)/(2V-1))^2: the printed algorithm loses acceptance when K grows."""
    V = 50
    z = np.zeros((1, 2, 2, V), np.float32)
    zp = np.zeros((1, 2, 1, V), np.float32)
    tok = np.array([[[3], [7]]], np.int32)
    res = oracle.verify(z, zp, tok, np.array([[0.9, 0.9, 0.5]], np.float32))
    assert res.h[0, 0, 0] == pytest.approx(V / (2 * V - 1), rel=1e-12)
    assert res.tau[0] == 0 and res.status[0] & oracle.STATUS_DEGENERATE_RESIDUAL
    res1 = oracle.verify(z[:, :1], zp[:, :1], tok[:, :1], np.array([[0.9, 0.5]], np.float32))
    assert res1.h[0, 0, 0] == 1.0 and res1.tau[0] == 1
