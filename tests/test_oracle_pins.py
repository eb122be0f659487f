"""Pins of the float64 oracle against what the paper and the mathematics fix (CPU only).

Each test names the passage it rests on.  None of them compares the oracle with itself: the
other side is a hand-derived value, a closed form, an exhaustive enumeration written here from
the definitions, or an independently written single-draft algorithm.
"""
import itertools
import os

import numpy as np
import pytest

import oracle
from treemodel import TreeModel, gbv_single_draft, np_softmax, py_scan_outcomes, scan_law

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _logits_of(prob):
    return np.log(np.asarray(prob, dtype=np.float64)).astype(np.float32)


# --------------------------------------------------------------------------------------------
# Hand-derived worked example (Algorithm 1 + Eqs. 3, 4 on V=2, gamma=1, K=2).
# --------------------------------------------------------------------------------------------
def _read_golden(name):
    vals = {}
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            line = line.split("#")[0].strip()
            if line:
                k, v = line.split("=")
                num, _, den = v.partition("/")
                vals[k.strip()] = float(num) / float(den) if den else float(num)
    return vals


def test_two_token_example_weights_and_law():
    gold = _read_golden("two_token_example.txt")
    p = np.array([0.5, 0.5])
    q = np.array([0.6, 0.4])
    K = 2
    # Eq. 3 weights of the two possible one-token blocks
    assert oracle.h_full(q[0], p[0], K) == pytest.approx(gold["h_token0"], abs=1e-14)
    assert oracle.h_full(q[1], p[1], K) == pytest.approx(gold["h_token1"], abs=1e-14)
    # Eq. 4 residual of the empty prefix: all mass on token 0
    S, w = oracle.resmass(q, p, 1.0, 1.0, K)
    assert S == pytest.approx(gold["residual_mass"], abs=1e-15)
    assert w[1] == 0.0
    # law of the first output token and E[tau], enumerating the 4 draft pairs through the
    # oracle's own scan with uniforms placed inside each outcome cell
    zq = np.tile(_logits_of(q), (1, K, 2, 1)).astype(np.float32)
    zp = np.tile(_logits_of(p), (1, K, 1, 1)).astype(np.float32)
    p_first0, e_tau = 0.0, 0.0
    for d0, d1 in itertools.product(range(2), repeat=2):
        tok = np.array([[[d0], [d1]]], np.int32)
        res0 = oracle.verify(zq, zp, tok, np.array([[0.0, 0.0, 0.5]], np.float32))
        h = res0.h[0, :, 0]
        for bits in itertools.product((0, 1), repeat=2):
            pr = np.prod([h[k] if bits[k] else 1 - h[k] for k in range(2)])
            eta = [0.5 * h[k] if bits[k] else 0.5 * (1 + h[k]) for k in range(2)]
            res = oracle.verify(zq, zp, tok, np.array([eta + [0.5]], np.float32))
            first = res.tokens[0, 0]
            p_first0 += 0.25 * pr * (first == 0)
            e_tau += 0.25 * pr * res.tau[0]
    assert p_first0 == pytest.approx(gold["p_first_token0"], abs=1e-7)
    assert e_tau == pytest.approx(gold["expected_tau"], abs=1e-7)


# --------------------------------------------------------------------------------------------
# K = 1, gamma = 1: token-level speculative sampling (accept min{1,q/p}, residual max(q-p,0)).
# --------------------------------------------------------------------------------------------
def test_k1_gamma1_is_token_level_speculative_sampling():
    rng = np.random.default_rng(3)
    for _ in range(20):
        V = 7
        q = rng.dirichlet(np.ones(V))
        p = rng.dirichlet(np.ones(V))
        for x in range(V):
            assert oracle.h_full(q[x], p[x], 1) == pytest.approx(min(1.0, q[x] / p[x]), rel=1e-13)
        S, w = oracle.resmass(q, p, 1.0, 1.0, 1)
        ref = np.maximum(q - p, 0.0)
        np.testing.assert_allclose(w, ref, atol=1e-15)
        assert S == pytest.approx(ref.sum(), rel=1e-13)


# --------------------------------------------------------------------------------------------
# K = 1: equality with an independently written single-draft GBV on the same uniforms.
# --------------------------------------------------------------------------------------------
@pytest.mark.parametrize("seed", range(6))
def test_k1_equals_single_draft_gbv(seed):
    rng = np.random.default_rng(100 + seed)
    V, g, T = 11, 4, 0.8
    tm = TreeModel(V, 1, seed)  # only used for its softmax convention
    del tm
    for trial in range(40):
        zq = (1.5 * rng.standard_normal((1, 1, g + 1, V))).astype(np.float32)
        zp = (0.7 * zq[:, :, :g] + 1.0 * rng.standard_normal((1, 1, g, V))).astype(np.float32)
        p_rows = [np_softmax(zp[0, 0, i], T) for i in range(g)]
        q_rows = [np_softmax(zq[0, 0, i], T) for i in range(g + 1)]
        tok = np.array([[[rng.choice(V, p=p_rows[i]) for i in range(g)]]], np.int32)
        u = rng.random((1, g + 1)).astype(np.float32)
        res = oracle.verify(zq, zp, tok, u, temperature=T)
        alpha, tau, y = gbv_single_draft(q_rows, p_rows, tok[0, 0], u[0, :g], float(u[0, g]))
        np.testing.assert_allclose(res.h[0, 0], alpha, rtol=1e-9, atol=1e-12)
        assert res.tau[0] == tau
        assert res.tokens[0, tau] == y
        assert list(res.tokens[0, :tau]) == list(tok[0, 0, :tau])
        assert res.f[0] == (0 if tau > 0 else -1)


# --------------------------------------------------------------------------------------------
# K = 1: the output law is exactly q (Theorem 4.2) and E[tau] = sum min{p,q} (Remark 5.2),
# by exhaustive enumeration over drafts, Bernoulli paths, residual draws and the distribution
# modification of Algorithm 2 for the tokens after y.
# --------------------------------------------------------------------------------------------
def _modified_next(tm, seq, K):
    """Algorithm 2: law of the token after `seq` when it lies in the modified region -- taken from the oracle's
    own Algorithm 2 (sgbv_oracle_modify) with the carried joint log-probabilities of `seq`, so that the
    enumeration below pins that function too."""
    a, b = tm.joint(seq)
    res = oracle.modify(tm.zq[tuple(seq)][None], tm.zp[tuple(seq)][None], np.array([np.log(a)]),
                        np.array([np.log(b)]), np.array([0.5], np.float32), K, tm.T, want_qnew=True)
    return res.qnew[0]


@pytest.mark.parametrize("V,g,seed", [(3, 2, 0), (3, 3, 1), (4, 2, 2), (2, 3, 3)])
def test_k1_output_law_is_target_law(V, g, seed):
    tm = TreeModel(V, g, seed, T=1.0)
    law = {}          # first g output tokens -> probability
    e_tau = 0.0
    lemma = {}        # (accepted block) -> P(tau >= i, block)   (Lemma A.1 at K = 1)
    for draft in itertools.product(range(V), repeat=g):
        _, pd = tm.joint(draft)
        zq, zp, tok = tm.verify_inputs([draft])
        res = oracle.verify(zq, zp, tok, np.zeros((1, g + 1), np.float32))
        for (tau, f), pr in scan_law(res.h[0], tok[0]).items():
            e_tau += pd * pr * tau
            for i in range(1, tau + 1):
                lemma[draft[:i]] = lemma.get(draft[:i], 0.0) + pd * pr
            if tau == g:
                law[draft] = law.get(draft, 0.0) + pd * pr
                continue
            a, b = tm.joint(draft[:tau])
            S, w = oracle.resmass(tm.q(draft[:tau]), tm.p(draft[:tau]), a, b, 1)
            assert S == pytest.approx(res.S[0, 0, tau], rel=1e-9)
            # continuation: y from the residual, later tokens from Algorithm 2's q_new
            stack = [(draft[:tau] + (y,), pd * pr * w[y] / S) for y in range(V) if w[y] > 0]
            while stack:
                seq, prs = stack.pop()
                if len(seq) == g:
                    law[seq] = law.get(seq, 0.0) + prs
                    continue
                nxt = _modified_next(tm, seq, 1)
                stack.extend((seq + (x,), prs * nxt[x]) for x in range(V) if nxt[x] > 0)
    for seq in itertools.product(range(V), repeat=g):
        a, _ = tm.joint(seq)
        assert law.get(seq, 0.0) == pytest.approx(a, abs=1e-12), seq
    bound = 0.0
    for i in range(1, g + 1):
        for seq in itertools.product(range(V), repeat=i):
            a, b = tm.joint(seq)
            bound += min(a, b)
            assert lemma.get(seq, 0.0) == pytest.approx(min(a, b), abs=1e-12)
    assert e_tau == pytest.approx(bound, abs=1e-12)


# --------------------------------------------------------------------------------------------
# Lemma A.1's backward recursion, which Eq. 2 is solved from: with G(x^i) = q(x^i) g(min{p/q,1}),
#   sum_x G(x^i,x) + (g(p(x^i)) - sum_x G(x^i,x)) h = G(x^i)      and      h_L g(p(x^L)) = G(x^L).
# G is evaluated here element by element from its definition.
# --------------------------------------------------------------------------------------------
@pytest.mark.parametrize("K", [1, 2, 3, 5, 8])
def test_weights_satisfy_lemma_recursion(K):
    rng = np.random.default_rng(7 + K)
    checked = 0
    for _ in range(200):
        V = int(rng.integers(2, 9))
        q = rng.dirichlet(np.ones(V) * rng.uniform(0.2, 2))
        p = rng.dirichlet(np.ones(V) * rng.uniform(0.2, 2))
        a = rng.uniform(0.01, 1.0)
        b = min(1.0, a * np.exp(rng.normal(0, 1.5)))
        G = lambda aa, bb: aa * (1 - (1 - min(bb / aa, 1.0)) ** K)  # noqa: E731
        sumG = sum(G(a * q[x], b * p[x]) for x in range(V))
        S, _ = oracle.resmass(q, p, a, b, K)
        assert S == pytest.approx(a - sumG, abs=1e-13)
        h = oracle.h_sub(a, b, S, K)
        has = 1 - (1 - b) ** K
        if 1e-9 < h < 1 - 1e-9:   # away from the clamp the recursion must close exactly
            assert sumG + (has - sumG) * h == pytest.approx(G(a, b), rel=1e-9)
            checked += 1
        hL = oracle.h_full(a, b, K)
        assert hL * has == pytest.approx(G(a, b), rel=1e-10)
        assert 0.0 <= h <= 1.0 and 0.0 <= hL <= 1.0 and -1e-15 <= S <= a + 1e-15
    assert checked > 50


# --------------------------------------------------------------------------------------------
# Closed forms of the residual mass on special rows.
# --------------------------------------------------------------------------------------------
@pytest.mark.parametrize("K", [1, 2, 4, 8])
def test_residual_mass_closed_forms(K):
    rng = np.random.default_rng(K)
    V = 13
    q = rng.dirichlet(np.ones(V))
    for c in (0.0, 0.3, 1.0, 2.5):
        a = 0.37
        b = a * c
        # identical rows: every ratio equals c
        S, w = oracle.resmass(q, q, a, b, K)
        assert S == pytest.approx(a * max(1 - c, 0.0) ** K, abs=1e-14)
        np.testing.assert_allclose(w, a * q * max(1 - c, 0.0) ** K, atol=1e-15)
        # uniform target, one-hot draft on token 3: only token 3 is reduced
        onehot = np.zeros(V)
        onehot[3] = 1.0
        uq = np.full(V, 1.0 / V)
        S, _ = oracle.resmass(uq, onehot, a, b, K)
        assert S == pytest.approx(a * ((V - 1) / V + (1 / V) * max(1 - c * V, 0.0) ** K), abs=1e-14)
    # K = 1: S = a - sum_x min(a q, b p)
    p = rng.dirichlet(np.ones(V))
    S, _ = oracle.resmass(q, p, 0.4, 0.3, 1)
    assert S == pytest.approx(0.4 - np.minimum(0.4 * q, 0.3 * p).sum(), abs=1e-14)
    # zero target probability contributes nothing, whatever the draft puts there
    q0 = q.copy()
    q0[5] = 0.0
    S, w = oracle.resmass(q0, p, 1.0, 1.0, K)
    assert w[5] == 0.0 and np.isfinite(S)


def test_softmax_invariances():
    rng = np.random.default_rng(11)
    z = (2.0 * rng.standard_normal(50)).astype(np.float32)
    prob, lse = oracle.softmax(z, 0.7)
    np.testing.assert_allclose(prob, np_softmax(z, 0.7), rtol=1e-13)
    assert prob.sum() == pytest.approx(1.0, abs=1e-14)
    assert lse == pytest.approx(np.log(np.exp(z.astype(np.float64) / 0.7).sum()), rel=1e-13)
    # temperature = pre-divided logits (exactly representable division by 0.5)
    prob2, _ = oracle.softmax((z * 2).astype(np.float32), 1.0)
    prob3, _ = oracle.softmax(z, 0.5)
    np.testing.assert_allclose(prob2, prob3, rtol=1e-14)
    # shift invariance (power-of-two shift keeps float32 inputs exact enough)
    prob4, lse4 = oracle.softmax(z + np.float32(8.0), 0.7)
    np.testing.assert_allclose(prob4, np_softmax(z + np.float32(8.0), 0.7), rtol=1e-13)
    # -inf logits are allowed and get probability 0
    z2 = z.copy()
    z2[4] = -np.inf
    prob5, _ = oracle.softmax(z2, 1.0)
    assert prob5[4] == 0.0 and prob5.sum() == pytest.approx(1.0, abs=1e-14)


# --------------------------------------------------------------------------------------------
# gamma = 1: the per-position K-draft problem.  Whole-block trials only; weight and residual
# follow Eq. 3 / Eq. 4 with single-token probabilities.
# --------------------------------------------------------------------------------------------
@pytest.mark.parametrize("K", [2, 3, 5])
def test_gamma1_is_per_position_multi_draft(K):
    rng = np.random.default_rng(20 + K)
    V = 9
    zq = (1.2 * rng.standard_normal((1, K, 2, V))).astype(np.float32)
    zq[0, :, 0] = zq[0, 0, 0]
    zp = (1.2 * rng.standard_normal((1, K, 1, V))).astype(np.float32)
    zp[0, :, 0] = zp[0, 0, 0]
    q, p = np_softmax(zq[0, 0, 0]), np_softmax(zp[0, 0, 0])
    tok = rng.choice(V, size=(1, K, 1), p=p).astype(np.int32)
    u = rng.random((1, K + 1)).astype(np.float32)
    res = oracle.verify(zq, zp, tok, u)
    for k in range(K):
        x = tok[0, k, 0]
        expect = q[x] * (1 - (1 - min(p[x] / q[x], 1.0)) ** K) / (1 - (1 - p[x]) ** K)
        assert res.h[0, k, 0] == pytest.approx(min(expect, 1.0), rel=1e-12)
    # first accepted distinct token in draft order wins
    tau, f = 0, -1
    seen = set()
    for k in range(K):
        x = int(tok[0, k, 0])
        if u[0, k] < res.h[0, k, 0] and x not in seen:
            tau, f = 1, k
            break
        seen.add(x)
    assert (res.tau[0], res.f[0]) == (tau, f)
    if tau == 0:
        w = q * (1 - np.minimum(p / q, 1.0)) ** K
        cum = np.cumsum(w)
        assert res.tokens[0, 0] == int(np.searchsorted(cum, float(u[0, K]) * cum[-1], side="right"))


# --------------------------------------------------------------------------------------------
# Scan semantics: two independently written scans (C with uniforms, Python with outcome bits).
# --------------------------------------------------------------------------------------------
def test_scan_matches_python_scan_on_random_cases():
    rng = np.random.default_rng(5)
    for _ in range(3000):
        K, g = int(rng.integers(1, 5)), int(rng.integers(1, 5))
        tok = rng.integers(0, 2, size=(K, g)).astype(np.int32)   # tiny alphabet: many duplicates
        h = rng.random((K, g))
        h[rng.random((K, g)) < 0.15] = 1.0
        h[rng.random((K, g)) < 0.15] = 0.0
        eta = rng.random((K, g)).astype(np.float32)
        bits = [[int(eta[k, j] < h[k, j]) for j in range(g)] for k in range(K)]
        assert oracle.scan(h, tok, eta) == py_scan_outcomes(bits, tok)


def test_scan_documented_cases():
    # a later draft replaces the accepted block wholesale; only the length carries over
    tok = np.array([[1, 2, 3], [4, 5, 6]], np.int32)
    h = np.array([[1.0, 0.0, 0.0], [0.0, 1.0, 0.0]])
    eta = np.full((2, 3), 0.5, np.float32)
    assert oracle.scan(h, tok, eta) == (2, 1)
    # whole-block accept stops the scan: draft 1 is never looked at
    h = np.array([[0.0, 0.0, 1.0], [1.0, 1.0, 1.0]])
    assert oracle.scan(h, tok, eta) == (3, 0)
    # a duplicate of a rejected sub-block is skipped even when its own trial would pass
    tok = np.array([[1, 2, 3], [1, 2, 9]], np.int32)
    h = np.array([[0.0, 0.0, 0.0], [1.0, 1.0, 0.0]])
    assert oracle.scan(h, tok, eta) == (0, -1)
    # strict inequality: eta == h rejects; h = 1 always accepts; h = 0 never
    tok = np.array([[7]], np.int32)
    assert oracle.scan(np.array([[0.5]]), tok, np.array([[0.5]], np.float32)) == (0, -1)
    assert oracle.scan(np.array([[1.0]]), tok, np.array([[0.99999994]], np.float32)) == (1, 0)
    assert oracle.scan(np.array([[0.0]]), tok, np.array([[0.0]], np.float32)) == (0, -1)


def test_sample_inverse_cdf():
    w = np.array([0.0, 2.0, 0.0, 1.0, 1.0, 0.0])
    assert oracle.sample(w, 0.0)[0] == 1
    assert oracle.sample(w, 0.4999)[0] == 1
    assert oracle.sample(w, 0.5)[0] == 3          # cumulative 2 is not > 2
    assert oracle.sample(w, 0.74)[0] == 3
    assert oracle.sample(w, 0.75)[0] == 4
    assert oracle.sample(w, 0.99999)[0] == 4
    assert oracle.sample(np.zeros(4), 0.3)[0] == -1
    y, margin = oracle.sample(w, 0.6)
    assert y == 3 and margin == pytest.approx(0.1)


def test_degenerate_residual_and_status_flags():
    rng = np.random.default_rng(9)
    V, K, g = 6, 2, 2
    zq = (rng.standard_normal((1, K, g + 1, V))).astype(np.float32)
    zq[0, :, 0] = zq[0, 0, 0]
    zp = zq[:, :, :g].copy()                       # p == q everywhere: zero residual mass
    tok = rng.integers(0, V, size=(1, K, g)).astype(np.int32)
    u = np.array([[0.99, 0.99, 0.99, 0.99, 0.3]], np.float32)
    res = oracle.verify(zq, zp, tok, u)
    # joint ratio is 1 everywhere, so a whole-block weight is q(x)g(1)/g(p(x)) = a/g(a) <= 1 and
    # with eta = 0.99 nothing is accepted here
    assert res.tau[0] == 0 and res.f[0] == -1
    assert res.status[0] & oracle.STATUS_DEGENERATE_RESIDUAL
    q = np_softmax(zq[0, 0, 0])
    assert res.tokens[0, 0] == int(np.searchsorted(np.cumsum(q), 0.3 * np.cumsum(q)[-1], side="right"))
    bad_tok = tok.copy()
    bad_tok[0, 1, 0] = V
    assert oracle.verify(zq, zp, bad_tok, u).status[0] & oracle.STATUS_TOKEN_RANGE
    bad = zq.copy()
    bad[0, 0, 1, 2] = np.nan
    r = oracle.verify(bad, zp, tok, u)
    assert r.status[0] & oracle.STATUS_NONFINITE and r.tau[0] == -1 and (r.tokens[0] == -1).all()
