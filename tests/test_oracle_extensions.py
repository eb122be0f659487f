"""Pins of the oracle's extensions: one position of Algorithm 2 (distribution modification) and the comparison
verifiers of Section 3 (token-level speculative sampling, SpecTr's K-SEQ).  CPU only.

Algorithm 2 is also pinned by the K = 1 exact-law enumeration of test_oracle_pins.py, whose continuation after
the extra token goes through ``oracle.modify``."""
import itertools

import numpy as np
import pytest

import oracle
from treemodel import TreeModel, np_softmax


# ---- Algorithm 2 -------------------------------------------------------------------------------------------
def test_modify_weights_from_the_definition_and_carried_logs():
    """q_new(x) = norm(q(s,x)(1 - min{p(s,x)/q(s,x), 1})^K) with JOINT probabilities, written out with numpy;
    the drawn token is the inverse CDF of it; the carried logs gain log q(y|s) and log p(y|s)."""
    rng = np.random.default_rng(5)
    B, V, T = 6, 9, 0.8
    zq = (1.3 * rng.standard_normal((B, V))).astype(np.float32)
    zp = (0.7 * zq + rng.standard_normal((B, V))).astype(np.float32)
    loga = -3.0 * rng.random(B)
    logb = loga + rng.normal(0.0, 0.7, B)
    u = rng.random(B).astype(np.float32)
    for K in (1, 2, 5):
        res = oracle.modify(zq, zp, loga, logb, u, K, T, want_qnew=True)
        for b in range(B):
            q, p = np_softmax(zq[b], T), np_softmax(zp[b], T)
            a, bb = np.exp(loga[b]), np.exp(logb[b])
            w = (a * q) * (1.0 - np.minimum((bb * p) / (a * q), 1.0)) ** K
            np.testing.assert_allclose(res.qnew[b], w / w.sum(), rtol=1e-12, atol=1e-15)
            assert res.R[b] == pytest.approx(w.sum() / a, rel=1e-12)
            cum = np.cumsum(w / w.sum())
            y = int(np.searchsorted(cum, float(u[b]), side="right"))
            assert res.token[b] == min(y, V - 1)
            assert res.loga[b] == pytest.approx(loga[b] + np.log(q[res.token[b]]), abs=1e-12)
            assert res.logb[b] == pytest.approx(logb[b] + np.log(p[res.token[b]]), abs=1e-12)
            assert res.status[b] == 0


def test_modify_special_cases():
    """K = 1 is single-draft GBV's modified target norm(max(nu q - p, 0)) with nu = a/b; p == q leaves q
    unchanged when b < a and has no residual mass at all when b >= a (the draw then comes from q, flagged)."""
    rng = np.random.default_rng(6)
    V = 7
    zq = rng.standard_normal((1, V)).astype(np.float32)
    zp = rng.standard_normal((1, V)).astype(np.float32)
    q, p = np_softmax(zq[0]), np_softmax(zp[0])
    la, lb = np.array([-1.2]), np.array([-1.5])
    res = oracle.modify(zq, zp, la, lb, np.array([0.4], np.float32), 1, 1.0, want_qnew=True)
    nu = np.exp(la[0] - lb[0])
    w = np.maximum(nu * q - p, 0.0)
    np.testing.assert_allclose(res.qnew[0], w / w.sum(), rtol=1e-12, atol=1e-15)
    same = oracle.modify(zq, zq, la, lb, np.array([0.4], np.float32), 3, 1.0, want_qnew=True)
    np.testing.assert_allclose(same.qnew[0], q, rtol=1e-12)
    assert same.R[0] == pytest.approx((1.0 - np.exp(lb[0] - la[0])) ** 3, rel=1e-12)
    none = oracle.modify(zq, zq, lb, la, np.array([0.4], np.float32), 3, 1.0, want_qnew=True)
    assert none.status[0] & oracle.STATUS_DEGENERATE_RESIDUAL and none.R[0] == 0.0
    np.testing.assert_allclose(none.qnew[0], q, rtol=1e-12)
    # a long sequence: joint probabilities far below the float64 range change nothing but the carried logs
    far = oracle.modify(zq, zp, la - 2000.0, lb - 2000.0, np.array([0.4], np.float32), 1, 1.0, want_qnew=True)
    np.testing.assert_allclose(far.qnew[0], res.qnew[0], rtol=1e-9)
    assert far.token[0] == res.token[0]


# ---- K-SEQ and token-level speculative sampling --------------------------------------------------------------
def test_kseq_rho_solves_its_equation():
    rng = np.random.default_rng(7)
    for n in (1, 2, 3, 5, 8):
        for _ in range(5):
            q = np_softmax(2.0 * rng.standard_normal(11))
            p = np_softmax(2.0 * rng.standard_normal(11))
            rho = oracle.kseq_rho(q, p, n)
            assert 1.0 <= rho <= n
            beta = np.minimum(p, q / rho).sum()
            assert 1.0 - (1.0 - beta) ** n == pytest.approx(rho * beta, abs=1e-12)
    q = np_softmax(rng.standard_normal(6))
    assert oracle.kseq_rho(q, q, 4) == pytest.approx(1.0, abs=1e-12)   # p == q: every token is accepted


def _token_level_sd(q_rows, p_rows, tok, eta, u_s):
    """Token-level speculative sampling from its definition (Section 3.1)."""
    g = len(tok)
    for i in range(g):
        x = tok[i]
        if not eta[i] < min(1.0, q_rows[i][x] / p_rows[i][x]):
            w = np.maximum(q_rows[i] - p_rows[i], 0.0)
            cum = np.cumsum(w)
            return i, min(int(np.searchsorted(cum, u_s * cum[-1], side="right")), len(w) - 1)
    cum = np.cumsum(q_rows[g])
    return g, min(int(np.searchsorted(cum, u_s * cum[-1], side="right")), len(cum) - 1)


def test_kseq_with_one_draft_is_token_level_speculative_sampling():
    rng = np.random.default_rng(8)
    V, g, T = 12, 4, 0.9
    for _ in range(60):
        zq = (1.5 * rng.standard_normal((1, 1, g + 1, V))).astype(np.float32)
        zp = (0.7 * zq[:, :, :g] + rng.standard_normal((1, 1, g, V))).astype(np.float32)
        q_rows = [np_softmax(zq[0, 0, i], T) for i in range(g + 1)]
        p_rows = [np_softmax(zp[0, 0, i], T) for i in range(g)]
        tok = np.array([[[rng.choice(V, p=p_rows[i]) for i in range(g)]]], np.int32)
        u = rng.random((1, g + 1)).astype(np.float32)
        res = oracle.kseq_verify(zq, zp, tok, u, T)
        tau, y = _token_level_sd(q_rows, p_rows, tok[0, 0], u[0, :g], float(u[0, g]))
        assert res.tau[0] == tau and res.tokens[0, tau] == y
        assert list(res.tokens[0, :tau]) == list(tok[0, 0, :tau]) and (res.tokens[0, tau + 1:] == -1).all()
        assert np.nanmax(np.abs(res.rho[0, :min(tau + 1, g)] - 1.0)) == 0.0


@pytest.mark.parametrize("V,K,seed", [(3, 2, 0), (3, 3, 1), (4, 2, 2), (2, 4, 3)])
def test_kseq_first_token_follows_the_target_law(V, K, seed):
    """K-SEQ is a valid coupling of K i.i.d. draft tokens with the target: over all draft tuples, acceptance
    paths and residual draws the emitted token has law q exactly.  The acceptance probabilities, rho and the
    residual are the oracle's (read back through sgbv_oracle_kseq_verify with chosen uniforms)."""
    tm = TreeModel(V, 1, seed)
    q = tm.q(())
    p = tm.p(())
    law = np.zeros(V)
    for draft in itertools.product(range(V), repeat=K):
        pd = float(np.prod([p[x] for x in draft]))
        zq = np.repeat(tm.zq[()][None, None, None], K, axis=1)            # [1,K,1,V] position-0 rows
        zq = np.concatenate([zq, np.zeros((1, K, 1, V), np.float32)], axis=2)
        zp = np.repeat(tm.zp[()][None, None, None], K, axis=1)
        tok = np.array(draft, np.int32).reshape(1, K, 1)
        # every trial that can fail does (eta = 1 - eps), so that every draft up to the first sure accept is
        # tried and the oracle reports its acceptance probability
        u = np.full((1, K + 1), np.float32(0.9999999), np.float32)
        res = oracle.kseq_verify(zq, zp, tok, u)
        acc, rho = res.acc[0, :, 0], res.rho[0, 0]
        stay = 1.0
        for k in range(K):
            if np.isnan(acc[k]):
                assert stay == 0.0      # only after a token that is accepted with probability 1
                break
            law[draft[k]] += pd * stay * acc[k]
            stay *= 1.0 - acc[k]
        w = np.maximum(q - rho * p, 0.0)
        if stay > 0 and w.sum() > 0:
            law += pd * stay * w / w.sum()
    np.testing.assert_allclose(law, q, atol=1e-9)


def test_kseq_keeps_the_drafts_that_match_and_stops_at_the_first_position_without_an_accept():
    V, K, g = 5, 3, 3
    zq = np.zeros((1, K, g + 1, V), np.float32)      # uniform rows everywhere: q/p = 1, rho = 1, always accept
    zp = np.zeros((1, K, g, V), np.float32)
    tok = np.array([[[1, 2, 3], [1, 4, 0], [2, 2, 2]]], np.int32)
    u = np.full((1, K * g + 1), 0.5, np.float32)
    res = oracle.kseq_verify(zq, zp, tok, u)
    assert res.tau[0] == 3 and list(res.tokens[0, :3]) == [1, 2, 3]
    # position 0: draft 0 accepted, drafts {0,1} retained (draft 2 has another token); draft 2 is never tried later
    assert np.isnan(res.acc[0, 2]).all() and np.isnan(res.acc[0, 1]).all()
    # a target that forbids every draft token at position 1: no accept there, y from the residual
    zq[0, :, 1, :] = np.array([0, -np.inf, -np.inf, 0, -np.inf], np.float32)
    tok[0, :, 1] = [1, 2, 4]
    res = oracle.kseq_verify(zq, zp, tok, u)
    assert res.tau[0] == 1 and res.tokens[0, 0] == 1 and res.tokens[0, 1] in (0, 3) and res.tokens[0, 2] == -1


# ---- Algorithm 3's draft draw -------------------------------------------------------------------------------
def test_draw_tokens_follow_the_softmax_law_on_a_grid_of_uniforms():
    """Inverse CDF: of N equally spaced uniforms exactly the share p(x) (up to one grid point per cell edge) maps to
    token x, tokens come out in non-decreasing order, and the reported log-probability is log softmax."""
    rng = np.random.default_rng(11)
    V, N, T = 13, 4000, 0.7
    row = (2.0 * rng.standard_normal(V)).astype(np.float32)
    row[4] = -np.inf
    p = np_softmax(row, T)
    u = ((np.arange(N) + 0.5) / N).astype(np.float32)
    tok, lp, _ = oracle.draw_tokens(np.repeat(row[None], N, 0), u, T)
    assert (np.diff(tok) >= 0).all() and (tok != 4).all()
    counts = np.bincount(tok, minlength=V)
    assert np.abs(counts - p * N).max() <= 1.0 + 1e-6
    np.testing.assert_allclose(lp, np.log(p[tok]), atol=1e-12)
    bad = row.copy()
    bad[2] = np.nan
    assert oracle.draw_tokens(bad[None], u[:1], T)[0][0] == -1
