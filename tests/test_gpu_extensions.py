"""GPU parity of the entry points beyond the verify step: Algorithm 2's draw (``sgbv_modify``) and the
comparison verifiers, against the oracle's functions on the same seeded inputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_25925_b200 import binding, workloads

pytestmark = pytest.mark.gpu


def _position_rows(cfg, device="cuda"):
    """[B,V] target and draft logits of one position: the position-0 rows of a seeded verify input set."""
    inp = workloads.make_inputs(cfg, device=device)
    return inp.target_logits[:, 0, 0].contiguous(), inp.draft_logits[:, 0, 0].contiguous()


@pytest.mark.parametrize("B,K,V,dtype,T", [(5, 3, 4099, "fp32", 0.8), (7, 1, 32000, "fp32", 1.0), (40, 4, 32000, "bf16", 0.7),
                                          (3, 8, 151936, "fp32", 1.0), (2, 2, 17, "fp32", 1.0), (200, 3, 9000, "bf16", 0.4)])
def test_modify_matches_the_oracle(B, K, V, dtype, T):
    cfg = workloads.VerifyConfig("mod", B=B, K=1, gamma=1, V=V, dtype=dtype, temperature=T, alpha=0.8, seed=900 + V % 97)
    zq, zp = _position_rows(cfg)
    g = torch.Generator().manual_seed(B * 131 + K)
    la = (-6.0 * torch.rand(B, generator=g, dtype=torch.float64)).cuda()
    lb = (la.cpu() + 0.8 * torch.randn(B, generator=g, dtype=torch.float64)).cuda()
    la[0], lb[0] = 0.0, 0.0                                    # an empty carried sequence: c = 1
    u = torch.rand(B, generator=g, dtype=torch.float32).cuda()
    out = binding.sgbv_modify(zq, zp, la, lb, u, K, T)
    torch.cuda.synchronize()
    ref = oracle.modify(zq.float().cpu().numpy(), zp.float().cpu().numpy(), la.cpu().numpy(), lb.cpu().numpy(),
                        u.cpu().numpy(), K, T)
    tok, st = out.token.cpu().numpy(), out.status.cpu().numpy()
    R = out.resmass.cpu().numpy()
    np.testing.assert_allclose(R, ref.R, rtol=1e-5, atol=1e-9)
    assert (st == ref.status).all()
    near = ref.margin < 1e-6                                    # draws within 1e-6 of a CDF edge may differ: counted
    assert near.sum() <= max(2, B // 3)
    assert (tok[~near] == ref.token[~near]).all()
    same = tok == ref.token
    np.testing.assert_allclose(out.log_a.cpu().numpy()[same], ref.loga[same], rtol=0, atol=2e-5)
    np.testing.assert_allclose(out.log_b.cpu().numpy()[same], ref.logb[same], rtol=0, atol=2e-5)


def test_modify_flags_and_degenerate_rows():
    cfg = workloads.VerifyConfig("modf", B=4, K=1, gamma=1, V=700, alpha=0.8, seed=77)
    zq, zp = _position_rows(cfg)
    zq, zp = zq.clone(), zp.clone()
    zp[1] = zq[1]                          # p == q and b >= a: no residual mass, the draw comes from q
    zq[2, 5] = float("nan")
    zq[3, 9] = float("-inf")               # allowed
    la = torch.tensor([-1.0, -2.0, -1.0, -1.0], dtype=torch.float64).cuda()
    lb = torch.tensor([-1.5, -1.0, -1.0, -0.5], dtype=torch.float64).cuda()
    u = torch.tensor([0.2, 0.5, 0.5, 0.9], dtype=torch.float32).cuda()
    out = binding.sgbv_modify(zq, zp, la, lb, u, 2, 1.0)
    torch.cuda.synchronize()
    ref = oracle.modify(zq.cpu().numpy(), zp.cpu().numpy(), la.cpu().numpy(), lb.cpu().numpy(), u.cpu().numpy(), 2, 1.0)
    st = out.status.cpu().numpy()
    assert (st == ref.status).all()
    assert st[1] & binding.STATUS_DEGENERATE_RESIDUAL and st[2] & binding.STATUS_NONFINITE_LOGIT
    assert out.token[2].item() == -1 and (out.token.cpu().numpy()[[0, 1, 3]] == ref.token[[0, 1, 3]]).all()


def test_modify_over_several_positions_follows_the_oracle_chain():
    """A few positions in a row, the carried logs fed back (in place), as a decode loop would do."""
    B, V, K, T = 6, 12000, 3, 0.9
    g = torch.Generator().manual_seed(5)
    la = torch.zeros(B, dtype=torch.float64).cuda() - 0.7
    lb = torch.zeros(B, dtype=torch.float64).cuda() - 1.1
    rla, rlb = la.cpu().numpy().copy(), lb.cpu().numpy().copy()
    for pos in range(4):
        cfg = workloads.VerifyConfig("modp", B=B, K=1, gamma=1, V=V, temperature=T, alpha=0.85, seed=300 + pos)
        zq, zp = _position_rows(cfg)
        u = torch.rand(B, generator=g, dtype=torch.float32).cuda()
        out = binding.sgbv_modify(zq, zp, la, lb, u, K, T)
        torch.cuda.synchronize()
        ref = oracle.modify(zq.cpu().numpy(), zp.cpu().numpy(), rla, rlb, u.cpu().numpy(), K, T)
        ok = ref.margin >= 1e-6
        assert (out.token.cpu().numpy()[ok] == ref.token[ok]).all()
        # carry on from the oracle's state where the draws agree (they all do unless a uniform sits on an edge)
        la, lb = out.log_a, out.log_b
        rla, rlb = ref.loga, ref.logb
        np.testing.assert_allclose(la.cpu().numpy()[ok], rla[ok], atol=5e-5)
        la = torch.from_numpy(rla).cuda()
        lb = torch.from_numpy(rlb).cuda()


def _kseq_compare(inp, T):
    out = binding.sgbv_verify_kseq(inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms, T)
    torch.cuda.synchronize()
    ref = oracle.kseq_verify(inp.target_logits.float().cpu().numpy(), inp.draft_logits.float().cpu().numpy(),
                             inp.draft_tokens.cpu().numpy(), inp.uniforms.cpu().numpy(), T)
    tau, tokens, st = out.accept_len.cpu().numpy(), out.tokens.cpu().numpy(), out.status.cpu().numpy()
    rho, acc = out.rho.cpu().numpy(), out.accept_prob.cpu().numpy()
    B = tau.shape[0]
    near = (ref.margin_accept < 1e-6) | (ref.margin_sample < 1e-6)     # a uniform on a threshold: counted, excused
    assert near.sum() <= max(2, B // 3)
    ok = ~near
    assert (st[ok] == ref.status[ok]).all()
    assert (tau[ok] == ref.tau[ok]).all() and (tokens[ok] == ref.tokens[ok]).all()
    # rho and the acceptance probabilities of what both sides tried
    both = ok[:, None] & ~np.isnan(ref.rho) & ~np.isnan(rho)
    np.testing.assert_allclose(rho[both], ref.rho[both], rtol=1e-5)
    assert (np.isnan(rho[ok]) == np.isnan(ref.rho[ok])).all()
    both = ok[:, None, None] & ~np.isnan(ref.acc) & ~np.isnan(acc)
    np.testing.assert_allclose(acc[both], ref.acc[both], rtol=1e-5, atol=1e-9)
    return out, ref


@pytest.mark.parametrize("B,K,gamma,V,dtype,T,alpha", [(6, 3, 4, 4099, "fp32", 0.8, 0.8), (8, 4, 4, 32000, "fp32", 1.0, 0.85),
                                                      (5, 1, 5, 9000, "fp32", 0.9, 0.9), (4, 8, 3, 32000, "bf16", 0.7, 0.7),
                                                      (2, 2, 2, 151936, "fp32", 1.0, 0.9), (3, 5, 2, 17, "fp32", 1.0, 0.5)])
def test_kseq_matches_the_oracle(B, K, gamma, V, dtype, T, alpha):
    cfg = workloads.VerifyConfig("ks", B=B, K=K, gamma=gamma, V=V, dtype=dtype, temperature=T, alpha=alpha, seed=640 + K)
    inp = workloads.make_inputs(cfg, device="cuda")
    _kseq_compare(inp, T)
    assert binding.last_main_kernel() == "kseq_kernel"


def test_kseq_flags():
    cfg = workloads.VerifyConfig("ksf", B=4, K=2, gamma=2, V=300, alpha=0.8, seed=9)
    inp = workloads.make_inputs(cfg, device="cuda")
    zq, tok = inp.target_logits.clone(), inp.draft_tokens.clone()
    tok[1, 0, 1] = 300
    zq[2, :, 0, 17] = float("nan")
    mod = workloads.VerifyInputs(cfg, zq, inp.draft_logits, tok, inp.uniforms)
    out, ref = _kseq_compare(mod, 1.0)
    st = out.status.cpu().numpy()
    assert st[1] & binding.STATUS_TOKEN_RANGE and st[2] & binding.STATUS_NONFINITE_LOGIT and st[0] == 0
    assert (out.accept_len.cpu().numpy()[1:3] == -1).all()


def test_single_draft_entry_points():
    """Token-level speculative sampling = K-SEQ with one draft; single-draft greedy block verification = the block
    verifier with K = 1 (whose parity with an independent GBV is covered by the verify-step tests)."""
    cfg = workloads.VerifyConfig("sd", B=7, K=1, gamma=5, V=12000, temperature=0.8, alpha=0.85, seed=12)
    inp = workloads.make_inputs(cfg, device="cuda")
    zq, zp, tok = inp.target_logits[:, 0].contiguous(), inp.draft_logits[:, 0].contiguous(), inp.draft_tokens[:, 0].contiguous()
    sd = binding.sgbv_verify_token(zq, zp, tok, inp.uniforms, cfg.temperature)
    ks = binding.sgbv_verify_kseq(inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms, cfg.temperature)
    gb = binding.sgbv_verify_gbv(zq, zp, tok, inp.uniforms, cfg.temperature)
    ex = binding.sgbv_verify_ex(inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms, cfg.temperature)
    torch.cuda.synchronize()
    assert torch.equal(sd.accept_len, ks.accept_len) and torch.equal(sd.tokens, ks.tokens)
    assert torch.equal(gb.accept_len, ex.accept_len) and torch.equal(gb.tokens, ex.tokens)
    assert torch.equal(gb.accept_prob[:, 0], ex.h[:, 0])
    ref = oracle.kseq_verify(inp.target_logits.cpu().numpy(), inp.draft_logits.cpu().numpy(), inp.draft_tokens.cpu().numpy(),
                             inp.uniforms.cpu().numpy(), cfg.temperature)
    ok = (ref.margin_accept >= 1e-6) & (ref.margin_sample >= 1e-6)
    assert (sd.accept_len.cpu().numpy()[ok] == ref.tau[ok]).all()


@pytest.mark.parametrize("N,V,dtype,T", [(9, 4099, "fp32", 0.8), (64, 32000, "fp32", 1.0), (33, 128256, "bf16", 0.7),
                                        (3, 17, "fp32", 1.0), (300, 9000, "bf16", 0.4)])
def test_draft_token_draw_matches_the_oracle(N, V, dtype, T):
    cfg = workloads.VerifyConfig("dr", B=N, K=1, gamma=1, V=V, dtype=dtype, temperature=T, alpha=0.8, seed=40 + V % 89)
    _, zp = _position_rows(cfg)
    g = torch.Generator().manual_seed(N)
    u = torch.rand(N, generator=g, dtype=torch.float32).cuda()
    tok, lp, st = binding.sgbv_draw_tokens(zp, u, T)
    torch.cuda.synchronize()
    rtok, rlp, margin = oracle.draw_tokens(zp.float().cpu().numpy(), u.cpu().numpy(), T)
    near = margin < 1e-6
    assert near.sum() <= max(2, N // 3) and (st.cpu().numpy() == 0).all()
    tok = tok.cpu().numpy()
    assert (tok[~near] == rtok[~near]).all()
    same = tok == rtok
    np.testing.assert_allclose(lp.cpu().numpy()[same], rlp[same], atol=2e-5)
    assert binding.last_main_kernel() == "draw_rows_kernel"
    # the draws feed the verify step as draft tokens: in range, and a flagged row for a NaN logit
    assert ((tok >= 0) & (tok < V)).all()
    zbad = zp.clone()
    zbad[0, 3] = float("nan")
    tok2, _, st2 = binding.sgbv_draw_tokens(zbad, u, T)
    assert tok2[0].item() == -1 and st2[0].item() & binding.STATUS_NONFINITE_LOGIT
