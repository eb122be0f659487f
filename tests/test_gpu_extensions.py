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
