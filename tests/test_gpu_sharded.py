"""GPU parity of the vocabulary-sharded verify step: every rank's phases run in lockstep on one device (no kernel
waits for another rank; the exchanges are a stack and a maximum), and the result must be what the oracle gets on the
whole vocabulary: sharding the logits must not change Algorithm 1's outcome."""
import numpy as np
import pytest
import torch

import oracle
from oracle.compare import compare
from paper_2604_25925_b200 import binding, sharded, workloads
from test_gpu_parity import assert_parity, _to_np32

pytestmark = pytest.mark.gpu


def split(inp, bounds):
    return [(inp.target_logits[..., lo:hi].contiguous(), inp.draft_logits[..., lo:hi].contiguous(), lo)
            for lo, hi in bounds]


def run_sharded(inp, bounds):
    cfg = inp.cfg
    outs = sharded.verify_all_ranks_on_one_device(split(inp, bounds), inp.draft_tokens, inp.uniforms,
                                                  cfg.temperature, cfg.V)
    torch.cuda.synchronize()
    first = outs[0]
    for o in outs[1:]:   # every rank reaches the same decisions, bit for bit
        for name in ("accept_len", "draft_idx", "tokens", "status"):
            assert torch.equal(getattr(o, name), getattr(first, name)), name
        assert torch.equal(o.h.nan_to_num(-7.0), first.h.nan_to_num(-7.0))
        assert torch.equal(o.resmass.nan_to_num(-7.0), first.resmass.nan_to_num(-7.0))
    ref = oracle.verify(_to_np32(inp.target_logits), _to_np32(inp.draft_logits), inp.draft_tokens.cpu().numpy(),
                        inp.uniforms.cpu().numpy(), cfg.temperature)
    rep = compare(ref, first.accept_len.cpu().numpy(), first.draft_idx.cpu().numpy(), first.tokens.cpu().numpy(),
                  first.h.cpu().numpy(), first.resmass.cpu().numpy(), first.status.cpu().numpy())
    print(cfg.name, len(bounds), rep.summary())
    for d in rep.detail:
        print("   ", d)
    return rep, first, ref


@pytest.mark.parametrize("n_ranks", [1, 2, 4, 8])
def test_config2_sharded_over_equal_ranges(n_ranks):
    inp = workloads.make_inputs(workloads.CONFIGS["c2"], device="cuda")
    rep, out, _ = run_sharded(inp, sharded.shard_bounds(inp.cfg.V, n_ranks))
    assert_parity(rep)
    # and the one-device path on the same inputs decides alike wherever the oracle's margins are not razor thin
    one = binding.sgbv_verify_ex(inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms, inp.cfg.temperature)
    assert (one.accept_len == out.accept_len).float().mean() >= 0.75
    np.testing.assert_allclose(out.h.cpu().numpy(), one.h.cpu().numpy(), rtol=3e-5, atol=1e-9)


def test_bf16_shards_of_a_large_vocabulary():
    cfg = workloads.with_batch(workloads.CONFIGS["c3"], 6)
    inp = workloads.make_inputs(cfg, device="cuda")
    rep, _, _ = run_sharded(inp, sharded.shard_bounds(cfg.V, 4))
    assert_parity(rep)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_ragged_ranges_with_odd_starts(dtype):
    """Ranges of very different sizes whose starts are not multiples of anything (the shards' rows are then not
    16-byte aligned), one of them a single entry, one shorter than a cell."""
    cfg = workloads.VerifyConfig(f"ragged_{dtype}", B=5, K=3, gamma=4, V=3001, dtype=dtype, temperature=0.8, alpha=0.85,
                                 boost=4.0, seed=99)
    inp = workloads.make_inputs(cfg, device="cuda")
    bounds = [(0, 1), (1, 778), (778, 781), (781, 2999), (2999, 3001)]
    rep, _, _ = run_sharded(inp, bounds)
    assert_parity(rep)


def test_paper_operating_point_sharded():
    cfg = workloads.with_batch(workloads.CONFIGS["paper_l12"], 3)
    inp = workloads.make_inputs(cfg, device="cuda")
    rep, _, _ = run_sharded(inp, sharded.shard_bounds(cfg.V, 8))
    assert_parity(rep)


def test_many_trials_on_a_tiny_vocabulary():
    """20,000 fresh uniforms on fixed logits over 16 entries split in three: every accept length, every owner rank
    and the fall-backs of the split inverse CDF are hit."""
    cfg = workloads.CONFIGS["c1"]
    inp = workloads.make_inputs(cfg).to("cuda")
    n = 20000
    big = workloads.VerifyInputs(
        workloads.with_batch(cfg, n),
        inp.target_logits.expand(n, -1, -1, -1).contiguous(), inp.draft_logits.expand(n, -1, -1, -1).contiguous(),
        inp.draft_tokens.expand(n, -1, -1).contiguous(),
        workloads.make_uniforms(n, cfg.K, cfg.gamma, seed=cfg.seed + 5, device="cuda"))
    rep, out, ref = run_sharded(big, [(0, 5), (5, 6), (6, 16)])
    assert_parity(rep)
    assert abs(rep.block_efficiency_got - rep.block_efficiency_ref) < 1e-3


def test_degenerate_and_flagged_rows_sharded():
    cfg = workloads.VerifyConfig("flags_sharded", B=7, K=2, gamma=2, V=300, alpha=0.8, seed=7)
    inp = workloads.make_inputs(cfg, device="cuda")
    zq, zp = inp.target_logits.clone(), inp.draft_logits.clone()
    tok, u = inp.draft_tokens.clone(), inp.uniforms.clone()
    zp[1] = zq[1, :, :2]                 # row 1: p == q everywhere -> zero residual mass, draw from q across shards
    u[1, :4] = 0.999
    tok[2, 1, 0] = 300                   # row 2: token out of range
    zq[3, 0, 1, 17] = float("nan")       # row 3: NaN logit (in the first shard only)
    zp[4, 1, 0, 205] = float("inf")      # row 4: +inf logit (in the last shard only)
    zq[5, :, :, 11] = float("-inf")      # row 5: -inf is allowed (probability 0)
    zp[5, :, :, 12] = float("-inf")
    zq[6, :, :, 100:200] = float("-inf")  # row 6: a whole shard carries no target mass
    mod = workloads.VerifyInputs(cfg, zq, zp, tok, u)
    rep, out, ref = run_sharded(mod, [(0, 100), (100, 200), (200, 300)])
    assert_parity(rep)
    st = out.status.cpu().numpy()
    assert st[1] & binding.STATUS_DEGENERATE_RESIDUAL
    assert st[2] & binding.STATUS_TOKEN_RANGE and st[3] & binding.STATUS_NONFINITE_LOGIT
    assert st[4] & binding.STATUS_NONFINITE_LOGIT and st[0] == 0 and (st[5] & 3) == 0 and (st[6] & 3) == 0
    assert (out.tokens[2:5].cpu().numpy() == -1).all() and (out.accept_len[2:5].cpu().numpy() == -1).all()
    y6 = int(out.tokens[6, int(out.accept_len[6])])
    assert 0 <= y6 < 300 and not (100 <= y6 < 200)


def test_argument_checks():
    cfg = workloads.VerifyConfig("args", B=2, K=2, gamma=2, V=512, seed=3)
    inp = workloads.make_inputs(cfg, device="cuda")
    (zq, zp, _), = split(inp, [(0, 512)])
    with pytest.raises(binding.SgbvError):   # the range does not fit the vocabulary
        binding.sgbv_shard_stats(zq, zp, inp.draft_tokens, 8, 512, 1.0)
    with pytest.raises(binding.SgbvError):   # temperature
        binding.sgbv_shard_stats(zq, zp, inp.draft_tokens, 0, 512, 0.0)
    stats = binding.sgbv_shard_stats(zq, zp, inp.draft_tokens, 0, 512, 1.0).unsqueeze(0).contiguous()
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.SgbvError) as e:
        binding.sgbv_shard_sums(zq, zp, 1.0, stats, small)
    assert "workspace" in str(e.value).lower()
    assert binding.sgbv_shard_workspace_bytes(2, 2, 2, 512) > 0


def test_one_rank_over_nccl_runs_the_real_exchanges():
    """The collectives of ``sharded.verify`` (two all-gathers, one max-all-reduce) on the device through NCCL, with a
    process group of one rank that holds the whole vocabulary: the only multi-rank plumbing one GPU can exercise."""
    import socket
    import torch.distributed as dist
    if dist.is_initialized():
        pytest.skip("a process group is already up in this process")
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1,
                            device_id=torch.device("cuda", torch.cuda.current_device()))
    try:
        cfg = workloads.VerifyConfig("nccl1", B=6, K=3, gamma=4, V=4096, temperature=0.7, alpha=0.85, seed=21)
        inp = workloads.make_inputs(cfg, device="cuda")
        out = sharded.verify(inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms, cfg.temperature, 0,
                             cfg.V, sharded.TorchExchange())
        torch.cuda.synchronize()
    finally:
        dist.destroy_process_group()
    ref = oracle.verify(_to_np32(inp.target_logits), _to_np32(inp.draft_logits), inp.draft_tokens.cpu().numpy(),
                        inp.uniforms.cpu().numpy(), cfg.temperature)
    rep = compare(ref, out.accept_len.cpu().numpy(), out.draft_idx.cpu().numpy(), out.tokens.cpu().numpy(),
                  out.h.cpu().numpy(), out.resmass.cpu().numpy(), out.status.cpu().numpy())
    assert_parity(rep)


@pytest.mark.parametrize("B,K,gamma,V,n_ranks", [(2, 64, 64, 768, 3), (1, 1, 1, 40, 2), (3, 5, 7, 1000, 64), (2, 2, 3, 70000, 2)])
def test_edge_shapes_sharded(B, K, gamma, V, n_ranks):
    """The largest draft count and length the interface takes, the smallest problem, as many ranks as it allows (most of
    them with a handful of entries), and shards longer than the fused kernel's CTA slice."""
    cfg = workloads.VerifyConfig(f"edge_sharded_{B}_{K}_{gamma}_{V}", B=B, K=K, gamma=gamma, V=V, temperature=0.9, alpha=0.8,
                                 boost=4.0, seed=77 + V)
    inp = workloads.make_inputs(cfg, device="cuda")
    bounds = sharded.shard_bounds(V, n_ranks)
    bounds = [(lo, hi) for lo, hi in bounds if hi > lo]   # (ranks whose range would be empty hold nothing: left out)
    rep, _, _ = run_sharded(inp, bounds)
    assert_parity(rep)
