"""GPU parity: the CUDA path (through the C ABI) against the float64 oracle on the same seeded
inputs.  Rules are those of ``oracle/compare.py``: decisions bit-exact except rows within 1e-6 of
a threshold (counted), weights and residual masses within 1e-5 relative."""
import numpy as np
import pytest
import torch

import oracle
from oracle.compare import compare
from paper_2604_25925_b200 import binding, workloads
from treemodel import chi_square, gbv_single_draft, np_softmax

pytestmark = pytest.mark.gpu


def _to_np32(t):
    return t.detach().to("cpu", torch.float32).numpy()


def run_both(inp, rows=None, host_inp=None):
    """GPU on the whole batch; oracle on the batch rows `rows` (all if None). Returns the report."""
    cfg = inp.cfg
    out = binding.sgbv_verify_ex(inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms,
                                 cfg.temperature)
    torch.cuda.synchronize()
    sel = slice(None) if rows is None else torch.as_tensor(rows, device=inp.target_logits.device)
    ref = oracle.verify(_to_np32(inp.target_logits[sel]), _to_np32(inp.draft_logits[sel]),
                        inp.draft_tokens[sel].cpu().numpy(), inp.uniforms[sel].cpu().numpy(), cfg.temperature)
    rep = compare(ref, out.accept_len[sel].cpu().numpy(), out.draft_idx[sel].cpu().numpy(),
                  out.tokens[sel].cpu().numpy(), out.h[sel].cpu().numpy(), out.resmass[sel].cpu().numpy(),
                  out.status[sel].cpu().numpy())
    print(cfg.name, rep.summary())
    for d in rep.detail:
        print("   ", d)
    return rep, out, ref


def assert_parity(rep):
    assert rep.decision_mismatches == 0, rep.detail
    assert rep.status_mismatches == 0, rep.detail
    assert rep.h_violations == 0, rep.detail
    assert rep.S_violations == 0, rep.detail
    # cells of Eq. 4 narrower than 2e-6 are always within 1e-6 of an edge, so on flat rows a fair
    # share of draws is excused by the rule; they are counted, and must still mostly agree
    assert rep.threshold_exceptions <= max(2, rep.rows // 3)
    assert rep.exceptions_matching >= rep.threshold_exceptions // 2


def test_config1_parity_and_20000_trials():
    cfg = workloads.CONFIGS["c1"]
    inp = workloads.make_inputs(cfg).to("cuda")
    rep, _, _ = run_both(inp)
    assert_parity(rep)
    # 20,000 trials on fixed logits/tokens with fresh uniforms: exact parity row by row and the
    # empirical law of (tau, f, y) against the exhaustively enumerated law
    n = 20000
    big = workloads.VerifyInputs(
        workloads.with_batch(cfg, n),
        inp.target_logits.expand(n, -1, -1, -1).contiguous(), inp.draft_logits.expand(n, -1, -1, -1).contiguous(),
        inp.draft_tokens.expand(n, -1, -1).contiguous(),
        workloads.make_uniforms(n, cfg.K, cfg.gamma, seed=cfg.seed + 1, device="cuda"))
    rep, out, ref = run_both(big)
    assert_parity(rep)
    from test_oracle_montecarlo import _chi2_critical, _exact_law_fixed_drafts
    law = _exact_law_fixed_drafts(_to_np32(inp.target_logits)[0], _to_np32(inp.draft_logits)[0],
                                  inp.draft_tokens.cpu().numpy()[0], cfg.temperature, cfg.K)
    tau = out.accept_len.cpu().numpy()
    f = out.draft_idx.cpu().numpy()
    tokens = out.tokens.cpu().numpy()
    counts = {}
    for t, ff, row in zip(tau, f, tokens):
        key = (int(t), int(ff), int(row[t]))
        counts[key] = counts.get(key, 0) + 1
    stat, dof = chi_square(counts, law)
    assert stat < _chi2_critical(dof), (stat, dof)
    assert abs(rep.block_efficiency_got - rep.block_efficiency_ref) < 1e-3


def test_config2_parity_full():
    inp = workloads.make_inputs(workloads.CONFIGS["c2"], device="cuda")
    rep, _, _ = run_both(inp)
    assert_parity(rep)


def test_config3_bf16_parity_full():
    inp = workloads.make_inputs(workloads.CONFIGS["c3"], device="cuda")
    assert inp.target_logits.dtype == torch.bfloat16
    rep, _, _ = run_both(inp)
    assert_parity(rep)


def test_config4_parity_sampled_rows():
    """Full-size launch (the configuration the benchmark times); the oracle recomputes a sample of
    whole batch rows, which are independent units."""
    inp = workloads.make_inputs(workloads.CONFIGS["c4"], device="cuda")
    rep, out, _ = run_both(inp, rows=[0, 7, 21, 38, 50, 63])
    assert_parity(rep)
    # properties that hold at any size, on all rows
    tau = out.accept_len.cpu().numpy()
    f = out.draft_idx.cpu().numpy()
    tokens = out.tokens.cpu().numpy()
    tok = inp.draft_tokens.cpu().numpy()
    cfg = inp.cfg
    assert ((tau >= 0) & (tau <= cfg.gamma)).all()
    assert ((f == -1) == (tau == 0)).all()
    for b in range(cfg.B):
        assert list(tokens[b, :tau[b]]) == list(tok[b, f[b], :tau[b]])
        assert 0 <= tokens[b, tau[b]] < cfg.V and (tokens[b, tau[b] + 1:] == -1).all()
    h = out.h.cpu().numpy()
    assert ((h >= 0) & (h <= 1)).all()


@pytest.mark.parametrize("K", [1, 2, 4, 8])
def test_config5_sweep_parity_sampled_rows(K):
    rows = list(range(0, 256, 16))
    for cfg in [c for c in workloads.sweep_c5() if c.K == K]:
        inp = workloads.make_inputs(cfg, device="cuda")
        rep, out, ref = run_both(inp, rows=rows)
        assert_parity(rep)
        if K == 1:   # K = 1 must reproduce single-draft GBV
            zq, zp = _to_np32(inp.target_logits), _to_np32(inp.draft_logits)
            tok, u = inp.draft_tokens.cpu().numpy(), inp.uniforms.cpu().numpy()
            for b in rows[:4]:
                q_rows = [np_softmax(zq[b, 0, i], cfg.temperature) for i in range(cfg.gamma + 1)]
                p_rows = [np_softmax(zp[b, 0, i], cfg.temperature) for i in range(cfg.gamma)]
                alpha, tau, y = gbv_single_draft(q_rows, p_rows, tok[b, 0], u[b, :cfg.gamma], float(u[b, cfg.gamma]))
                np.testing.assert_allclose(out.h[b, 0].cpu().numpy(), alpha, rtol=1e-5, atol=1e-9)
                if min(abs(u[b, j] - alpha[j]) for j in range(cfg.gamma)) > 1e-6:
                    assert int(out.accept_len[b]) == tau


@pytest.mark.parametrize("name", ["paper_l12", "paper_l8", "paper_l24"])
def test_paper_operating_points(name):
    """K = 3 drafts of 12, 8 or 24 tokens at T = 0.4 over a 32k vocabulary (the paper's Table 2 settings and
    the longest draft of its sweep over L),
    as a batch of 6 prompts so that several chains share the machine."""
    cfg = workloads.with_batch(workloads.CONFIGS[name], 6)
    inp = workloads.make_inputs(cfg, device="cuda")
    rep, _, _ = run_both(inp)
    assert_parity(rep)


@pytest.mark.parametrize("K,dtype", [(5, "fp32"), (6, "bf16"), (7, "fp32"), (16, "fp32")])
def test_draft_counts_without_a_specialised_kernel(K, dtype):
    """K outside {1,2,3,4,8} takes the run-time-K code of the fused kernel (rows are 16-byte aligned)."""
    cfg = workloads.VerifyConfig(f"k{K}", B=3, K=K, gamma=3, V=8192, dtype=dtype, temperature=0.8, alpha=0.85,
                                 seed=500 + K)
    inp = workloads.make_inputs(cfg, device="cuda")
    rep, _, _ = run_both(inp)
    assert_parity(rep)
    assert binding.last_main_kernel() == "fused_chain_kernel"


@pytest.mark.parametrize("B,K,gamma,V,dtype", [(50, 3, 4, 2048, "fp32"), (75, 2, 7, 4096, "bf16"), (149, 1, 5, 1024, "fp32"),
                                              (33, 4, 6, 40000, "fp32")])
def test_chains_cut_between_clusters(B, K, gamma, V, dtype):
    """The chain walk gives every cluster an equal share of the rows, so with a chain count that is no multiple of the
    clusters most chains begin on one cluster and end on another (the ratio c is handed over through global memory).
    Every batch row is compared."""
    cfg = workloads.VerifyConfig(f"cut_{B}_{K}_{gamma}", B=B, K=K, gamma=gamma, V=V, dtype=dtype, temperature=0.9,
                                 alpha=0.85, seed=700 + B)
    inp = workloads.make_inputs(cfg, device="cuda")
    rep, _, _ = run_both(inp)
    assert_parity(rep)
    assert binding.last_main_kernel() == "fused_chain_kernel"
    binding.set_option("walk", 1)            # and with the chain walk forced where the row walk would be chosen
    try:
        small = workloads.VerifyConfig("cut_small", B=7, K=3, gamma=5, V=3000, dtype=dtype, temperature=0.8, seed=701)
        rep, _, _ = run_both(workloads.make_inputs(small, device="cuda"))
        assert_parity(rep)
    finally:
        binding.set_option("walk", 0)


EDGE_SHAPES = [
    # B, K, gamma, V
    (3, 1, 1, 1), (2, 2, 3, 7), (5, 3, 2, 1000), (2, 2, 2, 1025), (2, 4, 3, 32001), (1, 1, 1, 5000),
    (4, 8, 1, 333), (1, 64, 2, 50), (2, 2, 64, 40), (1, 5, 7, 4099),
]


@pytest.mark.parametrize("B,K,gamma,V", EDGE_SHAPES)
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_edge_shapes(B, K, gamma, V, dtype):
    cfg = workloads.VerifyConfig(f"edge_{B}_{K}_{gamma}_{V}_{dtype}", B=B, K=K, gamma=gamma, V=V, dtype=dtype,
                                 temperature=0.9, alpha=0.8, boost=4.0, seed=4242 + V)
    inp = workloads.make_inputs(cfg, device="cuda")
    rep, _, _ = run_both(inp)
    assert_parity(rep)


@pytest.mark.parametrize("T", [0.05, 0.2, 3.0, 25.0])
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_temperature_extremes(T, dtype):
    """Very low temperatures turn rows into near point masses (exponentials underflow to zero away from the
    maximum, residual masses become tiny); very high ones flatten them (every CDF cell is narrow)."""
    cfg = workloads.VerifyConfig(f"temp_{T}_{dtype}", B=4, K=3, gamma=4, V=12288, dtype=dtype, temperature=T,
                                 alpha=0.9, seed=int(1000 * T) + 77)
    inp = workloads.make_inputs(cfg, device="cuda")
    rep, _, _ = run_both(inp)
    assert_parity(rep)


def test_vocabulary_beyond_the_fused_kernel_capacity():
    """Rows longer than 8 CTAs x 32,768 entries (the tensor memory of the largest cluster) take the generic
    two-sweep kernels, aligned or not."""
    cfg = workloads.VerifyConfig("bigv", B=2, K=2, gamma=2, V=8 * 32768 + 4096, alpha=0.85, seed=606)
    inp = workloads.make_inputs(cfg, device="cuda")
    rep, _, _ = run_both(inp)
    assert_parity(rep)
    assert binding.last_main_kernel() == "otreduce_kernel"


@pytest.mark.parametrize("V,dtype", [(8 * 32768, "fp32"), (8 * 32768 - 8, "bf16"), (5 * 32768 + 264, "fp32")])
def test_vocabulary_at_the_fused_kernel_capacity(V, dtype):
    """The longest rows the fused kernel takes (clusters of 8 with every tensor-memory column in use), and a
    row that needs a cluster of 6."""
    cfg = workloads.VerifyConfig("capv", B=2, K=2, gamma=2, V=V, dtype=dtype, alpha=0.85, seed=607)
    inp = workloads.make_inputs(cfg, device="cuda")
    rep, _, _ = run_both(inp)
    assert_parity(rep)
    assert binding.last_main_kernel() == "fused_chain_kernel"


def test_more_than_2_to_the_31_logits_per_tensor():
    """Element offsets beyond 32 bits: 2.8e9 bf16 logits in the target tensor (5.6 GB), 2.5e9 in the draft tensor.
    The oracle recomputes sampled batch rows from both ends of the tensors."""
    cfg = workloads.VerifyConfig("huge", B=256, K=8, gamma=8, V=151936, dtype="bf16", temperature=0.9, alpha=0.9,
                                 seed=808)
    assert cfg.B * cfg.K * (cfg.gamma + 1) * cfg.V > 2 ** 31
    inp = workloads.make_inputs(cfg, device="cuda")
    rep, out, _ = run_both(inp, rows=[0, 131, 255])
    assert_parity(rep)
    tau = out.accept_len.cpu().numpy()
    assert ((tau >= 0) & (tau <= cfg.gamma)).all() and (out.status.cpu().numpy() == 0).all()
    del inp, out
    torch.cuda.empty_cache()


def _slice_fits(V, cluster):
    """A CTA of the fused kernel holds at most 128 cells of 256 entries of a row in tensor memory."""
    cells = -(-V // 256)
    return -(-cells // cluster) <= 128


@pytest.mark.parametrize("option", [("path", 1), ("path", 2), ("cluster", 1), ("cluster", 2), ("cluster", 3),
                                    ("cluster", 4), ("cluster", 5), ("cluster", 7), ("cluster", 8),
                                    ("max_clusters", 3), ("walk", 1), ("walk", 2), ("aux", 1), ("aux", 2)])
def test_every_kernel_path_and_launch_shape_matches(option):
    """The generic two-sweep kernels and the fused kernel at every cluster size / walk /
    persistent-grid size must all agree with the oracle (automatic choice is covered elsewhere)."""
    cfgs = [workloads.VerifyConfig("paths_a", B=5, K=3, gamma=3, V=20480, temperature=0.8, alpha=0.8, seed=21),
            workloads.VerifyConfig("paths_b", B=3, K=2, gamma=2, V=33000, dtype="bf16", temperature=1.1, alpha=0.7,
                                   seed=22),
            workloads.VerifyConfig("paths_c", B=2, K=2, gamma=5, V=1000, alpha=0.9, seed=23),
            workloads.VerifyConfig("paths_d", B=40, K=2, gamma=3, V=9000, temperature=0.9, alpha=0.85, seed=24)]
    binding.set_option(*option)
    try:
        for cfg in cfgs:
            if option[0] == "cluster" and not _slice_fits(cfg.V, option[1]):
                continue   # forced cluster size whose slices do not fit the tensor memory
            if option == ("walk", 2) and cfg.B * cfg.K * cfg.gamma > 256:
                continue   # the row walk has one ratio word per row, 256 in all
            inp = workloads.make_inputs(cfg, device="cuda")
            rep, _, _ = run_both(inp)
            assert_parity(rep)
    finally:
        binding.set_option(option[0], 0)


@pytest.mark.parametrize("K,dtype,alpha,T", [(1, "fp32", 0.8, 1.0), (2, "bf16", 0.9, 0.7), (8, "fp32", 0.9, 1.0),
                                             (3, "fp32", 0.9995, 1.0), (5, "fp32", 0.99, 0.4), (8, "bf16", 0.9999, 1.0)])
def test_extra_sums_in_kernels_of_their_own(K, dtype, alpha, T):
    """Chain walk with the two extra sums of Eq. 2 (rows with c < 1) left to the kernels behind the fused kernel, which
    only do the rows whose plain numerator would cancel: ordinary drafts (few such rows), drafts nearly equal to the
    target (nearly all rows with c < 1 qualify), and a draft count without a specialised kernel; and the same inputs
    with the sums worked out in the fused kernel must give the same weights."""
    cfg = workloads.VerifyConfig(f"aux_{K}_{dtype}_{alpha}", B=24, K=K, gamma=5, V=40192, dtype=dtype, temperature=T,
                                 alpha=alpha, seed=300 + K)
    inp = workloads.make_inputs(cfg, device="cuda")
    res = {}
    for aux in (2, 1):
        binding.set_option("walk", 1)
        binding.set_option("aux", aux)
        try:
            rep, out, _ = run_both(inp)
            assert_parity(rep)
            res[aux] = out.h.cpu().numpy()
            assert binding.last_launch_count() == (4 if aux == 2 else 2)
        finally:
            binding.set_option("walk", 0)
            binding.set_option("aux", 0)
    np.testing.assert_allclose(res[2], res[1], rtol=2e-5, atol=1e-9)


def test_unaligned_views_and_repeated_calls_are_deterministic():
    cfg = workloads.VerifyConfig("unaligned", B=3, K=2, gamma=3, V=4099, alpha=0.8, seed=99)
    inp = workloads.make_inputs(cfg, device="cuda")
    # place the logits one element past a 16-byte boundary
    def shifted(t):
        buf = torch.empty(t.numel() + 1, dtype=t.dtype, device=t.device)
        v = buf[1:].view(t.shape)
        v.copy_(t)
        return v
    sh = workloads.VerifyInputs(cfg, shifted(inp.target_logits), shifted(inp.draft_logits), inp.draft_tokens,
                                inp.uniforms)
    assert sh.target_logits.data_ptr() % 16 != 0
    rep, out1, _ = run_both(sh)
    assert_parity(rep)
    out2 = binding.sgbv_verify_ex(inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms,
                                  cfg.temperature)
    out3 = binding.sgbv_verify_ex(inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms,
                                  cfg.temperature)
    torch.cuda.synchronize()
    for a, b in ((out2, out3), (out1, out2)):
        assert torch.equal(a.accept_len, b.accept_len) and torch.equal(a.tokens, b.tokens)
        assert torch.equal(a.h, b.h) and torch.equal(a.resmass, b.resmass)


def test_degenerate_and_flagged_rows():
    cfg = workloads.VerifyConfig("flags", B=6, K=2, gamma=2, V=300, alpha=0.8, seed=7)
    inp = workloads.make_inputs(cfg, device="cuda")
    zq, zp = inp.target_logits.clone(), inp.draft_logits.clone()
    tok, u = inp.draft_tokens.clone(), inp.uniforms.clone()
    zp[1] = zq[1, :, :2]                 # row 1: p == q everywhere -> zero residual mass
    u[1, :4] = 0.999
    tok[2, 1, 0] = 300                   # row 2: token out of range
    zq[3, 0, 1, 17] = float("nan")       # row 3: NaN logit
    zp[4, 1, 0, 5] = float("inf")        # row 4: +inf logit
    zq[5, :, :, 11] = float("-inf")      # row 5: -inf is allowed (probability 0)
    zp[5, :, :, 12] = float("-inf")
    mod = workloads.VerifyInputs(cfg, zq, zp, tok, u)
    rep, out, ref = run_both(mod)
    assert_parity(rep)
    st = out.status.cpu().numpy()
    assert st[1] & binding.STATUS_DEGENERATE_RESIDUAL
    assert st[2] & binding.STATUS_TOKEN_RANGE and st[3] & binding.STATUS_NONFINITE_LOGIT
    assert st[4] & binding.STATUS_NONFINITE_LOGIT and st[0] == 0 and (st[5] & 3) == 0
    assert (out.tokens[2:5].cpu().numpy() == -1).all() and (out.accept_len[2:5].cpu().numpy() == -1).all()


def test_repeated_calls_on_the_library_scratch_match_calls_on_a_fresh_workspace():
    """The row walk's "not published yet" words are cleared by a memset on a caller's workspace, but on the
    library's own scratch they are put back by the finishing kernel for the next call of the same layout.
    Sequences of calls (same shape repeated, another shape in between) must give what a fresh workspace gives."""
    row_cfg = workloads.with_batch(workloads.CONFIGS["paper_l8"], 2)
    other_cfg = workloads.VerifyConfig("other", B=16, K=4, gamma=4, V=8192, alpha=0.85, seed=31)
    sets = [workloads.make_inputs(row_cfg, device="cuda", set_index=i) for i in range(4)]
    other = workloads.make_inputs(other_cfg, device="cuda")

    def fresh(inp):
        ws = torch.empty(binding.workspace_bytes(inp.cfg.B, inp.cfg.K, inp.cfg.gamma, inp.cfg.V) + 256,
                         dtype=torch.uint8, device="cuda")
        ws.fill_(0x5a)
        off = (-ws.data_ptr()) % 256
        return binding.sgbv_verify_ex(inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms,
                                      inp.cfg.temperature, workspace=ws[off:off + ws.numel() - 256])

    order = [sets[0], sets[1], sets[1], other, sets[2], sets[3], other, other, sets[0]]
    for inp in order:
        got = binding.sgbv_verify_ex(inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms,
                                     inp.cfg.temperature)
        want = fresh(inp)
        torch.cuda.synchronize()
        assert torch.equal(got.accept_len, want.accept_len) and torch.equal(got.draft_idx, want.draft_idx)
        assert torch.equal(got.tokens, want.tokens) and torch.equal(got.status, want.status)
        assert torch.equal(got.h, want.h) and torch.equal(got.resmass, want.resmass)
    rep, _, _ = run_both(sets[2])
    assert_parity(rep)


@pytest.mark.parametrize("name", ["c2", "paper_l8"])
def test_calls_replayed_from_a_cuda_graph_give_the_eager_results(name):
    """After a warm-up call per shape a call only enqueues kernels (the chain walk of c2, the row walk of the
    one-prompt shape): a captured sequence of calls, replayed, must reproduce the eager outputs."""
    cfg = workloads.CONFIGS[name]
    sets = [workloads.make_inputs(cfg, device="cuda", set_index=i) for i in range(3)]
    eager = [binding.sgbv_verify(i.target_logits, i.draft_logits, i.draft_tokens, i.uniforms, cfg.temperature)
             for i in sets]
    torch.cuda.synchronize()
    outs = [binding.VerifyOutput(torch.full_like(e.accept_len, -7), torch.full_like(e.draft_idx, -7),
                                 torch.full_like(e.tokens, -7)) for e in eager]
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for i, o in zip(sets, outs):
                binding.sgbv_verify(i.target_logits, i.draft_logits, i.draft_tokens, i.uniforms, cfg.temperature,
                                    out=o)
    for _ in range(2):
        for o in outs:
            o.accept_len.fill_(-7), o.draft_idx.fill_(-7), o.tokens.fill_(-7)
        graph.replay()
        torch.cuda.synchronize()
        for e, o in zip(eager, outs):
            assert torch.equal(e.accept_len, o.accept_len) and torch.equal(e.draft_idx, o.draft_idx)
            assert torch.equal(e.tokens, o.tokens)


def _full_out(cfg):
    dev = "cuda"
    return binding.VerifyOutput(torch.full((cfg.B,), -7, dtype=torch.int32, device=dev),
                                torch.full((cfg.B,), -7, dtype=torch.int32, device=dev),
                                torch.full((cfg.B, cfg.gamma + 1), -7, dtype=torch.int32, device=dev),
                                torch.zeros((cfg.B, cfg.K, cfg.gamma), dtype=torch.float64, device=dev),
                                torch.zeros((cfg.B, cfg.K, cfg.gamma), dtype=torch.float64, device=dev),
                                torch.full((cfg.B,), -7, dtype=torch.int32, device=dev))


def _fresh_workspace_result(inp):
    ws = torch.empty(binding.workspace_bytes(inp.cfg.B, inp.cfg.K, inp.cfg.gamma, inp.cfg.V) + 256,
                     dtype=torch.uint8, device="cuda")
    ws.fill_(0x5a)
    off = (-ws.data_ptr()) % 256
    out = binding.sgbv_verify_ex(inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms,
                                 inp.cfg.temperature, workspace=ws[off:off + ws.numel() - 256])
    torch.cuda.synchronize()
    return out


def _assert_identical(got, want):
    assert torch.equal(got.accept_len, want.accept_len) and torch.equal(got.draft_idx, want.draft_idx)
    assert torch.equal(got.tokens, want.tokens) and torch.equal(got.status, want.status)
    assert torch.equal(got.h, want.h) and torch.equal(got.resmass, want.resmass)


def _capture_call(inp, out):
    """A CUDA graph holding one verify call on the library's own scratch (warmed up first, so nothing allocates)."""
    args = (inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms, inp.cfg.temperature)
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            binding.sgbv_verify_ex(*args, out=out)
    return graph


def test_graph_replays_and_eager_calls_of_other_shapes_in_any_order():
    """The row walk relies on words of the scratch that hold a "not published yet" pattern when a call starts.
    That must hold whatever ran before on the library's scratch: captures that never ran, replays of graphs of
    other shapes, eager calls in between.  Every result equals the one computed on a fresh caller workspace."""
    row_a = workloads.make_inputs(workloads.with_batch(workloads.CONFIGS["paper_l8"], 2), device="cuda")
    row_b = workloads.make_inputs(workloads.VerifyConfig("rowb", B=3, K=2, gamma=5, V=12288, temperature=0.7,
                                                         alpha=0.8, seed=41), device="cuda")
    c2 = workloads.make_inputs(workloads.CONFIGS["c2"], device="cuda")
    big = workloads.make_inputs(workloads.VerifyConfig("bigger", B=64, K=4, gamma=4, V=32000, alpha=0.85, seed=42),
                                device="cuda")
    want = {id(x): _fresh_workspace_result(x) for x in (row_a, row_b, c2, big)}

    def eager(inp):
        out = binding.sgbv_verify_ex(inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms,
                                     inp.cfg.temperature)
        torch.cuda.synchronize()
        assert_row_walk = inp is row_a or inp is row_b
        assert binding.last_main_kernel() == "fused_chain_kernel"
        _assert_identical(out, want[id(inp)])
        return assert_row_walk

    for inp in (big, row_a, row_b, c2):   # warm-up: the scratch has its final size from here on
        eager(inp)
    # (i) capture the row walk, run another shape eagerly, replay
    out_a = _full_out(row_a.cfg)
    graph_a = _capture_call(row_a, out_a)
    eager(c2)
    graph_a.replay()
    torch.cuda.synchronize()
    _assert_identical(out_a, want[id(row_a)])
    # (ii) a large shape eagerly, a capture that is not replayed, then the captured shape eagerly
    eager(big)
    out_b = _full_out(row_b.cfg)
    graph_b = _capture_call(row_b, out_b)
    eager(row_b)
    eager(row_a)
    # (iii) graphs of two row-walk shapes replayed alternately, eager calls in between
    for _ in range(3):
        graph_a.replay()
        graph_b.replay()
        torch.cuda.synchronize()
        _assert_identical(out_a, want[id(row_a)])
        _assert_identical(out_b, want[id(row_b)])
        eager(c2)
        graph_b.replay()
        graph_a.replay()
        torch.cuda.synchronize()
        _assert_identical(out_a, want[id(row_a)])
        _assert_identical(out_b, want[id(row_b)])


def test_a_bounded_wait_that_runs_out_flags_every_row_and_the_next_call_is_correct():
    """Failure detection without a fault: in the row walk a row waits (bounded) for the ratios that the rows
    before it publish.  With the first row of every chain withholding its ratio and the limit of that poll
    shortened, the poll expires; the kernel runs to its end, every batch row comes back flagged TIMEOUT with
    -1 outputs, and the next ordinary call on the same scratch is correct."""
    cfg = workloads.with_batch(workloads.CONFIGS["paper_l8"], 2)
    inp = workloads.make_inputs(cfg, device="cuda")
    args = (inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms, cfg.temperature)
    binding.set_option("withhold", 1)
    binding.set_option("poll_us", 300)
    try:
        out = binding.sgbv_verify_ex(*args)
        torch.cuda.synchronize()
    finally:
        binding.set_option("withhold", 0)
        binding.set_option("poll_us", 0)
    assert binding.last_main_kernel() == "fused_chain_kernel"
    st = out.status.cpu().numpy()
    assert ((st & binding.STATUS_TIMEOUT) != 0).all()
    assert (out.accept_len.cpu().numpy() == -1).all() and (out.draft_idx.cpu().numpy() == -1).all()
    assert (out.tokens.cpu().numpy() == -1).all()
    rep, again, _ = run_both(inp)
    assert_parity(rep)
    assert (again.status.cpu().numpy() & binding.STATUS_TIMEOUT == 0).all()


def test_plain_bf16_and_host_entry_points_agree_with_extended():
    for name in ("c2",):
        cfg = workloads.CONFIGS[name]
        inp = workloads.make_inputs(cfg, device="cuda")
        ex = binding.sgbv_verify_ex(inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms,
                                    cfg.temperature)
        plain = binding.sgbv_verify(inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms,
                                    cfg.temperature)
        ws = torch.empty(binding.workspace_bytes(cfg.B, cfg.K, cfg.gamma, cfg.V) + 256, dtype=torch.uint8,
                         device="cuda")
        off = (-ws.data_ptr()) % 256
        ex2 = binding.sgbv_verify_ex(inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms,
                                     cfg.temperature, workspace=ws[off:off + ws.numel() - 256])
        host = binding.sgbv_verify_host(inp.target_logits.cpu().pin_memory(), inp.draft_logits.cpu().pin_memory(),
                                        inp.draft_tokens.cpu().pin_memory(), inp.uniforms.cpu().pin_memory(),
                                        cfg.temperature)
        torch.cuda.synchronize()
        for o in (plain, ex2):
            assert torch.equal(o.accept_len, ex.accept_len) and torch.equal(o.tokens, ex.tokens)
            assert torch.equal(o.draft_idx, ex.draft_idx)
        assert torch.equal(host.accept_len, ex.accept_len.cpu()) and torch.equal(host.tokens, ex.tokens.cpu())
        assert binding.last_launch_count() > 0
    small = workloads.VerifyConfig("bf", B=2, K=2, gamma=2, V=2048, dtype="bf16", seed=5)
    inp = workloads.make_inputs(small, device="cuda")
    a = binding.sgbv_verify(inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms, 1.0)
    b = binding.sgbv_verify_ex(inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms, 1.0)
    torch.cuda.synchronize()
    assert torch.equal(a.tokens, b.tokens)
