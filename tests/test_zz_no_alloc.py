"""The allocation-free entry point (``sgbv_verify_static``) against the ordinary one.

Collected last on purpose: a run that stops at the first failure has then already run every other
test.  The new entry point takes its scratch from a fixed array inside the library instead of
allocating, for callers that must not allocate device memory once they are running (their pool
owns all of it, or an allocation's device-wide stall is not acceptable).  Same kernels, other
scratch: the results have to agree with ``sgbv_verify_ex`` -- decisions exactly, weights and
residual masses within the 1e-5 relative tolerance of the parity tests -- on two calls in a row
that leave different leftovers in the shared array.
"""
import pytest
import torch

from paper_2604_25925_b200 import binding, workloads

pytestmark = pytest.mark.gpu


def _same(a, b):
    assert torch.equal(a.accept_len, b.accept_len)
    assert torch.equal(a.draft_idx, b.draft_idx)
    assert torch.equal(a.tokens, b.tokens)
    assert torch.equal(a.status, b.status)
    torch.testing.assert_close(a.h, b.h, rtol=1e-5, atol=1e-9)
    torch.testing.assert_close(a.resmass, b.resmass, rtol=1e-5, atol=1e-30)


def test_static_scratch_entry_point_matches_on_two_calls_in_a_row():
    first = workloads.make_inputs(workloads.CONFIGS["c2"], device="cuda")
    second = workloads.make_inputs(
        workloads.VerifyConfig("na2", B=5, K=3, gamma=2, V=4099, dtype="bf16", temperature=0.8, alpha=0.7,
                               seed=31), device="cuda")
    for inp in (first, second):       # the second call finds the first call's leftovers in the array
        args = (inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms, inp.cfg.temperature)
        got = binding.sgbv_verify_static(*args)
        ref = binding.sgbv_verify_ex(*args)
        torch.cuda.synchronize()
        _same(got, ref)
    # a shape that takes the row walk of the fused kernel, the one path that reads words of the shared array
    # before writing them: before and after a larger shape that overwrites that part of the array
    walk = workloads.make_inputs(workloads.with_batch(workloads.CONFIGS["paper_l8"], 2), device="cuda")
    for inp in (walk, first, walk, walk):
        args = (inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms, inp.cfg.temperature)
        got = binding.sgbv_verify_static(*args)
        assert binding.last_main_kernel() == "fused_chain_kernel"
        ref = binding.sgbv_verify_ex(*args)
        torch.cuda.synchronize()
        _same(got, ref)
    # and once more on the first inputs, now over the second call's leftovers
    args = (first.target_logits, first.draft_logits, first.draft_tokens, first.uniforms, first.cfg.temperature)
    got = binding.sgbv_verify_static(*args)
    ref = binding.sgbv_verify_ex(*args)
    torch.cuda.synchronize()
    _same(got, ref)


def test_static_scratch_entry_point_refuses_shapes_beyond_its_array():
    B, K, gamma, V = 4096, 8, 8, 32000
    assert binding.workspace_bytes(B, K, gamma, V) > binding.STATIC_SCRATCH_BYTES
    lib = binding.load()
    d = torch.zeros(64, device="cuda")
    p = d.data_ptr()
    rc = lib.sgbv_verify_static(p, p, 0, p, p, B, K, gamma, V, 1.0, p, p, p, None, None, None, None)
    assert rc == -5 and "WORKSPACE" in binding.status_string(rc)
