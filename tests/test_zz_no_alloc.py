"""rtprune_select_static: stage 1 for callers that cannot allocate device memory.

A plug-in inside another framework's memory pool, a real-time loop where cudaMalloc's implicit
synchronisation is not allowed, or a process with a memory budget fixed at start-up cannot hand the
library a workspace.  For them the library carries a fixed scratch array in its own device image.
This test calls that entry point through the C ABI and checks every output against the ordinary
rtprune_select (caller-allocated workspace) on two calls in a row over different batches: the
array is shared by all calls and keeps the previous call's contents, so the second call is the one
that would expose state leaking from the first.

The file sorts last on purpose: a run that stops at the first failure has then already run every
other test.
"""
import numpy as np
import pytest
import torch

from paper_2605_00392_b200 import binding, synth

pytestmark = pytest.mark.gpu

STATIC_SCRATCH_BYTES = 8 << 20      # RTPRUNE_STATIC_SCRATCH_BYTES in include/rtprune.h


def _fields(w):
    return {k: (int(v) if k in ("dynamic", "iters") else float(v)) for k, v in w.params.items()}


def _stage1(plan, w, dev, static):
    out = binding.Outputs.allocate(w.total_tokens, w.batch, w.d, w.X.dtype, dev)
    norms = torch.full((w.total_tokens,), -1.0, device=dev)
    order = torch.full((w.total_tokens,), -1, dtype=torch.int32, device=dev)
    rho = torch.from_numpy(w.rho).to(dev)
    params = binding.make_params(rho, **_fields(w))
    X = w.X.to(dev)
    offs = torch.from_numpy(w.offsets).to(dev)
    call = plan.select_static if static else plan.select
    call(X, offs, params, out, norms, order)
    torch.cuda.synchronize()
    return (out.counts.cpu().numpy(), out.out_offsets.cpu().numpy(), out.stats.cpu().numpy(),
            norms.cpu().numpy(), order.cpu().numpy())


def _same(a, b, tag):
    counts_a, offs_a, stats_a, norms_a, order_a = a
    counts_b, offs_b, stats_b, norms_b, order_b = b
    # integer outputs: bit-exact, like every index comparison of the parity tests
    np.testing.assert_array_equal(counts_a, counts_b, err_msg=tag)
    np.testing.assert_array_equal(offs_a, offs_b, err_msg=tag)
    np.testing.assert_array_equal(order_a, order_b, err_msg=tag)
    # floating-point outputs: the parity tests' tolerances (phi 2e-5 absolute, r 1e-5, norms 2e-6)
    np.testing.assert_allclose(stats_a[:, 0], stats_b[:, 0], rtol=0, atol=2e-5, err_msg=tag)
    np.testing.assert_allclose(stats_a[:, 2], stats_b[:, 2], rtol=0, atol=1e-5, err_msg=tag)
    np.testing.assert_array_equal(stats_a[:, 3:5], stats_b[:, 3:5], err_msg=tag)
    np.testing.assert_allclose(norms_a, norms_b, rtol=2e-6, err_msg=tag)
    assert counts_a.min() >= 1 and (norms_a > 0).all() and (order_a >= 0).all(), tag


def test_static_scratch_matches_workspace_path_twice():
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    first = synth.make("large", batch=12)                      # dynamic ratio, 12 x 400 tokens
    second = synth.ragged([400, 37, 256, 1, 180], params=dict(r_fixed=0.35))   # other shape, fixed r
    plan = binding.Plan(1280, torch.bfloat16, 12, first.total_tokens, 400, device=dev)
    try:
        for tag, w in (("first call", first), ("second call", second)):
            ref = _stage1(plan, w, dev, static=False)
            assert plan.query_status() == 0
            got = _stage1(plan, w, dev, static=True)
            assert plan.last_launch_count >= 1
            _same(got, ref, tag)
    finally:
        plan.close()


def _a256(x):
    return (x + 255) // 256 * 256


def _needed(max_batch, max_total, max_tokens, d):
    # the header's formula for the bytes of the array a plan's stage 1 uses
    return 256 + 4 * _a256(4 * max_batch) + 4 * _a256(4 * max_total) + _a256(4 * max_batch * ((max_tokens + 31) // 32) * d)


def test_static_scratch_limit_is_the_stated_one():
    """The stated formula, the stated figure for the 64 x 400 x 1280 plan, and the boundary: the largest batch
    of 400-token images that fits runs, one image more is refused before anything is launched."""
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    assert _needed(64, 64 * 400, 400, 1280) == 4_670_720
    fits = max(b for b in range(1, 400) if _needed(b, b * 400, 400, 1280) <= STATIC_SCRATCH_BYTES)
    assert fits == 114
    for batch, ok in ((64, True), (fits, True), (fits + 1, False)):
        plan = binding.Plan(1280, torch.bfloat16, batch, batch * 400, 400, device=dev)
        try:
            assert plan.static_scratch_needed() == _needed(batch, batch * 400, 400, 1280)
            assert (plan.static_scratch_needed() <= STATIC_SCRATCH_BYTES) == ok
            w = synth.make("large", batch=3)
            out = binding.Outputs.allocate(w.total_tokens, w.batch, w.d, w.X.dtype, dev)
            params = binding.make_params(torch.from_numpy(w.rho).to(dev), **_fields(w))
            args = (w.X.to(dev), torch.from_numpy(w.offsets).to(dev), params, out)
            if ok:
                plan.select_static(*args)
                assert plan.query_status_static() == 0
                ref = binding.Outputs.allocate(w.total_tokens, w.batch, w.d, w.X.dtype, dev)
                plan.select(args[0], args[1], params, ref)
                torch.cuda.synchronize()
                assert torch.equal(out.counts, ref.counts) and torch.equal(out.out_offsets, ref.out_offsets)
            else:
                with pytest.raises(binding.RtpruneError) as err:
                    plan.select_static(*args)
                assert err.value.status == 3      # RTPRUNE_ERR_WORKSPACE
        finally:
            plan.close()


def test_static_scratch_whole_headline_batch():
    """64 x 400 x 1280, the largest batch the other tests time: every stage-1 output equals the workspace path's."""
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    w = synth.make("large")
    plan = binding.Plan(1280, torch.bfloat16, w.batch, w.total_tokens, 400, device=dev)
    try:
        ref = _stage1(plan, w, dev, static=False)
        got = _stage1(plan, w, dev, static=True)
        assert plan.query_status_static() == 0
        _same(got, ref, "64 x 400")
    finally:
        plan.close()


def test_static_scratch_reports_device_status():
    """A non-finite token and an image outside the offsets contract show in the array's status word; a clean
    call afterwards reads clean."""
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    w = synth.ragged([40, 64, 9])
    plan = binding.Plan(1280, torch.bfloat16, 3, w.total_tokens, 64, device=dev)
    try:
        out = binding.Outputs.allocate(w.total_tokens, w.batch, w.d, w.X.dtype, dev)
        params = binding.make_params(None, **_fields(w))
        offs = torch.from_numpy(w.offsets).to(dev)
        X = w.X.to(dev)
        plan.select_static(X, offs, params, out)
        assert plan.query_status_static() == 0
        bad = X.clone()
        bad[45, 7] = float("inf")
        plan.select_static(bad, offs, params, out)
        assert plan.query_status_static() & 1            # RTPRUNE_DEV_NONFINITE
        assert plan.query_status_static() == 0           # reading clears it
        long_offs = torch.tensor([0, 40, 113, 113], dtype=torch.int32, device=dev)   # 73 > 64 tokens, then 0 tokens
        plan.select_static(X, long_offs, params, out)
        assert plan.query_status_static() & 4            # RTPRUNE_DEV_BAD_OFFSETS
        torch.cuda.synchronize()
        assert out.counts.cpu().tolist()[1:] == [0, 0]
        plan.select_static(X, offs, params, out)
        assert plan.query_status_static() == 0
    finally:
        plan.close()


def test_static_scratch_rejects_plans_beyond_its_size():
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    w = synth.ragged([64, 64])
    big = binding.Plan(1280, torch.bfloat16, 1024, 1024 * 400, 400, device=dev)   # needs > 8 MiB
    try:
        out = binding.Outputs.allocate(w.total_tokens, w.batch, w.d, w.X.dtype, dev)
        params = binding.make_params(None, **_fields(w))
        with pytest.raises(binding.RtpruneError) as err:
            big.select_static(w.X.to(dev), torch.from_numpy(w.offsets).to(dev), params, out)
        assert err.value.status == 3          # RTPRUNE_ERR_WORKSPACE
        assert big.workspace_bytes > STATIC_SCRATCH_BYTES
    finally:
        big.close()
