"""The exit at the fixed point (an iteration that moves no dual by more than rounding ends the loop, Appendix C's
T = 100 being an upper limit) against the same kernel's own T = 100 iterations, for every Sinkhorn kernel at a
tile of the largest kind it takes.  The profiling record names the kernel that ran.  Marked gpu."""
import numpy as np
import pytest
import torch

from paper_2605_00392_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def parity():
    import parity as _p
    return _p


@pytest.fixture(scope="module")
def binding():
    from paper_2605_00392_b200 import binding as _b
    return _b


def _run(binding, plan, w, dev, **over):
    p = dict(w.params)
    p.update(over)
    fields = {k: (int(v) if k in ("dynamic", "iters", "form", "stop_at_fixed_point", "criterion", "schedule") else float(v))
              for k, v in p.items()}
    params = binding.make_params(torch.from_numpy(w.rho.copy()).to(dev), **fields)
    out = binding.Outputs.allocate(w.total_tokens, w.batch, w.d, w.X.dtype, dev)
    plan.run(w.X.to(dev), torch.from_numpy(w.offsets.copy()).to(dev), params, out)
    names = [n for n, _ in plan.profile_read()]
    assert plan.query_status() == 0
    return out, names


# (case, image lengths, dtype, d, fixed r, extra parameters, kernel that must run, weight rtol)
CASES = [
    # register-resident K, clusters of two: 200 x 200, the largest tile of a 400-token image
    ("reg", [400] * 6, torch.bfloat16, 1280, 0.5, {}, "sinkhorn_reg", 2e-6),
    # more images than clusters of the register kernel fit at once: the shared-memory cluster kernel
    ("cluster", [400] * 80, torch.bfloat16, 1280, 0.25, {}, "sinkhorn_cluster", 2e-6),
    # the same batch at the ratio cap: 200 x 200 tiles no longer fit one CTA each, the instance for wide tiles takes them
    ("cluster_at_cap", [400] * 80, torch.bfloat16, 1280, 0.5, {}, "sinkhorn_wide", 2e-6),
    # 578 columns (more than 256): the cluster kernel's instance for wide tiles, K in the workspace
    ("wide", [1156, 1156, 900], torch.bfloat16, 1280, 0.5, {}, "sinkhorn_wide", 2e-6),
    # 1729 columns: clusters of 8 or 16 CTAs iterate on K in the workspace (exit within 4 ulp: long sums)
    ("tall", [4512], torch.bfloat16, 1280, 0.3832, {}, "sinkhorn_tall", 2e-5),
    # log-domain form, one CTA per image (exit when the duals repeat bit for bit)
    ("log", [400, 256], torch.bfloat16, 1280, 0.5, dict(form=1), "sinkhorn", 2e-5),
    # fp32 storage takes the cluster kernel with the plan written in place
    ("fp32", [400] * 4, torch.float32, 64, 0.5, {}, "sinkhorn_cluster", 2e-6),
]


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_exit_at_fixed_point_equals_all_iterations(binding, case):
    name, lengths, dtype, d, r, extra, kernel, wtol = case
    dev = torch.device("cuda", 0)
    w = synth.ragged(lengths, d=d, dtype=dtype, params=dict(r_fixed=r))
    plan = binding.Plan(w.d, w.X.dtype, w.batch, w.total_tokens, w.max_tokens, device=dev)
    plan.profile_enable(True)
    try:
        a, names_a = _run(binding, plan, w, dev, stop_at_fixed_point=1, **extra)
        b, names_b = _run(binding, plan, w, dev, stop_at_fixed_point=0, **extra)
    finally:
        plan.profile_enable(False)
        plan.close()
    assert kernel in names_a and names_a == names_b, (names_a, names_b)
    nb = w.batch
    ita, itb = a.stats[:nb, 5].cpu().numpy(), b.stats[:nb, 5].cpu().numpy()
    assert np.all(itb == 100.0), itb
    assert np.all(ita >= 1) and ita.max() < 100.0, ita          # the exit was taken
    assert torch.equal(a.kept_idx, b.kept_idx) and torch.equal(a.merged_idx, b.merged_idx)
    n = int(a.out_offsets[nb])
    npr = w.total_tokens - n
    wa, wb = a.merge_weight[:npr].cpu(), b.merge_weight[:npr].cpu()
    torch.testing.assert_close(wa, wb, rtol=wtol, atol=0)
    # partners: identical wherever the two runs' weights are not a rounding tie
    pa, pb = a.merge_partner[:npr].cpu(), b.merge_partner[:npr].cpu()
    differ = pa != pb
    assert float(differ.float().mean()) < 0.02, float(differ.float().mean())
    ya, yb = a.Y[:n].float().cpu(), b.Y[:n].float().cpu()
    if dtype == torch.bfloat16:
        assert (ya - yb).abs().max() <= 2.0 ** -8 * yb.abs().max()          # at most one bf16 rounding apart
        assert float((ya != yb).float().mean()) < 2e-3
    else:
        torch.testing.assert_close(ya, yb, rtol=1e-5, atol=1e-6)
