"""Host-side behaviour of the library on a GPU: a bounded device-side wait that runs out is reported and leaves
the context usable; function attributes set by one plan survive a later, smaller plan.  Marked gpu."""
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


def test_expired_wait_is_reported_and_the_next_run_is_clean(parity, binding):
    """The waits give up after 64 polls on flags that nothing sets (no fault, no trap: the kernel returns),
    the status word says so, and the same plan and workspace then pass the parity check."""
    dev = torch.device("cuda", 0)
    w = synth.make("large", batch=4)
    plan = binding.Plan(w.d, w.X.dtype, w.batch, w.total_tokens, w.max_tokens, device=dev)
    try:
        assert plan.query_status() == 0
        assert plan.expire_waits(64) == 2                 # the flag wait and the barrier wait both gave up
        flags = plan.query_status()
        assert flags == binding.DEV_TIMEOUT
        st = binding.lib().rtprune_query_status(plan.handle, None, plan.workspace.data_ptr(), None)
        assert st == 0                                    # reading cleared it
        plan.expire_waits(1)
        st = binding.lib().rtprune_query_status(plan.handle, None, plan.workspace.data_ptr(), None)
        assert st == 6                                    # RTPRUNE_ERR_TIMEOUT
        with pytest.raises(binding.RtpruneError):
            plan.expire_waits(0)                          # limit out of range: nothing is launched
        rep = parity.check_workload(w, plan=plan)
        assert rep["images_compared"] == 4
    finally:
        plan.close()


def test_smaller_plan_does_not_shrink_an_earlier_plans_kernels(parity, binding):
    """Shared-memory limits are attributes of the kernels, not of a plan: a plan for 400-token images, then a plan
    for 32-token images, then the first plan's run in the log-domain form (its Sinkhorn kernel takes the most
    shared memory of all) must still launch and pass."""
    dev = torch.device("cuda", 0)
    big = synth.make("large", batch=3)
    small = synth.ragged([32, 20], params=dict(r_fixed=0.25))
    plan_big = binding.Plan(big.d, big.X.dtype, big.batch, big.total_tokens, 400, device=dev)
    plan_small = binding.Plan(small.d, small.X.dtype, small.batch, small.total_tokens, 32, device=dev)
    try:
        for form in (binding.SINKHORN_LOG, binding.SINKHORN_EXACT, binding.SINKHORN_AUTO):
            if form == binding.SINKHORN_EXACT:
                parity.check_exact(big, plan=plan_big)
            else:
                parity.check_workload(big, overrides=dict(form=form), plan=plan_big)
        parity.check_workload(small, overrides=dict(form=binding.SINKHORN_LOG), plan=plan_small)
    finally:
        plan_small.close()
        plan_big.close()


def test_two_slices_concatenate_to_the_one_call_result(binding):
    """What two ranks would do, on one GPU: each slice of the batch (the package's shard_slice) through a plan
    of its own, the second slice's offsets shifted by the first one's kept rows; the concatenation must equal
    the one-call result bit for bit (counts, offsets, indices, pairs, Y)."""
    dev = torch.device("cuda", 0)
    w = synth.make("large", batch=7)                     # dynamic ratio, 4 + 3 images
    fields = {k: (int(v) if k in ("dynamic", "iters") else float(v)) for k, v in w.params.items()}

    def run(X, offsets, rho):
        batch, total = len(offsets) - 1, X.shape[0]
        plan = binding.Plan(w.d, X.dtype, batch, total, w.max_tokens, device=dev)
        rho_dev = torch.from_numpy(rho.copy()).to(dev)
        out = binding.Outputs.allocate(total, batch, w.d, X.dtype, dev)
        plan.run(X.to(dev), torch.from_numpy(offsets.copy()).to(dev), binding.make_params(rho_dev, **fields), out)
        assert plan.query_status() == 0
        plan.close()
        return binding.Outputs(**{k: getattr(out, k).cpu() for k in out.__dataclass_fields__})

    whole = run(w.X, w.offsets, w.rho)
    parts, kept_rows = [], []
    for rank in range(2):
        (lo, hi), (row_lo, row_hi), local_offsets = binding.shard_slice(w.offsets, 2, rank)
        parts.append(((lo, hi), (row_lo, row_hi), run(w.X[row_lo:row_hi], local_offsets, w.rho[lo:hi])))
        kept_rows.append(int(parts[-1][2].out_offsets[hi - lo]))
    assert parts[0][0] == (0, 4) and parts[1][0] == (4, 7)
    nb = w.batch
    total_kept = int(whole.out_offsets[nb])
    assert sum(kept_rows) == total_kept
    counts = torch.cat([p[2].counts[:p[0][1] - p[0][0]] for p in parts])
    assert torch.equal(counts, whole.counts[:nb])
    offs = torch.cat([parts[0][2].out_offsets[:4] + binding.packed_row_base(kept_rows, 0),
                      parts[1][2].out_offsets[:4] + binding.packed_row_base(kept_rows, 1)])
    assert torch.equal(offs, whole.out_offsets[:nb + 1])
    Y = torch.cat([p[2].Y[:k] for p, k in zip(parts, kept_rows)])
    assert torch.equal(Y, whole.Y[:total_kept])
    kept_idx = torch.cat([p[2].kept_idx[:k] for p, k in zip(parts, kept_rows)])
    assert torch.equal(kept_idx, whole.kept_idx[:total_kept])
    pruned = [(p[1][1] - p[1][0]) - k for p, k in zip(parts, kept_rows)]
    for name in ("merged_idx", "merge_partner"):
        got = torch.cat([getattr(p[2], name)[:n] for p, n in zip(parts, pruned)])
        assert torch.equal(got, getattr(whole, name)[:sum(pruned)]), name
