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
