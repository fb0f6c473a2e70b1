"""Edge cases, parameter ranges and device-side error reporting of the CUDA path.  Marked gpu."""
import ctypes

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


RAGGED = [1, 2, 3, 5, 63, 64, 65, 127, 129, 400, 1]


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_ragged_lengths_fixed_ratio(parity, dtype):
    w = synth.ragged(RAGGED, dtype=dtype, params=dict(r_fixed=0.3))
    parity.check_workload(w)


def test_ragged_dynamic(parity):
    w = synth.ragged(RAGGED, params=dict(dynamic=1, phi_lo=0.0, phi_hi=0.6, r_max=0.5))
    parity.check_workload(w)


def test_retention_one_is_identity(parity):
    w = synth.ragged([7, 64, 200], params=dict(r_fixed=0.0))
    rep = parity.check_workload(w)
    assert rep["mean_retention"] == 1.0 and rep["launches"] == 2   # stage 1 + merge: stage 2 is not launched


def test_rho_one_prunes_nothing(parity):
    w = synth.ragged([50, 70], params=dict(dynamic=1, phi_hi=0.5))
    w.rho[:] = 1.0
    assert parity.check_workload(w)["mean_retention"] == 1.0


def test_single_kept_token(parity):
    w = synth.ragged([9, 40], params=dict(r_fixed=0.999))
    rep = parity.check_workload(w)
    assert rep["mean_retention"] == pytest.approx(2.0 / 49.0)


def test_alpha_zero_is_plain_pruning(parity, binding):
    w = synth.ragged([33, 90], params=dict(r_fixed=0.25, alpha=0.0))
    parity.check_workload(w)
    g = parity.run_gpu(w).out
    for i in range(2):
        o0, o1 = int(g.out_offsets[i]), int(g.out_offsets[i + 1])
        rows = w.X[int(w.offsets[i]):int(w.offsets[i + 1])][g.kept_idx[o0:o1].long()]
        assert torch.equal(g.Y[o0:o1], rows)


@pytest.mark.parametrize("over", [dict(form=1), dict(eps=0.1), dict(eps=0.3, z=0.6),
                                  dict(iters=0), dict(iters=1), dict(iters=7, stop_at_fixed_point=0),
                                  dict(z=1.0), dict(z=0.0, alpha=0.5), dict(eps=0.05, iters=300),
                                  dict(eps=0.1, form=1), dict(eps=0.05, form=2), dict(eps=0.04), dict(eps=0.02, iters=200),
                                  dict(eps=0.06, z=-1.0), dict(eps=0.25, z=4.0), dict(eps=0.25, z=-4.0)])
def test_ot_parameter_ranges(parity, over):
    w = synth.ragged([64, 150, 31], params=dict(r_fixed=0.25))
    parity.check_workload(w, overrides=over)


def test_fixed_point_stop_equals_all_iterations(parity):
    # leaving the loop at the fixed point (duals within one unit in the last place) must give what all
    # 100 iterations give, to fp32 accuracy: same pairs, weights and features equal to a few ulps
    w = synth.make("base", batch=6)
    a = parity.run_gpu(w, overrides=dict(stop_at_fixed_point=1)).out
    b = parity.run_gpu(w, overrides=dict(stop_at_fixed_point=0)).out
    assert torch.equal(a.kept_idx, b.kept_idx) and torch.equal(a.merged_idx, b.merged_idx)
    n = int(a.out_offsets[6])
    nb = int(w.offsets[6]) - n
    assert torch.equal(a.merge_partner[:nb], b.merge_partner[:nb])
    torch.testing.assert_close(a.merge_weight[:nb], b.merge_weight[:nb], rtol=2e-6, atol=0)
    ya, yb = a.Y[:n].float(), b.Y[:n].float()
    assert (ya - yb).abs().max() <= 2.0 ** -8 * yb.abs().max()      # at most one bf16 rounding apart
    assert (ya != yb).float().mean() < 1e-3
    assert float(b.stats[:6, 5].min()) == 100.0 and float(a.stats[:6, 5].max()) < 40.0


def test_tolerance_stop_runs_fewer_iterations(parity):
    w = synth.make("base", batch=4)
    a = parity.run_gpu(w, overrides=dict(tol=1e-4)).out
    assert 1.0 <= float(a.stats[:4, 5].max()) < 30.0 and float(a.stats[:4, 6].max()) <= 1e-4
    parity.check_workload(w, overrides=dict(tol=1e-6))


def test_large_tile_leaves_shared_memory(parity):
    # N = 1156 at r = 0.5: a 579 x 579 matrix (1.3 MB) that cannot stay in one CTA's shared memory
    w = synth.ragged([1156, 456], params=dict(r_fixed=0.5))
    parity.check_workload(w)


def test_tile_wider_than_the_cluster_kernel_takes(parity):
    # N = 1400 at r = 0.5: 700 pruned tokens, more than the 640 columns the cluster kernels cover, so
    # this image is solved by the kernel for wide tiles (clusters of 8 CTAs, K iterated in the workspace)
    # while the other two are solved by the two instances of the cluster kernel in the same run
    w = synth.ragged([1400, 300, 1000], params=dict(r_fixed=0.5))
    rep = parity.check_workload(w)
    assert rep["launches"] == 6      # stage1, gather, scores, sinkhorn_wide, sinkhorn_tall, merge


def test_exact_ties_keep_lower_index(parity):
    w = synth.ragged([40], params=dict(r_fixed=0.5))
    w.X[21] = w.X[3]
    w.X[30] = w.X[3]
    w.X[35] = w.X[8]
    parity.check_workload(w)
    w.X[:] = w.X[0]                      # every token identical
    g = parity.run_gpu(w).out
    assert g.kept_idx[:20].tolist() == list(range(20))
    assert g.merge_partner[:20].tolist() == [0] * 20
    parity.check_workload(w)


@pytest.mark.parametrize("d,dtype", [(8, torch.bfloat16), (64, torch.float32), (264, torch.bfloat16),
                                     (1000, torch.float32), (4096, torch.bfloat16)])
def test_other_widths(parity, d, dtype):
    w = synth.ragged([70, 33], d=d, dtype=dtype, params=dict(r_fixed=0.3))
    parity.check_workload(w)


def test_select_entry_point(parity, binding):
    w = synth.make("base", batch=3)
    parity.settle_rho(w, range(3))
    dev = torch.device("cuda", 0)
    plan = binding.Plan(w.d, w.X.dtype, 3, w.total_tokens, 256, device=dev)
    out = binding.Outputs.allocate(w.total_tokens, 3, w.d, w.X.dtype, dev)
    norms = torch.zeros(w.total_tokens, device=dev)
    order = torch.zeros(w.total_tokens, dtype=torch.int32, device=dev)
    rho = torch.from_numpy(w.rho).to(dev)
    fields = {k: (int(v) if k in ("dynamic", "iters") else float(v)) for k, v in w.params.items()}
    plan.select(w.X.to(dev), torch.from_numpy(w.offsets).to(dev), binding.make_params(rho, **fields),
                out, norms, order)
    assert plan.query_status() == 0 and plan.last_launch_count == 1
    from oracle import oracle
    ref = oracle.run_batch(w.X_f64(), w.offsets, parity.oracle_params(w.params), w.rho)
    for i, im in enumerate(ref.images):
        a = int(w.offsets[i])
        np.testing.assert_allclose(norms[a:a + 256].cpu().numpy(), im.C, rtol=2e-6)
        assert int(out.counts[i]) == im.M
        np.testing.assert_array_equal(order[a:a + im.M].cpu().numpy(), im.kept)
        np.testing.assert_array_equal(order[a + im.M:a + 256].cpu().numpy(), im.prop)
    plan.close()


def test_empty_batch(binding):
    dev = torch.device("cuda", 0)
    plan = binding.Plan(1280, torch.bfloat16, 4, 100, 50, device=dev)
    out = binding.Outputs.allocate(0, 0, 1280, torch.bfloat16, dev)
    out.out_offsets.fill_(9)
    plan.run(torch.empty((0, 1280), dtype=torch.bfloat16, device=dev),
             torch.zeros(1, dtype=torch.int32, device=dev), binding.make_params(), out)
    torch.cuda.synchronize()
    assert out.out_offsets.tolist() == [0] and plan.last_launch_count == 0
    plan.close()


def test_device_status_word(parity, binding):
    dev = torch.device("cuda", 0)
    w = synth.ragged([20, 30])
    plan = binding.Plan(w.d, w.X.dtype, 2, 50, 30, device=dev)
    out = binding.Outputs.allocate(50, 2, w.d, w.X.dtype, dev)
    X = w.X.to(dev)
    X[25, 7] = float("nan")
    offs = torch.from_numpy(w.offsets).to(dev)
    plan.run(X, offs, binding.make_params(), out)
    assert plan.query_status() & binding.DEV_NONFINITE
    assert plan.query_status() == 0                        # reading clears it
    # offsets that break the contract (image longer than the plan allows) are reported, not chased
    bad = torch.tensor([0, 45, 50], dtype=torch.int32, device=dev)
    plan.run(w.X.to(dev), bad, binding.make_params(), out)
    assert plan.query_status() & binding.DEV_BAD_OFFSETS
    # and the plan still works afterwards
    plan.run(w.X.to(dev), offs, binding.make_params(), out)
    assert plan.query_status() == 0 and int(out.out_offsets[2]) == 15 + 22
    plan.close()


def test_host_side_argument_errors(binding):
    dev = torch.device("cuda", 0)
    with pytest.raises(binding.RtpruneError) as e:
        binding.Plan(1281, torch.bfloat16, 1, 10, 10, device=dev)
    assert e.value.status == 2
    with pytest.raises(binding.RtpruneError):
        binding.Plan(1280, torch.bfloat16, 1, 10 ** 5, 9000, device=dev)
    plan = binding.Plan(1280, torch.bfloat16, 2, 100, 60, device=dev)
    out = binding.Outputs.allocate(100, 2, 1280, torch.bfloat16, dev)
    X = torch.zeros((100, 1280), dtype=torch.bfloat16, device=dev)
    offs = torch.tensor([0, 50, 100], dtype=torch.int32, device=dev)
    for bad in [dict(r_fixed=1.0), dict(r_fixed=-0.1), dict(eps=0.0), dict(iters=-1), dict(form=7),
                dict(dynamic=1, phi_lo=0.5, phi_hi=0.5), dict(dynamic=1, r_max=0.0),
                dict(form=2, eps=0.04), dict(form=2, eps=0.1, z=4.0), dict(tol=-1.0), dict(z=float("inf"))]:
        with pytest.raises(binding.RtpruneError) as e:
            plan.run(X, offs, binding.make_params(**bad), out)
        assert e.value.status == 1, bad
    with pytest.raises(binding.RtpruneError):                 # more tokens than planned
        plan.run(torch.zeros((101, 1280), dtype=torch.bfloat16, device=dev), offs,
                 binding.make_params(), out)
    with pytest.raises(binding.RtpruneError):                 # misaligned X
        lib = binding.lib()
        p = binding.make_params()
        binding._check(lib.rtprune_run(plan.handle, None, X.data_ptr() + 2, offs.data_ptr(), 2, 100,
                                       ctypes.byref(p), plan.workspace.data_ptr(),
                                       plan.workspace_bytes, out.Y.data_ptr(),
                                       out.out_offsets.data_ptr(), out.counts.data_ptr(),
                                       out.kept_idx.data_ptr(), out.merged_idx.data_ptr(),
                                       out.merge_partner.data_ptr(), out.merge_weight.data_ptr(),
                                       out.stats.data_ptr()), "rtprune_run")
    with pytest.raises(binding.RtpruneError) as e:            # workspace too small
        lib = binding.lib()
        p = binding.make_params()
        binding._check(lib.rtprune_run(plan.handle, None, X.data_ptr(), offs.data_ptr(), 2, 100,
                                       ctypes.byref(p), plan.workspace.data_ptr(), 1024,
                                       out.Y.data_ptr(), out.out_offsets.data_ptr(),
                                       out.counts.data_ptr(), out.kept_idx.data_ptr(),
                                       out.merged_idx.data_ptr(), out.merge_partner.data_ptr(),
                                       out.merge_weight.data_ptr(), out.stats.data_ptr()),
                       "rtprune_run")
    assert e.value.status == 3
    plan.close()


def test_runs_back_to_back_on_one_plan_leave_no_state(parity, binding):
    # Three workloads alternate on ONE plan and workspace without a synchronisation between the runs:
    # a batch whose images all take the fast Sinkhorn kernel (the merge kernel then follows the list of
    # finished images), a ragged one with images that prune nothing, and one at retention 1 (no stage
    # 2 at all).  Counters, the list and the unit counter in the workspace must be left as a fresh run
    # expects them: the second round must reproduce the first bit for bit, and match the oracle.
    dev = torch.device("cuda", 0)
    wa = synth.make("large", batch=6)
    wb = synth.ragged([1, 400, 2, 77, 300], params=dict(dynamic=1, phi_lo=0.0, phi_hi=0.6, r_max=0.5))
    wb.rho[3] = 1.0                                   # image 3 keeps every token
    wc = synth.ragged([64, 200, 9], params=dict(r_fixed=0.0))
    ws = [wa, wb, wc]
    plan = binding.Plan(1280, torch.bfloat16, 6, max(w.total_tokens for w in ws), 400, device=dev)
    try:
        ins, outs = [], []
        for w in ws:
            rho = torch.from_numpy(w.rho.copy()).to(dev)
            fields = {k: (int(v) if k in ("dynamic", "iters") else float(v)) for k, v in w.params.items()}
            ins.append((w.X.to(dev), torch.from_numpy(w.offsets.copy()).to(dev),
                        binding.make_params(rho, **fields), rho))
        for rnd in range(2):
            for w, (X, offs, params, _) in zip(ws, ins):
                out = binding.Outputs.allocate(w.total_tokens, w.batch, w.d, w.X.dtype, dev)
                plan.run(X, offs, params, out)
                outs.append(out)
        torch.cuda.synchronize()
        assert plan.query_status() == 0
        for k, w in enumerate(ws):
            a, b = outs[k], outs[k + 3]
            n = int(a.out_offsets[w.batch])
            nb = w.total_tokens - n
            assert torch.equal(a.out_offsets, b.out_offsets) and torch.equal(a.counts, b.counts)
            assert torch.equal(a.kept_idx[:n], b.kept_idx[:n]) and torch.equal(a.Y[:n], b.Y[:n])
            assert torch.equal(a.merged_idx[:nb], b.merged_idx[:nb])
            assert torch.equal(a.merge_partner[:nb], b.merge_partner[:nb])
            assert torch.equal(a.merge_weight[:nb], b.merge_weight[:nb])
    finally:
        plan.close()
    for w in ws:                                      # and each of them is what the oracle computes
        parity.check_workload(w)


@pytest.mark.parametrize("name,batch,bursts", [("base", 32, 40), ("large", 64, 12), ("gundam", 24, 8),
                                               ("sweep", 160, 6)])
def test_many_runs_in_bursts_reproduce_bit_for_bit(binding, name, batch, bursts):
    # The kernels of a run hand images to one another through counters and lists in the workspace while
    # later kernels of the run (programmatic dependents) may already be resident.  Bursts of runs
    # without a synchronisation, on inputs that alternate, must each reproduce the first result of
    # their input bit for bit: a kernel that reads a counter left by the run before shows up here (the
    # small batch leaves SMs free for dependents to become resident early).  The ragged batch and the batch
    # of 160 images take the cluster kernel's instance for wide tiles, which then also feeds the merge
    # kernel image by image (clusters of 4 and single CTAs, the largest tiles iterating in the workspace).
    dev = torch.device("cuda", 0)
    sets = [synth.make(name, seed_offset=s, batch=batch) for s in range(3)]
    w0 = sets[0]
    fields = {k: (int(v) if k in ("dynamic", "iters") else float(v)) for k, v in w0.params.items()}
    plan = binding.Plan(w0.d, w0.X.dtype, batch, max(s.total_tokens for s in sets),
                        max(s.max_tokens for s in sets), device=dev)
    keys = ("out_offsets", "counts", "kept_idx", "Y", "merged_idx", "merge_partner", "merge_weight")
    try:
        ins, ref = [], []
        for w in sets:
            rho = torch.from_numpy(w.rho.copy()).to(dev)
            ins.append((w, w.X.to(dev), torch.from_numpy(w.offsets.copy()).to(dev), binding.make_params(rho, **fields), rho))
            out = binding.Outputs.allocate(w.total_tokens, w.batch, w.d, w.X.dtype, dev)
            plan.run(ins[-1][1], ins[-1][2], ins[-1][3], out)
            torch.cuda.synchronize()
            ref.append(out)
        outs = [binding.Outputs.allocate(ins[j % 3][0].total_tokens, batch, w0.d, w0.X.dtype, dev) for j in range(6)]
        for _ in range(bursts):
            for j in range(6):
                plan.run(ins[j % 3][1], ins[j % 3][2], ins[j % 3][3], outs[j])
            torch.cuda.synchronize()
            for j in range(6):
                w, rf, o = ins[j % 3][0], ref[j % 3], outs[j]
                n = int(rf.out_offsets[batch])
                nb = w.total_tokens - n
                for k in keys:
                    m = n if k in ("kept_idx", "Y") else (nb if k.startswith("merge") else None)
                    a, b = getattr(o, k), getattr(rf, k)
                    assert torch.equal(a[:m] if m is not None else a, b[:m] if m is not None else b), k
                o.Y.zero_()
        assert plan.query_status() == 0
    finally:
        plan.close()
