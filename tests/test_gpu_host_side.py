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


@pytest.mark.parametrize("name,batch", [("large", 16), ("base", 32), ("ragged", 6)])
def test_run_captured_into_a_cuda_graph_replays(binding, name, batch):
    """rtprune_run captured once into a CUDA graph and replayed on changing inputs (copied into the captured
    buffers) gives, replay after replay and without a synchronisation in between, what the direct call gives
    bit for bit: the run number the kernels tell their hand-over lists by is counted on the device, not
    baked into the launches."""
    dev = torch.device("cuda", 0)
    if name == "ragged":      # tiles of up to 578 pruned tokens: the cluster kernel's instance for wide tiles
        sets = [synth.ragged([456, 1156, 700, 64, 300, 900], seed=40 + s, params=dict(r_fixed=0.5)) for s in range(3)]
    else:
        sets = [synth.make(name, seed_offset=s, batch=batch) for s in range(3)]
    total = max(s.total_tokens for s in sets)
    w0 = sets[0]
    fields = {k: (int(v) if k in ("dynamic", "iters") else float(v)) for k, v in w0.params.items()}
    plan = binding.Plan(w0.d, w0.X.dtype, batch, total, max(s.max_tokens for s in sets), device=dev)
    keys = ("out_offsets", "counts", "kept_idx", "Y", "merged_idx", "merge_partner", "merge_weight")
    try:
        # direct calls: the reference of each input set
        ref = []
        for w in sets:
            rho = torch.from_numpy(w.rho.copy()).to(dev)
            out = binding.Outputs.allocate(total, batch, w.d, w.X.dtype, dev)
            Xp = torch.zeros((total, w.d), dtype=w.X.dtype, device=dev)
            Xp[:w.total_tokens] = w.X.to(dev)
            plan.run(Xp[:w.total_tokens], torch.from_numpy(w.offsets.copy()).to(dev), binding.make_params(rho, **fields), out)
            torch.cuda.synchronize()
            ref.append(out)
        # the captured buffers (the sets of a named batch have the same token counts, so one capture serves all)
        assert all(s.total_tokens == w0.total_tokens and (s.offsets == w0.offsets).all() for s in sets)
        Xc = torch.empty((w0.total_tokens, w0.d), dtype=w0.X.dtype, device=dev)
        offs = torch.from_numpy(w0.offsets.copy()).to(dev)
        rho_c = torch.empty(batch, dtype=torch.float32, device=dev)
        params = binding.make_params(rho_c, **fields)
        out_c = binding.Outputs.allocate(total, batch, w0.d, w0.X.dtype, dev)
        Xc.copy_(sets[0].X.to(dev))
        rho_c.copy_(torch.from_numpy(sets[0].rho.copy()).to(dev))
        side = torch.cuda.Stream(device=dev)
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            plan.run(Xc, offs, params, out_c)                # warm-up on the capture stream
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            plan.run(Xc, offs, params, out_c)
        dev_in = [(s.X.to(dev), torch.from_numpy(s.rho.copy()).to(dev)) for s in sets]
        keep = [binding.Outputs.allocate(total, batch, w0.d, w0.X.dtype, dev) for _ in range(9)]
        for burst in range(4):
            for j in range(9):                               # nine replays back to back, inputs changing
                Xc.copy_(dev_in[j % 3][0])
                rho_c.copy_(dev_in[j % 3][1])
                graph.replay()
                for k in keys:
                    getattr(keep[j], k).copy_(getattr(out_c, k))
            torch.cuda.synchronize()
            for j in range(9):
                rf = ref[j % 3]
                n = int(rf.out_offsets[batch])
                nb = w0.total_tokens - n
                for k in keys:
                    m = n if k in ("kept_idx", "Y") else (nb if k.startswith("merge") else None)
                    a, b = getattr(keep[j], k), getattr(rf, k)
                    assert torch.equal(a[:m] if m is not None else a, b[:m] if m is not None else b), (burst, j, k)
        assert plan.query_status() == 0
    finally:
        plan.close()


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_stage1_gives_up_cleanly_and_recovers(parity, binding, dtype):
    """Stage 1's waits on the copies that stream X are given no polls at all: every CTA gives up although its
    copies are on their way, reports it, waits them out with the default limit, and its image passes through
    unpruned.  Nothing faults; with the default limit restored the same plan passes the parity check."""
    dev = torch.device("cuda", 0)
    w = synth.ragged([400, 37, 256, 1, 180, 129], dtype=dtype, params=dict(r_fixed=0.3))
    plan = binding.Plan(w.d, w.X.dtype, w.batch, w.total_tokens, w.max_tokens, device=dev)
    try:
        plan.set_poll_limit(0)
        fields = {k: (int(v) if k in ("dynamic", "iters") else float(v)) for k, v in w.params.items()}
        out = binding.Outputs.allocate(w.total_tokens, w.batch, w.d, w.X.dtype, dev)
        X = w.X.to(dev)
        for _ in range(2):
            plan.run(X, torch.from_numpy(w.offsets.copy()).to(dev), binding.make_params(None, **fields), out)
            assert plan.query_status() == binding.DEV_TIMEOUT
            lens = torch.from_numpy((w.offsets[1:] - w.offsets[:-1]).copy())
            assert torch.equal(out.counts.cpu()[:w.batch], lens.to(torch.int32))
            assert torch.equal(out.out_offsets.cpu(), torch.from_numpy(w.offsets.copy()))
            assert torch.equal(out.Y, X)                       # every image passed through, bit for bit
        with pytest.raises(binding.RtpruneError):
            plan.set_poll_limit(1 << 30)
        plan.set_poll_limit(-1)
        rep = parity.check_workload(w, plan=plan)
        assert rep["mean_retention"] < 0.75
    finally:
        plan.close()
