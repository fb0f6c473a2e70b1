#!/usr/bin/env python
"""Benchmark of the RTPrune pruning path on B200.

A step is one pass of the whole path (norms + statistics -> ratio -> top-M -> cosine scores ->
Sinkhorn -> merge + pack) over one synthetic DeepSeek-OCR-Large-shaped batch: 64 images x 400 tokens
x 1280 bf16, dynamic ratio with mean retention ~0.84.  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--repeats R] [--impl reference]

N > 1 runs one rank per GPU under torch.distributed.run (started by the caller, or by bench.py itself when
it is run plainly with --gpus N); images are independent, so every rank prunes its own batch and there is no
data-path collective (weak scaling).  The K-step region is timed R times; `value` is the median region.
--impl reference times the fp64 CPU oracle on the host cores instead (a deliberately slow program).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

WORKLOAD = "large"
WORKLOAD_DESC = "large: 64 images x 400 tokens x 1280 bf16, dynamic ratio (mean retention 0.84), T=100"
ROTATE = 4                 # input/output buffer sets cycled so that no step finds its input in L2
FP32_FMA_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12   # SMs x FP32 lanes x 2 flop x max SM clock
REFERENCE_SAMPLE = 64      # images per step of the --impl reference arm: the whole Large batch, as cpu_baseline
# dram__bytes_read.sum + dram__bytes_write.sum per launch from an ncu capture (profiles/), by kernel
# (kernels changed since their capture, or never captured, have no entry and report null)
NCU_TRAFFIC_BYTES = {"stage1": 66078208, "gather": 10355200, "scores": 87525888, "sinkhorn_reg": 4935424,
                     "merge": 118104064, "density_tile": 318402048}


def cpu_threads() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return os.cpu_count() or 1


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            pk = json.load(f)
        return float(pk["hbm_gbs"]), float(pk.get("bf16_tflops_sustained", pk["bf16_tflops"])), "measured"
    return 6650.0, 1400.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) >= 6:
                self.rows.append(parts)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        if self.thread:
            self.thread.join(timeout=2)
        sm = [float(r[0]) for r in self.rows if r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for k, n in enumerate(names) if any(r[2 + k] == "Active" for r in self.rows)]
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": reasons,
                "samples": len(self.rows)}


def time_oracle(w, images, threads):
    from oracle import oracle
    p = w.params
    op = oracle.Params(dynamic=bool(p["dynamic"]), r_fixed=p["r_fixed"], phi_lo=p["phi_lo"],
                       phi_hi=p["phi_hi"], r_max=p["r_max"], z=p["z"], alpha=p["alpha"],
                       eps=p["eps"], iters=int(p["iters"]))
    X = w.X_f64()
    t0 = time.perf_counter()
    oracle.run_batch(X, w.offsets, op, w.rho, images=images, threads=threads)
    return time.perf_counter() - t0


def run_reference(args, rank: int) -> None:
    """The oracle as it stands, on the host cores: rank 0 only."""
    if rank != 0:
        return
    from paper_2605_00392_b200 import synth
    threads = cpu_threads()
    w = synth.make(WORKLOAD, batch=REFERENCE_SAMPLE)
    images = list(range(REFERENCE_SAMPLE))
    for _ in range(args.warmup):
        time_oracle(w, images, threads)
    t = 0.0
    for _ in range(args.steps):
        t += time_oracle(w, images, threads)
    ms = 1e3 * t / max(args.steps, 1)
    value = REFERENCE_SAMPLE / (ms / 1e3)
    sample = "all %d images of the Large batch per step, all host cores" % REFERENCE_SAMPLE
    line = {"impl": "reference", "metric": "pruned images/sec", "value": value, "unit": "images/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "tokens_per_s": value * 400,
            "config": {"workload": WORKLOAD_DESC, "sample": sample},
            "cpu_baseline": {"value": value, "unit": "images/s", "cores": threads, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": "images/s", "h2d_bytes_per_step": 0,
                    "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def run_density(args) -> None:
    """`--step density`: the textual-density kernel (Eq. 9) alone, on the pages of one Large batch (64
    pages of 1280 x 1280 RGB, 8 bits per channel).  One GPU; prints one JSON line of its own."""
    print(json.dumps(density_line(args)))


def density_line(args) -> dict:
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device")
    from paper_2605_00392_b200 import binding, synth
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    batch, H, W, patch, tau = 64, 1280, 1280, synth.PAGE_PATCH, 0.2
    host = synth.pages(8, H, W, seed=1)
    sets = [torch.roll(host, k, 0).repeat(batch // 8, 1, 1, 1).contiguous().to(dev) for k in range(2)]   # 2 x 315 MB > L2
    warm = max(args.warmup, 3)
    sampler = ClockSampler(0)       # a step is 0.15 ms: the sampler runs over the warm-up and both legs
    sampler.start()
    for i in range(warm):
        binding.density(sets[i % 2], patch, tau)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda._sleep(2000000)
    e0.record()
    for i in range(args.steps):
        binding.density(sets[i % 2], patch, tau)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    # end to end from pinned host pages: copy in, kernel, rho back
    pinned = sets[0].cpu().pin_memory()
    stage = torch.empty_like(sets[0])
    rho_host = torch.empty(batch, dtype=torch.float32).pin_memory()
    e2e_steps = max(3, min(args.steps, 20))
    torch.cuda.synchronize()
    e0.record()
    for i in range(e2e_steps):
        stage.copy_(pinned, non_blocking=True)
        rho, _, _ = binding.density(stage, patch, tau)
        rho_host.copy_(rho, non_blocking=True)
    e1.record()
    torch.cuda.synchronize()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps
    clocks = sampler.stop()
    hbm_peak, _, src = measured_peaks()
    nbytes = batch * H * W * 3
    line = {"metric": "pages/sec (textual density)", "value": batch / ms * 1e3, "unit": "images/s", "n_gpus": 1,
            "steps": args.steps, "warmup": warm, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "u8 -> int64 (exact)", "data": "synthetic",
            "config": {"workload": "density: 64 pages x 1280 x 1280 x RGB8, patch 64, tau 0.2",
                       "l2": "pages rotate over 2 buffer sets (629 MB > L2)"},
            "roofline": {"kernel": "density_tile", "bound": "hbm", "achieved": nbytes / ms / 1e6, "peak": hbm_peak,
                         "unit": "GB/s", "frac": nbytes / ms / 1e6 / hbm_peak, "peak_source": src,
                         "traffic": NCU_TRAFFIC_BYTES["density_tile"]},
            "e2e": {"value": batch / e2e_ms * 1e3, "unit": "images/s", "h2d_bytes_per_step": nbytes,
                    "d2h_bytes_per_step": 4 * batch, "ms_per_step": e2e_ms},
            "gpu_launches": 2 * args.steps, "clocks": clocks}
    if not args.no_cpu_baseline:
        from oracle import density as od
        sample = host[:4].numpy()
        t0 = time.perf_counter()
        od.density_batch(sample, patch, float(np.float32(tau)))
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": len(sample) / dt, "unit": "images/s", "cores": 1, "kind": "oracle",
                                "sample": "4 pages of the batch, numpy fp64, one thread"}
    return line


LARGE_N = {   # token counts before -> after pruning of the OCR models with large visual token sets (the paper's
              # cross-model table); the fixed ratio is 1 - after / before
    "2137": dict(tokens=2137, kept=1238, batch=16),
    "4512": dict(tokens=4512, kept=2783, batch=8),
}


def run_large_n(args) -> None:
    """`--step largen`: the whole path on images of thousands of tokens (score tiles of 4 to 19 MB that
    no cluster's shared memory holds: the Sinkhorn kernel for wide tiles).  One GPU; one JSON line with
    one entry per shape."""
    print(json.dumps(large_n_line(args)), flush=True)


def large_n_line(args) -> dict:
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the pruning path has no CPU fallback")
    from paper_2605_00392_b200 import binding, synth
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    hbm_peak, _, peak_kind = measured_peaks()
    steps, warm = max(1, min(args.steps, 30)), max(args.warmup, 3)
    shapes = {}
    for name, cfg in LARGE_N.items():
        n, batch = cfg["tokens"], cfg["batch"]
        r = float(np.float32(1.0 - cfg["kept"] / n))
        w = synth.ragged([n] * batch, seed=21, params=dict(r_fixed=r))
        plan = binding.Plan(w.d, w.X.dtype, w.batch, w.total_tokens, w.max_tokens, device=dev)
        fields = {k: (int(v) if k in ("dynamic", "iters") else float(v)) for k, v in w.params.items()}
        params = binding.make_params(None, **fields)
        out = binding.Outputs.allocate(w.total_tokens, w.batch, w.d, w.X.dtype, dev)
        X, offs = w.X.to(dev), torch.from_numpy(w.offsets.copy()).to(dev)
        flush = torch.empty(160 << 20, dtype=torch.uint8, device=dev)      # larger than L2
        for _ in range(warm):
            plan.run(X, offs, params, out)
        torch.cuda.synchronize()
        assert plan.query_status() == 0
        plan.profile_enable(True)
        total_ms, per_kernel = 0.0, {}
        for _ in range(steps):
            flush.zero_()                                  # no step finds its input in L2
            plan.run(X, offs, params, out)
            for kname, ms in plan.profile_read():
                per_kernel.setdefault(kname, []).append(ms)
                total_ms += ms
        plan.profile_enable(False)
        st = out.stats.cpu().numpy()[:batch]
        M, B, it = st[:, 3].astype(np.int64), st[:, 4].astype(np.int64), st[:, 5]
        avg = {k: float(np.mean(v)) for k, v in per_kernel.items()}
        ms_step = total_ms / steps
        # the wide-tile Sinkhorn kernel must read K (M rows of pitch (B+4)&~3 floats) once per iteration
        k_bytes = float(np.sum(it * M * ((B + 4) & ~3) * 4))
        tall_ms = avg.get("sinkhorn_tall", 0.0)
        path_bytes = w.total_tokens * w.d * 2 + int(M.sum()) * w.d * 2 + 12 * w.total_tokens
        shapes[name] = {
            "workload": "%d images x %d tokens x %d bf16, fixed r = %.4f (%d kept), T=100" % (batch, n, w.d, r, int(M[0])),
            "ms_per_step": ms_step, "images_per_s": batch / (ms_step / 1e3),
            "tokens_per_s": w.total_tokens / (ms_step / 1e3), "kernel_ms": avg,
            "mean_iterations_run": float(it.mean()), "max_iterations_run": float(it.max()),
            "roofline": {"kernel": "sinkhorn_tall", "bound": "hbm", "achieved": k_bytes / (tall_ms / 1e3) / 1e9 if tall_ms else None,
                         "peak": hbm_peak, "unit": "GB/s", "frac": k_bytes / (tall_ms / 1e3) / 1e9 / hbm_peak if tall_ms else None,
                         "peak_source": peak_kind, "traffic": None, "avg_launch_ms": tall_ms,
                         "note": "bytes = executed iterations x the image's K tile; the tiles of a batch stay in L2 when they fit"},
            "path_roofline": {"bound": "hbm", "algorithmic_bytes": path_bytes,
                              "frac": path_bytes / (ms_step / 1e3) / 1e9 / hbm_peak},
            "gpu_launches": plan.last_launch_count * steps,
        }
        if name == "2137" and not args.no_cpu_baseline:
            threads = cpu_threads()
            sec = time_oracle(w, list(range(batch)), threads)
            shapes[name]["cpu_baseline"] = {"value": batch / sec, "unit": "images/s", "cores": threads, "kind": "oracle",
                                            "sample": "all %d images of this batch, once" % batch}
        plan.close()
    return {"metric": "pruned images/sec", "unit": "images/s", "n_gpus": 1, "steps": steps, "warmup": warm,
            "higher_is_better": True, "dtype": "bf16", "data": "synthetic",
            "timing": "sum of the kernels' CUDA-event times per step, L2 flushed between steps",
            "shapes": shapes}


def sweep_line(w0, steps: int, warm: int) -> dict:
    """1024 images x 400 tokens (the Large batch tiled 16 times on the device: 1.05 GB of tokens, far beyond L2):
    the batch on which the path's HBM bound can be approached.  One GPU."""
    from paper_2605_00392_b200 import binding
    dev = torch.device("cuda", 0)
    reps = 16
    batch, total, d = w0.batch * reps, w0.total_tokens * reps, w0.d
    X = w0.X.to(dev).repeat(reps, 1)
    lens = np.tile(np.diff(w0.offsets.astype(np.int64)), reps)
    offs = torch.from_numpy(np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)).to(dev)
    rho = torch.from_numpy(np.tile(w0.rho, reps)).to(dev)
    fields = {k: (int(v) if k in ("dynamic", "iters") else float(v)) for k, v in w0.params.items()}
    params = binding.make_params(rho, **fields)
    plan = binding.Plan(d, torch.bfloat16, batch, total, w0.max_tokens, device=dev)
    out = binding.Outputs.allocate(total, batch, d, torch.bfloat16, dev)
    for _ in range(warm):
        plan.run(X, offs, params, out)
    torch.cuda.synchronize()
    assert plan.query_status() == 0
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        plan.run(X, offs, params, out)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    kept = int(out.out_offsets[batch])
    launches = plan.last_launch_count
    plan.close()
    hbm_peak, _, peak_kind = measured_peaks()
    path_bytes = total * d * 2 + kept * d * 2 + 12 * total
    return {"workload": "sweep: %d images x 400 tokens x %d bf16 (the Large batch tiled %d times), dynamic ratio, T=100"
                        % (batch, d, reps),
            "ms_per_step": ms, "images_per_s": batch / (ms / 1e3), "steps": steps, "gpu_launches": launches * steps,
            "path_roofline": {"bound": "hbm", "algorithmic_bytes": path_bytes, "achieved": path_bytes / (ms / 1e3) / 1e9,
                              "peak": hbm_peak, "unit": "GB/s", "frac": path_bytes / (ms / 1e3) / 1e9 / hbm_peak,
                              "peak_source": peak_kind}}


def accuracy_against_oracle(w, out, threads: int) -> dict:
    """Part of the cpu_baseline leg: the oracle's results for the timed batch against the device's (set 0 of the
    rotation), as the figures the parity tests bound: largest feature error |y - y*| / max(|y*|, rms(y* row)), largest
    regret of a chosen partner in log P below the oracle's column maximum, and whether every index output agrees."""
    from oracle import oracle
    p = w.params
    op = oracle.Params(dynamic=bool(p["dynamic"]), r_fixed=p["r_fixed"], phi_lo=p["phi_lo"], phi_hi=p["phi_hi"],
                       r_max=p["r_max"], z=p["z"], alpha=p["alpha"], eps=p["eps"], iters=int(p["iters"]))
    refs = oracle.run_batch(w.X_f64(), w.offsets, op, w.rho, threads=threads, want_plan=True).images
    Y = out.Y.cpu().to(torch.float64).numpy()
    oo = out.out_offsets.cpu().numpy()
    kept_idx, merged_idx = out.kept_idx.cpu().numpy(), out.merged_idx.cpu().numpy()
    partner = out.merge_partner.cpu().numpy()
    worst_feature, worst_regret, indices_equal = 0.0, 0.0, True
    for i, ref in enumerate(refs):
        o0, o1 = int(oo[i]), int(oo[i + 1])
        seg = int(w.offsets[i]) - o0
        indices_equal &= (o1 - o0 == ref.M and np.array_equal(kept_idx[o0:o1], ref.kept)
                          and np.array_equal(merged_idx[seg:seg + ref.B], ref.prop))
        if o1 - o0 != ref.M:
            continue
        rms = np.sqrt(np.mean(ref.Y * ref.Y, axis=1, keepdims=True))
        denom = np.maximum(np.abs(ref.Y), rms)
        worst_feature = max(worst_feature, float((np.abs(Y[o0:o1] - ref.Y) / np.where(denom > 0, denom, 1.0)).max()))
        if ref.B:
            logP = np.log(ref.Pbar[:-1, :-1])
            gp = np.clip(partner[seg:seg + ref.B], 0, ref.M - 1)
            worst_regret = max(worst_regret, float((logP.max(axis=0) - logP[gp, np.arange(ref.B)]).max()))
    return {"images": len(refs), "indices_equal": bool(indices_equal), "max_feature_err": worst_feature,
            "max_partner_regret": worst_regret}


def self_launch(args) -> None:
    """`python bench.py --gpus N` outside torch.distributed.run: start the N ranks (one per GPU) on this node."""
    import socket
    import tempfile
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    env = dict(os.environ)
    if "NCCL_DEBUG" not in env:      # the communicator's log (transports, NVLS) goes to a file, not into the JSON line
        env["NCCL_DEBUG"] = "INFO"
        env["NCCL_DEBUG_FILE"] = os.path.join(tempfile.gettempdir(), "rtprune_bench_nccl_%h_%p.log")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    sys.stdout.flush()
    os.execve(sys.executable, cmd, env)


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--step", default="prune", choices=["prune", "density", "largen"],
                    help="prune: the pruning path (the headline); density: the textual-density kernel alone; "
                         "largen: the pruning path on images of 2137 and 4512 tokens")
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--repeats", type=int, default=10, help="how many times the K-step region is timed")
    ap.add_argument("--schedule", default="auto", choices=["auto", "separate", "fused"],
                    help="which kernels carry out stage 2 (rtprune_schedule_t); auto is the library's choice")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the one-shot summaries of the other workloads (density, large N, 1024 images)")
    args = ap.parse_args()
    if args.gpus > 1 and args.impl == "ours" and args.step == "prune" and "WORLD_SIZE" not in os.environ:
        self_launch(args)

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.step == "density":
        if rank == 0:
            run_density(args)
        return
    if args.step == "largen":
        if rank == 0:
            run_large_n(args)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the pruning path has no CPU fallback")
    import torch.distributed as dist
    from paper_2605_00392_b200 import binding, synth

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    # ---- workload: every rank prunes its own Large batch (independent images, no exchange) --------
    sets = []
    w0 = None
    for s in range(ROTATE):
        w = synth.make(WORKLOAD, seed_offset=rank * ROTATE + s)
        if w0 is None:
            w0 = w
        sets.append(w)
    batch, total, d = w0.batch, w0.total_tokens, w0.d
    plan = binding.Plan(d, torch.bfloat16, batch, total, w0.max_tokens, device=dev)
    fields = {k: (int(v) if k in ("dynamic", "iters") else float(v)) for k, v in w0.params.items()}
    fields["schedule"] = {"auto": binding.SCHEDULE_AUTO, "separate": binding.SCHEDULE_SEPARATE,
                          "fused": binding.SCHEDULE_FUSED}[args.schedule]
    dev_sets = []
    for w in sets:
        rho = torch.from_numpy(w.rho).to(dev)
        dev_sets.append(dict(X=w.X.to(dev), offs=torch.from_numpy(w.offsets).to(dev), rho=rho,
                             params=binding.make_params(rho, **fields),
                             out=binding.Outputs.allocate(total, batch, d, torch.bfloat16, dev)))
    stream = torch.cuda.current_stream()

    def step(i: int) -> None:
        s = dev_sets[i % ROTATE]
        plan.run(s["X"], s["offs"], s["params"], s["out"])

    def barrier() -> None:
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(args.warmup, 3)):
        step(i)
    barrier()
    assert plan.query_status() == 0

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    # ---- timed region: K steps back to back, CUDA events on the launching stream; R such regions --
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    repeats = max(1, args.repeats)
    region_ms = []
    for _ in range(repeats):
        barrier()
        torch.cuda._sleep(2000000)     # about 1 ms: the host is ahead of the device when the timed region starts
        e0.record(stream)
        for i in range(args.steps):
            step(i)
        e1.record(stream)
        barrier()
        region_ms.append(e0.elapsed_time(e1))
    launches = plan.last_launch_count * args.steps

    # ---- host time of a call: the library's own clock around rtprune_run, and the binding's on top ----
    barrier()
    host_ns = []
    t_host = time.perf_counter()
    for i in range(50):
        step(i)
        host_ns.append(plan.last_host_ns)
    t_host = (time.perf_counter() - t_host) / 50
    barrier()

    # ---- the same K steps as replays of CUDA graphs (one captured step per buffer set) -------------
    side = torch.cuda.Stream(device=dev)
    side.wait_stream(stream)
    graphs = []
    with torch.cuda.stream(side):
        step(0)
    stream.wait_stream(side)
    torch.cuda.synchronize()
    for k in range(ROTATE):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            step(k)
        graphs.append(g)
    for i in range(3):
        graphs[i % ROTATE].replay()
    barrier()
    e0.record(stream)
    for i in range(args.steps):
        graphs[i % ROTATE].replay()
    e1.record(stream)
    barrier()
    ms_graph = e0.elapsed_time(e1) / args.steps
    t_host_graph = time.perf_counter()
    for i in range(50):
        graphs[i % ROTATE].replay()
    t_host_graph = (time.perf_counter() - t_host_graph) / 50
    barrier()
    assert plan.query_status() == 0

    # ---- the same K steps with every image running all T iterations (no exit at the fixed point) --
    for s_ in dev_sets:
        s_["params_all"] = binding.make_params(s_["rho"], **dict(fields, stop_at_fixed_point=0))
    for i in range(3):
        plan.run(dev_sets[i % ROTATE]["X"], dev_sets[i % ROTATE]["offs"], dev_sets[i % ROTATE]["params_all"],
                 dev_sets[i % ROTATE]["out"])
    barrier()
    e0.record(stream)
    for i in range(args.steps):
        s_ = dev_sets[i % ROTATE]
        plan.run(s_["X"], s_["offs"], s_["params_all"], s_["out"])
    e1.record(stream)
    barrier()
    ms_all_iters = e0.elapsed_time(e1) / args.steps
    step(0)                            # set 0 holds the default run's outputs again (read below)
    barrier()

    # ---- same steps again with per-kernel events (feeds the roofline of the dominant kernel) -----
    plan.profile_enable(True)
    per_kernel = {}
    nprof = min(args.steps, 50)
    for i in range(nprof):
        torch.cuda._sleep(300000)      # the host gets ahead: no launch gaps inside the measured kernels
        step(i)
        for name, ms in plan.profile_read():
            per_kernel.setdefault(name, []).append(ms)
    plan.profile_enable(False)
    clocks = sampler.stop() if rank == 0 else None

    # ---- end to end through the host-buffer entry point ------------------------------------------
    # Two plans (each with its own device arena) on two streams take the steps in turn, the way a caller
    # with a queue of batches would: the upload of a step's inputs then runs while the step before it is
    # still downloading its outputs (the two directions of the link).  Every copy of every step, both
    # directions, is inside the timed region; each stream writes host outputs of its own.
    E2E_STREAMS = 2
    plans2 = [plan] + [binding.Plan(d, torch.bfloat16, batch, total, w0.max_tokens, device=dev)
                       for _ in range(E2E_STREAMS - 1)]
    streams2 = [torch.cuda.Stream(device=dev) for _ in range(E2E_STREAMS)]
    host_outs = [binding.Outputs.allocate(total, batch, d, torch.bfloat16, "cpu", pin=True)
                 for _ in range(E2E_STREAMS)]
    host_out = host_outs[0]
    hX = [w.X.pin_memory() for w in sets]
    hoffs = [torch.from_numpy(w.offsets).pin_memory() for w in sets]
    hrho = [torch.from_numpy(w.rho).pin_memory() for w in sets]
    hparams = binding.make_params(None, **fields)
    e2e_steps = 1 if args.no_e2e else max(4, min(args.steps, 20))

    def e2e_step(i: int) -> None:
        k = i % E2E_STREAMS
        plans2[k].run_host(hX[i % ROTATE], hoffs[i % ROTATE], hrho[i % ROTATE], hparams, host_outs[k],
                           stream=streams2[k])

    for i in range(0 if args.no_e2e else 2 * E2E_STREAMS):
        e2e_step(i)
    barrier()
    e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2.record(stream)
    for st2 in streams2:
        st2.wait_event(e2)
    for i in range(e2e_steps):
        e2e_step(i)
    for st2 in streams2:
        stream.wait_stream(st2)
    e3.record(stream)
    barrier()
    ms_e2e = e2.elapsed_time(e3) / e2e_steps

    # ---- device-resident steps again, two batches in flight (the same two plans and streams): the
    # latency-bound stretches of one batch run under the bandwidth-bound stretches of the other.
    # Reported beside `value`, which stays the one-stream figure.
    def step2(i: int) -> None:
        sset = dev_sets[i % ROTATE]
        k = i % E2E_STREAMS
        plans2[k].run(sset["X"], sset["offs"], sset["params"], outs2[k], stream=streams2[k])

    outs2 = [binding.Outputs.allocate(total, batch, d, torch.bfloat16, dev) for _ in range(E2E_STREAMS)]
    for i in range(2 * E2E_STREAMS):
        step2(i)
    barrier()
    e4, e5 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda._sleep(2000000)
    e4.record(stream)
    for st2 in streams2:
        st2.wait_event(e4)
    for i in range(args.steps):
        step2(i)
    for st2 in streams2:
        stream.wait_stream(st2)
    e5.record(stream)
    barrier()
    ms_two = e4.elapsed_time(e5) / args.steps
    for pl2 in plans2[1:]:
        assert pl2.query_status() == 0
        pl2.close()
    kept_total = int(host_out.out_offsets[batch])
    esz = 2
    h2d = total * d * esz + (batch + 1) * 4 + batch * 4
    d2h = total * d * esz + (batch + 1) * 4 + batch * 4 + 4 * total * 4 + batch * 8 * 4

    # ---- max over ranks ---------------------------------------------------------------------------
    t = torch.tensor([ms_e2e, ms_two, ms_all_iters] + region_ms, dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms_e2e, ms_two, ms_all_iters = float(t[0]), float(t[1]), float(t[2])
    region_ms = sorted(float(x) for x in t[3:])
    ms_total = float(np.median(region_ms))           # `value` is the median region (max over ranks of each)
    ms_step = ms_total / args.steps
    images_s = world * batch / (ms_step / 1e3)
    e2e_images_s = world * batch / (ms_e2e / 1e3)

    if rank == 0:
        hbm_peak, tensor_peak, peak_kind = measured_peaks()
        stats = dev_sets[0]["out"].stats.cpu().numpy()[:batch]
        M = stats[:, 3].astype(np.int64)
        B = stats[:, 4].astype(np.int64)
        iters_run = stats[:, 5]
        sumM, sumMB = int(M.sum()), int((M * B).sum())
        avg = {k: float(np.mean(v)) for k, v in per_kernel.items()}
        dominant = max(avg, key=avg.get)
        x_bytes = total * d * esz
        y_bytes = sumM * d * esz
        sink_flops = float(np.sum(iters_run * 2 * 2 * (M + 1) * (B + 1)))
        xp_bytes = int(B.sum()) * d * esz
        algo = {   # algorithmic bytes / flops per launch, by kernel
            "stage1": ("hbm", x_bytes + total * 4 * 3 + batch * 48),
            "gather": ("hbm", 2 * xp_bytes),
            "scores": ("hbm", x_bytes + xp_bytes + 4 * sumMB),
            "sinkhorn_cluster": ("alu", sink_flops),
            "sinkhorn_wide": ("alu", sink_flops),
            "sinkhorn_reg": ("alu", sink_flops),
            "sinkhorn": ("alu", sink_flops),
            "merge": ("hbm", x_bytes + y_bytes + sumM * 4),
            # scores, Sinkhorn and merge in one kernel: it must read X and write Y, the pairs and the indices
            "stage2_fused": ("hbm", x_bytes + y_bytes + 16 * total),
        }
        bound, units = algo[dominant]
        dur_s = avg[dominant] / 1e3
        if bound == "hbm":
            achieved, peak, unit = units / dur_s / 1e9, hbm_peak, "GB/s"
        else:
            achieved, peak, unit = units / dur_s / 1e12, FP32_FMA_PEAK_TFLOPS, "TFLOP/s"
        path_bytes = x_bytes + y_bytes + 12 * total
        # the same figures for every kernel of the step (the per-kernel times come from events between the
        # kernels, which serialise them: in the timed steps above they overlap)
        per_kernel_roofline = {}
        for name, t_ms in avg.items():
            kb, ku = algo[name]
            ach = ku / (t_ms / 1e3) / (1e9 if kb == "hbm" else 1e12)
            pk = hbm_peak if kb == "hbm" else FP32_FMA_PEAK_TFLOPS
            per_kernel_roofline[name] = {"bound": kb, "achieved": ach, "unit": "GB/s" if kb == "hbm" else "TFLOP/s",
                                         "frac": ach / pk, "avg_launch_ms": t_ms,
                                         "traffic": NCU_TRAFFIC_BYTES.get(name)}
        line = {
            "metric": "pruned images/sec", "value": images_s, "unit": "images/s",
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "tokens_per_s": images_s * total / batch,
            "repeats": {"n": repeats, "steps_each": args.steps, "value_is": "median",
                        "ms_per_step": {"median": ms_step, "min": region_ms[0] / args.steps,
                                        "max": region_ms[-1] / args.steps}},
            "all_iterations": {"ms_per_step": ms_all_iters, "value": world * batch / (ms_all_iters / 1e3),
                               "unit": "images/s", "note": "stop_at_fixed_point = 0: every image runs T = 100 iterations"},
            "host_call": {"library_us": float(np.median(host_ns)) / 1e3, "with_binding_us": t_host * 1e6,
                          "graph_replay_us": t_host_graph * 1e6,
                          "note": "host time of one rtprune_run call (5 launches), device busy; of one replay of the "
                                  "captured step"},
            "graph_replay": {"ms_per_step": ms_graph, "value": world * batch / (ms_graph / 1e3), "unit": "images/s",
                             "note": "the K steps as replays of CUDA graphs, one captured rtprune_run per buffer set"},
            "config": {"workload": WORKLOAD_DESC, "global_batch": world * batch,
                       "accumulate": "fp32", "sinkhorn": "T=100 with exit at the fixed point (no dual moves by more than 1 ulp)",
                       "mean_iterations_run": float(iters_run.mean()),
                       "mean_retention": float(sumM) / total,
                       "l2": "inputs and outputs rotate over %d buffer sets (%.0f MB > L2)"
                             % (ROTATE, ROTATE * (x_bytes + y_bytes) / 1e6),
                       "schedule": args.schedule,
                       "parallelism": "dp%d (independent images, no collective)" % world},
            "roofline": {"kernel": dominant, "bound": bound, "achieved": achieved, "peak": peak,
                         "unit": unit, "frac": achieved / peak, "peak_source": peak_kind,
                         "traffic": NCU_TRAFFIC_BYTES.get(dominant),
                         "avg_launch_ms": avg[dominant]},
            "path_roofline": {"bound": "hbm", "algorithmic_bytes": path_bytes,
                              "achieved": path_bytes / (ms_step / 1e3) / 1e9, "peak": hbm_peak,
                              "unit": "GB/s", "frac": path_bytes / (ms_step / 1e3) / 1e9 / hbm_peak,
                              "peak_source": peak_kind},
            "kernel_ms": avg,
            "kernel_rooflines": per_kernel_roofline,
            "e2e": {"value": e2e_images_s, "unit": "images/s", "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e, "kept_rows": kept_total,
                    "streams": E2E_STREAMS},
            "two_batches_in_flight": {"value": world * batch / (ms_two / 1e3), "unit": "images/s",
                                      "ms_per_step": ms_two, "streams": E2E_STREAMS},
            "gpu_launches": launches,
            "clocks": clocks,
        }
        if world == 1 and not args.no_cpu_baseline:
            threads = cpu_threads()
            sec = time_oracle(w0, list(range(batch)), threads)
            line["cpu_baseline"] = {"value": batch / sec, "unit": "images/s", "cores": threads,
                                    "kind": "oracle",
                                    "sample": "all %d images of the Large batch, once" % batch}
            line["accuracy"] = accuracy_against_oracle(w0, dev_sets[0]["out"], threads)
        if world == 1 and not args.no_extras:
            # one-shot records of the other workloads (each has a --step of its own for the full figures)
            sub = argparse.Namespace(steps=20, warmup=3, no_cpu_baseline=True)
            dl = density_line(sub)
            ln = large_n_line(argparse.Namespace(steps=5, warmup=3, no_cpu_baseline=True))
            line["also"] = {
                "density": {"workload": dl["config"]["workload"], "ms_per_step": dl["ms_per_step"],
                            "roofline_frac": dl["roofline"]["frac"]},
                "largen": {k: {"workload": v["workload"], "ms_per_step": v["ms_per_step"],
                               "path_roofline_frac": v["path_roofline"]["frac"]} for k, v in ln["shapes"].items()},
                "sweep1024": sweep_line(w0, steps=10, warm=3),
            }
        print(json.dumps(line), flush=True)
    plan.close()
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
