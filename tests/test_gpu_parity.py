"""GPU-vs-oracle parity on the five configurations, through the C ABI.  Marked gpu."""
import numpy as np
import pytest
import torch

from paper_2605_00392_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def parity():
    import parity as _p
    return _p


def test_tiny(parity):
    rep = parity.check_workload(synth.make("tiny"))
    assert rep["mean_retention"] == 0.75 and rep["launches"] == 5
    # Gaussian directions: no near-duplicate tokens, so (nearly) every pair is decisive and held to bit-exactness
    assert rep["bit_exact_pair_share"] >= 0.9


def test_base(parity):
    rep = parity.check_workload(synth.make("base"))
    assert 0.6 < rep["mean_retention"] < 1.0


def test_large_full_batch(parity):
    rep = parity.check_workload(synth.make("large"))
    assert abs(rep["mean_retention"] - 0.8425) < 0.01       # the retention the paper reports
    assert rep["max_partner_regret"] <= 5e-5 and rep["pairs"] > 3000


def test_gundam_ragged(parity):
    # every one of the 128 ragged images against the oracle
    w = synth.make("gundam")
    rep = parity.check_workload(w)
    assert rep["images_compared"] == 128


@pytest.fixture(scope="module")
def sweep_batch():
    return synth.make("sweep")


@pytest.mark.parametrize("r_fixed", [0.5, 0.35, 0.2, 0.05, None])
def test_sweep_1024(parity, sweep_batch, r_fixed):
    w = sweep_batch
    if r_fixed is None:
        over = dict(synth.DYNAMIC_PARAMS)
    else:
        over = dict(dynamic=0, r_fixed=r_fixed, phi_lo=0.0, phi_hi=1.0, r_max=1.0)
    rep = parity.check_workload(w, overrides=over)       # all 1024 images against the oracle
    assert rep["images_compared"] == 1024
    if r_fixed is not None:
        assert abs(rep["mean_retention"] - (1.0 - r_fixed)) < 1e-9


def test_sweep_fp32(parity):
    w = synth.make("sweep_fp32")
    assert w.X.dtype == torch.float32
    rep = parity.check_workload(w)                        # all 256 images, dynamic ratio
    assert rep["images_compared"] == 256
    rep = parity.check_workload(w, overrides=dict(dynamic=0, r_fixed=0.35, phi_lo=0.0, phi_hi=1.0, r_max=1.0))
    assert rep["images_compared"] == 256


def test_host_buffer_path_matches(parity):
    w = synth.make("base", batch=4)
    parity.check_workload(w, host_path=True)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_known_pairing_is_recovered(parity, dtype):
    """Images whose answer is known by construction (pruned tokens are low-norm noisy copies of kept tokens):
    every pair is decisive, so the whole pair output is held to bit-exactness against the oracle, and the
    partners are the anchors the generator used."""
    d = 1280 if dtype == torch.bfloat16 else 256
    w, truth = synth.paired([400] * 6 + [64, 100, 37, 256], 0.25, d=d, dtype=dtype)
    rep = parity.check_workload(w)
    assert rep["bit_exact_pair_share"] == 1.0 and rep["pairs"] == 6 * 100 + 16 + 25 + 9 + 64
    g = parity.run_gpu(w).out
    for i, echo_of in enumerate(truth):
        o0 = int(g.out_offsets[i])
        seg = int(w.offsets[i]) - o0
        nb = int((echo_of >= 0).sum())
        kept = g.kept_idx[o0:o0 + int(g.counts[i])].numpy()
        pruned = g.merged_idx[seg:seg + nb].numpy()
        partner = g.merge_partner[seg:seg + nb].numpy()
        np.testing.assert_array_equal(kept[partner], echo_of[pruned])
