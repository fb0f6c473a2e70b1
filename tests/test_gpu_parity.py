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


def test_base(parity):
    rep = parity.check_workload(synth.make("base"))
    assert 0.6 < rep["mean_retention"] < 1.0


def test_large_full_batch(parity):
    rep = parity.check_workload(synth.make("large"))
    assert abs(rep["mean_retention"] - 0.8425) < 0.01       # the retention the paper reports
    assert rep["max_partner_regret"] <= 5e-5 and rep["pairs"] > 3000


def test_gundam_ragged(parity):
    w = synth.make("gundam")
    lens = np.diff(w.offsets)
    sample = sorted({int(np.argmin(lens)), int(np.argmax(lens)), 0, 5, 17, 64, 127})
    parity.check_workload(w, images=sample)


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
    rep = parity.check_workload(w, images=[0, 1, 333, 1023], overrides=over)
    if r_fixed is not None:
        assert abs(rep["mean_retention"] - (1.0 - r_fixed)) < 1e-9


def test_sweep_fp32(parity):
    w = synth.make("sweep_fp32")
    assert w.X.dtype == torch.float32
    parity.check_workload(w, images=[0, 7, 100, 255])
    parity.check_workload(w, images=[3, 200], overrides=dict(dynamic=0, r_fixed=0.35, phi_lo=0.0,
                                                             phi_hi=1.0, r_max=1.0))


def test_host_buffer_path_matches(parity):
    w = synth.make("base", batch=4)
    parity.check_workload(w, host_path=True)
