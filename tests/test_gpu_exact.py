"""Exact pairing mode (the linear program of Eq. 2-6 solved on the device) against the oracle's exact solver:
objective value, validity of the matching, hard-pair merge (Eq. 7).  Marked gpu."""
import pytest
import torch

from paper_2605_00392_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def parity():
    import parity as _p
    return _p


def test_tiny(parity):
    rep = parity.check_exact(synth.make("tiny"))
    assert rep["launches"] == 5                 # stage 1, gather, scores, exact pairing, merge
    assert rep["pruned"] == 16


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_ragged(parity, dtype):
    w = synth.ragged([1, 2, 3, 5, 63, 64, 65, 127, 129, 400, 1], dtype=dtype, params=dict(r_fixed=0.3))
    rep = parity.check_exact(w)
    assert rep["pairs"] > 0


def test_more_pruned_than_kept(parity):
    # B > M: the kept side is the one inserted token by token
    w = synth.ragged([10, 90, 257, 400], params=dict(r_fixed=0.7))
    rep = parity.check_exact(w)
    assert 0 < rep["pairs"] <= 3 + 27 + 77 + 120


@pytest.mark.parametrize("z", [0.2, 0.0, 0.9, -0.5])
def test_dustbin_score(parity, z):
    # a higher dustbin score leaves more tokens unpaired; below every cosine all of the smaller side is paired
    w = synth.ragged([75, 150], params=dict(r_fixed=0.25, z=z))
    rep = parity.check_exact(w)
    assert rep["pruned"] == 19 + 38
    if z == -0.5:
        assert rep["pairs"] == rep["pruned"]
    if z == 0.9:
        assert rep["pairs"] < rep["pruned"]


def test_named_batches(parity):
    parity.check_exact(synth.make("base", batch=8))
    parity.check_exact(synth.make("large", batch=12))


def test_large_image(parity):
    # gains too many for shared memory: the search reads the workspace tile
    w = synth.ragged([1156], params=dict(r_fixed=0.5))
    rep = parity.check_exact(w)
    assert rep["pruned"] == 578
