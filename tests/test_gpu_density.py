"""rtprune_density (textual density rho, Eq. 9) against the fp64 oracle, through the C ABI.  Marked gpu.

Tolerances: the per-patch and per-image edge counts are integers and must be bit-exact (the CUDA path
decides G >= tau in exact integer arithmetic; the thresholds used here are checked not to sit on a
value G can take, so the oracle's fp64 decision is the exact one too); rho is one fp32 division of
the image count: 1e-6 relative.
"""
import numpy as np
import pytest
import torch

from oracle import density as od
from paper_2605_00392_b200 import binding, synth

pytestmark = pytest.mark.gpu

DEV = torch.device("cuda", 0)


def _no_tie(tau):
    """(255000 tau)^2 is not within 1e-3 of an integer: no pixel can sit exactly on the threshold."""
    t2 = (float(np.float32(tau)) * 255000.0) ** 2
    return abs(t2 - round(t2)) > 1e-3


def _check(pages: torch.Tensor, patch: int, tau: float):
    assert _no_tie(tau) or tau == 0.0
    rho, counts, per_patch = binding.density(pages.to(DEV), patch, tau, want_patch_counts=True)
    torch.cuda.synchronize()
    ref_rho, ref_counts = od.density_batch(pages.numpy(), patch, float(np.float32(tau)))
    np.testing.assert_array_equal(per_patch.cpu().numpy(), ref_counts)
    np.testing.assert_array_equal(counts.cpu().numpy().astype(np.int64), ref_counts.sum(axis=(1, 2)))
    np.testing.assert_allclose(rho.cpu().numpy(), ref_rho, rtol=1e-6, atol=1e-9)
    return ref_rho


@pytest.mark.parametrize("patch", [16, 32, 64])
def test_small_pages_every_patch(patch):
    pages = synth.pages(3, 192, 320, seed=3)             # 3 x 5 patches of 64: not square, several tiles
    rho = _check(pages, patch, 0.2)
    assert 0.02 < rho.min() and rho.max() < 0.6


@pytest.mark.parametrize("tau", [0.1, 0.2, 0.7, 1.3, 2.9])
def test_thresholds(tau):
    rng = np.random.default_rng(4)
    noise = torch.from_numpy(rng.integers(0, 256, size=(2, 128, 128, 3), dtype=np.uint8))
    _check(noise, 32, tau)                               # white noise: gradients of every size
    _check(synth.pages(2, 128, 256, seed=5), 64, tau)


def test_large_mode_pages():
    # the Large resolution mode: 1280 x 1280 pixels = 20 x 20 token patches of 64 x 64
    frac = np.array([0.0, 0.25, 0.6, 1.0])
    pages = synth.pages(4, 1280, 1280, seed=1, text_fraction=frac)
    rho = _check(pages, 64, 0.2)
    assert rho[0] == 0.0 and np.all(np.diff(rho) > 0)    # more text patches, more edges


def test_degenerate_images():
    flat = torch.full((2, 64, 64, 3), 200, dtype=torch.uint8)
    flat[1] = 0
    rho, counts, per_patch = binding.density(flat.to(DEV), 64, 0.2, want_patch_counts=True)
    assert rho.tolist() == [0.0, 0.0] and counts.tolist() == [0, 0]
    # tau = 0: every pixel is an edge; a threshold above the largest possible magnitude: none
    pages = synth.pages(2, 128, 128, seed=8)
    rho0, c0, _ = binding.density(pages.to(DEV), 16, 0.0)
    assert rho0.tolist() == [1.0, 1.0] and c0.tolist() == [128 * 128] * 2
    rho9, c9, _ = binding.density(pages.to(DEV), 16, 6.0)                # G <= 4 sqrt(2)
    assert rho9.tolist() == [0.0, 0.0]
    # one patch per image: every side of the patch is the replicated border
    one = synth.pages(5, 64, 64, seed=9)
    _check(one, 64, 0.2)
    # a step edge along the image border rows and columns (the ring of the corner patches)
    edge = torch.full((1, 128, 128, 3), 255, dtype=torch.uint8)
    edge[0, 0, :] = 0
    edge[0, :, 127] = 0
    _check(edge, 64, 0.2)


def test_empty_batch_and_argument_errors():
    lib = binding.lib()
    z = torch.zeros((0, 64, 64, 3), dtype=torch.uint8, device=DEV)
    rho, counts, _ = binding.density(z, 64, 0.2)
    assert rho.numel() == 0
    pages = synth.pages(1, 128, 128, seed=2).to(DEV)
    with pytest.raises(binding.RtpruneError) as e:
        binding.density(pages, 48, 0.2)
    assert e.value.status == 2                                            # RTPRUNE_ERR_UNSUPPORTED
    with pytest.raises(binding.RtpruneError) as e:
        binding.density(pages[:, :96].contiguous(), 64, 0.2)             # height not a multiple of the patch
    assert e.value.status == 2
    for bad_tau in (-0.1, float("nan"), float("inf")):
        with pytest.raises(binding.RtpruneError) as e:
            binding.density(pages, 64, bad_tau)
        assert e.value.status == 1
    rho = torch.empty(1, device=DEV)
    cnt = torch.empty(1, dtype=torch.int32, device=DEV)
    status = lib.rtprune_density(None, pages.data_ptr() + 3, 1, 128, 128, 64, 0.2, rho.data_ptr(), cnt.data_ptr(), None)
    assert status == 1                                                    # misaligned images


def test_rho_feeds_the_dynamic_ratio():
    # Algorithm 1 end to end on the device: rho from the pages goes straight into rtprune_run's params
    import parity as P
    w = synth.make("base", batch=4)
    pages = synth.pages(4, 1024, 1024, seed=6)           # Base mode: 1024 x 1024 <-> 256 tokens
    rho_dev, _, _ = binding.density(pages.to(DEV), 64, 0.2)
    ref_rho, _ = od.density_batch(pages.numpy(), 64, float(np.float32(0.2)))
    np.testing.assert_allclose(rho_dev.cpu().numpy(), ref_rho, rtol=1e-6)
    w.rho[:] = rho_dev.cpu().numpy()                       # the device's rho is the input of Eq. 10 from here on
    P.check_workload(w)
