"""Pins of the textual-density oracle (Eq. 9, Appendix B) to things other than itself: closed forms on
hand-made images, the thresholds that the BT.601 weights imply, and scipy's Sobel filter."""
import numpy as np
import pytest

from oracle import density as od


def _flat(h, w, rgb):
    im = np.empty((h, w, 3), dtype=np.uint8)
    im[:] = np.array(rgb, dtype=np.uint8)
    return im


def test_uniform_page_has_no_edges_even_at_the_border():
    for rgb in [(255, 255, 255), (0, 0, 0), (13, 200, 77)]:
        rho, rho_k, counts = od.density(_flat(64, 96, rgb), 32, tau=1e-9)
        assert rho == 0.0 and counts.sum() == 0


def test_vertical_step_marks_exactly_the_two_columns_beside_it():
    # black | white: G_x = 4 on the two columns next to the step, 0 elsewhere; G_y = 0 everywhere
    H, W = 64, 128
    im = _flat(H, W, (0, 0, 0))
    im[:, 70:] = 255
    gx, gy = od.sobel(od.grayscale(im))
    assert np.all(gy == 0)
    assert np.allclose(np.abs(gx[:, 69:71]), 4.0, atol=1e-12) and np.all(gx[:, :69] == 0) and np.all(gx[:, 71:] == 0)
    rho, rho_k, counts = od.density(im, 64, tau=0.2)
    assert counts.tolist() == [[0, 2 * H]]               # columns 69 and 70 lie in the second patch
    assert rho == pytest.approx(2.0 / W)                  # = 2 H / (H W)


def test_horizontal_step_is_seen_by_g_y_alone():
    im = _flat(64, 64, (255, 255, 255))
    im[40:] = 0
    gx, gy = od.sobel(od.grayscale(im))
    assert np.all(gx == 0) and np.allclose(np.abs(gy[39:41]), 4.0, atol=1e-12)
    assert od.density(im, 64)[2].tolist() == [[2 * 64]]


def test_single_bright_pixel_lights_its_eight_neighbours():
    # responses around an isolated unit impulse: 2 at the four edge neighbours, sqrt(2) at the four
    # corner neighbours, 0 at the pixel itself
    im = _flat(32, 32, (0, 0, 0))
    im[10, 20] = 255
    gx, gy = od.sobel(od.grayscale(im))
    G = np.sqrt(gx * gx + gy * gy)
    assert G[10, 20] == 0
    for dy, dx in [(-1, 0), (1, 0), (0, -1), (0, 1)]:
        assert G[10 + dy, 20 + dx] == pytest.approx(2.0, abs=1e-12)
    for dy, dx in [(-1, -1), (-1, 1), (1, -1), (1, 1)]:
        assert G[10 + dy, 20 + dx] == pytest.approx(np.sqrt(2.0), abs=1e-12)
    assert od.density(im, 32, tau=0.2)[2].sum() == 8
    assert od.density(im, 32, tau=1.5)[2].sum() == 4       # only the edge neighbours reach 1.5
    assert od.density(im, 32, tau=2.5)[2].sum() == 0


@pytest.mark.parametrize("channel,weight", [(0, 0.299), (1, 0.587), (2, 0.114)])
def test_channel_weights_fix_the_level_at_which_a_step_becomes_an_edge(channel, weight):
    # a step of one channel from 0 to v gives G = 4 * weight * v / 255: an edge from
    # v >= tau * 255 / (4 * weight) on (43 for red, 22 for green, 112 for blue at tau = 0.2)
    tau = 0.2
    v_min = int(np.ceil(tau * 255.0 / (4.0 * weight)))
    assert v_min == {0: 43, 1: 22, 2: 112}[channel]
    for v, edges in [(v_min - 1, 0), (v_min, 2 * 32)]:
        im = _flat(32, 64, (0, 0, 0))
        im[:, 30:, channel] = v
        assert od.density(im, 32, tau)[2].sum() == edges


def test_matches_scipy_sobel_on_a_random_image():
    ndi = pytest.importorskip("scipy.ndimage")
    rng = np.random.default_rng(5)
    im = rng.integers(0, 256, size=(48, 80, 3), dtype=np.uint8)
    gray = od.grayscale(im)
    gx, gy = od.sobel(gray)
    sx = ndi.sobel(gray, axis=1, mode="nearest")          # derivative along x, smoothing along y
    sy = ndi.sobel(gray, axis=0, mode="nearest")
    assert np.allclose(np.abs(gx), np.abs(sx), atol=1e-12)
    assert np.allclose(np.abs(gy), np.abs(sy), atol=1e-12)
    G = np.hypot(sx, sy)
    for tau in (0.2, 0.7, 1.3):
        E = G >= tau
        counts = E.reshape(3, 16, 5, 16).sum(axis=(1, 3))
        rho, rho_k, c = od.density(im, 16, tau)
        assert np.array_equal(c, counts)
        assert rho == pytest.approx(E.mean(), abs=1e-15)   # equal patches: mean of means = overall mean


def test_density_falls_as_the_threshold_rises_and_lies_in_unit_interval():
    rng = np.random.default_rng(9)
    im = rng.integers(0, 256, size=(64, 64, 3), dtype=np.uint8)
    last = 1.0
    for tau in (0.0, 0.1, 0.2, 0.5, 1.0, 2.0, 6.0):
        rho = od.density(im, 16, tau)[0]
        assert 0.0 <= rho <= last
        last = rho
    assert od.density(im, 16, 0.0)[0] == 1.0 and od.density(im, 16, 6.0)[0] == 0.0   # G <= 4 sqrt(2)


def test_transposed_image_gives_transposed_counts():
    rng = np.random.default_rng(2)
    im = rng.integers(0, 256, size=(32, 96, 3), dtype=np.uint8)
    c = od.density(im, 16, 0.6)[2]
    ct = od.density(np.ascontiguousarray(im.transpose(1, 0, 2)), 16, 0.6)[2]
    assert np.array_equal(c.T, ct)
