"""The seeded input generators: shapes, determinism, structure, and the spacing of row norms."""
import numpy as np
import torch

from paper_2605_00392_b200 import synth


def _min_rel_gap(x: torch.Tensor) -> float:
    n = np.sort(np.linalg.norm(x.to(torch.float64).numpy(), axis=1))
    return float(np.min(np.diff(n) / n[:-1]))


def test_tiny_shape_and_determinism():
    a, b = synth.make("tiny"), synth.make("tiny")
    assert a.X.shape == (64, 1280) and a.X.dtype == torch.bfloat16
    assert torch.equal(a.X, b.X) and list(a.offsets) == [0, 64]
    assert a.params["dynamic"] == 0 and a.params["r_fixed"] == 0.25
    assert (a.params["z"], a.params["alpha"], a.params["eps"], a.params["iters"]) == (0.2, 0.1, 1.0, 100)
    assert _min_rel_gap(a.X) >= 1.2e-3
    n = np.linalg.norm(a.X_f64(), axis=1)
    assert np.sum(n > 2.5 * np.median(n)) >= 4          # the x4 outliers are there


def test_prefix_and_single_image_regeneration():
    full = synth.make("large", batch=3)
    one = synth.make("large", images=[2])
    assert full.batch == 3 and full.total_tokens == 1200 and full.max_tokens == 400
    assert torch.equal(full.X[800:1200], one.X) and full.rho[2] == one.rho[0]
    assert all(0.2 <= r <= 0.9 for r in full.rho)
    assert full.params["dynamic"] == 1 and full.params["phi_hi"] == 0.737


def test_document_structure_and_gap():
    w = synth.make("base", batch=2)
    assert w.X.shape == (512, 1280) and np.allclose(w.rho, 0.7)
    for i in range(2):
        x = w.image_f64(i)
        assert _min_rel_gap(w.X[i * 256:(i + 1) * 256]) >= 1.2e-3
        xh = x / np.linalg.norm(x, axis=1, keepdims=True)
        g = xh @ xh.T
        near_dup = (g > 0.999).sum(axis=1) - 1
        assert 70 <= np.sum(near_dup >= 50) <= 84       # ~30 % of 256 tokens are background copies


def test_gundam_is_ragged():
    w = synth.make("gundam", batch=12)
    lens = np.diff(w.offsets)
    assert set(int((n - 256) // 100) for n in lens) <= set(range(2, 10))
    assert all((n - 256) % 100 == 0 for n in lens) and len(set(lens)) > 1
    assert w.offsets[0] == 0 and w.total_tokens == lens.sum()


def test_fp32_variant_and_fixed_ratio():
    w = synth.make("sweep_fp32", batch=1, r_fixed=0.35)
    assert w.X.dtype == torch.float32 and w.params["dynamic"] == 0 and w.params["r_fixed"] == 0.35
    assert _min_rel_gap(w.X) >= 1.2e-3
    w2 = synth.make("sweep", batch=1)
    assert w2.params["dynamic"] == 1 and w2.X.dtype == torch.bfloat16


def test_ragged_helper():
    w = synth.ragged([1, 7, 130], d=64, dtype=torch.float32)
    assert list(w.offsets) == [0, 1, 8, 138] and w.d == 64 and w.batch == 3
