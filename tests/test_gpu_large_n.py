"""Parity on images with thousands of visual tokens (the token counts of the OCR models with large
visual token sets in the paper's cross-model table: 2137 -> 1238 and 4512 -> 2783 tokens), whose
score tiles are far wider than one CTA's or one cluster's shared memory: the Sinkhorn kernel for wide
tiles iterates on K in the workspace with a cluster of 8 CTAs per image."""
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


def _names(plan):
    return [n for n, _ in plan.profile_read()]


def test_2137_tokens_to_1238(parity):
    # r = 1 - 1238 / 2137: B = 899 pruned tokens, a 1238 x 899 tile (4.4 MB); the second image is solved by
    # the cluster kernel in the same run
    w = synth.ragged([2137, 700], params=dict(r_fixed=0.4207))
    rep = parity.check_workload(w)
    assert rep["launches"] == 6      # stage1, gather, scores, sinkhorn_wide, sinkhorn_tall, merge


def test_4512_tokens_to_2783(parity):
    # B = 1729: one 16-byte chunk per thread over all 512 threads of a row group
    w = synth.ragged([4512], params=dict(r_fixed=0.3832))
    parity.check_workload(w)


def test_two_chunks_per_thread_and_fp32_storage(parity):
    # B = 2500 (rows wider than 2048 floats: two chunks per thread); a small width and fewer iterations keep
    # the oracle short (rows that short can only be told apart by length in fp32 storage)
    w = synth.ragged([5000, 1300], d=64, dtype=torch.float32, params=dict(r_fixed=0.5, iters=20))
    parity.check_workload(w)
    w = synth.ragged([1500, 2200], d=64, dtype=torch.float32, params=dict(r_fixed=0.5, iters=30))
    parity.check_workload(w)


def test_many_images_with_narrow_wide_tiles_take_clusters_of_four(parity):
    # 20 images whose clusters of 8 would not all run at once, tiles of 700 columns: clusters of 4 CTAs
    w = synth.ragged([1400] * 20, d=64, dtype=torch.float32, params=dict(r_fixed=0.5, iters=30))
    parity.check_workload(w)
    w = synth.ragged([1400] * 19 + [700], params=dict(r_fixed=0.5))
    parity.check_workload(w, images=[0, 7, 18, 19])


def test_single_kept_row_leaves_seven_ctas_without_rows(parity):
    w = synth.ragged([1400], d=64, dtype=torch.float32, params=dict(r_fixed=0.9995, iters=25))
    rep = parity.check_workload(w)
    assert rep["mean_retention"] == pytest.approx(1.0 / 1400.0)


def test_largest_image_goes_to_the_general_kernel(parity):
    # N = 8192, the plan's limit, with more than 4092 pruned tokens: wider than the wide-tile kernel takes
    w = synth.ragged([8192], d=64, dtype=torch.float32, params=dict(r_fixed=0.55, iters=8))
    rep = parity.check_workload(w)
    assert rep["launches"] == 6      # stage1, scores, sinkhorn_wide, sinkhorn_tall (leaves it), sinkhorn, merge


def test_wide_tile_runs_reproduce_bit_for_bit(parity, binding):
    dev = torch.device("cuda", 0)
    w = synth.ragged([2137, 1500], params=dict(r_fixed=0.45))
    plan = binding.Plan(w.d, w.X.dtype, w.batch, w.total_tokens, w.max_tokens, device=dev)
    a = parity.run_gpu(w, plan=plan).out
    b = parity.run_gpu(w, plan=plan).out
    n = int(a.out_offsets[w.batch])                  # rows of Y and entries of kept_idx that are written
    nb = w.total_tokens - n
    assert torch.equal(a.out_offsets, b.out_offsets) and torch.equal(a.counts, b.counts)
    assert torch.equal(a.stats, b.stats)
    assert torch.equal(a.kept_idx[:n], b.kept_idx[:n]) and torch.equal(a.Y[:n], b.Y[:n])
    assert torch.equal(a.merged_idx[:nb], b.merged_idx[:nb])
    assert torch.equal(a.merge_partner[:nb], b.merge_partner[:nb])
    assert torch.equal(a.merge_weight[:nb], b.merge_weight[:nb])
    plan.close()


def test_wide_tile_fixed_point_stop_equals_all_iterations(parity):
    # leaving the loop once no dual moves by more than one unit in the last place gives the result of all
    # T = 100 iterations to fp32 accuracy
    w = synth.ragged([2137], params=dict(r_fixed=0.4207))
    a = parity.run_gpu(w, overrides=dict(stop_at_fixed_point=1)).out
    b = parity.run_gpu(w, overrides=dict(stop_at_fixed_point=0)).out
    assert float(b.stats[0, 5]) == 100.0 and 1.0 <= float(a.stats[0, 5]) < 100.0
    n, nb = int(a.out_offsets[1]), 2137 - int(a.out_offsets[1])
    np.testing.assert_allclose(a.merge_weight[:nb].numpy(), b.merge_weight[:nb].numpy(), rtol=2e-5)
    ya, yb = a.Y[:n].to(torch.float32), b.Y[:n].to(torch.float32)
    assert float((ya - yb).abs().max()) <= 2.0 ** -7 * float(yb.abs().max())      # at most a bf16 rounding apart
    assert float((ya != yb).float().mean()) < 1e-3
