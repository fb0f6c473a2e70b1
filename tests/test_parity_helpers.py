"""The comparison the GPU parity tests apply (tests/parity.py) is itself checked here, on the CPU: an
output built from the oracle's own result (rounded to the storage type, as the device would) passes,
and the same output with a mistake planted in it fails.  No GPU, no product code in the loop."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2605_00392_b200 import binding, synth


@pytest.fixture(scope="module")
def parity():
    import parity as _p
    return _p


def _outputs_from_oracle(w, refs, dtype, mutate=None):
    """binding.Outputs filled from the oracle's results; `mutate(i, ref, Y)` may plant a mistake in Y."""
    out = binding.Outputs.allocate(w.total_tokens, w.batch, w.d, dtype, "cpu")
    o = 0
    for i, ref in enumerate(refs.images):
        Y = ref.Y.copy()
        if dtype == torch.bfloat16 and ref.B > 0:
            # what the tensor-core merge computes: the plan rounded to bf16 (alpha folded in) before the product
            Xi = w.image_f64(i)
            aP = torch.from_numpy(np.float32(w.params["alpha"]) * ref.Pbar[:-1, :-1].astype(np.float32)).to(torch.bfloat16)
            Y = Xi[ref.kept] + aP.to(torch.float64).numpy() @ Xi[ref.prop]
        if mutate is not None:
            Y = mutate(i, ref, Y)
        out.Y[o:o + ref.M] = torch.from_numpy(Y).to(dtype)
        out.kept_idx[o:o + ref.M] = torch.from_numpy(ref.kept)
        seg = int(w.offsets[i]) - o
        out.merged_idx[seg:seg + ref.B] = torch.from_numpy(ref.prop)
        out.merge_partner[seg:seg + ref.B] = torch.from_numpy(ref.partner)
        out.merge_weight[seg:seg + ref.B] = torch.from_numpy(ref.weight.astype(np.float32))
        out.counts[i] = ref.M
        out.out_offsets[i] = o
        out.stats[i, 0], out.stats[i, 2] = ref.phi, ref.r
        out.stats[i, 3], out.stats[i, 4], out.stats[i, 5] = ref.M, ref.B, 100
        o += ref.M
    out.out_offsets[w.batch] = o
    return out


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_oracle_output_in_storage_precision_passes(parity, dtype):
    w = synth.ragged([150, 64], dtype=dtype, params=dict(r_fixed=0.25))
    refs = oracle.run_batch(w.X_f64(), w.offsets, parity.oracle_params(w.params), w.rho, want_plan=True)
    g = _outputs_from_oracle(w, refs, dtype)
    rep = {}
    for i, ref in enumerate(refs.images):
        parity.compare_image(w, i, ref, g, rep)
    if dtype == torch.float32:
        assert rep["max_merge_gain_err"] <= parity.MERGE_GAIN_TOL[dtype] / 3
    else:
        assert rep["max_rounding_mismatch"] == 0.0


def test_output_with_fp32_sized_noise_before_the_rounding_passes(parity):
    # what a correct device produces: the value to ~1e-5 (bf16 plan, fp32 accumulation), then one rounding;
    # elements next to a rounding boundary then round the other way, which must not trip the merge-term checks
    w = synth.make("base", batch=3)
    refs = oracle.run_batch(w.X_f64(), w.offsets, parity.oracle_params(w.params), w.rho, want_plan=True)
    rng = np.random.default_rng(5)

    def jitter(i, ref, Y):
        xk = w.image_f64(i)[ref.kept]
        return xk + (Y - xk) * (1.0 + 2e-3 * rng.standard_normal(Y.shape)) + 3e-6 * np.abs(Y) * rng.standard_normal(Y.shape)

    g = _outputs_from_oracle(w, refs, torch.bfloat16, mutate=jitter)
    rep = {}
    for i, ref in enumerate(refs.images):
        parity.compare_image(w, i, ref, g, rep)
    assert 0.0 < rep["max_rounding_mismatch"] < parity.BF16_MODEL_MISMATCH


@pytest.mark.parametrize("lost", [0.36, 0.01])
def test_a_partly_missing_merge_term_fails(parity, lost):
    # the feature tolerance alone would accept this: with alpha = 0.1 the merge term is a few percent of a row
    w = synth.ragged([150], params=dict(r_fixed=0.25))
    refs = oracle.run_batch(w.X_f64(), w.offsets, parity.oracle_params(w.params), w.rho, want_plan=True)
    xk = w.X_f64()[refs.images[0].kept]

    def drop(i, ref, Y):
        return xk + (1.0 - lost) * (Y - xk)

    g = _outputs_from_oracle(w, refs, torch.bfloat16, mutate=drop)
    # the larger loss already breaks the feature tolerance; the smaller one only the merge-term checks
    with pytest.raises(AssertionError, match=None if lost > 0.2 else "merge-term"):
        parity.compare_image(w, 0, refs.images[0], g, {})


def test_a_term_missing_from_a_few_rows_fails(parity):
    w = synth.ragged([150], params=dict(r_fixed=0.25))
    refs = oracle.run_batch(w.X_f64(), w.offsets, parity.oracle_params(w.params), w.rho, want_plan=True)
    xk = w.X_f64()[refs.images[0].kept]

    def drop(i, ref, Y):
        Y = Y.copy()
        Y[5:8] = xk[5:8] + 0.7 * (Y[5:8] - xk[5:8])
        return Y

    g = _outputs_from_oracle(w, refs, torch.bfloat16, mutate=drop)
    with pytest.raises(AssertionError):
        parity.compare_image(w, 0, refs.images[0], g, {})


def test_a_wrong_partner_outside_the_regret_bound_fails(parity):
    w = synth.make("tiny")
    refs = oracle.run_batch(w.X_f64(), w.offsets, parity.oracle_params(w.params), w.rho, want_plan=True)
    g = _outputs_from_oracle(w, refs, torch.bfloat16)
    ref = refs.images[0]
    j = int(np.argmax(ref.gap))
    g.merge_partner[int(w.offsets[0]) - 0 + j] = (int(ref.partner[j]) + 1) % ref.M
    with pytest.raises(AssertionError):
        parity.compare_image(w, 0, ref, g, {})
