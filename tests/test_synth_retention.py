"""The dynamic-ratio constants of the Large configuration give the retention the paper reports."""
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

from paper_2605_00392_b200 import synth

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def test_large_mean_retention_is_about_84_percent(oracle):
    vals = dict(ln.split() for ln in open(os.path.join(GOLDEN, "large_phi_hi.txt"))
                if ln.strip() and not ln.startswith("#"))
    assert float(vals["phi_hi"]) == synth.DYNAMIC_PARAMS["phi_hi"]
    w = synth.make("large")
    X = w.X_f64()
    with ThreadPoolExecutor(os.cpu_count() or 1) as ex:
        phis = list(ex.map(lambda i: oracle.phi(X[w.offsets[i]:w.offsets[i + 1]]), range(w.batch)))
    p = synth.DYNAMIC_PARAMS
    kept = [oracle.ratio(ph, float(r), 400, dynamic=True, phi_lo=p["phi_lo"], phi_hi=p["phi_hi"],
                         r_max=p["r_max"])[2] for ph, r in zip(phis, w.rho)]
    assert abs(np.mean(kept) / 400.0 - 0.8425) < 0.005        # abstract: 84.25 % retention
    assert abs(np.mean(kept) / 400.0 - float(vals["mean_retention"])) < 1e-6
