"""The end-to-end set criterion on the CPU: a selection made on perturbed scores must pass against the unperturbed
scores, and a selection that drops or adds tokens well away from the cut must fail."""
import numpy as np
import pytest

from oracle import rtp_oracle as orc
from tests.set_checks import e2e_set_check


def _case(seed, n, sigma, noise):
    rng = np.random.default_rng(seed)
    so = (sigma * rng.standard_normal(n)).astype(np.float32)
    so[rng.integers(0, n, 4)] += np.float32(2.0 * sigma)
    sg = (so.astype(np.float64) + noise * rng.uniform(-1.0, 1.0, n) * np.maximum(1.0, np.abs(so))).astype(np.float32)
    tol = np.full(n, 0.0) + noise * np.maximum(1.0, np.abs(so)) + 1e-6
    return so, sg, tol


@pytest.mark.parametrize("seed", range(12))
@pytest.mark.parametrize("noise", [0.0, 1e-5, 1e-3, 2e-2])
def test_selection_on_perturbed_scores_passes(seed, noise):
    so, sg, tol = _case(seed, 3000, 1.0 + 0.5 * (seed % 4), noise)
    p = [0.5, 0.9, 0.99][seed % 3]
    got = set(orc.topp_select(sg, p)[0].tolist())
    e2e_set_check(so, sg, got, p, tol, "case")


def test_dropped_and_added_tokens_fail():
    so, sg, tol = _case(3, 3000, 2.0, 1e-4)
    ids, _, _, thr, order, _ = orc.topp_select(sg, 0.9)
    got = set(ids.tolist())
    with pytest.raises(AssertionError, match="missing"):
        e2e_set_check(so, sg, got - {int(order[0])}, 0.9, tol, "case")
    with pytest.raises(AssertionError, match="present"):
        e2e_set_check(so, sg, got | {int(order[-1])}, 0.9, tol, "case")
    with pytest.raises(AssertionError, match="tolerance"):
        bad = sg.copy()
        bad[5] += np.float32(1.0)
        e2e_set_check(so, bad, got, 0.9, tol, "case")
