"""Set comparisons used by the parity tests (host arithmetic on oracle results only)."""
import numpy as np

from oracle import rtp_oracle as orc

def e2e_set_check(so, s_gpu, got, p, tol, tag):
    """The GPU's set against the oracle's own scores `so` (fp32, from the raw inputs through the oracle's projections).
    With d = max |s_gpu - so| and A = sum_n P_n |exp(delta_n) - 1| (P = softmax of so), the mass of any subset moves by at
    most eps = 2A / (1 - A) between the two score vectors.  A set that reaches mass p on the GPU's scores therefore holds
    every token scoring more than 2d above the oracle's threshold for the target p - eps - band, and none scoring more than
    2d below the oracle's threshold for p + eps + band."""
    delta = np.abs(s_gpu.astype(np.float64) - so.astype(np.float64))
    assert np.all(delta <= tol), f"{tag}: score differs by {float((delta - tol).max()):.3g} beyond the tolerance"
    d = float(delta.max())
    _, _, P = orc.softmax_mass(so)
    A = float(np.sum(P * np.abs(np.expm1(s_gpu.astype(np.float64) - so.astype(np.float64)))))
    eps = 2.0 * A / (1.0 - A) + 1e-4
    t_hi = orc.topp_select(so, max(p - eps, 1e-6))[3]
    t_lo = orc.topp_select(so, min(p + eps, 1.0))[3]
    member = np.zeros(so.shape[0], dtype=bool)
    member[sorted(got)] = True
    missing = np.nonzero((so > t_hi + 2.0 * d) & ~member)[0]
    extra = np.nonzero((so < t_lo - 2.0 * d) & member)[0]
    assert missing.size == 0, f"{tag}: {missing.size} tokens above the cut are missing (eps {eps:.2g}, d {d:.2g})"
    assert extra.size == 0, f"{tag}: {extra.size} tokens below the cut are present (eps {eps:.2g}, d {d:.2g})"
    return eps

