"""The parity rule between a BMU implementation's outputs and the CPU oracle.

TEST INFRASTRUCTURE ONLY (tests, smoke check, benchmark self-check).

Rule (from the build target; Section 3.1 of the paper concedes that accumulation order
flips a few assignments between near-tied neurons, and that fp64 removes them):

* a sample is *unambiguous* when the oracle's best-to-second-best gap exceeds
  ``GAP_REL`` (1e-4) relative to the best squared distance d1; then the index must equal
  the oracle's exactly;
* otherwise (near tie) any index g whose fp64 distance is within the same band of d1 is
  accepted, and the case is counted;
* the reported squared distance must match the oracle's fp64 distance *to the reported
  neuron* within ``DIST_REL`` (1e-5) relative (``DIST_ABS`` 1e-6 absolute floor for
  distances that are exactly or nearly zero);
* the hit-count histogram built from unambiguous samples must be identical.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

GAP_REL = 1e-4
DIST_REL = 1e-5
DIST_ABS = 1e-6


@dataclass
class ParityReport:
    n: int
    unambiguous: int
    near_ties: int
    index_mismatch_unambiguous: int
    near_tie_outside_band: int
    max_dist_rel_err: float
    dist_violations: int
    histogram_equal: bool

    @property
    def ok(self) -> bool:
        return (self.index_mismatch_unambiguous == 0 and self.near_tie_outside_band == 0
                and self.dist_violations == 0 and self.histogram_equal)

    def __str__(self):
        return ("n=%d unambiguous=%d near_ties=%d idx_mismatch=%d outside_band=%d "
                "max_dist_rel_err=%.3g dist_violations=%d hist_equal=%s"
                % (self.n, self.unambiguous, self.near_ties, self.index_mismatch_unambiguous,
                   self.near_tie_outside_band, self.max_dist_rel_err, self.dist_violations,
                   self.histogram_equal))


def check(g_bmu, g_dist, top2, d_at_g, M: int) -> ParityReport:
    """g_bmu/g_dist: implementation outputs; top2: oracle Top2; d_at_g: oracle fp64 distance of
    each sample to g_bmu (``som_oracle.dist_at``)."""
    g = np.asarray(g_bmu).astype(np.int64)
    gd = np.asarray(g_dist).astype(np.float64)
    d1, d2, b1 = top2.d1, top2.d2, top2.b1
    n = g.size
    in_range = (g >= 0) & (g < M)
    scale = np.where(np.abs(d1) > 1e-30, np.abs(d1), 1.0)
    unamb = (d2 - d1) > GAP_REL * scale
    idx_bad = int(np.sum(unamb & (g != b1)))
    band_bad = int(np.sum(~unamb & (~in_range | ((d_at_g - d1) > GAP_REL * scale))))
    tol = DIST_REL * np.abs(d_at_g) + DIST_ABS
    err = np.abs(gd - d_at_g)
    viol = int(np.sum(~(err <= tol)))
    rel = float(np.max(err / np.maximum(np.abs(d_at_g), 1e-30), initial=0.0, where=np.abs(d_at_g) > 1e-3))
    hg = np.bincount(g[unamb & in_range], minlength=M)
    ho = np.bincount(b1[unamb], minlength=M)
    return ParityReport(n, int(unamb.sum()), int((~unamb).sum()), idx_bad, band_bad, rel, viol,
                        bool(np.array_equal(hg, ho)))
