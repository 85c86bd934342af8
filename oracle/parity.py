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

Second-best unit (the search of Algorithm 2 keeps the two best units): the reported second
unit g2 must differ from the reported best unit, and its fp64 distance may exceed the oracle's
second-best distance d2 by at most the same relative band (it may be lower: when the two best
are near-tied and the implementation ranks them the other way round, g2 is the oracle's best).
Where the oracle's second and third are further apart than the band this forces g2 == b2, so no
third-best distance is needed.  Its reported distance follows the same ``DIST_REL`` rule.
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


@dataclass
class SecondReport:
    n: int
    differs_from_oracle: int   # g2 != b2 (allowed only inside the band)
    same_as_best: int          # g2 == g1: never allowed
    outside_band: int
    dist_violations: int
    max_dist_rel_err: float

    @property
    def ok(self) -> bool:
        return self.same_as_best == 0 and self.outside_band == 0 and self.dist_violations == 0

    def __str__(self):
        return ("n=%d second_differs=%d same_as_best=%d outside_band=%d dist_violations=%d "
                "max_dist_rel_err=%.3g" % (self.n, self.differs_from_oracle, self.same_as_best,
                                           self.outside_band, self.dist_violations, self.max_dist_rel_err))


def check_second(g_bmu, g_bmu2, g_dist2, top2, d_at_g2, M: int) -> SecondReport:
    """g_bmu/g_bmu2/g_dist2: implementation outputs; top2: oracle Top2; d_at_g2: oracle fp64
    distance of each sample to g_bmu2.  Requires M >= 2 (with one neuron there is no second)."""
    g1 = np.asarray(g_bmu).astype(np.int64)
    g2 = np.asarray(g_bmu2).astype(np.int64)
    gd = np.asarray(g_dist2).astype(np.float64)
    d2 = top2.d2
    in_range = (g2 >= 0) & (g2 < M)
    scale = np.where(np.abs(d2) > 1e-30, np.abs(d2), 1.0)
    same = int(np.sum(g2 == g1))
    band_bad = int(np.sum(~in_range | ((d_at_g2 - d2) > GAP_REL * scale)))
    tol = DIST_REL * np.abs(d_at_g2) + DIST_ABS
    err = np.abs(gd - d_at_g2)
    viol = int(np.sum(~(err <= tol)))
    rel = float(np.max(err / np.maximum(np.abs(d_at_g2), 1e-30), initial=0.0, where=np.abs(d_at_g2) > 1e-3))
    return SecondReport(g1.size, int(np.sum(g2 != top2.b2)), same, band_bad, viol, rel)
