"""Shared test plumbing: builds a site (inputs + calibration + library layout) from a workload."""
from __future__ import annotations

import numpy as np

from paper_2304_01089_b200 import calibration, workloads


class Site:
    def __init__(self, w: workloads.Workload, tokens=None, calib=None, bits=None, g=None):
        self.w = w
        self.bits = w.bits if bits is None else bits
        self.g = w.clusters if g is None else g
        self.gamma, self.beta = workloads.ln_params(w)
        self.x = workloads.test_tokens(w, tokens)
        x_cal = workloads.calib_tokens(w, calib)
        self.draws = workloads.kmeans_draws(w, 0, self.g)
        self.cal = calibration.calibrate(x_cal, self.gamma, self.beta, self.g, self.bits, self.draws)

    def layout(self, order=0):
        from paper_2304_01089_b200 import binding
        return binding.Layout(self.cal.perm, self.cal.size, self.cal.scale, self.cal.zero, self.bits, order=order)


def random_layout_params(rng, C, g, bits, allow_empty=True):
    """A random reorder index with random cluster sizes (some empty) and parameters."""
    perm = rng.permutation(C).astype(np.int32)
    cuts = np.sort(rng.integers(0, C + 1, size=g - 1)) if g > 1 else np.array([], int)
    size = np.diff(np.concatenate([[0], cuts, [C]])).astype(np.int32)
    if not allow_empty:
        assert C >= g
        size = np.ones(g, np.int32)
        extra = rng.multinomial(C - g, np.ones(g) / g)
        size += extra.astype(np.int32)
    scale = rng.uniform(0.05, 1.5, size=g).astype(np.float32)
    zero = rng.integers(0, 1 << bits, size=g).astype(np.int32)
    return perm, size, scale, zero
