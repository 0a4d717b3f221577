"""Calibration on the device (Sec. 4.1): Eq. 3's per-channel ranges at a LayerNorm site and the K-Means
of the channels, through the C boundary against the CPU oracle."""
import numpy as np
import pytest

import oracle
from paper_2304_01089_b200 import calibration, workloads
from helpers import Site

pytestmark = pytest.mark.gpu

EPS = 1e-5


def _kmeans_gpu(pts, g, u, iters):
    import torch
    from paper_2304_01089_b200 import binding
    n, dim = pts.shape
    p = torch.from_numpy(np.ascontiguousarray(pts, np.float64)).cuda()
    labels = torch.full((n + 1,), -5, dtype=torch.int32, device="cuda")
    centres = torch.empty((g, dim), dtype=torch.float64, device="cuda")
    inertia = torch.empty(max(iters, 1), dtype=torch.float64, device="cuda")
    work = torch.empty(binding.kmeans_workspace_bytes(n, g), dtype=torch.uint8, device="cuda")
    binding.kmeans(p, g, torch.from_numpy(np.ascontiguousarray(u, np.float64)).cuda(), iters, labels, centres, inertia, work)
    torch.cuda.synchronize()
    lab = labels.cpu().numpy()
    assert lab[n] == -5
    return lab[:n], centres.cpu().numpy(), inertia.cpu().numpy()[:iters]


@pytest.mark.parametrize("n,dim,g,seed", [(40, 2, 3, 0), (1000, 2, 8, 1), (1531, 4, 17, 2), (300, 2, 64, 3), (9, 2, 12, 4)])
def test_kmeans_takes_the_oracles_decisions(n, dim, g, seed):
    """Same seeding draws, same steps: labels, centres and the inertia of every iteration equal the
    oracle's (the kernel sums in point order and never fuses a multiply with an add). The last case
    has fewer points than centres (empty centres stay empty); duplicates force exact ties."""
    rng = np.random.default_rng(seed)
    pts = rng.normal(size=(n, dim)) * rng.lognormal(0, 1, size=(n, 1))
    pts[n // 2:n // 2 + 3] = pts[0]                       # duplicates: distance ties
    u = rng.uniform(size=g)
    want_l, want_c, want_i = oracle.kmeans(pts, g, u, 20)
    got_l, got_c, got_i = _kmeans_gpu(pts, g, u, 20)
    assert np.array_equal(got_l, want_l)
    used = np.bincount(want_l, minlength=g) > 0
    assert np.array_equal(got_c[used], want_c[used]) and np.array_equal(got_i, want_i)


@pytest.mark.parametrize("name", ["opt-125m", "opt-66b"])
def test_ranges_and_clustering_of_a_workload_site(name):
    import torch
    from paper_2304_01089_b200 import binding
    site = Site(workloads.WORKLOADS[name])
    w = site.w
    x_cal = workloads.calib_tokens(w)
    Cn = w.hidden
    # Eq. 3 on the device (fp32 LayerNorm) against the fp64 oracle
    xd = torch.from_numpy(x_cal).cuda()
    gd, bd = torch.from_numpy(site.gamma).cuda(), torch.from_numpy(site.beta).cuda()
    x_min = torch.full((Cn + 1,), 77.0, dtype=torch.float32, device="cuda")
    x_max = torch.full((Cn + 1,), 77.0, dtype=torch.float32, device="cuda")
    binding.ln_channel_minmax(xd, gd, bd, EPS, x_min, x_max)
    torch.cuda.synchronize()
    lo, hi = x_min.cpu().numpy(), x_max.cpu().numpy()
    assert lo[Cn] == 77.0 and hi[Cn] == 77.0
    y64 = oracle.layernorm(x_cal, site.gamma, site.beta, EPS)
    want_lo, want_hi = oracle.channel_minmax(y64)
    tol = 8e-6 * np.abs(y64).max()
    assert np.max(np.abs(lo[:Cn] - want_lo)) <= tol and np.max(np.abs(hi[:Cn] - want_hi)) <= tol
    # the kernel's K-Means on the oracle's points: the oracle's labels
    pts = np.stack([want_lo, want_hi], axis=1)
    want_l, want_c, want_i = oracle.kmeans(pts, site.g, site.draws, 20)
    got_l, got_c, got_i = _kmeans_gpu(pts, site.g, site.draws, 20)
    assert np.array_equal(got_l, want_l) and np.array_equal(got_i, want_i)
    # the whole device calibration gives a usable layout: a bijection, every channel inside its cluster's range
    cal = calibration.calibrate_on_device(xd, gd, bd, site.g, site.bits, site.draws, EPS)
    assert np.array_equal(np.sort(cal.perm), np.arange(Cn)) and int(cal.size.sum()) == Cn
    L = binding.Layout(cal.perm, cal.size, cal.scale, cal.zero, site.bits)
    j = 0
    for c, n_c in enumerate(cal.size):
        ch = cal.perm[j:j + n_c]; j += n_c
        if n_c:
            s, z = oracle.minmax_params(float(lo[ch].min()), float(hi[ch].max()), site.bits)
            assert np.float32(s) == cal.scale[c] and z == cal.zero[c]
    L.destroy()
