"""Host-side calibration (off the hot path): what produces the inputs of rptq_layout_create.

Sec. 4.1 of the paper: run calibration data through the layer, take each channel's minimum and
maximum (Eq. 3), cluster the channels with K-Means on the points (min, max), concatenate the
clusters' index sets into the reorder index S, and give each cluster Min-Max parameters (Eq. 2,
Sec. 5.1). K-Means stays on the host by design; it runs once per site before deployment.

numpy only. This module is part of the product (the benchmark and any user calibrate with it) and
is independent of the test oracle, which has its own plain-C statement of the same steps.
"""
from __future__ import annotations

from typing import NamedTuple, Optional

import numpy as np


class Calibration(NamedTuple):
    perm: np.ndarray      # int32 [C]  S = [S^1 .. S^g]
    size: np.ndarray      # int32 [g]  n_c in S order
    scale: np.ndarray     # fp32  [g]  s_c
    zero: np.ndarray      # int32 [g]  z_c for codes in [0, 2^k - 1]
    x_min: np.ndarray     # fp64  [C]
    x_max: np.ndarray     # fp64  [C]


def layernorm_fp64(x16: np.ndarray, gamma16: np.ndarray, beta16: np.ndarray, eps: float = 1e-5,
                   block: int = 256) -> np.ndarray:
    """Reference-precision LayerNorm of fp16 inputs, used only to observe calibration ranges."""
    g, b = gamma16.astype(np.float64), beta16.astype(np.float64)
    out = np.empty(x16.shape, np.float64)
    for lo in range(0, x16.shape[0], block):
        x = x16[lo:lo + block].astype(np.float64)
        mu = x.mean(axis=1, keepdims=True)
        xc = x - mu
        var = (xc * xc).mean(axis=1, keepdims=True)
        out[lo:lo + block] = xc / np.sqrt(var + eps) * g + b
    return out


def channel_minmax(y: np.ndarray):
    """Eq. 3: per-channel extrema over every calibration sample and token. y is [tokens][C]."""
    return y.min(axis=0).astype(np.float64), y.max(axis=0).astype(np.float64)


def minmax_params(x_min: float, x_max: float, k: int):
    """Eq. 2 as printed: s = (max - min) / 2^k, z = -round((max + min) / (2 s)), with the zero
    point shifted by 2^(k-1) because codes are stored in [0, 2^k - 1]. A zero range gets s = 1."""
    s = (float(x_max) - float(x_min)) / float(1 << k)
    if not s > 0.0:
        s = 1.0
    z = -int(np.rint((float(x_max) + float(x_min)) / (2.0 * s)))
    return s, z + (1 << (k - 1))


def _seq_sum(a: np.ndarray) -> np.ndarray:
    """Sum over axis 0 in index order (numpy's default reduction is pairwise)."""
    return np.cumsum(a, axis=0)[-1] if a.shape[0] else np.zeros(a.shape[1:])


def kmeans(points: np.ndarray, g: int, draws: np.ndarray, iters: int = 20):
    """K-Means with k-means++ seeding driven by `draws` (uniform [0,1), one per centre), `iters`
    Lloyd iterations, squared Euclidean distance on the raw points, ties to the lowest centre; a
    centre left without points takes over the point farthest from its own centre.
    Returns (labels int32 [n], centres [g][dim], inertia per iteration)."""
    pts = np.ascontiguousarray(points, dtype=np.float64)
    n, dim = pts.shape
    centres = np.zeros((g, dim))

    def dist2(c):
        acc = np.zeros(n)
        for a in range(dim):
            t = pts[:, a] - c[a]
            acc = acc + t * t
        return acc

    first = min(int(np.floor(draws[0] * n)), n - 1)
    centres[0] = pts[first]
    d2 = np.full(n, np.inf)
    for k in range(1, g):
        d2 = np.minimum(d2, dist2(centres[k - 1]))
        run = np.cumsum(d2)
        pick = int(np.searchsorted(run, draws[k] * run[-1], side="right"))
        centres[k] = pts[min(pick, n - 1)]

    labels = np.zeros(n, np.int32)
    inertia = np.zeros(iters)
    for it in range(iters):
        all_d = np.stack([dist2(centres[k]) for k in range(g)], axis=1)
        labels = np.argmin(all_d, axis=1).astype(np.int32)
        best = all_d[np.arange(n), labels]
        inertia[it] = np.cumsum(best)[-1]
        count = np.bincount(labels, minlength=g)
        for k in range(g):
            if count[k]:
                continue
            movable = count[labels] > 1
            if not movable.any():
                continue
            far = int(np.argmax(np.where(movable, best, -1.0)))
            count[labels[far]] -= 1
            labels[far] = k
            count[k] = 1
            best[far] = 0.0
        for k in range(g):
            if count[k]:
                centres[k] = _seq_sum(pts[labels == k]) / count[k]
    return labels, centres, inertia


def reorder_index(labels: np.ndarray, x_min: np.ndarray, x_max: np.ndarray, g: int):
    """S = [S^1 .. S^g]. The paper fixes neither order: clusters are placed by ascending merged
    range (max - min), then ascending minimum, then smallest member; empty clusters last; channels
    inside a cluster by ascending index. Returns (perm, size, new_of_old)."""
    keys = []
    for k in range(g):
        members = np.flatnonzero(labels == k)
        if members.size:
            lo, hi = x_min[members].min(), x_max[members].max()
            keys.append((0, hi - lo, lo, int(members[0]), k))
        else:
            keys.append((1, 0.0, 0.0, k, k))
    order = [t[-1] for t in sorted(keys)]
    perm = np.concatenate([np.flatnonzero(labels == k) for k in order]).astype(np.int32)
    size = np.array([(labels == k).sum() for k in order], np.int32)
    new_of_old = np.empty(g, np.int32)
    new_of_old[order] = np.arange(g, dtype=np.int32)
    return perm, size, new_of_old


def calibrate_from_minmax(x_min, x_max, g: int, k: int, draws, iters: int = 20, labels=None) -> Calibration:
    """`labels`: the clustering of the channels when it was computed elsewhere (on the device)."""
    x_min, x_max = np.asarray(x_min, np.float64), np.asarray(x_max, np.float64)
    if labels is None:
        labels, _, _ = kmeans(np.stack([x_min, x_max], axis=1), g, draws, iters)
    perm, size, _ = reorder_index(np.asarray(labels), x_min, x_max, g)
    scale, zero = np.ones(g, np.float32), np.full(g, 1 << (k - 1), np.int32)
    pos = 0
    for c in range(g):
        n = int(size[c])
        if n:
            seg = perm[pos:pos + n]
            s, z = minmax_params(x_min[seg].min(), x_max[seg].max(), k)
            scale[c], zero[c] = np.float32(s), z
        pos += n
    return Calibration(perm, size, scale, zero, x_min, x_max)


def calibrate(x_cal16, gamma16, beta16, g: int, k: int, draws, eps: float = 1e-5, iters: int = 20) -> Calibration:
    """Full calibration of a LayerNorm output site from fp16 calibration activations."""
    y = layernorm_fp64(x_cal16, gamma16, beta16, eps)
    x_min, x_max = channel_minmax(y)
    return calibrate_from_minmax(x_min, x_max, g, k, draws, iters)


def calibrate_on_device(x_cal, gamma, beta, g: int, k: int, draws, eps: float = 1e-5, iters: int = 20) -> Calibration:
    """The same calibration with the two heavy steps on the GPU (Sec. 4.1): the per-channel ranges of
    Eq. 3 over the calibration tokens (rptq_ln_channel_minmax) and the K-Means of the channels
    (rptq_kmeans). x_cal fp16 [T][C], gamma / beta fp16 [C]: CUDA tensors. The reorder index and the
    per-cluster parameters of Eq. 2 are a few thousand operations and stay on the host."""
    import torch
    from . import binding
    Cn = int(gamma.shape[0])
    x_min = torch.empty(Cn, dtype=torch.float32, device=x_cal.device)
    x_max = torch.empty_like(x_min)
    binding.ln_channel_minmax(x_cal, gamma, beta, eps, x_min, x_max)
    pts = torch.stack([x_min, x_max], dim=1).to(torch.float64).contiguous()
    u = torch.from_numpy(np.ascontiguousarray(draws, dtype=np.float64)).to(x_cal.device)
    labels = torch.empty(Cn, dtype=torch.int32, device=x_cal.device)
    centres = torch.empty((g, 2), dtype=torch.float64, device=x_cal.device)
    work = torch.empty(binding.kmeans_workspace_bytes(Cn, g), dtype=torch.uint8, device=x_cal.device)
    binding.kmeans(pts, g, u, iters, labels, centres, None, work)
    return calibrate_from_minmax(x_min.cpu().numpy(), x_max.cpu().numpy(), g, k, draws, iters, labels=labels.cpu().numpy())


class HeadCalibration(NamedTuple):
    """Per-head reorder of an attention site: head h owns channels h*d .. (h+1)*d - 1 and clusters
    h*g_head .. (h+1)*g_head - 1. One (scale, zero) pair per tensor that shares the index."""
    perm: np.ndarray      # int32 [H*d]
    size: np.ndarray      # int32 [H*g_head]
    scale: tuple          # of fp32 [H*g_head]
    zero: tuple           # of int32 [H*g_head]


def _kmeans_host_or_device(points: np.ndarray, g: int, draws, iters: int, device):
    if device is None:
        return kmeans(points, g, draws, iters)[0]
    import torch
    from . import binding
    n, dim = points.shape
    pts = torch.from_numpy(np.ascontiguousarray(points, dtype=np.float64)).to(device)
    u = torch.from_numpy(np.ascontiguousarray(draws, dtype=np.float64)).to(device)
    labels = torch.empty(n, dtype=torch.int32, device=device)
    centres = torch.empty((g, dim), dtype=torch.float64, device=device)
    work = torch.empty(binding.kmeans_workspace_bytes(n, g), dtype=torch.uint8, device=device)
    binding.kmeans(pts, g, u, iters, labels, centres, None, work)
    return labels.cpu().numpy()


def calibrate_heads(ranges, n_heads: int, g_head: int, bits, draws, iters: int = 20, device=None) -> HeadCalibration:
    """Sec. 4.2 / 5.1: the reorder of an attention site, computed per head. `ranges` is a list of
    (x_min, x_max) pairs, one per tensor that must share the index: [(Q), (K)] for R2 -- the head's
    channels are clustered on the points (Q max, Q min, K max, K min) -- and [(V)] for R3. Every tensor
    gets its own Min-Max parameters per cluster (Eq. 2) with its own bit width bits[t]. draws: [H][g_head]
    uniform numbers for the K-Means seeding. device: a torch device to run the K-Means there (rptq_kmeans).
    The clusters of a head are ordered by the union of the tensors' ranges."""
    ranges = [(np.asarray(lo, np.float64), np.asarray(hi, np.float64)) for lo, hi in ranges]
    Cn = ranges[0][0].shape[0]
    d = Cn // n_heads
    assert d * n_heads == Cn and len(bits) == len(ranges)
    lo_all = np.min([r[0] for r in ranges], axis=0)
    hi_all = np.max([r[1] for r in ranges], axis=0)
    perm, size = [], []
    scale = [[] for _ in ranges]
    zero = [[] for _ in ranges]
    for h in range(n_heads):
        sl = slice(h * d, (h + 1) * d)
        pts = np.stack([a[sl] for r in ranges for a in (r[1], r[0])], axis=1)      # (max, min) per tensor
        labels = _kmeans_host_or_device(pts, g_head, np.asarray(draws)[h], iters, device)
        p_h, size_h, _ = reorder_index(np.asarray(labels), lo_all[sl], hi_all[sl], g_head)
        perm.append(h * d + p_h)
        size.append(size_h)
        pos = 0
        for c in range(g_head):
            n = int(size_h[c])
            seg = h * d + p_h[pos:pos + n]
            for t, (lo, hi) in enumerate(ranges):
                s, z = minmax_params(lo[seg].min(), hi[seg].max(), bits[t]) if n else (1.0, 1 << (bits[t] - 1))
                scale[t].append(np.float32(s)); zero[t].append(z)
            pos += n
    return HeadCalibration(np.concatenate(perm).astype(np.int32), np.concatenate(size).astype(np.int32),
                           tuple(np.array(s, np.float32) for s in scale), tuple(np.array(z, np.int32) for z in zero))


def segment_offsets(size: np.ndarray):
    """Padded segment layout of the library: segments start at multiples of 32, rows are a
    multiple of 128 long. Returns (seg_off int32 [g+1], K_pad)."""
    padded = (np.asarray(size, np.int64) + 31) // 32 * 32
    off = np.concatenate([[0], np.cumsum(padded)]).astype(np.int32)
    return off, max(128, int((int(off[-1]) + 127) // 128 * 128))
