"""Seeded synthetic inputs shaped like OPT decoder-layer activations and weights.

This module only draws random tensors. It holds none of the method's arithmetic (no LayerNorm,
no min/max, no clustering, no quantisation): both the CUDA path and the CPU checker are fed from
here so that they see the same bytes, and neither borrows code from the other.

Value structure follows the paper's observation that a few channels carry much larger ranges than
the rest (Sec. 3.2, Fig. 1): the LayerNorm gain has a log-normal body and a small fraction of
channels multiplied by a large factor, so the LayerNorm output has outlier channels and channel
ranges that differ by orders of magnitude.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, Iterator, Optional, Tuple

import numpy as np


@dataclasses.dataclass(frozen=True)
class Linear:
    name: str
    n_out: int


@dataclasses.dataclass(frozen=True)
class Workload:
    """One OPT-shaped site: LayerNorm over `hidden` channels followed by linear layer(s)."""
    name: str
    seed: int
    tokens: int          # M of the test batch
    hidden: int          # C
    clusters: int        # g
    bits: int            # activation bits b
    calib_tokens: int
    outlier_frac: float
    outlier_gain: float
    linears: Tuple[Linear, ...]
    token_sweep: Tuple[int, ...] = ()
    # second linear of an FC1 -> ReLU -> FC2 chain (its input is FC1's output space)
    chain_out: Optional[int] = None
    chain_clusters: Optional[int] = None


WORKLOADS: Dict[str, Workload] = {
    w.name: w for w in (
        Workload("opt-125m", 0, 128, 768, 4, 4, 256, 0.01, 40.0, (Linear("fc", 3072),)),
        Workload("opt-1.3b", 1, 2048, 2048, 8, 4, 512, 0.01, 40.0, (Linear("qkv", 6144),)),
        Workload("opt-6.7b", 2, 8192, 4096, 16, 4, 1024, 0.02, 60.0, (Linear("fc1", 16384),)),
        Workload("opt-66b", 3, 4096, 9216, 32, 3, 1024, 0.01, 40.0,
                 (Linear("qkv", 27648), Linear("fc1", 36864)), token_sweep=(16, 256, 4096)),
        Workload("opt-175b", 4, 2048, 12288, 64, 4, 2048, 0.01, 40.0,
                 (Linear("fc1", 49152),), chain_out=12288, chain_clusters=64),
    )
}

# stream tags keep the different tensors of one workload statistically independent
_TAG_LN, _TAG_TEST, _TAG_CALIB, _TAG_W, _TAG_KMEANS, _TAG_BIAS, _TAG_HEADS = 11, 12, 13, 14, 15, 16, 17


def _rng(seed: int, tag: int, *extra: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64([int(seed), int(tag), *[int(e) for e in extra]]))


def scaled(w: Workload, *, tokens: Optional[int] = None, hidden: Optional[int] = None,
           clusters: Optional[int] = None, bits: Optional[int] = None,
           calib_tokens: Optional[int] = None, linears: Optional[Tuple[Linear, ...]] = None,
           chain_out: Optional[int] = None, chain_clusters: Optional[int] = None,
           seed: Optional[int] = None, name: Optional[str] = None) -> Workload:
    """A copy of `w` with some sizes replaced (small cases for tests)."""
    return dataclasses.replace(
        w,
        name=name or (w.name + "-scaled"),
        seed=w.seed if seed is None else seed,
        tokens=w.tokens if tokens is None else tokens,
        hidden=w.hidden if hidden is None else hidden,
        clusters=w.clusters if clusters is None else clusters,
        bits=w.bits if bits is None else bits,
        calib_tokens=w.calib_tokens if calib_tokens is None else calib_tokens,
        linears=w.linears if linears is None else linears,
        chain_out=w.chain_out if chain_out is None and linears is None else chain_out,
        chain_clusters=w.chain_clusters if chain_clusters is None and linears is None else chain_clusters,
    )


def ln_params(w: Workload) -> Tuple[np.ndarray, np.ndarray]:
    """LayerNorm gain and bias as fp16 [C]: gain ~ LogNormal(0, 0.75) with `outlier_frac` of the
    channels multiplied by `outlier_gain`; bias ~ N(0, (0.5 * gain)^2)."""
    r = _rng(w.seed, _TAG_LN)
    C = w.hidden
    gain = r.lognormal(0.0, 0.75, size=C)
    n_out = max(1, int(round(w.outlier_frac * C)))
    idx = r.choice(C, size=n_out, replace=False)
    gain[idx] *= w.outlier_gain
    bias = r.normal(0.0, 1.0, size=C) * 0.5 * gain
    return gain.astype(np.float16), bias.astype(np.float16)


def _draw_tokens(r: np.random.Generator, n: int, C: int) -> np.ndarray:
    out = np.empty((n, C), dtype=np.float16)
    step = max(1, (1 << 22) // C)
    for lo in range(0, n, step):
        hi = min(n, lo + step)
        body = r.standard_normal((hi - lo, C), dtype=np.float32)
        tok_scale = r.lognormal(0.0, 0.3, size=(hi - lo, 1)).astype(np.float32)
        out[lo:hi] = (body * tok_scale).astype(np.float16)
    return out


def test_tokens(w: Workload, n: Optional[int] = None) -> np.ndarray:
    """Pre-LayerNorm test activations, fp16 [n, C]: N(0,1) rows times a LogNormal(0,0.3) per-token
    scale."""
    return _draw_tokens(_rng(w.seed, _TAG_TEST), w.tokens if n is None else n, w.hidden)


def calib_tokens(w: Workload, n: Optional[int] = None) -> np.ndarray:
    """Calibration activations from the same generator, disjoint from the test tokens."""
    return _draw_tokens(_rng(w.seed, _TAG_CALIB), w.calib_tokens if n is None else n, w.hidden)


def weight_rows(w: Workload, linear_index: int, n_out: int, n_in: int,
                row_lo: int = 0, row_hi: Optional[int] = None,
                chunk: int = 1024) -> Iterator[Tuple[int, np.ndarray]]:
    """Yield (first_row, W[first_row:first_row+k, :]) fp32 blocks of a linear layer's weight
    matrix W[n_out][n_in] ~ N(0, 0.02^2) in the PyTorch [out][in] orientation. Each block of
    `chunk` rows has its own stream, so any row range can be regenerated without the rest."""
    row_hi = n_out if row_hi is None else row_hi
    first_chunk = row_lo // chunk
    for ci in range(first_chunk, (row_hi + chunk - 1) // chunk):
        lo, hi = ci * chunk, min(n_out, (ci + 1) * chunk)
        blk = _rng(w.seed, _TAG_W, linear_index, ci).standard_normal((hi - lo, n_in), dtype=np.float32)
        blk *= np.float32(0.02)
        a, b = max(lo, row_lo), min(hi, row_hi)
        if a < b:
            yield a, blk[a - lo:b - lo]


def weight_matrix(w: Workload, linear_index: int, n_out: int, n_in: int) -> np.ndarray:
    out = np.empty((n_out, n_in), dtype=np.float32)
    for lo, blk in weight_rows(w, linear_index, n_out, n_in):
        out[lo:lo + blk.shape[0]] = blk
    return out


def bias_vector(w: Workload, linear_index: int, n_out: int) -> np.ndarray:
    """fp32 bias ~ N(0, 0.02^2) for a linear layer (OPT linears carry biases)."""
    return (_rng(w.seed, _TAG_BIAS, linear_index).standard_normal(n_out) * 0.02).astype(np.float32)


def kmeans_draws(w: Workload, site: int, g: int) -> np.ndarray:
    """Uniform [0,1) numbers consumed by the k-means++ seeding, one per centre. They are drawn
    here and handed to whichever clustering code runs, so two implementations that follow the
    same steps pick the same seeds."""
    return _rng(w.seed, _TAG_KMEANS, site).random(g)


def attention_site(w: Workload, head_dim: int = 128, clusters_per_head: int = 4):
    """Seeded stand-in for the calibrated attention sites of the workload's model (reorders R2 / R3 of the
    paper, computed per head with four clusters): per head a random permutation of its channels, cluster
    sizes drawn around head_dim / clusters_per_head, and per-cluster scales and zero points for Q, K and
    V. Returns dict(heads, perm_qk, size_qk, perm_v, size_v, scale={q,k,v}, zero={q,k,v}); Q and K share
    perm_qk / size_qk. Code tensors come from attention_codes."""
    r = _rng(w.seed, _TAG_HEADS)
    heads = w.hidden // head_dim
    def index():
        perm, size = [], []
        for h in range(heads):
            perm.append(h * head_dim + r.permutation(head_dim))
            size.append(1 + r.multinomial(head_dim - clusters_per_head, np.ones(clusters_per_head) / clusters_per_head))
        return np.concatenate(perm).astype(np.int32), np.concatenate(size).astype(np.int32)
    perm_qk, size_qk = index()
    perm_v, size_v = index()
    g = heads * clusters_per_head
    scale = {t: r.uniform(0.05, 0.3, size=g).astype(np.float32) for t in "qkv"}
    zero = {t: r.integers(0, 1 << w.bits, size=g).astype(np.int32) for t in "qkv"}
    return dict(heads=heads, perm_qk=perm_qk, size_qk=size_qk, perm_v=perm_v, size_v=size_v, scale=scale, zero=zero)


def attention_codes(w: Workload, tokens: int, real_position: np.ndarray, tensor: int) -> np.ndarray:
    """uint8 [tokens][K_pad] uniform codes of w.bits bits at the real positions of a layout (real_position:
    bool [K_pad]), zero at its pad positions. tensor: 0, 1, 2 for Q, K, V."""
    r = _rng(w.seed, _TAG_HEADS, 1 + tensor)
    codes = r.integers(0, 1 << w.bits, size=(tokens, real_position.shape[0]), dtype=np.uint8)
    codes[:, ~real_position] = 0
    return codes
