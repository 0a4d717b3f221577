"""rptq_attention_kv (key / value cache quantised only, Sec. 5.2) against the oracle's definition.

The kernel multiplies fp16 operands with fp32 sums: the query is fp16 as given, the K and V codes are exact
in fp16, the scores' error is that of fp32 sums (~1e-6 relative), and the probabilities are rounded to fp16
before the second product. A probability moves by at most 2^-11 of itself, so
    |O - O_oracle| <= 2^-10 sum_j P[i][j] |V^[j][p]|  +  2^-11 |O|  +  1e-5 max|V^|
(the first term with a factor 2 for the exp2 approximation and the score error, the second for the fp16
result); the oracle computes in fp64 from the same fp16 query values.
"""
import numpy as np
import pytest

import oracle
from test_attention_gpu import Case, channel_of_oracle_position

pytestmark = pytest.mark.gpu


def _check(c, q16, causal, n_seq=1):
    """c: a Case (its K layout is LK, V layout LV); q16: fp16 [n_seq * Tq][C] in the original channel order."""
    import torch
    from scipy.special import softmax
    from paper_2304_01089_b200 import binding
    Tq, Tk, H, hd, gh = c.Tq // n_seq, c.Tk // n_seq, c.H, c.hd, c.gh
    Cn = H * hd
    out = torch.full((n_seq * Tq + 1, Cn + 8), float("nan"), dtype=torch.float16, device="cuda")
    qd = torch.from_numpy(q16).cuda()
    binding.attention_kv(c.LK, c.LV, H, qd, c.dk, c.dv, out, c.qk_scale, causal, Tq=Tq, Tk=Tk, n_seq=n_seq)
    torch.cuda.synchronize()
    o = out.float().cpu().numpy()
    assert np.isnan(o[n_seq * Tq]).all() and np.isnan(o[:, Cn:]).all()
    o = o[:n_seq * Tq, :Cn].astype(np.float64)
    ch_k = channel_of_oracle_position(c.perm_qk, c.size_qk).astype(np.int32)
    ch_v = channel_of_oracle_position(c.perm_v, c.size_v)
    real_v = ch_v >= 0
    off_v, _ = oracle.segment_offsets(c.size_v)
    Vh = np.zeros(c.v.shape)
    for cl in range(len(c.size_v)):
        sl = slice(off_v[cl], off_v[cl] + c.size_v[cl])
        Vh[:, sl] = float(c.sV[cl]) * (c.v[:, sl].astype(np.float64) - c.zV[cl])
    off_k, _ = oracle.segment_offsets(c.size_qk)
    for s in range(n_seq):
        qs, ks = slice(s * Tq, (s + 1) * Tq), slice(s * Tk, (s + 1) * Tk)
        q64 = q16[qs].astype(np.float64)
        want = oracle.attention_kv(q64, ch_k, c.k[ks], c.v[ks], H, gh, c.size_qk, c.sK.astype(np.float64), c.zK,
                                   c.size_v, c.sV.astype(np.float64), c.zV, c.qk_scale, causal)
        got = np.zeros_like(want)
        got[:, real_v] = o[qs][:, ch_v[real_v]]
        # the bound needs P: recomputed here from the oracle's own inputs (test-side arithmetic for the bound only)
        for h in range(H):
            lo, hi = off_k[h * gh], off_k[(h + 1) * gh]
            real_k = ch_k[lo:hi] >= 0
            Kh = np.zeros((Tk, hi - lo))
            for cl in range(h * gh, (h + 1) * gh):
                sl = slice(off_k[cl] - lo, off_k[cl] - lo + c.size_qk[cl])
                Kh[:, sl] = float(c.sK[cl]) * (c.k[ks][:, off_k[cl]:off_k[cl] + c.size_qk[cl]].astype(np.float64) - c.zK[cl])
            A = c.qk_scale * q64[:, ch_k[lo:hi][real_k]] @ Kh[:, real_k].T
            if causal:
                A = np.where(np.arange(Tk)[None, :] <= np.arange(Tq)[:, None] + (Tk - Tq), A, -np.inf)
            P = softmax(A, axis=1)
            vs = slice(off_v[h * gh], off_v[(h + 1) * gh])
            bound = 2.0 ** -10 * (P @ np.abs(Vh[ks][:, vs])) + 2.0 ** -11 * np.abs(want[:, vs]) + 1e-5 * np.abs(Vh).max()
            assert np.all(np.abs(got[:, vs] - want[:, vs]) <= bound), (s, h, np.abs(got[:, vs] - want[:, vs]).max())
        assert np.abs(want).max() > 0


def _query(rng, T, Cn, scale=1.0):
    return (rng.normal(size=(T, Cn)) * scale).astype(np.float16)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("bits", [(4, 4, 4), (4, 3, 3), (4, 8, 8)])
def test_small_heads_ragged_tiles(causal, bits):
    c = Case(41, H=3, hd=40, gh=4, Tq=150, Tk=150, bits=bits)
    _check(c, _query(np.random.default_rng(1), 150, 120), causal)


@pytest.mark.parametrize("causal", [False, True])
def test_head_of_128_channels_four_clusters(causal):
    c = Case(42, H=2, hd=128, gh=4, Tq=200, Tk=200, allow_empty=False)
    _check(c, _query(np.random.default_rng(2), 200, 256, 0.5), causal)


@pytest.mark.parametrize("Tq,Tk", [(1, 1), (1, 130), (70, 200), (65, 129)])
def test_queries_are_the_last_tokens_of_the_cache(Tq, Tk):
    c = Case(43 + Tq, H=2, hd=64, gh=4, Tq=Tq, Tk=Tk)
    _check(c, _query(np.random.default_rng(3), Tq, 128), True)


def test_several_sequences_and_empty_clusters():
    c = Case(44, H=2, hd=48, gh=4, Tq=3 * 40, Tk=3 * 70)
    _check(c, _query(np.random.default_rng(4), 120, 96), True, n_seq=3)


def test_refusals_and_empty_calls():
    import torch
    from paper_2304_01089_b200 import binding
    c = Case(45, H=2, hd=32, gh=2, Tq=8, Tk=8)
    q = torch.zeros((8, 64), dtype=torch.float16, device="cuda")
    out = torch.full((8, 64), 7.0, dtype=torch.float16, device="cuda")
    binding.attention_kv(c.LK, c.LV, 2, q, c.dk, c.dv, out, c.qk_scale, True, Tq=0, Tk=8)
    binding.attention_kv(c.LK, c.LV, 2, q, c.dk, c.dv, out, c.qk_scale, True, Tq=8, Tk=8, n_seq=0)
    torch.cuda.synchronize()
    assert bool((out == 7.0).all())
    with pytest.raises(binding.RptqError) as e:      # more queries than keys
        binding.attention_kv(c.LK, c.LV, 2, q, c.dk, c.dv, out, c.qk_scale, True, Tq=8, Tk=4)
    assert e.value.status == binding.ERR_INVALID_ARG
    with pytest.raises(binding.RptqError) as e:      # heads that do not divide the clusters
        binding.attention_kv(c.LK, c.LV, 3, q, c.dk, c.dv, out, c.qk_scale, True)
    assert e.value.status == binding.ERR_INVALID_ARG


def test_layouts_whose_heads_do_not_own_their_channels_are_refused():
    import torch
    from paper_2304_01089_b200 import binding
    from helpers import random_layout_params
    rng = np.random.default_rng(9)
    perm, size, scale, zero = random_layout_params(rng, 64, 4, 4, allow_empty=False)     # one permutation across both heads
    L = binding.Layout(perm, size, scale, zero, 4)
    q = torch.zeros((8, 64), dtype=torch.float16, device="cuda")
    codes = torch.zeros((8, L.row_bytes), dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.RptqError) as e:
        binding.attention_kv(L, L, 2, q, codes, codes, torch.zeros_like(q), 0.1, True)
    assert e.value.status == binding.ERR_INVALID_ARG


def test_opt66b_heads_sampled_rows():
    """72 heads of 128 channels, 2048 tokens, 4-bit cache, causal; sampled (head, query) rows against the oracle
    run on that head and that query alone."""
    import torch
    from paper_2304_01089_b200 import binding
    H, hd, gh, T = 72, 128, 4, 2048
    c = Case(46, H=H, hd=hd, gh=gh, Tq=T, Tk=T, allow_empty=False)
    rng = np.random.default_rng(6)
    q16 = _query(rng, T, H * hd, 0.5)
    out = torch.empty((T, H * hd), dtype=torch.float16, device="cuda")
    binding.attention_kv(c.LK, c.LV, H, torch.from_numpy(q16).cuda(), c.dk, c.dv, out, c.qk_scale, True)
    torch.cuda.synchronize()
    o = out.float().cpu().numpy().astype(np.float64)
    off_k, _ = oracle.segment_offsets(c.size_qk)
    off_v, _ = oracle.segment_offsets(c.size_v)
    ch_k = channel_of_oracle_position(c.perm_qk, c.size_qk)
    ch_v = channel_of_oracle_position(c.perm_v, c.size_v)
    pad = lambda a: np.pad(a, ((0, 0), (0, (-a.shape[1]) % 128)))
    for h, i in [(0, 0), (71, T - 1), (35, 63), (35, 64)] + [(int(rng.integers(H)), int(rng.integers(T))) for _ in range(8)]:
        cl = slice(h * gh, (h + 1) * gh)
        ks = slice(off_k[h * gh], off_k[(h + 1) * gh]); vs = slice(off_v[h * gh], off_v[(h + 1) * gh])
        chk = ch_k[ks] - h * hd                                  # channels of the head, relative; pads stay negative
        chk = np.where(ch_k[ks] >= 0, chk, -1)
        chk = np.pad(chk, (0, (-len(chk)) % 128), constant_values=-1).astype(np.int32)
        want = oracle.attention_kv(q16[i:i + 1, h * hd:(h + 1) * hd].astype(np.float64), chk, pad(c.k[:i + 1, ks]), pad(c.v[:i + 1, vs]),
                                   1, gh, c.size_qk[cl], c.sK[cl].astype(np.float64), c.zK[cl],
                                   c.size_v[cl], c.sV[cl].astype(np.float64), c.zV[cl], c.qk_scale, True)
        chans = ch_v[vs]
        real = chans >= 0
        got, w = o[i, chans[real]], want[0, :vs.stop - vs.start][real]
        vmax = float(c.sV[cl].max()) * 15
        assert np.all(np.abs(got - w) <= 2.0 ** -10 * vmax + 2.0 ** -11 * np.abs(w) + 1e-5 * vmax)
