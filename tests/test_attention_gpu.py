"""rptq_attention against the oracle's attention on quantised Q, K, V (Sec. 4.2, 5.1).

The softmax codes are an integer decision taken from floating point: the kernel takes it in fp32 (exp2
of scaled scores), the oracle in fp64, so a code may differ by one where P / s_P lies within the
fp32 error of a half. The tests therefore check three things:
  - the kernel's codes equal the oracle's nearly everywhere and never differ by more than 1;
  - from the kernel's OWN codes, the oracle's last step (integer sums, exact) reproduces the kernel's
    output up to the rounding of the fp16 result;
  - the kernel's output lies within s_P sum_j |dP_q| |V^| (what the differing codes can move) of the
    oracle's end-to-end result.
"""
import numpy as np
import pytest

import oracle

pytestmark = pytest.mark.gpu

FP16 = 2.0 ** -11


def head_layout_params(rng, H, hd, gh, bits, allow_empty=True):
    """Per-head reorder index and clusters: head h owns channels h*hd..(h+1)*hd-1 and clusters h*gh..h*gh+gh-1."""
    perm, size = [], []
    for h in range(H):
        perm.append(h * hd + rng.permutation(hd))
        if allow_empty:
            cuts = np.sort(rng.integers(0, hd + 1, size=gh - 1))
            size.append(np.diff(np.concatenate([[0], cuts, [hd]])))
        else:
            size.append(1 + rng.multinomial(hd - gh, np.ones(gh) / gh))
    return np.concatenate(perm).astype(np.int32), np.concatenate(size).astype(np.int32)


def params(rng, g, bits, lo=0.05, hi=0.3):
    return rng.uniform(lo, hi, size=g).astype(np.float32), rng.integers(0, 1 << bits, size=g).astype(np.int32)


def codes_in_oracle_order(rng, T, size, bits):
    off, k_pad = oracle.segment_offsets(size)
    a = np.zeros((T, k_pad), np.uint8)
    for c in range(len(size)):
        a[:, off[c]:off[c] + size[c]] = rng.integers(0, 1 << bits, size=(T, size[c]))
    return a


def channel_of_oracle_position(perm, size):
    """int [K_pad]: the channel at each position of the oracle's contiguous order, -1 at pads."""
    off, k_pad = oracle.segment_offsets(size)
    out = np.full(k_pad, -1, np.int64)
    j = 0
    for c in range(len(size)):
        out[off[c]:off[c] + size[c]] = perm[j:j + size[c]]
        j += size[c]
    return out


class Case:
    def __init__(self, seed, H, hd, gh, Tq, Tk, bits=(4, 4, 4), allow_empty=True):
        import torch
        from paper_2304_01089_b200 import binding
        rng = np.random.default_rng(seed)
        self.H, self.hd, self.gh, self.Tq, self.Tk = H, hd, gh, Tq, Tk
        self.perm_qk, self.size_qk = head_layout_params(rng, H, hd, gh, bits[0], allow_empty)
        self.perm_v, self.size_v = head_layout_params(rng, H, hd, gh, bits[2], allow_empty)
        g = H * gh
        (self.sQ, self.zQ), (self.sK, self.zK), (self.sV, self.zV) = params(rng, g, bits[0]), params(rng, g, bits[1]), params(rng, g, bits[2])
        self.LQ = binding.Layout(self.perm_qk, self.size_qk, self.sQ, self.zQ, bits[0])
        self.LK = binding.Layout(self.perm_qk, self.size_qk, self.sK, self.zK, bits[1])
        self.LV = binding.Layout(self.perm_v, self.size_v, self.sV, self.zV, bits[2])
        self.q = codes_in_oracle_order(rng, Tq, self.size_qk, bits[0])
        self.k = codes_in_oracle_order(rng, Tk, self.size_qk, bits[1])
        self.v = codes_in_oracle_order(rng, Tk, self.size_v, bits[2])
        mq, mv = self.LQ.contiguous_position(), self.LV.contiguous_position()
        dev = lambda a, m, b: torch.from_numpy(oracle.pack(np.ascontiguousarray(a[:, m]), b)).cuda()
        self.dq, self.dk, self.dv = dev(self.q, mq, bits[0]), dev(self.k, mq, bits[1]), dev(self.v, mv, bits[2])
        self.qk_scale = 1.0 / np.sqrt(hd)
        self.s_P = 1.0 / 256

    def run(self, causal, want_p=True):
        import torch
        from paper_2304_01089_b200 import binding
        C = self.H * self.hd
        out = torch.full((self.Tq + 1, C + 8), float("nan"), dtype=torch.float16, device="cuda")
        pc = torch.zeros((self.H, self.Tq, self.Tk), dtype=torch.uint8, device="cuda") if want_p else None
        binding.attention(self.LQ, self.LK, self.LV, self.H, self.dq, self.dk, self.dv, out, self.s_P, self.qk_scale, causal,
                          Tq=self.Tq, p_codes=pc)
        torch.cuda.synchronize()
        assert binding.get_device_status() == 0
        o = out.float().cpu().numpy()
        assert np.isnan(o[self.Tq]).all() and np.isnan(o[:, C:]).all()           # nothing written outside [Tq][C]
        return o[:self.Tq, :C].astype(np.float64), (pc.cpu().numpy() if want_p else None)

    def oracle_args(self):
        return (self.H, self.gh, self.size_qk, self.sQ.astype(np.float64), self.zQ, self.sK.astype(np.float64), self.zK,
                self.size_v, self.sV.astype(np.float64), self.zV, self.s_P, 0, self.qk_scale)

    def check(self, causal):
        o, pq = self.run(causal)
        want, pq_want = oracle.attention(self.q, self.k, self.v, *self.oracle_args(), causal, return_p=True)
        ch = channel_of_oracle_position(self.perm_v, self.size_v)
        real = ch >= 0
        got = np.zeros_like(want)
        got[:, real] = o[:, ch[real]]
        # 1. the codes
        d = np.abs(pq.astype(np.int32) - pq_want.astype(np.int32))
        assert d.max() <= 1
        nz = pq_want > 0
        assert (d[nz] == 0).mean() >= 0.99 if nz.any() else True
        # 2. the second product from the kernel's own codes: integer sums, one fp32 scaling, fp16 result
        from_own = oracle.attention_output(pq, self.v, self.H, self.gh, self.size_v, self.sV.astype(np.float64), self.zV, self.s_P, 0)
        assert np.all(np.abs(got - from_own) <= 1.01 * FP16 * np.abs(from_own) + 1e-7)
        # 3. end to end: what the differing codes can move, plus the fp16 rounding
        off_v, _ = oracle.segment_offsets(self.size_v)
        Vh = np.zeros(self.v.shape)
        for c in range(len(self.size_v)):
            sl = slice(off_v[c], off_v[c] + self.size_v[c])
            Vh[:, sl] = float(self.sV[c]) * (self.v[:, sl].astype(np.float64) - self.zV[c])
        for h in range(self.H):
            sl = slice(off_v[h * self.gh], off_v[(h + 1) * self.gh])
            bound = self.s_P * d[h].astype(np.float64) @ np.abs(Vh[:, sl]) + 1.01 * FP16 * np.abs(want[:, sl]) + 1e-7
            assert np.all(np.abs(got[:, sl] - want[:, sl]) <= bound)
        assert np.abs(want).max() > 0
        return d


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("bits", [(4, 4, 4), (3, 3, 3), (8, 8, 8), (4, 3, 3)])
def test_small_heads_ragged_tiles(causal, bits):
    Case(11, H=3, hd=40, gh=4, Tq=150, Tk=150, bits=bits).check(causal)


@pytest.mark.parametrize("causal", [False, True])
def test_head_of_128_channels_four_clusters(causal):
    """The paper's setting for R2 / R3: four clusters per head; 128 channels take five to seven units."""
    Case(12, H=2, hd=128, gh=4, Tq=200, Tk=200, allow_empty=False).check(causal)


@pytest.mark.parametrize("Tq,Tk", [(1, 1), (1, 130), (70, 200), (64, 64), (65, 129)])
def test_queries_are_the_last_tokens_of_the_cache(Tq, Tk):
    """Decoding and chunked prefill: Tq queries against a cache of Tk >= Tq keys, causal offset Tk - Tq."""
    Case(13 + Tq, H=2, hd=64, gh=4, Tq=Tq, Tk=Tk).check(True)


def test_one_cluster_per_head_and_empty_clusters():
    Case(14, H=4, hd=32, gh=1, Tq=90, Tk=90).check(True)
    c = Case(15, H=2, hd=48, gh=4, Tq=50, Tk=50)
    c.check(False)


def test_refusals():
    import torch
    from paper_2304_01089_b200 import binding
    c = Case(16, H=2, hd=32, gh=2, Tq=8, Tk=8)
    out = torch.zeros((8, 64), dtype=torch.float16, device="cuda")
    with pytest.raises(binding.RptqError) as e:      # a zero point of the softmax codes
        binding.attention(c.LQ, c.LK, c.LV, 2, c.dq, c.dk, c.dv, out, c.s_P, c.qk_scale, True, z_P=3)
    assert e.value.status == binding.ERR_UNSUPPORTED
    with pytest.raises(binding.RptqError) as e:      # Q and K with different reorder indices
        binding.attention(c.LQ, c.LV, c.LV, 2, c.dq, c.dk, c.dv, out, c.s_P, c.qk_scale, True)
    assert e.value.status == binding.ERR_INVALID_ARG
    with pytest.raises(binding.RptqError) as e:      # more queries than keys
        binding.attention(c.LQ, c.LK, c.LV, 2, c.dq, c.dk, c.dv, out, c.s_P, c.qk_scale, True, Tq=8, Tk=4)
    assert e.value.status == binding.ERR_INVALID_ARG


def test_opt66b_heads_sampled_rows():
    """72 heads of 128 channels, 2048 tokens, 4-bit codes, causal: the launch shape of the OPT-66b
    attention sites; sampled (head, query) rows against the oracle run on that head and that query alone."""
    H, hd, gh, T = 72, 128, 4, 2048
    c = Case(17, H=H, hd=hd, gh=gh, Tq=T, Tk=T, allow_empty=False)
    o, _ = c.run(True, want_p=False)
    rng = np.random.default_rng(5)
    off_qk, _ = oracle.segment_offsets(c.size_qk)
    off_v, _ = oracle.segment_offsets(c.size_v)
    ch = channel_of_oracle_position(c.perm_v, c.size_v)
    for h, i in [(0, 0), (71, T - 1), (35, 63), (35, 64)] + [(int(rng.integers(H)), int(rng.integers(T))) for _ in range(8)]:
        cl = slice(h * gh, (h + 1) * gh)
        qs = slice(off_qk[h * gh], off_qk[(h + 1) * gh]); vs = slice(off_v[h * gh], off_v[(h + 1) * gh])
        pad = lambda a: np.pad(a, ((0, 0), (0, (-a.shape[1]) % 128)))
        want, pq = oracle.attention(pad(c.q[i:i + 1, qs]), pad(c.k[:i + 1, qs]), pad(c.v[:i + 1, vs]), 1, gh,
                                    c.size_qk[cl], c.sQ[cl].astype(np.float64), c.zQ[cl], c.sK[cl].astype(np.float64), c.zK[cl],
                                    c.size_v[cl], c.sV[cl].astype(np.float64), c.zV[cl], c.s_P, 0, c.qk_scale, True, return_p=True)
        chans = ch[vs]
        real = chans >= 0
        got = o[i, chans[real]]
        w = want[0, :vs.stop - vs.start][real]
        # up to a handful of codes of this row may differ by one: each moves the output by at most s_P max|V^|
        vmax = float(c.sV[cl].max()) * 15
        assert np.all(np.abs(got - w) <= 8 * c.s_P * vmax + 1.01 * FP16 * np.abs(w) + 1e-7)
        assert np.abs(got - w).max() <= 0.05 * np.abs(w).max() + 8 * c.s_P * vmax


def test_projections_write_the_cache_and_attention_reads_it():
    """Sec. 4.2: the Q, K and V projections' rows follow the attention sites' reorder indices, so their
    epilogues write the quantised query and the quantised key / value cache directly (RPTQ_OUT_CODES); the
    indices come from the per-head calibration with the K-Means on the device (Q and K clustered together
    on 4-D points). rptq_attention on those buffers against the oracle on the same codes."""
    import torch
    from paper_2304_01089_b200 import binding, calibration
    from helpers import random_layout_params
    rng = np.random.default_rng(21)
    H, d, gh, T, C_in, g_in = 4, 64, 4, 130, 256, 6
    perm1, size1, scale1, zero1 = random_layout_params(rng, C_in, g_in, 4)
    L1 = binding.Layout(perm1, size1, scale1, zero1, 4)
    a = codes_in_oracle_order(rng, T, size1, 4)
    da = torch.from_numpy(oracle.pack(np.ascontiguousarray(a[:, L1.contiguous_position()]), 4)).cuda()
    Ws = [(rng.normal(size=(H * d, C_in)) * 0.05 * rng.lognormal(0, 0.7, size=(H * d, 1))).astype(np.float32) for _ in range(3)]

    def project(W, L_out):
        n = H * d if L_out is None else L_out.K_pad
        rows = None if L_out is None else L_out.padded_index().astype(np.int32)
        w, s_w, wsum = binding.weight_pack(L1, W, out_perm=rows, n_pad=n)
        dw, ds, dws = torch.from_numpy(w).cuda(), torch.from_numpy(s_w).cuda(), torch.from_numpy(wsum).cuda()
        if L_out is None:
            y = torch.empty((T, n), dtype=torch.float32, device="cuda")
            binding.cluster_gemm(L1, da, T, dw, ds, dws, n, y)
        else:
            y = torch.empty((T, L_out.row_bytes), dtype=torch.uint8, device="cuda")
            binding.cluster_gemm(L1, da, T, dw, ds, dws, n, y, layout_out=L_out, y_dtype=binding.OUT_CODES)
        torch.cuda.synchronize()
        return y

    ranges = []
    for W in Ws:                                   # calibration ranges from the projections' own outputs
        y = project(W, None).cpu().numpy().astype(np.float64)
        ranges.append((y.min(axis=0), y.max(axis=0)))
    draws = rng.uniform(size=(H, gh))
    cal_qk = calibration.calibrate_heads(ranges[:2], H, gh, (4, 4), draws, device="cuda")
    cal_v = calibration.calibrate_heads(ranges[2:], H, gh, (3,), draws, device="cuda")
    host_qk = calibration.calibrate_heads(ranges[:2], H, gh, (4, 4), draws)
    assert np.array_equal(cal_qk.perm, host_qk.perm) and np.array_equal(cal_qk.size, host_qk.size)

    c = Case.__new__(Case)
    c.H, c.hd, c.gh, c.Tq, c.Tk = H, d, gh, T, T
    c.perm_qk, c.size_qk, c.perm_v, c.size_v = cal_qk.perm, cal_qk.size, cal_v.perm, cal_v.size
    (c.sQ, c.sK), (c.zQ, c.zK), c.sV, c.zV = cal_qk.scale, cal_qk.zero, cal_v.scale[0], cal_v.zero[0]
    c.LQ = binding.Layout(c.perm_qk, c.size_qk, c.sQ, c.zQ, 4)
    c.LK = binding.Layout(c.perm_qk, c.size_qk, c.sK, c.zK, 4)
    c.LV = binding.Layout(c.perm_v, c.size_v, c.sV, c.zV, 3)
    c.dq, c.dk, c.dv = project(Ws[0], c.LQ), project(Ws[1], c.LK), project(Ws[2], c.LV)
    back = lambda t, L, b: oracle.unpack(t.cpu().numpy(), L.K_pad, b)[:, np.argsort(L.contiguous_position())]
    c.q, c.k, c.v = back(c.dq, c.LQ, 4), back(c.dk, c.LK, 4), back(c.dv, c.LV, 3)
    assert c.q.max() > 8 and c.k.max() > 8 and c.v.max() > 4          # the ranges are used
    c.qk_scale, c.s_P = 1.0 / np.sqrt(d), 1.0 / 256
    c.check(True)


def test_several_sequences_in_one_call():
    """Three sequences of 40 queries against 70 keys each, rows stacked: every sequence attends to its own keys only."""
    import torch
    from paper_2304_01089_b200 import binding
    n_seq, Tq, Tk = 3, 40, 70
    c = Case(31, H=2, hd=64, gh=4, Tq=n_seq * Tq, Tk=n_seq * Tk)        # the stacked tensors; the calls below see them per sequence
    out = torch.full((n_seq * Tq, c.H * c.hd), float("nan"), dtype=torch.float16, device="cuda")
    pc = torch.zeros((n_seq, c.H, Tq, Tk), dtype=torch.uint8, device="cuda")
    binding.attention(c.LQ, c.LK, c.LV, c.H, c.dq, c.dk, c.dv, out, c.s_P, c.qk_scale, True, n_seq=n_seq, p_codes=pc)
    torch.cuda.synchronize()
    o, pq = out.float().cpu().numpy().astype(np.float64), pc.cpu().numpy()
    ch = channel_of_oracle_position(c.perm_v, c.size_v)
    real = ch >= 0
    for s in range(n_seq):
        qs, ks = slice(s * Tq, (s + 1) * Tq), slice(s * Tk, (s + 1) * Tk)
        want, pq_want = oracle.attention(c.q[qs], c.k[ks], c.v[ks], *c.oracle_args(), True, return_p=True)
        d = np.abs(pq[s].astype(np.int32) - pq_want.astype(np.int32))
        assert d.max() <= 1 and (d[pq_want > 0] == 0).mean() >= 0.99
        from_own = oracle.attention_output(pq[s], c.v[ks], c.H, c.gh, c.size_v, c.sV.astype(np.float64), c.zV, c.s_P, 0)
        got = np.zeros_like(from_own)
        got[:, real] = o[qs][:, ch[real]]
        assert np.all(np.abs(got - from_own) <= 1.01 * FP16 * np.abs(from_own) + 1e-7)
    # one sequence of the same call shape gives the same rows as the batch did
    out1 = torch.full((Tq, c.H * c.hd), float("nan"), dtype=torch.float16, device="cuda")
    binding.attention(c.LQ, c.LK, c.LV, c.H, c.dq[Tq:2 * Tq].contiguous(), c.dk[Tk:2 * Tk].contiguous(), c.dv[Tk:2 * Tk].contiguous(),
                      out1, c.s_P, c.qk_scale, True)
    torch.cuda.synchronize()
    assert torch.equal(out1, out[Tq:2 * Tq])


def test_empty_and_oversized_calls():
    import torch
    from paper_2304_01089_b200 import binding
    c = Case(32, H=2, hd=32, gh=2, Tq=8, Tk=8)
    out = torch.full((8, 64), 7.0, dtype=torch.float16, device="cuda")
    binding.attention(c.LQ, c.LK, c.LV, 2, c.dq, c.dk, c.dv, out, c.s_P, c.qk_scale, True, Tq=0, Tk=8)      # no queries: nothing runs
    binding.attention(c.LQ, c.LK, c.LV, 2, c.dq, c.dk, c.dv, out, c.s_P, c.qk_scale, True, Tq=8, Tk=8, n_seq=0)
    torch.cuda.synchronize()
    assert bool((out == 7.0).all())
    with pytest.raises(binding.RptqError) as e:      # more keys than the int32 sums of the second product can take
        binding.attention(c.LQ, c.LK, c.LV, 2, c.dq, c.dk, c.dv, out, c.s_P, c.qk_scale, True, Tq=8, Tk=40000)
    assert e.value.status == binding.ERR_UNSUPPORTED
