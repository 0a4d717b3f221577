"""The large workload configurations at full size, in the launch configuration the benchmark times:
the whole product path (host calibration -> rptq_ln_reorder_quant -> rptq_weight_pack ->
rptq_cluster_gemm) runs on the device, and sampled token rows are checked against the CPU oracle.

Sampled rows of the GEMM's input are overwritten with the oracle's own packed codes before the
launch, so that every expected value comes from the oracle alone while the launch keeps its full
shape."""
import numpy as np
import pytest

import oracle
from paper_2304_01089_b200 import calibration, workloads
from helpers import Site

pytestmark = pytest.mark.gpu

TOL = 1e-4
EPS = 1e-5


def _sample_rows(M, n=12, seed=0):
    rows = set(np.random.default_rng(seed).choice(M, size=min(n, M), replace=False).tolist())
    rows |= {0, M - 1}
    if M > 130:
        rows |= {127, 128}          # both sides of a tile boundary
    return np.array(sorted(rows))


def _pack_weights_both(L, site_w, li, n_out, hidden, out_perm=None, n_pad=None):
    """Library packing (chunked over output rows when there is no output index) and the oracle's,
    compared bit for bit. Returns device tensors and the oracle's codes."""
    import torch
    from paper_2304_01089_b200 import binding
    W = workloads.weight_matrix(site_w, li, n_out, hidden)
    w_codes_o, s_w_o, wsum_o = oracle.weight_quantize(W, L._perm, L._size, out_perm, n_pad)
    packed, s_w, wsum = binding.weight_pack(L, W, out_perm, n_pad)
    del W
    in_lib_order = np.ascontiguousarray(w_codes_o[:, L.contiguous_position()])
    assert np.array_equal(packed, oracle.pack_weights(in_lib_order)), "packed weights differ from the oracle's"
    del in_lib_order
    assert np.array_equal(s_w, s_w_o) and np.array_equal(wsum, wsum_o)
    dev = dict(w=torch.from_numpy(packed).cuda(), s_w=torch.from_numpy(s_w).cuda(), wsum=torch.from_numpy(wsum).cuda())
    return dev, w_codes_o, s_w_o, wsum_o


def _ln_codes(site, L, M):
    """Kernel (a) on the first M test tokens; returns the device code buffer and the oracle's codes
    for the sampled rows (which replace the kernel's in the buffer). The oracle's codes are in the
    contiguous unit order; `pos` moves them to the layout's."""
    import torch
    from paper_2304_01089_b200 import binding
    x = site.x[:M]
    xd = torch.from_numpy(x).cuda()
    codes = torch.empty((M, L.row_bytes), dtype=torch.uint8, device="cuda")
    binding.ln_reorder_quant(L, xd, torch.from_numpy(site.gamma).cuda(), torch.from_numpy(site.beta).cuda(), EPS, codes)
    torch.cuda.synchronize()
    rows = _sample_rows(M)
    y64 = oracle.reorder(oracle.layernorm(x[rows], site.gamma, site.beta, EPS), site.cal.perm)
    want = oracle.quantize(y64, site.cal.size, site.cal.scale.astype(np.float64), site.cal.zero, site.bits)
    pos = L.contiguous_position()
    want_lib = np.ascontiguousarray(want[:, pos])
    got = oracle.unpack(codes[torch.from_numpy(rows).cuda()].cpu().numpy(), L.K_pad, site.bits)
    diff = np.abs(got.astype(int) - want_lib.astype(int))
    # the bar of the LayerNorm kernel against the fp64 oracle: all within +-1, >= 99.99 % equal (over the
    # real positions of the sampled rows; pads always agree)
    assert diff.max() <= 1 and (diff != 0).sum() <= 1e-4 * len(rows) * site.w.hidden
    codes[torch.from_numpy(rows).cuda()] = torch.from_numpy(oracle.pack(want_lib, site.bits)).cuda()
    return codes, rows, want


@pytest.mark.parametrize("name,li,Ms", [("opt-6.7b", 0, (8192,)), ("opt-66b", 0, (4096,)), ("opt-66b", 1, (16, 256, 4096))])
def test_layernorm_to_linear_full_size(name, li, Ms):
    import torch
    from paper_2304_01089_b200 import binding
    site = Site(workloads.WORKLOADS[name])
    w = site.w
    L = site.layout(order=binding.ORDER_INTERLEAVED)
    n_out = w.linears[li].n_out
    dev, w_codes_o, s_w_o, wsum_o = _pack_weights_both(L, w, li, n_out, w.hidden)
    bias = workloads.bias_vector(w, li, n_out)
    bias_d = torch.from_numpy(bias).cuda()
    for M in Ms:
        codes, rows, a_rows = _ln_codes(site, L, M)
        want = oracle.cluster_gemm(a_rows, w_codes_o, site.cal.size, site.cal.scale.astype(np.float64), site.cal.zero,
                                   s_w_o, wsum_o, bias=bias)
        ymax = np.abs(want).max()
        y32 = torch.full((M, n_out), float("nan"), dtype=torch.float32, device="cuda")
        binding.cluster_gemm(L, codes, M, dev["w"], dev["s_w"], dev["wsum"], n_out, y32, bias=bias_d)
        y16 = torch.empty((M, n_out), dtype=torch.float16, device="cuda")
        binding.cluster_gemm(L, codes, M, dev["w"], dev["s_w"], dev["wsum"], n_out, y16, bias=bias_d, y_dtype=binding.OUT_F16)
        torch.cuda.synchronize()
        assert binding.get_device_status() == 0
        assert not bool(torch.isnan(y32).any())
        ridx = torch.from_numpy(rows).cuda()
        got = y32[ridx].cpu().numpy()
        err = np.max(np.abs(got - want)) / ymax
        print(f"{name} linear {li} M={M}: max|dy|/max|y| = {err:.2e} on {len(rows)} rows x {n_out}")
        assert err <= TOL
        assert np.array_equal(y16[ridx].cpu().numpy(), got.astype(np.float16))
        # raw accumulators of a window, bit for bit (integer debug kernel vs brute force)
        m0 = int(rows[1]) if len(rows) > 1 else 0
        acc = torch.empty((L.g, 1, 64), dtype=torch.int32, device="cuda")
        binding.cluster_gemm_debug_acc(L, codes, M, dev["w"], n_out, m0, m0 + 1, n_out - 64, n_out, acc)
        torch.cuda.synchronize()
        k = int(np.where(rows == m0)[0][0])
        assert np.array_equal(acc.cpu().numpy()[:, 0, :].astype(np.int64),
                              oracle.cluster_acc(a_rows[k:k + 1], w_codes_o[n_out - 64:], site.cal.size)[:, 0, :])
        if M >= 4096:
            # The same accumulators out of the tensor-core path of this very launch shape (persistent
            # tiles, every K block, both accumulator buffers): the cluster under test gets scale 1 and
            # every other one a vanishing scale, with s_w = 1, z = 0 and no Wsum, so the fp32 output is
            # that cluster's integer accumulator. Sampled rows, two column windows, three clusters.
            order = np.argsort(site.cal.size)
            picks = [int(order[-1]), int(order[len(order) // 2]), int(order[np.nonzero(site.cal.size[order])[0][0]])]
            ones = torch.ones(n_out, dtype=torch.float32, device="cuda")
            zeros_ws = torch.zeros_like(dev["wsum"])
            cols = np.r_[0:48, n_out - 48:n_out]
            want_acc = oracle.cluster_acc(a_rows, np.ascontiguousarray(w_codes_o[cols]), site.cal.size)
            for c in picks:
                sc = np.full(L.g, 2.0 ** -80, np.float32)
                sc[c] = 1.0
                Lc = binding.Layout(site.cal.perm, site.cal.size, sc, np.zeros(L.g, np.int32), site.bits, order=binding.ORDER_INTERLEAVED)
                assert np.array_equal(Lc.padded_index(), L.padded_index())
                binding.cluster_gemm(Lc, codes, M, dev["w"], ones, zeros_ws, n_out, y32)
                torch.cuda.synchronize()
                assert binding.get_device_status() == 0
                got_acc = y32[ridx][:, torch.from_numpy(cols).cuda()].cpu().numpy()
                assert np.array_equal(np.rint(got_acc).astype(np.int64), want_acc[c]) and np.all(np.abs(got_acc - np.rint(got_acc)) < 1e-6), \
                    f"cluster {c} (n_c = {site.cal.size[c]}) through the tensor-core path"


def test_fc1_relu_requantise_fc2_chain_full_size():
    """OPT-175b shapes: LN -> FC1 12288x49152 -> ReLU -> codes in the next site's cluster order
    -> FC2 49152x12288, whose output keeps the original channel order (Sec. 4.2)."""
    import torch
    from paper_2304_01089_b200 import binding
    site = Site(workloads.WORKLOADS["opt-175b"])
    w = site.w
    M, C, H = w.tokens, w.hidden, w.linears[0].n_out
    g2, bits2 = w.chain_clusters, w.bits
    L1 = site.layout(order=binding.ORDER_INTERLEAVED)
    b1 = workloads.bias_vector(w, 0, H)

    # --- calibrate the FC1-output site from the product path itself on the calibration tokens
    dev1_id, w1_o_id, s1_o_id, ws1_o_id = _pack_weights_both(L1, w, 0, H, C)
    x_cal = torch.from_numpy(workloads.calib_tokens(w)).cuda()
    n_cal = x_cal.shape[0]
    cal_codes = torch.empty((n_cal, L1.row_bytes), dtype=torch.uint8, device="cuda")
    binding.ln_reorder_quant(L1, x_cal, torch.from_numpy(site.gamma).cuda(), torch.from_numpy(site.beta).cuda(), EPS, cal_codes)
    h_cal = torch.empty((n_cal, H), dtype=torch.float32, device="cuda")
    binding.cluster_gemm(L1, cal_codes, n_cal, dev1_id["w"], dev1_id["s_w"], dev1_id["wsum"], H, h_cal,
                         bias=torch.from_numpy(b1).cuda(), act=binding.ACT_RELU)
    torch.cuda.synchronize()
    h_min, h_max = h_cal.amin(0).cpu().numpy().astype(np.float64), h_cal.amax(0).cpu().numpy().astype(np.float64)
    del h_cal, cal_codes, dev1_id, w1_o_id
    cal2 = calibration.calibrate_from_minmax(h_min, h_max, g2, bits2, workloads.kmeans_draws(w, 1, g2))
    L2 = binding.Layout(cal2.perm, cal2.size, cal2.scale, cal2.zero, bits2, order=binding.ORDER_INTERLEAVED)
    idx = L2.padded_index()          # original hidden channel at each position of the second site's rows
    K2 = L2.K_pad
    pos2 = L2.contiguous_position()
    where = np.empty(H, np.int64)    # position of each hidden channel in the second site's rows
    where[idx[idx >= 0]] = np.nonzero(idx >= 0)[0]
    in_S_order = where[cal2.perm]    # ... of the channels in the order of the reorder index
    print(f"FC1-output site: K_pad {K2}, cluster sizes {sorted(cal2.size.tolist())[:8]} ... {sorted(cal2.size.tolist())[-4:]}")

    # --- FC1 with its rows in the next site's padded order, FC2 on that site's codes
    dev1, w1_o, s1_o, ws1_o = _pack_weights_both(L1, w, 0, H, C, out_perm=idx, n_pad=K2)
    b1p = np.where(idx >= 0, b1[np.maximum(idx, 0)], 0).astype(np.float32)
    dev2, w2_o, s2_o, ws2_o = _pack_weights_both(L2, workloads.scaled(w, seed=w.seed + 1, name="fc2"), 0, C, H)

    codes1, rows, a_rows = _ln_codes(site, L1, M)
    ridx = torch.from_numpy(rows).cuda()
    h_codes = torch.full((M, L2.row_bytes), 0xEE, dtype=torch.uint8, device="cuda")
    binding.cluster_gemm(L1, codes1, M, dev1["w"], dev1["s_w"], dev1["wsum"], K2, h_codes, bias=torch.from_numpy(b1p).cuda(),
                         act=binding.ACT_RELU, layout_out=L2, y_dtype=binding.OUT_CODES)
    torch.cuda.synchronize()
    assert binding.get_device_status() == 0
    # oracle: FC1 (+bias, ReLU) on the sampled rows, then the cluster quantiser of the next site
    h64 = oracle.cluster_gemm(a_rows, w1_o, site.cal.size, site.cal.scale.astype(np.float64), site.cal.zero, s1_o, ws1_o,
                              bias=b1p, relu=True)
    real = idx >= 0
    want2 = oracle.quantize(h64[:, in_S_order], cal2.size, cal2.scale.astype(np.float64), cal2.zero, bits2)
    want2_lib = np.ascontiguousarray(want2[:, pos2])
    got2 = oracle.unpack(h_codes[ridx].cpu().numpy(), K2, bits2)
    diff = np.abs(got2.astype(int) - want2_lib.astype(int))
    print(f"re-quantised FC1 output: {(diff != 0).mean():.2e} of codes differ from the fp64 oracle, max {diff.max()}")
    # the epilogue decides from the GEMM's fp32 output, whose error (~1e-6 of max|h|) moves a value
    # across a rounding boundary with probability ~ 4 * 2^bits * 1e-6: 1e-4 + 2^bits * 4e-6 is the bar
    assert diff.max() <= 1 and (diff != 0).sum() <= (1e-4 + (1 << bits2) * 4e-6) * len(rows) * H
    assert not got2[:, ~real].any()
    # FC2 at full size with the oracle's codes planted in the sampled rows
    h_codes[ridx] = torch.from_numpy(oracle.pack(want2_lib, bits2)).cuda()
    y = torch.full((M, C), float("nan"), dtype=torch.float32, device="cuda")
    binding.cluster_gemm(L2, h_codes, M, dev2["w"], dev2["s_w"], dev2["wsum"], C, y)
    torch.cuda.synchronize()
    assert binding.get_device_status() == 0 and not bool(torch.isnan(y).any())
    want_y = oracle.cluster_gemm(want2, w2_o, cal2.size, cal2.scale.astype(np.float64), cal2.zero, s2_o, ws2_o)
    err = np.max(np.abs(y[ridx].cpu().numpy() - want_y)) / np.abs(want_y).max()
    print(f"FC2 output (original channel order): max|dy|/max|y| = {err:.2e}")
    assert err <= TOL
