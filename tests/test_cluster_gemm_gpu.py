"""Parity of rptq_cluster_gemm (tcgen05 path, through the C boundary) against the CPU oracle.

Inputs of the GEMM (packed activation codes, packed weights, s_w, Wsum) are produced by the
oracle here, so a fault in rptq_ln_reorder_quant or rptq_weight_pack cannot hide one in the GEMM.
"""
import numpy as np
import pytest

import oracle
from paper_2304_01089_b200 import workloads
from helpers import Site, random_layout_params

pytestmark = pytest.mark.gpu

TOL = 1e-4   # max |dy| <= TOL * max |y| on the fp32 output


def _case(rng, M, N, C, g, bits, n_pad=None, allow_empty=True):
    perm, size, scale, zero = random_layout_params(rng, C, g, bits, allow_empty)
    n_pad = N if n_pad is None else n_pad
    W = (rng.normal(size=(N, C)) * 0.02).astype(np.float32)
    w_codes, s_w, wsum = oracle.weight_quantize(W, perm, size, None, n_pad)
    off, k_pad = oracle.segment_offsets(size)
    a = np.zeros((M, k_pad), np.uint8)
    for c in range(g):
        a[:, off[c]:off[c] + size[c]] = rng.integers(0, 1 << bits, size=(M, size[c]))
    return dict(perm=perm, size=size, scale=scale, zero=zero, w_codes=w_codes, s_w=s_w, wsum=wsum,
                a=a, k_pad=k_pad, bits=bits, M=M, N=N, n_pad=n_pad)


def _dev(case, order=0):
    """Device inputs of a case. The oracle's arrays are in the contiguous unit order; their columns
    are moved to the layout's own order before packing."""
    import torch
    from paper_2304_01089_b200 import binding
    L = binding.Layout(case["perm"], case["size"], case["scale"], case["zero"], case["bits"], order=order)
    assert L.K_pad == case["k_pad"]
    m = L.contiguous_position()
    d = dict(L=L,
             a=torch.from_numpy(oracle.pack(np.ascontiguousarray(case["a"][:, m]), case["bits"])).cuda(),
             w=torch.from_numpy(oracle.pack_weights(np.ascontiguousarray(case["w_codes"][:, m]))).cuda(),
             s_w=torch.from_numpy(case["s_w"]).cuda(),
             wsum=torch.from_numpy(case["wsum"]).cuda())
    return d


def _gemm(case, d, y_dtype=0, bias=None, act=0, layout_out=None, ldy=None, s_w=None, wsum=None, L=None):
    import torch
    from paper_2304_01089_b200 import binding
    M, N = case["M"], case["N"]
    L = d["L"] if L is None else L
    if y_dtype == binding.OUT_CODES:
        y = torch.full((M + 1, layout_out.row_bytes), 0xA5, dtype=torch.uint8, device="cuda")
    else:
        ldy = N if ldy is None else ldy
        dt = torch.float32 if y_dtype == binding.OUT_F32 else torch.float16
        y = torch.full((M + 1, ldy), float("nan"), dtype=dt, device="cuda")
    bd = None if bias is None else torch.from_numpy(bias).cuda()
    binding.cluster_gemm(L, d["a"], M, d["w"], d["s_w"] if s_w is None else s_w, d["wsum"] if wsum is None else wsum,
                         N, y, ld_w=case["n_pad"], bias=bd, act=act, layout_out=layout_out, y_dtype=y_dtype,
                         ldy=None if y_dtype == binding.OUT_CODES else y.stride(0))
    torch.cuda.synchronize()
    assert binding.get_device_status() == 0
    out = y.cpu().numpy()
    if y_dtype == binding.OUT_CODES:
        assert np.all(out[M] == 0xA5)
    else:
        assert np.all(np.isnan(out[M].astype(np.float32))), "wrote past the last row"
        if out.shape[1] > N:
            assert np.all(np.isnan(out[:M, N:].astype(np.float32))), "wrote past the last column"
    return out[:M]


def _oracle_y(case, bias=None, relu=False, rows=None):
    a = case["a"] if rows is None else case["a"][rows]
    return oracle.cluster_gemm(a, case["w_codes"][:case["N"]], case["size"], case["scale"].astype(np.float64),
                               case["zero"], case["s_w"], case["wsum"], bias=bias, relu=relu)


@pytest.mark.parametrize("bits", [4, 3, 8])
def test_per_cluster_accumulators_are_bit_exact(bits):
    """Each cluster's integer accumulator, read out through the epilogue by giving that cluster
    scale 1 and every other cluster a vanishing scale, with s_w = 1 and z = 0; and the same
    accumulators from the integer-instruction debug kernel."""
    import torch
    from paper_2304_01089_b200 import binding
    rng = np.random.default_rng(bits)
    case = _case(rng, M=200, N=300, C=448, g=4, bits=bits, n_pad=304)
    d = _dev(case)
    want = oracle.cluster_acc(case["a"], case["w_codes"][:case["N"]], case["size"])
    ones = torch.ones(case["n_pad"], dtype=torch.float32, device="cuda")
    zeros_ws = torch.zeros_like(d["wsum"])
    for c in range(4):
        if case["size"][c] == 0:
            continue
        scale = np.full(4, 2.0 ** -80, np.float32)
        scale[c] = 1.0
        L = binding.Layout(case["perm"], case["size"], scale, np.zeros(4, np.int32), bits)
        y = _gemm(case, d, s_w=ones, wsum=zeros_ws, L=L, ldy=304)[:, :case["N"]]
        assert np.array_equal(y.astype(np.int64), want[c]), f"cluster {c}"
    acc = torch.full((4, 200, 300), -1, dtype=torch.int32, device="cuda")
    binding.cluster_gemm_debug_acc(d["L"], d["a"], 200, d["w"], 300, 0, 200, 0, 300, acc)
    torch.cuda.synchronize()
    assert np.array_equal(acc.cpu().numpy().astype(np.int64), want)
    win = torch.full((4, 7, 9), -1, dtype=torch.int32, device="cuda")
    binding.cluster_gemm_debug_acc(d["L"], d["a"], 200, d["w"], 300, 100, 107, 250, 259, win)
    torch.cuda.synchronize()
    assert np.array_equal(win.cpu().numpy().astype(np.int64), want[:, 100:107, 250:259])


@pytest.mark.parametrize("bits", [4, 3, 8])
@pytest.mark.parametrize("M,N,C,g", [(1, 256, 128, 1), (127, 200, 384, 5), (129, 520, 640, 7), (300, 256, 1024, 33)])
def test_small_and_ragged_shapes(bits, M, N, C, g):
    from paper_2304_01089_b200 import binding
    rng = np.random.default_rng(1000 * bits + M + N)
    n_pad = (N + 7) // 8 * 8
    case = _case(rng, M, N, C, g, bits, n_pad=n_pad)
    d = _dev(case)
    want = _oracle_y(case)
    y32 = _gemm(case, d, ldy=n_pad + 8)[:, :N]
    assert np.max(np.abs(y32 - want)) <= TOL * np.abs(want).max()
    # fp16 output: the same fp32 result rounded once to fp16
    y16 = _gemm(case, d, y_dtype=binding.OUT_F16, ldy=n_pad + 8)[:, :N]
    assert np.array_equal(y16, y32.astype(np.float16))
    # bias and ReLU
    bias = (rng.normal(size=n_pad) * np.abs(want).mean()).astype(np.float32)
    yb = _gemm(case, d, bias=bias, act=binding.ACT_RELU, ldy=n_pad + 8)[:, :N]
    want_b = _oracle_y(case, bias=bias[:N], relu=True)
    assert np.max(np.abs(yb - want_b)) <= TOL * np.abs(want).max()
    assert yb.min() >= 0.0


@pytest.mark.parametrize("bits,M", [(3, 300), (4, 100), (8, 257)])
def test_interleaved_unit_order(bits, M):
    """Many one- and two-unit clusters among a few large ones, as calibration produces them: the
    interleaved layout gives the oracle's result, and each cluster's accumulator bit for bit."""
    import torch
    from paper_2304_01089_b200 import binding
    rng = np.random.default_rng(900 + bits)
    size = np.array([1, 1, 2, 3, 9, 13, 0, 40, 5, 53, 173, 434, 530, 7, 64, 33, 664, 300, 2, 1, 1, 6], np.int32)
    size[-1] += (-int(size.sum())) % 8
    C, g, N = int(size.sum()), len(size), 520
    perm = rng.permutation(C).astype(np.int32)
    scale = rng.uniform(0.05, 1.5, size=g).astype(np.float32)
    zero = rng.integers(0, 1 << bits, size=g).astype(np.int32)
    W = (rng.normal(size=(N, C)) * 0.02).astype(np.float32)
    w_codes, s_w, wsum = oracle.weight_quantize(W, perm, size, None, N)
    off, k_pad = oracle.segment_offsets(size)
    a = np.zeros((M, k_pad), np.uint8)
    for c in range(g):
        a[:, off[c]:off[c] + size[c]] = rng.integers(0, 1 << bits, size=(M, size[c]))
    case = dict(perm=perm, size=size, scale=scale, zero=zero, w_codes=w_codes, s_w=s_w, wsum=wsum,
                a=a, k_pad=k_pad, bits=bits, M=M, N=N, n_pad=N)
    d = _dev(case, order=binding.ORDER_INTERLEAVED)
    assert not np.array_equal(d["L"].contiguous_position(), np.arange(k_pad))
    want = _oracle_y(case)
    y = _gemm(case, d)
    assert np.max(np.abs(y - want)) <= TOL * np.abs(want).max()
    y_contig = _gemm(case, _dev(case))
    assert np.max(np.abs(y - y_contig)) <= 1e-5 * np.abs(want).max()      # same sums, another order
    acc = torch.full((g, M, N), -1, dtype=torch.int32, device="cuda")
    binding.cluster_gemm_debug_acc(d["L"], d["a"], M, d["w"], N, 0, M, 0, N, acc)
    torch.cuda.synchronize()
    assert np.array_equal(acc.cpu().numpy().astype(np.int64), oracle.cluster_acc(a, w_codes, size))
    # one cluster at a time through the tensor-core path (scale 1 for it, vanishing for the others)
    ones = torch.ones(N, dtype=torch.float32, device="cuda")
    zeros_ws = torch.zeros_like(d["wsum"])
    want_acc = oracle.cluster_acc(a, w_codes, size)
    for c in (0, 3, 7, 11, 12, 16, 21):
        sc = np.full(g, 2.0 ** -80, np.float32)
        sc[c] = 1.0
        L1 = binding.Layout(perm, size, sc, np.zeros(g, np.int32), bits, order=binding.ORDER_INTERLEAVED)
        y1 = _gemm(case, d, s_w=ones, wsum=zeros_ws, L=L1)
        assert np.array_equal(y1.astype(np.int64), want_acc[c]), f"cluster {c}"


def test_two_launches_on_two_streams_give_identical_bytes():
    import torch
    from paper_2304_01089_b200 import binding
    rng = np.random.default_rng(77)
    case = _case(rng, 513, 768, 1536, 9, 4)
    d = _dev(case)
    y1 = _gemm(case, d)
    s2 = torch.cuda.Stream()
    y = torch.empty((513, 768), dtype=torch.float32, device="cuda")
    binding.cluster_gemm(d["L"], d["a"], 513, d["w"], d["s_w"], d["wsum"], 768, y, stream=s2)
    torch.cuda.synchronize()
    assert np.array_equal(y.cpu().numpy(), y1)


@pytest.mark.parametrize("out_bits", [4, 3, 8])
def test_requantised_output_feeds_the_next_layer(out_bits):
    """FC1 -> ReLU -> quantise in the next site's cluster order -> FC2 (Sec. 4.2: FC1's rows follow
    the next reorder index; FC2's output keeps the original channel order)."""
    import torch
    from paper_2304_01089_b200 import binding
    rng = np.random.default_rng(40 + out_bits)
    M, C, H, g1, g2 = 150, 256, 800, 4, 6          # hidden width H is the second site's channel count
    perm1, size1, scale1, zero1 = random_layout_params(rng, C, g1, 4)
    perm2, size2, _, _ = random_layout_params(rng, H, g2, out_bits)
    off2, k_pad2 = oracle.segment_offsets(size2)
    # where the second site's layout puts each hidden channel does not depend on its parameters
    L2p = binding.Layout(perm2, size2, np.ones(g2, np.float32), np.zeros(g2, np.int32), out_bits)
    # FC1's output rows in the second site's padded order: row r = original hidden channel or a zero pad
    out_rows = L2p.padded_index().astype(np.int64)
    m2 = L2p.contiguous_position()                      # the oracle's contiguous order -> that layout's
    real = out_rows >= 0
    where = np.empty(H, np.int64)
    where[out_rows[real]] = np.nonzero(real)[0]
    in_S_order = where[perm2]                           # position of the channels in the order of the reorder index
    cluster_of_pos = np.repeat(L2p.unit_cluster, 32)
    W1 = (rng.normal(size=(H, C)) * 0.02).astype(np.float32)
    W1p = np.zeros((k_pad2, C), np.float32)
    W1p[real] = W1[out_rows[real]]
    b1 = np.zeros(k_pad2, np.float32)
    b1[real] = (rng.normal(size=H) * 0.05).astype(np.float32)[out_rows[real]]
    w1_codes, s_w1, wsum1 = oracle.weight_quantize(W1p, perm1, size1, None, k_pad2)
    off1, k_pad1 = oracle.segment_offsets(size1)
    a = np.zeros((M, k_pad1), np.uint8)
    for c in range(g1):
        a[:, off1[c]:off1[c] + size1[c]] = rng.integers(0, 16, size=(M, size1[c]))
    case1 = dict(perm=perm1, size=size1, scale=scale1, zero=zero1, w_codes=w1_codes, s_w=s_w1, wsum=wsum1, a=a,
                 k_pad=k_pad1, bits=4, M=M, N=k_pad2, n_pad=k_pad2)
    d1 = _dev(case1)
    h64 = _oracle_y(case1, bias=b1, relu=True)                     # [M][k_pad2], the second site's padded order
    # second-site parameters from the observed range of h (Eq. 2 per cluster)
    scale2, zero2 = np.ones(g2, np.float32), np.zeros(g2, np.int32)
    for c in range(g2):
        if size2[c]:
            seg = h64[:, real & (cluster_of_pos == c)]
            s, z = oracle.minmax_params(seg.min(), seg.max(), out_bits)
            scale2[c], zero2[c] = s, z
    L2 = binding.Layout(perm2, size2, scale2, zero2, out_bits)
    assert L2.K_pad == k_pad2 and np.array_equal(L2.padded_index(), out_rows)
    # GPU: fp32 output and re-quantised output of the same launch parameters
    h32 = _gemm(case1, d1, bias=b1, act=binding.ACT_RELU)
    packed = _gemm(case1, d1, y_dtype=binding.OUT_CODES, bias=b1, act=binding.ACT_RELU, layout_out=L2)
    got = oracle.unpack(packed, k_pad2, out_bits)[:, np.argsort(m2)]           # back to the oracle's order
    # the decision, bit for bit, from the GPU's own fp32 values (real positions in reordered order)
    want32 = oracle.quantize_f32(h32[:, in_S_order], size2, scale2, zero2, out_bits)
    assert np.array_equal(got, want32)
    want64 = oracle.quantize(h64[:, in_S_order], size2, scale2.astype(np.float64), zero2, out_bits)
    diff = np.abs(got.astype(int) - want64.astype(int))
    # the decision is taken from the GEMM's fp32 output (error ~1e-6 of max|h|): a value crosses a
    # rounding boundary with probability ~ 4 * 2^bits * 1e-6, so the bar is 1e-4 + 2^bits * 4e-6
    assert diff.max() <= 1 and (diff != 0).mean() <= 1e-4 + (1 << out_bits) * 4e-6
    # FC2 on those codes, original output order
    W2 = (rng.normal(size=(C, H)) * 0.02).astype(np.float32)
    w2_codes, s_w2, wsum2 = oracle.weight_quantize(W2, perm2, size2, None, C)
    case2 = dict(perm=perm2, size=size2, scale=scale2, zero=zero2, w_codes=w2_codes, s_w=s_w2, wsum=wsum2, a=got,
                 k_pad=k_pad2, bits=out_bits, M=M, N=C, n_pad=C)
    d2 = _dev(case2)
    d2["a"] = torch.from_numpy(packed).cuda()
    y = _gemm(case2, d2)
    want_y = _oracle_y(case2)
    assert np.max(np.abs(y - want_y)) <= TOL * np.abs(want_y).max()


@pytest.mark.parametrize("out_bits", [4, 3, 8])
def test_requantised_outputs_far_outside_the_code_range(out_bits):
    """Eq. 1's clamp for every finite v / s: the output site's steps are so small that v / s' reaches
    +-1e6 ... +-1e9 on both sides (no ReLU), through and beyond the range where the rounded integer
    no longer fits the mantissa trick; zero points of both parities. Bit for bit against the oracle's
    fp32-decision quantiser on the GPU's own fp32 outputs."""
    from paper_2304_01089_b200 import binding
    rng = np.random.default_rng(140 + out_bits)
    M, C, H, g1, g2 = 130, 256, 416, 3, 5
    perm1, size1, scale1, zero1 = random_layout_params(rng, C, g1, 4)
    perm2, size2, _, _ = random_layout_params(rng, H, g2, out_bits, allow_empty=False)
    off2, k_pad2 = oracle.segment_offsets(size2)
    scale2 = np.array([3e-9, 2e-8, 7e-8, 4e-7, 0.05], np.float32)
    zero2 = np.array([0, 1, (1 << out_bits) - 1, 6, 3], np.int32)
    L2 = binding.Layout(perm2, size2, scale2, zero2, out_bits)
    out_rows = L2.padded_index().astype(np.int64)
    m2 = L2.contiguous_position()
    real = out_rows >= 0
    where = np.empty(H, np.int64)
    where[out_rows[real]] = np.nonzero(real)[0]
    in_S_order = where[perm2]
    W1 = (rng.normal(size=(H, C)) * 0.02).astype(np.float32)
    W1p = np.zeros((k_pad2, C), np.float32)
    W1p[real] = W1[out_rows[real]]
    w1_codes, s_w1, wsum1 = oracle.weight_quantize(W1p, perm1, size1, None, k_pad2)
    off1, k_pad1 = oracle.segment_offsets(size1)
    a = np.zeros((M, k_pad1), np.uint8)
    for c in range(g1):
        a[:, off1[c]:off1[c] + size1[c]] = rng.integers(0, 16, size=(M, size1[c]))
    case1 = dict(perm=perm1, size=size1, scale=scale1, zero=zero1, w_codes=w1_codes, s_w=s_w1, wsum=wsum1, a=a,
                 k_pad=k_pad1, bits=4, M=M, N=k_pad2, n_pad=k_pad2)
    d1 = _dev(case1)
    h32 = _gemm(case1, d1)
    packed = _gemm(case1, d1, y_dtype=binding.OUT_CODES, layout_out=L2)
    got = oracle.unpack(packed, k_pad2, out_bits)[:, np.argsort(m2)]
    h_S = h32[:, in_S_order]
    want32 = oracle.quantize_f32(h_S, size2, scale2, zero2, out_bits)
    assert np.array_equal(got, want32)
    # the case does reach the far windows on both sides
    t = h_S[:, :size2[0]].astype(np.float64) / float(scale2[0])
    for lo, hi in ((4e6, 1.2e7), (1.3e7, 2.5e7), (2.6e7, 1e12)):
        assert ((t > lo) & (t < hi)).any() and ((t < -lo) & (t > -hi)).any(), (lo, hi)
    assert np.all(want32[:, :size2[0]][t < -4e6] == 0) and np.all(want32[:, :size2[0]][t > 4e6] == (1 << out_bits) - 1)


def _workload_linear(site, li, rows):
    """Oracle inputs and expected outputs of one LN -> linear site on sampled token rows."""
    w = site.w
    lin = w.linears[li]
    W = workloads.weight_matrix(w, li, lin.n_out, w.hidden)
    w_codes, s_w, wsum = oracle.weight_quantize(W, site.cal.perm, site.cal.size, None, lin.n_out)
    y64 = oracle.reorder(oracle.layernorm(site.x[rows], site.gamma, site.beta, 1e-5), site.cal.perm)
    a = oracle.quantize(y64, site.cal.size, site.cal.scale.astype(np.float64), site.cal.zero, site.bits)
    return W, w_codes, s_w, wsum, a


@pytest.mark.parametrize("name", ["opt-125m", "opt-1.3b"])
def test_workload_configs_checked_in_full(name):
    import torch
    from paper_2304_01089_b200 import binding
    site = Site(workloads.WORKLOADS[name])
    w = site.w
    rows = np.arange(w.tokens)
    W, w_codes, s_w, wsum, a = _workload_linear(site, 0, rows)
    N = w.linears[0].n_out
    case = dict(perm=site.cal.perm, size=site.cal.size, scale=site.cal.scale, zero=site.cal.zero, w_codes=w_codes,
                s_w=s_w, wsum=wsum, a=a, k_pad=a.shape[1], bits=site.bits, M=w.tokens, N=N, n_pad=N)
    d = _dev(case)
    # the library's own offline weight preparation must give the same bytes as the oracle's
    packed_w, s_w_l, wsum_l = binding.weight_pack(d["L"], W)
    in_lib_order = np.ascontiguousarray(w_codes[:, d["L"].contiguous_position()])
    assert np.array_equal(packed_w, oracle.pack_weights(in_lib_order)) and np.array_equal(s_w_l, s_w) and np.array_equal(wsum_l, wsum)
    y = _gemm(case, d)
    want = _oracle_y(case)
    err = np.max(np.abs(y - want)) / np.abs(want).max()
    print(f"{name}: max|dy|/max|y| = {err:.2e}")
    assert err <= TOL
    # the integer method agrees with de-quantise-then-matmul on the same codes (Appendix)
    sub = slice(0, 8)
    ref = oracle.dequant_matmul(a[sub], w_codes, site.cal.size, site.cal.scale.astype(np.float64), site.cal.zero, s_w)
    assert np.max(np.abs(ref - want[sub])) <= 1e-10 * np.abs(want).max()


@pytest.mark.parametrize("order", [0, 1])
@pytest.mark.parametrize("bits", [4, 3, 8])
def test_few_tokens_take_the_direct_kernel_and_give_the_same_bits(bits, order):
    """Calls with at most 16 tokens run the kernel that feeds the weights straight into mma.sync (no
    tensor-memory tile); its result is right against the oracle and bit-identical to what the large
    kernel gives for the same tokens as part of a longer batch."""
    from paper_2304_01089_b200 import binding
    rng = np.random.default_rng(77 + bits + 10 * order)
    M_all, N, C, g = 40, 300, 1024, 33
    case = _case(rng, M_all, N, C, g, bits, n_pad=304)
    d = _dev(case, order=order)
    bias = (rng.normal(size=N) * 0.05).astype(np.float32)
    want = _oracle_y(case, bias=bias, relu=True)
    big = _gemm(case, d, bias=bias, act=binding.ACT_RELU, ldy=304)[:, :N]            # 40 tokens: the tcgen05 kernel
    assert np.max(np.abs(big - want)) <= TOL * np.abs(want).max()
    for M in (1, 7, 8, 9, 16):
        sub = dict(case, M=M)
        y32 = _gemm(sub, d, bias=bias, act=binding.ACT_RELU, ldy=304)[:, :N]
        assert np.max(np.abs(y32 - want[:M])) <= TOL * np.abs(want).max()
        assert np.array_equal(y32, big[:M])
        y16 = _gemm(sub, d, y_dtype=binding.OUT_F16, bias=bias, act=binding.ACT_RELU, ldy=304)[:, :N]
        assert np.array_equal(y16, big[:M].astype(np.float16))
    # no bias, no activation, an output pitch wider than N
    y = _gemm(dict(case, M=5), d, ldy=320)[:, :N]
    assert np.max(np.abs(y - _oracle_y(case)[:5])) <= TOL * np.abs(want).max()
