"""Per-cluster asymmetric weight parameters (Appendix: W~_q,i = Q_k(W~_i, s^W_i, z^W_i) and the second
computation method with all four terms) through the C boundary against the CPU oracle."""
import numpy as np
import pytest

import oracle
from paper_2304_01089_b200 import workloads
from helpers import Site, random_layout_params

pytestmark = pytest.mark.gpu

TOL = 1e-4


def _signed_in_layout_order(codes_u, L, size):
    """The oracle's unsigned codes (contiguous order, pads 0) as the library stores them: code - 8 at the
    real positions, 0 at the pads, columns in the layout's order."""
    off, k_pad = oracle.segment_offsets(size)
    real = np.zeros(k_pad, bool)
    for o, n in zip(off, size):
        real[o:o + n] = True
    signed = np.where(real[None, :], codes_u.astype(np.int16) - 8, 0).astype(np.int8)
    return np.ascontiguousarray(signed[:, L.contiguous_position()])


def _run_case(rng, M, N, C, g, bits, order=0, bias=True, relu=False, y_dtype=None, n_pad=None):
    import torch
    from paper_2304_01089_b200 import binding
    perm, size, scale, zero = random_layout_params(rng, C, g, bits)
    L = binding.Layout(perm, size, scale, zero, bits, order=order)
    n_pad = (N + 3) // 4 * 4 if n_pad is None else n_pad
    W = (rng.normal(size=(N, C)) * rng.lognormal(0, 0.7, size=C) * 0.02).astype(np.float32)
    # offline weight preparation: the library's bytes and tables equal the oracle's
    w_o, s_o, z_o, ws_o = oracle.weight_quantize_clustered(W, perm, size, 4, n_pad)
    packed, s_w, z_w, wsum = binding.weight_pack_clustered(L, W, n_pad)
    assert np.array_equal(s_w, s_o) and np.array_equal(z_w, z_o) and np.array_equal(wsum, ws_o)
    assert np.array_equal(packed, oracle.pack_weights(_signed_in_layout_order(w_o, L, size)))
    # activation codes from the oracle's side
    off, k_pad = oracle.segment_offsets(size)
    a = np.zeros((M, k_pad), np.uint8)
    for c in range(g):
        a[:, off[c]:off[c] + size[c]] = rng.integers(0, 1 << bits, size=(M, size[c]))
    a_dev = torch.from_numpy(oracle.pack(np.ascontiguousarray(a[:, L.contiguous_position()]), bits)).cuda()
    xsum = torch.full((M + 1, g), -7, dtype=torch.int32, device="cuda")
    binding.code_rowsums(L, a_dev, M, xsum)
    torch.cuda.synchronize()
    xs = xsum.cpu().numpy()
    assert np.array_equal(xs[:M], oracle.code_rowsums(a, size)) and np.all(xs[M] == -7)
    b = (rng.normal(size=n_pad) * 0.05).astype(np.float32) if bias else None
    want = oracle.cluster_gemm_asym(a, w_o[:N], size, scale.astype(np.float64), zero, s_o, z_o,
                                    bias=None if b is None else b[:N], relu=relu)
    dt = torch.float32 if y_dtype in (None, binding.OUT_F32) else torch.float16
    y = torch.full((M + 1, n_pad + 8), float("nan"), dtype=dt, device="cuda")
    binding.cluster_gemm_clustered(L, a_dev, M, xsum, torch.from_numpy(packed).cuda(), torch.from_numpy(s_w).cuda(),
                                   torch.from_numpy(z_w).cuda(), torch.from_numpy(wsum).cuda(), N, y,
                                   bias=None if b is None else torch.from_numpy(b).cuda(),
                                   act=binding.ACT_RELU if relu else binding.ACT_NONE,
                                   y_dtype=binding.OUT_F32 if y_dtype is None else y_dtype)
    torch.cuda.synchronize()
    assert binding.get_device_status() == 0
    out = y.float().cpu().numpy()
    assert np.all(np.isnan(out[M])) and np.all(np.isnan(out[:M, N:]))
    return out[:M, :N], want


@pytest.mark.parametrize("bits", [4, 3, 8])
@pytest.mark.parametrize("M,N,C,g", [(1, 256, 128, 1), (127, 200, 384, 5), (129, 520, 640, 7), (300, 260, 1024, 33)])
def test_small_and_ragged_shapes(bits, M, N, C, g):
    rng = np.random.default_rng(7000 + 10 * bits + M)
    got, want = _run_case(rng, M, N, C, g, bits)
    assert np.max(np.abs(got - want)) <= TOL * np.abs(want).max()


def test_interleaved_order_relu_and_fp16_output():
    from paper_2304_01089_b200 import binding
    rng = np.random.default_rng(7100)
    got, want = _run_case(rng, 260, 512, 1536, 40, 4, order=binding.ORDER_INTERLEAVED, relu=True)
    assert np.max(np.abs(got - want)) <= TOL * np.abs(want).max() and got.min() >= 0
    rng = np.random.default_rng(7100)
    got16, _ = _run_case(rng, 260, 512, 1536, 40, 4, order=binding.ORDER_INTERLEAVED, relu=True, y_dtype=binding.OUT_F16)
    assert np.array_equal(got16.astype(np.float16), got.astype(np.float16))


def test_reduces_to_the_symmetric_entry_point():
    """s^W_c the same for every cluster and z^W = 8: the four-term path must reproduce rptq_cluster_gemm
    on the same stored nibbles."""
    import torch
    from paper_2304_01089_b200 import binding
    rng = np.random.default_rng(7200)
    M, N, C, g, bits = 200, 384, 768, 6, 4
    perm, size, scale, zero = random_layout_params(rng, C, g, bits)
    L = binding.Layout(perm, size, scale, zero, bits)
    W = (rng.normal(size=(N, C)) * 0.02).astype(np.float32)
    packed, s_w, wsum = binding.weight_pack(L, W)
    off, k_pad = oracle.segment_offsets(size)
    a = np.zeros((M, k_pad), np.uint8)
    for c in range(g):
        a[:, off[c]:off[c] + size[c]] = rng.integers(0, 16, size=(M, size[c]))
    a_dev = torch.from_numpy(oracle.pack(np.ascontiguousarray(a[:, L.contiguous_position()]), bits)).cuda()
    y_sym = torch.empty((M, N), dtype=torch.float32, device="cuda")
    binding.cluster_gemm(L, a_dev, M, torch.from_numpy(packed).cuda(), torch.from_numpy(s_w).cuda(), torch.from_numpy(wsum).cuda(), N, y_sym)
    xsum = torch.empty((M, g), dtype=torch.int32, device="cuda")
    binding.code_rowsums(L, a_dev, M, xsum)
    # unsigned view of the same nibbles: W_q = w + 8, z^W = 8, Wsum_u = Wsum + 8 n_c
    wsum_u = (wsum + 8 * size[:, None]).astype(np.int32)
    y_asym = torch.empty((M, N), dtype=torch.float32, device="cuda")
    binding.cluster_gemm_clustered(L, a_dev, M, xsum, torch.from_numpy(packed).cuda(), torch.from_numpy(np.tile(s_w, (g, 1))).cuda(),
                                   torch.full((g, N), 8, dtype=torch.int32, device="cuda"), torch.from_numpy(wsum_u).cuda(), N, y_asym)
    torch.cuda.synchronize()
    ref = y_sym.cpu().numpy()
    assert np.max(np.abs(y_asym.cpu().numpy() - ref)) <= 1e-5 * np.abs(ref).max()


@pytest.mark.parametrize("name", ["opt-125m", "opt-1.3b"])
def test_workload_configs_checked_in_full(name):
    """LN -> linear with clustered weights on the calibrated layout, every token, against the oracle."""
    import torch
    from paper_2304_01089_b200 import binding
    site = Site(workloads.WORKLOADS[name])
    w = site.w
    N = w.linears[0].n_out
    L = site.layout(order=binding.ORDER_INTERLEAVED)
    W = workloads.weight_matrix(w, 0, N, w.hidden)
    w_o, s_o, z_o, ws_o = oracle.weight_quantize_clustered(W, site.cal.perm, site.cal.size, 4)
    packed, s_w, z_w, wsum = binding.weight_pack_clustered(L, W)
    assert np.array_equal(packed, oracle.pack_weights(_signed_in_layout_order(w_o, L, site.cal.size)))
    assert np.array_equal(s_w, s_o) and np.array_equal(z_w, z_o) and np.array_equal(wsum, ws_o)
    y64 = oracle.reorder(oracle.layernorm(site.x, site.gamma, site.beta, 1e-5), site.cal.perm)
    a = oracle.quantize(y64, site.cal.size, site.cal.scale.astype(np.float64), site.cal.zero, site.bits)
    M = a.shape[0]
    a_dev = torch.from_numpy(oracle.pack(np.ascontiguousarray(a[:, L.contiguous_position()]), site.bits)).cuda()
    xsum = torch.empty((M, L.g), dtype=torch.int32, device="cuda")
    binding.code_rowsums(L, a_dev, M, xsum)
    y = torch.empty((M, N), dtype=torch.float32, device="cuda")
    binding.cluster_gemm_clustered(L, a_dev, M, xsum, torch.from_numpy(packed).cuda(), torch.from_numpy(s_w).cuda(),
                                   torch.from_numpy(z_w).cuda(), torch.from_numpy(wsum).cuda(), N, y)
    torch.cuda.synchronize()
    assert binding.get_device_status() == 0
    want = oracle.cluster_gemm_asym(a, w_o, site.cal.size, site.cal.scale.astype(np.float64), site.cal.zero, s_o, z_o)
    err = np.max(np.abs(y.cpu().numpy() - want)) / np.abs(want).max()
    print(f"{name}: clustered weights max|dy|/max|y| = {err:.2e}")
    assert err <= TOL
    assert np.array_equal(xsum.cpu().numpy(), oracle.code_rowsums(a, site.cal.size))


def test_opt66b_fc1_sampled_rows_full_launch_shape():
    """4096 x 9216 x 36864 (the benchmark's launch shape) with clustered weights: sampled rows."""
    import torch
    from paper_2304_01089_b200 import binding
    site = Site(workloads.WORKLOADS["opt-66b"])
    w = site.w
    N, M = w.linears[1].n_out, w.tokens
    L = site.layout(order=binding.ORDER_INTERLEAVED)
    W = workloads.weight_matrix(w, 1, N, w.hidden)
    packed, s_w, z_w, wsum = binding.weight_pack_clustered(L, W)
    rows = np.array(sorted(set(np.random.default_rng(5).choice(M, 10, replace=False).tolist()) | {0, 127, 128, M - 1}))
    cols = np.r_[0:40, 18000:18040, N - 40:N]
    w_o, s_o, z_o, ws_o = oracle.weight_quantize_clustered(np.ascontiguousarray(W[cols]), site.cal.perm, site.cal.size, 4)
    assert np.array_equal(s_w[:, cols], s_o) and np.array_equal(z_w[:, cols], z_o) and np.array_equal(wsum[:, cols], ws_o)
    del W
    xd = torch.from_numpy(site.x).cuda()
    codes = torch.empty((M, L.row_bytes), dtype=torch.uint8, device="cuda")
    binding.ln_reorder_quant(L, xd, torch.from_numpy(site.gamma).cuda(), torch.from_numpy(site.beta).cuda(), 1e-5, codes)
    y64 = oracle.reorder(oracle.layernorm(site.x[rows], site.gamma, site.beta, 1e-5), site.cal.perm)
    a = oracle.quantize(y64, site.cal.size, site.cal.scale.astype(np.float64), site.cal.zero, site.bits)
    ridx = torch.from_numpy(rows).cuda()
    codes[ridx] = torch.from_numpy(oracle.pack(np.ascontiguousarray(a[:, L.contiguous_position()]), site.bits)).cuda()
    xsum = torch.empty((M, L.g), dtype=torch.int32, device="cuda")
    binding.code_rowsums(L, codes, M, xsum)
    y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    binding.cluster_gemm_clustered(L, codes, M, xsum, torch.from_numpy(packed).cuda(), torch.from_numpy(s_w).cuda(),
                                   torch.from_numpy(z_w).cuda(), torch.from_numpy(wsum).cuda(), N, y)
    torch.cuda.synchronize()
    assert binding.get_device_status() == 0 and not bool(torch.isnan(y).any())
    want = oracle.cluster_gemm_asym(a, w_o, site.cal.size, site.cal.scale.astype(np.float64), site.cal.zero, s_o, z_o)
    got = y[ridx][:, torch.from_numpy(cols).cuda()].cpu().numpy()
    err = np.max(np.abs(got - want)) / np.abs(want).max()
    print(f"opt-66b FC1 clustered weights: max|dy|/max|y| = {err:.2e} on {len(rows)} rows x {len(cols)} columns")
    assert err <= TOL
    assert np.array_equal(xsum[ridx].cpu().numpy(), oracle.code_rowsums(a, site.cal.size))
