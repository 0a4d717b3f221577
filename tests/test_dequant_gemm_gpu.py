"""rptq_dequant_gemm (Appendix, first computation method as a bfloat16 tensor-core product) against the
oracle's statement of it with bfloat16 operands, and its distance from the exact first method."""
import numpy as np
import pytest

import oracle
from paper_2304_01089_b200 import workloads
from helpers import Site, random_layout_params

pytestmark = pytest.mark.gpu

TOL = 1e-4


def _run(rng, M, N, C, g, bits, order=0, relu=False, f16=False, zero=None):
    import torch
    from paper_2304_01089_b200 import binding
    perm, size, scale, zero_r = random_layout_params(rng, C, g, bits)
    zero = zero_r if zero is None else zero
    L = binding.Layout(perm, size, scale, zero, bits, order=order)
    n_pad = (N + 7) // 8 * 8
    W = (rng.normal(size=(N, C)) * 0.02).astype(np.float32)
    w_o, s_w, _ = oracle.weight_quantize(W, perm, size, None, n_pad)
    off, k_pad = oracle.segment_offsets(size)
    a = np.zeros((M, k_pad), np.uint8)
    for c in range(g):
        a[:, off[c]:off[c] + size[c]] = rng.integers(0, 1 << bits, size=(M, size[c]))
    m = L.contiguous_position()
    a_dev = torch.from_numpy(oracle.pack(np.ascontiguousarray(a[:, m]), bits)).cuda()
    w_dev = torch.from_numpy(oracle.pack_weights(np.ascontiguousarray(w_o[:, m]))).cuda()
    bias = (rng.normal(size=n_pad) * 0.05).astype(np.float32)
    y = torch.full((M + 1, n_pad + 8), float("nan"), dtype=torch.float16 if f16 else torch.float32, device="cuda")
    binding.dequant_gemm(L, a_dev, M, w_dev, torch.from_numpy(s_w).cuda(), N, y, ld_w=n_pad, bias=torch.from_numpy(bias).cuda(),
                         act=binding.ACT_RELU if relu else binding.ACT_NONE, y_dtype=binding.OUT_F16 if f16 else binding.OUT_F32)
    torch.cuda.synchronize()
    assert binding.get_device_status() == 0
    out = y.float().cpu().numpy()
    assert np.all(np.isnan(out[M])) and np.all(np.isnan(out[:M, N:]))
    want = oracle.dequant_matmul_bf16(a, w_o[:N], size, scale, zero, s_w, bias=bias[:N], relu=relu)
    exact = oracle.dequant_matmul(a, w_o[:N], size, scale.astype(np.float64), zero, s_w) + bias[:N]
    if relu:
        exact = np.maximum(exact, 0)
    return out[:M, :N], want, exact


@pytest.mark.parametrize("bits", [4, 3, 8])
@pytest.mark.parametrize("M,N,C,g", [(1, 256, 128, 1), (127, 200, 384, 5), (129, 520, 640, 7), (300, 256, 1024, 33)])
def test_small_and_ragged_shapes(bits, M, N, C, g):
    rng = np.random.default_rng(9000 + 10 * bits + M)
    got, want, exact = _run(rng, M, N, C, g, bits)
    assert np.max(np.abs(got - want)) <= TOL * np.abs(want).max()
    # the first method with bfloat16 operands stays within the rounding of its operands of the exact one
    assert np.max(np.abs(got - exact)) <= 2e-2 * np.abs(exact).max()


def test_interleaved_order_relu_fp16_and_large_zero_points():
    from paper_2304_01089_b200 import binding
    rng = np.random.default_rng(9100)
    got, want, _ = _run(rng, 260, 512, 1536, 40, 4, order=binding.ORDER_INTERLEAVED, relu=True)
    assert np.max(np.abs(got - want)) <= TOL * np.abs(want).max() and got.min() >= 0
    rng = np.random.default_rng(9100)
    got16, want, _ = _run(rng, 260, 512, 1536, 40, 4, order=binding.ORDER_INTERLEAVED, relu=True, f16=True)
    assert np.array_equal(got16.astype(np.float16), got.astype(np.float16))
    rng = np.random.default_rng(9101)
    z = np.array([-1000, 70000, 3, 0, 15, -7], np.int32)
    got, want, _ = _run(rng, 130, 256, 768, 6, 4, zero=z)
    assert np.max(np.abs(got - want)) <= TOL * np.abs(want).max()


@pytest.mark.parametrize("name,li,Ms", [("opt-1.3b", 0, (2048,)), ("opt-66b", 1, (16, 4096))])
def test_workload_sites_sampled_rows(name, li, Ms):
    import torch
    from paper_2304_01089_b200 import binding
    site = Site(workloads.WORKLOADS[name])
    w = site.w
    N = w.linears[li].n_out
    L = site.layout(order=binding.ORDER_INTERLEAVED)
    W = workloads.weight_matrix(w, li, N, w.hidden)
    packed, s_w, _ = binding.weight_pack(L, W)
    cols = np.r_[0:40, N // 2:N // 2 + 40, N - 40:N]
    w_o, s_o, _ = oracle.weight_quantize(np.ascontiguousarray(W[cols]), site.cal.perm, site.cal.size)
    del W
    wd, sd = torch.from_numpy(packed).cuda(), torch.from_numpy(s_w).cuda()
    for M in Ms:
        rows = np.array(sorted(set(np.random.default_rng(M).choice(M, min(10, M), replace=False).tolist()) | {0, M - 1}))
        y64 = oracle.reorder(oracle.layernorm(site.x[rows], site.gamma, site.beta, 1e-5), site.cal.perm)
        a = oracle.quantize(y64, site.cal.size, site.cal.scale.astype(np.float64), site.cal.zero, site.bits)
        codes = torch.zeros((M, L.row_bytes), dtype=torch.uint8, device="cuda")
        ridx = torch.from_numpy(rows).cuda()
        codes[ridx] = torch.from_numpy(oracle.pack(np.ascontiguousarray(a[:, L.contiguous_position()]), site.bits)).cuda()
        y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        binding.dequant_gemm(L, codes, M, wd, sd, N, y)
        torch.cuda.synchronize()
        assert binding.get_device_status() == 0 and not bool(torch.isnan(y).any())
        got = y[ridx][:, torch.from_numpy(cols).cuda()].cpu().numpy()
        want = oracle.dequant_matmul_bf16(a, w_o, site.cal.size, site.cal.scale, site.cal.zero, s_o)
        err = np.max(np.abs(got - want)) / np.abs(want).max()
        exact = oracle.dequant_matmul(a, w_o, site.cal.size, site.cal.scale.astype(np.float64), site.cal.zero, s_o)
        print(f"{name} M={M}: max|dy|/max|y| = {err:.2e} vs the bf16 statement, {np.max(np.abs(got - exact)) / np.abs(exact).max():.2e} vs the exact first method")
        assert err <= TOL
