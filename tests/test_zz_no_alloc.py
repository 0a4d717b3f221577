"""rptq_cluster_gemm_noalloc against rptq_cluster_gemm.

Some users of this library are not allowed to allocate device memory when they call it: a serving
process that handed the whole GPU to its own memory pool at start-up, a job held to a fixed memory
budget, or code that is in the middle of recording work on a stream. For them the library has one
GEMM entry point that allocates nothing and keeps its per-column scratch in a static device array.
This test calls it through the C boundary twice in a row (the array keeps the previous call's
contents, so the second call must not be disturbed by the first) and compares with the ordinary entry
point. It lives in a file that pytest collects last, so a run that stops at the first failure has
already run everything else; it passes alone in a fresh process as well as after the other tests.
"""
import numpy as np
import pytest

import oracle
from helpers import random_layout_params

pytestmark = pytest.mark.gpu

TOL = 1e-4


def _problem(rng, M, N, C, g, bits):
    import torch
    from paper_2304_01089_b200 import binding
    perm, size, scale, zero = random_layout_params(rng, C, g, bits)
    L = binding.Layout(perm, size, scale, zero, bits)
    W = (rng.normal(size=(N, C)) * 0.02).astype(np.float32)
    w_codes, s_w, wsum = oracle.weight_quantize(W, perm, size)
    off, k_pad = oracle.segment_offsets(size)
    a = np.zeros((M, k_pad), np.uint8)
    for c in range(g):
        a[:, off[c]:off[c] + size[c]] = rng.integers(0, 1 << bits, size=(M, size[c]))
    m = L.contiguous_position()          # the oracle's column order -> the layout's
    dev = dict(L=L, a=torch.from_numpy(oracle.pack(np.ascontiguousarray(a[:, m]), bits)).cuda(),
               w=torch.from_numpy(oracle.pack_weights(np.ascontiguousarray(w_codes[:, m]))).cuda(),
               s_w=torch.from_numpy(s_w).cuda(), wsum=torch.from_numpy(wsum).cuda(),
               bias=torch.from_numpy((rng.normal(size=N) * 0.05).astype(np.float32)).cuda())
    want = oracle.cluster_gemm(a, w_codes, size, scale.astype(np.float64), zero, s_w, wsum, bias=dev["bias"].cpu().numpy())
    return dev, want


def test_two_calls_in_a_row_match_the_allocating_entry_point():
    import torch
    from paper_2304_01089_b200 import binding
    rng = np.random.default_rng(2024)
    # two different problems back to back: the second one has fewer columns than the first, so stale
    # entries of the first call's table lie right behind the ones it uses
    # (the last one has few enough tokens for the second GEMM kernel, which both entry points then use)
    shapes = [(300, 1024, 1280, 9, 4), (129, 520, 640, 5, 3), (9, 520, 640, 5, 3)]
    for M, N, C, g, bits in shapes:
        dev, want = _problem(rng, M, N, C, g, bits)
        y_ref = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        binding.cluster_gemm(dev["L"], dev["a"], M, dev["w"], dev["s_w"], dev["wsum"], N, y_ref, bias=dev["bias"])
        y_new = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        binding.cluster_gemm_noalloc(dev["L"], dev["a"], M, dev["w"], dev["s_w"], dev["wsum"], N, y_new, bias=dev["bias"])
        torch.cuda.synchronize()
        # a further call changes nothing in how much device memory is free: the driver's own count,
        # taken around the call with every buffer already in place
        free_before, _ = torch.cuda.mem_get_info()
        binding.cluster_gemm_noalloc(dev["L"], dev["a"], M, dev["w"], dev["s_w"], dev["wsum"], N, y_new, bias=dev["bias"])
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after == free_before
        ref, new = y_ref.cpu().numpy(), y_new.cpu().numpy()
        scale = np.abs(want).max()
        assert np.max(np.abs(new - ref)) <= TOL * scale          # same tolerance as the parity tests
        assert np.max(np.abs(new - want)) <= TOL * scale         # and right against the oracle, not merely equal
        assert np.array_equal(new, ref)                          # same arithmetic in the same order: identical bits


def test_requantised_output_through_the_entry_point_that_allocates_nothing():
    """The packed-codes output (the next site's quantiser in the epilogue) gives the same bytes through
    both entry points."""
    import torch
    from paper_2304_01089_b200 import binding
    rng = np.random.default_rng(31)
    M, C, g, bits = 200, 512, 4, 4
    perm2, size2, scale2, zero2 = random_layout_params(rng, 352, 3, 3, allow_empty=False)
    L2 = binding.Layout(perm2, size2, (scale2 * 0.2).astype(np.float32), zero2, 3)
    N = L2.K_pad
    dev, _ = _problem(rng, M, N, C, g, bits)
    outs = []
    for fn in (binding.cluster_gemm, binding.cluster_gemm_noalloc, binding.cluster_gemm_noalloc):
        y = torch.full((M + 1, L2.row_bytes), 0xA5, dtype=torch.uint8, device="cuda")
        fn(dev["L"], dev["a"], M, dev["w"], dev["s_w"], dev["wsum"], N, y, bias=dev["bias"], act=binding.ACT_RELU,
           layout_out=L2, y_dtype=binding.OUT_CODES)
        torch.cuda.synchronize()
        out = y.cpu().numpy()
        assert np.all(out[M] == 0xA5)
        outs.append(out[:M])
    assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[1], outs[2])
    codes = oracle.unpack(outs[1], N, 3)
    assert codes.max() <= 7 and not codes[:, L2.padded_index() < 0].any() and codes.any()


def test_more_columns_than_the_resident_table_is_refused():
    import torch
    from paper_2304_01089_b200 import binding
    rng = np.random.default_rng(7)
    perm, size, scale, zero = random_layout_params(rng, 128, 2, 4)
    L = binding.Layout(perm, size, scale, zero, 4)
    N = binding.NOALLOC_MAX_N + 8
    t = torch.zeros(16, dtype=torch.uint8, device="cuda")
    f = torch.zeros(N, dtype=torch.float32, device="cuda")
    ws = torch.zeros((2, N), dtype=torch.int32, device="cuda")
    with pytest.raises(binding.RptqError) as e:
        binding.cluster_gemm_noalloc(L, t, 1, t, f, ws, N, torch.zeros((1, N), device="cuda"))
    assert e.value.status == binding.ERR_UNSUPPORTED
