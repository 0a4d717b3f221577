"""Parity of rptq_ln_reorder_quant (CUDA, through the C boundary) against the CPU oracle."""
import numpy as np
import pytest

import oracle
from paper_2304_01089_b200 import workloads
from helpers import Site, random_layout_params

pytestmark = pytest.mark.gpu

EPS = 1e-5
CANARY = 0xA5


def _run(layout, x16, gamma16, beta16, want_y=True, ldx=None, stream=None):
    import torch
    from paper_2304_01089_b200 import binding
    M, C = x16.shape
    ldx = C if ldx is None else ldx
    xd = torch.zeros((max(M, 1), ldx), dtype=torch.float16, device="cuda")
    xd[:M, :C] = torch.from_numpy(x16).cuda()
    gd, bd = torch.from_numpy(gamma16).cuda(), torch.from_numpy(beta16).cuda()
    # one extra row of canary bytes behind the output
    codes = torch.full((M + 1, layout.row_bytes), CANARY, dtype=torch.uint8, device="cuda")
    y_dbg = torch.full((M + 1, C), float("nan"), dtype=torch.float32, device="cuda") if want_y else None
    binding.ln_reorder_quant(layout, xd, gd, bd, EPS, codes, y_dbg, M=M, ldx=ldx, stream=stream)
    torch.cuda.synchronize()
    assert binding.get_device_status() == 0
    codes_h = codes.cpu().numpy()
    assert np.all(codes_h[M] == CANARY), "wrote past the last row"
    y_h = None
    if want_y:
        y_h = y_dbg.cpu().numpy()
        assert np.all(np.isnan(y_h[M]))
        y_h = y_h[:M]
    return codes_h[:M], y_h


def _check_against_oracle(x16, gamma16, beta16, perm, size, scale32, zero, bits, packed, y_dbg, full_rate=0.9999, pos=None, L=None):
    """`pos`: the layout's contiguous_position() when its unit order is not the contiguous one (the
    oracle's codes are in contiguous order)."""
    M, C = x16.shape
    _, k_pad = oracle.segment_offsets(size)
    pos = L.contiguous_position() if pos is None else pos
    got = oracle.unpack(packed, k_pad, bits)[:, np.argsort(pos)]          # back to contiguous order
    # (1) the decision, bit for bit, from the kernel's own fp32 LayerNorm outputs
    want32 = oracle.quantize_f32(y_dbg, size, scale32, zero, bits)
    assert np.array_equal(got, want32), "codes differ from the fp32-decision oracle on identical LN outputs"
    assert np.array_equal(packed, oracle.pack(np.ascontiguousarray(want32[:, pos]), bits)), "packed bytes differ from the documented format"
    # (2) the whole step against the fp64 oracle
    y64 = oracle.reorder(oracle.layernorm(x16, gamma16, beta16, EPS), perm)
    want64 = oracle.quantize(y64, size, scale32.astype(np.float64), zero, bits)
    diff = np.abs(got.astype(np.int16) - want64.astype(np.int16))
    assert diff.max() <= 1, f"a code is off by {diff.max()}"
    off, _ = oracle.segment_offsets(size)
    real = np.concatenate([np.arange(off[c], off[c] + size[c]) for c in range(len(size))])
    rate = 1.0 - diff[:, real].astype(bool).mean()
    assert rate >= full_rate, f"only {rate:.6f} of the codes equal the fp64 oracle's"
    # (3) the LayerNorm outputs themselves
    tol = 2e-6 * np.abs(y64).max() + 1e-6
    assert np.max(np.abs(y_dbg - y64)) <= 4 * tol
    return rate


@pytest.mark.parametrize("name", ["opt-125m", "opt-1.3b", "opt-6.7b", "opt-66b", "opt-175b"])
def test_workload_configs_full_size(name):
    from paper_2304_01089_b200 import binding
    site = Site(workloads.WORKLOADS[name])
    L = site.layout(order=binding.ORDER_INTERLEAVED)       # the order the benchmark uses
    packed, y_dbg = _run(L, site.x, site.gamma, site.beta)
    rate = _check_against_oracle(site.x, site.gamma, site.beta, site.cal.perm, site.cal.size, site.cal.scale,
                                 site.cal.zero, site.bits, packed, y_dbg, pos=L.contiguous_position())
    print(f"{name}: {rate:.6f} of codes equal the fp64 oracle")
    # same launch without the debug output and on another stream: identical bytes
    import torch
    s2 = torch.cuda.Stream()
    packed2, _ = _run(L, site.x, site.gamma, site.beta, want_y=False, stream=s2)
    assert np.array_equal(packed, packed2)


@pytest.mark.parametrize("bits", [3, 4, 8])
@pytest.mark.parametrize("M", [1, 2, 127, 129])
def test_small_and_ragged_shapes_all_bit_widths(bits, M):
    rng = np.random.default_rng(100 * bits + M)
    C, g = 384, 5
    perm, size, scale, zero = random_layout_params(rng, C, g, bits)
    from paper_2304_01089_b200 import binding
    L = binding.Layout(perm, size, scale, zero, bits)
    x = (rng.normal(size=(M, C)) * 2).astype(np.float16)
    gm = rng.lognormal(0, 0.5, C).astype(np.float16)
    bt = rng.normal(size=C).astype(np.float16)
    packed, y_dbg = _run(L, x, gm, bt, ldx=C + 24)
    _check_against_oracle(x, gm, bt, perm, size, scale, zero, bits, packed, y_dbg, L=L)


@pytest.mark.parametrize("bits", [3, 4, 8])
def test_degenerate_clusterings(bits):
    from paper_2304_01089_b200 import binding
    rng = np.random.default_rng(7 + bits)
    C, M = 128, 33
    x = rng.normal(size=(M, C)).astype(np.float16)
    gm = rng.lognormal(0, 0.5, C).astype(np.float16)
    bt = rng.normal(size=C).astype(np.float16)
    # g = 1 with the identity index: plain LayerNorm + per-tensor quantisation
    perm = np.arange(C, dtype=np.int32)
    one = (perm, np.array([C], np.int32), np.array([0.21], np.float32), np.array([(1 << bits) // 2], np.int32))
    # g = C: one channel per cluster (per-channel quantisation), K_pad = 32 * C
    per_ch = (rng.permutation(C).astype(np.int32), np.ones(C, np.int32),
              rng.uniform(0.05, 0.6, C).astype(np.float32), rng.integers(0, 1 << bits, C).astype(np.int32))
    # many empty clusters
    size = np.zeros(9, np.int32); size[2], size[7] = 100, 28
    empty = (rng.permutation(C).astype(np.int32), size, rng.uniform(0.1, 0.5, 9).astype(np.float32),
             rng.integers(0, 1 << bits, 9).astype(np.int32))
    for perm_, size_, scale_, zero_ in (one, per_ch, empty):
        L = binding.Layout(perm_, size_, scale_, zero_, bits)
        packed, y_dbg = _run(L, x, gm, bt)
        _check_against_oracle(x, gm, bt, perm_, size_, scale_, zero_, bits, packed, y_dbg, L=L)


def test_wide_rows_take_the_multi_unit_path_and_zero_tokens_launch_nothing():
    from paper_2304_01089_b200 import binding
    import torch
    rng = np.random.default_rng(11)
    C, g, bits, M = 13312, 256, 4, 9
    perm, size, scale, zero = random_layout_params(rng, C, g, bits)
    L = binding.Layout(perm, size, scale, zero, bits)
    assert L.K_pad // 32 > 512
    x = rng.normal(size=(M, C)).astype(np.float16)
    gm = rng.lognormal(0, 0.5, C).astype(np.float16)
    bt = rng.normal(size=C).astype(np.float16)
    packed, y_dbg = _run(L, x, gm, bt)
    _check_against_oracle(x, gm, bt, perm, size, scale, zero, bits, packed, y_dbg, L=L)
    codes = torch.full((4, L.row_bytes), CANARY, dtype=torch.uint8, device="cuda")
    xd = torch.zeros((1, C), dtype=torch.float16, device="cuda")
    binding.ln_reorder_quant(L, xd, torch.from_numpy(gm).cuda(), torch.from_numpy(bt).cuda(), EPS, codes, None, M=0)
    torch.cuda.synchronize()
    assert bool((codes == CANARY).all())


@pytest.mark.parametrize("ratio,bound", [(1.5, 8e-6), (4.0, 8e-6), (32.0, 8e-6)])
def test_row_mean_far_from_zero(ratio, bound):
    """The kernel takes the variance as sum(x^2)/C - mean^2 from fp32 sums unless the row's mean is
    more than two standard deviations from zero (then a centred second pass): LayerNorm outputs
    against the fp64 oracle on rows whose mean is `ratio` standard deviations away from zero, on both
    sides of that switch, relative to max|y|."""
    from paper_2304_01089_b200 import binding
    rng = np.random.default_rng(int(ratio))
    C, M, bits = 4096, 64, 4
    perm, size, scale, zero = random_layout_params(rng, C, 8, bits)
    L = binding.Layout(perm, size, scale, zero, bits)
    x = (rng.normal(size=(M, C)) + ratio).astype(np.float16)
    gm = rng.lognormal(0, 0.3, C).astype(np.float16)
    bt = rng.normal(size=C).astype(np.float16)
    _, y_dbg = _run(L, x, gm, bt)
    y64 = oracle.reorder(oracle.layernorm(x, gm, bt, EPS), perm)
    err = np.max(np.abs(y_dbg - y64)) / np.abs(y64).max()
    print(f"mean = {ratio} std: max|dy|/max|y| = {err:.2e}")
    assert err <= bound


def test_wide_then_narrow_then_wide_layouts():
    """The kernel's launch set-up is cached per shape; a narrow layout (little shared memory) between
    two uses of a wide one (nearly all of it) must not take the wide one's shared memory away."""
    from paper_2304_01089_b200 import binding
    rng = np.random.default_rng(21)
    cases = []
    for C in (9216, 256, 9216):
        perm, size, scale, zero = random_layout_params(rng, C, 6, 4)
        x = rng.normal(size=(5, C)).astype(np.float16)
        gm = rng.lognormal(0, 0.3, C).astype(np.float16)
        bt = rng.normal(size=C).astype(np.float16)
        L = binding.Layout(perm, size, scale, zero, 4)
        packed, y_dbg = _run(L, x, gm, bt, want_y=False)
        packed2, y_dbg = _run(L, x, gm, bt)
        assert np.array_equal(packed, packed2)
        _check_against_oracle(x, gm, bt, perm, size, scale, zero, 4, packed2, y_dbg, L=L)


@pytest.mark.parametrize("bits", [3, 4, 8])
def test_values_far_outside_the_code_range(bits):
    """Eq. 1's clamp for every finite y / s: large gains and small steps put y / s at +-1e5 ... +-1e9,
    through and beyond the range where rne(y / s) + z still fits the arithmetic trick of the kernel;
    zero points of both parities (odd ones take the mirrored-code path). Bit for bit against the
    oracle's fp32-decision quantiser on the kernel's own LayerNorm outputs."""
    from paper_2304_01089_b200 import binding
    rng = np.random.default_rng(300 + bits)
    C, M, g = 512, 70, 6
    perm = rng.permutation(C).astype(np.int32)
    size = np.array([100, 60, 37, 200, 3, 112], np.int32)
    scale = np.array([1e-4, 3e-3, 2e-5, 0.3, 1e-6, 5e-4], np.float32)
    zero = np.array([0, 1, (1 << bits) - 1, 5, 2, (1 << bits) + 3], np.int32)
    L = binding.Layout(perm, size, scale, zero, bits)
    x = rng.normal(size=(M, C)).astype(np.float16)
    gm = np.exp(rng.uniform(np.log(0.5), np.log(6e4), C)).astype(np.float16)      # gains up to the fp16 range
    bt = (rng.normal(size=C) * 10).astype(np.float16)
    packed, y_dbg = _run(L, x, gm, bt)
    pos = L.contiguous_position()
    got = oracle.unpack(packed, L.K_pad, bits)[:, np.argsort(pos)]
    want32 = oracle.quantize_f32(y_dbg, size, scale, zero, bits)
    assert np.array_equal(got, want32), "codes differ from the fp32-decision oracle"
    # the case does reach the far windows on both sides, in every cluster parity
    off, _ = oracle.segment_offsets(size)
    inv = np.concatenate([np.full(n, 1.0 / float(s)) for n, s in zip(size, scale)])
    t = y_dbg.astype(np.float64) * inv
    for lo, hi in ((4e6, 1.2e7), (1.3e7, 2.5e7), (2.6e7, 1e12)):
        assert ((t > lo) & (t < hi)).any() and ((t < -lo) & (t > -hi)).any(), (lo, hi)
    real = np.concatenate([np.arange(off[c], off[c] + size[c]) for c in range(g)])
    w = want32[:, real]
    assert np.all(w[t < -4e6] == 0) and np.all(w[t > 4e6] == (1 << bits) - 1)
    # and the LayerNorm outputs agree with the fp64 oracle
    y64 = oracle.reorder(oracle.layernorm(x, gm, bt, EPS), perm)
    assert np.max(np.abs(y_dbg - y64)) <= 8e-6 * np.abs(y64).max()


def test_non_finite_inputs_still_give_in_range_codes():
    from paper_2304_01089_b200 import binding
    rng = np.random.default_rng(12)
    C, bits = 256, 4
    perm, size, scale, zero = random_layout_params(rng, C, 3, bits)
    L = binding.Layout(perm, size, scale, zero, bits)
    x = rng.normal(size=(4, C)).astype(np.float16)
    x[1, 5] = np.inf
    x[2, 9] = np.nan
    gm = np.ones(C, np.float16); bt = np.zeros(C, np.float16)
    packed, _ = _run(L, x, gm, bt)
    got = oracle.unpack(packed, L.K_pad, bits)
    assert got.max() <= 15
    pads = L.padded_index() < 0
    assert not got[:, pads].any()


def test_a_wait_that_runs_out_is_reported_and_the_next_launch_is_clean():
    """The give-up path, made to happen without any fault: the library's self-test launch gives every
    row's barrier an expectation that cannot be met and a ~5 ms budget. The kernel must come back, the
    status word must read RPTQ_ERR_DEVICE_TIMEOUT exactly once, and an ordinary launch afterwards must
    give the same bytes as one before."""
    import time
    import torch
    from paper_2304_01089_b200 import binding
    rng = np.random.default_rng(55)
    C, M, bits = 1024, 600, 4
    perm, size, scale, zero = random_layout_params(rng, C, 6, bits)
    L = binding.Layout(perm, size, scale, zero, bits)
    x = rng.normal(size=(M, C)).astype(np.float16)
    gm = rng.lognormal(0, 0.3, C).astype(np.float16)
    bt = rng.normal(size=C).astype(np.float16)
    before, _ = _run(L, x, gm, bt, want_y=False)
    xd, gd, bd = torch.from_numpy(x).cuda(), torch.from_numpy(gm).cuda(), torch.from_numpy(bt).cuda()
    junk = torch.zeros((M + 1, L.row_bytes), dtype=torch.uint8, device="cuda")
    junk[M] = CANARY
    t0 = time.perf_counter()
    binding.selftest_ln_timeout(L, xd, gd, bd, EPS, junk, M=M)
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 5.0                       # it came back by itself
    assert binding.get_device_status() == binding.ERR_DEVICE_TIMEOUT
    assert binding.get_device_status() == 0                     # reading clears the word
    assert bool((junk[M] == CANARY).all())                      # even the drained launch stays inside its rows
    assert binding.status_string(binding.ERR_DEVICE_TIMEOUT) == "bounded wait inside a kernel ran out"
    after, _ = _run(L, x, gm, bt, want_y=False)
    assert np.array_equal(before, after)
