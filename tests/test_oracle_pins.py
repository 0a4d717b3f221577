"""Pins for the CPU oracle: every oracle function is checked against something that is not the
oracle -- values worked by hand from the paper's equations (tests/golden/), closed forms,
invariants, library routines on special cases, and brute force on tiny inputs."""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rng(seed):
    return np.random.default_rng(seed)


# ------------------------------------------------------------------ Eq. 2 (Min-Max parameters)
def _golden_rows(name):
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            line = line.strip()
            if line and not line.startswith("#"):
                yield line


def test_eq2_hand_worked_toy_ranges():
    n = 0
    for line in _golden_rows("eq2_toy_ranges.txt"):
        lo, hi, k, s, z_signed, z_unsigned = line.split()
        got_s, got_z = oracle.minmax_params(float(lo), float(hi), int(k))
        assert got_s == float(s)
        assert got_z == int(z_unsigned) == int(z_signed) + (1 << (int(k) - 1))
        n += 1
    assert n == 5


def test_eq2_maps_min_to_code_zero_and_max_clamps():
    r = _rng(1)
    for k in (3, 4, 8):
        for _ in range(50):
            lo = r.normal() * 10
            hi = lo + abs(r.normal()) * 5 + 1e-3
            s, z = oracle.minmax_params(lo, hi, k)
            y = np.array([[lo, hi]])
            q = oracle.quantize(y, [2], [s], [z], k)
            # min lands on 0 (or 1 when the half-to-even roundings of the two terms disagree)
            assert q[0, 0] <= 1
            assert q[0, 1] == (1 << k) - 1
            assert abs(s * (1 << k) - (hi - lo)) < 1e-12 * (hi - lo)


def test_eq2_degenerate_range_uses_unit_scale():
    s, z = oracle.minmax_params(3.0, 3.0, 4)
    assert s == 1.0 and z == 8 - 3


# ------------------------------------------------------------------ Eq. 1 per cluster
def _plain_quant(y, s, z, k):
    """Independent five-line statement of Eq. 1 with codes re-based to [0, 2^k-1]."""
    q = np.rint(y / s) + z
    return np.clip(q, 0, (1 << k) - 1).astype(np.uint8)


@pytest.mark.parametrize("k", [3, 4, 8])
def test_single_cluster_is_per_tensor_quantisation(k):
    r = _rng(10 + k)
    M, Cn = 7, 200
    y = r.normal(size=(M, Cn)) * 3
    s, z = 0.37, (1 << (k - 1)) + 1
    codes = oracle.quantize(y, [Cn], [s], [z], k)
    assert codes.shape == (M, 256)
    assert np.array_equal(codes[:, :Cn], _plain_quant(y, s, z, k))
    assert not codes[:, Cn:].any()


@pytest.mark.parametrize("k", [3, 4, 8])
def test_one_channel_per_cluster_is_per_channel_quantisation(k):
    r = _rng(20 + k)
    M, Cn = 5, 12
    y = r.normal(size=(M, Cn)) * 2
    s = r.uniform(0.05, 0.8, size=Cn)
    z = r.integers(0, 1 << k, size=Cn)
    codes = oracle.quantize(y, np.ones(Cn, np.int32), s, z, k)
    off, k_pad = oracle.segment_offsets(np.ones(Cn, np.int32))
    assert k_pad == 384 and np.array_equal(off[:-1], 32 * np.arange(Cn))
    for c in range(Cn):
        assert np.array_equal(codes[:, off[c]], _plain_quant(y[:, c], s[c], z[c], k))
    mask = np.ones(k_pad, bool)
    mask[off[:-1]] = False
    assert not codes[:, mask].any()


@pytest.mark.parametrize("k", [3, 4, 8])
def test_dequant_error_at_most_half_step_when_unclamped(k):
    r = _rng(30 + k)
    size = np.array([40, 0, 25, 63], np.int32)
    Cn = int(size.sum())
    s = np.array([0.5, 1.0, 0.02, 3.0])
    z = np.array([3, 1, 4, 2], np.int32)
    y = r.normal(size=(64, Cn)) * np.repeat(s, size) * (1 << k) * 0.4
    codes = oracle.quantize(y, size, s, z, k)
    assert codes.max() <= (1 << k) - 1
    x_hat = oracle.dequantize(codes, Cn, size, s, z)
    step = np.repeat(s, size)[None, :]
    pre = np.rint(y / step) + np.repeat(z, size)[None, :]
    unclamped = (pre >= 0) & (pre <= (1 << k) - 1)
    assert unclamped.mean() > 0.5
    assert np.all(np.abs(x_hat - y)[unclamped] <= step.repeat(64, 0)[unclamped] * 0.5 * (1 + 1e-12))
    # clamped elements saturate at the ends of the code range
    flat = codes[:, np.concatenate([np.arange(o, o + n) for o, n in
                                    zip(oracle.segment_offsets(size)[0][:-1], size)])]
    assert np.all((flat[~unclamped] == 0) | (flat[~unclamped] == (1 << k) - 1))


def test_quantiser_is_monotone_rounds_half_to_even_and_sends_nan_to_zero():
    y = np.linspace(-20, 20, 4001)[None, :]
    q = oracle.quantize(y, [y.shape[1]], [0.7], [8], 4)[0, :y.shape[1]]
    assert np.all(np.diff(q.astype(int)) >= 0) and q[0] == 0 and q[-1] == 15
    ties = np.array([[0.5, 1.5, 2.5, -0.5, -1.5]])
    assert oracle.quantize(ties, [5], [1.0], [4], 4)[0, :5].tolist() == [4, 6, 6, 4, 2]
    assert oracle.quantize(np.array([[np.nan, np.inf, -np.inf]]), [3], [1.0], [4], 4)[0, :3].tolist() == [0, 15, 0]


def test_fp32_decision_matches_fp64_decision_away_from_ties_and_its_own_definition():
    r = _rng(40)
    size = np.array([33, 31], np.int32)
    s32 = np.array([0.3, 1.7], np.float32)
    z = np.array([8, 3], np.int32)
    y32 = (r.normal(size=(50, 64)) * 4).astype(np.float32)
    got = oracle.quantize_f32(y32, size, s32, z, 4)
    inv = (1.0 / s32.astype(np.float64)).astype(np.float32)
    off, _ = oracle.segment_offsets(size)
    # exact product of the two fp32 numbers (fits fp64), rounded once to an integer
    t = y32.astype(np.float64) * np.repeat(inv, size)[None, :].astype(np.float64)
    want = np.clip(np.rint(t) + np.repeat(z, size)[None, :], 0, 15).astype(np.uint8)
    # a product that sits just below a tie: rounding it to fp32 first would lift it onto the tie
    # and change the code, the single rounding must not
    y_t = np.array([[np.float32(2.5) * (1 - 2.0 ** -24)]], np.float32)
    s_t = np.array([1.0], np.float32)
    assert oracle.quantize_f32(y_t, [1], s_t, [0], 4)[0, 0] == 2
    y_u = np.array([[np.float32(3.5)]], np.float32)
    assert oracle.quantize_f32(y_u, [1], s_t, [0], 4)[0, 0] == 4
    cols = np.concatenate([np.arange(off[0], off[0] + 33), np.arange(off[1], off[1] + 31)])
    assert np.array_equal(got[:, cols], want)
    q64 = oracle.quantize(y32.astype(np.float64), size, s32.astype(np.float64), z, 4)
    assert np.mean(q64 == got) > 0.999 and np.max(np.abs(q64.astype(int) - got.astype(int))) <= 1


def test_toy_ranges_two_clusters_beat_one_by_the_step_ratio():
    """Sec. 3.2's example channels: a shared quantiser over -100..100 has step 12.5, separate
    clusters have steps 3.125 and 1.25; uniform rounding error has variance step^2/12."""
    r = _rng(41)
    T = 20000
    y = np.stack([r.uniform(-100, -50, T), r.uniform(80, 100, T)], axis=1)
    k = 4
    s1, z1 = oracle.minmax_params(-100, 100, k)
    x1 = oracle.dequantize(oracle.quantize(y, [2], [s1], [z1], k), 2, [2], [s1], [z1])
    pa, pb = oracle.minmax_params(-100, -50, k), oracle.minmax_params(80, 100, k)
    s2, z2 = [pa[0], pb[0]], [pa[1], pb[1]]
    x2 = oracle.dequantize(oracle.quantize(y, [1, 1], s2, z2, k), 2, [1, 1], s2, z2)
    mse1 = ((x1 - y) ** 2).mean(0)
    mse2 = ((x2 - y) ** 2).mean(0)
    # Eq. 2 leaves the top step of each range clamped, which adds a little to the uniform model
    assert np.allclose(mse2, np.array([3.125, 1.25]) ** 2 / 12, rtol=0.25)
    assert mse1[0] / mse2[0] > 8 and mse1[1] / mse2[1] > 40


# ------------------------------------------------------------------ reorder index
def test_reorder_index_is_a_bijection_sorted_inside_clusters_and_ordered_by_range():
    r = _rng(50)
    Cn, g = 300, 6
    labels = r.integers(0, g - 1, size=Cn).astype(np.int32)      # label g-1 stays empty
    x_min = -r.uniform(0.1, 5, Cn) * (1 + labels)
    x_max = r.uniform(0.1, 5, Cn) * (1 + labels)
    perm, size, new_of_old = oracle.reorder_index(labels, x_min, x_max, g)
    assert np.array_equal(np.sort(perm), np.arange(Cn))
    assert size.sum() == Cn and size[-1] == 0 and new_of_old[g - 1] == g - 1
    pos, prev_range = 0, -1.0
    for c in range(g):
        seg = perm[pos:pos + size[c]]
        pos += size[c]
        if size[c] == 0:
            continue
        assert np.all(np.diff(seg) > 0)
        assert len(set(labels[seg])) == 1 and new_of_old[labels[seg[0]]] == c
        rng_c = x_max[seg].max() - x_min[seg].min()
        assert rng_c >= prev_range
        prev_range = rng_c


def test_identity_permutation_single_cluster_is_plain_layernorm_quant():
    r = _rng(51)
    M, Cn = 9, 128
    x = r.normal(size=(M, Cn)).astype(np.float16)
    gm = r.lognormal(0, 0.5, Cn).astype(np.float16)
    bt = r.normal(size=Cn).astype(np.float16)
    y = oracle.layernorm(x, gm, bt, 1e-5)
    y_r = oracle.reorder(y, np.arange(Cn, dtype=np.int32))
    assert np.array_equal(y, y_r)
    perm = r.permutation(Cn).astype(np.int32)
    assert np.array_equal(oracle.reorder(y, perm), y[:, perm])


# ------------------------------------------------------------------ LayerNorm
def test_layernorm_matches_library_routine_and_closed_forms():
    import torch
    r = _rng(60)
    M, Cn = 33, 768
    x = (r.normal(size=(M, Cn)) * r.lognormal(0, 0.3, (M, 1))).astype(np.float16)
    gm = r.lognormal(0, 0.75, Cn).astype(np.float16)
    bt = r.normal(size=Cn).astype(np.float16)
    y = oracle.layernorm(x, gm, bt, 1e-5)
    ref = torch.nn.functional.layer_norm(torch.from_numpy(x.astype(np.float64)), (Cn,),
                                         torch.from_numpy(gm.astype(np.float64)),
                                         torch.from_numpy(bt.astype(np.float64)), 1e-5).numpy()
    assert np.max(np.abs(y - ref)) < 1e-12 * max(1.0, np.abs(ref).max())
    ones, zeros = np.ones(Cn, np.float16), np.zeros(Cn, np.float16)
    y0 = oracle.layernorm(x, ones, zeros, 1e-5)
    assert np.max(np.abs(y0.mean(1))) < 1e-13
    var_x = x.astype(np.float64).var(1)
    assert np.allclose(y0.var(1), var_x / (var_x + 1e-5), rtol=1e-12)
    # a constant row normalises to beta exactly
    xc = np.full((1, Cn), 2.5, np.float16)
    assert np.array_equal(oracle.layernorm(xc, gm, bt, 1e-5)[0], bt.astype(np.float64))


# ------------------------------------------------------------------ packing
def test_pack_format_hand_examples():
    n = 0
    for line in _golden_rows("pack_format_examples.txt"):
        bits, codes, hexbytes = [p.strip() for p in line.split("|")]
        k = int(bits)
        codes = np.array(codes.split(), np.uint8)
        want = bytes.fromhex(hexbytes.replace(" ", ""))
        row = np.zeros((1, 128), np.uint8)
        row[0, :codes.size] = codes
        got = oracle.pack(row, k)
        assert got.shape == (1, 128 * k // 8)
        assert bytes(got[0, :len(want)]) == want
        assert not got[0, len(want):].any()
        n += 1
    assert n == 4


@pytest.mark.parametrize("k", [3, 4, 8])
def test_pack_unpack_round_trip_every_row_length(k):
    r = _rng(70 + k)
    for k_pad in (128, 256, 384, 896, 1280):
        codes = r.integers(0, 1 << k, size=(5, k_pad), dtype=np.uint8)
        packed = oracle.pack(codes, k)
        assert packed.shape == (5, k_pad * k // 8)
        assert np.array_equal(oracle.unpack(packed, k_pad, k), codes)
    # every packed bit is used: distinct code rows give distinct packed rows, and size is exact
    a = np.zeros((1, 128), np.uint8)
    seen = set()
    for p in range(128):
        for bit in range(k):
            a[:] = 0
            a[0, p] = 1 << bit
            packed = oracle.pack(a, k)
            assert packed.sum() in (1, 2, 4, 8, 16, 32, 64, 128)     # exactly one bit set
            seen.add(int(np.flatnonzero(np.unpackbits(packed[0], bitorder="little"))[0]))
    assert len(seen) == 128 * k


def test_weight_pack_round_trip_and_twos_complement_nibbles():
    r = _rng(75)
    w = r.integers(-8, 8, size=(6, 256), dtype=np.int8)
    packed = oracle.pack_weights(w)
    assert packed.shape == (128 * 128,)                       # 6 rows round up to one 128-row tile
    assert np.array_equal(oracle.unpack_weights(packed, 256, 6), w)
    one = np.zeros((1, 128), np.int8)
    one[0, 0], one[0, 4], one[0, 1] = -1, -8, 7
    p = oracle.pack_weights(one)
    assert p[0] == 0x8F and p[1] == 0x07
    # tile-major placement, worked by hand: row 129, position 130 of K_pad = 256 lies in tile
    # (1, 1) = tile number 1*2+1 = 3 (8192 bytes each), row 1 of the tile (64 bytes each), position 2
    # of the block = low nibble of byte 2
    big = np.zeros((130, 256), np.int8)
    big[129, 130] = -3
    pb = oracle.pack_weights(big)
    assert pb.shape == (2 * 128 * 128,) and pb[3 * 8192 + 64 + 2] == 0x0D and pb.sum() == 0x0D


# ------------------------------------------------------------------ weights
def test_weight_quantise_per_output_channel_symmetric_and_wsum_brute_force():
    r = _rng(80)
    N, Cn = 10, 96
    W = (r.normal(size=(N, Cn)) * 0.02).astype(np.float32)
    W[3] = 0
    size = np.array([20, 0, 50, 26], np.int32)
    perm = r.permutation(Cn).astype(np.int32)
    out_perm = np.full(16, -1, np.int32)                       # rows 2, 5, 9.. of the output are zero pads
    slots = np.sort(r.choice(16, size=N, replace=False))
    out_perm[slots] = r.permutation(N)
    w_codes, s_w, wsum = oracle.weight_quantize(W, perm, size, out_perm, n_pad=16)
    off, k_pad = oracle.segment_offsets(size)
    assert w_codes.shape == (16, k_pad) and wsum.shape == (4, 16)
    for rrow in slots:
        src = W[out_perm[rrow]]
        amax = np.abs(src).max()
        s = np.float32(amax) / np.float32(7) if amax > 0 else np.float32(1)
        assert s_w[rrow] == s
        q = np.clip(np.rint(src / s), -8, 7).astype(np.int8)
        assert np.abs(q).max() <= 7
        j = 0
        for c in range(4):
            seg = w_codes[rrow, off[c]:off[c] + 32 * ((size[c] + 31) // 32)]
            assert np.array_equal(seg[:size[c]], q[perm[j:j + size[c]]])
            assert not seg[size[c]:].any()
            assert wsum[c, rrow] == int(q[perm[j:j + size[c]]].astype(int).sum())
            j += size[c]
    pads = np.setdiff1d(np.arange(16), slots)
    assert not w_codes[pads].any() and np.all(s_w[pads] == 1) and not wsum[:, pads].any()
    assert np.all(s_w[list(out_perm).index(3)] == 1)
    # without an output index: identity rows, zero rows beyond N
    w2, s2, ws2 = oracle.weight_quantize(W, perm, size, None, n_pad=16)
    assert np.array_equal(w2[out_perm[slots]], w_codes[slots]) and not w2[N:].any() and np.all(s2[N:] == 1)


# ------------------------------------------------------------------ cluster-segmented integer GEMM
def _tiny_case(seed, M=5, N=7, size=(33, 0, 4, 70), k=4):
    r = _rng(seed)
    size = np.array(size, np.int32)
    g = size.size
    off, k_pad = oracle.segment_offsets(size)
    a = np.zeros((M, k_pad), np.uint8)
    w = np.zeros((N, k_pad), np.int8)
    for c in range(g):
        a[:, off[c]:off[c] + size[c]] = r.integers(0, 1 << k, size=(M, size[c]))
        w[:, off[c]:off[c] + size[c]] = r.integers(-7, 8, size=(N, size[c]))
        # activation pads may hold anything the kernel wrote (code 0); make them non-zero here to
        # show that zero weight pads alone keep them out of the result
        a[:, off[c] + size[c]:off[c + 1]] = 1
    scale = r.uniform(0.05, 2.0, g)
    zero = r.integers(0, 1 << k, g).astype(np.int32)
    s_w = r.uniform(0.001, 0.01, N).astype(np.float32)
    wsum = np.stack([w[:, off[c]:off[c] + size[c]].astype(np.int64).sum(1) for c in range(g)]).astype(np.int32)
    return a, w, size, off, scale, zero, s_w, wsum


def test_cluster_acc_brute_force_triple_loop():
    a, w, size, off, *_ = _tiny_case(90)
    acc = oracle.cluster_acc(a, w, size)
    for c in range(size.size):
        for m in range(a.shape[0]):
            for n in range(w.shape[0]):
                s = 0
                for p in range(off[c], off[c] + size[c]):
                    s += int(a[m, p]) * int(w[n, p])
                assert acc[c, m, n] == s


def test_integer_method_equals_dequantise_then_matmul():
    """Appendix: the two computation methods are the same function of the codes."""
    for seed, k in ((91, 4), (92, 3), (93, 8)):
        a, w, size, off, scale, zero, s_w, wsum = _tiny_case(seed, k=k)
        y2 = oracle.cluster_gemm(a, w, size, scale, zero, s_w, wsum)
        y1 = oracle.dequant_matmul(a, w, size, scale, zero, s_w)
        assert np.max(np.abs(y1 - y2)) <= 1e-12 * np.abs(y1).max()
        # and equal to the same thing spelled with library matmuls on de-quantised arrays
        cols = np.concatenate([np.arange(off[c], off[c] + size[c]) for c in range(size.size)])
        x_hat = (a[:, cols].astype(np.float64) - np.repeat(zero, size)) * np.repeat(scale, size)
        w_hat = w[:, cols].astype(np.float64) * s_w.astype(np.float64)[:, None]
        assert np.max(np.abs(x_hat @ w_hat.T - y2)) <= 1e-12 * np.abs(y2).max()


def test_unit_scale_zero_offset_reduces_to_integer_matmul_and_epilogue_options():
    a, w, size, off, scale, zero, s_w, wsum = _tiny_case(94)
    g = size.size
    ones = np.ones(w.shape[0], np.float32)
    y = oracle.cluster_gemm(a, w, size, np.ones(g), np.zeros(g, np.int32), ones, wsum)
    cols = np.concatenate([np.arange(off[c], off[c] + size[c]) for c in range(g)])
    assert np.array_equal(y, (a[:, cols].astype(np.int64) @ w[:, cols].astype(np.int64).T).astype(np.float64))
    bias = np.linspace(-1, 1, w.shape[0]).astype(np.float32)
    base = oracle.cluster_gemm(a, w, size, scale, zero, s_w, wsum)
    yb = oracle.cluster_gemm(a, w, size, scale, zero, s_w, wsum, bias=bias, relu=True)
    assert np.allclose(yb, np.maximum(base + bias.astype(np.float64), 0), rtol=0, atol=1e-15)


# ------------------------------------------------------------------ K-Means (invariants only)
def test_kmeans_partitions_never_increases_inertia_and_recovers_separated_blobs():
    r = _rng(100)
    centres = np.array([[-10, -8], [0, 1], [5, 9], [20, 30.0]])
    pts = np.concatenate([c + r.normal(size=(60, 2)) * 0.3 for c in centres])
    truth = np.repeat(np.arange(4), 60)
    u = np.array([0.1, 0.4, 0.7, 0.95])
    labels, cent, inertia = oracle.kmeans(pts, 4, u, iters=20)
    assert labels.min() >= 0 and labels.max() < 4
    assert np.all(np.diff(inertia) <= 1e-9 * inertia[0])
    for b in range(4):
        assert len(set(labels[truth == b])) == 1
    assert len(set(labels)) == 4
    # Lloyd's fixed point from the same seeds, by a library routine
    from sklearn.cluster import KMeans
    km = KMeans(n_clusters=4, init=cent, n_init=1, max_iter=1, algorithm="lloyd").fit(pts)
    assert np.isclose(km.inertia_, inertia[-1], rtol=1e-9)
    # more centres than distinct points: labels stay a valid partition
    few = np.repeat(np.array([[0.0, 1.0], [5.0, 6.0]]), 3, axis=0)
    lab2, _, _ = oracle.kmeans(few, 4, np.array([0.0, 0.9, 0.5, 0.5]), iters=5)
    assert not (set(lab2[:3]) & set(lab2[3:]))
    assert lab2.min() >= 0 and lab2.max() < 4


def test_calibration_pipeline_composes_the_pinned_pieces():
    r = _rng(101)
    Cn, g, k = 256, 4, 4
    x = r.normal(size=(64, Cn)).astype(np.float16)
    gm = r.lognormal(0, 0.75, Cn).astype(np.float16)
    bt = (r.normal(size=Cn) * 0.5 * gm).astype(np.float16)
    cal = oracle.calibrate(x, gm, bt, g, k, r.random(g))
    assert np.array_equal(np.sort(cal.perm), np.arange(Cn)) and cal.size.sum() == Cn
    y = oracle.layernorm(x, gm, bt, 1e-5)
    assert np.array_equal(cal.x_min, y.min(0)) and np.array_equal(cal.x_max, y.max(0))
    pos = 0
    for c in range(g):
        seg = cal.perm[pos:pos + cal.size[c]]
        pos += cal.size[c]
        if cal.size[c]:
            s, z = oracle.minmax_params(y[:, seg].min(), y[:, seg].max(), k)
            assert (s, z) == (cal.scale[c], cal.zero[c])
    # calibration tokens themselves quantise without leaving the code range by more than the
    # one clamped top step that Eq. 2 implies
    codes = oracle.quantize(oracle.reorder(y, cal.perm), cal.size, cal.scale, cal.zero, k)
    assert codes.max() == 15 and codes.min() == 0


# ------------------------------------------------------------------ per-cluster asymmetric weights (Appendix)
def test_asymmetric_hand_worked_examples():
    n = 0
    for line in _golden_rows("asym_toy.txt"):
        kind, fields, want = [p.strip() for p in line.split("|")]
        if kind == "gemm":
            f = [float(v) for v in fields.split()]
            yq0, yq1, y = [float(v) for v in want.split()]
            size = np.array([2, 2], np.int32)
            a = np.zeros((1, 128), np.uint8); w = np.zeros((1, 128), np.uint8)
            a[0, 0:2] = f[2:4]; a[0, 32:34] = f[10:12]
            w[0, 0:2] = f[6:8]; w[0, 32:34] = f[14:16]
            scale = np.array([f[0], f[8]]); zero = np.array([f[1], f[9]], np.int32)
            s_w = np.array([[f[4]], [f[12]]], np.float32); z_w = np.array([[f[5]], [f[13]]], np.int32)
            assert oracle.cluster_gemm_asym(a, w, size, scale, zero, s_w, z_w)[0, 0] == y
            assert oracle.dequant_matmul_asym(a, w, size, scale, zero, s_w, z_w)[0, 0] == y
            # the per-cluster integers, through unit scales on one cluster at a time
            for c, yq in ((0, yq0), (1, yq1)):
                sc = np.zeros(2); sc[c] = 1.0
                assert oracle.cluster_gemm_asym(a, w, size, sc, zero, np.ones((2, 1), np.float32), z_w)[0, 0] == yq
        else:
            f = fields.split()
            k, ws = int(f[0]), np.array([float(v) for v in f[1:]], np.float32)
            wv = want.split()
            W = np.zeros((1, 8), np.float32); W[0, :3] = ws
            # the three weights are one cluster, the other five channels another one
            codes, s_w, z_w, wsum = oracle.weight_quantize_clustered(W, np.arange(8), np.array([3, 5], np.int32), k)
            assert s_w[0, 0] == np.float32(float(wv[0])) and z_w[0, 0] == int(wv[1])
            assert codes[0, :3].tolist() == [int(v) for v in wv[2:]] and wsum[0, 0] == sum(int(v) for v in wv[2:])
            # the other cluster is all zeros: max == min, so s = 1, z = 2^(k-1) and every code equals z
            assert s_w[1, 0] == 1.0 and z_w[1, 0] == 1 << (k - 1) and np.all(codes[0, 32:37] == 1 << (k - 1))
        n += 1
    assert n == 3


def _asym_case(seed, M=5, N=7, C=96, g=4, k=4, bits=4):
    r = _rng(seed)
    perm = r.permutation(C).astype(np.int32)
    cuts = np.sort(r.integers(0, C + 1, size=g - 1))
    size = np.diff(np.concatenate([[0], cuts, [C]])).astype(np.int32)
    W = (r.normal(size=(N, C)) * r.lognormal(0, 1, size=C)).astype(np.float32)
    codes_w, s_w, z_w, wsum = oracle.weight_quantize_clustered(W, perm, size, k)
    off, k_pad = oracle.segment_offsets(size)
    a = np.zeros((M, k_pad), np.uint8)
    for c in range(g):
        a[:, off[c]:off[c] + size[c]] = r.integers(0, 1 << bits, size=(M, size[c]))
    scale = r.uniform(0.05, 1.5, g)
    zero = r.integers(-3, 1 << bits, g).astype(np.int32)
    return dict(perm=perm, size=size, W=W, w=codes_w, s_w=s_w, z_w=z_w, wsum=wsum, a=a, scale=scale, zero=zero, off=off, k_pad=k_pad, k=k)


def test_clustered_weight_quantiser_against_a_plain_restatement():
    for seed, k in ((1, 4), (2, 3), (3, 8)):
        c = _asym_case(seed, k=k)
        qmax = (1 << k) - 1
        j = 0
        for ci, n_c in enumerate(c["size"]):
            ch = c["perm"][j:j + n_c]; j += n_c
            if n_c == 0:
                assert np.all(c["s_w"][ci] == 1) and not c["z_w"][ci].any() and not c["wsum"][ci].any()
                continue
            for n in range(c["W"].shape[0]):
                w = c["W"][n, ch]
                s = np.float32(w.max() - w.min()) / np.float32(1 << k)
                s = s if s > 0 else np.float32(1)
                z = (1 << (k - 1)) - int(np.rint(np.float32(w.max() + w.min()) / (np.float32(2) * s)))
                q = np.clip(np.rint(w / s) + z, 0, qmax).astype(np.uint8)
                got = c["w"][n, c["off"][ci]:c["off"][ci] + n_c]
                assert c["s_w"][ci, n] == s and c["z_w"][ci, n] == z
                assert np.array_equal(got, q) and c["wsum"][ci, n] == int(q.sum())
                # Eq. 2's consequences: the minimum maps to code 0; inside the range the error is at most half a step
                assert got[np.argmin(w)] == 0
                err = np.abs(s * (got.astype(np.float64) - z) - w)
                inside = np.rint(w / s) + z <= qmax
                assert np.all(err[inside] <= 0.5 * s * (1 + 1e-5))
        assert not c["w"][:, np.setdiff1d(np.arange(c["k_pad"]), np.concatenate([np.arange(o, o + n) for o, n in zip(c["off"], c["size"])]))].any()


def test_asymmetric_integer_method_equals_dequantise_then_matmul():
    for seed in (11, 12, 13):
        c = _asym_case(seed, M=6, N=9, C=160, g=5)
        y2 = oracle.cluster_gemm_asym(c["a"], c["w"], c["size"], c["scale"], c["zero"], c["s_w"], c["z_w"])
        y1 = oracle.dequant_matmul_asym(c["a"], c["w"], c["size"], c["scale"], c["zero"], c["s_w"], c["z_w"])
        assert np.max(np.abs(y1 - y2)) <= 1e-12 * np.abs(y1).max()
        # and a library matmul on the de-quantised operands (contiguous real positions)
        xh = np.zeros(c["a"].shape); wh = np.zeros(c["w"].shape)
        for ci, (o, n_c) in enumerate(zip(c["off"], c["size"])):
            xh[:, o:o + n_c] = c["scale"][ci] * (c["a"][:, o:o + n_c].astype(np.float64) - c["zero"][ci])
            wh[:, o:o + n_c] = c["s_w"][ci][:, None].astype(np.float64) * (c["w"][:, o:o + n_c].astype(np.float64) - c["z_w"][ci][:, None])
        assert np.max(np.abs(xh @ wh.T - y2)) <= 1e-12 * np.abs(y2).max()
        # bias and ReLU
        b = _rng(seed).normal(size=9).astype(np.float32)
        yb = oracle.cluster_gemm_asym(c["a"], c["w"], c["size"], c["scale"], c["zero"], c["s_w"], c["z_w"], bias=b, relu=True)
        assert np.allclose(yb, np.maximum(y2 + b, 0), rtol=0, atol=1e-12 * np.abs(y2).max())


def test_asymmetric_method_reduces_to_the_symmetric_one():
    """z^W = const and s^W_i the same for every cluster: the four-term expression must give what the
    symmetric path gives on the same integers (codes shifted by 8)."""
    r = _rng(21)
    C, N, M, g = 128, 6, 4, 3
    perm = r.permutation(C).astype(np.int32)
    size = np.array([50, 0, 78], np.int32)
    W = (r.normal(size=(N, C)) * 0.02).astype(np.float32)
    w_sym, s_w, wsum = oracle.weight_quantize(W, perm, size)
    off, k_pad = oracle.segment_offsets(size)
    a = np.zeros((M, k_pad), np.uint8)
    for c in range(g):
        a[:, off[c]:off[c] + size[c]] = r.integers(0, 16, size=(M, size[c]))
    scale = r.uniform(0.1, 1, g); zero = r.integers(0, 16, g).astype(np.int32)
    want = oracle.cluster_gemm(a, w_sym, size, scale, zero, s_w, wsum)
    w_u = (w_sym.astype(np.int16) + 8).astype(np.uint8)
    got = oracle.cluster_gemm_asym(a, w_u, size, scale, zero, np.tile(s_w, (g, 1)), np.full((g, N), 8, np.int32))
    assert np.max(np.abs(got - want)) <= 1e-12 * np.abs(want).max()


def test_code_rowsums_brute_force():
    c = _asym_case(31, M=9, C=200, g=6)
    got = oracle.code_rowsums(c["a"], c["size"])
    for m in range(9):
        for ci, (o, n_c) in enumerate(zip(c["off"], c["size"])):
            assert got[m, ci] == sum(int(v) for v in c["a"][m, o:o + n_c])


# ------------------------------------------------------------------ first method with bfloat16 operands
def _bf16_round(v32):
    """An independent statement of round-to-nearest-even to bfloat16: the nearer of the two
    neighbouring 8-bit-significand values, the even one on a tie (by exact comparison in fp64)."""
    u = np.asarray(v32, np.float32).view(np.uint32)
    lo = (u & 0xFFFF0000).view(np.float32).astype(np.float64)             # truncation toward zero
    hi = ((u & 0xFFFF0000) + np.uint32(0x10000)).view(np.float32).astype(np.float64)
    x = np.asarray(v32, np.float64)
    dl, dh = np.abs(x - lo), np.abs(hi - x)
    even_lo = ((u >> 16) & 1) == 0
    return np.where((dl < dh) | ((dl == dh) & even_lo), lo, hi)


def test_bf16_first_method_against_numpy_and_within_its_rounding_bound():
    r = _rng(41)
    C, N, M, g = 160, 9, 7, 4
    perm = r.permutation(C).astype(np.int32)
    size = np.array([50, 3, 0, 107], np.int32)
    W = (r.normal(size=(N, C)) * 0.02).astype(np.float32)
    w, s_w, wsum = oracle.weight_quantize(W, perm, size)
    off, k_pad = oracle.segment_offsets(size)
    a = np.zeros((M, k_pad), np.uint8)
    for c in range(g):
        a[:, off[c]:off[c] + size[c]] = r.integers(0, 16, size=(M, size[c]))
    scale = r.uniform(0.01, 2.0, g).astype(np.float32)
    zero = r.integers(0, 16, g).astype(np.int32)
    got = oracle.dequant_matmul_bf16(a, w, size, scale, zero, s_w)
    xh = np.zeros((M, k_pad))
    for c, (o, n_c) in enumerate(zip(off, size)):
        xh[:, o:o + n_c] = _bf16_round(scale[c] * (a[:, o:o + n_c].astype(np.int32) - zero[c]).astype(np.float32))
    want = (xh @ w.astype(np.float64).T) * s_w.astype(np.float64)
    assert np.max(np.abs(got - want)) <= 1e-13 * np.abs(want).max()
    # against the exact first method: every operand is off by at most 2^-9 of its magnitude
    exact = oracle.dequant_matmul(a, w, size, scale.astype(np.float64), zero, s_w)
    xe = np.zeros((M, k_pad))
    for c, (o, n_c) in enumerate(zip(off, size)):
        xe[:, o:o + n_c] = float(scale[c]) * (a[:, o:o + n_c].astype(np.float64) - zero[c])
    bound = 2.0 ** -8 * (np.abs(xe) @ np.abs(w.astype(np.float64)).T) * s_w.astype(np.float64) + 1e-12
    assert np.all(np.abs(got - exact) <= bound)
    assert np.max(np.abs(got - exact)) > 0          # and the rounding is really there


# ------------------------------------------------------------------ attention sites (Sec. 4.2, 5.1)
def _toy_attention(causal):
    q = np.zeros((2, 128), np.uint8); k = np.zeros((2, 128), np.uint8); v = np.zeros((2, 128), np.uint8)
    q[0, 0:2] = (4, 2); q[0, 32] = 1; q[1, 0:2] = (6, 0); q[1, 32] = 1
    k[0, 0:2] = (2, 3); k[0, 32] = 5; k[1, 0:2] = (3, 1); k[1, 32] = 3
    v[0, 0] = 8; v[0, 32:34] = (3, 0); v[1, 0] = 0; v[1, 32:34] = (1, 2)
    return oracle.attention(q, k, v, 1, 2, [2, 1], [0.5, 2.0], [2, 0], [1.0, 0.5], [1, 3], [1, 2], [0.25, 2.0], [4, 1],
                            1.0 / 256, 0, np.log(3.0) / 2, causal, return_p=True)


def test_attention_hand_worked_example():
    n = 0
    for line in _golden_rows("attention_toy.txt"):
        kind, pq_want, o_want = [p.strip() for p in line.split("|")]
        if kind.startswith("kv_"):
            continue
        o, pq = _toy_attention(kind == "causal")
        assert pq.reshape(-1).tolist() == [int(t) for t in pq_want.split()]
        got = np.concatenate([o[:, 0:1], o[:, 32:34]], axis=1).reshape(-1)
        assert np.allclose(got, [float(t) for t in o_want.split()], rtol=0, atol=1e-15)
        assert not o[:, 1:32].any() and not o[:, 34:].any()         # pad positions stay 0
        # the last step alone, from the fixture's codes
        v = np.zeros((2, 128), np.uint8); v[0, 0] = 8; v[0, 32:34] = (3, 0); v[1, 32:34] = (1, 2)
        o2 = oracle.attention_output(np.array([int(t) for t in pq_want.split()], np.uint8).reshape(1, 2, 2), v, 1, 2,
                                     [1, 2], [0.25, 2.0], [4, 1], 1.0 / 256, 0)
        assert np.allclose(np.concatenate([o2[:, 0:1], o2[:, 32:34]], axis=1).reshape(-1), [float(t) for t in o_want.split()], rtol=0, atol=1e-15)
        n += 1
    assert n == 2


def _attention_case(seed, Tq=5, Tk=9, H=2, gh=3, hd=24, bits=4):
    r = _rng(seed)
    def sizes():
        out = []
        for _ in range(H):
            cuts = np.sort(r.integers(0, hd + 1, size=gh - 1))
            out.append(np.diff(np.concatenate([[0], cuts, [hd]])))
        return np.concatenate(out).astype(np.int32)
    size_qk, size_v = sizes(), sizes()
    g = H * gh
    par = lambda: (r.uniform(0.05, 0.3, size=g), r.integers(0, 1 << bits, size=g).astype(np.int32))
    (sQ, zQ), (sK, zK), (sV, zV) = par(), par(), par()
    def codes(T, size):
        off, k_pad = oracle.segment_offsets(size)
        a = np.zeros((T, k_pad), np.uint8)
        for c in range(g):
            a[:, off[c]:off[c] + size[c]] = r.integers(0, 1 << bits, size=(T, size[c]))
        return a, off
    (q, off_qk), (k, _), (v, off_v) = codes(Tq, size_qk), codes(Tk, size_qk), codes(Tk, size_v)
    return dict(q=q, k=k, v=v, H=H, gh=gh, size_qk=size_qk, sQ=sQ, zQ=zQ, sK=sK, zK=zK, size_v=size_v, sV=sV, zV=zV,
                off_qk=off_qk, off_v=off_v, hd=hd)


def _dequant_by_hand(codes, off, size, s, z):
    """Eq. 1 on the real positions of every cluster; other positions 0."""
    out = np.zeros(codes.shape)
    for c in range(len(size)):
        sl = slice(off[c], off[c] + size[c])
        out[:, sl] = s[c] * (codes[:, sl].astype(np.float64) - z[c])
    return out


@pytest.mark.parametrize("causal", [False, True])
def test_attention_is_within_the_softmax_quantisers_bound_of_plain_attention(causal):
    """With the 8-bit softmax output replaced by the exact probabilities the computation is ordinary
    attention on the de-quantised tensors (scipy's softmax); the quantiser moves a probability by at most
    s_P / 2 (plus the clamp of 256 to 255), so |O - O_exact| <= (s_P / 2 + s_P [P = 1]) sum_j |V^|."""
    from scipy.special import softmax
    for seed in (1, 2, 3):
        c = _attention_case(seed)
        Tq, Tk, H, gh = c["q"].shape[0], c["k"].shape[0], c["H"], c["gh"]
        scale = 1.0 / np.sqrt(c["hd"])
        o, pq = oracle.attention(c["q"], c["k"], c["v"], H, gh, c["size_qk"], c["sQ"], c["zQ"], c["sK"], c["zK"],
                                 c["size_v"], c["sV"], c["zV"], 1.0 / 256, 0, scale, causal, return_p=True)
        Qh = _dequant_by_hand(c["q"], c["off_qk"], c["size_qk"], c["sQ"], c["zQ"])
        Kh = _dequant_by_hand(c["k"], c["off_qk"], c["size_qk"], c["sK"], c["zK"])
        Vh = _dequant_by_hand(c["v"], c["off_v"], c["size_v"], c["sV"], c["zV"])
        for h in range(H):
            lo, hi = c["off_qk"][h * gh], c["off_qk"][(h + 1) * gh]
            A = scale * Qh[:, lo:hi] @ Kh[:, lo:hi].T
            if causal:
                A = np.where(np.arange(Tk)[None, :] <= np.arange(Tq)[:, None] + (Tk - Tq), A, -np.inf)
            P = softmax(A, axis=1)
            vlo, vhi = c["off_v"][h * gh], c["off_v"][(h + 1) * gh]
            exact = P @ Vh[:, vlo:vhi]
            bound = (1.5 / 256) * np.abs(Vh[:, vlo:vhi]).sum(axis=0)[None, :] + 1e-12
            assert np.all(np.abs(o[:, vlo:vhi] - exact) <= bound)
            assert np.abs(o[:, vlo:vhi] - exact).max() > 0                      # and the quantiser is really there
            assert np.all(np.abs(pq[h].astype(np.float64) - np.minimum(np.rint(P * 256), 255)) <= 1)
            if causal:
                assert not pq[h][np.arange(Tk)[None, :] > np.arange(Tq)[:, None] + (Tk - Tq)].any()


def test_attention_closed_forms():
    c = _attention_case(7, Tq=4, Tk=6)
    H, gh = c["H"], c["gh"]
    Vh = _dequant_by_hand(c["v"], c["off_v"], c["size_v"], c["sV"], c["zV"])
    args = lambda k, s: (c["q"], k, c["v"], H, gh, c["size_qk"], c["sQ"], c["zQ"], c["sK"], c["zK"], c["size_v"], c["sV"], c["zV"],
                         1.0 / 256, 0, s, False)
    # equal keys: every probability is 1/6 -> code round(256 / 6) = 43, O = 43/256 sum_j V^
    k_same = np.repeat(c["k"][:1], 6, axis=0)
    o, pq = oracle.attention(*args(k_same, 0.3), return_p=True)
    assert np.all(pq == 43)
    assert np.allclose(o, np.broadcast_to((43.0 / 256) * Vh.sum(axis=0), o.shape), rtol=0, atol=1e-12)
    # a score scale of 0 does the same whatever the keys are
    assert np.array_equal(oracle.attention(*args(c["k"], 0.0)), o)
    # a zero point of the softmax codes cancels in s_P (Pq - z_P) as long as nothing clamps
    a = list(args(k_same, 0.3)); a[14] = 100
    assert np.allclose(oracle.attention(*a), o, rtol=0, atol=1e-12)
    # a huge score scale picks, per query and head, the key with the largest product: P = 1 -> 255/256 V^[j*]
    o, pq = oracle.attention(*args(c["k"], 1e4), return_p=True)
    Qh = _dequant_by_hand(c["q"], c["off_qk"], c["size_qk"], c["sQ"], c["zQ"])
    Kh = _dequant_by_hand(c["k"], c["off_qk"], c["size_qk"], c["sK"], c["zK"])
    for h in range(H):
        lo, hi = c["off_qk"][h * gh], c["off_qk"][(h + 1) * gh]
        best = np.argmax(Qh[:, lo:hi] @ Kh[:, lo:hi].T, axis=1)
        vlo, vhi = c["off_v"][h * gh], c["off_v"][(h + 1) * gh]
        assert np.allclose(o[:, vlo:vhi], (255.0 / 256) * Vh[best, vlo:vhi], rtol=0, atol=1e-12)
        assert np.all(pq[h][np.arange(4), best] == 255) and pq[h].sum() == 4 * 255


def _toy_kv_inputs():
    k = np.zeros((2, 128), np.uint8); v = np.zeros((2, 128), np.uint8)
    k[0, 0:2] = (2, 3); k[0, 32] = 5; k[1, 0:2] = (3, 1); k[1, 32] = 3
    v[0, 0] = 8; v[0, 32:34] = (3, 0); v[1, 0] = 0; v[1, 32:34] = (1, 2)
    ch = np.full(128, -1, np.int32); ch[0:2] = (2, 0); ch[32] = 1            # K's positions hold channels 2, 0 | 1
    q = np.zeros((2, 3)); q[0, [2, 0, 1]] = (1, 0, 2); q[1, [2, 0, 1]] = (2, -1, 2)
    return q, ch, k, v


def test_kv_only_attention_hand_worked_example():
    n = 0
    for line in _golden_rows("attention_toy.txt"):
        kind, _, o_want = [p.strip() for p in line.split("|")]
        if not kind.startswith("kv_"):
            continue
        q, ch, k, v = _toy_kv_inputs()
        o = oracle.attention_kv(q, ch, k, v, 1, 2, [2, 1], [1.0, 0.5], [1, 3], [1, 2], [0.25, 2.0], [4, 1], np.log(3.0) / 2, kind == "kv_causal")
        got = np.concatenate([o[:, 0:1], o[:, 32:34]], axis=1).reshape(-1)
        assert np.allclose(got, [float(t) for t in o_want.split()], rtol=0, atol=1e-14)
        assert not o[:, 1:32].any() and not o[:, 34:].any()
        n += 1
    assert n == 2


@pytest.mark.parametrize("causal", [False, True])
def test_kv_only_attention_is_plain_attention_on_the_dequantised_cache(causal):
    """The definition itself, through library routines: scipy softmax and numpy matmul on K^, V^ de-quantised by hand,
    with the query's channels scattered over K's positions."""
    from scipy.special import softmax
    for seed in (4, 5):
        c = _attention_case(seed)
        r = _rng(100 + seed)
        Tq, Tk, H, gh, hd = c["q"].shape[0], c["k"].shape[0], c["H"], c["gh"], c["hd"]
        Cn = H * hd
        k_pad = c["k"].shape[1]
        ch = np.full(k_pad, -1, np.int32)                       # a random per-head assignment of channels to K's real positions
        for h in range(H):
            pos = np.concatenate([np.arange(c["off_qk"][cc], c["off_qk"][cc] + c["size_qk"][cc]) for cc in range(h * gh, (h + 1) * gh)])
            ch[pos] = h * hd + r.permutation(hd)
        q = r.normal(size=(Tq, Cn))
        scale = 1.0 / np.sqrt(hd)
        o = oracle.attention_kv(q, ch, c["k"], c["v"], H, gh, c["size_qk"], c["sK"], c["zK"], c["size_v"], c["sV"], c["zV"], scale, causal)
        Kh = _dequant_by_hand(c["k"], c["off_qk"], c["size_qk"], c["sK"], c["zK"])
        Vh = _dequant_by_hand(c["v"], c["off_v"], c["size_v"], c["sV"], c["zV"])
        for h in range(H):
            lo, hi = c["off_qk"][h * gh], c["off_qk"][(h + 1) * gh]
            real = ch[lo:hi] >= 0
            A = scale * q[:, ch[lo:hi][real]] @ Kh[:, lo:hi][:, real].T
            if causal:
                A = np.where(np.arange(Tk)[None, :] <= np.arange(Tq)[:, None] + (Tk - Tq), A, -np.inf)
            vlo, vhi = c["off_v"][h * gh], c["off_v"][(h + 1) * gh]
            assert np.allclose(o[:, vlo:vhi], softmax(A, axis=1) @ Vh[:, vlo:vhi], rtol=1e-12, atol=1e-12)
