"""CPU-side checks of the library boundary and of the host-side product code: the shared library
loads and exports every declared symbol, argument validation, the packed-format helpers and the
offline weight preparation against the oracle, and the numpy calibration against the oracle's."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
from paper_2304_01089_b200 import build as lib_build
from paper_2304_01089_b200 import calibration, workloads
from helpers import random_layout_params

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    lib_build.build()
    from paper_2304_01089_b200 import binding as b
    return b


def test_library_exports_every_declared_symbol(binding):
    header = open(os.path.join(ROOT, "include", "rptq.h")).read()
    declared = set(re.findall(r"\b(rptq_[a-z0-9_]+)\s*\(", header))
    declared -= {"rptq_layout_t"}
    assert declared == set(binding.EXPORTS)
    lib = ctypes.CDLL(binding.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name
    assert binding.format_version() == 2
    assert binding.status_string(-3) == "reorder index is not a bijection"


def test_layout_validation_and_padded_offsets(binding):
    rng = np.random.default_rng(0)
    C, g, bits = 256, 6, 4
    perm, size, scale, zero = random_layout_params(rng, C, g, bits)
    L = binding.Layout(perm, size, scale, zero, bits)
    off, k_pad = oracle.segment_offsets(size)
    assert L.K_pad == k_pad and L.row_bytes == k_pad // 2
    want_uc = np.full(k_pad // 32, -1, np.int32)
    for c in range(g):
        want_uc[off[c] // 32:off[c + 1] // 32] = c
    assert np.array_equal(L.unit_cluster, want_uc)
    # within a cluster the library places the channels as it likes; contiguous_position() maps back
    m = L.contiguous_position()
    assert sorted(m.tolist()) == list(range(k_pad))
    for c in range(g):
        assert np.all((m[off[c]:off[c + 1]] >= off[c]) & (m[off[c]:off[c + 1]] < off[c + 1]))
    off2, k_pad2 = calibration.segment_offsets(size)
    assert k_pad2 == k_pad and np.array_equal(off2, off)
    bad = perm.copy(); bad[3] = bad[4]
    with pytest.raises(binding.RptqError) as e:
        binding.Layout(bad, size, scale, zero, bits)
    assert e.value.status == binding.ERR_NOT_BIJECTION
    short = size.copy(); short[0] += 1
    with pytest.raises(binding.RptqError) as e:
        binding.Layout(perm, short, scale, zero, bits)
    assert e.value.status == binding.ERR_NOT_BIJECTION
    with pytest.raises(binding.RptqError) as e:
        binding.Layout(perm, size, scale, zero, 5)
    assert e.value.status == binding.ERR_UNSUPPORTED
    neg = scale.copy(); neg[1] = 0.0
    with pytest.raises(binding.RptqError) as e:
        binding.Layout(perm, size, neg, zero, bits)
    assert e.value.status == binding.ERR_INVALID_ARG
    with pytest.raises(binding.RptqError) as e:
        binding.Layout(np.arange(12, dtype=np.int32), [12], [1.0], [0], 4)
    assert e.value.status == binding.ERR_UNSUPPORTED      # C not a multiple of 8


@pytest.mark.parametrize("bits", [3, 4, 8])
def test_packed_format_helpers_agree_with_the_oracle(binding, bits):
    rng = np.random.default_rng(bits)
    for k_pad in (128, 640, 1152):
        codes = rng.integers(0, 1 << bits, size=(7, k_pad), dtype=np.uint8)
        packed = binding.codes_pack_host(codes, bits)
        assert np.array_equal(packed, oracle.pack(codes, bits))
        assert np.array_equal(binding.codes_unpack_host(packed, k_pad, bits), codes)
    w = rng.integers(-8, 8, size=(5, 256), dtype=np.int8)
    assert np.array_equal(binding.weight_unpack_host(oracle.pack_weights(w), 256, 5), w)
    assert binding.weight_codes_bytes(256, 5) == 128 * 128 == oracle.weight_codes_bytes(5, 256)


def test_weight_pack_matches_the_oracle_bit_for_bit(binding):
    rng = np.random.default_rng(5)
    C, g, N, n_pad = 320, 7, 50, 64
    perm, size, scale, zero = random_layout_params(rng, C, g, 4)
    L = binding.Layout(perm, size, scale, zero, 4)
    W = (rng.normal(size=(N, C)) * 0.02).astype(np.float32)
    W[11] = 0
    out_perm = np.full(n_pad, -1, np.int32)
    out_perm[np.sort(rng.choice(n_pad, size=N, replace=False))] = rng.permutation(N)
    for op in (None, out_perm):
        packed, s_w, wsum = binding.weight_pack(L, W, op, n_pad)
        w_codes, s_w_o, wsum_o = oracle.weight_quantize(W, perm, size, op, n_pad)
        assert np.array_equal(packed, oracle.pack_weights(np.ascontiguousarray(w_codes[:, L.contiguous_position()])))
        assert np.array_equal(s_w, s_w_o) and np.array_equal(wsum, wsum_o)
    with pytest.raises(binding.RptqError):
        binding.weight_pack(L, W, np.zeros(n_pad, np.int32), n_pad)
    # the padded index of a layout is what places a previous layer's rows for re-quantisation:
    # every channel appears once, inside its own cluster's positions, pads only at a cluster's end
    idx = L.padded_index()
    off, _ = oracle.segment_offsets(size)
    assert sorted(idx[idx >= 0].tolist()) == list(range(C))
    j = 0
    for c in range(g):
        seg = idx[off[c]:off[c + 1]]
        assert sorted(seg[:size[c]].tolist()) == sorted(perm[j:j + size[c]].tolist()) and np.all(seg[size[c]:] == -1)
        j += size[c]
    assert np.all(idx[off[g]:] == -1)
    # the same array in the oracle's order, moved by contiguous_position(), is the oracle's padded index
    want = np.full(L.K_pad, -1, np.int32)
    j = 0
    for c in range(g):
        want[off[c]:off[c] + size[c]] = perm[j:j + size[c]]
        j += size[c]
    assert np.array_equal(idx, want[L.contiguous_position()])


def test_interleaved_unit_order(binding):
    """Small clusters are placed between the units of the larger ones; every channel keeps its
    cluster and its order within the cluster; packed weights follow the same order."""
    rng = np.random.default_rng(5)
    size = np.array([1, 2, 33, 700, 0, 5, 64, 300, 40, 200, 7, 3, 133], np.int32)
    C, g, bits = int(size.sum()), len(size), 3
    assert C % 8 == 0
    perm = rng.permutation(C).astype(np.int32)
    scale = rng.uniform(0.05, 1.5, size=g).astype(np.float32)
    zero = rng.integers(0, 8, size=g).astype(np.int32)
    Lc = binding.Layout(perm, size, scale, zero, bits)
    Li = binding.Layout(perm, size, scale, zero, bits, order=binding.ORDER_INTERLEAVED)
    assert Li.K_pad == Lc.K_pad and Li.row_bytes == Lc.row_bytes
    units = (size + 31) // 32
    uc = Li.unit_cluster
    assert np.array_equal(np.bincount(uc[uc >= 0], minlength=g), units)
    assert np.all(uc[int(units.sum()):] == -1)
    # clusters of one or two units come after every seven units of larger clusters, each in one piece
    small = [c for c in range(g) if 1 <= units[c] <= 2]
    big_run, placed = 0, []
    u = 0
    while u < int(units.sum()):
        c = int(uc[u])
        if c in small:
            assert np.all(uc[u:u + units[c]] == c)
            placed.append((c, big_run))
            big_run = 0
            u += int(units[c])
        else:
            big_run += 1
            u += 1
    assert [c for c, _ in placed] == small
    n_big_units = int(units.sum()) - sum(int(units[c]) for c in small)
    assert all(run == 7 for _, run in placed[:n_big_units // 7])
    # larger clusters keep their relative order and the order of their own units
    firsts = [int(np.argmax(uc == c)) for c in range(g) if units[c] > 2]
    assert firsts == sorted(firsts)
    # every channel sits once, in a unit of its own cluster
    idx_i, m = Li.padded_index(), Li.contiguous_position()
    assert sorted(idx_i[idx_i >= 0].tolist()) == list(range(C))
    cluster_of = np.empty(C, np.int64)
    cluster_of[perm] = np.repeat(np.arange(g), size)
    real = idx_i >= 0
    assert np.array_equal(np.repeat(uc, 32)[real], cluster_of[idx_i[real]])
    assert sorted(m.tolist()) == list(range(Li.K_pad))
    # packed weights: the oracle's codes with their columns moved to this order
    W = rng.normal(size=(70, C)).astype(np.float32)
    packed, s_w, wsum = binding.weight_pack(Li, W, None, 72)
    w_codes, s_w_o, wsum_o = oracle.weight_quantize(W, perm, size, None, 72)
    assert np.array_equal(packed, oracle.pack_weights(np.ascontiguousarray(w_codes[:, m])))
    assert np.array_equal(s_w, s_w_o) and np.array_equal(wsum, wsum_o)
    # fewer than two small clusters: nothing to interleave
    size2 = np.array([100, 60, 96], np.int32)
    L2 = binding.Layout(rng.permutation(256).astype(np.int32), size2, scale[:3], zero[:3], 4, order=binding.ORDER_INTERLEAVED)
    assert np.array_equal(L2.unit_cluster, binding.Layout(L2._perm, size2, scale[:3], zero[:3], 4).unit_cluster)
    with pytest.raises(binding.RptqError):
        binding.Layout(perm, size, scale, zero, bits, order=2)


def test_numpy_calibration_agrees_with_the_oracle_calibration():
    w = workloads.scaled(workloads.WORKLOADS["opt-125m"], tokens=16, calib_tokens=96)
    gm, bt = workloads.ln_params(w)
    x_cal = workloads.calib_tokens(w)
    for bits in (3, 4, 8):
        u = workloads.kmeans_draws(w, 0, w.clusters)
        a = calibration.calibrate(x_cal, gm, bt, w.clusters, bits, u)
        b = oracle.calibrate(x_cal, gm, bt, w.clusters, bits, u)
        assert np.allclose(a.x_min, b.x_min, rtol=1e-12, atol=1e-12)
        assert np.array_equal(a.perm, b.perm) and np.array_equal(a.size, b.size)
        assert np.array_equal(a.zero, b.zero)
        assert np.allclose(a.scale, b.scale.astype(np.float32), rtol=1e-6)
    # Eq. 2 on the paper's example ranges
    assert calibration.minmax_params(-100, -50, 4) == (3.125, 32)
    assert calibration.minmax_params(80, 100, 4) == (1.25, -64)


def test_workload_generators_are_seeded_and_shaped():
    w = workloads.WORKLOADS["opt-125m"]
    x1, x2 = workloads.test_tokens(w), workloads.test_tokens(w)
    assert x1.dtype == np.float16 and x1.shape == (128, 768) and np.array_equal(x1, x2)
    assert not np.array_equal(x1[:16], workloads.calib_tokens(w, 16))
    gm, bt = workloads.ln_params(w)
    assert gm.shape == (768,) and (gm.astype(np.float32) > 20).sum() >= 1
    full = workloads.weight_matrix(w, 0, 3072, 768)
    part = list(workloads.weight_rows(w, 0, 3072, 768, 1000, 1100))
    assert np.array_equal(np.concatenate([b for _, b in part]), full[1000:1100])
    assert abs(full.std() - 0.02) < 1e-3


def _head_ranges(rng, H, d, planted):
    """Per-channel (min, max) of Q and K with `planted` groups per head: the groups differ in K's range
    only, so a clustering on Q's ranges alone cannot find them."""
    group = np.concatenate([rng.permutation(np.arange(d) % planted) for _ in range(H)])
    q_hi = rng.uniform(0.9, 1.1, size=H * d); q_lo = -rng.uniform(0.9, 1.1, size=H * d)
    k_hi = (1.0 + 4.0 * group) * rng.uniform(0.95, 1.05, size=H * d); k_lo = -k_hi * rng.uniform(0.95, 1.05, size=H * d)
    return (q_lo, q_hi), (k_lo, k_hi), group


def test_attention_sites_share_one_index_between_q_and_k():
    """Sec. 4.2: Q and K of a head are clustered together on (Q max, Q min, K max, K min); Sec. 5.1: per
    head. The numpy calibration agrees with the oracle's composition, finds groups that only K's ranges
    show, and gives each tensor its own Eq. 2 parameters on the shared clusters."""
    rng = np.random.default_rng(3)
    H, d, gh = 3, 32, 4
    q, k, group = _head_ranges(rng, H, d, gh)
    draws = rng.uniform(size=(H, gh))
    cal = calibration.calibrate_heads([q, k], H, gh, (4, 3), draws)
    perm, size, scale, zero = oracle.calibrate_heads([q, k], H, gh, (4, 3), draws)
    assert np.array_equal(cal.perm, perm) and np.array_equal(cal.size, size)
    for t in range(2):
        assert np.array_equal(cal.scale[t], scale[t].astype(np.float32)) and np.array_equal(cal.zero[t], zero[t])
    assert cal.size.shape == (H * gh,) and np.array_equal(np.sort(cal.perm), np.arange(H * d))
    pos = 0
    for h in range(H):
        assert cal.size[h * gh:(h + 1) * gh].sum() == d
        for c in range(gh):
            n = int(cal.size[h * gh + c])
            seg = cal.perm[pos:pos + n]
            pos += n
            assert np.all(seg // d == h)                        # a head's clusters hold that head's channels
            assert len(set(group[seg])) == 1                    # and are the planted groups
            for t, (lo, hi) in enumerate((q, k)):               # Eq. 2 on the cluster's merged range, per tensor
                bits = (4, 3)[t]
                s = (hi[seg].max() - lo[seg].min()) / (1 << bits)
                assert cal.scale[t][h * gh + c] == np.float32(s)
                assert cal.zero[t][h * gh + c] == -int(np.rint((hi[seg].max() + lo[seg].min()) / (2 * s))) + (1 << (bits - 1))
    # a single tensor (R3, the values): the same routine with 2-D points
    v = (k[0] * 0.5, k[1] * 0.5)
    cv = calibration.calibrate_heads([v], H, gh, (4,), draws)
    pv, sv, _, _ = oracle.calibrate_heads([v], H, gh, (4,), draws)
    assert np.array_equal(cv.perm, pv) and np.array_equal(cv.size, sv)


def test_the_layernorm_kernels_hot_instances_do_not_spill(tmp_path):
    """The LayerNorm kernel runs at its 128-register limit: a few more live values (two more fields in its
    parameter struct once did it) put spills into the gather loop of the 3-bit instance and cost 2 - 3 us of
    35. ptxas reports the spills at build time; this compiles the file the way the library build does and
    reads them."""
    import shutil
    import subprocess
    if shutil.which("nvcc") is None:
        pytest.skip("nvcc not available")
    src = os.path.join(lib_build.CSRC, "ln_reorder_quant.cu")
    r = subprocess.run(["nvcc", *lib_build.NVCC_FLAGS, "-Xptxas", "-v", "-c", src, "-o", str(tmp_path / "ln.o")],
                       capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = r.stderr.splitlines()
    spills = {}
    for i, line in enumerate(lines):
        m = re.search(r"ln_reorder_quant_kernelILi(\d)ELb(\d)ELb(\d)EEEv", line)
        if m and "Compiling entry function" in line:
            s = re.search(r"(\d+) bytes spill stores, (\d+) bytes spill loads", " ".join(lines[i + 1:i + 4]))
            spills[(int(m.group(1)), m.group(2) == "1", m.group(3) == "1")] = (int(s.group(1)), int(s.group(2)))
    # the plain instances (no debug output, no self-test): 3- and 8-bit spill nothing, 4-bit at most one register
    assert spills[(3, False, False)] == (0, 0) and spills[(8, False, False)] == (0, 0)
    assert spills[(4, False, False)][0] <= 8 and spills[(4, False, False)][1] <= 8
