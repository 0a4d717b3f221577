"""Python face of the CPU oracle (oracle/rptq_oracle.c), loaded through ctypes.

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the benchmark's CPU
baseline leg. The GPU library and its Python binding never import this package.

The functions below only marshal numpy arrays; all arithmetic is in the C file, whose comments
cite the passages of the paper. `calibrate` composes the calibration steps of Sec. 4.1.
"""
from __future__ import annotations

import ctypes as C
from typing import NamedTuple, Optional, Tuple

import numpy as np

from .build import build as _build

_lib = C.CDLL(_build())

_i64, _i32, _dbl = C.c_int64, C.c_int32, C.c_double
_P = C.c_void_p


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(_P)


def _arr(a, dt) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dt)


_lib.orc_segment_offsets.restype = _i32
_lib.orc_row_bytes.restype = _i64
_lib.orc_weight_codes_bytes.restype = _i64
_lib.orc_cluster_gemm.restype = _i64
_lib.orc_kmeans.restype = C.c_int


# ---------------------------------------------------------------- calibration (Sec. 4.1)
def channel_minmax(y: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    y = _arr(y, np.float64)
    T, Cn = y.shape
    mn, mx = np.empty(Cn), np.empty(Cn)
    _lib.orc_channel_minmax(_p(y), _i64(T), C.c_int(Cn), _p(mn), _p(mx))
    return mn, mx


def minmax_params(x_min: float, x_max: float, k: int) -> Tuple[float, int]:
    s, z = _dbl(), _i32()
    _lib.orc_minmax_params(_dbl(x_min), _dbl(x_max), C.c_int(k), C.byref(s), C.byref(z))
    return s.value, z.value


def kmeans(pts: np.ndarray, g: int, u: np.ndarray, iters: int = 20):
    pts = _arr(pts, np.float64)
    n, dim = pts.shape
    u = _arr(u, np.float64)
    assert u.shape[0] >= g
    labels = np.empty(n, np.int32)
    centres = np.zeros((g, dim))
    inertia = np.zeros(iters)
    rc = _lib.orc_kmeans(_p(pts), C.c_int(n), C.c_int(dim), C.c_int(g), _p(u), C.c_int(iters),
                         _p(labels), _p(centres), _p(inertia))
    assert rc == 0
    return labels, centres, inertia


def reorder_index(labels, x_min, x_max, g: int):
    labels = _arr(labels, np.int32)
    x_min, x_max = _arr(x_min, np.float64), _arr(x_max, np.float64)
    Cn = labels.shape[0]
    perm = np.empty(Cn, np.int32)
    size = np.empty(g, np.int32)
    new_of_old = np.empty(g, np.int32)
    _lib.orc_reorder_index(_p(labels), _p(x_min), _p(x_max), C.c_int(Cn), C.c_int(g),
                           _p(perm), _p(size), _p(new_of_old))
    return perm, size, new_of_old


def segment_offsets(size) -> Tuple[np.ndarray, int]:
    size = _arr(size, np.int32)
    off = np.empty(size.shape[0] + 1, np.int32)
    k_pad = _lib.orc_segment_offsets(_p(size), C.c_int(size.shape[0]), _p(off))
    return off, int(k_pad)


def row_bytes(k_pad: int, k: int) -> int:
    return int(_lib.orc_row_bytes(_i32(k_pad), C.c_int(k)))


# ---------------------------------------------------------------- hot path steps
def layernorm(x16: np.ndarray, gamma16: np.ndarray, beta16: np.ndarray, eps: float) -> np.ndarray:
    """fp16 inputs are widened exactly to fp64; result fp64 [M][C] in original channel order."""
    x = _arr(x16, np.float64)
    gm, bt = _arr(gamma16, np.float64), _arr(beta16, np.float64)
    M, Cn = x.shape
    y = np.empty((M, Cn))
    _lib.orc_layernorm(_p(x), _p(gm), _p(bt), _i64(M), C.c_int(Cn), _dbl(eps), _p(y))
    return y


def reorder(y: np.ndarray, perm) -> np.ndarray:
    y = _arr(y, np.float64)
    perm = _arr(perm, np.int32)
    out = np.empty_like(y)
    _lib.orc_reorder(_p(y), _i64(y.shape[0]), C.c_int(y.shape[1]), _p(perm), _p(out))
    return out


def quantize(y_r: np.ndarray, size, scale, zero, k: int) -> np.ndarray:
    """fp64 decision. Returns unpacked codes uint8 [M][K_pad] in the padded segment layout."""
    y_r = _arr(y_r, np.float64)
    size, zero = _arr(size, np.int32), _arr(zero, np.int32)
    scale = _arr(scale, np.float64)
    _, k_pad = segment_offsets(size)
    M, Cn = y_r.shape
    codes = np.empty((M, k_pad), np.uint8)
    _lib.orc_quantize_clusters(_p(y_r), _i64(M), C.c_int(Cn), C.c_int(size.shape[0]), _p(size),
                               _p(scale), _p(zero), C.c_int(k), _i32(k_pad), _p(codes))
    return codes


def quantize_f32(y_r32: np.ndarray, size, scale32, zero, k: int) -> np.ndarray:
    """fp32 decision on given fp32 LayerNorm outputs (the precision the GPU decides in)."""
    y_r32 = _arr(y_r32, np.float32)
    size, zero = _arr(size, np.int32), _arr(zero, np.int32)
    scale32 = _arr(scale32, np.float32)
    _, k_pad = segment_offsets(size)
    M, Cn = y_r32.shape
    codes = np.empty((M, k_pad), np.uint8)
    _lib.orc_quantize_clusters_f32(_p(y_r32), _i64(M), C.c_int(Cn), C.c_int(size.shape[0]), _p(size),
                                   _p(scale32), _p(zero), C.c_int(k), _i32(k_pad), _p(codes))
    return codes


def dequantize(codes: np.ndarray, Cn: int, size, scale, zero) -> np.ndarray:
    codes = _arr(codes, np.uint8)
    size, zero = _arr(size, np.int32), _arr(zero, np.int32)
    scale = _arr(scale, np.float64)
    M, k_pad = codes.shape
    out = np.empty((M, Cn))
    _lib.orc_dequantize_clusters(_p(codes), _i64(M), C.c_int(Cn), C.c_int(size.shape[0]), _p(size),
                                 _p(scale), _p(zero), _i32(k_pad), _p(out))
    return out


def pack(codes: np.ndarray, k: int) -> np.ndarray:
    codes = _arr(codes, np.uint8)
    M, k_pad = codes.shape
    out = np.empty((M, row_bytes(k_pad, k)), np.uint8)
    _lib.orc_pack_codes(_p(codes), _i64(M), _i32(k_pad), C.c_int(k), _p(out))
    return out


def unpack(packed: np.ndarray, k_pad: int, k: int) -> np.ndarray:
    packed = _arr(packed, np.uint8)
    M = packed.shape[0]
    assert packed.shape[1] == row_bytes(k_pad, k)
    out = np.empty((M, k_pad), np.uint8)
    _lib.orc_unpack_codes(_p(packed), _i64(M), _i32(k_pad), C.c_int(k), _p(out))
    return out


def weight_codes_bytes(n_rows: int, k_pad: int) -> int:
    return int(_lib.orc_weight_codes_bytes(_i64(n_rows), _i32(k_pad)))


def pack_weights(w_codes: np.ndarray) -> np.ndarray:
    """Tile-major packed weight buffer (flat uint8) of int8 codes [N][K_pad]."""
    w_codes = _arr(w_codes, np.int8)
    N, k_pad = w_codes.shape
    out = np.empty(weight_codes_bytes(N, k_pad), np.uint8)
    _lib.orc_pack_weight_codes(_p(w_codes), _i64(N), _i32(k_pad), _p(out))
    return out


def unpack_weights(packed: np.ndarray, k_pad: int, n_rows: int) -> np.ndarray:
    packed = _arr(packed, np.uint8).reshape(-1)
    assert packed.shape[0] >= weight_codes_bytes(n_rows, k_pad)
    out = np.empty((n_rows, k_pad), np.int8)
    _lib.orc_unpack_weight_codes(_p(packed), _i64(n_rows), _i32(k_pad), _p(out))
    return out


def weight_quantize(W: np.ndarray, perm, size, out_perm=None, n_pad: Optional[int] = None):
    """Returns (w_codes int8 [N_pad][K_pad], s_w fp32 [N_pad], wsum int32 [g][N_pad])."""
    W = _arr(W, np.float32)
    perm, size = _arr(perm, np.int32), _arr(size, np.int32)
    N, Cn = W.shape
    n_pad = N if n_pad is None else n_pad
    g = size.shape[0]
    _, k_pad = segment_offsets(size)
    op = None if out_perm is None else _arr(out_perm, np.int32)
    if op is not None:
        if n_pad == N and op.shape[0] != N:
            n_pad = int(op.shape[0])
        assert op.shape[0] == n_pad, "out_perm has one entry per output row"
    w_codes = np.empty((n_pad, k_pad), np.int8)
    s_w = np.empty(n_pad, np.float32)
    wsum = np.empty((g, n_pad), np.int32)
    _lib.orc_weight_quantize(_p(W), _i64(N), C.c_int(Cn), C.c_int(g), _p(perm), _p(size), _p(op),
                             _i64(n_pad), _i32(k_pad), _p(w_codes), _p(s_w), _p(wsum))
    return w_codes, s_w, wsum


def cluster_acc(a_codes: np.ndarray, w_codes: np.ndarray, size) -> np.ndarray:
    a_codes, w_codes = _arr(a_codes, np.uint8), _arr(w_codes, np.int8)
    size = _arr(size, np.int32)
    M, k_pad = a_codes.shape
    N = w_codes.shape[0]
    assert w_codes.shape[1] == k_pad
    acc = np.empty((size.shape[0], M, N), np.int64)
    _lib.orc_cluster_acc(_p(a_codes), _i64(M), _p(w_codes), _i64(N), _i32(k_pad),
                         C.c_int(size.shape[0]), _p(size), _p(acc))
    return acc


def cluster_gemm(a_codes, w_codes, size, scale, zero, s_w, wsum, bias=None, relu=False) -> np.ndarray:
    a_codes, w_codes = _arr(a_codes, np.uint8), _arr(w_codes, np.int8)
    size, zero = _arr(size, np.int32), _arr(zero, np.int32)
    scale = _arr(scale, np.float64)
    s_w = _arr(s_w, np.float32)
    wsum = _arr(wsum, np.int32)
    M, k_pad = a_codes.shape
    N = w_codes.shape[0]
    assert w_codes.shape[1] == k_pad and wsum.shape[0] == size.shape[0] and wsum.shape[1] >= N
    b = None if bias is None else _arr(bias, np.float32)
    y = np.empty((M, N))
    ovf = _lib.orc_cluster_gemm(_p(a_codes), _i64(M), _p(w_codes), _i64(N), _i32(k_pad),
                                C.c_int(size.shape[0]), _p(size), _p(scale), _p(zero), _p(s_w),
                                _p(wsum), _i64(wsum.shape[1]), _p(b), C.c_int(1 if relu else 0), _p(y))
    assert ovf == 0, f"{ovf} per-cluster accumulators exceed int32"
    return y


def dequant_matmul(a_codes, w_codes, size, scale, zero, s_w) -> np.ndarray:
    a_codes, w_codes = _arr(a_codes, np.uint8), _arr(w_codes, np.int8)
    size, zero = _arr(size, np.int32), _arr(zero, np.int32)
    scale = _arr(scale, np.float64)
    s_w = _arr(s_w, np.float32)
    M, k_pad = a_codes.shape
    N = w_codes.shape[0]
    y = np.empty((M, N))
    _lib.orc_dequant_matmul(_p(a_codes), _i64(M), _p(w_codes), _i64(N), _i32(k_pad),
                            C.c_int(size.shape[0]), _p(size), _p(scale), _p(zero), _p(s_w), _p(y))
    return y


def dequant_matmul_bf16(a_codes, w_codes, size, scale32, zero, s_w, bias=None, relu=False) -> np.ndarray:
    """First method with the de-quantised activation rounded to bfloat16 (the operand precision of a
    16-bit tensor-core product)."""
    a_codes, w_codes = _arr(a_codes, np.uint8), _arr(w_codes, np.int8)
    size, zero = _arr(size, np.int32), _arr(zero, np.int32)
    scale32, s_w = _arr(scale32, np.float32), _arr(s_w, np.float32)
    M, k_pad = a_codes.shape
    N = w_codes.shape[0]
    b = None if bias is None else _arr(bias, np.float32)
    y = np.empty((M, N))
    _lib.orc_dequant_matmul_bf16(_p(a_codes), _i64(M), _p(w_codes), _i64(N), _i32(k_pad), C.c_int(size.shape[0]), _p(size),
                                 _p(scale32), _p(zero), _p(s_w), _p(b), C.c_int(1 if relu else 0), _p(y))
    return y


# ---------------------------------------------------------------- per-cluster asymmetric weights
def weight_quantize_clustered(W: np.ndarray, perm, size, k: int = 4, n_pad: Optional[int] = None):
    """Returns (w_codes uint8 [N_pad][K_pad], s_w fp32 [g][N_pad], z_w int32 [g][N_pad], wsum int32 [g][N_pad])."""
    W = _arr(W, np.float32)
    perm, size = _arr(perm, np.int32), _arr(size, np.int32)
    N, Cn = W.shape
    n_pad = N if n_pad is None else n_pad
    g = size.shape[0]
    _, k_pad = segment_offsets(size)
    w_codes = np.empty((n_pad, k_pad), np.uint8)
    s_w = np.empty((g, n_pad), np.float32)
    z_w = np.empty((g, n_pad), np.int32)
    wsum = np.empty((g, n_pad), np.int32)
    _lib.orc_weight_quantize_clustered(_p(W), _i64(N), C.c_int(Cn), C.c_int(g), C.c_int(k), _p(perm), _p(size),
                                       _i64(n_pad), _i32(k_pad), _p(w_codes), _p(s_w), _p(z_w), _p(wsum))
    return w_codes, s_w, z_w, wsum


def code_rowsums(a_codes, size) -> np.ndarray:
    a_codes, size = _arr(a_codes, np.uint8), _arr(size, np.int32)
    M, k_pad = a_codes.shape
    out = np.empty((M, size.shape[0]), np.int32)
    _lib.orc_code_rowsums(_p(a_codes), _i64(M), _i32(k_pad), C.c_int(size.shape[0]), _p(size), _p(out))
    return out


def _asym_args(a_codes, w_codes, size, scale, zero, s_w, z_w):
    a_codes, w_codes = _arr(a_codes, np.uint8), _arr(w_codes, np.uint8)
    size, zero = _arr(size, np.int32), _arr(zero, np.int32)
    scale, s_w, z_w = _arr(scale, np.float64), _arr(s_w, np.float32), _arr(z_w, np.int32)
    M, k_pad = a_codes.shape
    N = w_codes.shape[0]
    g = size.shape[0]
    assert w_codes.shape[1] == k_pad and s_w.shape == z_w.shape and s_w.shape[0] == g and s_w.shape[1] >= N
    return a_codes, w_codes, size, scale, zero, s_w, z_w, M, N, k_pad, g


def cluster_gemm_asym(a_codes, w_codes, size, scale, zero, s_w, z_w, bias=None, relu=False) -> np.ndarray:
    a_codes, w_codes, size, scale, zero, s_w, z_w, M, N, k_pad, g = _asym_args(a_codes, w_codes, size, scale, zero, s_w, z_w)
    b = None if bias is None else _arr(bias, np.float32)
    y = np.empty((M, N))
    _lib.orc_cluster_gemm_asym(_p(a_codes), _i64(M), _p(w_codes), _i64(N), _i32(k_pad), C.c_int(g), _p(size), _p(scale),
                               _p(zero), _p(s_w), _p(z_w), _i64(s_w.shape[1]), _p(b), C.c_int(1 if relu else 0), _p(y))
    return y


def dequant_matmul_asym(a_codes, w_codes, size, scale, zero, s_w, z_w) -> np.ndarray:
    a_codes, w_codes, size, scale, zero, s_w, z_w, M, N, k_pad, g = _asym_args(a_codes, w_codes, size, scale, zero, s_w, z_w)
    y = np.empty((M, N))
    _lib.orc_dequant_matmul_asym(_p(a_codes), _i64(M), _p(w_codes), _i64(N), _i32(k_pad), C.c_int(g), _p(size), _p(scale),
                                 _p(zero), _p(s_w), _p(z_w), _i64(s_w.shape[1]), _p(y))
    return y


# ---------------------------------------------------------------- attention sites (Sec. 4.2, 5.1)
def attention(q_codes, k_codes, v_codes, H: int, gh: int, size_qk, sQ, zQ, sK, zK, size_v, sV, zV,
              s_P: float, z_P: int, qk_scale: float, causal: bool, return_p: bool = False):
    """Codes at padded positions: q [Tq][K_pad_qk], k [Tk][K_pad_qk], v [Tk][K_pad_v]; head h owns
    clusters h*gh .. h*gh+gh-1 of both layouts. Returns O [Tq][K_pad_v] (and Pq [H][Tq][Tk])."""
    q_codes, k_codes, v_codes = _arr(q_codes, np.uint8), _arr(k_codes, np.uint8), _arr(v_codes, np.uint8)
    size_qk, size_v = _arr(size_qk, np.int32), _arr(size_v, np.int32)
    sQ, sK, sV = _arr(sQ, np.float64), _arr(sK, np.float64), _arr(sV, np.float64)
    zQ, zK, zV = _arr(zQ, np.int32), _arr(zK, np.int32), _arr(zV, np.int32)
    Tq, kp = q_codes.shape
    Tk, kpv = v_codes.shape
    g = H * gh
    assert k_codes.shape == (Tk, kp) and Tq <= Tk
    for a in (size_qk, size_v, sQ, sK, sV, zQ, zK, zV):
        assert a.shape == (g,)
    out = np.empty((Tq, kpv))
    pq = np.empty((H, Tq, Tk), np.uint8) if return_p else None
    _lib.orc_attention(_p(q_codes), _p(k_codes), _p(v_codes), _i64(Tq), _i64(Tk), C.c_int(H), C.c_int(gh),
                       _i32(kp), _p(size_qk), _p(sQ), _p(zQ), _p(sK), _p(zK),
                       _i32(kpv), _p(size_v), _p(sV), _p(zV),
                       _dbl(s_P), _i32(z_P), _dbl(qk_scale), C.c_int(1 if causal else 0), _p(out), _p(pq))
    return (out, pq) if return_p else out


def attention_kv(q, ch_of_pos_k, k_codes, v_codes, H: int, gh: int, size_k, sK, zK, size_v, sV, zV,
                 qk_scale: float, causal: bool) -> np.ndarray:
    """Sec. 5.2, key / value cache quantised only: q [Tq][C] floating point in the original channel order,
    ch_of_pos_k int [K_pad_k] the channel at each padded position of K's layout (-1 at pads), codes at
    padded positions. Returns O [Tq][K_pad_v]."""
    q = _arr(q, np.float64)
    ch = _arr(ch_of_pos_k, np.int32)
    k_codes, v_codes = _arr(k_codes, np.uint8), _arr(v_codes, np.uint8)
    size_k, size_v = _arr(size_k, np.int32), _arr(size_v, np.int32)
    sK, sV, zK, zV = _arr(sK, np.float64), _arr(sV, np.float64), _arr(zK, np.int32), _arr(zV, np.int32)
    Tq, Cn = q.shape
    Tk, kpk = k_codes.shape
    kpv = v_codes.shape[1]
    assert ch.shape == (kpk,) and v_codes.shape[0] == Tk and Tq <= Tk and size_k.shape == (H * gh,) == size_v.shape
    out = np.empty((Tq, kpv))
    _lib.orc_attention_kv(_p(q), C.c_int(Cn), _p(ch), _p(k_codes), _p(v_codes), _i64(Tq), _i64(Tk), C.c_int(H), C.c_int(gh),
                          _i32(kpk), _p(size_k), _p(sK), _p(zK), _i32(kpv), _p(size_v), _p(sV), _p(zV),
                          _dbl(qk_scale), C.c_int(1 if causal else 0), _p(out))
    return out


def attention_output(p_codes, v_codes, H: int, gh: int, size_v, sV, zV, s_P: float, z_P: int) -> np.ndarray:
    """O from given softmax codes p_codes [H][Tq][Tk] and V codes [Tk][K_pad_v]."""
    p_codes, v_codes = _arr(p_codes, np.uint8), _arr(v_codes, np.uint8)
    size_v, sV, zV = _arr(size_v, np.int32), _arr(sV, np.float64), _arr(zV, np.int32)
    Hn, Tq, Tk = p_codes.shape
    assert Hn == H and v_codes.shape[0] == Tk and size_v.shape == (H * gh,)
    out = np.empty((Tq, v_codes.shape[1]))
    _lib.orc_attention_output(_p(p_codes), _p(v_codes), _i64(Tq), _i64(Tk), C.c_int(H), C.c_int(gh), _i32(v_codes.shape[1]),
                              _p(size_v), _p(sV), _p(zV), _dbl(s_P), _i32(z_P), _p(out))
    return out


# ---------------------------------------------------------------- calibration pipeline
class Calibration(NamedTuple):
    perm: np.ndarray      # int32 [C]  reorder index S
    size: np.ndarray      # int32 [g]  cluster sizes in S order
    scale: np.ndarray     # fp64  [g]
    zero: np.ndarray      # int32 [g]  unsigned-range zero points
    x_min: np.ndarray     # fp64  [C]  per-channel calibration minimum (original order)
    x_max: np.ndarray
    labels: np.ndarray    # int32 [C]  cluster of each channel, in S's cluster numbering


def calibrate_from_minmax(x_min, x_max, g: int, k: int, u, iters: int = 20) -> Calibration:
    """Sec. 4.1 + Sec. 5.1: cluster channels on (min, max), build S, then Min-Max parameters
    (Eq. 2) from the merged range of each cluster."""
    x_min, x_max = _arr(x_min, np.float64), _arr(x_max, np.float64)
    pts = np.stack([x_min, x_max], axis=1)
    labels, _, _ = kmeans(pts, g, u, iters)
    perm, size, new_of_old = reorder_index(labels, x_min, x_max, g)
    scale = np.ones(g)
    zero = np.zeros(g, np.int32)
    pos = 0
    for c in range(g):
        n = int(size[c])
        if n:
            members = perm[pos:pos + n]
            scale[c], zero[c] = minmax_params(float(x_min[members].min()), float(x_max[members].max()), k)
        else:
            scale[c], zero[c] = 1.0, 1 << (k - 1)
        pos += n
    return Calibration(perm, size, scale, zero, x_min, x_max, new_of_old[labels].astype(np.int32))


def calibrate(x_cal16, gamma16, beta16, g: int, k: int, u, eps: float = 1e-5, iters: int = 20) -> Calibration:
    y = layernorm(x_cal16, gamma16, beta16, eps)
    x_min, x_max = channel_minmax(y)
    return calibrate_from_minmax(x_min, x_max, g, k, u, iters)


def calibrate_heads(ranges, n_heads: int, g_head: int, bits, u, iters: int = 20):
    """Sec. 4.2 / 5.1: per-head reorder of an attention site. `ranges`: [(min, max)] per tensor that shares
    the index -- for Q and K the head's channels are clustered on the 4-D points (Q max, Q min, K max,
    K min). Composition of orc_kmeans, orc_reorder_index (on the union of the ranges) and
    orc_minmax_params per tensor and cluster. Returns (perm, size, [scale per tensor], [zero per tensor])."""
    ranges = [(_arr(lo, np.float64), _arr(hi, np.float64)) for lo, hi in ranges]
    Cn = ranges[0][0].shape[0]
    d = Cn // n_heads
    lo_all = np.min([r[0] for r in ranges], axis=0)
    hi_all = np.max([r[1] for r in ranges], axis=0)
    perm, size = [], []
    scale = [[] for _ in ranges]
    zero = [[] for _ in ranges]
    for h in range(n_heads):
        sl = slice(h * d, (h + 1) * d)
        pts = np.stack([a[sl] for r in ranges for a in (r[1], r[0])], axis=1)
        labels, _, _ = kmeans(pts, g_head, np.asarray(u)[h], iters)
        p_h, size_h, _ = reorder_index(labels, lo_all[sl], hi_all[sl], g_head)
        perm.append(h * d + p_h)
        size.append(size_h)
        pos = 0
        for c in range(g_head):
            n = int(size_h[c])
            seg = h * d + p_h[pos:pos + n]
            for t, (lo, hi) in enumerate(ranges):
                s, z = minmax_params(lo[seg].min(), hi[seg].max(), bits[t]) if n else (1.0, 1 << (bits[t] - 1))
                scale[t].append(s); zero[t].append(z)
            pos += n
    return (np.concatenate(perm).astype(np.int32), np.concatenate(size).astype(np.int32),
            [np.array(x, np.float64) for x in scale], [np.array(x, np.int32) for x in zero])
