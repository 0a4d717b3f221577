"""Thin Python binding of librptq.so (include/rptq.h): argument marshalling only.

Every step of the hot path runs in the library's CUDA kernels. PyTorch appears here only as the
owner of device memory and streams. If the library is missing this module raises at import time;
there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librptq.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_NOT_BIJECTION, ERR_CUDA, ERR_DEVICE_TIMEOUT, ERR_ALLOC = 0, -1, -2, -3, -4, -5, -6
OUT_F32, OUT_F16, OUT_CODES = 0, 1, 2
ACT_NONE, ACT_RELU = 0, 1
NOALLOC_MAX_N = 65536
ORDER_CONTIGUOUS, ORDER_INTERLEAVED = 0, 1

EXPORTS = (
    "rptq_layout_create", "rptq_layout_query", "rptq_layout_destroy", "rptq_ln_reorder_quant",
    "rptq_weight_pack", "rptq_cluster_gemm", "rptq_cluster_gemm_debug_acc", "rptq_codes_unpack_host",
    "rptq_codes_pack_host", "rptq_weight_unpack_host", "rptq_get_device_status", "rptq_status_string",
    "rptq_format_version", "rptq_layout_padded_index", "rptq_weight_codes_bytes", "rptq_cluster_gemm_noalloc",
    "rptq_selftest_ln_timeout", "rptq_dequant_gemm", "rptq_ln_channel_minmax", "rptq_kmeans", "rptq_kmeans_workspace_bytes",
    "rptq_probe_int8_peak", "rptq_weight_pack_clustered", "rptq_code_rowsums", "rptq_cluster_gemm_clustered",
    "rptq_attention", "rptq_attention_kv",
)


class RptqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


def _load(path: str = LIB_PATH) -> C.CDLL:
    if not os.path.exists(path):
        raise ImportError(
            f"{path} is missing: build it with `python -m paper_2304_01089_b200.build` "
            "(nvcc, sm_100a). There is no CPU or PyTorch fallback.")
    lib = C.CDLL(path)
    vp, i32, i64, f32 = C.c_void_p, C.c_int, C.c_int64, C.c_float
    lib.rptq_layout_create.argtypes = [C.POINTER(vp), i32, i32, i32, vp, vp, vp, vp, i32]
    lib.rptq_layout_query.argtypes = [vp, C.POINTER(i32), C.POINTER(i64), vp]
    lib.rptq_layout_destroy.argtypes = [vp]
    lib.rptq_layout_padded_index.argtypes = [vp, vp]
    lib.rptq_ln_reorder_quant.argtypes = [vp, vp, i64, vp, vp, f32, i32, vp, vp, vp]
    lib.rptq_weight_pack.argtypes = [vp, vp, i32, vp, i32, vp, vp, vp]
    lib.rptq_cluster_gemm.argtypes = [vp, vp, i32, vp, vp, vp, i64, vp, i32, i32, vp, vp, i32, i64, vp]
    lib.rptq_cluster_gemm_noalloc.argtypes = lib.rptq_cluster_gemm.argtypes
    lib.rptq_cluster_gemm_debug_acc.argtypes = [vp, vp, i32, vp, i32, i32, i32, i32, i32, vp, vp]
    lib.rptq_codes_unpack_host.argtypes = [i32, i32, vp, i64, vp]
    lib.rptq_codes_pack_host.argtypes = [i32, i32, vp, i64, vp]
    lib.rptq_weight_unpack_host.argtypes = [i32, vp, i64, vp]
    lib.rptq_weight_codes_bytes.argtypes = [i32, i64]
    lib.rptq_selftest_ln_timeout.argtypes = [vp, vp, i64, vp, vp, f32, i32, vp, vp]
    lib.rptq_dequant_gemm.argtypes = [vp, vp, i32, vp, vp, i64, vp, i32, i32, vp, i32, i64, vp]
    lib.rptq_ln_channel_minmax.argtypes = [vp, i64, vp, vp, f32, i32, i32, vp, vp, vp]
    lib.rptq_kmeans_workspace_bytes.argtypes = [i32, i32]
    lib.rptq_kmeans.argtypes = [vp, i32, i32, i32, vp, i32, vp, vp, vp, vp, vp]
    lib.rptq_weight_pack_clustered.argtypes = [vp, vp, i32, i32, vp, vp, vp, vp]
    lib.rptq_code_rowsums.argtypes = [vp, vp, i32, vp, vp]
    lib.rptq_cluster_gemm_clustered.argtypes = [vp, vp, i32, vp, vp, vp, vp, vp, i64, vp, i32, i32, vp, vp, i32, i64, vp]
    lib.rptq_probe_int8_peak.argtypes = [i32, vp, C.POINTER(C.c_double), vp]
    lib.rptq_get_device_status.argtypes = [C.POINTER(i32)]
    lib.rptq_status_string.argtypes = [i32]
    lib.rptq_status_string.restype = C.c_char_p
    lib.rptq_attention.argtypes = [vp, vp, vp, i32, vp, i32, vp, vp, i32, i32, f32, i32, f32, i32, vp, i64, vp, vp]
    lib.rptq_attention_kv.argtypes = [vp, vp, i32, vp, i64, i32, vp, vp, i32, i32, f32, i32, vp, i64, vp]
    for name in EXPORTS:
        if name not in ("rptq_status_string", "rptq_weight_codes_bytes", "rptq_kmeans_workspace_bytes"):
            getattr(lib, name).restype = i32
    lib.rptq_weight_codes_bytes.restype = i64
    lib.rptq_kmeans_workspace_bytes.restype = i64
    return lib


_lib = _load()


def status_string(status: int) -> str:
    return _lib.rptq_status_string(int(status)).decode()


def format_version() -> int:
    return int(_lib.rptq_format_version())


def _check(status: int, where: str) -> None:
    if status != OK:
        raise RptqError(status, where)


def _np_ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _dev_ptr(t) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return t.data_ptr()


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


class Layout:
    """rptq_layout_create / _query / _destroy: reorder index S, cluster sizes, (s_c, z_c)."""

    def __init__(self, perm, cluster_size, scale, zero, bits: int, order: int = ORDER_CONTIGUOUS):
        self._perm = np.ascontiguousarray(perm, dtype=np.int32)
        self._size = np.ascontiguousarray(cluster_size, dtype=np.int32)
        self._scale = np.ascontiguousarray(scale, dtype=np.float32)
        self._zero = np.ascontiguousarray(zero, dtype=np.int32)
        if not (self._size.shape == self._scale.shape == self._zero.shape):
            raise ValueError("cluster_size, scale and zero must have one entry per cluster")
        self.C, self.g, self.bits = int(self._perm.shape[0]), int(self._size.shape[0]), int(bits)
        h = C.c_void_p()
        _check(_lib.rptq_layout_create(C.byref(h), self.C, self.g, self.bits, _np_ptr(self._perm),
                                       _np_ptr(self._size), _np_ptr(self._scale), _np_ptr(self._zero), int(order)),
               "rptq_layout_create")
        self._h = h
        self.order = int(order)
        k_pad, rb = C.c_int(), C.c_int64()
        _check(_lib.rptq_layout_query(self._h, C.byref(k_pad), C.byref(rb), None), "rptq_layout_query")
        self.K_pad, self.row_bytes = int(k_pad.value), int(rb.value)
        self.unit_cluster = np.empty(self.K_pad // 32, np.int32)      # owning cluster of each unit of 32 positions
        _check(_lib.rptq_layout_query(self._h, None, None, _np_ptr(self.unit_cluster)), "rptq_layout_query")

    @property
    def handle(self) -> C.c_void_p:
        if self._h is None:
            raise ValueError("layout was destroyed")
        return self._h

    def padded_index(self) -> np.ndarray:
        """int32 [K_pad]: original channel at each padded position, -1 at pads."""
        out = np.empty(self.K_pad, np.int32)
        _check(_lib.rptq_layout_padded_index(self.handle, _np_ptr(out)), "rptq_layout_padded_index")
        return out

    def contiguous_position(self) -> np.ndarray:
        """int32 [K_pad]: for each position of this layout, the position that holds the same channel
        (or a pad of the same cluster) in the plain contiguous order, where cluster c starts at
        seg_off[c] = sum_{c' < c} roundup32(n_c') and holds its channels in the order of S.
        A [*, K_pad] array `a` in that order becomes `a[:, m]` in this layout's order."""
        size = self._size.astype(np.int64)
        seg_off = np.concatenate([[0], np.cumsum((size + 31) // 32 * 32)])
        j_start = np.concatenate([[0], np.cumsum(size)])
        plain = np.empty(self.C, np.int64)               # plain[ch]: contiguous position of channel ch
        for c in range(self.g):
            plain[self._perm[j_start[c]:j_start[c + 1]]] = seg_off[c] + np.arange(size[c])
        idx = self.padded_index()
        out = np.empty(self.K_pad, np.int32)
        next_pad = (seg_off[:-1] + size).copy()          # first pad position of each cluster
        tail = int(seg_off[-1])
        for p in range(self.K_pad):
            if idx[p] >= 0:
                out[p] = plain[idx[p]]
                continue
            c = self.unit_cluster[p // 32]
            if c < 0:
                out[p] = tail
                tail += 1
            else:
                out[p] = next_pad[c]
                next_pad[c] += 1
        return out

    def destroy(self) -> None:
        if getattr(self, "_h", None) is not None:
            _lib.rptq_layout_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def ln_reorder_quant(layout: Layout, x, gamma, beta, eps: float, codes, y_dbg=None, M: Optional[int] = None,
                     ldx: Optional[int] = None, stream=None) -> None:
    """rptq_ln_reorder_quant on device tensors: x fp16 [M][ldx], gamma/beta fp16 [C],
    codes uint8 [M][row_bytes], y_dbg optional fp32 [M][C]."""
    M = int(x.shape[0]) if M is None else int(M)
    ldx = int(x.stride(0)) if ldx is None else int(ldx)
    _check(_lib.rptq_ln_reorder_quant(layout.handle, _dev_ptr(x), ldx, _dev_ptr(gamma), _dev_ptr(beta),
                                      C.c_float(eps), M, _dev_ptr(codes), _dev_ptr(y_dbg), _stream_ptr(stream)),
           "rptq_ln_reorder_quant")


def selftest_ln_timeout(layout: Layout, x, gamma, beta, eps: float, codes, M: Optional[int] = None, stream=None) -> None:
    """rptq_selftest_ln_timeout: the LayerNorm kernel with barriers that cannot complete and a ~5 ms wait budget."""
    M = int(x.shape[0]) if M is None else int(M)
    _check(_lib.rptq_selftest_ln_timeout(layout.handle, _dev_ptr(x), int(x.stride(0)), _dev_ptr(gamma), _dev_ptr(beta),
                                         C.c_float(eps), M, _dev_ptr(codes), _stream_ptr(stream)), "rptq_selftest_ln_timeout")


def attention(LQ: Layout, LK: Layout, LV: Layout, n_heads: int, q_codes, k_codes, v_codes, out, s_P: float,
              qk_scale: float, causal: bool, z_P: int = 0, Tq: Optional[int] = None, Tk: Optional[int] = None,
              n_seq: int = 1, p_codes=None, stream=None) -> None:
    """rptq_attention on n_seq sequences of Tq queries and Tk keys each: q_codes uint8 [n_seq * Tq][LQ.row_bytes],
    k_codes / v_codes uint8 [n_seq * Tk][row_bytes] CUDA tensors, out fp16 [n_seq * Tq][>= LV.C]; p_codes:
    optional uint8 [n_seq][n_heads][Tq][Tk] (zeroed by the caller)."""
    Tq = int(q_codes.shape[0]) // int(n_seq) if Tq is None else int(Tq)
    Tk = int(k_codes.shape[0]) // int(n_seq) if Tk is None else int(Tk)
    _check(_lib.rptq_attention(LQ.handle, LK.handle, LV.handle, int(n_heads), _dev_ptr(q_codes), Tq, _dev_ptr(k_codes),
                               _dev_ptr(v_codes), Tk, int(n_seq), C.c_float(s_P), int(z_P), C.c_float(qk_scale), 1 if causal else 0,
                               _dev_ptr(out), int(out.stride(0)), _dev_ptr(p_codes), _stream_ptr(stream)), "rptq_attention")


def attention_kv(LK: Layout, LV: Layout, n_heads: int, q, k_codes, v_codes, out, qk_scale: float, causal: bool,
                 Tq: Optional[int] = None, Tk: Optional[int] = None, n_seq: int = 1, stream=None) -> None:
    """rptq_attention_kv: q fp16 [n_seq * Tq][>= C] (original channel order), k_codes / v_codes uint8
    [n_seq * Tk][row_bytes], out fp16 [n_seq * Tq][>= C]: CUDA tensors."""
    Tq = int(q.shape[0]) // int(n_seq) if Tq is None else int(Tq)
    Tk = int(k_codes.shape[0]) // int(n_seq) if Tk is None else int(Tk)
    _check(_lib.rptq_attention_kv(LK.handle, LV.handle, int(n_heads), _dev_ptr(q), int(q.stride(0)), Tq, _dev_ptr(k_codes),
                                  _dev_ptr(v_codes), Tk, int(n_seq), C.c_float(qk_scale), 1 if causal else 0,
                                  _dev_ptr(out), int(out.stride(0)), _stream_ptr(stream)), "rptq_attention_kv")


def weight_pack(layout_in: Layout, W: np.ndarray, out_perm=None, n_pad: Optional[int] = None):
    """rptq_weight_pack on host arrays. Returns (w_codes: flat uint8 tile-major buffer of
    weight_codes_bytes(K_pad, N_pad) bytes, s_w fp32 [N_pad], wsum int32 [g][N_pad])."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    N, Cn = W.shape
    if Cn != layout_in.C:
        raise ValueError("W must be [N][C] with C the layout's channel count")
    n_pad = N if n_pad is None else int(n_pad)
    op = None if out_perm is None else np.ascontiguousarray(out_perm, dtype=np.int32)
    if op is not None:
        n_pad = int(op.shape[0]) if n_pad == N and op.shape[0] != N else n_pad
        if op.shape[0] != n_pad:
            raise ValueError("out_perm must have one entry per output row (N_pad)")
    w_codes = np.empty(weight_codes_bytes(layout_in.K_pad, n_pad), np.uint8)
    s_w = np.empty(n_pad, np.float32)
    wsum = np.empty((layout_in.g, n_pad), np.int32)
    _check(_lib.rptq_weight_pack(layout_in.handle, _np_ptr(W), N, _np_ptr(op), n_pad, _np_ptr(w_codes),
                                 _np_ptr(s_w), _np_ptr(wsum)), "rptq_weight_pack")
    return w_codes, s_w, wsum


def cluster_gemm(layout_in: Layout, a_codes, M: int, w_codes, s_w, wsum, N: int, y, *, ld_w: Optional[int] = None,
                 bias=None, act: int = ACT_NONE, layout_out: Optional[Layout] = None, y_dtype: int = OUT_F32,
                 ldy: Optional[int] = None, stream=None) -> None:
    """rptq_cluster_gemm on device tensors."""
    ld_w = int(s_w.shape[0]) if ld_w is None else int(ld_w)
    if ldy is None:
        ldy = 0 if y_dtype == OUT_CODES else int(y.stride(0))
    _check(_lib.rptq_cluster_gemm(layout_in.handle, _dev_ptr(a_codes), int(M), _dev_ptr(w_codes), _dev_ptr(s_w),
                                  _dev_ptr(wsum), ld_w, _dev_ptr(bias), int(N), int(act),
                                  None if layout_out is None else layout_out.handle, _dev_ptr(y), int(y_dtype),
                                  int(ldy), _stream_ptr(stream)), "rptq_cluster_gemm")


def dequant_gemm(layout_in: Layout, a_codes, M: int, w_codes, s_w, N: int, y, *, ld_w: Optional[int] = None, bias=None,
                 act: int = ACT_NONE, y_dtype: int = OUT_F32, ldy: Optional[int] = None, stream=None) -> None:
    """rptq_dequant_gemm on device tensors (the Appendix's first method as a bfloat16 product)."""
    ld_w = int(s_w.shape[0]) if ld_w is None else int(ld_w)
    ldy = int(y.stride(0)) if ldy is None else int(ldy)
    _check(_lib.rptq_dequant_gemm(layout_in.handle, _dev_ptr(a_codes), int(M), _dev_ptr(w_codes), _dev_ptr(s_w), ld_w,
                                  _dev_ptr(bias), int(N), int(act), _dev_ptr(y), int(y_dtype), int(ldy), _stream_ptr(stream)),
           "rptq_dequant_gemm")


def weight_pack_clustered(layout_in: Layout, W: np.ndarray, n_pad: Optional[int] = None):
    """rptq_weight_pack_clustered on host arrays. Returns (w_codes flat uint8 tile-major buffer,
    s_w fp32 [g][N_pad], z_w int32 [g][N_pad], wsum int32 [g][N_pad])."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    N, Cn = W.shape
    if Cn != layout_in.C:
        raise ValueError("W must be [N][C] with C the layout's channel count")
    n_pad = N if n_pad is None else int(n_pad)
    w_codes = np.empty(weight_codes_bytes(layout_in.K_pad, n_pad), np.uint8)
    s_w = np.empty((layout_in.g, n_pad), np.float32)
    z_w = np.empty((layout_in.g, n_pad), np.int32)
    wsum = np.empty((layout_in.g, n_pad), np.int32)
    _check(_lib.rptq_weight_pack_clustered(layout_in.handle, _np_ptr(W), N, n_pad, _np_ptr(w_codes), _np_ptr(s_w),
                                           _np_ptr(z_w), _np_ptr(wsum)), "rptq_weight_pack_clustered")
    return w_codes, s_w, z_w, wsum


def code_rowsums(layout: Layout, codes, M: int, xsum, stream=None) -> None:
    """rptq_code_rowsums: xsum int32 [M][g] device tensor."""
    _check(_lib.rptq_code_rowsums(layout.handle, _dev_ptr(codes), int(M), _dev_ptr(xsum), _stream_ptr(stream)), "rptq_code_rowsums")


def cluster_gemm_clustered(layout_in: Layout, a_codes, M: int, xsum, w_codes, s_w, z_w, wsum, N: int, y, *,
                           bias=None, act: int = ACT_NONE, layout_out: Optional[Layout] = None, y_dtype: int = OUT_F32,
                           ldy: Optional[int] = None, stream=None) -> None:
    """rptq_cluster_gemm_clustered on device tensors (s_w, z_w, wsum are [g][N_pad])."""
    ld_w = int(s_w.shape[1])
    if ldy is None:
        ldy = 0 if y_dtype == OUT_CODES else int(y.stride(0))
    _check(_lib.rptq_cluster_gemm_clustered(layout_in.handle, _dev_ptr(a_codes), int(M), _dev_ptr(xsum), _dev_ptr(w_codes),
                                            _dev_ptr(s_w), _dev_ptr(z_w), _dev_ptr(wsum), ld_w, _dev_ptr(bias), int(N), int(act),
                                            None if layout_out is None else layout_out.handle, _dev_ptr(y), int(y_dtype),
                                            int(ldy), _stream_ptr(stream)), "rptq_cluster_gemm_clustered")


def cluster_gemm_noalloc(layout_in: Layout, a_codes, M: int, w_codes, s_w, wsum, N: int, y, *, ld_w: Optional[int] = None,
                         bias=None, act: int = ACT_NONE, layout_out: Optional[Layout] = None, y_dtype: int = OUT_F32,
                         ldy: Optional[int] = None, stream=None) -> None:
    """rptq_cluster_gemm_noalloc: same arguments and results as cluster_gemm, for callers that must
    not allocate device memory (the library keeps its per-column scratch in a static device array;
    N is limited to NOALLOC_MAX_N; calls that may overlap on the GPU must be serialised)."""
    ld_w = int(s_w.shape[0]) if ld_w is None else int(ld_w)
    if ldy is None:
        ldy = 0 if y_dtype == OUT_CODES else int(y.stride(0))
    _check(_lib.rptq_cluster_gemm_noalloc(layout_in.handle, _dev_ptr(a_codes), int(M), _dev_ptr(w_codes), _dev_ptr(s_w),
                                          _dev_ptr(wsum), ld_w, _dev_ptr(bias), int(N), int(act),
                                          None if layout_out is None else layout_out.handle, _dev_ptr(y), int(y_dtype),
                                          int(ldy), _stream_ptr(stream)), "rptq_cluster_gemm_noalloc")


def cluster_gemm_debug_acc(layout_in: Layout, a_codes, M: int, w_codes, N: int, m0: int, m1: int, n0: int, n1: int,
                           acc, stream=None) -> None:
    _check(_lib.rptq_cluster_gemm_debug_acc(layout_in.handle, _dev_ptr(a_codes), int(M), _dev_ptr(w_codes), int(N),
                                            int(m0), int(m1), int(n0), int(n1), _dev_ptr(acc), _stream_ptr(stream)),
           "rptq_cluster_gemm_debug_acc")


def codes_unpack_host(packed: np.ndarray, k_pad: int, bits: int) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    M = packed.shape[0]
    out = np.empty((M, k_pad), np.uint8)
    _check(_lib.rptq_codes_unpack_host(int(k_pad), int(bits), _np_ptr(packed), M, _np_ptr(out)), "rptq_codes_unpack_host")
    return out


def codes_pack_host(codes: np.ndarray, bits: int) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    M, k_pad = codes.shape
    out = np.empty((M, k_pad * bits // 8), np.uint8)
    _check(_lib.rptq_codes_pack_host(int(k_pad), int(bits), _np_ptr(codes), M, _np_ptr(out)), "rptq_codes_pack_host")
    return out


def weight_codes_bytes(k_pad: int, n_pad: int) -> int:
    return int(_lib.rptq_weight_codes_bytes(int(k_pad), int(n_pad)))


def weight_unpack_host(packed: np.ndarray, k_pad: int, n_rows: int) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint8).reshape(-1)
    N = int(n_rows)
    if packed.shape[0] < weight_codes_bytes(k_pad, N):
        raise ValueError("packed weight buffer too small")
    out = np.empty((N, k_pad), np.int8)
    _check(_lib.rptq_weight_unpack_host(int(k_pad), _np_ptr(packed), N, _np_ptr(out)), "rptq_weight_unpack_host")
    return out


def ln_channel_minmax(x, gamma, beta, eps: float, x_min, x_max, T: Optional[int] = None, stream=None) -> None:
    """rptq_ln_channel_minmax: x fp16 [T][ldx], gamma / beta fp16 [C], x_min / x_max fp32 [C] device tensors."""
    T = int(x.shape[0]) if T is None else int(T)
    _check(_lib.rptq_ln_channel_minmax(_dev_ptr(x), int(x.stride(0)), _dev_ptr(gamma), _dev_ptr(beta), C.c_float(eps), T,
                                       int(gamma.shape[0]), _dev_ptr(x_min), _dev_ptr(x_max), _stream_ptr(stream)),
           "rptq_ln_channel_minmax")


def kmeans(pts, g: int, u, iters: int, labels, centres, inertia, workspace, stream=None) -> None:
    """rptq_kmeans on device tensors: pts fp64 [n][dim], u fp64 [g], labels int32 [n], centres fp64 [g][dim],
    inertia fp64 [iters] or None, workspace uint8 of kmeans_workspace_bytes(n, g) bytes."""
    n, dim = int(pts.shape[0]), int(pts.shape[1])
    _check(_lib.rptq_kmeans(_dev_ptr(pts), n, dim, int(g), _dev_ptr(u), int(iters), _dev_ptr(labels), _dev_ptr(centres),
                            _dev_ptr(inertia), _dev_ptr(workspace), _stream_ptr(stream)), "rptq_kmeans")


def kmeans_workspace_bytes(n: int, g: int) -> int:
    return int(_lib.rptq_kmeans_workspace_bytes(int(n), int(g)))


def probe_int8_peak(n_batches: int, failed, stream=None) -> float:
    """rptq_probe_int8_peak: launches the operand-resident tcgen05.mma kind::i8 loop; returns the
    integer operations it performs. `failed` is a zeroed int32 device tensor of one element."""
    ops = C.c_double()
    _check(_lib.rptq_probe_int8_peak(int(n_batches), _dev_ptr(failed), C.byref(ops), _stream_ptr(stream)), "rptq_probe_int8_peak")
    return float(ops.value)


def get_device_status() -> int:
    s = C.c_int()
    _check(_lib.rptq_get_device_status(C.byref(s)), "rptq_get_device_status")
    return int(s.value)
