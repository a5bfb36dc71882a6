"""ctypes front end of the CPU oracle (``nq_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the
CPU-baseline leg of the benchmark.  The CUDA package never imports this module and
this module never imports the CUDA package.

Every function takes and returns numpy arrays; unpacked weights are ``int8`` in
the paper's value ranges, packed tensors are ``uint8`` byte arrays (sliced layout)
or ``uint64`` words (the paper's packed-bit tensor).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "nq_oracle.c"
_LIB = _HERE / "libnq_oracle.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc.  No fast-math, no FMA contraction: every fp32
    operation in the dequantisation rounds once, as the definition says."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        cmd = ["gcc", "-std=c99", "-O2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
               "-fPIC", "-shared", "-o", str(_LIB), str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(str(_LIB))
        _lib.nqo_sliced_row_bytes.restype = ctypes.c_int64
        _lib.nqo_word64_row_words.restype = ctypes.c_int64
        _lib.nqo_word64_fields_per_word.restype = ctypes.c_int64
        _lib.nqo_conv_out_dim.restype = ctypes.c_int64
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _i64(v):
    return ctypes.c_int64(int(v))


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def num_threads() -> int:
    return int(_load().nqo_num_threads())


# --------------------------------------------------------------------------- O1-O3
def decompose(w_int, mask, n_bits: int, h_bits: int, compensate: bool = True):
    """Eq. 5 / Eq. 6 / Eq. 10 and the compensation subsection: returns (w_high, w_low)."""
    w = _c(w_int, np.int8)
    m = _c(mask, np.uint8)
    assert w.shape == m.shape
    wh = np.empty_like(w)
    wl = np.empty_like(w)
    rc = _load().nqo_decompose(_p(w), _p(m), _i64(w.size), n_bits, h_bits, int(bool(compensate)),
                               _p(wh), _p(wl))
    if rc != 0:
        raise ValueError(f"unsupported nesting INT({n_bits}|{h_bits})")
    return wh, wl


def mask_rtn(w_int, n_bits: int, h_bits: int):
    w = _c(w_int, np.int8)
    m = np.empty(w.shape, dtype=np.uint8)
    rc = _load().nqo_mask_rtn(_p(w), _i64(w.size), n_bits, h_bits, _p(m))
    if rc != 0:
        raise ValueError("unsupported nesting")
    return m


def recompose(w_high, w_low, n_bits: int, h_bits: int):
    """Eq. 5: w_high * 2^l + w_low, clipped to INTn."""
    wh = _c(w_high, np.int8)
    wl = _c(w_low, np.int8)
    out = np.empty_like(wh)
    rc = _load().nqo_recompose(_p(wh), _p(wl), _i64(wh.size), n_bits, h_bits, _p(out))
    if rc != 0:
        raise ValueError("unsupported nesting")
    return out


def drop_low(w_int, w_low, n_bits: int, h_bits: int):
    """Downgrade: (w_int - w_low) / 2^l."""
    w = _c(w_int, np.int8)
    wl = _c(w_low, np.int8)
    out = np.empty_like(w)
    rc = _load().nqo_drop_low(_p(w), _p(wl), _i64(w.size), n_bits, h_bits, _p(out))
    if rc != 0:
        raise ValueError("unsupported nesting")
    return out


# --------------------------------------------------------------------------- O4
def word64_fields_per_word(bits: int) -> int:
    return int(_load().nqo_word64_fields_per_word(bits))


def word64_row_words(cols: int, bits: int) -> int:
    return int(_load().nqo_word64_row_words(_i64(cols), bits))


def pack_word64(v, bits: int):
    v = _c(v, np.int8)
    rows, cols = v.shape
    out = np.empty((rows, word64_row_words(cols, bits)), dtype=np.uint64)
    _load().nqo_pack_word64(_p(v), _i64(rows), _i64(cols), bits, _p(out))
    return out


def unpack_word64(words, cols: int, bits: int):
    words = _c(words, np.uint64)
    rows = words.shape[0]
    out = np.empty((rows, cols), dtype=np.int8)
    _load().nqo_unpack_word64(_p(words), _i64(rows), _i64(cols), bits, _p(out))
    return out


def sliced_row_bytes(cols: int, bits: int) -> int:
    """Bytes per row of a packed tensor (a size unit: the tensor is stored in 128 x 128 blocks)."""
    return int(_load().nqo_sliced_row_bytes(_i64(cols), bits))


def sliced_padded_rows(rows: int) -> int:
    return -(-int(rows) // 128) * 128


def pack_sliced(v, bits: int):
    """-> uint8 [rows padded to 128, sliced_row_bytes(cols, bits)]: the packed tensor's bytes in storage order."""
    v = _c(v, np.int8)
    rows, cols = v.shape
    out = np.empty((sliced_padded_rows(rows), sliced_row_bytes(cols, bits)), dtype=np.uint8)
    rc = _load().nqo_pack_sliced(_p(v), _i64(rows), _i64(cols), bits, _p(out))
    if rc != 0:
        raise ValueError("unsupported field width")
    return out


def unpack_sliced(packed, rows: int, cols: int, bits: int):
    packed = _c(packed, np.uint8)
    assert packed.size == sliced_padded_rows(rows) * sliced_row_bytes(cols, bits)
    out = np.empty((rows, cols), dtype=np.int8)
    rc = _load().nqo_unpack_sliced(_p(packed), _i64(rows), _i64(cols), bits, _p(out))
    if rc != 0:
        raise ValueError("unsupported field width")
    return out


# --------------------------------------------------------------------------- O5-O7
def gemm_acc(x, w):
    """acc[m, j] = sum_k x[m, k] * w[j, k] in int32."""
    x = _c(x, np.int8)
    w = _c(w, np.int8)
    M, K = x.shape
    N, K2 = w.shape
    assert K == K2
    acc = np.empty((M, N), dtype=np.int32)
    _load().nqo_gemm_acc(_p(x), _i64(K), _p(w), _i64(K), _i64(M), _i64(N), _i64(K), _p(acc), _i64(N))
    return acc


def dequant(acc, w_scale, act_scale: float, l_shift: int = 0, bias=None, want_ref: bool = False):
    """fp32 output of Eq. 2 (l_shift = 0) or Eq. 9 (l_shift = l); optionally the fp64 value too."""
    acc = _c(acc, np.int32)
    lead = acc.shape[:-1]
    N = acc.shape[-1]
    acc2 = acc.reshape(-1, N)
    M = acc2.shape[0]
    ws = _c(w_scale, np.float32)
    assert ws.shape == (N,)
    b = None if bias is None else _c(bias, np.float32)
    y = np.empty((M, N), dtype=np.float32)
    yref = np.empty((M, N), dtype=np.float64) if want_ref else None
    _load().nqo_dequant(_p(acc2), _i64(N), _i64(M), _i64(N), _p(ws), ctypes.c_float(act_scale),
                        int(l_shift), None if b is None else _p(b), _p(y), _i64(N),
                        None if yref is None else _p(yref))
    y = y.reshape(*lead, N)
    if want_ref:
        return y, yref.reshape(*lead, N)
    return y


def requant(acc, w_scale, act_scale: float, l_shift: int, out_scale: float, bias=None, relu: bool = True):
    """INT8 activations for the next layer from a layer's accumulators (the library's own definition, fp32)."""
    acc = _c(acc, np.int32)
    lead = acc.shape[:-1]
    N = acc.shape[-1]
    acc2 = acc.reshape(-1, N)
    M = acc2.shape[0]
    ws = _c(w_scale, np.float32)
    assert ws.shape == (N,)
    b = None if bias is None else _c(bias, np.float32)
    q = np.empty((M, N), dtype=np.int8)
    _load().nqo_requant(_p(acc2), _i64(N), _i64(M), _i64(N), _p(ws), ctypes.c_float(act_scale), int(l_shift),
                        None if b is None else _p(b), int(bool(relu)), ctypes.c_float(out_scale), _p(q), _i64(N))
    return q.reshape(*lead, N)


def requant_res(acc, w_scale, act_scale: float, l_shift: int, out_scale: float, res, res_scale: float, bias=None,
                relu: bool = True):
    """requant with a residual connection: the INT8 skip tensor `res` (same shape as acc, scale res_scale) is added,
    dequantised, before the activation (the library's own definition, fp32)."""
    acc = _c(acc, np.int32)
    lead = acc.shape[:-1]
    N = acc.shape[-1]
    acc2 = acc.reshape(-1, N)
    M = acc2.shape[0]
    r = _c(res, np.int8).reshape(-1, N)
    assert r.shape == acc2.shape
    ws = _c(w_scale, np.float32)
    assert ws.shape == (N,)
    b = None if bias is None else _c(bias, np.float32)
    q = np.empty((M, N), dtype=np.int8)
    _load().nqo_requant_res(_p(acc2), _i64(N), _i64(M), _i64(N), _p(ws), ctypes.c_float(act_scale), int(l_shift),
                            None if b is None else _p(b), _p(r), _i64(N), ctypes.c_float(res_scale), int(bool(relu)),
                            ctypes.c_float(out_scale), _p(q), _i64(N))
    return q.reshape(*lead, N)


def maxpool_nhwc(x, ksize: int, stride: int, pad: int):
    """Integer max pooling of INT8 NHWC activations; padding never wins."""
    x = _c(x, np.int8)
    B, H, W, C = x.shape
    Ho, Wo = (H + 2 * pad - ksize) // stride + 1, (W + 2 * pad - ksize) // stride + 1
    y = np.empty((B, Ho, Wo, C), dtype=np.int8)
    _load().nqo_maxpool_nhwc(_p(x), _i64(B), _i64(H), _i64(W), _i64(C), _i64(ksize), _i64(stride), _i64(pad), _p(y))
    return y


def avgpool_requant_nhwc(x, in_scale: float, out_scale: float):
    """Global average pooling of INT8 NHWC activations, requantised to INT8 [B, C]."""
    x = _c(x, np.int8)
    B, H, W, C = x.shape
    y = np.empty((B, C), dtype=np.int8)
    _load().nqo_avgpool_requant_nhwc(_p(x), _i64(B), _i64(H), _i64(W), _i64(C), ctypes.c_float(in_scale),
                                     ctypes.c_float(out_scale), _p(y))
    return y


def f32_to_bf16_bits(x):
    x = _c(x, np.float32)
    out = np.empty(x.shape, dtype=np.uint16)
    _load().nqo_f32_to_bf16(_p(x), _i64(x.size), _p(out))
    return out


def conv_out_dim(size: int, ksize: int, stride: int, pad: int) -> int:
    return int(_load().nqo_conv_out_dim(_i64(size), _i64(ksize), _i64(stride), _i64(pad)))


def conv_acc(x_nchw, w_oihw, stride: int, pad: int):
    x = _c(x_nchw, np.int8)
    w = _c(w_oihw, np.int8)
    B, C, H, W = x.shape
    Cout, C2, R, S = w.shape
    assert C == C2
    Ho, Wo = conv_out_dim(H, R, stride, pad), conv_out_dim(W, S, stride, pad)
    acc = np.empty((B, Cout, Ho, Wo), dtype=np.int32)
    _load().nqo_conv_acc(_p(x), _i64(B), _i64(C), _i64(H), _i64(W), _p(w), _i64(Cout), _i64(R),
                         _i64(S), _i64(stride), _i64(pad), _p(acc))
    return acc


def conv_acc_pixels(x_nchw, w_oihw, stride: int, pad: int, pixels):
    """The convolution at listed output pixels (b, p, q): returns int32 [npix, Cout]."""
    x = _c(x_nchw, np.int8)
    w = _c(w_oihw, np.int8)
    pix = _c(pixels, np.int64).reshape(-1, 3)
    B, C, H, W = x.shape
    Cout, C2, R, S = w.shape
    assert C == C2
    out = np.empty((pix.shape[0], Cout), dtype=np.int32)
    _load().nqo_conv_acc_pixels(_p(x), _i64(B), _i64(C), _i64(H), _i64(W), _p(w), _i64(Cout),
                                _i64(R), _i64(S), _i64(stride), _i64(pad), _p(pix),
                                _i64(pix.shape[0]), _p(out))
    return out
