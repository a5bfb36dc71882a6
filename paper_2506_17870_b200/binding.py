"""ctypes binding of ``libnq_b200.so``: argument marshalling only.

Each ``nq_*`` function below has the name of the C entry point it calls (``include/nq.h``); it
takes torch CUDA tensors, checks their dtype / device, allocates the outputs through torch and passes
raw device pointers plus the current torch stream to the library.  No step of the computation runs
here, and there is no fallback: if the shared library cannot be loaded the import of a function
raises ``NqLibraryError``.
"""
from __future__ import annotations

import ctypes
from pathlib import Path
from typing import Optional, Sequence

import torch

_PKG = Path(__file__).resolve().parent
_LIB_PATH = _PKG / "libnq_b200.so"
_lib = None

NQ_OK = 0
NQ_F32, NQ_BF16 = 0, 1

EXPORTS = (
    "nq_status_str", "nq_low_bits", "nq_packed_row_bytes", "nq_packed_bytes",
    "nq_decompose", "nq_recompose", "nq_drop_low", "nq_unpack", "nq_pack",
    "nq_word64_row_words", "nq_word64_to_sliced", "nq_sliced_to_word64", "nq_rounding_mask",
    "nq_batch_table_bytes", "nq_batch_plan", "nq_recompose_batched", "nq_drop_low_batched",
    "nq_gemm_full", "nq_gemm_part", "nq_conv_workspace_bytes", "nq_conv_implicit_gemm",
    "nq_conv_implicit_gemm_static",
    "nq_gemm_full_q8", "nq_gemm_part_q8", "nq_conv_implicit_gemm_q8", "nq_gemm_nested", "nq_conv_implicit_gemm_nested", "nq_gemm_nested_q8",
    "nq_conv_implicit_gemm_nested_q8",
    "nq_i8_mma_ceiling", "nq_debug_set",
    "nq_conv_implicit_gemm_q8_res", "nq_conv_implicit_gemm_nested_q8_res", "nq_maxpool_nhwc_i8", "nq_avgpool_requant_nhwc_i8",
    "nq_device_status",
)


class NqLibraryError(RuntimeError):
    pass


class NqError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {status_str(status)} (nq_status {status})")


class nq_tensor_desc(ctypes.Structure):
    _fields_ = [("rows", ctypes.c_int64), ("cols", ctypes.c_int64), ("ld", ctypes.c_int64),
                ("packed_high", ctypes.c_void_p), ("packed_low", ctypes.c_void_p), ("w_int", ctypes.c_void_p)]


class nq_conv_desc(ctypes.Structure):
    _fields_ = [(k, ctypes.c_int32) for k in
                ("B", "Cin", "H", "W", "Cout", "R", "S", "stride", "pad", "x_nchw")]


def lib() -> ctypes.CDLL:
    """The loaded C library.  Raises NqLibraryError when it has not been built."""
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise NqLibraryError(
                f"{_LIB_PATH} is missing: build it with `python -m paper_2506_17870_b200.build` "
                "(needs nvcc); there is no CPU fallback")
        try:
            L = ctypes.CDLL(str(_LIB_PATH))
        except OSError as e:  # pragma: no cover
            raise NqLibraryError(f"cannot load {_LIB_PATH}: {e}") from e
        L.nq_status_str.restype = ctypes.c_char_p
        for name in ("nq_packed_row_bytes", "nq_packed_bytes", "nq_batch_table_bytes", "nq_conv_workspace_bytes",
                     "nq_word64_row_words"):
            getattr(L, name).restype = ctypes.c_int64
        _lib = L
    return _lib


def status_str(status: int) -> str:
    return lib().nq_status_str(int(status)).decode()


def _check(status: int, what: str):
    if status != NQ_OK:
        raise NqError(status, what)


def _ptr(t: Optional[torch.Tensor]):
    return ctypes.c_void_p(0 if t is None else t.data_ptr())


def _i64(v):
    return ctypes.c_int64(int(v))


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _need(t: torch.Tensor, dtype, name: str, ndim: Optional[int] = None):
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype:
        raise ValueError(f"{name} must be {dtype}, got {t.dtype}")
    if ndim is not None and t.dim() != ndim:
        raise ValueError(f"{name} must have {ndim} dimensions")
    if t.dim() >= 1 and t.stride(-1) != 1 and t.numel() > 0:
        raise ValueError(f"{name} must be contiguous in its last dimension")


def _ld(t: torch.Tensor) -> int:
    return t.stride(0) if t.dim() == 2 and t.shape[0] > 1 else max(t.shape[-1], 1)


# --------------------------------------------------------------------------- sizes (host, pure)
def nq_low_bits(n_bits: int, h_bits: int, compensate: bool = True) -> int:
    return int(lib().nq_low_bits(n_bits, h_bits, int(bool(compensate))))


def nq_packed_row_bytes(cols: int, bits: int) -> int:
    return int(lib().nq_packed_row_bytes(_i64(cols), bits))


def nq_packed_bytes(rows: int, cols: int, bits: int) -> int:
    return int(lib().nq_packed_bytes(_i64(rows), _i64(cols), bits))


def _empty_packed(rows: int, cols: int, bits: int, device) -> torch.Tensor:
    """Storage of a packed tensor: nq_packed_bytes(rows, cols, bits) bytes, shaped [rows padded to 128, bytes per row]
    (a container only: the layout stores 128 x 128 blocks, a row's bytes are not contiguous)."""
    return torch.empty((-(-rows // 128) * 128, max(nq_packed_row_bytes(cols, bits), 0)), dtype=torch.uint8, device=device)


# --------------------------------------------------------------------------- codec
def nq_decompose(w_int: torch.Tensor, mask: torch.Tensor, n_bits: int, h_bits: int, compensate: bool = True,
                 out_high: Optional[torch.Tensor] = None, out_low: Optional[torch.Tensor] = None):
    """-> (packed_high, packed_low): uint8 storage of the two sliced tensors."""
    _need(w_int, torch.int8, "w_int", 2)
    _need(mask, torch.uint8, "mask", 2)
    if mask.shape != w_int.shape or _ld(mask) != _ld(w_int):
        raise ValueError("mask must have the shape and row pitch of w_int")
    rows, cols = w_int.shape
    lb = nq_low_bits(n_bits, h_bits, compensate)
    if lb < 0:
        raise NqError(2, "nq_decompose")
    hi = out_high if out_high is not None else _empty_packed(rows, cols, h_bits, w_int.device)
    lo = out_low if out_low is not None else _empty_packed(rows, cols, lb, w_int.device)
    _check(lib().nq_decompose(_ptr(w_int), _ptr(mask), _i64(rows), _i64(cols), _i64(_ld(w_int)), n_bits, h_bits,
                              int(bool(compensate)), _ptr(hi), _ptr(lo), _stream()), "nq_decompose")
    return hi, lo


def nq_recompose(packed_high: torch.Tensor, packed_low: torch.Tensor, rows: int, cols: int, n_bits: int, h_bits: int,
                 compensate: bool = True, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    _need(packed_high, torch.uint8, "packed_high")
    _need(packed_low, torch.uint8, "packed_low")
    if out is None:
        out = torch.empty((rows, cols), dtype=torch.int8, device=packed_high.device)
    _need(out, torch.int8, "out", 2)
    _check(lib().nq_recompose(_ptr(packed_high), _ptr(packed_low), _i64(rows), _i64(cols), n_bits, h_bits,
                              int(bool(compensate)), _ptr(out), _i64(_ld(out)), _stream()), "nq_recompose")
    return out


def nq_drop_low(w_int: torch.Tensor, packed_low: torch.Tensor, n_bits: int, h_bits: int, compensate: bool = True,
                out_high: Optional[torch.Tensor] = None) -> torch.Tensor:
    _need(w_int, torch.int8, "w_int", 2)
    _need(packed_low, torch.uint8, "packed_low")
    rows, cols = w_int.shape
    hi = out_high if out_high is not None else _empty_packed(rows, cols, h_bits, w_int.device)
    _check(lib().nq_drop_low(_ptr(w_int), _i64(_ld(w_int)), _ptr(packed_low), _i64(rows), _i64(cols), n_bits, h_bits,
                             int(bool(compensate)), _ptr(hi), _stream()), "nq_drop_low")
    return hi


def nq_unpack(packed: torch.Tensor, bits: int, rows: int, cols: int, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    _need(packed, torch.uint8, "packed")
    if out is None:
        out = torch.empty((rows, cols), dtype=torch.int8, device=packed.device)
    _check(lib().nq_unpack(_ptr(packed), bits, _i64(rows), _i64(cols), _ptr(out), _i64(_ld(out)), _stream()),
           "nq_unpack")
    return out


def nq_pack(values: torch.Tensor, bits: int) -> torch.Tensor:
    _need(values, torch.int8, "values", 2)
    rows, cols = values.shape
    out = _empty_packed(rows, cols, bits, values.device)
    _check(lib().nq_pack(_ptr(values), _i64(_ld(values)), bits, _i64(rows), _i64(cols), _ptr(out), _stream()),
           "nq_pack")
    return out


NQ_ROUND_DOWN, NQ_ROUND_UP, NQ_ROUND_NEAREST = 0, 1, 2


def nq_rounding_mask(w_int: torch.Tensor, n_bits: int, h_bits: int, mode: int) -> torch.Tensor:
    """Rounding mask (uint8 0 / 1, same shape and pitch as w_int) of one of the baseline roundings."""
    _need(w_int, torch.int8, "w_int", 2)
    rows, cols = w_int.shape
    ld = _ld(w_int)
    buf = torch.empty((rows, ld), dtype=torch.uint8, device=w_int.device)
    _check(lib().nq_rounding_mask(_ptr(w_int), _i64(ld), _i64(rows), _i64(cols), n_bits, h_bits, int(mode), _ptr(buf),
                                  _i64(ld), _stream()), "nq_rounding_mask")
    return buf[:, :cols]


def nq_word64_row_words(cols: int, bits: int) -> int:
    return int(lib().nq_word64_row_words(_i64(cols), bits))


def nq_word64_to_sliced(words: torch.Tensor, bits: int, cols: int) -> torch.Tensor:
    """[rows, nq_word64_row_words(cols, bits)] int64 words (the paper's packed-bit tensor) -> sliced tensor."""
    _need(words, torch.int64, "words", 2)
    rows = words.shape[0]
    if not words.is_contiguous() or words.shape[1] != nq_word64_row_words(cols, bits):
        raise ValueError("words must be a dense [rows, nq_word64_row_words(cols, bits)] tensor")
    out = _empty_packed(rows, cols, bits, words.device)
    _check(lib().nq_word64_to_sliced(_ptr(words), bits, _i64(rows), _i64(cols), _ptr(out), _stream()), "nq_word64_to_sliced")
    return out


def nq_sliced_to_word64(packed: torch.Tensor, bits: int, rows: int, cols: int) -> torch.Tensor:
    """Sliced tensor -> [rows, nq_word64_row_words(cols, bits)] int64 words."""
    _need(packed, torch.uint8, "packed")
    if packed.numel() != nq_packed_bytes(rows, cols, bits):
        raise ValueError("packed has the wrong size for (rows, cols, bits)")
    out = torch.empty((rows, nq_word64_row_words(cols, bits)), dtype=torch.int64, device=packed.device)
    _check(lib().nq_sliced_to_word64(_ptr(packed), bits, _i64(rows), _i64(cols), _ptr(out), _stream()), "nq_sliced_to_word64")
    return out


class BatchPlan:
    """Device table of a model's tensors (nq_batch_plan) plus the work-item count the batched calls need."""

    def __init__(self, table: torch.Tensor, count: int, total_units: int, keep: Sequence[torch.Tensor]):
        self.table, self.count, self.total_units, self._keep = table, count, total_units, list(keep)


def nq_batch_plan(tensors: Sequence[dict]) -> BatchPlan:
    """tensors: dicts with 'w_int' (int8 [rows, cols]), 'packed_high', 'packed_low' (uint8)."""
    count = len(tensors)
    arr = (nq_tensor_desc * max(count, 1))()
    keep = []
    device = tensors[0]["w_int"].device if count else torch.device("cuda")
    for i, t in enumerate(tensors):
        w = t["w_int"]
        _need(w, torch.int8, "w_int", 2)
        _need(t["packed_high"], torch.uint8, "packed_high")
        _need(t["packed_low"], torch.uint8, "packed_low")
        arr[i] = nq_tensor_desc(w.shape[0], w.shape[1], _ld(w), t["packed_high"].data_ptr(),
                                t["packed_low"].data_ptr(), w.data_ptr())
        keep += [w, t["packed_high"], t["packed_low"]]
    nbytes = int(lib().nq_batch_table_bytes(arr, count))
    table = torch.empty(nbytes, dtype=torch.uint8, device=device)
    total = ctypes.c_int64(0)
    _check(lib().nq_batch_plan(arr, count, _ptr(table), _i64(nbytes), ctypes.byref(total), _stream()), "nq_batch_plan")
    return BatchPlan(table, count, total.value, keep)


def nq_recompose_batched(plan: BatchPlan, n_bits: int, h_bits: int, compensate: bool = True):
    _check(lib().nq_recompose_batched(_ptr(plan.table), plan.count, _i64(plan.total_units), n_bits, h_bits,
                                      int(bool(compensate)), _stream()), "nq_recompose_batched")


def nq_drop_low_batched(plan: BatchPlan, n_bits: int, h_bits: int, compensate: bool = True):
    _check(lib().nq_drop_low_batched(_ptr(plan.table), plan.count, _i64(plan.total_units), n_bits, h_bits,
                                     int(bool(compensate)), _stream()), "nq_drop_low_batched")


# --------------------------------------------------------------------------- GEMM
def _y_dtype(dtype) -> int:
    if dtype == torch.float32:
        return NQ_F32
    if dtype == torch.bfloat16:
        return NQ_BF16
    raise ValueError("output dtype must be float32 or bfloat16")


def _gemm_outputs(M, N, device, want_acc, y_dtype, acc_out, y_out):
    acc = acc_out if acc_out is not None else (torch.empty((M, N), dtype=torch.int32, device=device) if want_acc else None)
    y = y_out if y_out is not None else (torch.empty((M, N), dtype=y_dtype, device=device) if y_dtype is not None else None)
    return acc, y


def nq_gemm_full(X: torch.Tensor, W: torch.Tensor, w_scale: torch.Tensor, act_scale: float,
                 bias: Optional[torch.Tensor] = None, want_acc: bool = False, y_dtype=torch.float32,
                 acc_out: Optional[torch.Tensor] = None, y_out: Optional[torch.Tensor] = None):
    """-> (acc int32 [M, N] or None, Y [M, N] or None)."""
    _need(X, torch.int8, "X", 2)
    _need(W, torch.int8, "W", 2)
    _need(w_scale, torch.float32, "w_scale", 1)
    M, K = X.shape
    N = W.shape[0]
    if W.shape[1] != K or w_scale.shape[0] != N:
        raise ValueError("shape mismatch")
    acc, y = _gemm_outputs(M, N, X.device, want_acc, y_dtype, acc_out, y_out)
    _check(lib().nq_gemm_full(_ptr(X), _i64(_ld(X)), _ptr(W), _i64(_ld(W)), _ptr(w_scale), ctypes.c_float(act_scale),
                              _ptr(bias), _i64(M), _i64(N), _i64(K), _ptr(acc), _i64(_ld(acc) if acc is not None else 0),
                              _ptr(y), _i64(_ld(y) if y is not None else 0),
                              _y_dtype(y.dtype) if y is not None else NQ_F32, _stream()), "nq_gemm_full")
    return acc, y


def nq_gemm_part(X: torch.Tensor, packed_high: torch.Tensor, N: int, n_bits: int, h_bits: int, w_scale: torch.Tensor,
                 act_scale: float, bias: Optional[torch.Tensor] = None, want_acc: bool = False,
                 y_dtype=torch.float32, acc_out: Optional[torch.Tensor] = None, y_out: Optional[torch.Tensor] = None):
    _need(X, torch.int8, "X", 2)
    _need(packed_high, torch.uint8, "packed_high")
    _need(w_scale, torch.float32, "w_scale", 1)
    M, K = X.shape
    acc, y = _gemm_outputs(M, N, X.device, want_acc, y_dtype, acc_out, y_out)
    _check(lib().nq_gemm_part(_ptr(X), _i64(_ld(X)), _ptr(packed_high), n_bits, h_bits, _ptr(w_scale),
                              ctypes.c_float(act_scale), _ptr(bias), _i64(M), _i64(N), _i64(K), _ptr(acc),
                              _i64(_ld(acc) if acc is not None else 0), _ptr(y), _i64(_ld(y) if y is not None else 0),
                              _y_dtype(y.dtype) if y is not None else NQ_F32, _stream()), "nq_gemm_part")
    return acc, y


def nq_gemm_nested(X: torch.Tensor, packed_high: torch.Tensor, packed_low: torch.Tensor, N: int, n_bits: int,
                   h_bits: int, w_scale: torch.Tensor, act_scale: float, bias: Optional[torch.Tensor] = None,
                   want_acc: bool = False, y_dtype=torch.float32, acc_out: Optional[torch.Tensor] = None,
                   y_out: Optional[torch.Tensor] = None):
    """Full-bit layer computed from the packed higher-bit and compensated lower-bit tensors (no INT8 copy)."""
    _need(X, torch.int8, "X", 2)
    _need(packed_high, torch.uint8, "packed_high")
    _need(packed_low, torch.uint8, "packed_low")
    _need(w_scale, torch.float32, "w_scale", 1)
    M, K = X.shape
    acc, y = _gemm_outputs(M, N, X.device, want_acc, y_dtype, acc_out, y_out)
    _check(lib().nq_gemm_nested(_ptr(X), _i64(_ld(X)), _ptr(packed_high), _ptr(packed_low), n_bits, h_bits,
                                _ptr(w_scale), ctypes.c_float(act_scale), _ptr(bias), _i64(M), _i64(N), _i64(K),
                                _ptr(acc), _i64(_ld(acc) if acc is not None else 0), _ptr(y),
                                _i64(_ld(y) if y is not None else 0),
                                _y_dtype(y.dtype) if y is not None else NQ_F32, _stream()), "nq_gemm_nested")
    return acc, y


# --------------------------------------------------------------------------- convolution
def nq_gemm_full_q8(X: torch.Tensor, W: torch.Tensor, w_scale: torch.Tensor, act_scale: float, out_scale: float,
                    relu: bool = True, bias: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Full-bit layer whose output is the next layer's INT8 activations."""
    _need(X, torch.int8, "X", 2); _need(W, torch.int8, "W", 2); _need(w_scale, torch.float32, "w_scale", 1)
    M, K = X.shape
    N = W.shape[0]
    y = torch.empty((M, N), dtype=torch.int8, device=X.device)
    _check(lib().nq_gemm_full_q8(_ptr(X), _i64(_ld(X)), _ptr(W), _i64(_ld(W)), _ptr(w_scale), ctypes.c_float(act_scale),
                                 _ptr(bias), ctypes.c_float(out_scale), int(bool(relu)), _i64(M), _i64(N), _i64(K),
                                 _ptr(y), _i64(N), _stream()), "nq_gemm_full_q8")
    return y


def nq_gemm_part_q8(X: torch.Tensor, packed_high: torch.Tensor, N: int, n_bits: int, h_bits: int, w_scale: torch.Tensor,
                    act_scale: float, out_scale: float, relu: bool = True, bias: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Part-bit layer whose output is the next layer's INT8 activations."""
    _need(X, torch.int8, "X", 2); _need(packed_high, torch.uint8, "packed_high"); _need(w_scale, torch.float32, "w_scale", 1)
    M, K = X.shape
    y = torch.empty((M, N), dtype=torch.int8, device=X.device)
    _check(lib().nq_gemm_part_q8(_ptr(X), _i64(_ld(X)), _ptr(packed_high), n_bits, h_bits, _ptr(w_scale),
                                 ctypes.c_float(act_scale), _ptr(bias), ctypes.c_float(out_scale), int(bool(relu)),
                                 _i64(M), _i64(N), _i64(K), _ptr(y), _i64(N), _stream()), "nq_gemm_part_q8")
    return y


def nq_conv_implicit_gemm_q8(X: torch.Tensor, Wt: torch.Tensor, desc: nq_conv_desc, w_scale: torch.Tensor, act_scale: float,
                             out_scale: float, relu: bool = True, part_bit: bool = False, n_bits: int = 8, h_bits: int = 6,
                             bias: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                             y_out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Convolution whose NHWC output is the next layer's INT8 activations."""
    Ho = (desc.H + 2 * desc.pad - desc.R) // desc.stride + 1
    Wo = (desc.W + 2 * desc.pad - desc.S) // desc.stride + 1
    need = nq_conv_workspace_bytes(desc)
    if workspace is None:
        workspace = torch.empty(max(need, 0) + 2048, dtype=torch.uint8, device=X.device)
    off = (-workspace.data_ptr()) % 1024
    y = y_out if y_out is not None else torch.empty((desc.B, Ho, Wo, desc.Cout), dtype=torch.int8, device=X.device)
    ldw = _ld(Wt) if not part_bit else 0
    _check(lib().nq_conv_implicit_gemm_q8(_ptr(X), _ptr(Wt), _i64(ldw), int(bool(part_bit)), n_bits, h_bits,
                                          ctypes.byref(desc), _ptr(w_scale), ctypes.c_float(act_scale), _ptr(bias),
                                          ctypes.c_float(out_scale), int(bool(relu)), _ptr(y),
                                          ctypes.c_void_p(workspace.data_ptr() + off), _i64(workspace.numel() - off),
                                          _stream()), "nq_conv_implicit_gemm_q8")
    return y


def nq_gemm_nested_q8(X: torch.Tensor, packed_high: torch.Tensor, packed_low: torch.Tensor, N: int, n_bits: int,
                      h_bits: int, w_scale: torch.Tensor, act_scale: float, out_scale: float, relu: bool = True,
                      bias: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Nested full-bit layer whose output is the next layer's INT8 activations."""
    _need(X, torch.int8, "X", 2); _need(packed_high, torch.uint8, "packed_high"); _need(packed_low, torch.uint8, "packed_low")
    _need(w_scale, torch.float32, "w_scale", 1)
    M, K = X.shape
    y = torch.empty((M, N), dtype=torch.int8, device=X.device)
    _check(lib().nq_gemm_nested_q8(_ptr(X), _i64(_ld(X)), _ptr(packed_high), _ptr(packed_low), n_bits, h_bits,
                                   _ptr(w_scale), ctypes.c_float(act_scale), _ptr(bias), ctypes.c_float(out_scale),
                                   int(bool(relu)), _i64(M), _i64(N), _i64(K), _ptr(y), _i64(N), _stream()),
           "nq_gemm_nested_q8")
    return y


def nq_conv_implicit_gemm_nested_q8(X: torch.Tensor, packed_high: torch.Tensor, packed_low: torch.Tensor,
                                    desc: nq_conv_desc, w_scale: torch.Tensor, act_scale: float, out_scale: float,
                                    relu: bool = True, n_bits: int = 8, h_bits: int = 6,
                                    bias: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                                    y_out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Nested full-bit convolution whose NHWC output is the next layer's INT8 activations."""
    Ho = (desc.H + 2 * desc.pad - desc.R) // desc.stride + 1
    Wo = (desc.W + 2 * desc.pad - desc.S) // desc.stride + 1
    need = nq_conv_workspace_bytes(desc)
    if workspace is None:
        workspace = torch.empty(max(need, 0) + 2048, dtype=torch.uint8, device=X.device)
    off = (-workspace.data_ptr()) % 1024
    y = y_out if y_out is not None else torch.empty((desc.B, Ho, Wo, desc.Cout), dtype=torch.int8, device=X.device)
    _check(lib().nq_conv_implicit_gemm_nested_q8(_ptr(X), _ptr(packed_high), _ptr(packed_low), n_bits, h_bits,
                                                 ctypes.byref(desc), _ptr(w_scale), ctypes.c_float(act_scale), _ptr(bias),
                                                 ctypes.c_float(out_scale), int(bool(relu)), _ptr(y),
                                                 ctypes.c_void_p(workspace.data_ptr() + off), _i64(workspace.numel() - off),
                                                 _stream()), "nq_conv_implicit_gemm_nested_q8")
    return y


def nq_conv_implicit_gemm_q8_res(X: torch.Tensor, Wt: torch.Tensor, desc: nq_conv_desc, w_scale: torch.Tensor, act_scale: float,
                                 residual: torch.Tensor, residual_scale: float, out_scale: float, relu: bool = True,
                                 part_bit: bool = False, n_bits: int = 8, h_bits: int = 6,
                                 bias: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                                 y_out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Requantising convolution with a residual connection: `residual` (int8, the output's NHWC shape, scale
    residual_scale) is added, dequantised, before the activation."""
    Ho = (desc.H + 2 * desc.pad - desc.R) // desc.stride + 1
    Wo = (desc.W + 2 * desc.pad - desc.S) // desc.stride + 1
    _need(residual, torch.int8, "residual")
    if tuple(residual.shape) != (desc.B, Ho, Wo, desc.Cout) or not residual.is_contiguous():
        raise ValueError("residual must be a dense NHWC tensor of the output's shape")
    need = nq_conv_workspace_bytes(desc)
    if workspace is None:
        workspace = torch.empty(max(need, 0) + 2048, dtype=torch.uint8, device=X.device)
    off = (-workspace.data_ptr()) % 1024
    y = y_out if y_out is not None else torch.empty((desc.B, Ho, Wo, desc.Cout), dtype=torch.int8, device=X.device)
    ldw = _ld(Wt) if not part_bit else 0
    _check(lib().nq_conv_implicit_gemm_q8_res(_ptr(X), _ptr(Wt), _i64(ldw), int(bool(part_bit)), n_bits, h_bits,
                                              ctypes.byref(desc), _ptr(w_scale), ctypes.c_float(act_scale), _ptr(bias),
                                              _ptr(residual), ctypes.c_float(residual_scale), ctypes.c_float(out_scale),
                                              int(bool(relu)), _ptr(y), ctypes.c_void_p(workspace.data_ptr() + off),
                                              _i64(workspace.numel() - off), _stream()), "nq_conv_implicit_gemm_q8_res")
    return y


def nq_conv_implicit_gemm_nested_q8_res(X: torch.Tensor, packed_high: torch.Tensor, packed_low: torch.Tensor,
                                        desc: nq_conv_desc, w_scale: torch.Tensor, act_scale: float,
                                        residual: torch.Tensor, residual_scale: float, out_scale: float,
                                        relu: bool = True, n_bits: int = 8, h_bits: int = 6,
                                        bias: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                                        y_out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """The same in nested full-bit mode (weights rebuilt from the two packed parts inside the kernel)."""
    Ho = (desc.H + 2 * desc.pad - desc.R) // desc.stride + 1
    Wo = (desc.W + 2 * desc.pad - desc.S) // desc.stride + 1
    _need(residual, torch.int8, "residual")
    if tuple(residual.shape) != (desc.B, Ho, Wo, desc.Cout) or not residual.is_contiguous():
        raise ValueError("residual must be a dense NHWC tensor of the output's shape")
    need = nq_conv_workspace_bytes(desc)
    if workspace is None:
        workspace = torch.empty(max(need, 0) + 2048, dtype=torch.uint8, device=X.device)
    off = (-workspace.data_ptr()) % 1024
    y = y_out if y_out is not None else torch.empty((desc.B, Ho, Wo, desc.Cout), dtype=torch.int8, device=X.device)
    _check(lib().nq_conv_implicit_gemm_nested_q8_res(_ptr(X), _ptr(packed_high), _ptr(packed_low), n_bits, h_bits,
                                                     ctypes.byref(desc), _ptr(w_scale), ctypes.c_float(act_scale), _ptr(bias),
                                                     _ptr(residual), ctypes.c_float(residual_scale), ctypes.c_float(out_scale),
                                                     int(bool(relu)), _ptr(y), ctypes.c_void_p(workspace.data_ptr() + off),
                                                     _i64(workspace.numel() - off), _stream()),
           "nq_conv_implicit_gemm_nested_q8_res")
    return y


def nq_conv_workspace_bytes(desc: nq_conv_desc) -> int:
    return int(lib().nq_conv_workspace_bytes(ctypes.byref(desc)))


def nq_conv_implicit_gemm(X: torch.Tensor, Wt: torch.Tensor, desc: nq_conv_desc, w_scale: torch.Tensor,
                          act_scale: float, part_bit: bool = False, n_bits: int = 8, h_bits: int = 6,
                          bias: Optional[torch.Tensor] = None, want_acc: bool = False, y_dtype=torch.float32,
                          workspace: Optional[torch.Tensor] = None, acc_out: Optional[torch.Tensor] = None,
                          y_out: Optional[torch.Tensor] = None):
    """X int8 NHWC (or NCHW when desc.x_nchw); Wt int8 [Cout, ldw] (full-bit) or sliced uint8 (part-bit).
    -> (acc int32 [B, Ho, Wo, Cout] or None, Y [B, Ho, Wo, Cout] or None, workspace)."""
    _need(X, torch.int8, "X")
    _need(w_scale, torch.float32, "w_scale", 1)
    if part_bit:
        _need(Wt, torch.uint8, "Wt")
        ldw = 0
    else:
        _need(Wt, torch.int8, "Wt", 2)
        ldw = _ld(Wt)
    Ho = (desc.H + 2 * desc.pad - desc.R) // desc.stride + 1
    Wo = (desc.W + 2 * desc.pad - desc.S) // desc.stride + 1
    need = nq_conv_workspace_bytes(desc)
    if need < 0:
        raise NqError(1, "nq_conv_workspace_bytes")
    if workspace is None:
        workspace = torch.empty(max(need, 1024) + 1024, dtype=torch.uint8, device=X.device)
    off = (-workspace.data_ptr()) % 1024
    ws = workspace[off:]
    shape = (desc.B, Ho, Wo, desc.Cout)
    acc = acc_out if acc_out is not None else (torch.empty(shape, dtype=torch.int32, device=X.device) if want_acc else None)
    y = y_out if y_out is not None else (torch.empty(shape, dtype=y_dtype, device=X.device) if y_dtype is not None else None)
    _check(lib().nq_conv_implicit_gemm(_ptr(X), _ptr(Wt), _i64(ldw), int(bool(part_bit)), n_bits, h_bits,
                                       ctypes.byref(desc), _ptr(w_scale), ctypes.c_float(act_scale), _ptr(bias),
                                       _ptr(acc), _ptr(y), _y_dtype(y.dtype) if y is not None else NQ_F32,
                                       _ptr(ws), _i64(ws.numel()), _stream()), "nq_conv_implicit_gemm")
    return acc, y, workspace


def nq_conv_implicit_gemm_nested(X: torch.Tensor, packed_high: torch.Tensor, packed_low: torch.Tensor, desc: nq_conv_desc,
                                 w_scale: torch.Tensor, act_scale: float, n_bits: int = 8, h_bits: int = 6,
                                 bias: Optional[torch.Tensor] = None, want_acc: bool = False, y_dtype=torch.float32,
                                 workspace: Optional[torch.Tensor] = None, y_out: Optional[torch.Tensor] = None):
    """The full-bit convolution computed from the packed higher-bit and compensated lower-bit tensors.
    -> (acc int32 [B, Ho, Wo, Cout] or None, Y [B, Ho, Wo, Cout] or None, workspace)."""
    _need(X, torch.int8, "X")
    _need(packed_high, torch.uint8, "packed_high")
    _need(packed_low, torch.uint8, "packed_low")
    _need(w_scale, torch.float32, "w_scale", 1)
    Ho = (desc.H + 2 * desc.pad - desc.R) // desc.stride + 1
    Wo = (desc.W + 2 * desc.pad - desc.S) // desc.stride + 1
    need = nq_conv_workspace_bytes(desc)
    if need < 0:
        raise NqError(1, "nq_conv_workspace_bytes")
    if workspace is None:
        workspace = torch.empty(max(need, 1024) + 1024, dtype=torch.uint8, device=X.device)
    off = (-workspace.data_ptr()) % 1024
    ws = workspace[off:]
    shape = (desc.B, Ho, Wo, desc.Cout)
    acc = torch.empty(shape, dtype=torch.int32, device=X.device) if want_acc else None
    y = y_out if y_out is not None else (torch.empty(shape, dtype=y_dtype, device=X.device) if y_dtype is not None else None)
    _check(lib().nq_conv_implicit_gemm_nested(_ptr(X), _ptr(packed_high), _ptr(packed_low), n_bits, h_bits,
                                              ctypes.byref(desc), _ptr(w_scale), ctypes.c_float(act_scale), _ptr(bias),
                                              _ptr(acc), _ptr(y), _y_dtype(y.dtype) if y is not None else NQ_F32,
                                              _ptr(ws), _i64(ws.numel()), _stream()), "nq_conv_implicit_gemm_nested")
    return acc, y, workspace


NQ_CONV_STATIC_SCRATCH_BYTES = 16 * 1024 * 1024


def nq_conv_implicit_gemm_static(X: torch.Tensor, Wt: torch.Tensor, desc: nq_conv_desc, w_scale: torch.Tensor,
                                 act_scale: float, acc_out: Optional[torch.Tensor], y_out: Optional[torch.Tensor],
                                 part_bit: bool = False, n_bits: int = 8, h_bits: int = 6,
                                 bias: Optional[torch.Tensor] = None):
    """The convolution for callers that cannot allocate: no workspace argument, and this wrapper allocates
    nothing either -- the caller passes the output tensors (acc_out int32 and / or y_out fp32 / bf16, NHWC).
    Layers that need more than NQ_CONV_STATIC_SCRATCH_BYTES of staging raise NqError(NQ_ERR_WORKSPACE)."""
    _need(X, torch.int8, "X")
    _need(w_scale, torch.float32, "w_scale", 1)
    if acc_out is None and y_out is None:
        raise ValueError("pass acc_out and / or y_out")
    if part_bit:
        _need(Wt, torch.uint8, "Wt")
        ldw = 0
    else:
        _need(Wt, torch.int8, "Wt", 2)
        ldw = _ld(Wt)
    _check(lib().nq_conv_implicit_gemm_static(_ptr(X), _ptr(Wt), _i64(ldw), int(bool(part_bit)), n_bits, h_bits,
                                              ctypes.byref(desc), _ptr(w_scale), ctypes.c_float(act_scale), _ptr(bias),
                                              _ptr(acc_out), _ptr(y_out),
                                              _y_dtype(y_out.dtype) if y_out is not None else NQ_F32, _stream()),
           "nq_conv_implicit_gemm_static")
    return acc_out, y_out


NQ_DEBUG_PLAIN_STORES, NQ_DEBUG_PACKED_RING = 0, 1


def nq_debug_set(which: int, enabled: bool) -> None:
    """Test aid: force ordinary stores / the packed-tile ring (see nq.h)."""
    _check(lib().nq_debug_set(int(which), int(bool(enabled))), "nq_debug_set")


def nq_maxpool_nhwc_i8(X: torch.Tensor, ksize: int, stride: int, pad: int, y_out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """INT8 NHWC [B, H, W, C] -> [B, Ho, Wo, C], integer maximum over the taps inside the image."""
    _need(X, torch.int8, "X", 4)
    B, H, W, C = X.shape
    Ho, Wo = (H + 2 * pad - ksize) // stride + 1, (W + 2 * pad - ksize) // stride + 1
    y = y_out if y_out is not None else torch.empty((B, Ho, Wo, C), dtype=torch.int8, device=X.device)
    _check(lib().nq_maxpool_nhwc_i8(_ptr(X), B, H, W, C, ksize, stride, pad, _ptr(y), _stream()), "nq_maxpool_nhwc_i8")
    return y


def nq_avgpool_requant_nhwc_i8(X: torch.Tensor, in_scale: float, out_scale: float,
                               y_out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """INT8 NHWC [B, H, W, C] -> INT8 [B, C]: global average, requantised."""
    _need(X, torch.int8, "X", 4)
    B, H, W, C = X.shape
    y = y_out if y_out is not None else torch.empty((B, C), dtype=torch.int8, device=X.device)
    _check(lib().nq_avgpool_requant_nhwc_i8(_ptr(X), B, H, W, C, ctypes.c_float(in_scale), ctypes.c_float(out_scale),
                                            _ptr(y), _stream()), "nq_avgpool_requant_nhwc_i8")
    return y


def nq_i8_mma_ceiling(stage_iters: int) -> float:
    """Enqueues one launch of the MMA-issue-only kernel on the current stream; returns its integer operations."""
    ops = ctypes.c_double(0.0)
    _check(lib().nq_i8_mma_ceiling(_i64(stage_iters), ctypes.byref(ops), _stream()), "nq_i8_mma_ceiling")
    return float(ops.value)


def nq_device_status() -> int:
    """Synchronises the current stream; raises NqError(NQ_ERR_TIMEOUT) if a bounded device wait expired."""
    where = ctypes.c_int(0)
    st = lib().nq_device_status(_stream(), ctypes.byref(where))
    if st != NQ_OK:
        raise NqError(st, f"nq_device_status (wait code {where.value})")
    return 0
