"""Python binding of libqbert: argument marshalling only.

Every step of the path (activation quantizer, group-wise weight quantizer and packer, integer
GEMM with dequantizing epilogue, encoder-layer linear stack) runs in the CUDA kernels behind the C
ABI declared in ``include/qbert.h``.  torch is used for device buffers and the current stream.
There is no CPU fallback: if ``libqbert.so`` has not been built, importing works but the first call
raises ``QbertError``.
"""
from __future__ import annotations

import ctypes
from dataclasses import dataclass
from pathlib import Path
from typing import Optional, Sequence

import torch

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libqbert.so"

QB_OK = 0
QB_ERR_INVALID = -1
QB_ERR_ALIGN = -2
QB_ERR_WORKSPACE = -3
QB_ERR_CUDA = -4
QB_ERR_NONFINITE = -5
QB_ERR_TIMEOUT = -6

EXPORTS = (
    "qb_version", "qb_status_string", "qb_last_error", "qb_packed_words", "qb_workspace_bytes",
    "qb_workspace_init", "qb_read_status", "qb_quantize_act", "qb_quantize_pack_weights", "qb_gemm",
    "qb_layer_linears", "qb_quantize_pack_weights_noalloc", "qb_probe_i8_mma", "qb_quantize_act_batch",
    "qb_quantize_pack_weights_batch", "qb_gemm_bf16", "qb_layer_linears_bf16",
    "qb_fake_quantize_weights", "qb_fake_quantize_weights_batch", "qb_ste_backward", "qb_quantize_embedding", "qb_embedding_lookup",
    "qb_gemm_i8", "qb_rowsum_i8", "qb_layer_linears_i8", "qb_sensitivity_bits", "qb_probe_wait_limit", "qb_layer_linears_launch_count", "qb_quantize_pack_weights_launch_count", "qb_quantize_act_launch_count",
)
NOALLOC_MAX_GROUPS = 4096


class QbertError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{message} (status {status})")
        self.status = status


class LinearDescC(ctypes.Structure):
    """Mirror of ``qb_linear_desc``."""
    _fields_ = [
        ("xq", ctypes.c_void_p), ("act_scale", ctypes.c_void_p), ("rowsum", ctypes.c_void_p),
        ("packed", ctypes.c_void_p), ("delta", ctypes.c_void_p), ("q0", ctypes.c_void_p),
        ("bias", ctypes.c_void_p),
        ("M", ctypes.c_int64), ("N", ctypes.c_int64), ("K", ctypes.c_int64),
        ("bits", ctypes.c_int32), ("groups", ctypes.c_int32),
        ("y", ctypes.c_void_p),
    ]


class ActDescC(ctypes.Structure):
    """Mirror of ``qb_act_desc``."""
    _fields_ = [("x", ctypes.c_void_p), ("M", ctypes.c_int64), ("K", ctypes.c_int64), ("xq", ctypes.c_void_p),
                ("act_scale", ctypes.c_void_p), ("rowsum", ctypes.c_void_p)]


class WeightDescC(ctypes.Structure):
    """Mirror of ``qb_weight_desc``."""
    _fields_ = [("w", ctypes.c_void_p), ("N", ctypes.c_int64), ("K", ctypes.c_int64), ("bits", ctypes.c_int32),
                ("groups", ctypes.c_int32), ("range_lo", ctypes.c_void_p), ("range_hi", ctypes.c_void_p),
                ("packed", ctypes.c_void_p), ("delta", ctypes.c_void_p), ("q0", ctypes.c_void_p)]


_lib: Optional[ctypes.CDLL] = None


def lib() -> ctypes.CDLL:
    """Load ``libqbert.so`` (built in-tree by ``paper_1909_05840_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not LIB_PATH.exists():
        raise QbertError(QB_ERR_CUDA, f"{LIB_PATH} is missing: build it with "
                                      "`python -m paper_1909_05840_b200.build`; there is no CPU fallback")
    L = ctypes.CDLL(str(LIB_PATH))
    i64, i32, vp, sz = ctypes.c_int64, ctypes.c_int32, ctypes.c_void_p, ctypes.c_size_t
    L.qb_version.restype = ctypes.c_int
    L.qb_status_string.argtypes = [i32]
    L.qb_status_string.restype = ctypes.c_char_p
    L.qb_last_error.restype = ctypes.c_char_p
    L.qb_packed_words.argtypes = [i64, i64, ctypes.c_int]
    L.qb_packed_words.restype = sz
    L.qb_workspace_bytes.argtypes = [i64, i64, i64, ctypes.c_int, ctypes.c_int]
    L.qb_workspace_bytes.restype = sz
    L.qb_workspace_init.argtypes = [vp, sz, vp]
    L.qb_workspace_init.restype = i32
    L.qb_read_status.argtypes = [vp, vp]
    L.qb_read_status.restype = i32
    L.qb_quantize_act.argtypes = [vp, i64, i64, vp, vp, vp, vp, sz, vp]
    L.qb_quantize_act.restype = i32
    L.qb_quantize_pack_weights.argtypes = [vp, i64, i64, ctypes.c_int, ctypes.c_int, vp, vp, vp, vp, vp, vp, sz, vp]
    L.qb_quantize_pack_weights.restype = i32
    L.qb_quantize_pack_weights_noalloc.argtypes = [vp, i64, i64, ctypes.c_int, ctypes.c_int, vp, vp, vp, vp, vp, vp, vp]
    L.qb_quantize_pack_weights_noalloc.restype = i32
    L.qb_probe_i8_mma.argtypes = [i32, i32, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]
    L.qb_probe_i8_mma.restype = i32
    L.qb_layer_linears_launch_count.argtypes = [ctypes.POINTER(LinearDescC), i32]
    L.qb_layer_linears_launch_count.restype = i32
    L.qb_quantize_pack_weights_launch_count.argtypes = [ctypes.POINTER(WeightDescC), i32]
    L.qb_quantize_pack_weights_launch_count.restype = i32
    L.qb_quantize_act_launch_count.argtypes = [i32]
    L.qb_quantize_act_launch_count.restype = i32
    L.qb_probe_wait_limit.argtypes = [vp, sz, i64, vp, vp]
    L.qb_probe_wait_limit.restype = i32
    L.qb_sensitivity_bits.argtypes = [vp, i32, i32, vp, i32, vp, vp, vp]
    L.qb_sensitivity_bits.restype = i32
    L.qb_quantize_act_batch.argtypes = [ctypes.POINTER(ActDescC), i32, vp, sz, vp]
    L.qb_quantize_act_batch.restype = i32
    L.qb_quantize_pack_weights_batch.argtypes = [ctypes.POINTER(WeightDescC), i32, vp, sz, vp]
    L.qb_quantize_pack_weights_batch.restype = i32
    L.qb_gemm.argtypes = [vp, vp, vp, vp, vp, vp, vp, i64, i64, i64, ctypes.c_int, ctypes.c_int, vp, vp, vp, sz, vp]
    L.qb_gemm.restype = i32
    L.qb_layer_linears.argtypes = [ctypes.POINTER(LinearDescC), i32, vp, sz, vp]
    L.qb_layer_linears.restype = i32
    L.qb_fake_quantize_weights.argtypes = [vp, i64, i64, ctypes.c_int, ctypes.c_int, vp, vp, vp, vp, vp, vp, sz, vp]
    L.qb_fake_quantize_weights.restype = i32
    L.qb_fake_quantize_weights_batch.argtypes = [ctypes.POINTER(WeightDescC), i32, vp, sz, vp]
    L.qb_fake_quantize_weights_batch.restype = i32
    L.qb_ste_backward.argtypes = [vp, vp, i64, i64, ctypes.c_int, vp, vp, vp, vp]
    L.qb_ste_backward.restype = i32
    L.qb_quantize_embedding.argtypes = [vp, i64, i64, ctypes.c_int, ctypes.c_int, vp, vp, vp, vp, sz, vp]
    L.qb_quantize_embedding.restype = i32
    L.qb_embedding_lookup.argtypes = [vp, i64, vp, vp, vp, i64, i64, ctypes.c_int, ctypes.c_int, ctypes.c_int, vp, vp,
                                      sz, vp]
    L.qb_embedding_lookup.restype = i32
    L.qb_gemm_i8.argtypes = [vp, vp, vp, vp, vp, vp, vp, i64, i64, i64, ctypes.c_int, ctypes.c_int, vp, vp, vp, sz, vp]
    L.qb_gemm_i8.restype = i32
    L.qb_layer_linears_i8.argtypes = [ctypes.POINTER(LinearDescC), ctypes.POINTER(vp), i32, vp, sz, vp]
    L.qb_layer_linears_i8.restype = i32
    L.qb_rowsum_i8.argtypes = [vp, i64, i64, vp, vp]
    L.qb_rowsum_i8.restype = i32
    L.qb_gemm_bf16.argtypes = [vp, vp, vp, vp, vp, vp, vp, i64, i64, i64, ctypes.c_int, ctypes.c_int, vp, vp, sz, vp]
    L.qb_gemm_bf16.restype = i32
    L.qb_layer_linears_bf16.argtypes = [ctypes.POINTER(LinearDescC), i32, vp, sz, vp]
    L.qb_layer_linears_bf16.restype = i32
    _lib = L
    return L


def _check(status: int, what: str) -> None:
    if status != QB_OK:
        L = lib()
        name = L.qb_status_string(status).decode()
        raise QbertError(status, f"{what}: {name}: {L.qb_last_error().decode()}")


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def version() -> int:
    return int(lib().qb_version())


def packed_words(N: int, K: int, bits: int) -> int:
    return int(lib().qb_packed_words(N, K, bits))


def workspace_bytes(M: int = 0, N: int = 0, K: int = 0, bits: int = 0, groups: int = 0) -> int:
    return int(lib().qb_workspace_bytes(M, N, K, bits, groups))


def workspace(groups: int = 4096, device="cuda") -> torch.Tensor:
    """A zero-initialised workspace large enough for any call with up to ``groups`` groups."""
    ws = torch.empty(workspace_bytes(groups=groups), dtype=torch.uint8, device=device)
    _check(lib().qb_workspace_init(ws.data_ptr(), ws.numel(), _stream()), "qb_workspace_init")
    return ws


def read_status(ws: torch.Tensor) -> int:
    """Synchronise the current stream and return the workspace's status word."""
    return int(lib().qb_read_status(ws.data_ptr(), _stream()))


def quantize_act(x: torch.Tensor, ws: torch.Tensor, xq: Optional[torch.Tensor] = None,
                 act_scale: Optional[torch.Tensor] = None, rowsum: Optional[torch.Tensor] = None):
    """``qb_quantize_act``: fp32 [M,K] -> (int8 codes [M,K], fp32 scale [1], int32 row sums [M])."""
    assert x.is_cuda and x.dtype == torch.float32 and x.dim() == 2 and x.is_contiguous()
    M, K = x.shape
    xq = torch.empty((M, K), dtype=torch.int8, device=x.device) if xq is None else xq
    act_scale = torch.empty(1, dtype=torch.float32, device=x.device) if act_scale is None else act_scale
    rowsum = torch.empty(M, dtype=torch.int32, device=x.device) if rowsum is None else rowsum
    _check(lib().qb_quantize_act(x.data_ptr(), M, K, xq.data_ptr(), act_scale.data_ptr(), rowsum.data_ptr(),
                                 ws.data_ptr(), ws.numel(), _stream()), "qb_quantize_act")
    return xq, act_scale, rowsum


def quantize_pack_weights(w: torch.Tensor, bits: int, groups: int, ws: torch.Tensor,
                          range_lo: Optional[torch.Tensor] = None, range_hi: Optional[torch.Tensor] = None,
                          packed: Optional[torch.Tensor] = None, delta: Optional[torch.Tensor] = None,
                          q0: Optional[torch.Tensor] = None):
    """``qb_quantize_pack_weights``: fp32 [N,K] -> (int32-viewed packed words [N, K*bits/32], delta [G], q0 [G])."""
    assert w.is_cuda and w.dtype == torch.float32 and w.dim() == 2 and w.is_contiguous()
    N, K = w.shape
    if packed is None:
        words_per_row = max(1, K * bits // 32)
        packed = torch.empty((N, words_per_row), dtype=torch.int32, device=w.device)
    delta = torch.empty(max(groups, 1), dtype=torch.float32, device=w.device) if delta is None else delta
    q0 = torch.empty(max(groups, 1), dtype=torch.float32, device=w.device) if q0 is None else q0
    _check(lib().qb_quantize_pack_weights(w.data_ptr(), N, K, bits, groups, _ptr(range_lo), _ptr(range_hi),
                                          packed.data_ptr(), delta.data_ptr(), q0.data_ptr(), ws.data_ptr(),
                                          ws.numel(), _stream()), "qb_quantize_pack_weights")
    return packed, delta, q0


def fake_quantize_weights(w: torch.Tensor, bits: int, groups: int, ws: torch.Tensor,
                          range_lo: Optional[torch.Tensor] = None, range_hi: Optional[torch.Tensor] = None,
                          wq: Optional[torch.Tensor] = None):
    """``qb_fake_quantize_weights``: fp32 [N,K] -> (Q(W) fp32 [N,K], delta [G], q0 [G])."""
    assert w.is_cuda and w.dtype == torch.float32 and w.dim() == 2 and w.is_contiguous()
    N, K = w.shape
    wq = torch.empty_like(w) if wq is None else wq
    delta = torch.empty(groups, dtype=torch.float32, device=w.device)
    q0 = torch.empty(groups, dtype=torch.float32, device=w.device)
    _check(lib().qb_fake_quantize_weights(w.data_ptr(), N, K, bits, groups, _ptr(range_lo), _ptr(range_hi),
                                          wq.data_ptr(), delta.data_ptr(), q0.data_ptr(), ws.data_ptr(), ws.numel(),
                                          _stream()), "qb_fake_quantize_weights")
    return wq, delta, q0


def fake_quantize_weights_batch(items, ws: torch.Tensor) -> None:
    """``qb_fake_quantize_weights_batch`` over ``(w, bits, groups, wq, delta, q0)`` tuples (or a C array whose
    ``packed`` fields point to the fp32 outputs)."""
    arr = items if isinstance(items, ctypes.Array) else make_weight_desc_array(items)
    _check(lib().qb_fake_quantize_weights_batch(arr, len(arr), ws.data_ptr(), ws.numel(), _stream()),
           "qb_fake_quantize_weights_batch")


def ste_backward(grad_wq: torch.Tensor, w: torch.Tensor, groups: int, range_lo: Optional[torch.Tensor] = None,
                 range_hi: Optional[torch.Tensor] = None, grad_w: Optional[torch.Tensor] = None) -> torch.Tensor:
    """``qb_ste_backward``: straight-through gradient of the quantizer with respect to the weights."""
    assert grad_wq.is_cuda and grad_wq.dtype == torch.float32 and grad_wq.is_contiguous() and grad_wq.shape == w.shape
    N, K = w.shape
    grad_w = torch.empty_like(w) if grad_w is None else grad_w
    _check(lib().qb_ste_backward(grad_wq.data_ptr(), w.data_ptr(), N, K, groups, _ptr(range_lo), _ptr(range_hi),
                                 grad_w.data_ptr(), _stream()), "qb_ste_backward")
    return grad_w


def quantize_embedding(table: torch.Tensor, bits: int, groups: int, ws: torch.Tensor,
                       packed: Optional[torch.Tensor] = None):
    """``qb_quantize_embedding``: fp32 [V,D] -> (int32-viewed packed rows [V, D*bits/32], delta [G], q0 [G])."""
    assert table.is_cuda and table.dtype == torch.float32 and table.dim() == 2 and table.is_contiguous()
    V, D = table.shape
    if packed is None:
        packed = torch.empty((V, D * bits // 32), dtype=torch.int32, device=table.device)
    delta = torch.empty(groups, dtype=torch.float32, device=table.device)
    q0 = torch.empty(groups, dtype=torch.float32, device=table.device)
    _check(lib().qb_quantize_embedding(table.data_ptr(), V, D, bits, groups, packed.data_ptr(), delta.data_ptr(),
                                       q0.data_ptr(), ws.data_ptr(), ws.numel(), _stream()), "qb_quantize_embedding")
    return packed, delta, q0


def embedding_lookup(ids: torch.Tensor, packed: torch.Tensor, delta: torch.Tensor, q0: torch.Tensor, D: int,
                     bits: int, groups: int, ws: torch.Tensor, out: Optional[torch.Tensor] = None,
                     accumulate: bool = False) -> torch.Tensor:
    """``qb_embedding_lookup``: int32 ids [T] -> fp32 [T,D]; with ``accumulate`` the rows are added to ``out``."""
    assert ids.is_cuda and ids.dtype == torch.int32 and ids.is_contiguous()
    T = ids.numel()
    V = packed.shape[0]
    if out is None:
        assert not accumulate
        out = torch.empty((T, D), dtype=torch.float32, device=ids.device)
    _check(lib().qb_embedding_lookup(ids.data_ptr(), T, packed.data_ptr(), delta.data_ptr(), q0.data_ptr(), V, D, bits,
                                     groups, 1 if accumulate else 0, out.data_ptr(), ws.data_ptr(), ws.numel(),
                                     _stream()), "qb_embedding_lookup")
    return out


def make_act_desc_array(items):
    """``items``: sequence of ``(x, xq, act_scale, rowsum)`` tensors -> C array of ``qb_act_desc``."""
    arr = (ActDescC * len(items))()
    for i, (x, xq, sc, rs) in enumerate(items):
        assert x.is_cuda and x.dtype == torch.float32 and x.dim() == 2 and x.is_contiguous()
        arr[i] = ActDescC(x.data_ptr(), x.shape[0], x.shape[1], xq.data_ptr(), sc.data_ptr(), rs.data_ptr())
    return arr


def quantize_act_batch(items, ws: torch.Tensor) -> None:
    """``qb_quantize_act_batch`` over ``(x, xq, act_scale, rowsum)`` tuples (or a prepared C array)."""
    arr = items if isinstance(items, ctypes.Array) else make_act_desc_array(items)
    _check(lib().qb_quantize_act_batch(arr, len(arr), ws.data_ptr(), ws.numel(), _stream()), "qb_quantize_act_batch")


def make_weight_desc_array(items):
    """``items``: sequence of ``(w, bits, groups, packed, delta, q0)`` -> C array of ``qb_weight_desc``."""
    arr = (WeightDescC * len(items))()
    for i, (w, bits, groups, packed, delta, q0) in enumerate(items):
        assert w.is_cuda and w.dtype == torch.float32 and w.dim() == 2 and w.is_contiguous()
        arr[i] = WeightDescC(w.data_ptr(), w.shape[0], w.shape[1], bits, groups, None, None, packed.data_ptr(),
                             delta.data_ptr(), q0.data_ptr())
    return arr


def quantize_pack_weights_batch(items, ws: torch.Tensor) -> None:
    """``qb_quantize_pack_weights_batch`` over ``(w, bits, groups, packed, delta, q0)`` tuples (or a C array)."""
    arr = items if isinstance(items, ctypes.Array) else make_weight_desc_array(items)
    _check(lib().qb_quantize_pack_weights_batch(arr, len(arr), ws.data_ptr(), ws.numel(), _stream()),
           "qb_quantize_pack_weights_batch")


def quantize_pack_weights_noalloc(w: torch.Tensor, bits: int, groups: int, packed: torch.Tensor,
                                  delta: torch.Tensor, q0: torch.Tensor, status_out: Optional[torch.Tensor] = None,
                                  range_lo: Optional[torch.Tensor] = None, range_hi: Optional[torch.Tensor] = None):
    """``qb_quantize_pack_weights_noalloc``: same results as ``quantize_pack_weights`` for callers that
    cannot allocate a workspace (the scratch is a fixed array inside the library, at most
    ``NOALLOC_MAX_GROUPS`` groups).  Every buffer, outputs included, is the caller's: this wrapper
    allocates nothing either.  ``status_out`` (int32 [1], optional) receives the device status word."""
    assert w.is_cuda and w.dtype == torch.float32 and w.dim() == 2 and w.is_contiguous()
    N, K = w.shape
    _check(lib().qb_quantize_pack_weights_noalloc(w.data_ptr(), N, K, bits, groups, _ptr(range_lo), _ptr(range_hi),
                                                  packed.data_ptr(), delta.data_ptr(), q0.data_ptr(),
                                                  _ptr(status_out), _stream()), "qb_quantize_pack_weights_noalloc")
    return packed, delta, q0


def probe_i8_mma(tokens: int = 256, k_blocks: int = 20000):
    """``qb_probe_i8_mma``: (TOPS, SM cycles per K block) the tensor cores sustain for the GEMM's MMA."""
    tops, cyc = ctypes.c_double(0.0), ctypes.c_double(0.0)
    _check(lib().qb_probe_i8_mma(tokens, k_blocks, ctypes.byref(tops), ctypes.byref(cyc)), "qb_probe_i8_mma")
    return tops.value, cyc.value


def probe_wait_limit(ws: torch.Tensor, limit_cycles: int = 2_000_000) -> torch.Tensor:
    """``qb_probe_wait_limit``: a bounded wait that must run out; returns the cycles the two warps waited."""
    waited = torch.zeros(2, dtype=torch.int64, device=ws.device)
    _check(lib().qb_probe_wait_limit(ws.data_ptr(), ws.numel(), limit_cycles, waited.data_ptr(), _stream()),
           "qb_probe_wait_limit")
    return waited


def sensitivity_bits(lam, budget_bits, reverse: bool = False):
    """``qb_sensitivity_bits`` (host only): ``lam`` [layers, samples] eigenvalue samples, ``budget_bits`` the bit
    width for each rank of the descending Omega order.  Returns (omega f64 [L], order i32 [L], bits i32 [L])."""
    import numpy as np
    lam = np.ascontiguousarray(lam, dtype=np.float64)
    budget = np.ascontiguousarray(budget_bits, dtype=np.int32)
    layers, samples = lam.shape
    if budget.shape != (layers,):
        raise QbertError(QB_ERR_INVALID, "budget_bits must have one entry per layer")
    omega = np.empty(layers, np.float64)
    order = np.empty(layers, np.int32)
    bits = np.empty(layers, np.int32)
    _check(lib().qb_sensitivity_bits(lam.ctypes.data, layers, samples, budget.ctypes.data, int(reverse),
                                     omega.ctypes.data, order.ctypes.data, bits.ctypes.data), "qb_sensitivity_bits")
    return omega, order, bits


def gemm(xq: torch.Tensor, act_scale: torch.Tensor, rowsum: torch.Tensor, packed: torch.Tensor,
         delta: torch.Tensor, q0: torch.Tensor, bias: Optional[torch.Tensor], N: int, bits: int, groups: int,
         ws: torch.Tensor, y: Optional[torch.Tensor] = None, acc_out: Optional[torch.Tensor] = None,
         want_acc: bool = False):
    """``qb_gemm``: returns ``y`` fp32 [M,N] (and the int32 accumulators when ``want_acc``)."""
    assert xq.is_cuda and xq.dtype == torch.int8 and xq.is_contiguous()
    M, K = xq.shape
    y = torch.empty((M, N), dtype=torch.float32, device=xq.device) if y is None else y
    if want_acc and acc_out is None:
        acc_out = torch.empty((M, N), dtype=torch.int32, device=xq.device)
    _check(lib().qb_gemm(xq.data_ptr(), act_scale.data_ptr(), rowsum.data_ptr(), packed.data_ptr(),
                         delta.data_ptr(), q0.data_ptr(), _ptr(bias), M, N, K, bits, groups, y.data_ptr(),
                         _ptr(acc_out), ws.data_ptr(), ws.numel(), _stream()), "qb_gemm")
    return (y, acc_out) if (want_acc or acc_out is not None) else y


def gemm_bf16(xq: torch.Tensor, act_scale: torch.Tensor, rowsum: torch.Tensor, packed: torch.Tensor,
              delta: torch.Tensor, q0: torch.Tensor, bias: Optional[torch.Tensor], N: int, bits: int, groups: int,
              ws: torch.Tensor, y: Optional[torch.Tensor] = None) -> torch.Tensor:
    """``qb_gemm_bf16``: returns ``y`` bfloat16 [M,N]."""
    assert xq.is_cuda and xq.dtype == torch.int8 and xq.is_contiguous()
    M, K = xq.shape
    y = torch.empty((M, N), dtype=torch.bfloat16, device=xq.device) if y is None else y
    assert y.dtype == torch.bfloat16 and y.is_contiguous()
    _check(lib().qb_gemm_bf16(xq.data_ptr(), act_scale.data_ptr(), rowsum.data_ptr(), packed.data_ptr(),
                              delta.data_ptr(), q0.data_ptr(), _ptr(bias), M, N, K, bits, groups, y.data_ptr(),
                              ws.data_ptr(), ws.numel(), _stream()), "qb_gemm_bf16")
    return y


def gemm_i8(xq: torch.Tensor, act_scale: torch.Tensor, rowsum: torch.Tensor, packed: torch.Tensor,
            delta: torch.Tensor, q0: torch.Tensor, bias: Optional[torch.Tensor], N: int, bits: int, groups: int,
            out_scale: torch.Tensor, ws: torch.Tensor, yq: Optional[torch.Tensor] = None) -> torch.Tensor:
    """``qb_gemm_i8``: returns int8 codes [M,N] on the grid of step ``out_scale`` (device fp32 [1])."""
    assert xq.is_cuda and xq.dtype == torch.int8 and xq.is_contiguous()
    assert out_scale.is_cuda and out_scale.dtype == torch.float32
    M, K = xq.shape
    yq = torch.empty((M, N), dtype=torch.int8, device=xq.device) if yq is None else yq
    _check(lib().qb_gemm_i8(xq.data_ptr(), act_scale.data_ptr(), rowsum.data_ptr(), packed.data_ptr(),
                            delta.data_ptr(), q0.data_ptr(), _ptr(bias), M, N, K, bits, groups, out_scale.data_ptr(),
                            yq.data_ptr(), ws.data_ptr(), ws.numel(), _stream()), "qb_gemm_i8")
    return yq


def rowsum_i8(xq: torch.Tensor, rowsum: Optional[torch.Tensor] = None) -> torch.Tensor:
    """``qb_rowsum_i8``: int32 row sums of int8 codes [M,K]."""
    assert xq.is_cuda and xq.dtype == torch.int8 and xq.dim() == 2 and xq.is_contiguous()
    M, K = xq.shape
    rowsum = torch.empty(M, dtype=torch.int32, device=xq.device) if rowsum is None else rowsum
    _check(lib().qb_rowsum_i8(xq.data_ptr(), M, K, rowsum.data_ptr(), _stream()), "qb_rowsum_i8")
    return rowsum


@dataclass
class LinearDesc:
    """One linear of a stack: tensors as produced by ``quantize_act`` / ``quantize_pack_weights``."""
    xq: torch.Tensor
    act_scale: torch.Tensor
    rowsum: torch.Tensor
    packed: torch.Tensor
    delta: torch.Tensor
    q0: torch.Tensor
    bias: Optional[torch.Tensor]
    N: int
    bits: int
    groups: int
    y: torch.Tensor


def make_desc_array(descs: Sequence[LinearDesc]):
    """Marshal descriptors into a C array once; reuse it across calls on the same buffers."""
    arr = (LinearDescC * len(descs))()
    for i, d in enumerate(descs):
        M, K = d.xq.shape
        arr[i] = LinearDescC(d.xq.data_ptr(), d.act_scale.data_ptr(), d.rowsum.data_ptr(), d.packed.data_ptr(),
                             d.delta.data_ptr(), d.q0.data_ptr(), _ptr(d.bias), M, d.N, K, d.bits, d.groups,
                             d.y.data_ptr())
    return arr


def layer_linears(descs, ws: torch.Tensor) -> None:
    """``qb_layer_linears`` over a list of ``LinearDesc`` (or an array from ``make_desc_array``)."""
    arr = descs if isinstance(descs, ctypes.Array) else make_desc_array(descs)
    _check(lib().qb_layer_linears(arr, len(arr), ws.data_ptr(), ws.numel(), _stream()), "qb_layer_linears")


def quantize_act_launch_count(count: int) -> int:
    """``qb_quantize_act_launch_count``: kernel launches ``quantize_act_batch`` issues for ``count`` tensors."""
    return int(lib().qb_quantize_act_launch_count(int(count)))


def quantize_pack_weights_launch_count(items) -> int:
    """``qb_quantize_pack_weights_launch_count``: kernel launches ``quantize_pack_weights_batch`` issues for these matrices."""
    arr = items if isinstance(items, ctypes.Array) else make_weight_desc_array(items)
    return int(lib().qb_quantize_pack_weights_launch_count(arr, len(arr)))


def layer_linears_launch_count(descs) -> int:
    """``qb_layer_linears_launch_count``: GEMM kernel launches ``layer_linears`` issues for this stack."""
    arr = descs if isinstance(descs, ctypes.Array) else make_desc_array(descs)
    return int(lib().qb_layer_linears_launch_count(arr, len(arr)))


def layer_linears_i8(descs: Sequence[LinearDesc], out_scales: Sequence[torch.Tensor], ws: torch.Tensor) -> None:
    """``qb_layer_linears_i8``: every ``y`` an int8 [M,N] tensor, ``out_scales[i]`` a device fp32 [1] tensor."""
    assert len(descs) == len(out_scales) and all(d.y.dtype == torch.int8 for d in descs)
    arr = make_desc_array(descs)
    sc = (ctypes.c_void_p * len(descs))(*[t.data_ptr() for t in out_scales])
    _check(lib().qb_layer_linears_i8(arr, sc, len(arr), ws.data_ptr(), ws.numel(), _stream()), "qb_layer_linears_i8")


def layer_linears_bf16(descs, ws: torch.Tensor) -> None:
    """``qb_layer_linears_bf16``: as ``layer_linears``, every ``y`` a bfloat16 [M,N] tensor."""
    if not isinstance(descs, ctypes.Array):
        assert all(d.y.dtype == torch.bfloat16 for d in descs)
    arr = descs if isinstance(descs, ctypes.Array) else make_desc_array(descs)
    _check(lib().qb_layer_linears_bf16(arr, len(arr), ws.data_ptr(), ws.numel(), _stream()), "qb_layer_linears_bf16")
