"""numpy front end of the CPU oracle (``qbert_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the
CPU-baseline leg of ``bench.py``.  The CUDA library never imports this package
and this package never imports the CUDA library.

Two builds of the same source are kept side by side:

* ``libqbert_oracle.so``      ``-O2 -ffp-contract=off``, single thread: the parity oracle.
* ``libqbert_oracle_omp.so``  ``-O3 -ffp-contract=off -fopenmp``: the same loops on all host
  cores, used only when the oracle is *timed* as the CPU baseline.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "qbert_oracle.cpp"
_LIBS = {
    False: (_HERE / "libqbert_oracle.so", ["-O2"]),
    True: (_HERE / "libqbert_oracle_omp.so", ["-O3", "-fopenmp"]),
}
_loaded: dict[bool, ctypes.CDLL] = {}

OK = 0
ERR_INVALID = -1
ERR_NONFINITE = -5


def build(force: bool = False) -> None:
    """Compile both builds of the oracle with g++ if missing or older than the source."""
    for _omp, (lib, flags) in _LIBS.items():
        if not force and lib.exists() and lib.stat().st_mtime >= _SRC.stat().st_mtime:
            continue
        cmd = ["g++", "-std=c++17", *flags, "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
               str(_SRC), "-o", str(lib) + ".tmp"]
        subprocess.run(cmd, check=True)
        os.replace(str(lib) + ".tmp", lib)


def _lib(omp: bool = False) -> ctypes.CDLL:
    if omp not in _loaded:
        build()
        lib = ctypes.CDLL(str(_LIBS[omp][0]))
        i64, i32, vp, f32 = ctypes.c_int64, ctypes.c_int, ctypes.c_void_p, ctypes.c_float
        lib.qo_num_threads.restype = i32
        lib.qo_quantize_weights.argtypes = [vp, i64, i64, i32, i32, vp, vp, vp, vp, vp]
        lib.qo_quantize_weights.restype = i32
        lib.qo_dequantize_weights.argtypes = [vp, i64, i64, i32, vp, vp, vp]
        lib.qo_dequantize_weights.restype = None
        lib.qo_pack.argtypes = [vp, i64, i64, i32, vp]
        lib.qo_pack.restype = i32
        lib.qo_unpack.argtypes = [vp, i64, i64, i32, vp]
        lib.qo_unpack.restype = i32
        lib.qo_quantize_embedding.argtypes = [vp, i64, i64, i32, i32, vp, vp, vp]
        lib.qo_quantize_embedding.restype = i32
        lib.qo_embedding_lookup.argtypes = [vp, i64, vp, i64, i64, i32, vp, vp, i32, vp]
        lib.qo_embedding_lookup.restype = i32
        lib.qo_requantize_i8.argtypes = [vp, i64, f32, vp]
        lib.qo_requantize_i8.restype = i32
        lib.qo_rowsum_i8.argtypes = [vp, i64, i64, vp]
        lib.qo_rowsum_i8.restype = None
        lib.qo_ste_backward.argtypes = [vp, vp, i64, i64, i32, vp, vp, vp]
        lib.qo_ste_backward.restype = None
        lib.qo_sensitivity_bits.argtypes = [vp, i32, i32, vp, i32, vp, vp, vp]
        lib.qo_sensitivity_bits.restype = i32
        lib.qo_round_bf16.argtypes = [vp, i64, vp]
        lib.qo_round_bf16.restype = None
        lib.qo_quantize_act.argtypes = [vp, i64, i64, vp, vp, vp]
        lib.qo_quantize_act.restype = i32
        lib.qo_int_gemm.argtypes = [vp, vp, i64, i64, i64, vp, vp]
        lib.qo_int_gemm.restype = None
        lib.qo_dequant_epilogue.argtypes = [vp, vp, f32, vp, vp, vp, i64, i64, i32, i32, vp]
        lib.qo_dequant_epilogue.restype = None
        lib.qo_linear_fp64.argtypes = [vp, f32, vp, vp, vp, vp, i64, i64, i64, i32, vp]
        lib.qo_linear_fp64.restype = None
        _loaded[omp] = lib
    return _loaded[omp]


def num_threads(omp: bool = False) -> int:
    return int(_lib(omp).qo_num_threads())


def _c(a: np.ndarray, dtype) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def quantize_weights(w, bits: int, groups: int, range_lo=None, range_hi=None, omp: bool = False):
    """Group-wise uniform quantizer Q (Section 3.3, Appendix A).

    Returns ``(status, codes uint8 [N,K], delta f32 [G], q0 f32 [G])``.
    """
    w = _c(w, np.float32)
    N, K = w.shape
    codes = np.empty((N, K), np.uint8)
    delta = np.empty(groups, np.float32)
    q0 = np.empty(groups, np.float32)
    lo = None if range_lo is None else _c(range_lo, np.float32)
    hi = None if range_hi is None else _c(range_hi, np.float32)
    st = _lib(omp).qo_quantize_weights(_p(w), N, K, bits, groups, _p(lo), _p(hi), _p(codes), _p(delta),
                                       _p(q0))
    return st, codes, delta, q0


def dequantize_weights(codes, groups: int, delta, q0):
    """Q(W) = Delta * X^I + q0 (Appendix A) as fp32 fused multiply-add."""
    codes = _c(codes, np.uint8)
    N, K = codes.shape
    delta = _c(delta, np.float32)
    q0 = _c(q0, np.float32)
    out = np.empty((N, K), np.float32)
    _lib().qo_dequantize_weights(_p(codes), N, K, groups, _p(delta), _p(q0), _p(out))
    return out


def pack(codes, bits: int):
    """Dense little-endian k-bit packing: uint32 [N, K*bits/32]."""
    codes = _c(codes, np.uint8)
    N, K = codes.shape
    if (K * bits) % 32:
        raise ValueError("K*bits must be a multiple of 32")
    words = np.empty((N, K * bits // 32), np.uint32)
    st = _lib().qo_pack(_p(codes), N, K, bits, _p(words))
    if st != OK:
        raise ValueError(f"qo_pack status {st}")
    return words


def unpack(words, K: int, bits: int):
    words = _c(words, np.uint32)
    N = words.shape[0]
    codes = np.empty((N, K), np.uint8)
    st = _lib().qo_unpack(_p(words), N, K, bits, _p(codes))
    if st != OK:
        raise ValueError(f"qo_unpack status {st}")
    return codes


def quantize_act(x, omp: bool = False):
    """Per-tensor 8-bit activation quantizer: ``(status, xq int8 [M,K], scale f32, rowsum i32 [M])``."""
    x = _c(x, np.float32)
    M, K = x.shape
    xq = np.empty((M, K), np.int8)
    scale = np.empty(1, np.float32)
    rowsum = np.empty(M, np.int32)
    st = _lib(omp).qo_quantize_act(_p(x), M, K, _p(xq), _p(scale), _p(rowsum))
    return st, xq, np.float32(scale[0]), rowsum


def int_gemm(xq, codes, want64: bool = False, omp: bool = False):
    """acc[m,n] = sum_k xq[m,k] * u[n,k] in int32 (and int64 when ``want64``)."""
    xq = _c(xq, np.int8)
    codes = _c(codes, np.uint8)
    M, K = xq.shape
    N, K2 = codes.shape
    assert K == K2
    acc = np.empty((M, N), np.int32)
    acc64 = np.empty((M, N), np.int64) if want64 else None
    _lib(omp).qo_int_gemm(_p(xq), _p(codes), M, N, K, _p(acc), _p(acc64))
    return (acc, acc64) if want64 else acc


def dequant_epilogue(acc, rowsum, act_scale, delta, q0, bias, bits: int, groups: int, omp: bool = False):
    """fp32 'gathered dequantization' of the int32 accumulators (Appendix A)."""
    acc = _c(acc, np.int32)
    rowsum = _c(rowsum, np.int32)
    delta = _c(delta, np.float32)
    q0 = _c(q0, np.float32)
    b = None if bias is None else _c(bias, np.float32)
    M, N = acc.shape
    y = np.empty((M, N), np.float32)
    _lib(omp).qo_dequant_epilogue(_p(acc), _p(rowsum), float(act_scale), _p(delta), _p(q0), _p(b), M, N,
                                  bits, groups, _p(y))
    return y


def linear_fp64(xq, act_scale, codes, delta, q0, bias, groups: int, omp: bool = False):
    """The quantized linear layer from the definitions, accumulated in double precision."""
    xq = _c(xq, np.int8)
    codes = _c(codes, np.uint8)
    delta = _c(delta, np.float32)
    q0 = _c(q0, np.float32)
    b = None if bias is None else _c(bias, np.float32)
    M, K = xq.shape
    N = codes.shape[0]
    y = np.empty((M, N), np.float64)
    _lib(omp).qo_linear_fp64(_p(xq), float(act_scale), _p(codes), _p(delta), _p(q0), _p(b), M, N, K, groups,
                             _p(y))
    return y


def linear(x, w, bias, bits: int, groups: int, omp: bool = False):
    """Whole path on the CPU: quantize activations and weights, pack, integer GEMM, epilogue.

    Returns a dict with every intermediate the parity tests compare.
    """
    st_a, xq, s_a, rowsum = quantize_act(x, omp=omp)
    st_w, codes, delta, q0 = quantize_weights(w, bits, groups, omp=omp)
    words = pack(codes, bits)
    acc = int_gemm(xq, codes, omp=omp)
    y = dequant_epilogue(acc, rowsum, s_a, delta, q0, bias, bits, groups, omp=omp)
    return dict(status_act=st_a, status_w=st_w, xq=xq, act_scale=s_a, rowsum=rowsum, codes=codes,
                delta=delta, q0=q0, words=words, acc=acc, y=y)


def round_bf16(y) -> np.ndarray:
    """fp32 -> bfloat16 bit patterns (uint16), round to nearest, ties to even; same shape as ``y``."""
    y = _c(np.asarray(y), np.float32)
    out = np.empty(y.shape, dtype=np.uint16)
    _lib().qo_round_bf16(_p(y), y.size, _p(out))
    return out


def fake_quantize_weights(w, bits: int, groups: int, range_lo=None, range_hi=None, omp: bool = False):
    """Q(W) of Appendix A in fp32: (status, Q(w) [N,K], delta [G], q0 [G]); quantize, then Delta * code + q0."""
    st, codes, delta, q0 = quantize_weights(w, bits, groups, range_lo, range_hi, omp=omp)
    return st, dequantize_weights(codes, groups, delta, q0), delta, q0


def ste_backward(grad_q, w, groups: int, lo, hi) -> np.ndarray:
    """Straight-through gradient of the quantizer: grad_q where lo_g <= w <= hi_g, else 0."""
    grad_q = _c(grad_q, np.float32)
    w = _c(w, np.float32)
    lo = _c(lo, np.float32)
    hi = _c(hi, np.float32)
    N, K = w.shape
    out = np.empty((N, K), dtype=np.float32)
    _lib().qo_ste_backward(_p(grad_q), _p(w), N, K, groups, _p(lo), _p(hi), _p(out))
    return out


def quantize_embedding(e, bits: int, groups: int):
    """Column-group quantizer of an embedding table E [V,D]: (status, codes uint8 [V,D], delta [G], q0 [G])."""
    e = _c(e, np.float32)
    V, D = e.shape
    codes = np.empty((V, D), dtype=np.uint8)
    delta = np.empty(groups, dtype=np.float32)
    q0 = np.empty(groups, dtype=np.float32)
    st = _lib().qo_quantize_embedding(_p(e), V, D, bits, groups, _p(codes), _p(delta), _p(q0))
    return st, codes, delta, q0


def embedding_lookup(ids, codes, groups: int, delta, q0, out=None) -> np.ndarray:
    """Dequantizing lookup; with ``out`` given the looked-up rows are added to it."""
    ids = _c(ids, np.int32)
    codes = _c(codes, np.uint8)
    V, D = codes.shape
    acc = out is not None
    out = np.empty((ids.size, D), dtype=np.float32) if out is None else _c(out, np.float32).copy()
    st = _lib().qo_embedding_lookup(_p(ids), ids.size, _p(codes), V, D, groups, _p(_c(delta, np.float32)),
                                    _p(_c(q0, np.float32)), int(acc), _p(out))
    assert st == OK, "id out of range"
    return out


def requantize_i8(y, s_out: float) -> np.ndarray:
    """fp32 -> int8 codes on the grid of step ``s_out``: clamp(round_half_even(y / s_out), -127, 127)."""
    y = _c(np.asarray(y), np.float32)
    out = np.empty(y.shape, dtype=np.int8)
    st = _lib().qo_requantize_i8(_p(y), y.size, ctypes.c_float(s_out), _p(out))
    assert st == OK, "s_out must be finite and positive"
    return out


def rowsum_i8(xq) -> np.ndarray:
    xq = _c(xq, np.int8)
    M, K = xq.shape
    out = np.empty(M, dtype=np.int32)
    _lib().qo_rowsum_i8(_p(xq), M, K, _p(out))
    return out


def sensitivity_bits(lam, budget, reverse: bool = False):
    """Eq. 2: ``(status, omega f64 [L], order i32 [L], bits i32 [L])`` from eigenvalue samples ``lam`` [L, S]
    and ``budget``, the bit width for each rank of the descending order."""
    lam = _c(np.asarray(lam), np.float64)
    L, S = lam.shape
    budget = _c(np.asarray(budget), np.int32)
    assert budget.shape == (L,)
    omega = np.empty(L, np.float64)
    order = np.empty(L, np.int32)
    bits = np.empty(L, np.int32)
    st = _lib().qo_sensitivity_bits(_p(lam), L, S, _p(budget), int(reverse), _p(omega), _p(order), _p(bits))
    return st, omega, order, bits
