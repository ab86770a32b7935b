"""Helpers shared by the GPU parity tests: run the CUDA path through the binding and compare it
with the CPU oracle on the same arrays."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import paper_1909_05840_b200 as qb
from paper_1909_05840_b200 import build as qb_build

Y_RTOL = 1e-6  # fp32 outputs: relative tolerance of the parity gate


def ensure_built():
    qb_build.build()
    return qb.lib()


def dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def poison(t: torch.Tensor) -> torch.Tensor:
    """Fill an output buffer with 0xFF bytes so that unwritten elements are caught."""
    t.view(torch.uint8).fill_(0xFF)
    return t


def gpu_quantize_act(x: np.ndarray, ws):
    xd = dev(x)
    M, K = x.shape
    xq = poison(torch.empty((M, K), dtype=torch.int8, device="cuda"))
    sc = poison(torch.empty(1, dtype=torch.float32, device="cuda"))
    rs = poison(torch.empty(M, dtype=torch.int32, device="cuda"))
    qb.quantize_act(xd, ws, xq, sc, rs)
    return xq, sc, rs


def gpu_quantize_weights(w: np.ndarray, bits: int, groups: int, ws, range_lo=None, range_hi=None):
    wd = dev(w)
    N, K = w.shape
    packed = poison(torch.empty((N, K * bits // 32), dtype=torch.int32, device="cuda"))
    delta = poison(torch.empty(groups, dtype=torch.float32, device="cuda"))
    q0 = poison(torch.empty(groups, dtype=torch.float32, device="cuda"))
    lo = None if range_lo is None else dev(range_lo)
    hi = None if range_hi is None else dev(range_hi)
    qb.quantize_pack_weights(wd, bits, groups, ws, lo, hi, packed, delta, q0)
    return packed, delta, q0


def words_np(packed: torch.Tensor) -> np.ndarray:
    return packed.cpu().numpy().view(np.uint32)


def assert_y_close(y_gpu: np.ndarray, y_ref: np.ndarray):
    """Spec tolerance: |y_gpu - y_ref| <= 1e-6 * |y_ref| element by element."""
    diff = np.abs(y_gpu.astype(np.float64) - y_ref.astype(np.float64))
    tol = Y_RTOL * np.abs(y_ref.astype(np.float64))
    bad = diff > tol
    assert not bad.any(), (f"{int(bad.sum())} of {bad.size} outputs differ by more than 1e-6 relative; "
                           f"worst abs diff {diff.max():.3e}")


def check_linear(x, w, b, bits, groups, ws, rows=None, use_omp=False):
    """Run quantize_act -> quantize_pack_weights -> gemm on the GPU and compare every stage with the
    oracle.  ``rows``: optional subset of token rows on which accumulators and outputs are compared
    (all quantizer outputs are always compared in full)."""
    M, K = x.shape
    N = w.shape[0]
    xq, sc, rs = gpu_quantize_act(x, ws)
    packed, delta, q0 = gpu_quantize_weights(w, bits, groups, ws)
    bd = None if b is None else dev(b)
    y = poison(torch.empty((M, N), dtype=torch.float32, device="cuda"))
    acc = poison(torch.empty((M, N), dtype=torch.int32, device="cuda"))
    qb.gemm(xq, sc, rs, packed, delta, q0, bd, N, bits, groups, ws, y=y, acc_out=acc)
    assert qb.read_status(ws) == qb.QB_OK

    st_a, o_xq, o_s, o_rs = oracle.quantize_act(x, omp=use_omp)
    st_w, o_codes, o_delta, o_q0 = oracle.quantize_weights(w, bits, groups, omp=use_omp)
    assert st_a == oracle.OK and st_w == oracle.OK
    o_words = oracle.pack(o_codes, bits)

    # integer / byte work: bit exact
    assert np.array_equal(xq.cpu().numpy(), o_xq), "activation codes differ"
    assert np.array_equal(rs.cpu().numpy(), o_rs), "row sums differ"
    assert sc.cpu().numpy()[0] == o_s, "activation scale differs"
    assert np.array_equal(words_np(packed), o_words), "packed weight words differ"
    assert np.array_equal(delta.cpu().numpy(), o_delta), "Delta differs"
    assert np.array_equal(q0.cpu().numpy(), o_q0), "q0 differs"

    if rows is None:
        sel = slice(None)
        o_acc = oracle.int_gemm(o_xq, o_codes, omp=use_omp)
        o_y = oracle.dequant_epilogue(o_acc, o_rs, o_s, o_delta, o_q0, b, bits, groups)
        acc_g, y_g = acc.cpu().numpy(), y.cpu().numpy()
    else:
        sel = np.asarray(rows)
        o_acc = oracle.int_gemm(o_xq[sel], o_codes, omp=use_omp)
        o_y = oracle.dequant_epilogue(o_acc, o_rs[sel], o_s, o_delta, o_q0, b, bits, groups)
        idx = torch.from_numpy(sel).cuda()
        acc_g, y_g = acc[idx].cpu().numpy(), y[idx].cpu().numpy()
    assert np.array_equal(acc_g, o_acc), "int32 accumulators differ"
    assert_y_close(y_g, o_y)
    return dict(xq=xq, act_scale=sc, rowsum=rs, packed=packed, delta=delta, q0=q0, y=y, acc=acc,
                exact_y=bool(np.array_equal(y_g, o_y)))


def sample_rows(M: int, tile: int = 256, per_tile: int = 2, seed: int = 0) -> np.ndarray:
    """Rows covering the first and last token tile completely-ish and every tile residue sparsely."""
    rng = np.random.default_rng(seed)
    rows = set(range(min(M, 4))) | set(range(max(0, M - 4), M))
    for t0 in range(0, M, tile):
        hi = min(M, t0 + tile)
        rows |= set(int(r) for r in rng.integers(t0, hi, size=per_tile))
    return np.array(sorted(rows), dtype=np.int64)
