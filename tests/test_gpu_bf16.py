"""Narrow-output epilogue on the GPU: qb_gemm_bf16 / qb_layer_linears_bf16 against the oracle.

The oracle evaluates the fp32 epilogue and rounds it to bfloat16 (round to nearest even); the GPU does
the same two steps, so the 16-bit patterns are compared bit for bit.  The fp32 gate of the library is
1e-6 relative; should an fp32 value ever differ in its last bits, its bfloat16 pattern may differ only
when that value sits within 1e-6 relative of a rounding boundary, which the check reports separately."""
import numpy as np
import pytest
import torch

import oracle
import paper_1909_05840_b200 as qb
from paper_1909_05840_b200 import synth

import gpu_util as gu

pytestmark = pytest.mark.gpu

BITS = (2, 3, 4, 8)


@pytest.fixture(scope="module")
def ws():
    return qb.workspace(groups=4096)


def _bf16_bits(t: torch.Tensor) -> np.ndarray:
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def _assert_bf16_equal(got: np.ndarray, o_y: np.ndarray):
    want = oracle.round_bf16(o_y)
    bad = got != want
    if bad.any():
        # tolerated only next to a rounding boundary (one step apart and the fp32 value within 1e-6 of the tie)
        y = o_y[bad].astype(np.float64)
        lo = (np.minimum(got[bad], want[bad]).astype(np.uint32) << 16).view(np.float32).astype(np.float64)
        hi = (np.maximum(got[bad], want[bad]).astype(np.uint32) << 16).view(np.float32).astype(np.float64)
        one_step = np.abs(got[bad].astype(np.int64) - want[bad].astype(np.int64)) == 1
        near_tie = np.abs(y - 0.5 * (lo + hi)) <= 1e-6 * np.abs(y)
        assert np.all(one_step & near_tie), f"{int(bad.sum())} bfloat16 outputs differ away from a tie"


@pytest.mark.parametrize("bits", BITS)
@pytest.mark.parametrize("M,N,K,groups", [
    (200, 264, 384, 11),     # ragged everywhere, N % 8 == 0: TMA store path
    (515, 384, 768, 64),     # several token tiles and a ragged tail
    (131, 100, 256, 4),      # N % 8 != 0: direct 16-bit stores
    (64, 128, 128, 1),
])
def test_gemm_bf16_matches_oracle(ws, bits, M, N, K, groups):
    x = synth.activations(M, K, seed=31 * M + bits)
    w = synth.weights(N, K, seed=37 * N + bits)
    b = synth.bias(N, seed=41 * N + bits)
    xq, sc, rs = gu.gpu_quantize_act(x, ws)
    packed, delta, q0 = gu.gpu_quantize_weights(w, bits, groups, ws)
    y16 = gu.poison(torch.empty((M, N), dtype=torch.bfloat16, device="cuda"))
    qb.gemm_bf16(xq, sc, rs, packed, delta, q0, gu.dev(b), N, bits, groups, ws, y=y16)
    y32 = qb.gemm(xq, sc, rs, packed, delta, q0, gu.dev(b), N, bits, groups, ws)
    assert qb.read_status(ws) == qb.QB_OK
    st_a, o_xq, o_s, o_rs = oracle.quantize_act(x)
    st_w, codes, o_delta, o_q0 = oracle.quantize_weights(w, bits, groups)
    o_acc = oracle.int_gemm(o_xq, codes)
    o_y = oracle.dequant_epilogue(o_acc, o_rs, o_s, o_delta, o_q0, b, bits, groups)
    _assert_bf16_equal(_bf16_bits(y16), o_y)
    # and against the library's own fp32 result, converted by a library routine
    assert torch.equal(y16, y32.to(torch.bfloat16))


def test_gemm_bf16_without_bias_wide_tiles(ws):
    M, N, K, bits, groups = 1100, 256, 512, 4, 8
    x = np.abs(synth.activations(M, K, seed=77))
    w = synth.weights(N, K, seed=78)
    xq, sc, rs = gu.gpu_quantize_act(x, ws)
    packed, delta, q0 = gu.gpu_quantize_weights(w, bits, groups, ws)
    y16 = qb.gemm_bf16(xq, sc, rs, packed, delta, q0, None, N, bits, groups, ws)
    st_a, o_xq, o_s, o_rs = oracle.quantize_act(x, omp=True)
    st_w, codes, o_delta, o_q0 = oracle.quantize_weights(w, bits, groups, omp=True)
    o_y = oracle.dequant_epilogue(oracle.int_gemm(o_xq, codes, omp=True), o_rs, o_s, o_delta, o_q0, None, bits, groups)
    _assert_bf16_equal(_bf16_bits(y16), o_y)


def test_layer_linears_bf16_equals_single_calls_and_oracle(ws):
    # a small mixed-precision stack (side-by-side launches) and the config-1 layer at full size, sampled
    M = 128
    shapes = [(256, 256, 2, 4), (384, 512, 4, 6), (128, 1024, 8, 2), (256, 256, 3, 1)]
    descs, refs = [], []
    for i, (N, K, bits, G) in enumerate(shapes):
        x = synth.activations(M, K, seed=700 + i)
        w = synth.weights(N, K, seed=750 + i)
        b = synth.bias(N, seed=790 + i)
        xq, sc, rs = gu.gpu_quantize_act(x, ws)
        packed, delta, q0 = gu.gpu_quantize_weights(w, bits, G, ws)
        y = gu.poison(torch.empty((M, N), dtype=torch.bfloat16, device="cuda"))
        descs.append(qb.LinearDesc(xq, sc, rs, packed, delta, q0, gu.dev(b), N, bits, G, y))
        refs.append((x, w, b, bits, G))
    qb.layer_linears_bf16(descs, ws)
    assert qb.read_status(ws) == qb.QB_OK
    for d, (x, w, b, bits, G) in zip(descs, refs):
        y1 = qb.gemm_bf16(d.xq, d.act_scale, d.rowsum, d.packed, d.delta, d.q0, d.bias, d.N, bits, G, ws)
        assert torch.equal(y1, d.y)
        o = oracle.linear(x, w, b, bits, G)
        _assert_bf16_equal(_bf16_bits(d.y), o["y"])


def test_config1_layer_bf16_sampled(ws):
    wl = synth.workload(1)
    descs, refs = [], []
    for mi, s in enumerate(wl.linears):
        seed = synth.seed_for(wl.config, 0, mi)
        x = synth.activations(wl.M, s.K, seed)
        w = synth.weights(s.N, s.K, seed)
        b = synth.bias(s.N, seed)
        xq, sc, rs = gu.gpu_quantize_act(x, ws)
        packed, delta, q0 = gu.gpu_quantize_weights(w, wl.bits[0], s.groups, ws)
        y = gu.poison(torch.empty((wl.M, s.N), dtype=torch.bfloat16, device="cuda"))
        descs.append(qb.LinearDesc(xq, sc, rs, packed, delta, q0, gu.dev(b), s.N, wl.bits[0], s.groups, y))
        refs.append((x, w, b, s))
    qb.layer_linears_bf16(descs, ws)
    assert qb.read_status(ws) == qb.QB_OK
    for d, (x, w, b, s) in zip(descs, refs):
        rows = gu.sample_rows(wl.M, per_tile=2, seed=s.N)
        st_a, o_xq, o_s, o_rs = oracle.quantize_act(x, omp=True)
        st_w, codes, o_delta, o_q0 = oracle.quantize_weights(w, wl.bits[0], s.groups, omp=True)
        o_acc = oracle.int_gemm(o_xq[rows], codes, omp=True)
        o_y = oracle.dequant_epilogue(o_acc, o_rs[rows], o_s, o_delta, o_q0, b, wl.bits[0], s.groups)
        got = _bf16_bits(d.y[torch.from_numpy(rows).cuda()])
        _assert_bf16_equal(got, o_y)
