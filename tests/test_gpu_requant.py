"""int8 re-quantized output of the GEMM (qb_gemm_i8) and int8 row sums against the oracle, and two
linears chained with no fp32 tensor and no activation-quantizer pass between them."""
import numpy as np
import pytest
import torch

import oracle
import paper_1909_05840_b200 as qb
from paper_1909_05840_b200 import synth

import gpu_util as gu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ws():
    return qb.workspace(groups=4096)


def _check_codes(got: np.ndarray, o_y: np.ndarray, s_out: float):
    want = oracle.requantize_i8(o_y, s_out)
    bad = got != want
    if bad.any():
        # tolerated only one code apart and with the fp32 value within 1e-6 relative of the tie between them
        t = o_y[bad].astype(np.float64) / s_out
        assert np.all(np.abs(got[bad].astype(np.int64) - want[bad].astype(np.int64)) == 1)
        assert np.all(np.abs(t - 0.5 * (got[bad].astype(np.float64) + want[bad])) <= 1e-6 * np.abs(t) + 1e-9)


@pytest.mark.parametrize("bits", (2, 3, 4, 8))
@pytest.mark.parametrize("M,N,K,groups", [(200, 272, 384, 17), (515, 384, 768, 64), (131, 100, 256, 4), (64, 128, 128, 1)])
def test_gemm_i8_matches_oracle(ws, bits, M, N, K, groups):
    x = synth.activations(M, K, seed=51 * M + bits)
    w = synth.weights(N, K, seed=53 * N + bits)
    b = synth.bias(N, seed=57 * N + bits)
    xq, sc, rs = gu.gpu_quantize_act(x, ws)
    packed, delta, q0 = gu.gpu_quantize_weights(w, bits, groups, ws)
    o = oracle.linear(x, w, b, bits, groups)
    s_out = float(np.float32(np.abs(o["y"]).max() / 200.0))          # outputs beyond 127 steps saturate
    yq = gu.poison(torch.empty((M, N), dtype=torch.int8, device="cuda"))
    qb.gemm_i8(xq, sc, rs, packed, delta, q0, gu.dev(b), N, bits, groups, torch.tensor([s_out], device="cuda"), ws, yq=yq)
    assert qb.read_status(ws) == qb.QB_OK
    got = yq.cpu().numpy()
    _check_codes(got, o["y"], s_out)
    assert got.max() == 127 or got.min() == -127
    # row sums of the codes
    if N % 128 == 0:
        assert np.array_equal(qb.rowsum_i8(yq).cpu().numpy(), oracle.rowsum_i8(got))


def test_two_linears_chained_in_int8(ws):
    M, K, H, N, bits, G = 384, 256, 512, 256, 4, 8
    x = synth.activations(M, K, seed=5)
    w1, b1 = synth.weights(H, K, seed=6), synth.bias(H, seed=7)
    w2, b2 = synth.weights(N, H, seed=8), synth.bias(N, seed=9)
    o1 = oracle.linear(x, w1, b1, bits, G)
    s_mid = float(np.float32(np.abs(o1["y"]).max() / 127.0))
    xq, sc, rs = gu.gpu_quantize_act(x, ws)
    p1, d1, z1 = gu.gpu_quantize_weights(w1, bits, G, ws)
    p2, d2, z2 = gu.gpu_quantize_weights(w2, bits, G, ws)
    s_dev = torch.tensor([s_mid], device="cuda")
    hq = qb.gemm_i8(xq, sc, rs, p1, d1, z1, gu.dev(b1), H, bits, G, s_dev, ws)
    hrs = qb.rowsum_i8(hq)
    y = qb.gemm(hq, s_dev, hrs, p2, d2, z2, gu.dev(b2), N, bits, G, ws)
    assert qb.read_status(ws) == qb.QB_OK
    # oracle: the same chain
    o_hq = oracle.requantize_i8(o1["y"], s_mid)
    _check_codes(hq.cpu().numpy(), o1["y"], s_mid)
    st, c2, od2, oz2 = oracle.quantize_weights(w2, bits, G)
    o_hq_gpu = hq.cpu().numpy()                         # continue from the GPU's codes (equal unless a tie was tolerated)
    o_acc = oracle.int_gemm(o_hq_gpu, c2)
    o_y = oracle.dequant_epilogue(o_acc, oracle.rowsum_i8(o_hq_gpu), np.float32(s_mid), od2, oz2, b2, bits, G)
    gu.assert_y_close(y.cpu().numpy(), o_y)
    assert np.array_equal(hrs.cpu().numpy(), oracle.rowsum_i8(o_hq_gpu))
    assert (o_hq != o_hq_gpu).mean() < 1e-4


def test_rowsum_i8_matches_oracle():
    rng = np.random.default_rng(1)
    for M, K in ((1, 128), (37, 256), (1000, 768), (4096, 3072)):
        xq = rng.integers(-127, 128, (M, K)).astype(np.int8)
        got = qb.rowsum_i8(torch.from_numpy(xq).cuda()).cpu().numpy()
        assert np.array_equal(got, oracle.rowsum_i8(xq))


def test_layer_linears_i8_equals_single_calls(ws):
    # a small mixed-precision stack (side-by-side launches) with one output scale per linear
    M = 128
    shapes = [(256, 256, 2, 4), (384, 512, 4, 6), (128, 1024, 8, 2), (256, 256, 3, 1), (272, 384, 4, 17)]
    descs, scales, singles = [], [], []
    for i, (N, K, bits, G) in enumerate(shapes):
        x = synth.activations(M, K, seed=300 + i)
        w = synth.weights(N, K, seed=350 + i)
        b = synth.bias(N, seed=390 + i)
        xq, sc, rs = gu.gpu_quantize_act(x, ws)
        packed, delta, q0 = gu.gpu_quantize_weights(w, bits, G, ws)
        o = oracle.linear(x, w, b, bits, G)
        s_out = torch.tensor([float(np.float32(np.abs(o["y"]).max() / (90.0 + 10 * i)))], device="cuda")
        yq = gu.poison(torch.empty((M, N), dtype=torch.int8, device="cuda"))
        descs.append(qb.LinearDesc(xq, sc, rs, packed, delta, q0, gu.dev(b), N, bits, G, yq))
        scales.append(s_out)
        singles.append(qb.gemm_i8(xq, sc, rs, packed, delta, q0, gu.dev(b), N, bits, G, s_out, ws))
        _check_codes(singles[-1].cpu().numpy(), o["y"], float(s_out.item()))
    qb.layer_linears_i8(descs, scales, ws)
    assert qb.read_status(ws) == qb.QB_OK
    for d, y1 in zip(descs, singles):
        assert torch.equal(d.y, y1)


def test_gemm_i8_large_launch_ragged(ws):
    # a launch large enough for the CTA-pair kernel (256 x 256 tiles), ragged in M and N: int8 outputs through
    # TMA stores (N % 16 == 0) must equal the oracle's re-quantization of the oracle's fp32 result
    M, N, K, bits, G = 2500, 2448, 384, 4, 12
    x = synth.activations(M, K, seed=71)
    w = synth.weights(N, K, seed=72)
    b = synth.bias(N, seed=73)
    o = oracle.linear(x, w, b, bits, G, omp=True)
    xq, sc, rs = gu.gpu_quantize_act(x, ws)
    packed, delta, q0 = gu.gpu_quantize_weights(w, bits, G, ws)
    s_out = float(np.float32(np.abs(o["y"]).max() / 127.0))
    yq = qb.gemm_i8(xq, sc, rs, packed, delta, q0, gu.dev(b), N, bits, G, torch.tensor([s_out], device="cuda"), ws)
    assert qb.read_status(ws) == qb.QB_OK
    _check_codes(yq.cpu().numpy(), o["y"], s_out)
