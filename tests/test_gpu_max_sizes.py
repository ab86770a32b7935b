"""GPU parity at the largest inner dimension the interface allows (K = QB_MAX_K = 65536: 512 K blocks per
tile, 512 units per weight row) and with the operands that drive the int32 accumulators as far as they go.

|acc| <= 127 * (2^k - 1) * K; with 8-bit codes and K = 65536 that is 2.12e9 < 2^31: the bound the header
states.  The tensor cores are fed (code - 128) as s8 and the epilogue adds 128 * rowsum back, so the test
with every activation at +-127 and every code at 0 or 255 also drives the recentred sum to its extremes.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_1909_05840_b200 as qb
from paper_1909_05840_b200 import synth

import gpu_util as gu

pytestmark = pytest.mark.gpu

MAX_K = 65536


@pytest.fixture(scope="module")
def ws():
    return qb.workspace(groups=256)


def test_quantizers_at_max_k(ws):
    # activations: three rows of 65536; weights: rows of 512 units in groups held by a cluster of four CTAs
    # (2 rows per group), by a cluster of two (1 row per group), and by the two passes (one range per tensor)
    x = synth.activations(3, MAX_K, seed=1)
    xq, sc, rs = gu.gpu_quantize_act(x, ws)
    st, o_xq, o_s, o_rs = oracle.quantize_act(x)
    assert st == oracle.OK and np.array_equal(xq.cpu().numpy(), o_xq) and np.array_equal(rs.cpu().numpy(), o_rs)
    assert sc.item() == o_s
    w = synth.weights(8, MAX_K, seed=2)
    for bits, groups in ((2, 4), (3, 8), (4, 1), (8, 2)):
        packed, delta, q0 = gu.gpu_quantize_weights(w, bits, groups, ws)
        st, codes, o_delta, o_q0 = oracle.quantize_weights(w, bits, groups)
        assert st == oracle.OK
        assert np.array_equal(gu.words_np(packed), oracle.pack(codes, bits)), (bits, groups)
        assert np.array_equal(delta.cpu().numpy(), o_delta) and np.array_equal(q0.cpu().numpy(), o_q0)
    assert qb.read_status(ws) == qb.QB_OK


@pytest.mark.parametrize("bits", (2, 3, 4, 8))
def test_linear_at_max_k(ws, bits):
    # one ragged token tile and two neuron tiles, 512 K blocks each: the ring and both accumulator phases wrap
    # hundreds of times; every stage against the oracle
    M, N, G = 130, 136, 8
    x = synth.activations(M, MAX_K, seed=10 + bits)
    w = synth.weights(N, MAX_K, seed=20 + bits)
    b = synth.bias(N, seed=30 + bits)
    gu.check_linear(x, w, b, bits, G, ws, use_omp=True)


def test_accumulators_at_their_bound(ws):
    # every activation +-127, every 8-bit code 0 or 255, K = 65536: sums of up to 127 * 255 * 65536
    M, N, K, bits, G = 64, 128, MAX_K, 8, 1
    rng = np.random.default_rng(3)
    xq_h = np.where(rng.random((M, K)) < 0.5, -127, 127).astype(np.int8)
    xq_h[0] = 127          # the all-positive row against an all-255 neuron: the largest sum there is
    xq_h[1] = -127
    codes = np.where(rng.random((N, K)) < 0.5, 0, 255).astype(np.uint8)
    codes[0] = 255
    codes[1] = 0
    xq = torch.from_numpy(xq_h).cuda()
    rs_h = xq_h.astype(np.int64).sum(axis=1).astype(np.int32)
    rs = torch.from_numpy(rs_h).cuda()
    sc = torch.tensor([0.01], dtype=torch.float32, device="cuda")
    packed = torch.from_numpy(oracle.pack(codes, bits).view(np.int32)).cuda()
    delta = torch.tensor([0.002], dtype=torch.float32, device="cuda")
    q0 = torch.tensor([-0.25], dtype=torch.float32, device="cuda")
    y = gu.poison(torch.empty((M, N), dtype=torch.float32, device="cuda"))
    acc = gu.poison(torch.empty((M, N), dtype=torch.int32, device="cuda"))
    qb.gemm(xq, sc, rs, packed, delta, q0, None, N, bits, G, ws, y=y, acc_out=acc)
    assert qb.read_status(ws) == qb.QB_OK
    o_acc = oracle.int_gemm(xq_h, codes, omp=True)
    assert int(np.abs(o_acc.astype(np.int64)).max()) == 127 * 255 * K          # 2,122,383,360 < 2^31
    assert np.array_equal(acc.cpu().numpy(), o_acc)
    o_y = oracle.dequant_epilogue(o_acc, rs_h, np.float32(0.01), delta.cpu().numpy(), q0.cpu().numpy(), None, bits, G)
    gu.assert_y_close(y.cpu().numpy(), o_y)


def test_a_million_rows():
    # M = N = 2^20 at the smallest K: row counts far beyond one wave of any kernel, one range per weight row
    # (18 groups per warp, thousands of CTA items), a million token rows through 4,096 token tiles of one linear
    R, K = 1 << 20, 128
    ws_big = qb.workspace(groups=R)
    w = synth.weights(R, K, seed=5)
    packed, delta, q0 = gu.gpu_quantize_weights(w, 4, R, ws_big)
    st, codes, o_delta, o_q0 = oracle.quantize_weights(w, 4, R, omp=True)
    assert st == oracle.OK and qb.read_status(ws_big) == qb.QB_OK
    assert np.array_equal(gu.words_np(packed), oracle.pack(codes, 4))
    assert np.array_equal(delta.cpu().numpy(), o_delta) and np.array_equal(q0.cpu().numpy(), o_q0)
    del packed, delta, q0, codes
    x = synth.activations(R, K, seed=6)
    w2 = synth.weights(128, K, seed=7)
    b2 = synth.bias(128, seed=8)
    rows = gu.sample_rows(R, tile=256, per_tile=1, seed=9)
    gu.check_linear(x, w2, b2, 3, 16, ws_big, rows=rows[:: max(1, len(rows) // 2048)], use_omp=True)
