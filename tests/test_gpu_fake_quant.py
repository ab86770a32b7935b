"""Fake quantization (forward Q(W) in fp32) and the straight-through backward on the GPU, against the
oracle: both are bit-exact (the forward runs the same IEEE operations in the same order; the backward
only selects)."""
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


@pytest.mark.parametrize("bits", (2, 3, 4, 8))
@pytest.mark.parametrize("N,K,groups", [(768, 768, 12), (264, 384, 11), (96, 3072, 96), (128, 128, 1), (3072, 768, 128),
                                        (70, 256, 70),     # two units per group: nine groups per warp, a last warp with fewer
                                        (12, 30720, 2),    # 1,440 units per group: a cluster of five CTAs
                                        (74, 8192, 2)])    # 2,368 units per group: the two-pass path
def test_fake_quantize_matches_oracle(ws, bits, N, K, groups):
    w = synth.weights(N, K, seed=3 * N + K + groups + bits)
    wq = gu.poison(torch.empty((N, K), dtype=torch.float32, device="cuda"))
    wq, delta, q0 = qb.fake_quantize_weights(gu.dev(w), bits, groups, ws, wq=wq)
    assert qb.read_status(ws) == qb.QB_OK
    st, o_q, o_delta, o_q0 = oracle.fake_quantize_weights(w, bits, groups)
    assert st == oracle.OK
    assert np.array_equal(delta.cpu().numpy(), o_delta) and np.array_equal(q0.cpu().numpy(), o_q0)
    assert np.array_equal(wq.cpu().numpy().view(np.uint32), o_q.view(np.uint32))
    # and it is the dequantized form of what the packer stores
    packed, d2, z2 = qb.quantize_pack_weights(gu.dev(w), bits, groups, ws)
    codes = oracle.unpack(gu.words_np(packed), K, bits)
    assert np.array_equal(oracle.dequantize_weights(codes, groups, d2.cpu().numpy(), z2.cpu().numpy()).view(np.uint32),
                          wq.cpu().numpy().view(np.uint32))


def test_fake_quantize_clipped_ranges_constant_group_and_nonfinite(ws):
    N, K, G = 64, 256, 4
    w = synth.weights(N, K, seed=21)
    w[16:32] = 0.25                                   # a constant group
    lo = np.quantile(w.reshape(G, -1), 0.02, axis=1).astype(np.float32)
    hi = np.quantile(w.reshape(G, -1), 0.98, axis=1).astype(np.float32)
    for bits in (2, 3, 4, 8):
        wq, delta, q0 = qb.fake_quantize_weights(gu.dev(w), bits, G, ws)
        st, o_q, o_delta, o_q0 = oracle.fake_quantize_weights(w, bits, G)
        assert np.array_equal(wq.cpu().numpy().view(np.uint32), o_q.view(np.uint32))
        assert delta.cpu().numpy()[1] == 1.0 and np.all(wq.cpu().numpy()[16:32] == 0.25)
        wq, delta, q0 = qb.fake_quantize_weights(gu.dev(w), bits, G, ws, gu.dev(lo), gu.dev(hi))
        st, o_q, o_delta, o_q0 = oracle.fake_quantize_weights(w, bits, G, lo, hi)
        assert np.array_equal(wq.cpu().numpy().view(np.uint32), o_q.view(np.uint32))
        assert np.array_equal(delta.cpu().numpy(), o_delta) and np.array_equal(q0.cpu().numpy(), o_q0)
    assert qb.read_status(ws) == qb.QB_OK
    bad = w.copy(); bad[3, 7] = np.inf
    ws2 = qb.workspace(groups=64)
    qb.fake_quantize_weights(gu.dev(bad), 4, G, ws2)
    assert qb.read_status(ws2) == qb.QB_ERR_NONFINITE


def test_fake_quantize_batch_equals_single_calls_and_the_oracle():
    # a stack in one call: mixed bit widths, groups held by one CTA, by clusters, several per warp, caller
    # ranges, and one matrix whose groups take the two passes
    shapes = [(768, 768, 4, 128, False), (3072, 768, 2, 128, False), (768, 3072, 3, 128, False), (70, 256, 8, 70, False),
              (768, 768, 3, 12, False), (12, 30720, 4, 2, False), (74, 8192, 2, 2, False), (264, 384, 4, 11, True),
              (768, 768, 8, 1, True)]
    ws_big = qb.workspace(groups=4096)
    arr = (qb.WeightDescC * len(shapes))()
    keep, host = [], []
    for i, (N, K, bits, G, ranged) in enumerate(shapes):
        w = synth.weights(N, K, seed=17 * i + N + K + G)
        lo = hi = None
        if ranged:
            lo = np.quantile(w.reshape(G, -1), 0.03, axis=1).astype(np.float32)
            hi = np.quantile(w.reshape(G, -1), 0.97, axis=1).astype(np.float32)
        wd = gu.dev(w)
        wq = gu.poison(torch.empty((N, K), dtype=torch.float32, device="cuda"))
        dl = gu.poison(torch.empty(G, dtype=torch.float32, device="cuda"))
        z0 = gu.poison(torch.empty(G, dtype=torch.float32, device="cuda"))
        lod, hid = (gu.dev(lo), gu.dev(hi)) if ranged else (None, None)
        arr[i] = qb.WeightDescC(wd.data_ptr(), N, K, bits, G, lod.data_ptr() if ranged else None,
                                hid.data_ptr() if ranged else None, wq.data_ptr(), dl.data_ptr(), z0.data_ptr())
        keep.append((wd, wq, dl, z0, lod, hid))
        host.append((w, lo, hi))
    qb.fake_quantize_weights_batch(arr, ws_big)
    assert qb.read_status(ws_big) == qb.QB_OK
    for (N, K, bits, G, ranged), (wd, wq, dl, z0, lod, hid), (w, lo, hi) in zip(shapes, keep, host):
        st, o_q, o_delta, o_q0 = oracle.fake_quantize_weights(w, bits, G, lo, hi)
        assert st == oracle.OK
        assert np.array_equal(wq.cpu().numpy().view(np.uint32), o_q.view(np.uint32)), (N, K, bits, G)
        assert np.array_equal(dl.cpu().numpy(), o_delta) and np.array_equal(z0.cpu().numpy(), o_q0)
        one, d1, z1 = qb.fake_quantize_weights(wd, bits, G, ws_big, lod, hid)
        assert torch.equal(one, wq) and torch.equal(d1, dl) and torch.equal(z1, z0)


def test_fake_quantize_products_that_round_onto_ties(ws):
    # weights within a few ulp of the midpoints between grid points (see the packer's test of the same name)
    N, K, G, bits = 96, 1152, 12, 4
    rng = np.random.default_rng(5)
    L = (1 << bits) - 1
    w = np.empty((N, K), np.float32)
    R = N // G
    for g in range(G):
        lo = np.float32(-0.05 - 0.02 * rng.random())
        hi = np.float32(0.04 + 0.03 * rng.random())
        d = np.float32((hi - lo) / np.float32(L))
        m = rng.integers(0, L, size=(R, K)).astype(np.float32)
        x = (lo + (m + np.float32(0.5)) * d).astype(np.float32)
        x = (x.view(np.int32) + rng.integers(-4, 5, size=x.shape).astype(np.int32)).view(np.float32)
        x[0, 0], x[0, 1] = lo, hi
        w[g * R:(g + 1) * R] = np.clip(x, lo, hi)
    wq, delta, q0 = qb.fake_quantize_weights(gu.dev(w), bits, G, ws)
    st, o_q, o_delta, o_q0 = oracle.fake_quantize_weights(w, bits, G)
    assert st == oracle.OK and qb.read_status(ws) == qb.QB_OK
    assert np.array_equal(wq.cpu().numpy().view(np.uint32), o_q.view(np.uint32))


@pytest.mark.parametrize("N,K,groups", [(768, 768, 12), (264, 384, 11), (3072, 768, 128), (8, 128, 1)])
def test_ste_backward_matches_oracle(N, K, groups):
    rng = np.random.default_rng(N + K)
    w = synth.weights(N, K, seed=N + groups)
    grad = rng.standard_normal((N, K)).astype(np.float32)
    lo = np.quantile(w.reshape(groups, -1), 0.05, axis=1).astype(np.float32)
    hi = np.quantile(w.reshape(groups, -1), 0.95, axis=1).astype(np.float32)
    w[0, 0], w[0, 1] = lo[0], hi[0]                  # the ends of the range count as inside
    out = gu.poison(torch.empty((N, K), dtype=torch.float32, device="cuda"))
    qb.ste_backward(gu.dev(grad), gu.dev(w), groups, gu.dev(lo), gu.dev(hi), grad_w=out)
    ref = oracle.ste_backward(grad, w, groups, lo, hi)
    assert np.array_equal(out.cpu().numpy().view(np.uint32), ref.view(np.uint32))
    assert 0 < (ref == 0).sum() < ref.size
    # default range: the gradient passes unchanged, also in place
    out2 = qb.ste_backward(gu.dev(grad), gu.dev(w), groups)
    assert np.array_equal(out2.cpu().numpy(), grad)
    g_dev = gu.dev(grad)
    assert qb.ste_backward(g_dev, gu.dev(w), groups, grad_w=g_dev) is g_dev and np.array_equal(g_dev.cpu().numpy(), grad)
    # masked in place
    g_dev = gu.dev(grad)
    qb.ste_backward(g_dev, gu.dev(w), groups, gu.dev(lo), gu.dev(hi), grad_w=g_dev)
    assert np.array_equal(g_dev.cpu().numpy(), ref)
