"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by element.

Integer results (activation codes, row sums, packed words, int32 accumulators) must be bit exact;
fp32 outputs must agree within 1e-6 relative.
"""
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
    gu.ensure_built()
    return qb.workspace(groups=8192)


# ------------------------------------------------------------------ quantizers alone
@pytest.mark.parametrize("M,K", [(1, 128), (7, 256), (300, 384), (1024, 768), (129, 3072)])
def test_quantize_act_matches_oracle(ws, M, K):
    x = synth.activations(M, K, seed=M + K)
    xq, sc, rs = gu.gpu_quantize_act(x, ws)
    st, o_xq, o_s, o_rs = oracle.quantize_act(x)
    assert qb.read_status(ws) == qb.QB_OK
    assert np.array_equal(xq.cpu().numpy(), o_xq)
    assert np.array_equal(rs.cpu().numpy(), o_rs)
    assert sc.cpu().numpy()[0] == o_s


def test_quantize_act_ties_zero_and_nonfinite(ws):
    # exact midpoints (a = 127 makes x*inv = x): half-to-even on both sides
    x = np.zeros((2, 128), np.float32)
    x[0, :8] = [127.0, -127.0, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5]
    xq, sc, rs = gu.gpu_quantize_act(x, ws)
    st, o_xq, o_s, o_rs = oracle.quantize_act(x)
    assert xq.cpu().numpy()[0, :8].tolist() == [127, -127, 0, 2, 2, 0, -2, -2]
    assert np.array_equal(xq.cpu().numpy(), o_xq) and sc.cpu().numpy()[0] == o_s == 1.0
    # all-zero tensor: scale 1, zero codes
    xq, sc, rs = gu.gpu_quantize_act(np.zeros((3, 128), np.float32), ws)
    assert sc.item() == 1.0 and not xq.any().item() and not rs.any().item()
    assert qb.read_status(ws) == qb.QB_OK
    # NaN / Inf: reported through the status word of the workspace, as the oracle reports it
    for bad in (np.nan, np.inf, -np.inf):
        ws2 = qb.workspace(groups=16)
        x = synth.activations(5, 128, seed=3)
        x[4, 100] = bad
        gu.gpu_quantize_act(x, ws2)
        assert qb.read_status(ws2) == qb.QB_ERR_NONFINITE
        assert oracle.quantize_act(x)[0] == oracle.ERR_NONFINITE


@pytest.mark.parametrize("bits", BITS)
@pytest.mark.parametrize("N,K,groups", [(12, 128, 1), (12, 128, 12), (24, 384, 4), (768, 768, 128),
                                        (768, 768, 12), (264, 256, 11), (96, 3072, 96), (768, 768, 1)])
def test_quantize_pack_weights_matches_oracle(ws, bits, N, K, groups):
    w = synth.weights(N, K, seed=N + K + groups + bits)
    packed, delta, q0 = gu.gpu_quantize_weights(w, bits, groups, ws)
    assert qb.read_status(ws) == qb.QB_OK
    st, codes, o_delta, o_q0 = oracle.quantize_weights(w, bits, groups)
    assert np.array_equal(gu.words_np(packed), oracle.pack(codes, bits))
    assert np.array_equal(delta.cpu().numpy(), o_delta)
    assert np.array_equal(q0.cpu().numpy(), o_q0)
    # run-to-run determinism (order-independent integer reductions): any difference would be a race
    packed2, delta2, q02 = gu.gpu_quantize_weights(w, bits, groups, ws)
    assert torch.equal(packed, packed2) and torch.equal(delta, delta2) and torch.equal(q0, q02)


@pytest.mark.parametrize("bits", BITS)
@pytest.mark.parametrize("N,K,groups", [
    (2304, 768, 384),    # more groups than SMs, 36 units per group: teams of two warps
    (2560, 1536, 80),    # 384 units per group: clusters of two CTAs, more groups than resident clusters
    (2640, 1536, 80),    # 396 units per group: clusters of two, ragged slices
    (2048, 9600, 512),   # 300 units per group: clusters of two, seven items per cluster
    (296, 128, 148),     # two units per group
])
def test_quantize_weights_single_read_shapes(bits, N, K, groups):
    ws_big = qb.workspace(groups=1024)
    w = synth.weights(N, K, seed=7 * N + K + groups + bits)
    packed, delta, q0 = gu.gpu_quantize_weights(w, bits, groups, ws_big)
    assert qb.read_status(ws_big) == qb.QB_OK
    st, codes, o_delta, o_q0 = oracle.quantize_weights(w, bits, groups)
    assert np.array_equal(gu.words_np(packed), oracle.pack(codes, bits))
    assert np.array_equal(delta.cpu().numpy(), o_delta)
    assert np.array_equal(q0.cpu().numpy(), o_q0)


@pytest.mark.parametrize("bits,shapes", [
    # thirteen matrices of 384-unit groups (clusters of two): 156 groups on 74 resident clusters
    (4, [(768, 768, 12)] * 13),
    # group sizes from 6 to 240 units in one launch, hundreds of groups per CTA
    (3, [(768, 768, 768), (768, 7680, 768), (3072, 768, 768), (768, 768, 128), (768, 3072, 768)]),
    (2, [(768, 768, 128), (3072, 768, 128), (768, 3072, 128), (2304, 768, 384)] * 3),
])
def test_quantize_weights_single_read_batches(bits, shapes):
    ws_big = qb.workspace(groups=8192)
    items, host = [], []
    for i, (N, K, G) in enumerate(shapes):
        w = synth.weights(N, K, seed=31 * i + N + K + G)
        packed = gu.poison(torch.empty((N, K * bits // 32), dtype=torch.int32, device="cuda"))
        delta = gu.poison(torch.empty(G, dtype=torch.float32, device="cuda"))
        q0 = gu.poison(torch.empty(G, dtype=torch.float32, device="cuda"))
        items.append((gu.dev(w), bits, G, packed, delta, q0))
        host.append(w)
    for _ in range(3):  # repeated: a race between teams would not show every time
        qb.quantize_pack_weights_batch(items, ws_big)
    assert qb.read_status(ws_big) == qb.QB_OK
    for (wd, _, G, packed, delta, q0), w in zip(items, host):
        st, codes, o_delta, o_q0 = oracle.quantize_weights(w, bits, G)
        assert np.array_equal(gu.words_np(packed), oracle.pack(codes, bits))
        assert np.array_equal(delta.cpu().numpy(), o_delta)
        assert np.array_equal(q0.cpu().numpy(), o_q0)


def test_quantize_weights_single_read_edge_cases():
    # enough small groups for the single-read path: constant groups, caller ranges, non-finite input
    N, K, G = 256, 128, 128
    w = synth.weights(N, K, seed=11)
    w[:2] = -0.25
    w[4, :8] = [0.0, 0.5, 1.5, 2.5, 3.0, 1.0, 2.0, 0.25]
    w[4, 8:] = 1.0
    w[5] = w[4]
    ws1 = qb.workspace(groups=G)
    for bits in BITS:
        packed, delta, q0 = gu.gpu_quantize_weights(w, bits, G, ws1)
        st, codes, o_delta, o_q0 = oracle.quantize_weights(w, bits, G)
        assert np.array_equal(gu.words_np(packed), oracle.pack(codes, bits))
        assert np.array_equal(delta.cpu().numpy(), o_delta) and np.array_equal(q0.cpu().numpy(), o_q0)
        assert delta.cpu().numpy()[0] == 1.0
        lo = np.linspace(-0.05, -0.01, G).astype(np.float32)
        hi = np.linspace(0.02, 0.06, G).astype(np.float32)
        packed, delta, q0 = gu.gpu_quantize_weights(w, bits, G, ws1, lo, hi)
        st, codes, o_delta, o_q0 = oracle.quantize_weights(w, bits, G, lo, hi)
        assert st == oracle.OK
        assert np.array_equal(gu.words_np(packed), oracle.pack(codes, bits))
        assert np.array_equal(delta.cpu().numpy(), o_delta) and np.array_equal(q0.cpu().numpy(), o_q0)
    assert qb.read_status(ws1) == qb.QB_OK
    ws2 = qb.workspace(groups=G)
    w[200, 77] = np.inf
    gu.gpu_quantize_weights(w, 3, G, ws2)
    assert qb.read_status(ws2) == qb.QB_ERR_NONFINITE
    assert oracle.quantize_weights(w, 3, G)[0] == oracle.ERR_NONFINITE


def _check_weight_batch(shapes, seed0, ws_groups=16384):
    ws_big = qb.workspace(groups=ws_groups)
    items, host = [], []
    for i, (N, K, bits, G) in enumerate(shapes):
        w = synth.weights(N, K, seed=seed0 + 31 * i + N + K + G)
        packed = gu.poison(torch.empty((N, K * bits // 32), dtype=torch.int32, device="cuda"))
        delta = gu.poison(torch.empty(G, dtype=torch.float32, device="cuda"))
        q0 = gu.poison(torch.empty(G, dtype=torch.float32, device="cuda"))
        items.append((gu.dev(w), bits, G, packed, delta, q0))
        host.append(w)
    for _ in range(2):
        qb.quantize_pack_weights_batch(items, ws_big)
    assert qb.read_status(ws_big) == qb.QB_OK
    for (wd, bits, G, packed, delta, q0), w in zip(items, host):
        st, codes, o_delta, o_q0 = oracle.quantize_weights(w, bits, G)
        assert np.array_equal(gu.words_np(packed), oracle.pack(codes, bits)), (w.shape, bits, G)
        assert np.array_equal(delta.cpu().numpy(), o_delta) and np.array_equal(q0.cpu().numpy(), o_q0), (w.shape, bits, G)


def test_quantize_weights_register_path_shapes():
    # one launch, all bit widths: groups cut over 1, 2, 4, 8 and 16 warps with ragged last slices and warps
    # that get nothing (37 and 130 units), several whole groups per warp (1, 2, 5 and 9 units per group, a
    # last warp with fewer groups), last CTA items with fewer groups than teams, the largest group (288 units)
    _check_weight_batch([(760, 640, 3, 40), (1000, 1152, 2, 100), (777, 128, 4, 777), (777, 256, 8, 111),
                         (96, 2432, 4, 96), (1536, 2304, 2, 384), (130, 1280, 3, 13), (3072, 768, 4, 96),
                         (64, 4608, 8, 8), (2304, 768, 3, 2304), (37, 128, 2, 1), (74, 640, 8, 2),
                         (35, 640, 4, 7), (288, 1152, 3, 9), (9, 1152, 2, 9), (130, 128, 4, 1)], seed0=5)


def test_quantize_weights_cluster_path_shapes():
    # groups of 289 to 2,304 units are held by a thread-block cluster of 2 to 8 CTAs: every cluster size, slices
    # with ragged ends and warps that get nothing, more groups than resident clusters (several items per
    # cluster), all bit widths; 2,368 units is past the largest cluster and takes the two passes
    _check_weight_batch([(34, 2176, 4, 2), (36, 4096, 2, 2), (40, 3712, 3, 2), (12, 30720, 8, 2), (72, 8192, 4, 2),
                         (74, 8192, 3, 2), (2560, 1536, 2, 80), (2048, 9600, 4, 512), (2640, 1536, 8, 80),
                         (1000, 2560, 3, 50), (1400, 1408, 2, 40), (96, 16384, 4, 8), (36, 4096, 3, 1), (63, 4096, 4, 1)], seed0=9)


def test_quantize_weights_cluster_path_nonfinite():
    # an Inf in the slice of the last CTA of a cluster of five must reach the group's published range check
    N, K, G = 12, 30720, 2
    w = synth.weights(N, K, seed=3)
    ws_ok, ws_bad = qb.workspace(groups=G), qb.workspace(groups=G)
    gu.gpu_quantize_weights(w, 3, G, ws_ok)
    assert qb.read_status(ws_ok) == qb.QB_OK
    w[11, 30000] = np.inf
    gu.gpu_quantize_weights(w, 3, G, ws_bad)
    assert qb.read_status(ws_bad) == qb.QB_ERR_NONFINITE
    w[11, 30000] = np.nan
    ws_bad2 = qb.workspace(groups=G)
    gu.gpu_quantize_weights(w, 3, G, ws_bad2)
    assert qb.read_status(ws_bad2) == qb.QB_ERR_NONFINITE


@pytest.mark.parametrize("N,K,G", [(74, 8192, 2),      # 2,368 units per group: nine items per group
                                   (768, 768, 1),      # one range for the tensor: 4,608 units, sixteen items
                                   (3072, 768, 128),   # 144 units: teams of eight warps
                                   (70, 256, 70),      # two units per group: several groups per warp
                                   (40, 3712, 2)])     # 580 units: three items per group, the last one ragged
def test_quantize_weights_caller_ranges_any_group_size(N, K, G):
    # ranges that clip about 4 % of the weights (Appendix A: the range "can be a subinterval of [min, max]");
    # with ranges supplied nothing is reduced, so a group of any size stays on the single-read path
    w = synth.weights(N, K, seed=N + K + G)
    lo = np.quantile(w.reshape(G, -1), 0.02, axis=1).astype(np.float32)
    hi = np.quantile(w.reshape(G, -1), 0.98, axis=1).astype(np.float32)
    ws1 = qb.workspace(groups=max(32, G))
    for bits in BITS:
        packed, delta, q0 = gu.gpu_quantize_weights(w, bits, G, ws1, lo, hi)
        st, codes, o_delta, o_q0 = oracle.quantize_weights(w, bits, G, lo, hi)
        assert st == oracle.OK
        assert np.array_equal(gu.words_np(packed), oracle.pack(codes, bits)), bits
        assert np.array_equal(delta.cpu().numpy(), o_delta) and np.array_equal(q0.cpu().numpy(), o_q0)
        wq, d2, z2 = qb.fake_quantize_weights(gu.dev(w), bits, G, ws1, gu.dev(lo), gu.dev(hi))
        st, o_q, _, _ = oracle.fake_quantize_weights(w, bits, G, lo, hi)
        assert np.array_equal(wq.cpu().numpy().view(np.uint32), o_q.view(np.uint32)), bits
    assert qb.read_status(ws1) == qb.QB_OK
    # a NaN among the weights is still reported, and so is a range that is not ordered
    ws2, ws3 = qb.workspace(groups=max(32, G)), qb.workspace(groups=max(32, G))
    bad = w.copy()
    bad[N - 1, K - 3] = np.nan
    gu.gpu_quantize_weights(bad, 4, G, ws2, lo, hi)
    assert qb.read_status(ws2) == qb.QB_ERR_NONFINITE
    assert oracle.quantize_weights(bad, 4, G, lo, hi)[0] == oracle.ERR_NONFINITE
    lo_bad = lo.copy()
    lo_bad[G - 1] = hi[G - 1] + 1.0
    gu.gpu_quantize_weights(w, 4, G, ws3, lo_bad, hi)
    assert qb.read_status(ws3) == qb.QB_ERR_NONFINITE
    assert oracle.quantize_weights(w, 4, G, lo_bad, hi)[0] == oracle.ERR_NONFINITE


def test_quantize_weights_register_path_more_matrices_than_one_launch():
    # 100 small matrices of mixed widths and group sizes: two launches
    shapes = [((24 + 8 * (i % 5)), 128 * (1 + i % 3), (2, 3, 4, 8)[i % 4], (1, 2, 4, 8)[(i // 4) % 4]) for i in range(100)]
    _check_weight_batch(shapes, seed0=77)


@pytest.mark.parametrize("bits", BITS)
def test_quantize_weights_products_that_round_onto_ties(bits):
    # Every weight sits within a few ulp of the midpoint between two grid points, so that thousands of
    # products (w - q0) * (1/Delta) round to k + 0.5 exactly while the exact product does not: a fused
    # multiply-add in the rounding step, or a rounding other than half-to-even, shows here.
    N, K, G = 96, 1152, 12
    rng = np.random.default_rng(100 + bits)
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
    ws1 = qb.workspace(groups=G)
    packed, delta, q0 = gu.gpu_quantize_weights(w, bits, G, ws1)
    assert qb.read_status(ws1) == qb.QB_OK
    st, codes, o_delta, o_q0 = oracle.quantize_weights(w, bits, G)
    prod = (w.reshape(G, -1) - o_q0[:, None]) * (np.float32(1.0) / o_delta)[:, None]
    assert np.count_nonzero(prod - np.floor(prod) == 0.5) > 1000
    assert np.array_equal(delta.cpu().numpy(), o_delta) and np.array_equal(q0.cpu().numpy(), o_q0)
    assert np.array_equal(gu.words_np(packed), oracle.pack(codes, bits))


def test_quantize_weights_register_path_nonfinite():
    # NaN in a warp that holds several groups, -Inf in one slice of a group cut over eight warps
    for N, K, G, r, c, bad in ((64, 256, 64, 41, 200, np.nan), (128, 4608, 32, 77, 4000, -np.inf)):
        w = synth.weights(N, K, seed=N + G)
        ws_ok, ws_bad = qb.workspace(groups=G), qb.workspace(groups=G)
        gu.gpu_quantize_weights(w, 4, G, ws_ok)
        assert qb.read_status(ws_ok) == qb.QB_OK
        w[r, c] = bad
        gu.gpu_quantize_weights(w, 4, G, ws_bad)
        assert qb.read_status(ws_bad) == qb.QB_ERR_NONFINITE
        assert oracle.quantize_weights(w, 4, G)[0] == oracle.ERR_NONFINITE


def test_quantize_weights_edge_cases(ws):
    # constant group, exact ties, caller-supplied (clipping) ranges, non-finite input
    w = synth.weights(8, 128, seed=1)
    w[:2] = 0.125
    w[2, :8] = [0.0, 0.5, 1.5, 2.5, 3.0, 1.0, 2.0, 0.25]
    w[2, 8:] = 1.0
    w[3] = w[2]
    for bits in BITS:
        packed, delta, q0 = gu.gpu_quantize_weights(w, bits, 4, ws)
        st, codes, o_delta, o_q0 = oracle.quantize_weights(w, bits, 4)
        assert np.array_equal(gu.words_np(packed), oracle.pack(codes, bits))
        assert np.array_equal(delta.cpu().numpy(), o_delta) and np.array_equal(q0.cpu().numpy(), o_q0)
        assert delta.cpu().numpy()[0] == 1.0
        lo = np.full(4, -0.03, np.float32)
        hi = np.full(4, 0.05, np.float32)
        packed, delta, q0 = gu.gpu_quantize_weights(w, bits, 4, ws, lo, hi)
        st, codes, o_delta, o_q0 = oracle.quantize_weights(w, bits, 4, lo, hi)
        assert st == oracle.OK
        assert np.array_equal(gu.words_np(packed), oracle.pack(codes, bits))
        assert np.array_equal(delta.cpu().numpy(), o_delta) and np.array_equal(q0.cpu().numpy(), o_q0)
    assert qb.read_status(ws) == qb.QB_OK
    ws2 = qb.workspace(groups=16)
    w[5, 77] = np.nan
    gu.gpu_quantize_weights(w, 4, 4, ws2)
    assert qb.read_status(ws2) == qb.QB_ERR_NONFINITE
    assert oracle.quantize_weights(w, 4, 4)[0] == oracle.ERR_NONFINITE


# ------------------------------------------------------------------ whole linear layer
@pytest.mark.parametrize("bits", BITS)
@pytest.mark.parametrize("M,N,K,groups", [
    (128, 128, 128, 1),      # exactly one tile, one K block
    (1, 8, 128, 8),          # smallest: one token, one row per group
    (127, 24, 256, 4),       # ragged token tile, tiny N (6-row groups as in 128-group BERT-base)
    (300, 264, 384, 11),     # several token and neuron tiles, both ragged, groups straddle tiles
    (260, 768, 1024, 128),   # more K blocks than pipeline stages
])
def test_linear_matches_oracle(ws, bits, M, N, K, groups):
    x = synth.activations(M, K, seed=11 * M + bits)
    w = synth.weights(N, K, seed=13 * N + bits)
    b = synth.bias(N, seed=17 * N + bits)
    gu.check_linear(x, w, b, bits, groups, ws)


@pytest.mark.parametrize("bits", BITS)
def test_linear_wide_token_tiles(ws, bits):
    # enough tiles that the 256-token tile configuration is selected; ragged in M and N
    M, N, K, groups = 2040, 4730, 128, 10
    x = synth.activations(M, K, seed=bits)
    w = synth.weights(N, K, seed=100 + bits)
    b = synth.bias(N, seed=200 + bits)
    gu.check_linear(x, w, b, bits, groups, ws, use_omp=True)


@pytest.mark.parametrize("bits", BITS)
def test_linear_cta_pairs_ragged_tiles_through_tma_stores(ws, bits):
    # enough 256 x 256 tiles for the CTA-pair kernel; the last neuron tile leaves the second CTA of the pair
    # with 8 valid rows of 128, the last token tile is ragged (its second half partly outside M), K is
    # five K blocks (the depth of the pair's ring); N % 4 == 0, so outputs leave through TMA stores
    M, N, K, groups = 2500, 2440, 640, 10
    x = synth.activations(M, K, seed=300 + bits)
    w = synth.weights(N, K, seed=400 + bits)
    b = synth.bias(N, seed=500 + bits) if bits != 3 else None
    gu.check_linear(x, w, b, bits, groups, ws, use_omp=True)


def test_small_mixed_stack_larger_than_one_launch(ws):
    # 50 small linears of mixed bit widths and ragged shapes: more than one launch holds (48), every launch
    # mixes bit widths; each result must equal the single call bit for bit and the oracle
    rng = np.random.default_rng(77)
    M = 96
    descs, refs = [], []
    for i in range(50):
        N = int(rng.choice([24, 136, 264]))
        K = int(rng.choice([128, 256, 640]))
        bits = int(rng.choice(BITS))
        G = int(rng.choice([1, 2, 4]))
        x = synth.activations(M, K, seed=2000 + i)
        w = synth.weights(N, K, seed=3000 + i)
        b = synth.bias(N, seed=4000 + i)
        xq, sc, rs = qb.quantize_act(gu.dev(x), ws)
        packed, delta, q0 = qb.quantize_pack_weights(gu.dev(w), bits, G, ws)
        y = gu.poison(torch.empty((M, N), dtype=torch.float32, device="cuda"))
        descs.append(qb.LinearDesc(xq, sc, rs, packed, delta, q0, gu.dev(b), N, bits, G, y))
        refs.append((x, w, b, bits, G))
    assert qb.layer_linears_launch_count(descs) == 2
    qb.layer_linears(descs, ws)
    assert qb.read_status(ws) == qb.QB_OK
    for d, (x, w, b, bits, G) in zip(descs, refs):
        y1 = qb.gemm(d.xq, d.act_scale, d.rowsum, d.packed, d.delta, d.q0, d.bias, d.N, bits, G, ws)
        assert torch.equal(y1, d.y)
        ref = oracle.linear(x, w, b, bits, G)
        gu.assert_y_close(d.y.cpu().numpy(), ref["y"])


def test_linear_without_bias_and_with_positive_activations(ws):
    M, N, K, groups = 200, 256, 512, 32
    x = np.abs(synth.activations(M, K, seed=5))   # large row sums: the offset term dominates
    w = synth.weights(N, K, seed=6)
    for bits in BITS:
        gu.check_linear(x, w, None, bits, groups, ws)


def test_gemm_one_hot_and_extreme_codes(ws):
    # one-hot activations return single weight codes: a layout or descriptor slip shows as a permutation
    K, N = 256, 136
    x = np.zeros((K, K), np.float32)
    np.fill_diagonal(x, 1.0)
    w = synth.weights(N, K, seed=9)
    for bits in BITS:
        r = gu.check_linear(x, w, None, bits, 1, ws)
        st, codes, _, _ = oracle.quantize_weights(w, bits, 1)
        assert np.array_equal(r["acc"].cpu().numpy(), 127 * codes.T.astype(np.int32))
    # largest magnitudes: every activation code +-127, every weight code 0 or 2^k-1
    x = np.where(np.random.default_rng(1).random((130, 4096)) < 0.5, -1.0, 1.0).astype(np.float32)
    w = np.where(np.random.default_rng(2).random((128, 4096)) < 0.5, -1.0, 1.0).astype(np.float32)
    for bits in BITS:
        gu.check_linear(x, w, None, bits, 1, ws)


def test_gemm_is_deterministic(ws):
    M, N, K, bits, groups = 515, 384, 768, 3, 64
    x = synth.activations(M, K, seed=1)
    w = synth.weights(N, K, seed=2)
    b = synth.bias(N, seed=3)
    r1 = gu.check_linear(x, w, b, bits, groups, ws)
    y2 = torch.empty_like(r1["y"])
    qb.gemm(r1["xq"], r1["act_scale"], r1["rowsum"], r1["packed"], r1["delta"], r1["q0"], gu.dev(b), N, bits,
            groups, ws, y=y2)
    assert torch.equal(r1["y"], y2)


# ------------------------------------------------------------------ the benchmark configurations
def test_config0_query_projection(ws):
    wl = synth.workload(0)
    s = wl.linears[0]
    x = synth.activations(wl.M, s.K, seed=0)
    w = synth.weights(s.N, s.K, seed=0)
    b = synth.bias(s.N, seed=0)
    gu.check_linear(x, w, b, wl.bits[0], s.groups, ws, use_omp=True)


def _check_stack(ws, wl, layers, rows_per_tile=2):
    """quantize everything, run the stack through qb_layer_linears, compare with the oracle."""
    descs, refs, acts, mats = [], [], [], []
    for layer in layers:
        bits = wl.bits[layer]
        for mi, s in enumerate(wl.linears):
            seed = synth.seed_for(wl.config, layer, mi)
            x = synth.activations(wl.M, s.K, seed)
            w = synth.weights(s.N, s.K, seed)
            b = synth.bias(s.N, seed)
            # outputs poisoned, then filled by the batched quantizers below
            xq = gu.poison(torch.empty((wl.M, s.K), dtype=torch.int8, device="cuda"))
            sc = gu.poison(torch.empty(1, dtype=torch.float32, device="cuda"))
            rs = gu.poison(torch.empty(wl.M, dtype=torch.int32, device="cuda"))
            packed = gu.poison(torch.empty((s.N, s.K * bits // 32), dtype=torch.int32, device="cuda"))
            delta = gu.poison(torch.empty(s.groups, dtype=torch.float32, device="cuda"))
            q0 = gu.poison(torch.empty(s.groups, dtype=torch.float32, device="cuda"))
            acts.append((gu.dev(x), xq, sc, rs))
            mats.append((gu.dev(w), bits, s.groups, packed, delta, q0))
            y = gu.poison(torch.empty((wl.M, s.N), dtype=torch.float32, device="cuda"))
            descs.append(qb.LinearDesc(xq, sc, rs, packed, delta, q0, gu.dev(b), s.N, bits, s.groups, y))
            refs.append((x, w, b, bits, s))
    ws = qb.workspace(groups=max(32, sum(m[2] for m in mats)))
    qb.quantize_act_batch(acts, ws)
    qb.quantize_pack_weights_batch(mats, ws)
    qb.layer_linears(descs, ws)
    assert qb.read_status(ws) == qb.QB_OK
    for d, (x, w, b, bits, s) in zip(descs, refs):
        rows = gu.sample_rows(wl.M, per_tile=rows_per_tile, seed=s.N + bits)
        st_a, o_xq, o_s, o_rs = oracle.quantize_act(x, omp=True)
        st_w, codes, o_delta, o_q0 = oracle.quantize_weights(w, bits, s.groups, omp=True)
        assert np.array_equal(d.xq.cpu().numpy(), o_xq)
        assert np.array_equal(d.rowsum.cpu().numpy(), o_rs)
        assert np.array_equal(gu.words_np(d.packed), oracle.pack(codes, bits))
        assert np.array_equal(d.delta.cpu().numpy(), o_delta) and np.array_equal(d.q0.cpu().numpy(), o_q0)
        o_acc = oracle.int_gemm(o_xq[rows], codes, omp=True)
        o_y = oracle.dequant_epilogue(o_acc, o_rs[rows], o_s, o_delta, o_q0, b, bits, s.groups)
        gu.assert_y_close(d.y[torch.from_numpy(rows).cuda()].cpu().numpy(), o_y)
        # the stack must equal the single call bit for bit
        y1, acc1 = qb.gemm(d.xq, d.act_scale, d.rowsum, d.packed, d.delta, d.q0, d.bias, d.N, bits, s.groups, ws,
                           want_acc=True)
        assert torch.equal(y1, d.y)
        assert np.array_equal(acc1[torch.from_numpy(rows).cuda()].cpu().numpy(), o_acc)


def test_batched_quantizers_equal_single_calls(ws):
    # mixed bit widths and group counts, more tensors than one launch holds (32)
    rng = np.random.default_rng(3)
    acts, mats, single_a, single_w = [], [], [], []
    shapes = [(5, 128), (129, 384), (64, 768), (300, 256)] * 9          # 36 activation tensors
    for i, (M, K) in enumerate(shapes):
        x = gu.dev(synth.activations(M, K, seed=700 + i))
        single_a.append(qb.quantize_act(x, ws))
        acts.append((x, gu.poison(torch.empty((M, K), dtype=torch.int8, device="cuda")),
                     gu.poison(torch.empty(1, dtype=torch.float32, device="cuda")),
                     gu.poison(torch.empty(M, dtype=torch.int32, device="cuda"))))
    wshapes = [(24, 128, 4), (768, 768, 128), (264, 256, 11), (12, 384, 1), (96, 3072, 96)] * 8   # 40 matrices
    for i, (N, K, G) in enumerate(wshapes):
        bits = int(rng.choice(BITS))
        w = gu.dev(synth.weights(N, K, seed=800 + i))
        single_w.append(qb.quantize_pack_weights(w, bits, G, ws))
        mats.append((w, bits, G, gu.poison(torch.empty((N, K * bits // 32), dtype=torch.int32, device="cuda")),
                     gu.poison(torch.empty(G, dtype=torch.float32, device="cuda")),
                     gu.poison(torch.empty(G, dtype=torch.float32, device="cuda"))))
    ws2 = qb.workspace(groups=sum(m[2] for m in mats))
    qb.quantize_act_batch(acts, ws2)
    qb.quantize_pack_weights_batch(mats, ws2)
    assert qb.read_status(ws2) == qb.QB_OK
    for (x, xq, sc, rs), (xq1, sc1, rs1) in zip(acts, single_a):
        assert torch.equal(xq, xq1) and torch.equal(sc, sc1) and torch.equal(rs, rs1)
    for (w, bits, G, packed, delta, q0), (p1, d1, z1) in zip(mats, single_w):
        assert torch.equal(packed, p1) and torch.equal(delta, d1) and torch.equal(q0, z1)
    # a non-finite tensor in the middle of a batch is reported
    bad = acts[7][0].clone()
    bad[0, 3] = float("nan")
    acts[7] = (bad,) + acts[7][1:]
    ws3 = qb.workspace(groups=64)
    qb.quantize_act_batch(acts, ws3)
    assert qb.read_status(ws3) == qb.QB_ERR_NONFINITE


def test_config1_encoder_layer_linears(ws):
    _check_stack(ws, synth.workload(1), layers=[0])


def test_config2_mixed_precision_stack(ws):
    wl = synth.workload(2)
    assert sum(b == 2 for b in wl.bits) >= 6 and set(wl.bits) <= set(synth.BITS_CHOICES)
    _check_stack(ws, wl, layers=range(wl.layers), rows_per_tile=8)


def test_mixed_stack_in_a_graph(ws):
    # A small stack that mixes bit widths is one launch whose problems carry their own width.  Captured
    # into a CUDA graph on a non-default stream and replayed, it must still equal the single calls bit for
    # bit (everything the call enqueues is on the capturing stream).
    M = 128
    shapes = [(256, 256, 2, 4), (384, 512, 4, 6), (128, 1024, 8, 2), (256, 256, 3, 1), (256, 768, 2, 8)]
    descs, singles = [], []
    for i, (N, K, bits, G) in enumerate(shapes):
        x = synth.activations(M, K, seed=900 + i)
        w = synth.weights(N, K, seed=950 + i)
        b = synth.bias(N, seed=990 + i)
        xq, sc, rs = qb.quantize_act(gu.dev(x), ws)
        packed, delta, q0 = qb.quantize_pack_weights(gu.dev(w), bits, G, ws)
        y = gu.poison(torch.empty((M, N), dtype=torch.float32, device="cuda"))
        descs.append(qb.LinearDesc(xq, sc, rs, packed, delta, q0, gu.dev(b), N, bits, G, y))
        singles.append(qb.gemm(xq, sc, rs, packed, delta, q0, gu.dev(b), N, bits, G, ws).clone())
    arr = qb.make_desc_array(descs)
    qb.layer_linears(arr, ws)  # first call on the device sets kernel attributes: before any capture
    torch.cuda.synchronize()
    for d, y1 in zip(descs, singles):
        assert torch.equal(d.y, y1)
        gu.poison(d.y)
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            qb.layer_linears(arr, ws)
        for _ in range(2):
            graph.replay()
    stream.synchronize()
    torch.cuda.synchronize()
    assert qb.read_status(ws) == qb.QB_OK
    for d, y1 in zip(descs, singles):
        assert torch.equal(d.y, y1)


@pytest.mark.parametrize("preset", ["2/3-MP SST-2", "2/4-MP SST-2"])
def test_paper_bit_presets_stack(ws, preset):
    # the per-layer bit widths printed in the paper's appendix tables, first four layers' worth of bits
    base = synth.workload(2)
    wl = synth.Workload(2, preset, 128, 12, base.linears, synth.MP_PRESETS[preset])
    _check_stack(ws, wl, layers=[0, 2, 3, 5], rows_per_tile=8)


def test_config3_bert_large_layer_sampled(ws):
    # full-size M = 24576 in the launch configuration the benchmark times; one layer, sampled rows
    _check_stack(ws, synth.workload(3), layers=[0], rows_per_tile=1)


def test_config4_quantizer_sweep_sample(ws):
    # the distinct shapes of the sweep (incl. the 768 x 30720 embedding-shaped matrix) at every k and
    # a spread of group counts; the activation tensor of the sweep at full size
    shapes = sorted(set(synth.quantizer_sweep_shapes()))
    for i, (N, K) in enumerate(shapes):
        w = synth.weights(N, K, seed=synth.seed_for(4, 0, i))
        for bits, groups in ((2, 1), (3, 12), (4, 128), (8, 768)):
            packed, delta, q0 = gu.gpu_quantize_weights(w, bits, groups, ws)
            st, codes, o_delta, o_q0 = oracle.quantize_weights(w, bits, groups, omp=True)
            assert np.array_equal(gu.words_np(packed), oracle.pack(codes, bits)), (N, K, bits, groups)
            assert np.array_equal(delta.cpu().numpy(), o_delta) and np.array_equal(q0.cpu().numpy(), o_q0)
    M, K = synth.QUANTIZER_SWEEP_ACT
    x = synth.activations(M, K, seed=synth.seed_for(4))
    xq, sc, rs = gu.gpu_quantize_act(x, ws)
    st, o_xq, o_s, o_rs = oracle.quantize_act(x, omp=True)
    assert np.array_equal(xq.cpu().numpy(), o_xq) and np.array_equal(rs.cpu().numpy(), o_rs)
    assert sc.item() == o_s
    assert qb.read_status(ws) == qb.QB_OK
