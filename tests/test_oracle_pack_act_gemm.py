"""Pins for the oracle's packing, activation quantizer, integer GEMM and epilogue."""
from pathlib import Path

import numpy as np
import pytest
import torch

import oracle
from paper_1909_05840_b200 import synth

BITS = (2, 3, 4, 8)
GOLDEN = Path(__file__).parent / "golden"


# ---------------------------------------------------------------- packing
@pytest.mark.parametrize("bits", BITS)
def test_pack_round_trip(bits):
    rng = np.random.default_rng(bits)
    codes = rng.integers(0, 1 << bits, size=(5, 384), dtype=np.uint8)
    words = oracle.pack(codes, bits)
    assert words.shape == (5, 384 * bits // 32)
    assert np.array_equal(oracle.unpack(words, 384, bits), codes)


def test_pack_hand_checked_words():
    # dense little-endian bit stream: code j sits at stream bits [k*j, k*j+k)
    assert oracle.pack(np.arange(8, dtype=np.uint8)[None], 4)[0, 0] == 0x76543210
    assert oracle.pack(np.tile(np.arange(4, dtype=np.uint8), 4)[None], 2)[0, 0] == 0xE4E4E4E4
    assert oracle.pack(np.arange(4, dtype=np.uint8)[None], 8)[0, 0] == 0x03020100
    c3 = np.zeros((1, 32), np.uint8)
    c3[0, :8] = np.arange(8)
    w3 = oracle.pack(c3, 3)
    assert w3.shape == (1, 3) and w3[0, 0] == 0xFAC688 and w3[0, 1] == 0 and w3[0, 2] == 0
    # a 3-bit code that straddles a word boundary: code 10 occupies stream bits 30..32
    c3[:] = 0
    c3[0, 10] = 0b111
    w3 = oracle.pack(c3, 3)
    assert w3[0, 0] == 0xC0000000 and w3[0, 1] == 0x1 and w3[0, 2] == 0


@pytest.mark.parametrize("bits", BITS)
def test_pack_matches_python_big_integer_stream(bits):
    # independent restatement: the row as one big little-endian integer
    rng = np.random.default_rng(40 + bits)
    K = 128
    codes = rng.integers(0, 1 << bits, size=(3, K), dtype=np.uint8)
    words = oracle.pack(codes, bits)
    for n in range(3):
        big = 0
        for j in range(K):
            big |= int(codes[n, j]) << (bits * j)
        raw = big.to_bytes(K * bits // 8, "little")
        assert np.array_equal(np.frombuffer(raw, dtype="<u4"), words[n])


def _golden_sizes():
    out = {}
    for line in (GOLDEN / "table1_sizes.txt").read_text().splitlines():
        if line.startswith("#") or not line.strip():
            continue
        k, v = line.split()
        out[k] = float(v)
    return out


def _golden_bits():
    out = {}
    for line in (GOLDEN / "bits_tables.txt").read_text().splitlines():
        if line.startswith("#") or not line.strip():
            continue
        parts = line.split()
        out[" ".join(parts[:2])] = tuple(int(b) for b in parts[2:])
    return out


def _layer_words(bits):
    """32-bit words the oracle's packing produces for the 4 linears of one BERT-base layer."""
    total = 0
    for s in synth.BERT_BASE:
        total += oracle.pack(np.zeros((s.N, s.K), np.uint8), bits).size
    return total


def test_packed_size_reproduces_table1():
    # Table 1 "Size-w/o-e": exactly k bits per weight.  The paper's 7.1 M parameters per layer
    # include biases and LayerNorm; the packed matrices are 7,077,888 of them.
    gold = _golden_sizes()
    mats = sum(s.N * s.K for s in synth.BERT_BASE)
    assert mats == 7077888
    per_layer = mats + sum(s.N for s in synth.BERT_BASE) + 4 * 768
    assert abs(per_layer / 1e6 - gold["params_per_layer_M"]) < 0.05
    assert abs(12 * per_layer * 4 / 2 ** 20 - gold["fp32"]) < 0.3
    words = {b: _layer_words(b) for b in BITS}
    for b in BITS:
        assert words[b] * 32 == mats * b                       # dense: k bits per weight
        assert abs(12 * words[b] * 4 / 2 ** 20 - gold[str(b)]) < 0.3
    tables = _golden_bits()
    for label, task in (("2/3-MP:SST-2", "2/3-MP SST-2"), ("2/3-MP:SQuAD", "2/3-MP SQuAD"),
                        ("2/3-MP:MNLI", "2/3-MP MNLI"), ("2/3-MP:CoNLL-03", "2/3-MP CoNLL-03"),
                        ("2/4-MP", "2/4-MP SST-2")):
        mib = sum(words[b] for b in tables[task]) * 4 / 2 ** 20
        assert abs(mib - gold[label]) < 0.4, (label, mib)


def test_bit_presets_match_the_papers_tables():
    assert _golden_bits() == synth.MP_PRESETS


# ---------------------------------------------------------------- activations
def test_act_codes_bruteforce_nearest():
    rng = np.random.default_rng(1)
    x = (rng.standard_normal((7, 64)) * 3).astype(np.float32)
    st, xq, s, rowsum = oracle.quantize_act(x)
    assert st == oracle.OK
    a = np.abs(x).max()
    assert np.isclose(float(s), float(a) / 127.0, rtol=1e-6)
    grid = np.arange(-127, 128, dtype=np.float64) * (float(a) / 127.0)   # 255-point symmetric grid
    dist = np.abs(x.astype(np.float64)[..., None] - grid)
    chosen = np.take_along_axis(dist, (xq.astype(np.int64) + 127)[..., None], -1)[..., 0]
    assert np.all(chosen <= dist.min(-1) + float(a) * 2.0 ** -20)
    assert np.array_equal(rowsum, xq.astype(np.int64).sum(1))
    assert xq.min() >= -127 and xq.max() <= 127


def test_act_special_points_and_symmetry():
    x = np.array([[2.5, -2.5, 0.0, 1.25, -1.25, 2.5 / 127 * 0.5, 0.1, -0.1]], np.float32)
    st, xq, s, rowsum = oracle.quantize_act(x)
    assert xq[0, 0] == 127 and xq[0, 1] == -127 and xq[0, 2] == 0
    assert xq[0, 3] == -xq[0, 4]
    st2, xq2, s2, rs2 = oracle.quantize_act(-x)
    assert np.array_equal(xq2, -xq) and s2 == s and rs2[0] == -rowsum[0]
    # hand-checkable row: a = 1 -> codes 127, -127, round(63.5) = 64 (half to even), 0
    st, xq, s, rowsum = oracle.quantize_act(np.array([[1.0, -1.0, 0.5, 0.0]], np.float32))
    assert xq[0].tolist() == [127, -127, 64, 0] and rowsum[0] == 64
    assert np.isclose(float(s), 1 / 127)


def test_act_zero_tensor_and_nonfinite():
    st, xq, s, rowsum = oracle.quantize_act(np.zeros((3, 16), np.float32))
    assert st == oracle.OK and s == 1.0 and not xq.any() and not rowsum.any()
    x = np.ones((2, 16), np.float32)
    x[1, 3] = np.nan
    assert oracle.quantize_act(x)[0] == oracle.ERR_NONFINITE
    x[1, 3] = -np.inf
    assert oracle.quantize_act(x)[0] == oracle.ERR_NONFINITE


# ---------------------------------------------------------------- integer GEMM
def _rand_q(M, N, K, bits, seed):
    rng = np.random.default_rng(seed)
    xq = rng.integers(-127, 128, size=(M, K), dtype=np.int8)
    codes = rng.integers(0, 1 << bits, size=(N, K), dtype=np.uint8)
    return xq, codes


@pytest.mark.parametrize("bits", BITS)
def test_int_gemm_matches_library_matmul_and_int64(bits):
    xq, codes = _rand_q(9, 11, 160, bits, bits)
    acc, acc64 = oracle.int_gemm(xq, codes, want64=True)
    assert np.array_equal(acc.astype(np.int64), acc64)
    ref = xq.astype(np.int64) @ codes.astype(np.int64).T            # numpy library product
    assert np.array_equal(acc64, ref)
    tref = torch.from_numpy(xq.astype(np.int32)) @ torch.from_numpy(codes.astype(np.int32)).T
    assert np.array_equal(acc, tref.numpy())                         # torch CPU integer matmul


def test_int_gemm_extreme_values_do_not_overflow():
    K = 4096
    xq = np.full((2, K), 127, np.int8)
    xq[1] = -127
    codes = np.full((2, K), 255, np.uint8)
    acc, acc64 = oracle.int_gemm(xq, codes, want64=True)
    assert acc[0, 0] == 127 * 255 * K and acc[1, 1] == -127 * 255 * K
    assert np.array_equal(acc.astype(np.int64), acc64)


def test_int_gemm_one_hot_and_all_ones():
    xq, codes = _rand_q(6, 5, 64, 4, 3)
    onehot = np.zeros((64, 64), np.int8)
    np.fill_diagonal(onehot, 127)
    assert np.array_equal(oracle.int_gemm(onehot, codes), 127 * codes.T.astype(np.int32))
    ones = np.ones_like(codes)
    assert np.array_equal(oracle.int_gemm(xq, ones), np.repeat(xq.astype(np.int32).sum(1)[:, None], 5, 1))


# ---------------------------------------------------------------- epilogue / whole layer
def test_hand_worked_layer():
    # X = [1, -1, 0.5, 0]: a = 1, codes [127, -127, 64, 0], rowsum 64, scale 1/127.
    # W rows [0,1,2,3] and [3,3,0,0] at k = 2, per-row groups: Delta = 1, q0 = 0, codes = values.
    # acc = [127*0 - 127*1 + 64*2, 127*3 - 127*3] = [1, 0];  y = acc/127 + bias.
    x = np.array([[1.0, -1.0, 0.5, 0.0] + [0.0] * 28], np.float32)
    w = np.zeros((2, 32), np.float32)
    w[0, :4] = [0, 1, 2, 3]
    w[1, :4] = [3, 3, 0, 0]
    b = np.array([0.5, -0.25], np.float32)
    r = oracle.linear(x, w, b, bits=2, groups=2)
    assert r["acc"].tolist() == [[1, 0]]
    assert np.allclose(r["y"], [[1 / 127 + 0.5, -0.25]], rtol=1e-6)


@pytest.mark.parametrize("bits", BITS)
@pytest.mark.parametrize("positive", (False, True))
def test_epilogue_equals_fp64_definition(bits, positive):
    # sum_k (s*xq) * (Delta*u + q0) + b, evaluated in double precision straight from Appendix A
    M, N, K, G = 17, 24, 256, 4
    x = synth.activations(M, K, seed=bits)
    if positive:
        x = np.abs(x)                       # large row sums: the hard case for cancellation
    w = synth.weights(N, K, seed=bits + 10)
    b = synth.bias(N, seed=bits + 20)
    r = oracle.linear(x, w, b, bits, G)
    # an independent float64 evaluation in numpy (not the oracle's own fp64 routine)
    wq = r["delta"].astype(np.float64).repeat(N // G)[:, None] * r["codes"] + \
        r["q0"].astype(np.float64).repeat(N // G)[:, None]
    y64 = (np.float64(r["act_scale"]) * r["xq"].astype(np.float64)) @ wq.T + b.astype(np.float64)
    # fp32 rounding enters through alpha, beta and the two fused multiply-adds: a few ulp of the
    # magnitudes of the two terms about the centre code c = 2^(k-1), and of the bias
    c = 1 << (bits - 1)
    sa, D, z = np.float64(r["act_scale"]), r["delta"].astype(np.float64).repeat(N // G), \
        r["q0"].astype(np.float64).repeat(N // G)
    rs = r["rowsum"].astype(np.float64)[:, None]
    mag = np.abs(sa * D[None] * (r["acc"] - c * rs)) + np.abs(sa * (D * c + z)[None] * rs) + np.abs(b)
    assert np.all(np.abs(r["y"] - y64) <= 4e-7 * mag + 1e-9)
    assert np.allclose(oracle.linear_fp64(r["xq"], r["act_scale"], r["codes"], r["delta"], r["q0"], b, G),
                       y64, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("bits", BITS)
def test_end_to_end_error_bound(bits):
    # propagate the quantizers' half-step bounds through the product:
    # |y - (x.w + b)| <= sum_k |x| D/2 + |w| s/2 + s D/4
    M, N, K, G = 8, 12, 128, 3
    x = synth.activations(M, K, seed=50 + bits)
    w = synth.weights(N, K, seed=60 + bits)
    b = synth.bias(N, seed=70 + bits)
    r = oracle.linear(x, w, b, bits, G)
    exact = x.astype(np.float64) @ w.astype(np.float64).T + b
    D = r["delta"].astype(np.float64).repeat(N // G)
    s = float(r["act_scale"])
    bound = (np.abs(x).astype(np.float64).sum(1)[:, None] * D[None, :] / 2
             + np.abs(w).astype(np.float64).sum(1)[None, :] * s / 2 + K * s * D[None, :] / 4)
    assert np.all(np.abs(r["y"] - exact) <= bound * (1 + 1e-4) + 1e-5)
    # and the bound is not vacuous: 8-bit weights are much closer than 2-bit ones
    if bits == 8:
        r2 = oracle.linear(x, w, b, 2, G)
        assert np.abs(r["y"] - exact).mean() < np.abs(r2["y"] - exact).mean() / 5


def test_epilogue_bias_optional_and_group_lookup():
    M, N, K, G = 4, 6, 32, 3
    xq, codes = _rand_q(M, N, K, 4, 9)
    acc = oracle.int_gemm(xq, codes)
    rowsum = xq.astype(np.int32).sum(1)
    delta = np.array([0.5, 2.0, 1.0], np.float32)
    q0 = np.array([0.0, -1.0, 3.0], np.float32)
    y0 = oracle.dequant_epilogue(acc, rowsum, 0.25, delta, q0, None, 4, G)
    want = 0.25 * (acc * delta.repeat(2)[None] + rowsum[:, None] * q0.repeat(2)[None])
    assert np.allclose(y0, want, rtol=1e-6, atol=1e-6)
    b = np.arange(N, dtype=np.float32)
    assert np.allclose(oracle.dequant_epilogue(acc, rowsum, 0.25, delta, q0, b, 4, G), want + b, rtol=1e-6,
                       atol=1e-5)
