"""Quantized embedding tables on the GPU against the oracle: codes, packed rows, Delta, q0 and the
looked-up fp32 rows are bit-exact (same IEEE operations in the same order)."""
import numpy as np
import pytest
import torch

import oracle
import paper_1909_05840_b200 as qb

import gpu_util as gu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ws():
    return qb.workspace(groups=4096)


def _table(V, D, seed):
    rng = np.random.default_rng(seed)
    e = (rng.standard_normal((V, D)) * 0.02).astype(np.float32)
    e[:, 5] *= 8.0
    e[rng.integers(0, V, 16), rng.integers(0, D, 16)] = rng.laplace(0, 0.2, 16).astype(np.float32)
    return e


@pytest.mark.parametrize("bits", (2, 3, 4, 8))
@pytest.mark.parametrize("V,D,groups", [(1000, 768, 128), (513, 768, 768), (77, 128, 1), (2050, 1024, 128), (300, 768, 12)])
def test_quantize_embedding_and_lookup_match_oracle(ws, bits, V, D, groups):
    e = _table(V, D, seed=V + D + bits)
    packed = gu.poison(torch.empty((V, D * bits // 32), dtype=torch.int32, device="cuda"))
    packed, delta, q0 = qb.quantize_embedding(gu.dev(e), bits, groups, ws, packed=packed)
    assert qb.read_status(ws) == qb.QB_OK
    st, codes, o_delta, o_q0 = oracle.quantize_embedding(e, bits, groups)
    assert st == oracle.OK
    assert np.array_equal(delta.cpu().numpy(), o_delta) and np.array_equal(q0.cpu().numpy(), o_q0)
    assert np.array_equal(gu.words_np(packed), oracle.pack(codes, bits))
    rng = np.random.default_rng(bits)
    ids = np.concatenate([[0, V - 1, V - 1, 0], rng.integers(0, V, 601)]).astype(np.int32)
    out = gu.poison(torch.empty((ids.size, D), dtype=torch.float32, device="cuda"))
    qb.embedding_lookup(torch.from_numpy(ids).cuda(), packed, delta, q0, D, bits, groups, ws, out=out)
    ref = oracle.embedding_lookup(ids, codes, groups, o_delta, o_q0)
    assert np.array_equal(out.cpu().numpy().view(np.uint32), ref.view(np.uint32))
    assert qb.read_status(ws) == qb.QB_OK


def test_word_plus_position_mixed_precision_and_bad_id():
    # the paper's mixed-precision embedding: 4-bit word table, 8-bit position table, 128 groups each
    ws = qb.workspace(groups=4096)
    D, G = 768, 128
    words, positions = _table(4096, D, seed=1), _table(512, D, seed=2)
    pw, dw, zw = qb.quantize_embedding(gu.dev(words), 4, G, ws)
    pp, dp, zp = qb.quantize_embedding(gu.dev(positions), 8, G, ws)
    rng = np.random.default_rng(3)
    ids = rng.integers(0, 4096, 8 * 128).astype(np.int32)
    pos = np.tile(np.arange(128, dtype=np.int32), 8)
    out = qb.embedding_lookup(torch.from_numpy(ids).cuda(), pw, dw, zw, D, 4, G, ws)
    qb.embedding_lookup(torch.from_numpy(pos).cuda(), pp, dp, zp, D, 8, G, ws, out=out, accumulate=True)
    _, cw, odw, ozw = oracle.quantize_embedding(words, 4, G)
    _, cp, odp, ozp = oracle.quantize_embedding(positions, 8, G)
    ref = oracle.embedding_lookup(pos, cp, G, odp, ozp, out=oracle.embedding_lookup(ids, cw, G, odw, ozw))
    assert np.array_equal(out.cpu().numpy().view(np.uint32), ref.view(np.uint32))
    assert qb.read_status(ws) == qb.QB_OK
    # an id outside the table: zeros for that token, QB_ERR_INVALID in the status word, no out-of-bounds read
    bad = ids.copy(); bad[5] = 4096; bad[9] = -1
    out2 = qb.embedding_lookup(torch.from_numpy(bad).cuda(), pw, dw, zw, D, 4, G, ws)
    assert qb.read_status(ws) == qb.QB_ERR_INVALID
    o2 = out2.cpu().numpy()
    assert np.all(o2[5] == 0) and np.all(o2[9] == 0)
    good = np.ones(len(bad), bool); good[[5, 9]] = False
    assert np.array_equal(o2[good], oracle.embedding_lookup(ids, cw, G, odw, ozw)[good])


def test_embedding_nonfinite_and_constant_group():
    ws = qb.workspace(groups=4096)
    e = _table(200, 256, seed=9)
    e[:, 8:16] = -0.125                    # a constant group (G = 32: 8 columns per group)
    packed, delta, q0 = qb.quantize_embedding(gu.dev(e), 4, 32, ws)
    st, codes, o_delta, o_q0 = oracle.quantize_embedding(e, 4, 32)
    assert np.array_equal(gu.words_np(packed), oracle.pack(codes, 4))
    assert delta.cpu().numpy()[1] == 1.0 and q0.cpu().numpy()[1] == -0.125
    assert qb.read_status(ws) == qb.QB_OK
    e[17, 3] = np.nan
    qb.quantize_embedding(gu.dev(e), 4, 32, ws)
    assert qb.read_status(ws) == qb.QB_ERR_NONFINITE
