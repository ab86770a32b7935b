"""Pins of the oracle's embedding-table quantizer (column groups) and dequantizing lookup against the
row-group weight quantizer on the transposed table (itself pinned by brute force and closed forms),
against numpy indexing of the dequantized table, and against the size the paper prints."""
import numpy as np

import oracle


def _table(V=300, D=768, seed=0):
    rng = np.random.default_rng(seed)
    e = (rng.standard_normal((V, D)) * 0.02).astype(np.float32)
    e[:, 5] *= 8.0          # a column with a wide range: its group gets a coarser grid than its neighbours
    return e


def test_column_groups_equal_row_groups_of_the_transposed_table():
    e = _table()
    for bits, G in ((4, 128), (8, 128), (2, 768), (3, 1), (4, 12)):
        st, codes, delta, q0 = oracle.quantize_embedding(e, bits, G)
        st2, codes_t, delta_t, q0_t = oracle.quantize_weights(np.ascontiguousarray(e.T), bits, G)
        assert st == oracle.OK and st2 == oracle.OK
        assert np.array_equal(codes, codes_t.T)
        assert np.array_equal(delta, delta_t) and np.array_equal(q0, q0_t)
    # groups matter: the wide column's group has a larger step than the next group
    st, codes, delta, q0 = oracle.quantize_embedding(e, 4, 128)
    assert delta[0] > 4 * delta[1]


def test_lookup_is_indexing_of_the_dequantized_table_and_accumulates():
    e = _table(seed=1)
    V, D = e.shape
    G, bits = 128, 4
    st, codes, delta, q0 = oracle.quantize_embedding(e, bits, G)
    deq = oracle.dequantize_weights(np.ascontiguousarray(codes.T), G, delta, q0).T   # Q(E), via the row-group routine
    ids = np.array([0, V - 1, 7, 7, 123, 1], dtype=np.int32)
    out = oracle.embedding_lookup(ids, codes, G, delta, q0)
    assert np.array_equal(out, deq[ids])
    # |E - Q(E)| <= Delta/2 per group (the quantizer's own bound, now through the lookup)
    C = D // G
    err = np.abs(e[ids].astype(np.float64) - out.astype(np.float64)).reshape(len(ids), G, C).max(axis=(0, 2))
    assert np.all(err <= 0.5 * delta.astype(np.float64) * (1 + 2.0**-18) + 1e-9)
    # word + position: the second lookup adds, one fp32 addition per element
    st, pcodes, pdelta, pq0 = oracle.quantize_embedding(_table(V=64, seed=2), 8, G)
    pos = np.arange(len(ids), dtype=np.int32)
    both = oracle.embedding_lookup(pos, pcodes, G, pdelta, pq0, out=out)
    pdeq = oracle.dequantize_weights(np.ascontiguousarray(pcodes.T), G, pdelta, pq0).T
    assert np.array_equal(both, out + pdeq[pos])


def test_packed_size_of_the_mixed_precision_embedding():
    # Appendix on mixed-precision embedding: 4-bit word and 8-bit position embedding bring the table to
    # about 11.6 MB.  BERT-base: 30522 words + 2 token types at 4 bits, 512 positions at 8 bits, 768 dims.
    words = (30522 + 2) * 768 * 4 / 8
    positions = 512 * 768 * 8 / 8
    assert abs((words + positions) / 2**20 - 11.6) < 0.1
    st, codes, _, _ = oracle.quantize_embedding(_table(V=16), 4, 128)
    assert oracle.pack(codes, 4).nbytes == 16 * 768 * 4 // 8
