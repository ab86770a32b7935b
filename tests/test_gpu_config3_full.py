"""GPU parity at the largest single-GPU workload, in the launch shape the benchmark times.

The 24-layer BERT-large stack (M = 24576, 4-bit weights, 128 groups per matrix) goes through ONE
qb_layer_linears call over all 96 linears, exactly as ``bench.py --config 3`` issues it: the library
sorts the linears by K, cuts them into launches of 48 (CTA pairs: tiles of 256 neurons x 256 tokens) and
walks each launch's tiles in identity order.  Checked against the CPU oracle:

* layer 0: every fp32 output and every int32 accumulator of its four linears;
* layers 1..23: a strided sample of 256 token rows per linear that covers every row position inside a
  256-token tile (so every TMEM column / staging row of the epilogue) and moves over the token tiles;
* every packed word, Delta and q0 of all 96 weight matrices, every activation code and row sum.

Activations are shared by the linears of one shape (as the benchmark does for deep stacks: four host
arrays instead of 96); every layer has its own weights and bias.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_1909_05840_b200 as qb
from paper_1909_05840_b200 import synth

import gpu_util as gu

pytestmark = pytest.mark.gpu


def _residue_rows(M: int, layer: int, matrix: int, tile: int = 256) -> np.ndarray:
    """One row for every position 0..tile-1 inside a token tile, spread over the tiles."""
    tiles = M // tile
    i = np.arange(tile, dtype=np.int64)
    return np.sort(i + tile * ((i * 37 + 5 * layer + matrix) % tiles))


def test_config3_whole_stack_in_the_benchmarked_launch_shape():
    gu.ensure_built()
    wl = synth.workload(3)
    M = wl.M
    assert M % 256 == 0 and wl.layers == 24 and len(wl.linears) == 4
    ws = qb.workspace(groups=max(32, wl.layers * sum(s.groups for s in wl.linears)))

    # activations: one tensor per linear shape, quantized once on each side
    act = {}
    for mi, s in enumerate(wl.linears):
        x = synth.activations(M, s.K, synth.seed_for(3, 0, mi))
        xq, sc, rs = gu.gpu_quantize_act(x, ws)
        st, o_xq, o_s, o_rs = oracle.quantize_act(x, omp=True)
        assert st == oracle.OK
        assert np.array_equal(xq.cpu().numpy(), o_xq), "activation codes differ"
        assert np.array_equal(rs.cpu().numpy(), o_rs) and sc.item() == o_s
        act[mi] = (xq, sc, rs, o_xq, o_s, o_rs)
        del x

    descs, refs, mats = [], [], []
    for layer in range(wl.layers):
        bits = wl.bits[layer]
        for mi, s in enumerate(wl.linears):
            seed = synth.seed_for(3, layer, mi)
            w = synth.weights(s.N, s.K, seed)
            b = synth.bias(s.N, seed)
            packed = gu.poison(torch.empty((s.N, s.K * bits // 32), dtype=torch.int32, device="cuda"))
            delta = gu.poison(torch.empty(s.groups, dtype=torch.float32, device="cuda"))
            q0 = gu.poison(torch.empty(s.groups, dtype=torch.float32, device="cuda"))
            mats.append((gu.dev(w), bits, s.groups, packed, delta, q0))
            y = gu.poison(torch.empty((M, s.N), dtype=torch.float32, device="cuda"))
            xq, sc, rs = act[mi][:3]
            descs.append(qb.LinearDesc(xq, sc, rs, packed, delta, q0, gu.dev(b), s.N, bits, s.groups, y))
            refs.append((layer, mi, w, b, bits, s))
    qb.quantize_pack_weights_batch(mats, ws)
    qb.layer_linears(descs, ws)   # 96 linears: two launches of 48, CTA pairs, BT = 256, identity tile order
    torch.cuda.synchronize()
    assert qb.read_status(ws) == qb.QB_OK

    for d, (layer, mi, w, b, bits, s) in zip(descs, refs):
        o_xq, o_s, o_rs = act[mi][3:]
        st, codes, o_delta, o_q0 = oracle.quantize_weights(w, bits, s.groups, omp=True)
        assert st == oracle.OK
        assert np.array_equal(gu.words_np(d.packed), oracle.pack(codes, bits)), (layer, mi, "packed words")
        assert np.array_equal(d.delta.cpu().numpy(), o_delta) and np.array_equal(d.q0.cpu().numpy(), o_q0)
        if layer == 0:
            # the whole linear: every output of the stack call, every accumulator of the single call
            o_acc = oracle.int_gemm(o_xq, codes, omp=True)
            o_y = oracle.dequant_epilogue(o_acc, o_rs, o_s, o_delta, o_q0, b, bits, s.groups, omp=True)
            y_g = d.y.cpu().numpy()
            gu.assert_y_close(y_g, o_y)
            assert np.array_equal(y_g, o_y), "same IEEE operations in the same order: expected bit-equal"
            y1, acc1 = qb.gemm(d.xq, d.act_scale, d.rowsum, d.packed, d.delta, d.q0, d.bias, d.N, bits, s.groups, ws,
                               want_acc=True)
            assert torch.equal(y1, d.y), "the stack must equal the single call bit for bit"
            assert np.array_equal(acc1.cpu().numpy(), o_acc), (layer, mi, "int32 accumulators")
            del o_acc, o_y, y_g, y1, acc1
        else:
            rows = _residue_rows(M, layer, mi)
            assert len(set(int(r) % 256 for r in rows)) == 256
            o_acc = oracle.int_gemm(o_xq[rows], codes, omp=True)
            o_y = oracle.dequant_epilogue(o_acc, o_rs[rows], o_s, o_delta, o_q0, b, bits, s.groups)
            y_g = d.y[torch.from_numpy(rows).cuda()].cpu().numpy()
            gu.assert_y_close(y_g, o_y)
        d.y = None  # free the 75-400 MB output as soon as it is checked
    assert qb.read_status(ws) == qb.QB_OK
