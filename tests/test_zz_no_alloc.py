"""GPU test of qb_quantize_pack_weights_noalloc, the entry point for callers that cannot allocate.

Collected last on purpose (file name): a run that stops at the first failure has then already run
every other test.  The entry point keeps its scratch in an array inside the library, shared by all
calls, so the test makes two calls in a row -- the second on a different matrix, bit width and group
count -- and compares each with qb_quantize_pack_weights (caller workspace) on the same input and with
the CPU oracle's quantizer and packer.  Packed words, Delta and q0 are integer / byte-exact results in
this library's tests, so they must be equal.  The shapes are chosen so that each of the quantizer's paths
runs against the built-in scratch (status word, and the range tables of the two-pass path): several groups
per warp, groups cut over the warps of a CTA, a group held by a thread-block cluster, and the two passes.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_1909_05840_b200 as qb
from paper_1909_05840_b200 import build as qb_build
from paper_1909_05840_b200 import synth

pytestmark = pytest.mark.gpu


def _outputs(N, K, bits, groups):
    packed = torch.empty((N, K * bits // 32), dtype=torch.int32, device="cuda")
    packed.view(torch.uint8).fill_(0xFF)
    delta = torch.full((groups,), float("nan"), dtype=torch.float32, device="cuda")
    q0 = torch.full((groups,), float("nan"), dtype=torch.float32, device="cuda")
    return packed, delta, q0


def test_noalloc_matches_workspace_entry_point_twice_in_a_row():
    qb_build.build()
    ws = qb.workspace(groups=qb.NOALLOC_MAX_GROUPS)
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    # second call: fewer groups, other width and shape, so that stale ranges of call 1 would show
    # (768, 768, 12 groups): 384 units per group -> a cluster of two CTAs; (768, 3072, 1 group): the two passes
    for call, (N, K, bits, groups) in enumerate([(768, 768, 3, 768), (264, 384, 4, 11), (3072, 768, 2, 128),
                                                 (768, 768, 4, 12), (768, 3072, 8, 1)]):
        w_host = synth.weights(N, K, seed=900 + call)
        w = torch.from_numpy(w_host).cuda()
        ref_packed, ref_delta, ref_q0 = qb.quantize_pack_weights(w, bits, groups, ws)
        packed, delta, q0 = _outputs(N, K, bits, groups)
        qb.quantize_pack_weights_noalloc(w, bits, groups, packed, delta, q0, status_out=status)
        torch.cuda.synchronize()
        assert status.item() == qb.QB_OK
        assert torch.equal(packed, ref_packed), f"call {call}: packed words differ"
        assert torch.equal(delta, ref_delta) and torch.equal(q0, ref_q0), f"call {call}: group tables differ"
        # and against the oracle directly, not only against the library's other entry point
        st, codes, o_delta, o_q0 = oracle.quantize_weights(w_host, bits, groups, omp=True)
        assert st == oracle.OK
        assert np.array_equal(packed.cpu().numpy().view(np.uint32), oracle.pack(codes, bits)), f"call {call}: words vs oracle"
        assert np.array_equal(delta.cpu().numpy(), o_delta) and np.array_equal(q0.cpu().numpy(), o_q0)
    assert qb.read_status(ws) == qb.QB_OK

    # a non-finite weight is reported through status_out for that call only; the next call is clean again
    w = synth.weights(24, 128, seed=5)
    w[7, 3] = np.inf
    packed, delta, q0 = _outputs(24, 128, 4, 4)
    qb.quantize_pack_weights_noalloc(torch.from_numpy(w).cuda(), 4, 4, packed, delta, q0, status_out=status)
    torch.cuda.synchronize()
    assert status.item() == qb.QB_ERR_NONFINITE
    w[7, 3] = 0.0
    wd = torch.from_numpy(w).cuda()
    qb.quantize_pack_weights_noalloc(wd, 4, 4, packed, delta, q0, status_out=status)
    torch.cuda.synchronize()
    assert status.item() == qb.QB_OK
    ref = qb.quantize_pack_weights(wd, 4, 4, ws)
    assert torch.equal(packed, ref[0]) and torch.equal(delta, ref[1]) and torch.equal(q0, ref[2])


def test_noalloc_rejects_more_groups_than_its_scratch_holds():
    qb_build.build()
    N = 2 * qb.NOALLOC_MAX_GROUPS
    w = torch.zeros((N, 128), dtype=torch.float32, device="cuda")
    packed, delta, q0 = _outputs(N, 128, 2, N)
    packed.zero_()
    with pytest.raises(qb.QbertError) as err:
        qb.quantize_pack_weights_noalloc(w, 2, N, packed, delta, q0)
    assert err.value.status == qb.QB_ERR_WORKSPACE and "QB_NOALLOC_MAX_GROUPS" in str(err.value)
    torch.cuda.synchronize()
    assert not packed.any().item()  # nothing was launched
