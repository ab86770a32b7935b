"""A bounded device-side wait that runs out, without hanging or faulting anything.

qb_probe_wait_limit launches one small kernel that waits, with the GEMM's own wait routines, on an
mbarrier at which nothing ever arrives.  The wait must give up after its cycle limit, the kernel must
record QB_ERR_TIMEOUT in the workspace's status word and exit normally, and the next ordinary call (on
a fresh workspace) must run and be bit-exact against the oracle."""
import numpy as np
import pytest
import torch

import paper_1909_05840_b200 as qb
from paper_1909_05840_b200 import synth

import gpu_util as gu

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("limit", [200_000, 2_000_000])
def test_wait_runs_out_and_reports_timeout(limit):
    gu.ensure_built()
    ws = qb.workspace(groups=32)
    assert qb.read_status(ws) == qb.QB_OK
    waited = qb.probe_wait_limit(ws, limit)
    torch.cuda.synchronize()
    assert qb.read_status(ws) == qb.QB_ERR_TIMEOUT
    w = waited.cpu().numpy()
    # both waiting warps gave up after the limit, and not long after it (the limit is checked every 64 polls
    # of at most about a microsecond each)
    assert np.all(w > limit) and np.all(w < limit + 2_000_000), w
    # the status word is sticky: a second expiry leaves the first record in place
    qb.probe_wait_limit(ws, limit)
    torch.cuda.synchronize()
    assert qb.read_status(ws) == qb.QB_ERR_TIMEOUT
    # the context is intact: an ordinary call on a fresh workspace is bit-exact against the oracle
    ws2 = qb.workspace(groups=32)
    x = synth.activations(300, 384, seed=41)
    wgt = synth.weights(264, 384, seed=42)
    b = synth.bias(264, seed=43)
    gu.check_linear(x, wgt, b, 3, 11, ws2)
    assert qb.read_status(ws2) == qb.QB_OK


def test_wait_limit_argument_errors():
    gu.ensure_built()
    ws = qb.workspace(groups=32)
    with pytest.raises(qb.QbertError) as e:
        qb.probe_wait_limit(ws, 10)
    assert e.value.status == qb.QB_ERR_INVALID
    torch.cuda.synchronize()
    assert qb.read_status(ws) == qb.QB_OK
