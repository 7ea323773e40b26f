"""GPU: the orderings the header promises for planes that change on the stream.

The linear kernels fetch planes before they wait for the kernel launched just before them, so a plane must
not be written by THAT kernel; planes written by dps_split_weights (which ends with a fence launch) or by an
asynchronous copy are safe without any synchronisation in between.  Here the same plane buffers are
rewritten again and again, alternating between two different weight tensors, and each rewrite is followed
at once -- same stream, no synchronisation -- by linears of every kernel family; a stale fetch would show up
as the other tensor's result."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_34380_b200 as dps
from paper_2609_34380_b200 import workloads
from tests.helpers import assert_close_to_oracle, to_np_words

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("M", [4, 16, 48, 600])          # streaming kernel, tcgen05 decode tiles, prefill tiles
def test_split_then_linear_and_copy_then_linear_without_synchronising(M):
    N, K = 1024, 2048
    ws = [workloads.weights(N, K, 8100 + i, device=DEV) for i in range(2)]
    refs = [oracle.split(to_np_words(w), oracle.ENC_E5M2) for w in ws]
    good = [dps.dps_split_weights(w, dps.DPS_ENC_E5M2) for w in ws]          # pristine planes to copy from
    x = workloads.activations(M, K, 8200, device=DEV)
    xn = to_np_words(x)
    want = {(i, mode): oracle.linear(mode, refs[i][2], xn, refs[i][0], refs[i][1], threads=8)
            for i in range(2) for mode in (0, 1)}
    p = torch.zeros((N, K), dtype=torch.uint8, device=DEV)
    r = torch.zeros((N, K), dtype=torch.uint8, device=DEV)
    outs = []
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for rep in range(6):
            i = rep % 2
            if rep < 3:       # split straight into the live planes (explicit E5M2: the call never synchronises)
                dps.dps_split_weights(ws[i], dps.DPS_ENC_E5M2, p, r, stream=stream)
            else:             # asynchronous device-to-device copies into the live planes
                p.copy_(good[i][0], non_blocking=True)
                r.copy_(good[i][1], non_blocking=True)
            for mode in (0, 1):
                outs.append((i, mode, dps.dps_linear(mode, dps.DPS_ENC_E5M2, x, p, r if mode else None, stream=stream)))
    stream.synchronize()
    for i, mode, y in outs:
        assert_close_to_oracle(y, want[(i, mode)], f"rewrite {i} mode {mode} M={M}")
    assert not np.allclose(want[(0, 1)], want[(1, 1)])
    assert dps.dps_stream_status() == dps.DPS_OK
