"""GPU: residual backup / restore in chunks, and fast-mode linears running beside a restore.

The paper's switch back to full mode first restores the lower byte of every weight from a host copy
while fast-mode steps keep running; fast mode never reads the residual plane, so its results must
not depend on what that plane holds at the time.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_34380_b200 as dps
from paper_2609_34380_b200 import workloads
from tests.helpers import assert_close_to_oracle, split_both, to_np_bytes, to_np_words

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("chunk", [0, 4096, 1 << 20, 3000])      # default 4 MiB, tiny, 1 MiB, ragged
def test_backup_poison_restore_is_bit_exact(chunk):
    w = workloads.weights(1024, 2064, 77, device=DEV)
    p, r, enc = dps.dps_split_weights(w, dps.DPS_ENC_AUTO)
    r_ref = r.clone()
    host = dps.dps_backup_residual(r, chunk_bytes=chunk)
    torch.cuda.synchronize()
    assert np.array_equal(host.numpy(), to_np_bytes(r_ref))
    r.fill_(0xAB)                                   # the plane's memory was lent out and overwritten
    dps.dps_restore_residual(r, host, chunk_bytes=chunk)
    torch.cuda.synchronize()
    assert torch.equal(r, r_ref)
    assert np.array_equal(workloads.as_words(dps.dps_reconstruct(p, r, enc)), to_np_words(w))


def test_empty_and_argument_checks():
    r = torch.empty(0, dtype=torch.uint8, device=DEV)
    host = torch.empty(0, dtype=torch.uint8).pin_memory()
    dps.dps_restore_residual(r, host)               # nothing to do, no error
    with pytest.raises(ValueError):
        dps.dps_restore_residual(torch.zeros(16, dtype=torch.uint8, device=DEV), torch.zeros(8, dtype=torch.uint8))
    with pytest.raises(ValueError):
        dps.dps_backup_residual(torch.zeros(16, dtype=torch.uint8, device=DEV),
                                torch.zeros(16, dtype=torch.uint8, device=DEV))


def test_fast_mode_steps_beside_a_restore_then_full_mode():
    n, k = 4096, 4096
    w = workloads.weights(n, k, 91, device=DEV)
    p, r, enc, p_ref, r_ref = split_both(w, dps.DPS_ENC_AUTO, DEV)
    host = dps.dps_backup_residual(r)
    x = workloads.activations(8, k, 92, device=DEV)
    y_alone = dps.dps_linear(dps.DPS_MODE_FAST, enc, x, p, None)
    torch.cuda.synchronize()
    r.fill_(0x5C)                                   # residual memory in other use
    copy_stream, compute = torch.cuda.Stream(), torch.cuda.Stream()
    restored = torch.cuda.Event()
    with torch.cuda.stream(copy_stream):
        dps.dps_restore_residual(r, host, chunk_bytes=1 << 20, stream=copy_stream)
        restored.record(copy_stream)
    ys = []
    with torch.cuda.stream(compute):
        for _ in range(20):                         # fast-mode steps while the copies are in flight; r passed on purpose
            ys.append(dps.dps_linear(dps.DPS_MODE_FAST, enc, x, p, r, stream=compute))
        compute.wait_event(restored)                # the switch to full mode is ordered after the restore
        y_full = dps.dps_linear(dps.DPS_MODE_FULL, enc, x, p, r, stream=compute)
    torch.cuda.synchronize()
    for y in ys:
        assert torch.equal(y, y_alone)
    assert np.array_equal(host.numpy(), r_ref)
    ref = oracle.linear(oracle.MODE_FULL, enc, to_np_words(x), p_ref, r_ref, threads=8)
    assert_close_to_oracle(y_full, ref, "full mode after restore")
    assert dps.dps_stream_status() == dps.DPS_OK
