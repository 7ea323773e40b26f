"""GPU: decode steps whose precision mode comes from the shared-region manager model.

The manager (Algorithm 1's allocation / release, section "KV-Cache-Pressure-aware DPS") is fed a bursty
KV occupancy trace.  When it evicts a layer's residual tensor the test overwrites that layer's residual
planes (as KV-cache writes would); when it restores one, the planes are copied back from the pinned host
backup in chunks on a copy stream, and a full-mode step runs only after every started copy has landed.
Every step's outputs must equal the fixed-mode outputs bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_34380_b200 as dps
from paper_2609_34380_b200 import sum_manager as sm, workloads
from tests.helpers import assert_close_to_oracle, to_np_words

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_manager_driven_schedule_with_eviction_poison_and_chunked_restore():
    layers, M = 6, 8
    shapes = [(384, 512), (256, 768)]                        # two linears per layer
    planes, enc_of, x_of = [], [], []
    for layer in range(layers):
        row = []
        for i, (n, k) in enumerate(shapes):
            w = workloads.weights(n, k, 6100 + 10 * layer + i)
            p_ref, r_ref, enc = oracle.split(to_np_words(w), oracle.ENC_AUTO)
            row.append((torch.from_numpy(p_ref).to(DEV), torch.from_numpy(r_ref).to(DEV), enc, p_ref, r_ref))
        planes.append(row)
    xs = [workloads.activations(M, k, 6200 + i, device=DEV) for i, (n, k) in enumerate(shapes)]

    def run(mode):
        return [dps.dps_linear(mode, enc, xs[i], p, r if mode else None)
                for row in planes for i, (p, r, enc, _, _) in enumerate(row)]

    want = {mode: run(mode) for mode in (dps.DPS_MODE_FAST, dps.DPS_MODE_FULL)}
    # the fixed-mode outputs themselves against the oracle (layer 0)
    for mode in (dps.DPS_MODE_FAST, dps.DPS_MODE_FULL):
        for i, (p, r, enc, p_ref, r_ref) in enumerate(planes[0]):
            ref = oracle.linear(mode, enc, to_np_words(xs[i]), p_ref, r_ref, threads=4)
            assert_close_to_oracle(want[mode][i], ref, f"layer 0 linear {i} mode {mode}")

    copy_stream = torch.cuda.Stream()
    store = sm.ResidualPlanes([[r for (_, r, _, _, _) in row] for row in planes], copy_stream, poison=True,
                              chunk_bytes=64 << 10)          # several chunks per plane
    units, bpu = 12, 4
    mgr = sm.SumManager(units, bpu, layers, on_evict=store.on_evict, on_restore=store.on_restore)
    demand = sm.kv_demand_trace(400, units * bpu, seed=6300)
    driver = sm.TraceDriver(mgr, demand, steps_per_restore=2, ready=store.landed)
    seen = {dps.DPS_MODE_FAST: 0, dps.DPS_MODE_FULL: 0}
    for step in range(len(demand)):
        mode = driver.mode()
        got = run(mode)
        for a, b in zip(got, want[mode]):
            assert torch.equal(a.view(torch.int16), b.view(torch.int16)), (step, mode)
        seen[mode] += 1
        driver.advance()
        mgr.check()
    assert seen[dps.DPS_MODE_FAST] > 20 and seen[dps.DPS_MODE_FULL] > 20, seen
    assert store.evictions > 0 and store.restored_bytes > 0
    # drain: give everything back, restore what is still evicted, and full mode works on the restored bytes
    mgr.free_kv_blocks(driver.held)
    mgr.restore_weights()
    copy_stream.synchronize()
    assert mgr.mode == sm.MODE_FULL and store.landed()
    for a, b in zip(run(dps.DPS_MODE_FULL), want[dps.DPS_MODE_FULL]):
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    for row in planes:                                       # and the planes are the original bytes again
        for (_, r, _, _, r_ref) in row:
            assert np.array_equal(r.cpu().numpy(), r_ref)
    assert dps.dps_stream_status() == dps.DPS_OK
