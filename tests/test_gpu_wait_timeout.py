"""GPU: the bounded device-side wait gives up, reports it through the status word, and leaves the
device and the library fully usable (nothing in this test faults, traps or spins without a limit)."""
import time

import numpy as np
import pytest
import torch

import oracle
import paper_2609_34380_b200 as dps
from paper_2609_34380_b200 import binding, workloads
from tests.helpers import assert_close_to_oracle, to_np_words

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_wait_runs_out_sets_the_status_word_and_the_library_carries_on():
    assert dps.dps_stream_status() == dps.DPS_OK
    t0 = time.perf_counter()
    dps.dps_debug_wait_timeout(1_000_000)                 # 1 ms on a barrier nothing ever signals
    assert dps.dps_stream_status() == binding.DPS_ERR_CUDA   # the waiter gave up and said so
    elapsed = time.perf_counter() - t0
    assert 0.5e-3 <= elapsed < 1.0, elapsed               # it did wait, and only as long as told
    assert dps.dps_stream_status() == dps.DPS_OK          # reading the status cleared it
    # a tensor-core launch (the kernels that use this wait) right after is still correct
    w = workloads.weights(512, 1024, 9901)
    p_ref, r_ref, enc = oracle.split(to_np_words(w), oracle.ENC_AUTO)
    p, r = torch.from_numpy(p_ref).to(DEV), torch.from_numpy(r_ref).to(DEV)
    x = workloads.activations(48, 1024, 9902, device=DEV)
    for mode in (dps.DPS_MODE_FAST, dps.DPS_MODE_FULL):
        y = dps.dps_linear(mode, enc, x, p, r if mode else None)
        ref = oracle.linear(mode, enc, to_np_words(x), p_ref, r_ref, threads=8)
        assert_close_to_oracle(y, ref, f"after timeout, mode={mode}")
    assert dps.dps_stream_status() == dps.DPS_OK


def test_limit_is_validated_on_the_host():
    before = dps.dps_launch_count()
    for bad in (0, 2_000_000_000):
        with pytest.raises(dps.DpsError) as ei:
            dps.dps_debug_wait_timeout(bad)
        assert ei.value.status == binding.DPS_ERR_SHAPE
    assert dps.dps_launch_count() == before
    assert np.isfinite(before)
