"""GPU: the allocation-free grouped linear (dps_moe_linear_static) against dps_moe_linear.

This file is collected last on purpose: should the new entry point misbehave, a run that stops at
the first failure has already exercised every other test.  The checks pass both in a fresh
process (where the first call performs the one-time address look-up of the built-in scratch) and
after the rest of the suite.

Who needs this entry point: callers that are not allowed to allocate device memory while they
run -- for instance a serving worker that committed all free memory to weight planes and KV
cache at start-up -- and therefore cannot provide the workspace dps_moe_linear asks for.
"""
import pytest
import torch

import paper_2609_34380_b200 as dps
from paper_2609_34380_b200 import binding, workloads

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _problem(E, N, K, T, seed):
    ps, rs, encs = [], [], []
    for e in range(E):
        w = workloads.weights(N, K, seed + e, device=DEV)
        if e % 3 == 1:
            w = workloads.with_outlier(w)                 # mixes E5M2 experts in
        p, r, enc = dps.dps_split_weights(w, dps.DPS_ENC_AUTO)
        ps.append(p), rs.append(r), encs.append(enc)
    x = workloads.activations(T, K, seed + 100, device=DEV)
    tor, eor = workloads.top2_routing(T, E, seed + 200)
    return (torch.stack(ps), torch.stack(rs), encs, x, torch.from_numpy(tor).to(DEV), torch.from_numpy(eor).to(DEV))


def _compare(mode, prob):
    p, r, encs, x, tor, eor = prob
    want = dps.dps_moe_linear(mode, encs, x, tor, eor, p, r if mode else None)
    got = torch.full_like(want, 7.0)
    dps.dps_moe_linear_static(mode, encs, x, tor, eor, p, r if mode else None, got)
    torch.cuda.synchronize()
    # the two entry points run the same deterministic kernels: the outputs must agree bit for bit
    assert bool(torch.isfinite(got).all())
    assert torch.equal(got.view(torch.int16), want.view(torch.int16))
    return got


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    first = _problem(8, 264, 528, 96, 9100)               # ragged tiles, several experts, 192 rows
    second = _problem(3, 136, 1040, 21, 9200)             # a different, smaller problem right after
    for mode in (dps.DPS_MODE_FAST, dps.DPS_MODE_FULL):
        out1 = _compare(mode, first)
        _compare(mode, second)                            # reuses the scratch the first call left behind
        out1_again = _compare(mode, first)                # and the first problem is unaffected by it
        assert torch.equal(out1.view(torch.int16), out1_again.view(torch.int16))
    assert dps.dps_stream_status() == dps.DPS_OK


def test_problem_beyond_the_built_in_scratch_is_rejected():
    A, E, K, N = 4096, 8, 4096, 64                        # 4096 x 4096 FP16 activations alone are 32 MiB
    assert dps.dps_moe_workspace_bytes(A, E, K) > binding.DPS_MOE_STATIC_SCRATCH_BYTES
    p = torch.zeros((E, N, K), dtype=torch.uint8, device=DEV)
    x = torch.zeros((A, K), dtype=torch.float16, device=DEV)
    eor = torch.zeros(A, dtype=torch.int32, device=DEV)
    y = torch.full((A, N), 3.0, dtype=torch.float16, device=DEV)
    before = dps.dps_launch_count()
    with pytest.raises(dps.DpsError) as ei:
        dps.dps_moe_linear_static(dps.DPS_MODE_FAST, [dps.DPS_ENC_E5M2] * E, x, None, eor, p, None, y)
    assert ei.value.status == binding.DPS_ERR_WORKSPACE
    assert dps.dps_launch_count() == before               # nothing was enqueued
    torch.cuda.synchronize()
    assert bool((y == 3.0).all())


def test_no_device_memory_is_allocated_by_the_call():
    prob = _problem(4, 128, 256, 16, 9300)
    p, r, encs, x, tor, eor = prob
    y = torch.empty((eor.numel(), p.shape[1]), dtype=torch.float16, device=DEV)
    dps.dps_moe_linear_static(dps.DPS_MODE_FULL, encs, x, tor, eor, p, r, y)      # set-up call
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    reserved_before = torch.cuda.memory_reserved()
    for _ in range(3):
        dps.dps_moe_linear_static(dps.DPS_MODE_FULL, encs, x, tor, eor, p, r, y)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert torch.cuda.memory_reserved() == reserved_before
    assert free_after == free_before
