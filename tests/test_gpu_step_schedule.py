"""GPU: per-step mode dispatch (one mode per forward pass, two CUDA graphs per batch size) and the
config-5 decoder shapes."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_34380_b200 as dps
from paper_2609_34380_b200 import workloads
from tests.helpers import assert_close_to_oracle, split_both, to_np_words, y_as_f64

gpu = pytest.mark.gpu
DEV = "cuda:0"


class MiniDecoder:
    """L layers x 4 linears with nested planes; one captured graph per mode for a fixed batch size."""

    def __init__(self, layers, shapes, M, seed):
        self.shapes, self.M = shapes, M
        self.planes, self.ref_planes = [], []              # GPU planes; the oracle's own planes of the same words
        for layer in range(layers):
            row, ref_row = {}, {}
            for i, (name, (n, k)) in enumerate(shapes.items()):
                w = workloads.weights(n, k, seed + layer * 4 + i, device=DEV)
                p, r, enc, p_ref, r_ref = split_both(w, dps.DPS_ENC_AUTO, DEV)
                row[name], ref_row[name] = (p, r, enc), (p_ref, r_ref)
            self.planes.append(row)
            self.ref_planes.append(ref_row)
        self.x = {name: workloads.activations(M, k, 5901 + i, device=DEV) for i, (name, (n, k)) in enumerate(shapes.items())}
        self.y = {(layer, name): torch.zeros((M, n), dtype=torch.float16, device=DEV)
                  for layer in range(layers) for name, (n, k) in shapes.items()}
        self.graphs = {}
        stream = torch.cuda.Stream()
        with torch.cuda.stream(stream):
            for mode in (dps.DPS_MODE_FAST, dps.DPS_MODE_FULL):
                self.enqueue(mode)                       # warm-up outside capture
            stream.synchronize()
            for mode in (dps.DPS_MODE_FAST, dps.DPS_MODE_FULL):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=stream):
                    self.enqueue(mode)
                self.graphs[mode] = g
        torch.cuda.synchronize()

    def enqueue(self, mode):
        for layer, row in enumerate(self.planes):
            for name, (p, r, enc) in row.items():
                dps.dps_linear(mode, enc, self.x[name], p, r if mode else None, self.y[(layer, name)])

    def step(self, mode):
        self.graphs[mode].replay()
        torch.cuda.synchronize()
        return {k: v.clone() for k, v in self.y.items()}


@gpu
@pytest.mark.parametrize("M", [1, 16])
def test_schedule_outputs_depend_only_on_the_mode_of_the_step(M):
    shapes = {"qkv": (1280, 1024), "o": (1024, 1024), "gate_up": (7168, 1024), "down": (1024, 3584)}
    model = MiniDecoder(3, shapes, M, 5000)
    schedule = workloads.mode_schedule(40, 5555)
    assert schedule[0] == 1 and 0 in schedule and 1 in schedule
    first = {}
    for t, mode in enumerate(schedule):
        if mode == dps.DPS_MODE_FAST:
            # the residual's memory may be reused between passes: poison it before a fast step
            poison = [(r, r.clone()) for row in model.planes for (p, r, enc) in row.values()]
            for r, _ in poison:
                r.fill_(0xEE)
        out = model.step(mode)
        if mode == dps.DPS_MODE_FAST:
            for r, keep in poison:
                r.copy_(keep)
        if mode not in first:
            first[mode] = out
        else:                                            # same mode => same bits, whatever came before
            for k, v in out.items():
                assert torch.equal(v.view(torch.int16), first[mode][k].view(torch.int16)), (t, mode, k)
    # layer 0 against the oracle, both modes
    for mode in (dps.DPS_MODE_FAST, dps.DPS_MODE_FULL):
        for name, (p, r, enc) in model.planes[0].items():
            p_ref, r_ref = model.ref_planes[0][name]
            ref = oracle.linear(mode, enc, to_np_words(model.x[name]), p_ref, r_ref, threads=16)
            assert_close_to_oracle(first[mode][(0, name)], ref, f"{name} mode={mode}")
    assert dps.dps_stream_status() == dps.DPS_OK


def test_schedule_generator_is_seeded_and_bursty():
    a, b = workloads.mode_schedule(256, 5555), workloads.mode_schedule(256, 5555)
    assert a == b and len(a) == 256 and a[0] == 1
    assert workloads.mode_schedule(256, 5556) != a
    fast_share = a.count(0) / len(a)
    assert 0.4 < fast_share < 0.85
    switches = sum(1 for i in range(1, len(a)) if a[i] != a[i - 1])
    assert 6 <= switches <= 40                           # long stretches, few transitions


@gpu
@pytest.mark.parametrize("M", [1, 16, 64, 256])
def test_decoder70_layer_shapes_sampled(M):
    """Config 5 shapes (hidden 8192, ffn 28672, GQA QKV): one layer at full size, sampled outputs."""
    for i, (name, (N, K)) in enumerate(workloads.DECODER70.items()):
        w = workloads.weights(N, K, 5000 + i, device=DEV)
        p, r, enc, p_ref, r_ref = split_both(w, dps.DPS_ENC_AUTO, DEV)
        del w
        x = workloads.activations(M, K, 5901 + i, device=DEV)
        ms, ns = workloads.sample_entries(M, N, 768, 5999 + M)
        ns[:4] = [0, 127, 128, N - 1]
        rows = np.unique(ns)
        pn, rn = p_ref[rows], r_ref[rows]                  # reference side: the oracle's own planes
        idx = np.searchsorted(rows, ns)
        xn = to_np_words(x)
        for mode in (dps.DPS_MODE_FAST, dps.DPS_MODE_FULL):
            y = dps.dps_linear(mode, enc, x, p, r if mode else None)
            ref = oracle.linear_at(mode, enc, xn, pn, rn, ms, idx)
            got = y_as_f64(y)[ms, ns]
            assert np.max(np.abs(got - ref)) <= 2e-3 * np.max(np.abs(ref)), (name, M, mode)
        del p, r
    assert dps.dps_stream_status() == dps.DPS_OK
