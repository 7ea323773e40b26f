"""GPU: the 32-layer decoder step of config 5 at full scale (hidden 8192, ffn 28672, GQA QKV; 27.4 GB of
persistent and 27.4 GB of residual planes), dispatched per step as one of two CUDA graphs per batch size.

Checked: (1) two steps of equal mode give the same bits in every output of every layer, whatever ran in
between (the residual planes are overwritten before fast steps and put back before full ones: fast mode must
not notice); (2) layer 0, every output of all four linears, against the FP64 oracle on the oracle's own
planes, at 1 and 16 tokens in both modes; (3) for the larger batch sizes, equal-mode steps again bit for bit.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_34380_b200 as dps
from paper_2609_34380_b200 import workloads
from tests.helpers import assert_close_to_oracle, split_both, to_np_words

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_32_layer_step_equal_modes_equal_bits_and_layer0_against_the_oracle():
    layers, shapes = workloads.DECODER70_LAYERS, workloads.DECODER70
    if torch.cuda.mem_get_info()[0] < 70 << 30:
        pytest.skip("needs 70 GB of free device memory")
    planes, ref0 = [], {}
    for layer in range(layers):
        row = {}
        for i, (name, (n, k)) in enumerate(shapes.items()):
            w = workloads.weights(n, k, 5000 + layer * 4 + i, device=DEV)
            if layer == 0:
                p, r, enc, p_ref, r_ref = split_both(w, dps.DPS_ENC_AUTO, DEV)
                ref0[name] = (p_ref, r_ref)
            else:
                p, r, enc = dps.dps_split_weights(w, dps.DPS_ENC_AUTO)
            row[name] = (p, r, enc)
            del w
        planes.append(row)
    layer0_r = [r for (_, r, _) in planes[0].values()]
    keep0 = [r.clone() for r in layer0_r]
    stream = torch.cuda.Stream()
    for M in workloads.STEP_M:
        xs = {name: workloads.activations(M, k, 5901 + i, device=DEV) for i, (name, (n, k)) in enumerate(shapes.items())}
        ys = {(layer, name): torch.zeros((M, n), dtype=torch.float16, device=DEV)
              for layer in range(layers) for name, (n, k) in shapes.items()}

        def enqueue(mode):
            for layer, row in enumerate(planes):
                for name, (p, r, enc) in row.items():
                    dps.dps_linear(mode, enc, xs[name], p, r if mode else None, ys[(layer, name)])

        graphs = {}
        with torch.cuda.stream(stream):
            for mode in (0, 1):
                enqueue(mode)
                stream.synchronize()
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=stream):
                    enqueue(mode)
                graphs[mode] = g
        first = {}
        for t, mode in enumerate([1, 0, 0, 1, 0, 1]):
            with torch.cuda.stream(stream):
                for r, keep in zip(layer0_r, keep0):          # residual memory in other use during fast steps
                    if mode == dps.DPS_MODE_FAST:
                        r.fill_(0xEE)
                    else:
                        r.copy_(keep)
                graphs[mode].replay()
            stream.synchronize()
            if mode not in first:
                first[mode] = {k: v.clone() for k, v in ys.items()}
            else:
                for k, v in ys.items():
                    assert torch.equal(v.view(torch.int16), first[mode][k].view(torch.int16)), (M, t, mode, k)
        if M in (1, 16):
            for mode in (dps.DPS_MODE_FAST, dps.DPS_MODE_FULL):
                for name, (p, r, enc) in planes[0].items():
                    p_ref, r_ref = ref0[name]
                    ref = oracle.linear(mode, enc, to_np_words(xs[name]), p_ref, r_ref, threads=32)
                    assert_close_to_oracle(first[mode][(0, name)], ref, f"layer 0 {name} M={M} mode={mode}")
        del graphs, ys, xs, first
    for r, keep in zip(layer0_r, keep0):
        assert torch.equal(r, keep)
    assert np.isfinite(float(layers))
    assert dps.dps_stream_status() == dps.DPS_OK
