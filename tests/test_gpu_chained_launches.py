"""GPU: chains of dependent launches on one stream, each layer's output the next layer's input.

Every dense kernel requests weight planes BEFORE it waits for the kernel in front of it (programmatic
dependent launch) and reads the activations only after; the tensor-core decode tiles additionally run planes
and activations as two streams with barriers of their own.  A mistake there does not show in a single launch:
it shows as a layer reading activations that the layer before it has not finished writing.  So the same chain
is run twice -- launches back to back, and with the device drained after every launch -- and the two results
must agree bit for bit; the first layer is also checked against the oracle.
"""
import pytest
import torch

import oracle
import paper_2609_34380_b200 as dps
from paper_2609_34380_b200 import workloads
from tests.helpers import assert_close_to_oracle, split_both, to_np_words

gpu = pytest.mark.gpu
DEV = "cuda:0"
LAYERS = 12


def _chain(planes, x0, mode, drain):
    x = x0
    outs = []
    for (p, r, enc) in planes:
        y = torch.empty((x.shape[0], p.shape[0]), dtype=torch.float16, device=DEV)
        dps.dps_linear(mode, enc, x, p, r if mode else None, y)
        if drain:
            torch.cuda.synchronize()
        outs.append(y)
        x = y
    torch.cuda.synchronize()
    return outs


@gpu
@pytest.mark.parametrize("mode", [dps.DPS_MODE_FAST, dps.DPS_MODE_FULL])
@pytest.mark.parametrize("M", [1, 8, 16, 32, 33, 64, 100, 200])
def test_back_to_back_chain_equals_drained_chain(M, mode):
    # square layers so that an output feeds the next input; weights scaled to keep the chain's magnitudes
    # level (row sums of K = 2048 terms); four distinct matrices in rotation
    N = K = 2048
    planes, refs = [], []
    for i in range(4):
        w = workloads.weights(N, K, 7100 + i, device=DEV)
        w = (w.float() * (1.0 / (w.float().std().item() * K ** 0.5))).to(torch.float16)
        p, r, enc, p_ref, r_ref = split_both(w, dps.DPS_ENC_AUTO, DEV)
        planes.append((p, r, enc))
        refs.append((p_ref, r_ref))
    planes = [planes[i % 4] for i in range(LAYERS)]
    x0 = workloads.activations(M, K, 7200 + M, device=DEV)
    drained = _chain(planes, x0, mode, drain=True)
    for attempt in range(3):      # the overlap of consecutive launches differs from run to run
        chained = _chain(planes, x0, mode, drain=False)
        for layer, (a, b) in enumerate(zip(chained, drained)):
            assert torch.equal(a.view(torch.int16), b.view(torch.int16)), f"layer {layer}, attempt {attempt}"
    assert torch.isfinite(drained[-1].float()).all()
    assert float(drained[-1].float().abs().max()) > 0.0
    p_ref, r_ref = refs[0]
    ref = oracle.linear(mode, planes[0][2], to_np_words(x0), p_ref, r_ref, threads=8)
    assert_close_to_oracle(drained[0], ref, f"first layer M={M} mode={mode}")
    assert dps.dps_stream_status() == dps.DPS_OK


@gpu
@pytest.mark.parametrize("mode", [dps.DPS_MODE_FAST, dps.DPS_MODE_FULL])
def test_chain_inside_a_cuda_graph(mode):
    # the same at 32 tokens with the chain captured once and replayed: replays overlap their own tail and head
    N = K = 2048
    M = 32
    planes = []
    for i in range(4):
        w = workloads.weights(N, K, 7300 + i, device=DEV)
        w = (w.float() * (1.0 / (w.float().std().item() * K ** 0.5))).to(torch.float16)
        p, r, enc, _, _ = split_both(w, dps.DPS_ENC_AUTO, DEV)
        planes.append((p, r, enc))
    planes = [planes[i % 4] for i in range(LAYERS)]
    x0 = workloads.activations(M, K, 7400, device=DEV)
    drained = _chain(planes, x0, mode, drain=True)
    bufs = [torch.empty((M, N), dtype=torch.float16, device=DEV) for _ in range(LAYERS)]

    def enqueue():
        x = x0
        for (p, r, enc), y in zip(planes, bufs):
            dps.dps_linear(mode, enc, x, p, r if mode else None, y)
            x = y

    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        enqueue()
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            enqueue()
        for _ in range(5):
            for y in bufs:
                y.zero_()
            g.replay()
            stream.synchronize()
            for layer, (a, b) in enumerate(zip(bufs, drained)):
                assert torch.equal(a.view(torch.int16), b.view(torch.int16)), f"layer {layer}"
    assert dps.dps_stream_status() == dps.DPS_OK


@gpu
@pytest.mark.parametrize("mode", [dps.DPS_MODE_FAST, dps.DPS_MODE_FULL])
@pytest.mark.parametrize("T", [24, 160])
def test_grouped_chain_equals_drained_chain(T, mode):
    # a gate/up-style call (token map) followed by down-style calls (rows are their own tokens), every output
    # the next input, with one workspace shared by all calls as a serving loop would
    E, N = 4, 1024
    K = N
    ps, rs, encs = [], [], []
    for e in range(E):
        w = workloads.weights(N, K, 7500 + e, device=DEV)
        w = (w.float() * (1.0 / (w.float().std().item() * K ** 0.5))).to(torch.float16)
        p, r, enc, _, _ = split_both(w, dps.DPS_ENC_AUTO, DEV)
        ps.append(p), rs.append(r), encs.append(enc)
    p, r = torch.stack(ps), torch.stack(rs)
    tor, eor = workloads.top2_routing(T, E, 7600 + T)
    tor_d, eor_d = torch.from_numpy(tor).to(DEV), torch.from_numpy(eor).to(DEV)
    A = eor.size
    x0 = workloads.activations(T, K, 7700 + T, device=DEV)
    ws = torch.empty(dps.dps_moe_workspace_bytes(A, E, K), dtype=torch.uint8, device=DEV)

    def chain(drain):
        outs = []
        x, tmap = x0, tor_d
        for _ in range(6):
            y = torch.empty((A, N), dtype=torch.float16, device=DEV)
            dps.dps_moe_linear(mode, encs, x, tmap, eor_d, p, r if mode else None, y, ws)
            if drain:
                torch.cuda.synchronize()
            outs.append(y)
            x, tmap = y, None
        torch.cuda.synchronize()
        return outs

    drained = chain(True)
    for attempt in range(3):
        for layer, (a, b) in enumerate(zip(chain(False), drained)):
            assert torch.equal(a.view(torch.int16), b.view(torch.int16)), f"layer {layer}, attempt {attempt}"
    assert torch.isfinite(drained[-1].float()).all()
    assert dps.dps_stream_status() == dps.DPS_OK
