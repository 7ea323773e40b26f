"""GPU parity: prefill-sized linears (config 3) on the tensor-core path."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_34380_b200 as dps
from paper_2609_34380_b200 import workloads
from tests.helpers import assert_close_to_oracle, split_both, to_np_words, y_as_f64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
MODES = [dps.DPS_MODE_FAST, dps.DPS_MODE_FULL]


def test_o_proj_m512_full_check():
    """O projection, 512 tokens: every output against the FP64 oracle, both modes."""
    N, K = workloads.LLAMA7B["o"]
    w = workloads.weights(N, K, 2002, device=DEV)
    p, r, enc, p_ref, r_ref = split_both(w, dps.DPS_ENC_AUTO, DEV)
    x = workloads.activations(512, K, 3001, device=DEV)
    for mode in MODES:
        y = dps.dps_linear(mode, enc, x, p, r if mode else None)
        ref = oracle.linear(mode, enc, to_np_words(x), p_ref, r_ref, threads=16)
        assert_close_to_oracle(y, ref, f"o M=512 mode={mode}")
    assert dps.dps_stream_status() == dps.DPS_OK


@pytest.mark.parametrize("M", [512, 2048, 8192])
def test_llama7b_prefill_sampled(M):
    """All four linears at prefill sizes: 16 whole output rows' worth of samples plus random entries."""
    for i, (name, (N, K)) in enumerate(workloads.LLAMA7B.items()):
        w = workloads.weights(N, K, 2001 + i, device=DEV)
        p, r, enc, pn, rn = split_both(w, dps.DPS_ENC_AUTO, DEV)
        del w
        x = workloads.activations(M, K, 3001 + i, device=DEV)
        xn = to_np_words(x)
        ms, ns = workloads.sample_entries(M, N, 1536, 3999)
        # corners and tile borders of the output
        ms[:8] = [0, 0, M - 1, M - 1, 127, 128, M - 129, M - 128]
        ns[:8] = [0, N - 1, 0, N - 1, 127, 128, N - 129, N - 128]
        for mode in MODES:
            y = dps.dps_linear(mode, enc, x, p, r if mode else None)
            ref = oracle.linear_at(mode, enc, xn, pn, rn, ms, ns)
            got = y_as_f64(y[torch.from_numpy(ms).to(DEV), torch.from_numpy(ns).to(DEV)])
            scale = np.max(np.abs(ref))
            assert np.max(np.abs(got - ref)) <= 2e-3 * scale, (name, M, mode)
            del y
        del x, p, r
    assert dps.dps_stream_status() == dps.DPS_OK


def test_prefill_determinism():
    N, K, M = 4096, 4096, 1024
    w = workloads.weights(N, K, 7, device=DEV)
    p, r, enc = dps.dps_split_weights(w, dps.DPS_ENC_E5M2)
    x = workloads.activations(M, K, 8, device=DEV)
    a = dps.dps_linear(dps.DPS_MODE_FULL, enc, x, p, r)
    b = dps.dps_linear(dps.DPS_MODE_FULL, enc, x, p, r)
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))


@pytest.mark.parametrize("enc_req", [dps.DPS_ENC_AUTO, dps.DPS_ENC_E5M2])
def test_persistent_kernel_ragged_shapes_every_output(enc_req):
    """More tiles than SMs with a short last round, ragged in every direction: N = 2056 (17 row
    tiles, the last with 8 rows), K = 1104 (a partial last K block, an odd number of blocks to halve),
    M = 2500 (partial last token tile).  Full mode walks 170 tiles of 256 tokens, fast mode 180
    two-row-block tiles; in both the last round is shared out as halves of K.  Every output is checked."""
    N, K, M = 2056, 1104, 2500
    w = workloads.weights(N, K, 611, device=DEV)
    p, r, enc, p_ref, r_ref = split_both(w, enc_req, DEV)
    x = workloads.activations(M, K, 612, device=DEV)
    for mode in MODES:
        y = dps.dps_linear(mode, enc, x, p, r if mode else None)
        ref = oracle.linear(mode, enc, to_np_words(x), p_ref, r_ref, threads=16)
        assert_close_to_oracle(y, ref, f"ragged persistent mode={mode} enc={enc}")
        again = dps.dps_linear(mode, enc, x, p, r if mode else None)
        assert torch.equal(y, again)              # the pair reduction adds in a fixed order
    assert dps.dps_stream_status() == dps.DPS_OK
