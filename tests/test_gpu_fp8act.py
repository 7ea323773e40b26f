"""GPU parity: fast mode with FP8 activations (per-token E4M3 quantisation + FP8 tensor-core linear)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_34380_b200 as dps
from paper_2609_34380_b200 import workloads
from tests.helpers import assert_close_to_oracle, split_both, to_np_bytes, to_np_words

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("M,K", [(1, 16), (7, 528), (300, 1040), (64, 4096), (5, 8192), (3, 8208), (4, 11008)])
def test_quantisation_is_bit_exact(M, K):
    """Rows of up to 8192 elements are held in registers between the two passes; longer ones are read twice."""
    x = workloads.activations(M, K, 21 + M, device=DEV)
    if M > 2:
        x[2] = 0                                   # an all-zero token
        x[1] *= 1e-3                               # a token of small values: the scale is per token, the codes stay spread
    q, scale = dps.dps_quantize_activations(x)
    q_ref, s_ref = oracle.quantize_activations(to_np_words(x))
    assert np.array_equal(scale.cpu().numpy(), s_ref)
    assert np.array_equal(to_np_bytes(q), q_ref)
    assert dps.dps_stream_status() == dps.DPS_OK


def test_non_finite_activation_raises_the_status_word():
    x = workloads.activations(4, 64, 5, device=DEV)
    x[1, 3] = float("inf")
    dps.dps_quantize_activations(x)
    assert dps.dps_stream_status() == dps.binding.DPS_ERR_DATA
    assert dps.dps_stream_status() == dps.DPS_OK


@pytest.mark.parametrize("enc_req", [dps.DPS_ENC_AUTO, dps.DPS_ENC_E5M2])
@pytest.mark.parametrize("N,K,M", [(264, 528, 10), (1024, 1040, 300), (136, 4112, 257), (2056, 272, 520)])
def test_linear_against_the_oracle(enc_req, N, K, M):
    """Ragged in N (not a multiple of 128), K (partial last block of 128) and M (partial token tile)."""
    w = workloads.weights(N, K, 31, device=DEV)
    p, r, enc, p_ref, _ = split_both(w, enc_req, DEV)
    x = workloads.activations(M, K, 32, device=DEV)
    q, scale = dps.dps_quantize_activations(x)
    y = dps.dps_linear_fp8act(enc, q, scale, p)
    ref = oracle.linear_fp8act(enc, *oracle.quantize_activations(to_np_words(x)), p_ref, threads=8)   # the oracle's own codes
    assert_close_to_oracle(y, ref, f"fp8act N={N} K={K} M={M} enc={enc}")
    assert torch.equal(y, dps.dps_linear_fp8act(enc, q, scale, p))
    assert dps.dps_stream_status() == dps.DPS_OK


def test_more_tiles_than_sms_on_256_token_tiles():
    """160 tiles of 128 x 256 on 148 persistent CTAs: both accumulators in use, a second tile for some CTAs."""
    N, K, M = 4096, 272, 1280
    w = workloads.weights(N, K, 33, device=DEV)
    p, r, enc, p_ref, _ = split_both(w, dps.DPS_ENC_AUTO, DEV)
    x = workloads.activations(M, K, 34, device=DEV)
    q, scale = dps.dps_quantize_activations(x)
    y = dps.dps_linear_fp8act(enc, q, scale, p)
    ref = oracle.linear_fp8act(enc, *oracle.quantize_activations(to_np_words(x)), p_ref, threads=16)   # the oracle's own codes
    assert_close_to_oracle(y, ref, "fp8act 160 tiles")


def test_llama_o_proj_512_tokens_and_distance_to_fp16_activations():
    N, K = workloads.LLAMA7B["o"]
    w = workloads.weights(N, K, 2002, device=DEV)
    p, r, enc, p_ref, _ = split_both(w, dps.DPS_ENC_AUTO, DEV)
    x = workloads.activations(512, K, 3001, device=DEV)
    q, scale = dps.dps_quantize_activations(x)
    y8 = dps.dps_linear_fp8act(enc, q, scale, p)
    ref = oracle.linear_fp8act(enc, *oracle.quantize_activations(to_np_words(x)), p_ref, threads=16)   # the oracle's own codes
    assert_close_to_oracle(y8, ref, "o-proj fp8act")
    y16 = dps.dps_linear(dps.DPS_MODE_FAST, enc, x, p, None)
    diff = (y8.double() - y16.double()).abs().max().item()
    assert diff <= 5e-2 * y16.double().abs().max().item()      # the price of E4M3 activations, not a parity bound


def test_one_hot_activations_pick_out_fast_mode_weights():
    """One-hot tokens: the single 1.0 quantises to the code of 448 with scale 1/448, so y[m][n] is W_fast[n][k]
    up to one binary32 rounding of the scale and the FP16 rounding of the store."""
    N, K, M = 256, 256, 16
    w = workloads.weights(N, K, 41, device=DEV)
    for enc_req in (dps.DPS_ENC_AUTO, dps.DPS_ENC_E5M2):
        p, r, enc, p_ref, _ = split_both(w, enc_req, DEV)
        x = torch.zeros((M, K), dtype=torch.float16, device=DEV)
        ks = [(7 * m + 3) % K for m in range(M)]
        for m, k in enumerate(ks):
            x[m, k] = 1.0
        q, scale = dps.dps_quantize_activations(x)
        y = dps.dps_linear_fp8act(enc, q, scale, p)
        wf = torch.from_numpy(oracle.fast_words(p_ref, enc).view(np.float16).astype(np.float64))
        want = torch.stack([wf[:, k] for k in ks]).to(torch.float64)
        # scale = 1/448 in binary32 and q = 448: scale * 448 differs from 1 by at most one binary32 rounding
        assert torch.allclose(y.cpu().double(), want, rtol=2 ** -10, atol=0)
