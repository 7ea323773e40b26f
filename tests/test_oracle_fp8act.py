"""Pins for the oracle's FP8-activation fast mode (per-token E4M3 quantisation of the activations).

None of these reuses the oracle's own arithmetic: the E4M3 code table and the rounding are pinned to
an independent library's float8 type, the scale rule to its definition, the product to a brute-force
loop, to a library matmul and to the FP16-activation fast mode on inputs that quantise exactly.
"""
import numpy as np
import torch

import oracle
from paper_2609_34380_b200 import workloads


def test_e4m3_code_table_matches_torch_float8():
    codes = torch.arange(256, dtype=torch.uint8)
    ref = codes.view(torch.float8_e4m3fn).to(torch.float64).numpy()
    mine = np.array([oracle.e4m3_to_double(c) for c in range(256)])
    assert np.isnan(mine[0x7F]) and np.isnan(mine[0xFF])
    keep = ~np.isnan(ref)
    assert keep.sum() == 254
    assert np.array_equal(ref[keep], mine[keep])
    assert mine[0x7E] == 448.0 and mine[0x01] == 2.0 ** -9 and mine[0x08] == 2.0 ** -6


def test_rounding_matches_torch_cast_below_saturation():
    rng = np.random.default_rng(0)
    ties = np.array([(oracle.e4m3_to_double(c) + oracle.e4m3_to_double(c + 1)) / 2 for c in range(0x7E)])
    v = np.concatenate([rng.normal(0, 100, 20000), rng.normal(0, 1, 20000), rng.normal(0, 0.01, 20000), ties, -ties,
                        [448.0, 449.0, 463.9, 464.0, 0.0, -0.0, 2.0 ** -9, 2.0 ** -10, 3 * 2.0 ** -10]]).astype(np.float32)
    v = v[np.abs(v) <= 464.0]                   # beyond 464 torch's cast gives NaN, the oracle saturates (next test)
    ref = torch.from_numpy(v).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    mine = np.array([oracle.float_to_e4m3(x) for x in v], np.uint8)
    assert np.array_equal(ref, mine)


def test_saturation_and_special_values():
    for v, code in [(465.0, 0x7E), (1e6, 0x7E), (-465.0, 0xFE), (-1e30, 0xFE), (float("inf"), 0x7E)]:
        assert oracle.float_to_e4m3(v) == code
    assert oracle.float_to_e4m3(float("nan")) == 0x7F
    assert oracle.float_to_e4m3(0.0) == 0x00 and oracle.float_to_e4m3(-0.0) == 0x80


def test_quantize_scale_rule_and_error_bound():
    x = workloads.activations(7, 96, 5)
    x[3] = 0                                            # an all-zero token
    xw = workloads.as_words(x)
    q, scale = oracle.quantize_activations(xw)
    xf = x.to(torch.float32).numpy()
    amax = np.abs(xf).max(axis=1)
    want = np.where(amax > 0, (amax / np.float32(448.0)).astype(np.float32), np.float32(1.0))
    assert np.array_equal(scale, want)
    assert np.all(q[3] == 0)
    deq = np.array([[oracle.e4m3_to_double(c) for c in row] for row in q]) * scale[:, None].astype(np.float64)
    # relative spacing of E4M3 normals is 2^-3: half of it bounds the error of every normal value
    err = np.abs(deq - xf)
    assert np.all(err <= np.maximum(np.abs(xf) * 2.0 ** -4, scale[:, None] * 2.0 ** -10) * 1.0001)
    # the largest element of every non-zero token lands on +-448
    for m in range(7):
        if amax[m] > 0:
            k = int(np.argmax(np.abs(xf[m])))
            assert q[m, k] & 0x7F == 0x7E


def test_linear_fp8act_brute_force_and_library_matmul():
    M, N, K = 3, 5, 16
    w = workloads.weights(N, K, 9)
    p, r, enc = oracle.split(workloads.as_words(w), oracle.ENC_AUTO)
    x = workloads.activations(M, K, 10)
    q, scale = oracle.quantize_activations(workloads.as_words(x))
    y = oracle.linear_fp8act(enc, q, scale, p)
    wf = np.array([[oracle.half_to_double(v) for v in row] for row in oracle.fast_words(p, enc)])
    brute = np.zeros((M, N))
    for m in range(M):
        for n in range(N):
            acc = 0.0
            for k in range(K):
                acc += oracle.e4m3_to_double(q[m, k]) * wf[n, k]
            brute[m, n] = acc * float(scale[m])
    assert np.allclose(y, brute, rtol=1e-15, atol=0)
    deq = torch.from_numpy(q).view(torch.float8_e4m3fn).to(torch.float64) * torch.from_numpy(scale).to(torch.float64)[:, None]
    lib = (deq @ torch.from_numpy(wf).T).numpy()
    assert np.allclose(y, lib, rtol=1e-12, atol=1e-300)


def test_reduces_to_fp16_activation_fast_mode_when_quantisation_is_exact():
    """Activations in {0, +-1, +-2, +-4}: amax = 4, x / scale in {0, +-112, +-224, +-448}, all E4M3 values."""
    M, N, K = 4, 24, 64
    rng = np.random.default_rng(3)
    vals = np.array([0.0, 1.0, -1.0, 2.0, -2.0, 4.0, -4.0])
    x = torch.from_numpy(vals[rng.integers(0, len(vals), (M, K))]).to(torch.float16)
    x[:, 0] = 4.0                                       # every token has amax 4
    w = workloads.weights(N, K, 11)
    for enc_req in (oracle.ENC_AUTO, oracle.ENC_E5M2):
        p, r, enc = oracle.split(workloads.as_words(w), enc_req)
        q, scale = oracle.quantize_activations(workloads.as_words(x))
        y8 = oracle.linear_fp8act(enc, q, scale, p)
        y16 = oracle.linear(oracle.MODE_FAST, enc, workloads.as_words(x), p, r)
        assert np.allclose(y8, y16, rtol=1e-6, atol=1e-12)


def test_close_to_fp16_activation_result_on_gaussian_inputs():
    """Not a parity bound, a sanity bound: quantising N(0,1) activations to E4M3 moves the output by a few per cent."""
    M, N, K = 8, 64, 1024
    w = workloads.weights(N, K, 12)
    p, r, enc = oracle.split(workloads.as_words(w), oracle.ENC_AUTO)
    x = workloads.activations(M, K, 13)
    q, scale = oracle.quantize_activations(workloads.as_words(x))
    y8 = oracle.linear_fp8act(enc, q, scale, p, threads=4)
    y16 = oracle.linear(oracle.MODE_FAST, enc, workloads.as_words(x), p, r, threads=4)
    assert np.max(np.abs(y8 - y16)) <= 5e-2 * np.max(np.abs(y16))
