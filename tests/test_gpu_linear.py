"""GPU parity: dense linear layers in fast and full mode against the FP64 oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_34380_b200 as dps
from paper_2609_34380_b200 import workloads
from tests.helpers import assert_close_to_oracle, split_both, to_np_bytes, to_np_words, y_as_f64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
MODES = [dps.DPS_MODE_FAST, dps.DPS_MODE_FULL]
ENCS = [dps.DPS_ENC_E4M3, dps.DPS_ENC_E5M2]


def planes(n, k, seed, enc, device=DEV):
    """GPU planes; the oracle's own planes of the same words ride along as p.ref / r.ref."""
    w = workloads.weights(n, k, seed, device=device).to(DEV)
    return (w,) + with_ref(w, enc)


def with_ref(w, enc_req):
    p, r, enc, p.ref, r.ref = split_both(w, enc_req, DEV)
    return p, r, enc


def run_and_check(mode, enc, x, p, r, what):
    y = dps.dps_linear(mode, enc, x, p, r if mode == dps.DPS_MODE_FULL else None)
    ref = oracle.linear(mode, enc, to_np_words(x), p.ref, r.ref, threads=8)   # reference side: oracle-made planes
    assert_close_to_oracle(y, ref, what)
    return y


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("enc", ENCS)
def test_config1(mode, enc):
    """512x512 layer, M=4 tokens, both modes, natural (E4M3) and forced (E5M2) encodings."""
    w, p, r, enc = planes(512, 512, 1001, enc, device="cpu")
    x = workloads.activations(4, 512, 1002).to(DEV)
    run_and_check(mode, enc, x, p, r, f"cfg1 mode={mode} enc={enc}")


@pytest.mark.parametrize("mode", MODES)
def test_config1_outlier_goes_e5m2(mode):
    w = workloads.with_outlier(workloads.weights(512, 512, 1001)).to(DEV)
    p, r, enc = with_ref(w, dps.DPS_ENC_AUTO)
    assert enc == dps.DPS_ENC_E5M2
    x = workloads.activations(4, 512, 1002).to(DEV)
    run_and_check(mode, enc, x, p, r, "cfg1 outlier")


@pytest.mark.parametrize("M", [1, 2, 3, 4, 5, 7, 8, 9, 16, 17, 31, 32, 33, 64, 100, 128, 129, 256, 300])
@pytest.mark.parametrize("mode", MODES)
def test_token_counts(M, mode):
    _, p, r, enc = planes(264, 1040, 11, dps.DPS_ENC_AUTO)
    x = workloads.activations(M, 1040, 12 + M, device=DEV)
    run_and_check(mode, enc, x, p, r, f"M={M}")


@pytest.mark.parametrize("N,K", [(8, 16), (8, 4096), (16, 48), (136, 4112), (1000, 272), (4096, 16),
                                 (520, 11008), (24, 28672), (2056, 8208)])
@pytest.mark.parametrize("M", [1, 4, 24])
@pytest.mark.parametrize("mode", MODES)
def test_ragged_shapes(N, K, M, mode):
    """Shapes that span several tiles and leave ragged tails in N, K and M."""
    for enc_req in ENCS:
        _, p, r, enc = planes(N, K, 100 + N + K, enc_req)
        x = workloads.activations(M, K, 7 + M, device=DEV)
        run_and_check(mode, enc, x, p, r, f"N={N} K={K} M={M} enc={enc}")


@pytest.mark.parametrize("M", [1, 4, 8, 32, 160])
@pytest.mark.parametrize("enc_req", ENCS)
def test_one_hot_activations_are_bit_exact(M, enc_req):
    """x = unit vectors: y must equal single effective weights exactly, which pins the in-kernel
    reconstruction bit for bit (full: the original FP16 word; fast: the truncated word)."""
    N, K = 392, 2064
    w, p, r, enc = planes(N, K, 21, enc_req)
    ks = np.random.default_rng(M).integers(0, K, M)
    ks[0], ks[-1] = 0, K - 1
    x = torch.zeros((M, K), dtype=torch.float16, device=DEV)
    for m, k in enumerate(ks):
        x[m, int(k)] = 1.0
    full = dps.dps_linear(dps.DPS_MODE_FULL, enc, x, p, r)
    fast = dps.dps_linear(dps.DPS_MODE_FAST, enc, x, p, None)
    w_words = to_np_words(w)
    fast_words = oracle.fast_words(p.ref, enc)
    # Equality of the FP16 VALUES: for non-zero values that is equality of the bits; a weight
    # that is -0 sums to +0 (0 + (-0) = +0 in IEEE arithmetic, in the oracle as well).
    for m, k in enumerate(ks):
        assert np.array_equal(to_np_words(full[m]).view(np.float16), w_words[:, k].view(np.float16)), (m, k)
        assert np.array_equal(to_np_words(fast[m]).view(np.float16), fast_words[:, k].view(np.float16)), (m, k)


def test_subnormal_weights_survive():
    """Weights in the FP16 subnormal range must not be flushed."""
    N, K = 64, 256
    words = np.random.default_rng(3).integers(1, 0x400, (N, K)).astype(np.uint16)   # all subnormal, positive
    w = torch.from_numpy(words.view(np.int16)).view(torch.float16).to(DEV)
    x = torch.full((2, K), 1024.0, dtype=torch.float16, device=DEV)
    for enc_req in ENCS:
        p, r, enc = with_ref(w, enc_req)
        for mode in MODES:
            run_and_check(mode, enc, x, p, r, f"subnormal enc={enc} mode={mode}")


@pytest.mark.parametrize("M", [1, 8, 48])
def test_fast_mode_never_reads_residual(M):
    """The residual's memory may hold KV-cache data in fast mode: results must not depend on it."""
    _, p, r, enc = planes(512, 1024, 31, dps.DPS_ENC_AUTO)
    x = workloads.activations(M, 1024, 32, device=DEV)
    clean = dps.dps_linear(dps.DPS_MODE_FAST, enc, x, p, None)
    poisoned = dps.dps_linear(dps.DPS_MODE_FAST, enc, x, p, torch.full_like(r, 0xFF))
    noise = torch.randint(0, 256, r.shape, dtype=torch.uint8, device=DEV)
    noisy = dps.dps_linear(dps.DPS_MODE_FAST, enc, x, p, noise)
    assert torch.equal(clean.view(torch.int16), poisoned.view(torch.int16))
    assert torch.equal(clean.view(torch.int16), noisy.view(torch.int16))


@pytest.mark.parametrize("M", [1, 4, 32, 512])
@pytest.mark.parametrize("mode", MODES)
def test_run_to_run_determinism_and_guard_bands(M, mode):
    """Same inputs, same bits; and nothing is written outside y (canaries on both sides)."""
    N, K = 1024, 2048
    _, p, r, enc = planes(N, K, 41, dps.DPS_ENC_AUTO)
    x = workloads.activations(M, K, 42, device=DEV)
    guard = 4096
    buf = torch.full((M * N + 2 * guard,), -7.0, dtype=torch.float16, device=DEV)
    y = buf[guard:guard + M * N].view(M, N)
    dps.dps_linear(mode, enc, x, p, r, y)
    first = y.clone()
    for _ in range(3):
        dps.dps_linear(mode, enc, x, p, r, y)
        assert torch.equal(first.view(torch.int16), y.view(torch.int16))
    assert bool((buf[:guard] == -7.0).all()) and bool((buf[guard + M * N:] == -7.0).all())


def test_llama7b_decode_shapes_sampled():
    """Config 2 at full size: every Llama-7B-shaped linear, M in {1, 8, 32}, both modes; the
    oracle recomputes whole output rows for the smallest layer and sampled entries elsewhere."""
    for i, (name, (N, K)) in enumerate(workloads.LLAMA7B.items()):
        w = workloads.weights(N, K, 2001 + i, device=DEV)
        p, r, enc, pn, rn = split_both(w, dps.DPS_ENC_AUTO, DEV)
        assert enc == dps.DPS_ENC_E4M3
        del w
        for M in workloads.DECODE_M:
            x = workloads.activations(M, K, 2011 + i, device=DEV)
            xn = to_np_words(x)
            ms, ns = workloads.sample_entries(M, N, 2048, 2999 + M)
            ns[:4] = [0, 1, N - 2, N - 1]
            for mode in MODES:
                y = dps.dps_linear(mode, enc, x, p, r if mode else None)
                if name == "o" and M == 1:
                    ref = oracle.linear(mode, enc, xn, pn, rn, threads=8)
                    assert_close_to_oracle(y, ref, f"{name} M={M} mode={mode}")
                    continue
                ref = oracle.linear_at(mode, enc, xn, pn, rn, ms, ns)
                got = y_as_f64(y)[ms, ns]
                scale = np.max(np.abs(ref))
                assert np.max(np.abs(got - ref)) <= 2e-3 * scale, (name, M, mode)
        # forced E5M2 on the same shape, M = 8
        w = workloads.weights(N, K, 2001 + i, device=DEV)
        p, r, enc, pn, rn = split_both(w, dps.DPS_ENC_E5M2, DEV)
        del w
        x = workloads.activations(8, K, 2011 + i, device=DEV)
        ms, ns = workloads.sample_entries(8, N, 1024, 2998)
        for mode in MODES:
            y = dps.dps_linear(mode, enc, x, p, r if mode else None)
            ref = oracle.linear_at(mode, enc, to_np_words(x), pn, rn, ms, ns)
            assert np.max(np.abs(y_as_f64(y)[ms, ns] - ref)) <= 2e-3 * np.max(np.abs(ref)), (name, "e5m2", mode)
    assert dps.dps_stream_status() == dps.DPS_OK


def test_launch_counter_moves():
    before = dps.dps_launch_count()
    _, p, r, enc = planes(64, 64, 51, dps.DPS_ENC_E5M2)
    x = workloads.activations(1, 64, 52, device=DEV)
    dps.dps_linear(dps.DPS_MODE_FULL, enc, x, p, r)
    assert dps.dps_launch_count() > before


def test_inf_and_nan_weights_follow_the_bit_rule():
    """Inf / NaN weights force E5M2; split and reconstruction stay bit-exact, and the products carry
    the same non-finite pattern as the oracle's (a NaN whose payload sits only in the low mantissa
    byte turns into Inf in fast mode: that is what dropping the residual means)."""
    N, K = 64, 256
    w = workloads.weights(N, K, 61).clone()
    words = to_np_words(w).copy()
    words[3, 7] = 0x7C00      # +inf
    words[5, 9] = 0xFC00      # -inf
    words[8, 1] = 0x7E01      # NaN, payload in both bytes
    words[9, 2] = 0x7C01      # NaN whose payload is in the residual byte only
    w = torch.from_numpy(words.view(np.int16)).view(torch.float16).to(DEV)
    p, r, enc = dps.dps_split_weights(w, dps.DPS_ENC_AUTO)
    assert enc == dps.DPS_ENC_E5M2
    p_ref, r_ref, _ = oracle.split(words, oracle.ENC_E5M2)
    assert np.array_equal(to_np_bytes(p), p_ref) and np.array_equal(to_np_bytes(r), r_ref)
    assert np.array_equal(to_np_words(dps.dps_reconstruct(p, r, enc)), words)
    for M in (1, 8, 40):
        x = workloads.activations(M, K, 62, device=DEV).abs() + 0.5      # no zeros: inf * x stays inf
        for mode in MODES:
            y = y_as_f64(dps.dps_linear(mode, enc, x, p, r if mode else None))
            with np.errstate(invalid="ignore", over="ignore"):
                ref = oracle.linear(mode, enc, to_np_words(x), p_ref, r_ref)
            assert np.array_equal(np.isnan(y), np.isnan(ref)), (M, mode)
            assert np.array_equal(np.isinf(y), np.isinf(ref)), (M, mode)
            assert np.array_equal(np.sign(y[np.isinf(y)]), np.sign(ref[np.isinf(ref)]))
            fin = np.isfinite(ref)
            assert np.max(np.abs(y[fin] - ref[fin])) <= 2e-3 * np.max(np.abs(ref[fin]))
            assert np.isinf(ref[:, 9]).all() if mode == dps.DPS_MODE_FAST else np.isnan(ref[:, 9]).all()


def test_randomised_shapes_modes_and_encodings():
    """Seeded sweep over awkward shapes: every kernel family and dispatch boundary sees ragged
    N (multiples of 8), ragged K (multiples of 16) and token counts on both sides of each threshold."""
    rng = np.random.default_rng(20261125)
    token_pool = [1, 2, 5, 8, 9, 15, 16, 17, 31, 32, 33, 63, 64, 65, 127, 128, 129, 200, 256, 257, 300, 513]
    for case in range(36):
        N = int(rng.integers(1, 400)) * 8
        K = int(rng.integers(1, 380)) * 16
        M = int(token_pool[int(rng.integers(0, len(token_pool)))])
        enc_req = ENCS[int(rng.integers(0, 2))]
        mode = MODES[int(rng.integers(0, 2))]
        _, p, r, enc = planes(N, K, 7000 + case, enc_req)
        x = workloads.activations(M, K, 8000 + case, device=DEV)
        run_and_check(mode, enc, x, p, r, f"random case {case}: M={M} N={N} K={K} mode={mode} enc={enc}")
    assert dps.dps_stream_status() == dps.DPS_OK
