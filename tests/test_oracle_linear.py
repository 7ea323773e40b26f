"""Pins for the oracle's dense and grouped linear layers.

The oracle's product is checked against a library matmul on the UNSPLIT FP16
weights (full mode must reproduce the FP16 model), against a float8 cast of the
persistent plane done by torch (fast mode), against a pure-Python triple loop on
tiny shapes, and against structural facts: one-hot activations pick out single
effective weights, +-1 activations give exactly representable sums, and the two
modes differ by the product with the truncated-away part.
"""
import numpy as np
import pytest
import torch

import oracle
from oracle import ENC_E4M3, ENC_E5M2, MODE_FAST, MODE_FULL
from paper_2609_34380_b200 import workloads


def f16(words):
    return np.asarray(words, np.uint16).view(np.float16)


def _case(n, k, m, seed, enc, std=0.02):
    w = workloads.weights(n, k, seed, std=std)
    x = workloads.activations(m, k, seed + 1)
    p, r, enc = oracle.split(workloads.as_words(w), enc)
    return w, x, p, r, enc


@pytest.mark.parametrize("enc", [ENC_E4M3, ENC_E5M2])
def test_full_mode_equals_library_matmul_on_unsplit_fp16_weights(enc):
    w, x, p, r, enc = _case(96, 160, 5, 11, enc)
    want = torch.matmul(x.double(), w.double().T).numpy()
    got = oracle.linear(MODE_FULL, enc, workloads.as_words(x), p, r)
    assert np.allclose(got, want, rtol=1e-13, atol=1e-15)


def test_fast_mode_equals_library_matmul_on_float8_view_of_persistent_plane():
    w, x, p, r, _ = _case(64, 128, 3, 21, ENC_E5M2, std=0.5)
    w_fast = torch.from_numpy(p.copy()).view(torch.float8_e5m2).to(torch.float64)
    want = torch.matmul(x.double(), w_fast.T).numpy()
    got = oracle.linear(MODE_FAST, ENC_E5M2, workloads.as_words(x), p, None)
    assert np.allclose(got, want, rtol=1e-13, atol=1e-15)

    w, x, p, r, _ = _case(64, 128, 3, 22, ENC_E4M3)
    w_fast = torch.from_numpy(p.copy()).view(torch.float8_e4m3fn).to(torch.float64) * 2.0 ** -8
    want = torch.matmul(x.double(), w_fast.T).numpy()
    got = oracle.linear(MODE_FAST, ENC_E4M3, workloads.as_words(x), p, None)
    assert np.allclose(got, want, rtol=1e-13, atol=1e-15)


@pytest.mark.parametrize("enc", [ENC_E4M3, ENC_E5M2])
@pytest.mark.parametrize("mode", [MODE_FAST, MODE_FULL])
def test_brute_force_tiny(mode, enc):
    M, N, K = 3, 5, 7
    w, x, p, r, enc = _case(N, K, M, 31, enc)
    weff = f16(oracle.reconstruct(p, r if mode == MODE_FULL else np.zeros_like(r), enc))
    xs = x.numpy()
    want = [[sum(float(xs[m, k]) * float(weff[n, k]) for k in range(K)) for n in range(N)] for m in range(M)]
    got = oracle.linear(mode, enc, workloads.as_words(x), p, r)
    assert np.allclose(got, np.array(want), rtol=1e-14, atol=0)


@pytest.mark.parametrize("enc", [ENC_E4M3, ENC_E5M2])
def test_one_hot_activations_return_single_effective_weights(enc):
    N, K = 40, 48
    w, _, p, r, enc = _case(N, K, 1, 41, enc)
    hot = [0, 7, K - 1]
    x = np.zeros((len(hot), K), np.float16)
    for i, k in enumerate(hot):
        x[i, k] = 1.0
    full, full_h = oracle.linear(MODE_FULL, enc, x, p, r, want_half=True)
    fast, fast_h = oracle.linear(MODE_FAST, enc, x, p, None, want_half=True)
    wn = w.numpy()
    for i, k in enumerate(hot):
        assert np.array_equal(full[i], wn[:, k].astype(np.float64))       # the original FP16 value
        assert np.array_equal(full_h[i], wn[:, k].view(np.uint16))
        assert np.array_equal(fast_h[i], oracle.fast_words(p, enc)[:, k])
        assert np.all(np.abs(fast[i]) <= np.abs(full[i]))


def test_plus_minus_one_activations_give_exact_sums():
    N, K = 16, 2048
    rng = np.random.default_rng(5)
    wi = rng.integers(-4, 5, (N, K))                       # small integers: exact in FP16 and E5M2-fast
    w = wi.astype(np.float16)
    x = rng.choice([-1.0, 1.0], (2, K)).astype(np.float16)
    p, r, _ = oracle.split(w, ENC_E5M2)
    got = oracle.linear(MODE_FULL, ENC_E5M2, x, p, r)
    want = x.astype(np.int64) @ wi.T
    assert np.array_equal(got, want.astype(np.float64))
    # integers up to 4 need at most 2 mantissa bits below the leading one: fast mode is exact too
    got_fast = oracle.linear(MODE_FAST, ENC_E5M2, x, p, None)
    assert np.array_equal(got_fast, want.astype(np.float64))


@pytest.mark.parametrize("enc", [ENC_E4M3, ENC_E5M2])
def test_modes_differ_by_the_truncated_part(enc):
    w, x, p, r, enc = _case(32, 96, 4, 51, enc)
    full = oracle.linear(MODE_FULL, enc, workloads.as_words(x), p, r)
    fast = oracle.linear(MODE_FAST, enc, workloads.as_words(x), p, None)
    delta = w.double().numpy() - f16(oracle.fast_words(p, enc)).astype(np.float64)
    want = x.double().numpy() @ delta.T
    assert np.allclose(full - fast, want, rtol=1e-9, atol=1e-15)
    assert np.any(full != fast)


def test_fast_mode_ignores_residual_contents():
    w, x, p, r, enc = _case(24, 64, 2, 61, ENC_E4M3)
    a = oracle.linear(MODE_FAST, enc, workloads.as_words(x), p, None)
    b = oracle.linear(MODE_FAST, enc, workloads.as_words(x), p, np.full_like(r, 0xFF))
    assert np.array_equal(a, b)


def test_threads_do_not_change_results_and_half_output_is_rounding_of_reference():
    w, x, p, r, enc = _case(64, 128, 4, 71, ENC_E4M3)
    y1, h1 = oracle.linear(MODE_FULL, enc, workloads.as_words(x), p, r, threads=1, want_half=True)
    y4, h4 = oracle.linear(MODE_FULL, enc, workloads.as_words(x), p, r, threads=4, want_half=True)
    assert np.array_equal(y1, y4) and np.array_equal(h1, h4)
    assert np.array_equal(h1, y1.astype(np.float16).view(np.uint16))


def test_linear_at_matches_full_product():
    w, x, p, r, enc = _case(48, 80, 6, 81, ENC_E5M2)
    y = oracle.linear(MODE_FULL, enc, workloads.as_words(x), p, r)
    ms, ns = workloads.sample_entries(6, 48, 50, 9)
    got = oracle.linear_at(MODE_FULL, enc, workloads.as_words(x), p, r, ms, ns)
    assert np.array_equal(got, y[ms, ns])


# ---- grouped (MoE) linear reduces to the dense one ----

def _moe_case(E, N, K, T, seed, mixed_enc=True):
    ps, rs, encs = [], [], []
    for e in range(E):
        w = workloads.weights(N, K, seed + e)
        if mixed_enc and e % 2 == 1:
            w = workloads.with_outlier(w)              # pushes this expert to E5M2
        p, r, enc = oracle.split(workloads.as_words(w), oracle.ENC_AUTO)
        ps.append(p), rs.append(r), encs.append(enc)
    x = workloads.activations(T, K, seed + 100)
    tor, eor = workloads.top2_routing(T, E, seed + 200)
    return np.stack(ps), np.stack(rs), np.array(encs, np.int32), x, tor, eor


@pytest.mark.parametrize("mode", [MODE_FAST, MODE_FULL])
def test_moe_equals_per_expert_dense(mode):
    E, N, K, T = 4, 24, 64, 10
    p, r, encs, x, tor, eor = _moe_case(E, N, K, T, 300)
    assert set(encs.tolist()) == {ENC_E4M3, ENC_E5M2}
    y, rc = oracle.moe_linear(mode, encs, workloads.as_words(x), tor, eor, p, r)
    assert rc == oracle.OK
    xw = workloads.as_words(x)
    for e in range(E):
        rows = np.nonzero(eor == e)[0]
        if rows.size == 0:
            continue
        dense = oracle.linear(mode, int(encs[e]), xw[tor[rows]], p[e], r[e])
        assert np.array_equal(y[rows], dense)
    for t in range(T):                                   # top-2: two distinct experts per token
        assert eor[2 * t] != eor[2 * t + 1]


def test_moe_all_rows_to_one_expert_is_dense_and_permutation_equivariant():
    E, N, K, T = 3, 16, 32, 6
    p, r, encs, x, _, _ = _moe_case(E, N, K, T, 400, mixed_enc=False)
    xw = workloads.as_words(x)
    eor = np.full(T, 2, np.int32)
    y, rc = oracle.moe_linear(MODE_FULL, encs, xw, None, eor, p, r)
    assert rc == oracle.OK
    assert np.array_equal(y, oracle.linear(MODE_FULL, int(encs[2]), xw, p[2], r[2]))
    perm = np.random.default_rng(1).permutation(T).astype(np.int32)
    y2, _ = oracle.moe_linear(MODE_FULL, encs, xw, perm, eor, p, r)
    assert np.array_equal(y2, y[perm])


def test_moe_bad_rows_are_skipped_and_reported():
    E, N, K, T = 2, 8, 16, 4
    p, r, encs, x, tor, eor = _moe_case(E, N, K, T, 500, mixed_enc=False)
    eor = eor.copy()
    tor = tor.copy()
    eor[1] = E            # expert out of range
    tor[5] = -1           # token out of range
    init = np.full((2 * T, N), 123.0)
    y, rc = oracle.moe_linear(MODE_FAST, encs, workloads.as_words(x), tor, eor, p, None, y_init=init)
    assert rc == oracle.ERR_DATA
    assert np.all(y[1] == 123.0) and np.all(y[5] == 123.0)
    good = [a for a in range(2 * T) if a not in (1, 5)]
    ref, _ = oracle.moe_linear(MODE_FAST, encs, workloads.as_words(x), workloads.top2_routing(T, E, 700)[0],
                               workloads.top2_routing(T, E, 700)[1], p, None)
    assert np.array_equal(y[good], ref[good])


def test_moe_row_subset():
    E, N, K, T = 4, 8, 32, 8
    p, r, encs, x, tor, eor = _moe_case(E, N, K, T, 600)
    y, _ = oracle.moe_linear(MODE_FULL, encs, workloads.as_words(x), tor, eor, p, r)
    rows = np.array([0, 3, 15])
    ys, _ = oracle.moe_linear(MODE_FULL, encs, workloads.as_words(x), tor, eor, p, r, rows=rows)
    assert np.array_equal(ys[rows], y[rows])
    others = np.setdiff1d(np.arange(2 * T), rows)
    assert not np.any(ys[others])
