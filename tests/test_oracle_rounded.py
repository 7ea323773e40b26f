"""Pins for the oracle's rounded nests (persistent byte = nearest FP8 value instead of the truncated one).

The paper describes bit selection only; the rounded nests are an extension, so what pins them is their
definition: the persistent byte is the FP8 value nearest to the weight, ties away from zero; the pair
(P, R) still rebuilds the FP16 word exactly; the legality limits are the largest words whose rounded
byte is still a finite FP8 code.  The FP8 value tables come from an independent library's float8
types, the search for the nearest value is a brute-force one written here.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_34380_b200 import workloads

ALL_WORDS = np.arange(65536, dtype=np.uint32).astype(np.uint16)
CASES = [(oracle.ENC_E5M2_RN, oracle.ENC_E5M2, 0x7B7F), (oracle.ENC_E4M3_RN, oracle.ENC_E4M3, 0x3F3F)]


def legal_words(max_mag):
    return ALL_WORDS[(ALL_WORDS & 0x7FFF) <= max_mag]


def fp8_magnitudes(base):
    """Every finite magnitude a persistent byte can stand for (the fast-mode weight values)."""
    codes = torch.arange(256, dtype=torch.uint8)
    if base == oracle.ENC_E5M2:
        t = codes.view(torch.float8_e5m2).to(torch.float64).numpy()
    else:
        t = codes.view(torch.float8_e4m3fn).to(torch.float64).numpy() * 2.0 ** -8
    return np.unique(np.abs(t[np.isfinite(t)]))


@pytest.mark.parametrize("enc,base,max_mag", CASES)
def test_split_then_reconstruct_is_the_identity_on_every_legal_word(enc, base, max_mag):
    w = legal_words(max_mag)
    assert oracle.rounded_legal(w, enc)
    p, r, used = oracle.split(w, enc)
    assert used == enc
    assert np.array_equal(oracle.reconstruct(p, r, enc), w)
    if base == oracle.ENC_E4M3:
        assert np.all(r < 0x80)                       # the spare residual bit stays clear
        assert not np.any((p & 0x7F) == 0x7F)         # never the NaN code


@pytest.mark.parametrize("enc,base,max_mag", CASES)
def test_persistent_byte_is_the_nearest_fp8_value_ties_away_from_zero(enc, base, max_mag):
    w = legal_words(max_mag)
    p, _, _ = oracle.split(w, enc)
    fast = oracle.fast_words(p, enc).view(np.float16).astype(np.float64)
    orig = w.view(np.float16).astype(np.float64)
    grid = fp8_magnitudes(base)
    a = np.abs(orig)
    # brute force: distance to every grid value, the larger value wins a tie
    want = np.empty_like(a)
    for lo in range(0, a.size, 4096):
        chunk = a[lo:lo + 4096, None]
        d = np.abs(chunk - grid[None, :])
        best = d.min(axis=1, keepdims=True)
        want[lo:lo + 4096] = np.where(d == best, grid[None, :], -1.0).max(axis=1)
    assert np.array_equal(np.abs(fast), want)
    assert np.array_equal(np.signbit(fast), np.signbit(orig))
    # the same bytes read through the truncated sibling's table: a rounded plane IS an FP8 plane
    assert np.array_equal(oracle.fast_words(p, base), oracle.fast_words(p, enc))


def test_agrees_with_a_library_cast_away_from_ties():
    """torch rounds ties to even; everywhere else its E5M2 cast and the rounded nest pick the same byte."""
    w = legal_words(0x7B7F)
    p, r, _ = oracle.split(w, oracle.ENC_E5M2_RN)
    lib = torch.from_numpy(w.view(np.float16).copy()).to(torch.float8_e5m2).view(torch.uint8).numpy()
    tie = (w & 0xFF) == 0x80
    assert np.array_equal(p[~tie], lib[~tie])
    assert tie.sum() == 2 * 0x7B and np.all(p[tie] == ((w[tie] >> 8) + 1).astype(np.uint8))   # ties go up in magnitude


@pytest.mark.parametrize("enc,base,max_mag", CASES)
def test_legality_limits(enc, base, max_mag):
    for sign in (0, 0x8000):
        assert oracle.rounded_legal(np.array([max_mag | sign], np.uint16), enc)
        assert not oracle.rounded_legal(np.array([(max_mag + 1) | sign], np.uint16), enc)
    assert not oracle.rounded_legal(np.array([0x7C00], np.uint16), enc)        # Inf
    assert not oracle.rounded_legal(np.array([0x7E00], np.uint16), enc)        # NaN
    assert not oracle.rounded_legal(np.array([0], np.uint16), base)            # not a rounded encoding
    with pytest.raises(oracle.OracleError):
        oracle.split(np.array([max_mag + 1, 0] * 8, np.uint16), enc)
    # the largest legal word rounds to the largest finite code
    p, r, _ = oracle.split(np.array([max_mag], np.uint16), enc)
    assert p[0] == (0x7B if base == oracle.ENC_E5M2 else 0x7E)


def test_rounding_removes_the_shrinking_bias_of_truncation():
    w = workloads.weights(256, 1024, 77)
    words = workloads.as_words(w)
    orig = w.to(torch.float64).numpy()
    nz = orig != 0
    for enc, base in [(oracle.ENC_E4M3_RN, oracle.ENC_E4M3), (oracle.ENC_E5M2_RN, oracle.ENC_E5M2)]:
        rel = {}
        for e in (enc, base):
            p, _, _ = oracle.split(words, e)
            fast = oracle.fast_words(p, e).view(np.float16).astype(np.float64)
            rel[e] = ((np.abs(fast) - np.abs(orig))[nz] / np.abs(orig)[nz])
        assert rel[base].mean() < -0.02 and rel[base].max() <= 0          # truncation only ever shrinks
        assert abs(rel[enc].mean()) < 0.004                                 # rounding is centred
        assert np.sqrt((rel[enc] ** 2).mean()) < 0.62 * np.sqrt((rel[base] ** 2).mean())


def test_linear_full_mode_is_unchanged_and_fast_mode_uses_the_rounded_weights():
    M, N, K = 3, 20, 64
    w = workloads.weights(N, K, 5)
    x = workloads.activations(M, K, 6)
    words, xw = workloads.as_words(w), workloads.as_words(x)
    for enc, base in [(oracle.ENC_E4M3_RN, oracle.ENC_E4M3), (oracle.ENC_E5M2_RN, oracle.ENC_E5M2)]:
        p, r, _ = oracle.split(words, enc)
        pb, rb, _ = oracle.split(words, base)
        full = oracle.linear(oracle.MODE_FULL, enc, xw, p, r)
        assert np.array_equal(full, oracle.linear(oracle.MODE_FULL, base, xw, pb, rb))
        fast = oracle.linear(oracle.MODE_FAST, enc, xw, p, r)
        wf = oracle.fast_words(p, enc).view(np.float16).astype(np.float64)
        xd = x.to(torch.float64).numpy()
        brute = np.zeros((M, N))
        for m in range(M):
            for n in range(N):
                acc = 0.0
                for k in range(K):
                    acc += xd[m, k] * wf[n, k]
                brute[m, n] = acc
        assert np.array_equal(fast, brute)
        # closer to the full-mode result than the truncated nest's fast mode
        fast_trunc = oracle.linear(oracle.MODE_FAST, base, xw, pb, rb)
        assert np.abs(fast - full).mean() < np.abs(fast_trunc - full).mean()


def test_auto_rule_answers_with_a_rounded_nest():
    w = workloads.weights(8, 64, 9)
    words = workloads.as_words(w)
    _, _, enc = oracle.split(words, oracle.ENC_AUTO_RN)
    assert enc == oracle.ENC_E4M3_RN and oracle.select_encoding(words) == oracle.ENC_E4M3
    _, _, enc = oracle.split(workloads.as_words(workloads.with_outlier(w)), oracle.ENC_AUTO_RN)
    assert enc == oracle.ENC_E5M2_RN
    assert oracle.half_to_double(0x7B80) == 61440.0                       # the first magnitude no rounded nest can hold
    with pytest.raises(oracle.OracleError):
        oracle.split(workloads.as_words(workloads.with_outlier(w, 61440.0)), oracle.ENC_AUTO_RN)
