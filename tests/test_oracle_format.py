"""Pins for the oracle's nested split / reconstruct / fast value / encoding choice.

None of these checks re-types the oracle's own shifts: they use the paper's
losslessness statement (full mode rebuilds the original FP16 values), byte
accounting, hand-derived fixtures, closed-form truncation bounds, and float8
casts done by an independent library (torch) and numpy's float16 decoder.
"""
from pathlib import Path

import numpy as np
import pytest
import torch

import oracle
from oracle import ENC_AUTO, ENC_E4M3, ENC_E5M2

GOLDEN = Path(__file__).parent / "golden" / "nested_split_hand_values.txt"

ALL_WORDS = np.arange(65536, dtype=np.uint32).astype(np.uint16)
E4M3_WORDS = ALL_WORDS[(ALL_WORDS & 0x4000) == 0]                       # exponent MSB zero
E4M3_LEGAL = E4M3_WORDS[((E4M3_WORDS >> 7) & 0x7F) != 0x7F]             # not the all-ones code


def f16(words):
    return np.asarray(words, np.uint16).view(np.float16)


def _golden_rows():
    rows = []
    for line in GOLDEN.read_text().splitlines():
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        rows.append(line.split())
    return rows


# ---- binary16 decoder/encoder against numpy (independent implementation) ----

def test_half_to_double_matches_numpy_on_all_words():
    got = np.array([oracle.half_to_double(int(w)) for w in ALL_WORDS])
    want = f16(ALL_WORDS).astype(np.float64)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], want[~nan])
    assert np.array_equal(np.signbit(got[~nan]), np.signbit(want[~nan]))


def test_double_to_half_round_trip_and_ties():
    finite = ALL_WORDS[np.isfinite(f16(ALL_WORDS))]
    vals = f16(finite).astype(np.float64)
    back = np.array([oracle.double_to_half(v) for v in vals], np.uint16)
    assert np.array_equal(back, finite)
    rng = np.random.default_rng(7)
    xs = np.concatenate([rng.normal(0, 1, 4000), rng.normal(0, 1e-5, 2000), rng.normal(0, 3e4, 2000),
                         [65519.9, 65520.0, -65520.0, 1e9, 2.0 ** -25, 2.0 ** -24 * 1.5, 2.0 ** -24 * 2.5,
                          1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11]])
    with np.errstate(over="ignore"):
        want = xs.astype(np.float16).view(np.uint16)
    got = np.array([oracle.double_to_half(v) for v in xs], np.uint16)
    assert np.array_equal(got, want)


# ---- the paper's invariant: full mode returns the original FP16 bits ----

@pytest.mark.parametrize("enc,words", [(ENC_E5M2, ALL_WORDS), (ENC_E4M3, E4M3_LEGAL)])
def test_round_trip_is_lossless_on_every_word(enc, words):
    p, r, used = oracle.split(words, enc)
    assert used == enc
    assert p.dtype == np.uint8 and r.dtype == np.uint8
    assert p.nbytes == words.size and r.nbytes == words.size      # one byte per parameter per plane
    assert np.array_equal(oracle.reconstruct(p, r, enc), words)


def test_e4m3_residual_bit7_written_zero_and_ignored_on_read():
    p, r, _ = oracle.split(E4M3_LEGAL, ENC_E4M3)
    assert not np.any(r & 0x80)
    assert np.array_equal(oracle.reconstruct(p, r | 0x80, ENC_E4M3), E4M3_LEGAL)


# ---- hand-derived fixtures ----

def test_hand_values():
    for word, value, enc_name, p_hex, r_hex, fast_word, fast_value in _golden_rows():
        w = np.array([int(word, 16)], np.uint16)
        assert float(f16(w)[0]) == float(value) or (np.isinf(float(value)) and np.isinf(f16(w)[0]))
        if enc_name.endswith("!"):
            assert not oracle.e4m3_legal(w)
            with pytest.raises(oracle.OracleError) as ei:
                oracle.split(w, ENC_E4M3)
            assert ei.value.code == oracle.ERR_DATA
            continue
        enc = {"E4M3": ENC_E4M3, "E5M2": ENC_E5M2}[enc_name]
        p, r, _ = oracle.split(w, enc)
        assert int(p[0]) == int(p_hex, 16), (word, enc_name)
        assert int(r[0]) == int(r_hex, 16), (word, enc_name)
        fw = oracle.fast_words(p, enc)
        assert int(fw[0]) == int(fast_word, 16), (word, enc_name)
        fv = float(f16(fw)[0])
        assert fv == float(fast_value) and np.signbit(fv) == np.signbit(float(fast_value))
        assert int(oracle.reconstruct(p, r, enc)[0]) == int(word, 16)


# ---- bit positions pinned by an independent library's float8 casts ----

def test_e5m2_persistent_byte_is_a_float8_e5m2_number():
    p, _, _ = oracle.split(ALL_WORDS, ENC_E5M2)
    fast = f16(oracle.fast_words(p, ENC_E5M2))
    lib = torch.from_numpy(p.copy()).view(torch.float8_e5m2).to(torch.float16).numpy()
    nan = np.isnan(lib)
    assert np.array_equal(np.isnan(fast), nan)
    assert np.array_equal(fast[~nan].view(np.uint16), lib[~nan].view(np.uint16))


def test_e4m3_persistent_byte_is_a_float8_e4m3_number_times_2_pow_minus_8():
    p, _, _ = oracle.split(E4M3_LEGAL, ENC_E4M3)
    fast = f16(oracle.fast_words(p, ENC_E4M3)).astype(np.float64)
    lib = torch.from_numpy(p.copy()).view(torch.float8_e4m3fn).to(torch.float32).numpy().astype(np.float64)
    assert not np.any(np.isnan(lib))
    assert np.array_equal(fast, lib * 2.0 ** -8)
    assert np.array_equal(np.signbit(fast), np.signbit(lib))


# ---- closed-form truncation properties of the fast value ----

@pytest.mark.parametrize("enc,words,kept", [(ENC_E5M2, ALL_WORDS, 2), (ENC_E4M3, E4M3_LEGAL, 3)])
def test_fast_value_is_truncation_toward_zero(enc, words, kept):
    words = words[np.isfinite(f16(words))]
    p, r, _ = oracle.split(words, enc)
    fw = oracle.fast_words(p, enc)
    w = f16(words).astype(np.float64)
    f = f16(fw).astype(np.float64)
    assert np.array_equal(np.signbit(w), np.signbit(f))
    assert np.all(np.abs(f) <= np.abs(w))
    exp_field = (words >> 10) & 0x1F
    quantum = np.ldexp(1.0, np.maximum(exp_field.astype(np.int64), 1) - 15 - kept)  # value of last kept bit
    assert np.all(np.abs(w) - np.abs(f) < quantum)
    # idempotent, and a fast value has an all-zero residual
    p2, r2, _ = oracle.split(fw, enc)
    assert np.array_equal(p2, p) and not np.any(r2)
    # the dropped part is exactly the residual's mantissa bits
    dropped = np.abs(w) - np.abs(f)
    rbits = (r & (0xFF if enc == ENC_E5M2 else 0x7F)).astype(np.float64)
    assert np.array_equal(dropped, rbits * np.ldexp(1.0, np.maximum(exp_field.astype(np.int64), 1) - 25))


# ---- encoding selection ----

def _t(vals):
    return np.array(vals, np.float16)


def test_select_encoding_rule():
    small = (np.random.default_rng(3).normal(0, 0.02, 4096)).astype(np.float16)
    assert oracle.select_encoding(small) == ENC_E4M3
    assert oracle.select_encoding(np.append(small, np.float16(1.75))) == ENC_E4M3
    assert oracle.select_encoding(np.append(small, np.float16(-1.75))) == ENC_E4M3
    assert oracle.select_encoding(np.append(small, np.float16(1.751))) == ENC_E5M2   # next fp16 above 1.75
    assert oracle.select_encoding(np.append(small, np.float16(1.76))) == ENC_E5M2
    assert oracle.select_encoding(np.append(small, np.float16(2.0))) == ENC_E5M2
    assert oracle.select_encoding(np.append(small, np.float16(-3.0))) == ENC_E5M2
    assert oracle.select_encoding(np.append(small, np.float16(np.inf))) == ENC_E5M2
    assert oracle.select_encoding(np.append(small, np.float16(np.nan))) == ENC_E5M2
    assert oracle.select_encoding(_t([0.0, -0.0, 6e-8])) == ENC_E4M3


def test_auto_split_uses_selected_encoding_and_explicit_e4m3_is_checked():
    small = (np.random.default_rng(4).normal(0, 0.02, 1024)).astype(np.float16)
    _, _, enc = oracle.split(small, ENC_AUTO)
    assert enc == ENC_E4M3
    big = np.append(small, np.float16(3.0))
    _, _, enc = oracle.split(big, ENC_AUTO)
    assert enc == ENC_E5M2
    with pytest.raises(oracle.OracleError):
        oracle.split(big, ENC_E4M3)
    # 1.8125 = 0x3F40: above 1.75 so AUTO says E5M2, yet an explicit E4M3 request is legal (p = 0x7E)
    mid = np.append(small, np.float16(1.8125))
    assert oracle.select_encoding(mid) == ENC_E5M2
    p, r, _ = oracle.split(mid, ENC_E4M3)
    assert np.array_equal(oracle.reconstruct(p, r, ENC_E4M3), mid.view(np.uint16))
    # 1.875 = 0x3F80 lands on the all-ones code 0x7F: rejected
    with pytest.raises(oracle.OracleError):
        oracle.split(np.append(small, np.float16(1.875)), ENC_E4M3)


def test_every_legal_e4m3_byte_is_not_the_nan_code():
    p, _, _ = oracle.split(E4M3_LEGAL, ENC_E4M3)
    assert not np.any((p & 0x7F) == 0x7F)
    # and the AUTO range (|w| <= 1.75) is a subset of the legal set
    auto_ok = E4M3_WORDS[np.abs(f16(E4M3_WORDS).astype(np.float64)) <= 1.75]
    assert np.all(((auto_ok >> 7) & 0x7F) != 0x7F)
