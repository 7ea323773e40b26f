"""GPU parity: rounded nests (persistent byte = nearest FP8 value) through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_34380_b200 as dps
from paper_2609_34380_b200 import workloads
from tests.helpers import assert_close_to_oracle, split_both, to_np_bytes, to_np_words

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
PAIRS = [(dps.DPS_ENC_E4M3_RN, dps.DPS_ENC_E4M3), (dps.DPS_ENC_E5M2_RN, dps.DPS_ENC_E5M2)]


@pytest.mark.parametrize("enc,base", PAIRS)
@pytest.mark.parametrize("rows,cols", [(1, 16), (37, 272), (640, 1040)])
def test_split_and_reconstruct_are_bit_exact(enc, base, rows, cols):
    w = workloads.weights(rows, cols, 90 + rows, device=DEV)
    if rows > 1:
        w[1, :8] = torch.tensor([0.0, -0.0, 6e-8, -6e-8, 1.0, -1.0, 1.5, -1.2421875], dtype=torch.float16, device=DEV)
    p, r, used = dps.dps_split_weights(w, enc)
    assert used == enc
    p_ref, r_ref, _ = oracle.split(to_np_words(w), enc)
    assert np.array_equal(to_np_bytes(p), p_ref) and np.array_equal(to_np_bytes(r), r_ref)
    back = dps.dps_reconstruct(p, r, enc)
    assert torch.equal(back.view(torch.int16), w.view(torch.int16))
    fast = dps.dps_reconstruct(p, None, enc)
    assert np.array_equal(to_np_words(fast), oracle.fast_words(p_ref, enc))
    assert dps.dps_stream_status() == dps.DPS_OK


def test_every_legal_word_round_trips():
    for enc, max_mag in [(dps.DPS_ENC_E5M2_RN, 0x7B7F), (dps.DPS_ENC_E4M3_RN, 0x3F3F)]:
        words = np.arange(65536, dtype=np.uint32).astype(np.uint16)
        words = words[(words & 0x7FFF) <= max_mag]
        words = np.resize(words, ((words.size + 15) // 16) * 16).reshape(-1, 16)
        w = torch.from_numpy(words.view(np.int16).copy()).to(DEV).view(torch.float16)
        p, r, _ = dps.dps_split_weights(w, enc)
        p_ref, r_ref, _ = oracle.split(words, enc)
        assert np.array_equal(to_np_bytes(p), p_ref) and np.array_equal(to_np_bytes(r), r_ref)
        assert torch.equal(dps.dps_reconstruct(p, r, enc).view(torch.int16), w.view(torch.int16))


@pytest.mark.parametrize("enc,bad", [(dps.DPS_ENC_E4M3_RN, 1.9765625), (dps.DPS_ENC_E5M2_RN, 65504.0),
                                     (dps.DPS_ENC_E5M2_RN, float("inf"))])
def test_ineligible_tensor_is_refused_and_planes_stay_untouched(enc, bad):
    w = workloads.weights(8, 64, 3, device=DEV)
    w[5, 7] = bad
    p = torch.full((8, 64), 0xAB, dtype=torch.uint8, device=DEV)
    r = torch.full((8, 64), 0xCD, dtype=torch.uint8, device=DEV)
    with pytest.raises(dps.DpsError) as e:
        dps.dps_split_weights(w, enc, p, r)
    assert e.value.status == dps.binding.DPS_ERR_DATA
    assert bool((p == 0xAB).all()) and bool((r == 0xCD).all())
    assert not oracle.rounded_legal(to_np_words(w), enc)


@pytest.mark.parametrize("enc,base", PAIRS)
@pytest.mark.parametrize("N,K,M", [(264, 528, 3), (1032, 1040, 12), (520, 2064, 32), (392, 272, 300), (8192, 272, 200)])
def test_linear_against_the_oracle_in_both_modes(enc, base, N, K, M):
    """Streaming kernel (3, 12 tokens), tcgen05 decode tiles (32), prefill tiles (300) and K halves on CTA
    pairs (200 tokens x 8192 rows); ragged N and K."""
    w = workloads.weights(N, K, 700 + N, device=DEV)
    p, r, _, pn, rn = split_both(w, enc, DEV)        # reference side: the oracle's own planes
    pb, rb, _ = dps.dps_split_weights(w, base)
    x = workloads.activations(M, K, 800 + M, device=DEV)
    for mode in (dps.DPS_MODE_FAST, dps.DPS_MODE_FULL):
        y = dps.dps_linear(mode, enc, x, p, r if mode else None)
        ref = oracle.linear(mode, enc, to_np_words(x), pn, rn, threads=8)
        assert_close_to_oracle(y, ref, f"rounded enc={enc} N={N} K={K} M={M} mode={mode}")
    # full mode rebuilds the same FP16 weights from either nest: the same bits come out
    y_rn = dps.dps_linear(dps.DPS_MODE_FULL, enc, x, p, r)
    y_tr = dps.dps_linear(dps.DPS_MODE_FULL, base, x, pb, rb)
    assert torch.equal(y_rn, y_tr)
    # fast mode reads a rounded plane exactly as it reads any FP8 plane of the sibling encoding
    assert torch.equal(dps.dps_linear(dps.DPS_MODE_FAST, enc, x, p, None), dps.dps_linear(dps.DPS_MODE_FAST, base, x, p, None))
    assert dps.dps_stream_status() == dps.DPS_OK


def test_fast_mode_error_shrinks_on_llama_o_projection():
    """What the extension is for: the fast-mode output is closer to the full-mode one."""
    N, K = workloads.LLAMA7B["o"]
    w = workloads.weights(N, K, 2002, device=DEV)
    x = workloads.activations(8, K, 3001, device=DEV)
    full = None
    err = {}
    for enc in (dps.DPS_ENC_E4M3, dps.DPS_ENC_E4M3_RN):
        p, r, _ = dps.dps_split_weights(w, enc)
        y_full = dps.dps_linear(dps.DPS_MODE_FULL, enc, x, p, r)
        full = y_full if full is None else full
        assert torch.equal(y_full, full)
        err[enc] = (dps.dps_linear(dps.DPS_MODE_FAST, enc, x, p, None).double() - y_full.double()).abs().mean().item()
    assert err[dps.DPS_ENC_E4M3_RN] < 0.8 * err[dps.DPS_ENC_E4M3]


def test_fp8_activation_fast_mode():
    N, K, M = 264, 528, 40
    w = workloads.weights(N, K, 31, device=DEV)
    x = workloads.activations(M, K, 32, device=DEV)
    q, scale = dps.dps_quantize_activations(x)
    for enc, base in PAIRS:
        p, r, _, p_ref, _ = split_both(w, enc, DEV)
        y = dps.dps_linear_fp8act(enc, q, scale, p)
        ref = oracle.linear_fp8act(enc, *oracle.quantize_activations(to_np_words(x)), p_ref, threads=4)   # the oracle's own codes
        assert_close_to_oracle(y, ref, f"fp8act rounded enc={enc}")
        assert torch.equal(y, dps.dps_linear_fp8act(base, q, scale, p))


def test_grouped_linear_with_rounded_and_truncated_experts():
    """Experts of all four encodings in one call; one expert with a second token tile, one empty."""
    E, N, K, T = 5, 392, 528, 140
    req = [dps.DPS_ENC_E4M3_RN, dps.DPS_ENC_E5M2, dps.DPS_ENC_E5M2_RN, dps.DPS_ENC_E4M3, dps.DPS_ENC_E4M3_RN]
    ps, rs, encs, p_refs, r_refs = [], [], [], [], []
    for e in range(E):
        w = workloads.weights(N, K, 150 + e, device=DEV)
        p, r, enc, p_ref, r_ref = split_both(w, req[e], DEV)
        ps.append(p), rs.append(r), encs.append(enc), p_refs.append(p_ref), r_refs.append(r_ref)
    assert encs == req
    p, r = torch.stack(ps), torch.stack(rs)
    p_ref, r_ref = np.stack(p_refs), np.stack(r_refs)
    x = workloads.activations(T, K, 160, device=DEV)
    tor, eor = workloads.top2_routing(T, E, 170)
    eor[eor == E - 1] = 0                         # the last expert stays empty, expert 0 gets two shares
    tor_d, eor_d = torch.from_numpy(tor).to(DEV), torch.from_numpy(eor).to(DEV)
    for mode in (dps.DPS_MODE_FAST, dps.DPS_MODE_FULL):
        y = dps.dps_moe_linear(mode, encs, x, tor_d, eor_d, p, r if mode else None)
        ref, rc = oracle.moe_linear(mode, encs, to_np_words(x), tor, eor, p_ref, r_ref, threads=8)
        assert rc == oracle.OK
        assert_close_to_oracle(y, ref, f"grouped rounded mode={mode}")
        y_static = torch.empty_like(y)
        dps.dps_moe_linear_static(mode, encs, x, tor_d, eor_d, p, r if mode else None, y_static)
        assert torch.equal(y, y_static)
    # full mode: the same outputs as with every expert stored as its truncated sibling
    base = {dps.DPS_ENC_E4M3_RN: dps.DPS_ENC_E4M3, dps.DPS_ENC_E5M2_RN: dps.DPS_ENC_E5M2}
    ps2, rs2, encs2 = [], [], []
    for e in range(E):
        w = workloads.weights(N, K, 150 + e, device=DEV)
        p2, r2, enc2 = dps.dps_split_weights(w, base.get(req[e], req[e]))
        ps2.append(p2), rs2.append(r2), encs2.append(enc2)
    y_rn = dps.dps_moe_linear(dps.DPS_MODE_FULL, encs, x, tor_d, eor_d, p, r)
    y_tr = dps.dps_moe_linear(dps.DPS_MODE_FULL, encs2, x, tor_d, eor_d, torch.stack(ps2), torch.stack(rs2))
    assert torch.equal(y_rn, y_tr)
    assert dps.dps_stream_status() == dps.DPS_OK


def test_auto_rule_answers_with_a_rounded_nest():
    w = workloads.weights(16, 64, 9, device=DEV)
    p, r, enc = dps.dps_split_weights(w, dps.DPS_ENC_AUTO_RN)
    assert enc == dps.DPS_ENC_E4M3_RN
    p_ref, r_ref, enc_ref = oracle.split(to_np_words(w), oracle.ENC_AUTO_RN)
    assert enc_ref == enc and np.array_equal(to_np_bytes(p), p_ref) and np.array_equal(to_np_bytes(r), r_ref)
    w2 = workloads.with_outlier(w)
    p, r, enc = dps.dps_split_weights(w2, dps.DPS_ENC_AUTO_RN)
    assert enc == dps.DPS_ENC_E5M2_RN
    assert torch.equal(dps.dps_reconstruct(p, r, enc).view(torch.int16), w2.view(torch.int16))
    with pytest.raises(dps.DpsError) as e:
        dps.dps_split_weights(workloads.with_outlier(w, 61440.0), dps.DPS_ENC_AUTO_RN)
    assert e.value.status == dps.binding.DPS_ERR_DATA
    # AUTO_RN names no stored format: the other calls refuse it
    with pytest.raises(dps.DpsError) as e:
        dps.dps_reconstruct(p, r, dps.DPS_ENC_AUTO_RN)
    assert e.value.status == dps.binding.DPS_ERR_ENCODING
