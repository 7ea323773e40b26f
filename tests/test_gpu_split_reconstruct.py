"""GPU parity: nested split, reconstruction and encoding choice are bit-exact vs the oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_34380_b200 as dps
from paper_2609_34380_b200 import workloads
from tests.helpers import to_np_bytes, to_np_words

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def words_tensor(words: np.ndarray, cols: int) -> torch.Tensor:
    assert words.size % cols == 0
    return torch.from_numpy(words.view(np.int16).reshape(-1, cols).copy()).view(torch.float16).to(DEV)


def check_split(w: torch.Tensor, enc_req: int):
    wn = to_np_words(w)
    p_ref, r_ref, enc_ref = oracle.split(wn, enc_req)
    p, r, enc = dps.dps_split_weights(w, enc_req)
    assert enc == enc_ref
    assert np.array_equal(to_np_bytes(p), p_ref)
    assert np.array_equal(to_np_bytes(r), r_ref)
    back = dps.dps_reconstruct(p, r, enc)
    assert np.array_equal(to_np_words(back), wn)                       # lossless, the paper's invariant
    assert np.array_equal(to_np_words(back), oracle.reconstruct(p_ref, r_ref, enc_ref))
    fast = dps.dps_reconstruct(p, None, enc)
    assert np.array_equal(to_np_words(fast), oracle.fast_words(p_ref, enc_ref))
    return enc


def test_every_fp16_word_e5m2():
    words = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    assert check_split(words_tensor(words, 4096), dps.DPS_ENC_E5M2) == dps.DPS_ENC_E5M2
    assert check_split(words_tensor(words, 4096), dps.DPS_ENC_AUTO) == dps.DPS_ENC_E5M2


def test_every_legal_word_e4m3():
    words = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    words = words[((words & 0x4000) == 0) & (((words >> 7) & 0x7F) != 0x7F)]
    words = words[: words.size // 16 * 16]
    assert check_split(words_tensor(words, 16), dps.DPS_ENC_E4M3) == dps.DPS_ENC_E4M3
    auto = words[np.abs(words.view(np.float16).astype(np.float64)) <= 1.75]
    auto = auto[: auto.size // 16 * 16]
    assert check_split(words_tensor(auto, 16), dps.DPS_ENC_AUTO) == dps.DPS_ENC_E4M3


def test_config1_tensors():
    w = workloads.weights(512, 512, 1001).to(DEV)
    assert check_split(w, dps.DPS_ENC_AUTO) == dps.DPS_ENC_E4M3
    assert check_split(w, dps.DPS_ENC_E5M2) == dps.DPS_ENC_E5M2
    assert check_split(w, dps.DPS_ENC_E4M3) == dps.DPS_ENC_E4M3
    assert check_split(workloads.with_outlier(w), dps.DPS_ENC_AUTO) == dps.DPS_ENC_E5M2


@pytest.mark.parametrize("rows,cols", [(1, 16), (3, 48), (257, 4112), (1000, 1008), (4096, 4096)])
def test_ragged_and_multi_tile_shapes(rows, cols):
    w = workloads.weights(rows, cols, 77 + rows).to(DEV)
    check_split(w, dps.DPS_ENC_AUTO)
    check_split(w, dps.DPS_ENC_E5M2)


@pytest.mark.parametrize("value,auto_enc,e4m3_ok", [(1.75, 1, True), (-1.75, 1, True), (1.751, 2, True),
                                                    (1.8125, 2, True), (1.875, 2, False), (2.0, 2, False),
                                                    (float("inf"), 2, False)])
def test_encoding_thresholds(value, auto_enc, e4m3_ok):
    w = workloads.weights(64, 64, 5).to(DEV)
    w[17, 33] = value
    assert oracle.select_encoding(to_np_words(w)) == auto_enc
    _, _, enc = dps.dps_split_weights(w, dps.DPS_ENC_AUTO)
    assert enc == auto_enc
    assert oracle.e4m3_legal(to_np_words(w)) == e4m3_ok
    if e4m3_ok:
        check_split(w, dps.DPS_ENC_E4M3)
    else:
        p = torch.full((64, 64), 0xAB, dtype=torch.uint8, device=DEV)
        r = torch.full((64, 64), 0xCD, dtype=torch.uint8, device=DEV)
        with pytest.raises(dps.DpsError) as ei:
            dps.dps_split_weights(w, dps.DPS_ENC_E4M3, p, r)
        assert ei.value.status == dps.binding.DPS_ERR_DATA
        torch.cuda.synchronize()
        assert bool((p == 0xAB).all()) and bool((r == 0xCD).all())      # planes untouched


def test_e4m3_reconstruct_ignores_residual_bit7():
    w = workloads.weights(64, 64, 6).to(DEV)
    p, r, enc = dps.dps_split_weights(w, dps.DPS_ENC_E4M3)
    back = dps.dps_reconstruct(p, r | 0x80, enc)
    assert np.array_equal(to_np_words(back), to_np_words(w))


def test_llama_shaped_plane_full_size():
    n, k = workloads.LLAMA7B["down"]
    w = workloads.weights(n, k, 2004, device=DEV)
    p, r, enc = dps.dps_split_weights(w, dps.DPS_ENC_AUTO)
    assert enc == dps.DPS_ENC_E4M3 and p.numel() == n * k and r.numel() == n * k
    wn = to_np_words(w)
    p_ref, r_ref, _ = oracle.split(wn, enc)
    assert np.array_equal(to_np_bytes(p), p_ref) and np.array_equal(to_np_bytes(r), r_ref)
    assert torch.equal(dps.dps_reconstruct(p, r, enc).view(torch.int16), w.view(torch.int16))
    assert dps.dps_stream_status() == dps.DPS_OK
