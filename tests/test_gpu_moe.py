"""GPU parity: grouped (MoE) linear layers against the oracle."""
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


def expert_planes(E, N, K, seed, mixed=True):
    """Stacked GPU planes; the oracle's own planes of the same words ride along as p.ref / r.ref, so that
    the reference side of every comparison is built from the FP16 words, not from the GPU's planes."""
    ps, rs, encs, p_refs, r_refs = [], [], [], [], []
    for e in range(E):
        w = workloads.weights(N, K, seed + e, device=DEV)
        if mixed and e % 3 == 1:
            w = workloads.with_outlier(w)
        p, r, enc, p_ref, r_ref = split_both(w, dps.DPS_ENC_AUTO, DEV)
        ps.append(p), rs.append(r), encs.append(enc), p_refs.append(p_ref), r_refs.append(r_ref)
    p, r = torch.stack(ps), torch.stack(rs)
    p.ref, r.ref = np.stack(p_refs), np.stack(r_refs)
    return p, r, encs


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("E,N,K,T", [(4, 264, 528, 10), (8, 520, 1040, 96), (3, 136, 4112, 33)])
def test_top2_routing_small(mode, E, N, K, T):
    p, r, encs = expert_planes(E, N, K, 300)
    x = workloads.activations(T, K, 400, device=DEV)
    tor, eor = workloads.top2_routing(T, E, 500)
    y = dps.dps_moe_linear(mode, encs, x, torch.from_numpy(tor).to(DEV), torch.from_numpy(eor).to(DEV), p,
                           r if mode else None)
    ref, rc = oracle.moe_linear(mode, encs, to_np_words(x), tor, eor, p.ref, r.ref, threads=8)
    assert rc == oracle.OK
    assert_close_to_oracle(y, ref, f"moe E={E}")
    assert dps.dps_stream_status() == dps.DPS_OK


@pytest.mark.parametrize("mode", MODES)
def test_identity_token_map_and_empty_experts(mode):
    """token_of_row = NULL means row a reads x[a]; experts that receive no row are never touched."""
    E, N, K, A = 6, 128, 256, 40
    p, r, encs = expert_planes(E, N, K, 600)
    x = workloads.activations(A, K, 700, device=DEV)
    eor = np.random.default_rng(1).choice([0, 2, 5], A).astype(np.int32)     # experts 1, 3, 4 stay empty
    y = dps.dps_moe_linear(mode, encs, x, None, torch.from_numpy(eor).to(DEV), p, r if mode else None)
    ref, _ = oracle.moe_linear(mode, encs, to_np_words(x), None, eor, p.ref, r.ref, threads=8)
    assert_close_to_oracle(y, ref, "identity map")


def test_all_rows_one_expert_equals_dense():
    E, N, K, A = 3, 256, 512, 70
    p, r, encs = expert_planes(E, N, K, 800, mixed=False)
    x = workloads.activations(A, K, 900, device=DEV)
    eor = torch.full((A,), 1, dtype=torch.int32, device=DEV)
    for mode in MODES:
        y = dps.dps_moe_linear(mode, encs, x, None, eor, p, r if mode else None)
        ref = oracle.linear(mode, encs[1], to_np_words(x), p.ref[1], r.ref[1], threads=8)
        assert_close_to_oracle(y, ref, "one expert")


def test_bad_indices_are_skipped_and_flagged():
    E, N, K, T = 4, 64, 128, 8
    p, r, encs = expert_planes(E, N, K, 1000)
    x = workloads.activations(T, K, 1100, device=DEV)
    tor, eor = workloads.top2_routing(T, E, 1200)
    tor, eor = tor.copy(), eor.copy()
    eor[3] = E
    eor[6] = -1
    tor[9] = T
    y = torch.full((2 * T, N), 5.0, dtype=torch.float16, device=DEV)
    dps.dps_moe_linear(dps.DPS_MODE_FULL, encs, x, torch.from_numpy(tor).to(DEV), torch.from_numpy(eor).to(DEV), p, r, y)
    assert dps.dps_stream_status() == dps.binding.DPS_ERR_DATA
    assert dps.dps_stream_status() == dps.DPS_OK                      # reading clears the word
    ref, rc = oracle.moe_linear(dps.DPS_MODE_FULL, encs, to_np_words(x), tor, eor, p.ref, r.ref,
                                y_init=np.full((2 * T, N), 5.0))
    assert rc == oracle.ERR_DATA
    got = y_as_f64(y)
    for a in (3, 6, 9):
        assert np.all(got[a] == 5.0)                                  # skipped rows are left untouched
    assert_close_to_oracle(y, ref, "bad rows")


def test_fast_mode_ignores_residual_and_is_deterministic():
    E, N, K, T = 4, 128, 256, 24
    p, r, encs = expert_planes(E, N, K, 1300)
    x = workloads.activations(T, K, 1400, device=DEV)
    tor, eor = workloads.top2_routing(T, E, 1500)
    tor_d, eor_d = torch.from_numpy(tor).to(DEV), torch.from_numpy(eor).to(DEV)
    a = dps.dps_moe_linear(dps.DPS_MODE_FAST, encs, x, tor_d, eor_d, p, None)
    b = dps.dps_moe_linear(dps.DPS_MODE_FAST, encs, x, tor_d, eor_d, p, torch.full_like(r, 0xFF))
    c = dps.dps_moe_linear(dps.DPS_MODE_FAST, encs, x, tor_d, eor_d, p, None)
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    assert torch.equal(a.view(torch.int16), c.view(torch.int16))


def test_mixtral_shapes_sampled():
    """Config 4 at full size: 8 experts, hidden 4096, ffn 14336, 256 tokens routed top-2.  Per expert the
    oracle recomputes eight WHOLE output rows -- the first three, the last three (which sit in the expert's
    last token tile) and two from the middle of its row list -- and, beyond those, 2048 seeded entries spread
    over all rows.  The reference planes are the oracle's own split of the FP16 words."""
    E, T = workloads.MIXTRAL_EXPERTS, workloads.MIXTRAL_TOKENS
    tor, eor = workloads.top2_routing(T, E, 4200)
    rng = np.random.default_rng(4999)
    for li, (name, (N, K)) in enumerate(workloads.MIXTRAL_EXPERT.items()):
        p = torch.empty((E, N, K), dtype=torch.uint8, device=DEV)
        r = torch.empty((E, N, K), dtype=torch.uint8, device=DEV)
        encs, p_ref, r_ref = [], [], []
        for e in range(E):
            w = workloads.weights(N, K, 4001 + 10 * li + e, device=DEV)
            _, _, enc, pe, re_ = split_both(w, dps.DPS_ENC_AUTO, DEV, p[e], r[e])
            encs.append(enc), p_ref.append(pe), r_ref.append(re_)
            del w
        if name == "gate_up":
            x = workloads.activations(T, K, 4100, device=DEV)
            tmap = tor
        else:
            x = workloads.activations(2 * T, K, 4300, device=DEV)
            tmap = np.arange(2 * T, dtype=np.int32)
        tor_d = torch.from_numpy(tor).to(DEV) if name == "gate_up" else None
        eor_d = torch.from_numpy(eor).to(DEV)
        xn = to_np_words(x)
        whole = {}
        for e in range(E):
            mine = np.nonzero(eor == e)[0]
            assert len(mine) >= 8
            mid = mine[len(mine) // 2 - 1:len(mine) // 2 + 1]
            whole[e] = np.unique(np.concatenate([mine[:3], mid, mine[-3:]]))
        sa = rng.integers(0, 2 * T, 2048)                   # sampled entries (row a, column n)
        sn = rng.integers(0, N, 2048)
        sn[:4] = [0, 1, N - 2, N - 1]
        for mode in MODES:
            y = dps.dps_moe_linear(mode, encs, x, tor_d, eor_d, p, r if mode else None)
            got = y_as_f64(y)
            for e in range(E):
                rows = whole[e]
                ref = oracle.linear(mode, encs[e], xn[tmap[rows]], p_ref[e], r_ref[e], threads=16)
                scale = np.max(np.abs(ref))
                assert np.max(np.abs(got[rows] - ref)) <= 2e-3 * scale, (name, mode, e)
                sel = np.nonzero(eor[sa] == e)[0]
                ref_s = oracle.linear_at(mode, encs[e], xn, p_ref[e], r_ref[e], tmap[sa[sel]], sn[sel])
                assert np.max(np.abs(got[sa[sel], sn[sel]] - ref_s)) <= 2e-3 * np.max(np.abs(ref_s)), (name, mode, e)
        assert dps.dps_stream_status() == dps.DPS_OK
        del p, r, p_ref, r_ref


@pytest.mark.parametrize("mode", MODES)
def test_persistent_grouped_kernel_with_short_last_round(mode):
    """8 experts x 21 two-row-block tiles (N = 5128: the last tile has 8 rows) = 168 work items for 148
    CTAs: the grouped launch runs on the persistent kernel and shares its last round out as halves of K
    (K = 1040: a partial last K block).  Every output row is checked."""
    E, N, K, T = 8, 5128, 1040, 256
    p, r, encs = expert_planes(E, N, K, 900)
    x = workloads.activations(T, K, 901, device=DEV)
    tor, eor = workloads.top2_routing(T, E, 902)
    args = (mode, encs, x, torch.from_numpy(tor).to(DEV), torch.from_numpy(eor).to(DEV), p, r if mode else None)
    y = dps.dps_moe_linear(*args)
    ref, rc = oracle.moe_linear(mode, encs, to_np_words(x), tor, eor, p.ref, r.ref, threads=16)
    assert rc == oracle.OK
    assert_close_to_oracle(y, ref, "grouped persistent")
    assert torch.equal(y, dps.dps_moe_linear(*args))
    assert dps.dps_stream_status() == dps.DPS_OK
