"""GPU parity of the two-row-block tiles (256 weight rows per CTA) and of the persistent kernel on
small, ragged shapes.

The launchers pick those only for large problems; the tuning knobs DPS_DENSE_RB, DPS_GROUPED_RB and
DPS_PERSIST force them.  The library reads its knobs once per process, so each forced run is a child
process: this file executed as a script compares against the oracle and prints one line per case.
"""
import os
import subprocess
import sys

import pytest

REPO = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _cases():
    import numpy as np
    import torch

    import oracle
    import paper_2609_34380_b200 as dps
    from paper_2609_34380_b200 import workloads
    from tests.helpers import assert_close_to_oracle, split_both, to_np_words

    dev = "cuda:0"
    # dense: N not a multiple of 256 (second row block ragged or absent), K with a ragged last block,
    # token counts that leave a partial last token tile
    for (N, K, M) in [(640, 1088, 200), (128, 512, 65), (904, 2064, 300), (392, 272, 577)]:
        for forced_enc in (dps.DPS_ENC_AUTO, dps.DPS_ENC_E5M2):
            w = workloads.weights(N, K, 11 + N, device=dev)
            p, r, enc, p_ref, r_ref = split_both(w, forced_enc, dev)
            x = workloads.activations(M, K, 13 + M, device=dev)
            for mode in (dps.DPS_MODE_FAST, dps.DPS_MODE_FULL):
                y = dps.dps_linear(mode, enc, x, p, r if mode else None)
                ref = oracle.linear(mode, enc, to_np_words(x), p_ref, r_ref, threads=8)
                assert_close_to_oracle(y, ref, f"dense N={N} K={K} M={M} enc={enc} mode={mode}")
                print(f"ok dense N={N} K={K} M={M} enc={enc} mode={mode}")
    # grouped: experts with 0, few and more than one tile of rows; N ragged against 256
    for (E, N, K, T) in [(4, 384, 1040, 90), (3, 136, 528, 150)]:
        ps, rs, encs, p_refs, r_refs = [], [], [], [], []
        for e in range(E):
            w = workloads.weights(N, K, 50 + e, device=dev)
            if e == 1:
                w = workloads.with_outlier(w)
            p, r, enc, p_ref, r_ref = split_both(w, dps.DPS_ENC_AUTO, dev)
            ps.append(p), rs.append(r), encs.append(enc), p_refs.append(p_ref), r_refs.append(r_ref)
        p, r = torch.stack(ps), torch.stack(rs)
        p_ref, r_ref = np.stack(p_refs), np.stack(r_refs)
        x = workloads.activations(T, K, 60, device=dev)
        tor, eor = workloads.top2_routing(T, E, 70)
        eor[eor == E - 1] = 0                     # the last expert stays empty, expert 0 gets two shares
        for mode in (dps.DPS_MODE_FAST, dps.DPS_MODE_FULL):
            y = dps.dps_moe_linear(mode, encs, x, torch.from_numpy(tor).to(dev), torch.from_numpy(eor).to(dev), p,
                                   r if mode else None)
            ref, rc = oracle.moe_linear(mode, encs, to_np_words(x), tor, eor, p_ref, r_ref, threads=8)
            assert rc == oracle.OK
            assert_close_to_oracle(y, ref, f"grouped E={E} N={N} mode={mode}")
            print(f"ok grouped E={E} N={N} K={K} T={T} mode={mode}")
    assert dps.dps_stream_status() == dps.DPS_OK
    print("all row-block cases passed")


@pytest.mark.gpu
@pytest.mark.parametrize("persist", ["0", "2"])      # one CTA per tile / persistent kernel forced
def test_forced_two_row_blocks_in_child_process(persist):
    env = dict(os.environ, DPS_DENSE_RB="2", DPS_GROUPED_RB="2", DPS_PERSIST=persist, PYTHONPATH=REPO)
    out = subprocess.run([sys.executable, os.path.abspath(__file__)], cwd=REPO, env=env, capture_output=True,
                         text=True, timeout=600)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-4000:]
    assert "all row-block cases passed" in out.stdout
    assert out.stdout.count("ok dense") == 16 and out.stdout.count("ok grouped") == 4


@pytest.mark.gpu
@pytest.mark.parametrize("persist", ["0", "2"])
def test_forced_192_token_two_row_block_tiles_in_child_process(persist):
    """Fast mode, 256 rows x 192 tokens per CTA (the launcher picks it from two rounds of such tiles on): here
    forced on shapes with a ragged second row block, a ragged last K block and a short last token tile."""
    env = dict(os.environ, DPS_DENSE_RB="2", DPS_RB2_TN="192", DPS_PERSIST=persist, PYTHONPATH=REPO)
    out = subprocess.run([sys.executable, os.path.abspath(__file__)], cwd=REPO, env=env, capture_output=True,
                         text=True, timeout=600)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-4000:]
    assert "all row-block cases passed" in out.stdout


@pytest.mark.gpu
def test_forced_k_halves_for_every_tile_in_child_process():
    """Few 256-token tiles: two CTAs per tile, each with one half of K (forced; 1 to 8 tiles here)."""
    env = dict(os.environ, DPS_PAIR_ALL="2", DPS_FORCE_TN="256", PYTHONPATH=REPO)
    out = subprocess.run([sys.executable, os.path.abspath(__file__)], cwd=REPO, env=env, capture_output=True,
                         text=True, timeout=600)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-4000:]
    assert "all row-block cases passed" in out.stdout


@pytest.mark.gpu
def test_forced_persistent_kernel_with_default_tiles_in_child_process():
    """256-token tiles (forced: the shapes here are small) walked by the persistent kernel."""
    env = dict(os.environ, DPS_PERSIST="2", DPS_FORCE_TN="256", PYTHONPATH=REPO)
    out = subprocess.run([sys.executable, os.path.abspath(__file__)], cwd=REPO, env=env, capture_output=True,
                         text=True, timeout=600)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-4000:]
    assert "all row-block cases passed" in out.stdout


if __name__ == "__main__":
    _cases()
