"""GPU parity of the dense kernel families that the dispatcher does not pick by itself for a given shape:
the CUDA-core GEMV (split-K over a CTA's threads, warp-shuffle reduction) for any token count, the
register-streaming kernel for 9-16 tokens on large matrices, and the tensor-core kernel for one token.

DPS_FORCE_PATH pins the family; the library reads it once per process, so each forced run is a child
process: this file executed as a script compares against the oracle and prints one line per case.
"""
import os
import subprocess
import sys

import pytest

REPO = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CASES = {
    # family: (token counts, shapes (N, K))
    "gemv": ([1, 2, 3, 4, 7, 12], [(264, 1040), (1000, 272), (24, 4112), (2056, 528)]),
    "stream": ([1, 5, 8, 9, 13, 16], [(264, 1040), (1000, 272), (8200, 4112)]),
    "umma": ([1, 4, 9, 16], [(264, 1040), (1000, 272), (2056, 528)]),
}


def _cases(family):
    import torch

    import oracle
    import paper_2609_34380_b200 as dps
    from paper_2609_34380_b200 import workloads
    from tests.helpers import assert_close_to_oracle, split_both, to_np_words

    dev = "cuda:0"
    tokens, shapes = CASES[family]
    count = 0
    for (N, K) in shapes:
        for enc_req in (dps.DPS_ENC_AUTO, dps.DPS_ENC_E5M2, dps.DPS_ENC_E4M3_RN):
            w = workloads.weights(N, K, 17 + N, device=dev)
            p, r, enc, p_ref, r_ref = split_both(w, enc_req, dev)
            for M in tokens:
                x = workloads.activations(M, K, 19 + M, device=dev)
                for mode in (dps.DPS_MODE_FAST, dps.DPS_MODE_FULL):
                    y = dps.dps_linear(mode, enc, x, p, r if mode else None)
                    ref = oracle.linear(mode, enc, to_np_words(x), p_ref, r_ref, threads=8)
                    assert_close_to_oracle(y, ref, f"{family} N={N} K={K} M={M} enc={enc} mode={mode}")
                    assert torch.equal(y, dps.dps_linear(mode, enc, x, p, r if mode else None))   # run-to-run bits
                    count += 1
    assert dps.dps_stream_status() == dps.DPS_OK
    print(f"all {count} {family} cases passed")


@pytest.mark.gpu
@pytest.mark.parametrize("family", sorted(CASES))
def test_forced_kernel_family_in_child_process(family):
    env = dict(os.environ, DPS_FORCE_PATH=family, DPS_DEBUG="1", PYTHONPATH=REPO)
    out = subprocess.run([sys.executable, os.path.abspath(__file__), family], cwd=REPO, env=env, capture_output=True,
                         text=True, timeout=900)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-4000:]
    tokens, shapes = CASES[family]
    assert f"all {len(tokens) * len(shapes) * 3 * 2} {family} cases passed" in out.stdout


if __name__ == "__main__":
    _cases(sys.argv[1])
